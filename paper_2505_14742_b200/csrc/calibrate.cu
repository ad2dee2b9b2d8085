// Calibration before fine-tuning (Sec. 3.3, Eq. 6): count, per input channel, the calibration samples in
// which the channel's largest magnitude exceeds thr x the sample's mean magnitude, then pick the channels
// with the largest counts as the fixed outlier set O.
//
// The indicator is evaluated as one exact integer decision.  |x| is taken in units of 2^-16, truncated
// and saturating at 2^32 - 1:  a(x) = min(floor(|x| 2^16), 2^32 - 1); the test is
//     a(max_o) * (M K)  >  thr * sum a(X)
// in 128-bit integers.  a() is monotone, so the column maximum is taken on the raw bf16 magnitudes; the
// sum is a 64-bit integer (integer atomics: order-free, exact).
#include "common.cuh"

namespace quaff {

// a(x) from the 15 magnitude bits of a bf16 (finite input)
__device__ __forceinline__ unsigned long long abs_fix16(uint32_t mag15) {
    const int e = (int)(mag15 >> 7);                       // biased exponent
    if (e == 0) return 0ull;                               // zero and subnormals: far below 2^-16
    const unsigned long long man = 0x80ull | (mag15 & 0x7Fu);   // 1.mmmmmmm as an 8-bit integer, value = man 2^(e-127-7)
    const int sh = e - 127 - 7 + 16;                       // a = man 2^sh
    if (sh >= 25) return 4294967295ull;                    // >= 2^32: saturate
    if (sh <= -8) return 0ull;
    const unsigned long long v = sh >= 0 ? (man << sh) : (man >> (-sh));
    return v > 4294967295ull ? 4294967295ull : v;
}

// The same a(x) from |x| as fp32 bits, in the hot loop: |x| 2^16 is exact in fp32 (a power-of-two scaling of an
// 8-bit mantissa), and the float -> u32 conversion truncates toward zero and saturates at 2^32 - 1.
__device__ __forceinline__ uint32_t abs_fix16_fast(uint32_t abs_f32_bits) {
    return __float2uint_rz(__fmul_rn(__uint_as_float(abs_f32_bits), 65536.0f));
}

// Pass 1: a thread owns 8 consecutive channels (one 128-bit load per row) over every 8th row of a slice: packed
// 15-bit column maxima in registers, the fixed-point sum in a 64-bit register; merged by integer atomics.
//   ws: [K] u32 column maxima (magnitude bits) | u64 sum | u32 ticket.  The last block turns the maxima into
//   indicators and adds them to xi.
__global__ void __launch_bounds__(256) outlier_count_kernel(const uint16_t* __restrict__ X, int64_t ldx, int M, int K, int thr,
                                                            int32_t* __restrict__ xi, unsigned int* __restrict__ colmax,
                                                            unsigned long long* __restrict__ total,
                                                            unsigned int* __restrict__ ticket, int rows_per_block) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ unsigned long long red[8];
    __shared__ int is_last;
    // block = 32 column-threads (8 channels each: 256 channels) x 8 row groups (a warp reads 512 contiguous bytes of a row)
    __shared__ uint32_t smx[8][32][4];
    const int cx = threadIdx.x & 31, ry = threadIdx.x >> 5;
    const int r0 = blockIdx.y * rows_per_block, r1 = min(M, r0 + rows_per_block);
    const int k0 = (blockIdx.x * 32 + cx) * 8;
    unsigned long long sum = 0;
    uint32_t mx[4] = {0, 0, 0, 0};
    if (k0 < K) {
        const bool vec = (k0 + 8 <= K);
        int m = r0 + ry;
        if (vec) {
            for (; m + 24 < r1; m += 32) {           // four independent 128-bit loads in flight
                uint4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) v[u] = __ldg(reinterpret_cast<const uint4*>(X + (int64_t)(m + 8 * u) * ldx + k0));
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t a = w[i] & 0x7FFF7FFFu;
                        mx[i] = __vmaxu2(mx[i], a);
                        sum += (unsigned long long)abs_fix16_fast(a << 16) + abs_fix16_fast(a & 0xFFFF0000u);
                    }
                }
            }
        }
        for (; m < r1; m += 8) {
            const uint16_t* row = X + (int64_t)m * ldx + k0;
            uint32_t w[4] = {0, 0, 0, 0};
            if (vec) {
                const uint4 v = __ldg(reinterpret_cast<const uint4*>(row));
                w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
            } else {
                for (int e = 0; e < 8 && k0 + e < K; ++e) w[e >> 1] |= (uint32_t)row[e] << ((e & 1) * 16);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t a = w[i] & 0x7FFF7FFFu;
                mx[i] = __vmaxu2(mx[i], a);
                sum += (unsigned long long)abs_fix16_fast(a << 16) + abs_fix16_fast(a & 0xFFFF0000u);
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) smx[ry][cx][i] = mx[i];
    __syncthreads();
    if (ry == 0 && k0 < K) {
#pragma unroll
        for (int g = 1; g < 8; ++g)
#pragma unroll
            for (int i = 0; i < 4; ++i) mx[i] = __vmaxu2(mx[i], smx[g][cx][i]);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const uint32_t v = (mx[e >> 1] >> ((e & 1) * 16)) & 0x7FFFu;
            if (k0 + e < K && v) atomicMax(colmax + k0 + e, v);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long s = 0;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) s += red[w];
        if (s) atomicAdd(total, s);
        __threadfence();
        is_last = (atomicAdd(ticket, 1u) == gridDim.x * gridDim.y - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const unsigned long long S = *reinterpret_cast<volatile unsigned long long*>(total);
    const unsigned long long count = (unsigned long long)M * (unsigned long long)K;
    const unsigned long long rhs_lo = (unsigned long long)thr * S, rhs_hi = __umul64hi((unsigned long long)thr, S);
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        const unsigned long long a = abs_fix16(*reinterpret_cast<volatile unsigned int*>(colmax + k));
        const unsigned long long lhs_lo = a * count, lhs_hi = __umul64hi(a, count);
        if (lhs_hi > rhs_hi || (lhs_hi == rhs_hi && lhs_lo > rhs_lo)) xi[k] += 1;
    }
}

// Selection: channel k is taken if fewer than nO channels come before it in the order (xi descending, index
// ascending).  One thread per channel, the counts staged through shared memory.
__global__ void __launch_bounds__(256) outlier_rank_kernel(const int32_t* __restrict__ xi, int K, int nO, unsigned char* __restrict__ taken) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ int tile[1024];
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    const int mine = k < K ? xi[k] : 0;
    int before = 0;
    for (int c0 = 0; c0 < K; c0 += 1024) {
        for (int i = threadIdx.x; i < 1024; i += blockDim.x) tile[i] = c0 + i < K ? xi[c0 + i] : INT32_MIN;
        __syncthreads();
        const int n = min(1024, K - c0);
        for (int i = 0; i < n; ++i) before += (tile[i] > mine) || (tile[i] == mine && c0 + i < k);
        __syncthreads();
    }
    if (k < K) taken[k] = before < nO;
}

// Ordered compaction of the taken channels into O_idx (one block; chunks of 1024 channels with a block scan).
__global__ void __launch_bounds__(1024) outlier_compact_kernel(const unsigned char* __restrict__ taken, int K, int32_t* __restrict__ O_idx) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ int warp_sum[32];
    __shared__ int base;
    if (threadIdx.x == 0) base = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int c0 = 0; c0 < K; c0 += 1024) {
        const int k = c0 + threadIdx.x;
        const int f = (k < K && taken[k]) ? 1 : 0;
        int incl = f;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) warp_sum[warp] = incl;
        __syncthreads();
        int off = base;
        for (int w = 0; w < warp; ++w) off += warp_sum[w];
        if (f) O_idx[off + incl - 1] = k;
        __syncthreads();
        if (threadIdx.x == 1023) base = off + incl;
        __syncthreads();
    }
}

// Hit-rate monitor: ind[k] > 0 marks a real-time outlier channel of the batch; hits = {those inside O, all of them}.
__global__ void __launch_bounds__(1024) outlier_hits_kernel(const int32_t* __restrict__ ind, int K, const int32_t* __restrict__ O_idx,
                                                            int nO, int32_t* __restrict__ hits) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ int acc[2];
    if (threadIdx.x < 2) acc[threadIdx.x] = 0;
    __syncthreads();
    int in_set = 0, all = 0;
    for (int k = threadIdx.x; k < K; k += blockDim.x) all += ind[k] > 0;
    for (int i = threadIdx.x; i < nO; i += blockDim.x) {
        const int o = O_idx[i];
        if ((unsigned)o < (unsigned)K) in_set += ind[o] > 0;      // an index outside [0, K) is ignored
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        all += __shfl_xor_sync(0xffffffffu, all, o);
        in_set += __shfl_xor_sync(0xffffffffu, in_set, o);
    }
    if ((threadIdx.x & 31) == 0) {
        atomicAdd(&acc[0], in_set);
        atomicAdd(&acc[1], all);
    }
    __syncthreads();
    if (threadIdx.x < 2) hits[threadIdx.x] = acc[threadIdx.x];
}

// Eq. 6 indicator of one sample added to xi; ws = QUAFF_WS_CALIBRATE bytes (cleared here).
static quaff_status_t launch_outlier_count(const quaff_bf16* X, int64_t ldx, int M, int K, int thr, int32_t* xi, void* ws, cudaStream_t st) {
    const size_t need = quaff_workspace_bytes(QUAFF_WS_CALIBRATE, M, K, 0, 0, 0);
    if (cudaMemsetAsync(ws, 0, need, st) != cudaSuccess) return QUAFF_ERR_CUDA;
    unsigned int* colmax = reinterpret_cast<unsigned int*>(ws);
    unsigned char* tail = reinterpret_cast<unsigned char*>(ws) + round_up((size_t)K * 4, 256);
    const int bx = ceil_div(K, 256);
    const int by = max(1, min(ceil_div(M, 32), ceil_div(4 * sm_count(), bx)));
    const int rows_per_block = ceil_div(M, by);
    launch_pdl(outlier_count_kernel, dim3(bx, ceil_div(M, rows_per_block)), dim3(256), 0, st, 1, X, ldx, M, K, thr, xi, colmax,
               reinterpret_cast<unsigned long long*>(tail), reinterpret_cast<unsigned int*>(tail + 8), rows_per_block);
    return launch_status();
}

}  // namespace quaff

using namespace quaff;

extern "C" quaff_status_t quaff_outlier_count(const quaff_bf16* X, int64_t ldx, int M, int K, int thr, int32_t* xi,
                                              void* ws, size_t ws_bytes, quaff_stream_t stream) {
    QUAFF_RETURN_IF(!X || !xi || M <= 0 || K <= 0 || ldx < K || thr < 0, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(!aligned16(X) || (ldx % 8), QUAFF_ERR_ALIGNMENT);
    const size_t need = quaff_workspace_bytes(QUAFF_WS_CALIBRATE, M, K, 0, 0, 0);
    QUAFF_RETURN_IF(!ws || !aligned16(ws) || ws_bytes < need, QUAFF_ERR_WORKSPACE_TOO_SMALL);
    return launch_outlier_count(X, ldx, M, K, thr, xi, ws, (cudaStream_t)stream);
}

extern "C" quaff_status_t quaff_outlier_hits(const quaff_bf16* X, int64_t ldx, int M, int K, int thr, const int32_t* O_idx, int nO,
                                             int32_t* hits, void* ws, size_t ws_bytes, quaff_stream_t stream) {
    QUAFF_RETURN_IF(!X || !hits || M <= 0 || K <= 0 || ldx < K || thr < 0 || nO < 0 || nO > K || (nO > 0 && !O_idx), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(!aligned16(X) || (ldx % 8), QUAFF_ERR_ALIGNMENT);
    const size_t need = quaff_workspace_bytes(QUAFF_WS_HITS, M, K, 0, 0, 0);
    QUAFF_RETURN_IF(!ws || !aligned16(ws) || ws_bytes < need, QUAFF_ERR_WORKSPACE_TOO_SMALL);
    cudaStream_t st = (cudaStream_t)stream;
    // workspace: the counting pass's own scratch, then the indicator of this batch (one int32 per channel)
    const size_t off_ind = quaff_workspace_bytes(QUAFF_WS_CALIBRATE, M, K, 0, 0, 0);
    int32_t* ind = reinterpret_cast<int32_t*>(reinterpret_cast<unsigned char*>(ws) + off_ind);
    if (cudaMemsetAsync(ind, 0, (size_t)K * 4, st) != cudaSuccess) return QUAFF_ERR_CUDA;
    quaff_status_t rc = launch_outlier_count(X, ldx, M, K, thr, ind, ws, st);
    if (rc != QUAFF_OK) return rc;
    launch_pdl(outlier_hits_kernel, dim3(1), dim3(1024), 0, st, 1, (const int32_t*)ind, K, O_idx, nO, hits);
    return launch_status();
}

extern "C" quaff_status_t quaff_select_outliers(const int32_t* xi, int K, int nO, int32_t* O_idx, void* ws, size_t ws_bytes,
                                                quaff_stream_t stream) {
    QUAFF_RETURN_IF(!xi || K <= 0 || nO < 0 || nO > K || (nO > 0 && !O_idx), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(!ws || ws_bytes < quaff_workspace_bytes(QUAFF_WS_CALIBRATE, 1, K, 0, 0, 0), QUAFF_ERR_WORKSPACE_TOO_SMALL);
    if (nO == 0) return QUAFF_OK;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned char* taken = reinterpret_cast<unsigned char*>(ws);
    launch_pdl(outlier_rank_kernel, dim3(ceil_div(K, 256)), dim3(256), 0, st, 1, xi, K, nO, taken);
    quaff_status_t rc = launch_status();
    if (rc != QUAFF_OK) return rc;
    launch_pdl(outlier_compact_kernel, dim3(1), dim3(1024), 0, st, 1, (const unsigned char*)taken, K, O_idx);
    return launch_status();
}
