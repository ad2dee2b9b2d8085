// HBM-bound kernels of the Quaff linear layer: momentum scale update (Eq. 7-8), activation
// scaling + per-token INT8 quantization (Eq. 5, Eq. 1), outlier weight-row re-quantization
// (Eq. 5, Eq. 1 per output channel) and the one-time weight preprocessing.
//
// Bit-exactness contract: every value that decides an INT8 code, a step size or a scale factor is
// computed in fp32 with explicit round-to-nearest intrinsics (__fmul_rn, __fdiv_rn, __fsqrt_rn,
// __fadd_rn, __fsub_rn), which the compiler never contracts into FMAs.
#include "common.cuh"

namespace quaff {

std::atomic<unsigned long long> g_launch_count{0};

int sm_count() {
    static std::atomic<int> cached[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    int n = cached[dev].load();
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev].store(n);
    }
    return n;
}

// =====================================================================================
// Activation scaling + per-token quantization (one pass over X)
// =====================================================================================
// A small CTA (64..256 threads) owns one token row at a time and keeps it in registers as packed
// bf16 between the absmax reduction and the quantization, so X is read from HBM exactly once; the
// next row of the CTA is already being loaded while the current one is reduced and quantized, and
// many such CTAs are resident per SM, which is what keeps enough bytes in flight for HBM.
// A thread owns up to J "units" of 16 consecutive channels (two 128-bit loads, one 128-bit store of
// codes).  Which elements of a thread's units are outlier channels is the same for every row: it is
// found once per CTA (binary search in the sorted O) and kept as a 16-bit mask per unit.  The fast
// path treats masked elements as zero; the few outlier elements are handled one by one
// (x / s before both the absmax and the rounding, as Eq. 5 requires) and patched into the codes.
//
// Rounding: adding 1.5 * 2^23 to a float of magnitude < 2^22 rounds it to an integer, ties to even,
// and leaves that integer in the low mantissa bits; the low byte of the bit pattern is the two's
// complement INT8 code.  |x * (127 / amax)| <= 127 (1 + 2^-23) always rounds into [-127, 127].

constexpr float kRoundMagic = 12582912.0f;   // 1.5 * 2^23
#ifndef QUAFF_QA_MAX_THREADS
#define QUAFF_QA_MAX_THREADS 128
#endif
constexpr int kQuantActMaxThreads = QUAFF_QA_MAX_THREADS;   // CTA size the dispatch aims for (tuning constant)

__device__ __forceinline__ uint32_t code_bits(float x, float rinv) {   // low byte = Eq. 1 code of x
    return __float_as_uint(__fadd_rn(__fmul_rn(x, rinv), kRoundMagic));
}

// Largest 15-bit magnitude among the 8 packed bf16 of a 128-bit word, as two packed 16-bit maxima.
// `keep` has 0x7FFF on the halves that count and 0 on outlier elements (they enter scaled, separately).
__device__ __forceinline__ uint32_t absmax8(const uint4& a, const uint4& keep, uint32_t acc) {
    acc = __vmaxu2(acc, a.x & keep.x);
    acc = __vmaxu2(acc, a.y & keep.y);
    acc = __vmaxu2(acc, a.z & keep.z);
    acc = __vmaxu2(acc, a.w & keep.w);
    return acc;
}

// codes of the 8 packed bf16 of a 128-bit word -> two 32-bit words of 4 codes each
__device__ __forceinline__ uint2 codes8(const uint4& a, float rinv) {
    const uint32_t w[4] = {a.x, a.y, a.z, a.w};
    uint32_t c[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        c[2 * i] = code_bits(__uint_as_float(w[i] << 16), rinv);
        c[2 * i + 1] = code_bits(__uint_as_float(w[i] & 0xFFFF0000u), rinv);
    }
    uint2 r;
    r.x = __byte_perm(__byte_perm(c[0], c[1], 0x0040), __byte_perm(c[2], c[3], 0x0040), 0x5410);
    r.y = __byte_perm(__byte_perm(c[4], c[5], 0x0040), __byte_perm(c[6], c[7], 0x0040), 0x5410);
    return r;
}

// TAIL: K is not a multiple of 16 (the last unit of a row is loaded and stored element by element)
template <int J, bool TAIL>
__device__ __forceinline__ void load_row(uint4 (&raw)[J][2], const uint16_t* __restrict__ xrow, int tid, int T, int K) {
#pragma unroll
    for (int j = 0; j < J; ++j) {
        const int k0 = (tid + j * T) << 4;
        if (!TAIL && k0 >= K) {
            raw[j][0] = raw[j][1] = make_uint4(0, 0, 0, 0);
        } else if (!TAIL || k0 + 16 <= K) {
            const uint4* p = reinterpret_cast<const uint4*>(xrow + k0);
            raw[j][0] = __ldg(p);
            raw[j][1] = __ldg(p + 1);
        } else {
            uint32_t w[8] = {0, 0, 0, 0, 0, 0, 0, 0};
            for (int e = 0; e < 16; ++e)
                if (k0 + e < K) w[e >> 1] |= (uint32_t)xrow[k0 + e] << ((e & 1) * 16);
            raw[j][0] = make_uint4(w[0], w[1], w[2], w[3]);
            raw[j][1] = make_uint4(w[4], w[5], w[6], w[7]);
        }
    }
}

#ifndef QUAFF_QA_MIN_BLOCKS
#define QUAFF_QA_MIN_BLOCKS 2
#endif
#ifndef QUAFF_QA_PERSM_J2
#define QUAFF_QA_PERSM_J2 1024
#endif
// CTA size and residency the compiler may assume: rows of up to 4096 columns (J <= 2) run in CTAs of at most 128
// threads, eight of them per SM (64 registers per thread); wider rows keep more of the row per thread.
template <int J> struct QaBounds {
    static constexpr int kThreads = (J <= 6 && QUAFF_QA_MAX_THREADS <= 128) ? 128 : 256;
    static constexpr int kPerSm = J <= 2 ? QUAFF_QA_PERSM_J2 : (J <= 4 ? 640 : (J <= 6 ? 512 : 512));      // threads per SM the registers must allow
    static constexpr int kBlocks = kPerSm / kThreads;
};
template <int J, bool TAIL>
__global__ void __launch_bounds__(QaBounds<J>::kThreads, QaBounds<J>::kBlocks) quant_act_kernel(const uint16_t* __restrict__ X, int64_t ldx, int M, int K,
                                                        const int32_t* __restrict__ O_idx, int nO,
                                                        const float* __restrict__ s_O,
                                                        int8_t* __restrict__ Xq, int64_t ldxq,
                                                        int8_t* __restrict__ xq_O, int64_t ldxo, int nOp,
                                                        float* __restrict__ dx) {
    pdl_launch_dependents();
    pdl_wait();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int tid = threadIdx.x, T = blockDim.x;
    float* red = reinterpret_cast<float*>(smem_raw);            // [2][8]
    uint4* keep_s = reinterpret_cast<uint4*>(smem_raw + 64);    // [J][2][T]: magnitude masks of this thread's units
    int* O_s = reinterpret_cast<int*>(smem_raw + 64 + (size_t)J * 2 * T * 16);   // [nO]
    float* s_s = reinterpret_cast<float*>(O_s) + nO;                               // [nO]
    float* xo_s = s_s + nO;                                                        // [2][nO]: scaled outlier elements of the row

    const int lane = tid & 31, warp = tid >> 5, nwarps = T >> 5;
    const int nunits = (K + 15) >> 4;

    // the CTA's first row is requested before anything else: its latency covers the staging of O below
    uint4 raw[J][2];
    int m = blockIdx.x;
    if (m < M) load_row<J, TAIL>(raw, X + (int64_t)m * ldx, tid, T, K);

    for (int i = tid; i < nO; i += T) {
        O_s[i] = O_idx[i];
        s_s[i] = s_O[i];
    }
    __syncthreads();

    // outlier elements of this thread's units (mask bit e = channel 16 u + e is in O) -> magnitude masks in smem
#pragma unroll
    for (int j = 0; j < J; ++j) {
        const int u = tid + j * T;
        uint32_t mask = 0;
        if (u < nunits && nO > 0) {
            const int lo_key = u << 4;
            int lo = 0, hi = nO;
            while (lo < hi) {  // first index with O >= lo_key
                const int mid = (lo + hi) >> 1;
                if (O_s[mid] < lo_key) lo = mid + 1; else hi = mid;
            }
            for (int t = lo; t < nO && O_s[t] < lo_key + 16; ++t) mask |= 1u << (O_s[t] - lo_key);
        }
        uint32_t kw[8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
            kw[i] = ((mask >> (2 * i)) & 1u ? 0u : 0x00007FFFu) | ((mask >> (2 * i + 1)) & 1u ? 0u : 0x7FFF0000u);
        keep_s[(j * 2 + 0) * T + tid] = make_uint4(kw[0], kw[1], kw[2], kw[3]);
        keep_s[(j * 2 + 1) * T + tid] = make_uint4(kw[4], kw[5], kw[6], kw[7]);
    }

    int parity = 0;
    for (; m < M; m += gridDim.x, parity ^= 1) {
        const uint16_t* xrow = X + (int64_t)m * ldx;
        // the CTA's next row is on its way while this one is processed (measured: a second row in flight, in registers or
        // as L2 prefetches, does not help - the kernel is not bound by the bytes in flight)
        uint4 nxt[J][2];
        const int mn = m + gridDim.x;
        if (mn < M) load_row<J, TAIL>(nxt, X + (int64_t)mn * ldx, tid, T, K);

        uint32_t mag = 0;                               // two packed 15-bit magnitudes (bf16 bits order like the values)
#pragma unroll
        for (int j = 0; j < J; ++j) {
            mag = absmax8(raw[j][0], keep_s[(j * 2 + 0) * T + tid], mag);
            mag = absmax8(raw[j][1], keep_s[(j * 2 + 1) * T + tid], mag);
        }
        float amax = __uint_as_float(max(mag & 0xFFFFu, mag >> 16) << 16);
        // Eq. 5: the outlier channels enter the absmax as x / s.  They are spread over the CTA's threads
        // (thread i takes channels O[i], O[i + T], ...), whoever owns the unit they sit in.
        float* xo = xo_s + parity * nO;
        for (int i = tid; i < nO; i += T) {
            const float xs = __fdiv_rn(bf16_bits_to_f32(__ldg(xrow + O_s[i])), s_s[i]);
            xo[i] = xs;
            amax = fmaxf(amax, fabsf(xs));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        if (nwarps > 1) {
            if (lane == 0) red[parity * 8 + warp] = amax;
            __syncthreads();
            amax = red[parity * 8];
            for (int w = 1; w < nwarps; ++w) amax = fmaxf(amax, red[parity * 8 + w]);
        }
        const float rinv = amax > 0.0f ? __fdiv_rn(127.0f, amax) : 0.0f;
        if (tid == 0) dx[m] = __fdiv_rn(amax, 127.0f);

        int8_t* qrow = Xq + (int64_t)m * ldxq;
#pragma unroll
        for (int j = 0; j < J; ++j) {
            const int k0 = (tid + j * T) << 4;
            if (k0 >= K) continue;
            const uint2 c0 = codes8(raw[j][0], rinv), c1 = codes8(raw[j][1], rinv);
            if (!TAIL || k0 + 16 <= K) {
                *reinterpret_cast<uint4*>(qrow + k0) = make_uint4(c0.x, c0.y, c1.x, c1.y);
            } else {
                const uint32_t c[4] = {c0.x, c0.y, c1.x, c1.y};
                for (int e = 0; e < 16 && k0 + e < K; ++e) qrow[k0 + e] = (int8_t)((c[e >> 2] >> ((e & 3) * 8)) & 0xFFu);
            }
        }
        if (nO > 0) {
            // outlier channels: the code of x / s replaces the one just written by the unit's owner (the
            // barrier orders the two stores); Eq. 9: the outlier operand is a column gather of the codes
            __syncthreads();
            for (int i = tid; i < nO; i += T) {
                const int8_t q = (int8_t)(code_bits(xo[i], rinv) & 0xFFu);
                qrow[O_s[i]] = q;
                xq_O[(int64_t)m * ldxo + i] = q;
            }
        }
        for (int i = nO + tid; i < nOp; i += T) xq_O[(int64_t)m * ldxo + i] = 0;
#pragma unroll
        for (int j = 0; j < J; ++j) {
            raw[j][0] = nxt[j][0];
            raw[j][1] = nxt[j][1];
        }
    }
}

template <int J, bool TAIL>
static quaff_status_t launch_quant_act(int T, const uint16_t* X, int64_t ldx, int M, int K, const int32_t* O_idx, int nO,
                                       const float* s_O, int8_t* Xq, int64_t ldxq, int8_t* xq_O, int64_t ldxo, int nOp,
                                       float* dx, cudaStream_t st) {
    const size_t smem = 64 + (size_t)J * 2 * T * 16 + (size_t)nO * 16;
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(quant_act_kernel<J, TAIL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return QUAFF_ERR_UNSUPPORTED_SHAPE;
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, quant_act_kernel<J, TAIL>, T, smem) != cudaSuccess || per_sm < 1)
        per_sm = 1;
    const int grid = min(M, sm_count() * per_sm);
    launch_pdl(quant_act_kernel<J, TAIL>, dim3(grid), dim3(T), smem, st, 1, X, ldx, M, K, O_idx, nO, s_O, Xq, ldxq, xq_O, ldxo, nOp, dx);
    return launch_status();
}

static quaff_status_t quant_act_dispatch(const uint16_t* X, int64_t ldx, int M, int K, const int32_t* O_idx, int nO,
                                         const float* s_O, int8_t* Xq, int64_t ldxq, int8_t* xq_O, int64_t ldxo,
                                         int nOp, float* dx, cudaStream_t st) {
    const int nunits = (K + 15) / 16;
    if (nunits > 8 * 256) return QUAFF_ERR_UNSUPPORTED_SHAPE;  // K > 32768
    // units per thread: as many as keep the CTA at 128 threads or fewer (more, smaller CTAs per SM), at most 8
    int J = 1;
    while (J < 8 && ceil_div(nunits, J) > kQuantActMaxThreads) ++J;
    if (J == 5) J = 6;
    if (J == 7) J = 8;
    const int T = min(256, ceil_div(ceil_div(nunits, J), 32) * 32);
#define QA(JJ)                                                                                                    \
    return (K % 16) ? launch_quant_act<JJ, true>(T, X, ldx, M, K, O_idx, nO, s_O, Xq, ldxq, xq_O, ldxo, nOp, dx, st) \
                    : launch_quant_act<JJ, false>(T, X, ldx, M, K, O_idx, nO, s_O, Xq, ldxq, xq_O, ldxo, nOp, dx, st)
    switch (J) {
        case 1: QA(1);
        case 2: QA(2);
        case 3: QA(3);
        case 4: QA(4);
        case 6: QA(6);
        default: QA(8);
    }
#undef QA
}

// =====================================================================================
// INT8 grad-input variant: Z = dY * Delta_W[n], per-token quantization (one pass over dY)
// =====================================================================================
// The same row scheme as quant_act_kernel: a small CTA owns one row at a time and keeps it in registers as packed
// bf16 (J units of 16 columns per thread), the CTA's next row is in flight while this one is processed.  The column
// scales are re-read per row through the read-only path (all rows share them: L1 / L2 hits).  z = x * scale is one
// fp32 product with one rounding, evaluated twice with the same operands (absmax pass, rounding pass).
__device__ __forceinline__ void scaled8(const uint4& a, const float4& s0, const float4& s1, float (&z)[8]) {
    z[0] = __fmul_rn(bf16_lo(a.x), s0.x); z[1] = __fmul_rn(bf16_hi(a.x), s0.y);
    z[2] = __fmul_rn(bf16_lo(a.y), s0.z); z[3] = __fmul_rn(bf16_hi(a.y), s0.w);
    z[4] = __fmul_rn(bf16_lo(a.z), s1.x); z[5] = __fmul_rn(bf16_hi(a.z), s1.y);
    z[6] = __fmul_rn(bf16_lo(a.w), s1.z); z[7] = __fmul_rn(bf16_hi(a.w), s1.w);
}
template <int J>
__global__ void __launch_bounds__(256, 2) quant_grad_kernel(const uint16_t* __restrict__ dY, int64_t lddy, int M, int N,
                                                            const float* __restrict__ colscale, int8_t* __restrict__ Zq,
                                                            int64_t ldz, float* __restrict__ dz) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ float red[2][8];
    const int tid = threadIdx.x, T = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, nwarps = T >> 5;
    // this thread's column scales are the same for every row: with up to two units per thread they are read once and kept
    // in registers (16 per unit); with more units they are re-read per row (L1 / L2 hits), the registers go to the products
    constexpr bool kCacheScales = J <= 2;
    float sc[kCacheScales ? J : 1][16];
    auto load_scales = [&](int j, float (&dst)[16]) {
        const int k0 = (tid + j * T) << 4;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float4 v = k0 < N ? __ldg(reinterpret_cast<const float4*>(colscale + k0) + q) : make_float4(0.f, 0.f, 0.f, 0.f);
            dst[4 * q] = v.x; dst[4 * q + 1] = v.y; dst[4 * q + 2] = v.z; dst[4 * q + 3] = v.w;
        }
    };
    if (kCacheScales) {
#pragma unroll
        for (int j = 0; j < J; ++j) load_scales(j, sc[kCacheScales ? j : 0]);
    }
    uint4 raw[J][2];
    int m = blockIdx.x;
    if (m < M) load_row<J, false>(raw, dY + (int64_t)m * lddy, tid, T, N);
    int parity = 0;
    for (; m < M; m += gridDim.x, parity ^= 1) {
        uint4 nxt[J][2];
        const int mn = m + gridDim.x;
        if (mn < M) load_row<J, false>(nxt, dY + (int64_t)mn * lddy, tid, T, N);
        // z = x * scale (one fp32 product), kept for the rounding pass; absmax over the row
        float z[J][16];
        float amax = 0.0f;
#pragma unroll
        for (int j = 0; j < J; ++j) {
            float tmp[16];
            if (!kCacheScales) load_scales(j, tmp);
            const float (&scj)[16] = kCacheScales ? sc[kCacheScales ? j : 0] : tmp;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const uint32_t w[4] = {raw[j][h].x, raw[j][h].y, raw[j][h].z, raw[j][h].w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    z[j][8 * h + 2 * i] = __fmul_rn(bf16_lo(w[i]), scj[8 * h + 2 * i]);
                    z[j][8 * h + 2 * i + 1] = __fmul_rn(bf16_hi(w[i]), scj[8 * h + 2 * i + 1]);
                    amax = fmaxf(amax, fmaxf(fabsf(z[j][8 * h + 2 * i]), fabsf(z[j][8 * h + 2 * i + 1])));
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        if (nwarps > 1) {
            if (lane == 0) red[parity][warp] = amax;
            __syncthreads();
            amax = red[parity][0];
            for (int w = 1; w < nwarps; ++w) amax = fmaxf(amax, red[parity][w]);
        }
        const float rinv = amax > 0.0f ? __fdiv_rn(127.0f, amax) : 0.0f;
        if (tid == 0) dz[m] = __fdiv_rn(amax, 127.0f);
        int8_t* qrow = Zq + (int64_t)m * ldz;
#pragma unroll
        for (int j = 0; j < J; ++j) {
            const int k0 = (tid + j * T) << 4;
            if (k0 >= N) continue;
            uint32_t out[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t c0 = code_bits(z[j][4 * q], rinv), c1 = code_bits(z[j][4 * q + 1], rinv);
                const uint32_t c2 = code_bits(z[j][4 * q + 2], rinv), c3 = code_bits(z[j][4 * q + 3], rinv);
                out[q] = __byte_perm(__byte_perm(c0, c1, 0x0040), __byte_perm(c2, c3, 0x0040), 0x5410);
            }
            *reinterpret_cast<uint4*>(qrow + k0) = make_uint4(out[0], out[1], out[2], out[3]);
        }
#pragma unroll
        for (int j = 0; j < J; ++j) {
            raw[j][0] = nxt[j][0];
            raw[j][1] = nxt[j][1];
        }
    }
}

template <int J>
static quaff_status_t launch_quant_grad(int T, const uint16_t* dY, int64_t lddy, int M, int N, const float* colscale, int8_t* Zq,
                                        int64_t ldz, float* dz, cudaStream_t st) {
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, quant_grad_kernel<J>, T, 0) != cudaSuccess || per_sm < 1) per_sm = 1;
    const int grid = min(M, sm_count() * per_sm);
    launch_pdl(quant_grad_kernel<J>, dim3(grid), dim3(T), 0, st, 1, dY, lddy, M, N, colscale, Zq, ldz, dz);
    return launch_status();
}

quaff_status_t quant_grad_dispatch(const uint16_t* dY, int64_t lddy, int M, int N, const float* colscale, int8_t* Zq, int64_t ldz,
                                   float* dz, cudaStream_t st) {
    const int nunits = N / 16;
    if ((N % 16) || nunits > 4 * 256) return QUAFF_ERR_UNSUPPORTED_SHAPE;
    // units of 16 columns per thread: as few as keep the CTA at 256 threads or fewer (1..4); up to 4096 columns two units
    // per thread in CTAs of 128 threads or fewer
    int J = 1;
    while (J < 4 && ceil_div(nunits, J) > 256) ++J;
    if (J == 1 && nunits > kQuantActMaxThreads) J = 2;
    const int T = min(256, ceil_div(ceil_div(nunits, J), 32) * 32);
    switch (J) {
        case 1: return launch_quant_grad<1>(T, dY, lddy, M, N, colscale, Zq, ldz, dz, st);
        case 2: return launch_quant_grad<2>(T, dY, lddy, M, N, colscale, Zq, ldz, dz, st);
        case 3: return launch_quant_grad<3>(T, dY, lddy, M, N, colscale, Zq, ldz, dz, st);
        default: return launch_quant_grad<4>(T, dY, lddy, M, N, colscale, Zq, ldz, dz, st);
    }
}

// =====================================================================================
// Momentum scale update (Eq. 8 then Eq. 7), only over the channels of O
// =====================================================================================
// Column maxima of |X| over the nO outlier columns: each block scans a slice of rows (lane =
// channel, warp = row), reduces in shared memory and merges with an integer atomicMax on the
// fp32 bit pattern (non-negative floats order like integers, so the result is exact and
// order-free).  The last block to finish derives beta and updates s.
// colmax_in != null: the maxima are given (one block; nothing is scanned).  apply = 0: the maxima are only
// written to colmax_opt (Eq. 8 and Eq. 7 are left to a later call).
__global__ void __launch_bounds__(256) momentum_kernel(const uint16_t* __restrict__ X, int64_t ldx, int M,
                                                       const int32_t* __restrict__ O_idx, int nO,
                                                       const float* __restrict__ wmax_O, float gamma,
                                                       float* __restrict__ s_O, float* __restrict__ colmax_opt,
                                                       float* __restrict__ beta_opt, unsigned int* __restrict__ ws,
                                                       const float* __restrict__ colmax_in, int apply) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ unsigned int red[8][32];
    __shared__ int is_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (!colmax_in) {
        const int rows_per_block = (M + gridDim.x - 1) / gridDim.x;
        const int r0 = blockIdx.x * rows_per_block;
        const int r1 = min(M, r0 + rows_per_block);

        for (int c0 = 0; c0 < nO; c0 += 32) {
            const int i = c0 + lane;
            unsigned int best = 0;
            if (i < nO) {
                const uint16_t* xc = X + O_idx[i];
                int m = r0 + warp;
                for (; m + 24 < r1; m += 32) {     // four independent gathers in flight per thread
                    const unsigned int a = __ldg(xc + (int64_t)m * ldx), b = __ldg(xc + (int64_t)(m + 8) * ldx);
                    const unsigned int c = __ldg(xc + (int64_t)(m + 16) * ldx), d = __ldg(xc + (int64_t)(m + 24) * ldx);
                    best = max(best, max(max(a & 0x7FFFu, b & 0x7FFFu), max(c & 0x7FFFu, d & 0x7FFFu)));
                }
                for (; m < r1; m += 8) best = max(best, (unsigned int)__ldg(xc + (int64_t)m * ldx) & 0x7FFFu);
                best <<= 16;                       // |x| as fp32 bits
            }
            red[warp][lane] = best;
            __syncthreads();
            if (warp == 0) {
#pragma unroll
                for (int w = 1; w < 8; ++w) best = max(best, red[w][lane]);
                if (i < nO && best) atomicMax(&ws[i], best);
            }
            __syncthreads();
        }
        __threadfence();
        if (tid == 0) is_last = (atomicAdd(&ws[nO], 1u) == gridDim.x - 1);
        __syncthreads();
        if (!is_last) return;
        __threadfence();
    }
    const float one_minus_gamma = __fsub_rn(1.0f, gamma);
    for (int i = tid; i < nO; i += blockDim.x) {
        const float cmax = colmax_in ? colmax_in[i] : __uint_as_float(*reinterpret_cast<volatile unsigned int*>(&ws[i]));
        if (colmax_opt) colmax_opt[i] = cmax;
        if (!apply) continue;
        const float wmax = wmax_O[i];
        float beta = 1.0f;
        if (wmax > 0.0f) beta = fmaxf(1.0f, __fsqrt_rn(__fdiv_rn(cmax, wmax)));   // Eq. 8
        s_O[i] = __fadd_rn(__fmul_rn(gamma, s_O[i]), __fmul_rn(one_minus_gamma, beta));  // Eq. 7
        if (beta_opt) beta_opt[i] = beta;
    }
}

// =====================================================================================
// Outlier weight rows: what = (s_O - 1) W_O, per-output-channel quantization
// =====================================================================================
// A CTA of 8 warps owns 32 output channels: warp w takes the outlier rows w, w + 8, ... (a warp reads 32
// consecutive channels of one row of W_O: coalesced), the per-channel maxima meet in shared memory, and
// the codes go through a shared tile so that each row of wq_O leaves in 128-bit pieces.  The second
// read of W_O comes from L1/L2.
constexpr int kRqCols = 32, kRqRows = 128, kRqPitch = kRqRows + 16;
__global__ void __launch_bounds__(256) requant_rows_kernel(const uint16_t* __restrict__ W_O, int64_t ldwo, int nO, int N,
                                                           const float* __restrict__ s_O, int8_t* __restrict__ wq_O,
                                                           int64_t ldwq, int nOp, float* __restrict__ dw_O) {
    pdl_launch_dependents();
    pdl_wait();
    extern __shared__ __align__(16) unsigned char rq_smem[];
    float* sm1_s = reinterpret_cast<float*>(rq_smem);                 // [nO]: s - 1
    float* red = sm1_s + ((nO + 3) & ~3);                             // [8][32]
    unsigned char* tile = reinterpret_cast<unsigned char*>(red + 8 * kRqCols);   // [32][kRqPitch] codes
    const int tid = threadIdx.x, cx = tid & 31, ry = tid >> 5;
    const int n = blockIdx.x * kRqCols + cx;
    const bool live = n < N;
    for (int i = tid; i < nO; i += 256) sm1_s[i] = __fsub_rn(__ldg(s_O + i), 1.0f);
    __syncthreads();
    float amax = 0.0f;
    if (live) {
#pragma unroll 4
        for (int i = ry; i < nO; i += 8)
            amax = fmaxf(amax, fabsf(__fmul_rn(sm1_s[i], bf16_bits_to_f32(__ldg(W_O + (int64_t)i * ldwo + n)))));
    }
    red[ry * kRqCols + cx] = amax;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < 8; ++w) amax = fmaxf(amax, red[w * kRqCols + cx]);
    if (live && ry == 0) dw_O[n] = __fdiv_rn(amax, 127.0f);
    const float rinv = amax > 0.0f ? __fdiv_rn(127.0f, amax) : 0.0f;
    for (int c0 = 0; c0 < nOp; c0 += kRqRows) {
        const int cl = min(kRqRows, nOp - c0);                        // a multiple of 16
        if (live) {
#pragma unroll 4
            for (int i = c0 + ry; i < c0 + cl; i += 8) {
                int q = 0;
                if (i < nO) q = quant_code(__fmul_rn(sm1_s[i], bf16_bits_to_f32(__ldg(W_O + (int64_t)i * ldwo + n))), rinv);
                tile[cx * kRqPitch + (i - c0)] = (unsigned char)(q & 0xFF);
            }
        }
        __syncthreads();
        const int cpr = cl >> 4;                                      // 128-bit pieces per channel row
        for (int idx = tid; idx < kRqCols * cpr; idx += 256) {
            const int col = idx / cpr, ch = idx - col * cpr;
            const int nn = blockIdx.x * kRqCols + col;
            if (nn < N)
                *reinterpret_cast<uint4*>(wq_O + (int64_t)nn * ldwq + c0 + 16 * ch) =
                    *reinterpret_cast<const uint4*>(tile + col * kRqPitch + 16 * ch);
        }
        __syncthreads();
    }
}

// =====================================================================================
// Weight preprocessing helpers: gather the outlier rows W_O and their maxima
// =====================================================================================
__global__ void __launch_bounds__(256) gather_outlier_rows_kernel(const uint16_t* __restrict__ Wt, int64_t ldw, int N,
                                                                 const int32_t* __restrict__ O_idx,
                                                                 uint16_t* __restrict__ W_O, int64_t ldwo,
                                                                 float* __restrict__ wmax_O) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ unsigned int red[8];
    const int i = blockIdx.x;
    const int col = O_idx[i];
    unsigned int best = 0;
    for (int n = threadIdx.x; n < N; n += blockDim.x) {
        const uint16_t w = Wt[(int64_t)n * ldw + col];
        W_O[(int64_t)i * ldwo + n] = w;
        best = max(best, ((unsigned int)w & 0x7FFFu) << 16);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w) best = max(best, red[w]);
        wmax_O[i] = __uint_as_float(best);
    }
}

// Scratch of quaff_momentum_update_static: column-maximum bit patterns [0, nO) and the block
// ticket counter at [nO].  Lives in every device that loads the library until the process exits.
constexpr int kStaticMaxNO = 4096;
static __device__ __align__(256) unsigned int g_momentum_scratch[kStaticMaxNO + 1];

// The outlier set of every entry point: 0 <= nO <= K, at most kStaticMaxNO channels (the row kernels stage O and
// s_O in shared memory; the paper's largest budget, 10 % of an 11008-wide layer, is 1100).
static quaff_status_t check_outlier_args(const int32_t* O_idx, int nO, int K) {
    if (nO < 0 || nO > K || (nO > 0 && O_idx == nullptr)) return QUAFF_ERR_INVALID_ARG;
    if (nO > kStaticMaxNO) return QUAFF_ERR_UNSUPPORTED_SHAPE;
    return QUAFF_OK;
}
#define QUAFF_CHECK_OUTLIERS(O_idx, nO, K)                              \
    do {                                                                \
        const quaff_status_t rc_ = check_outlier_args(O_idx, nO, K);    \
        if (rc_ != QUAFF_OK) return rc_;                                \
    } while (0)

static int momentum_grid(int M) { return max(1, min(ceil_div(M, 16), sm_count() * 2)); }

}  // namespace quaff

using namespace quaff;

extern "C" quaff_status_t quaff_quant_act(const quaff_bf16* X, int64_t ldx, int M, int K, const int32_t* O_idx, int nO,
                                          const float* s_O, int8_t* Xq, int64_t ldxq, int8_t* xq_O, int64_t ldxo,
                                          int nOp, float* dx, quaff_stream_t stream) {
    QUAFF_RETURN_IF(!X || !Xq || !dx || M < 0 || K <= 0, QUAFF_ERR_INVALID_ARG);
    QUAFF_CHECK_OUTLIERS(O_idx, nO, K);
    QUAFF_RETURN_IF(nO > 0 && !s_O, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(nOp < nO || (nOp > 0 && !xq_O) || ldx < K || ldxq < K || (nOp > 0 && ldxo < nOp), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(!aligned16(X) || !aligned16(Xq) || (ldx % 8) || (ldxq % 16), QUAFF_ERR_ALIGNMENT);
    if (M == 0) return QUAFF_OK;
    return quant_act_dispatch(X, ldx, M, K, O_idx, nO, s_O, Xq, ldxq, xq_O, ldxo, nOp, dx, (cudaStream_t)stream);
}

extern "C" quaff_status_t quaff_momentum_update(const quaff_bf16* X, int64_t ldx, int M, int K, const int32_t* O_idx,
                                                int nO, const float* wmax_O, float gamma, float* s_O,
                                                float* colmax_O_opt, float* beta_O_opt, void* ws, size_t ws_bytes,
                                                quaff_stream_t stream) {
    QUAFF_RETURN_IF(!X || M < 0 || K <= 0 || ldx < K, QUAFF_ERR_INVALID_ARG);
    QUAFF_CHECK_OUTLIERS(O_idx, nO, K);
    QUAFF_RETURN_IF(!(gamma >= 0.0f && gamma <= 1.0f), QUAFF_ERR_INVALID_ARG);
    if (nO == 0) return QUAFF_OK;
    QUAFF_RETURN_IF(!wmax_O || !s_O, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(!ws || ws_bytes < quaff_workspace_bytes(QUAFF_WS_MOMENTUM, M, K, 0, nO, 0), QUAFF_ERR_WORKSPACE_TOO_SMALL);
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(ws, 0, (size_t)(nO + 1) * 4, st) != cudaSuccess) return QUAFF_ERR_CUDA;
    launch_pdl(momentum_kernel, dim3(momentum_grid(M)), dim3(256), 0, st, 1, X, ldx, M, O_idx, nO, wmax_O, gamma, s_O, colmax_O_opt,
               beta_O_opt, reinterpret_cast<unsigned int*>(ws), (const float*)nullptr, 1);
    return launch_status();
}

extern "C" quaff_status_t quaff_outlier_colmax(const quaff_bf16* X, int64_t ldx, int M, int K, const int32_t* O_idx, int nO,
                                               float* colmax_O, void* ws, size_t ws_bytes, quaff_stream_t stream) {
    QUAFF_RETURN_IF(!X || M < 0 || K <= 0 || ldx < K, QUAFF_ERR_INVALID_ARG);
    QUAFF_CHECK_OUTLIERS(O_idx, nO, K);
    if (nO == 0) return QUAFF_OK;
    QUAFF_RETURN_IF(!colmax_O, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(!ws || ws_bytes < quaff_workspace_bytes(QUAFF_WS_MOMENTUM, M, K, 0, nO, 0), QUAFF_ERR_WORKSPACE_TOO_SMALL);
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(ws, 0, (size_t)(nO + 1) * 4, st) != cudaSuccess) return QUAFF_ERR_CUDA;
    launch_pdl(momentum_kernel, dim3(momentum_grid(M)), dim3(256), 0, st, 1, X, ldx, M, O_idx, nO, (const float*)nullptr, 0.0f,
               (float*)nullptr, colmax_O, (float*)nullptr, reinterpret_cast<unsigned int*>(ws), (const float*)nullptr, 0);
    return launch_status();
}

extern "C" quaff_status_t quaff_momentum_apply(const float* colmax_O, const float* wmax_O, int nO, float gamma, float* s_O,
                                               float* beta_O_opt, quaff_stream_t stream) {
    QUAFF_RETURN_IF(nO < 0, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(!(gamma >= 0.0f && gamma <= 1.0f), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(nO > kStaticMaxNO, QUAFF_ERR_UNSUPPORTED_SHAPE);
    if (nO == 0) return QUAFF_OK;
    QUAFF_RETURN_IF(!colmax_O || !wmax_O || !s_O, QUAFF_ERR_INVALID_ARG);
    launch_pdl(momentum_kernel, dim3(1), dim3(256), 0, (cudaStream_t)stream, 1, (const uint16_t*)nullptr, (int64_t)0, 0,
               (const int32_t*)nullptr, nO, wmax_O, gamma, s_O, (float*)nullptr, beta_O_opt, (unsigned int*)nullptr, colmax_O, 1);
    return launch_status();
}

extern "C" quaff_status_t quaff_requant_weight_rows(const quaff_bf16* W_O, int64_t ldwo, int nO, int N, const float* s_O,
                                                    int8_t* wq_O, int64_t ldwq, int nOp, float* dw_O,
                                                    quaff_stream_t stream) {
    QUAFF_RETURN_IF(nO < 0 || N <= 0 || nOp < nO || !dw_O, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(nO > 0 && (!W_O || !s_O || ldwo < N), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(nOp > 0 && (!wq_O || ldwq < nOp), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(nOp % 16, QUAFF_ERR_UNSUPPORTED_SHAPE);
    QUAFF_RETURN_IF(nOp > 0 && (!aligned16(wq_O) || (ldwq % 16)), QUAFF_ERR_ALIGNMENT);
    const size_t smem = (size_t)((nO + 3) & ~3) * 4 + 8 * kRqCols * 4 + (size_t)kRqCols * kRqPitch;
    launch_pdl(requant_rows_kernel, dim3(ceil_div(N, kRqCols)), dim3(256), smem, (cudaStream_t)stream, 1, W_O, ldwo, nO, N, s_O, wq_O, ldwq, nOp, dw_O);
    return launch_status();
}

extern "C" quaff_status_t quaff_prepare_weight(const quaff_bf16* Wt, int64_t ldw, int N, int K, const int32_t* O_idx,
                                               int nO, int8_t* Wq, int64_t ldwq, float* dW, quaff_bf16* W_O,
                                               int64_t ldwo, float* wmax_O, quaff_stream_t stream) {
    QUAFF_RETURN_IF(!Wt || !Wq || !dW || N <= 0 || K <= 0 || ldw < K || ldwq < K, QUAFF_ERR_INVALID_ARG);
    QUAFF_CHECK_OUTLIERS(O_idx, nO, K);
    QUAFF_RETURN_IF(nO > 0 && (!W_O || !wmax_O || ldwo < N), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(!aligned16(Wt) || !aligned16(Wq) || (ldw % 8) || (ldwq % 16), QUAFF_ERR_ALIGNMENT);
    cudaStream_t st = (cudaStream_t)stream;
    // Eq. 1 per output channel of W = per row of the [N][K] layout: the per-token kernel without outliers
    quaff_status_t rc = quant_act_dispatch(Wt, ldw, N, K, nullptr, 0, nullptr, Wq, ldwq, nullptr, 0, 0, dW, st);
    if (rc != QUAFF_OK) return rc;
    if (nO > 0) {
        launch_pdl(gather_outlier_rows_kernel, dim3(nO), dim3(256), 0, st, 1, Wt, ldw, N, O_idx, W_O, ldwo, wmax_O);
        rc = launch_status();
    }
    return rc;
}

extern "C" quaff_status_t quaff_momentum_update_static(const quaff_bf16* X, int64_t ldx, int M, int K,
                                                       const int32_t* O_idx, int nO, const float* wmax_O, float gamma,
                                                       float* s_O, float* colmax_O_opt, float* beta_O_opt,
                                                       quaff_stream_t stream) {
    QUAFF_RETURN_IF(!X || M < 0 || K <= 0 || ldx < K, QUAFF_ERR_INVALID_ARG);
    QUAFF_CHECK_OUTLIERS(O_idx, nO, K);    // nO > 4096: more outlier channels than the built-in scratch (or any entry point) takes
    QUAFF_RETURN_IF(!(gamma >= 0.0f && gamma <= 1.0f), QUAFF_ERR_INVALID_ARG);
    if (nO == 0) return QUAFF_OK;
    QUAFF_RETURN_IF(!wmax_O || !s_O, QUAFF_ERR_INVALID_ARG);

    // In host code `g_momentum_scratch` is only a stand-in for the device array; the address a kernel
    // may use comes from cudaGetSymbolAddress, once per device, with that device current.
    static std::atomic<unsigned int*> scratch_of_device[64];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return QUAFF_ERR_CUDA;
    unsigned int* scratch = scratch_of_device[dev].load();
    if (!scratch) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_momentum_scratch) != cudaSuccess || !ptr) return QUAFF_ERR_CUDA;
        scratch = static_cast<unsigned int*>(ptr);
        scratch_of_device[dev].store(scratch);      // the same address whichever thread gets here first
    }
    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps the previous call's maxima and ticket count: both must start at zero
    if (cudaMemsetAsync(scratch, 0, (size_t)(nO + 1) * sizeof(unsigned int), st) != cudaSuccess) return QUAFF_ERR_CUDA;
    launch_pdl(momentum_kernel, dim3(momentum_grid(M)), dim3(256), 0, st, 1, X, ldx, M, O_idx, nO, wmax_O, gamma, s_O, colmax_O_opt,
               beta_O_opt, scratch, (const float*)nullptr, 1);
    return launch_status();
}

extern "C" quaff_status_t quaff_quant_grad(const quaff_bf16* dY, int64_t lddy, int M, int N, const float* dW, int8_t* Zq,
                                           int64_t ldz, float* dz, quaff_stream_t stream) {
    QUAFF_RETURN_IF(!dY || !dW || !Zq || !dz || M < 0 || N <= 0 || lddy < N || ldz < N, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF((N % 16) || N > 16384, QUAFF_ERR_UNSUPPORTED_SHAPE);
    QUAFF_RETURN_IF(!aligned16(dY) || !aligned16(Zq) || !aligned16(dW) || (lddy % 8) || (ldz % 16), QUAFF_ERR_ALIGNMENT);
    if (M == 0) return QUAFF_OK;
    return quant_grad_dispatch(dY, lddy, M, N, dW, Zq, ldz, dz, (cudaStream_t)stream);
}
