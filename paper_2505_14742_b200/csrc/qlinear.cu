// quaff_qlinear_fwd / quaff_qlinear_bwd: host side (validation, tensor maps, workspace carving,
// launches) and the small kernels around the two tcgen05 GEMMs (LoRA projections, weight
// dequantization for the backward, outlier-column fix-up, LoRA gradients).
#include <string.h>

#include "umma_gemm.cuh"

namespace quaff {

// ------------------------------------------------------------------ tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

quaff_status_t make_tmap_2d(CUtensorMap* map, const void* base, int elem_bytes, uint64_t rows, uint64_t cols,
                            uint64_t ld, uint32_t box_rows, uint32_t box_cols) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return QUAFF_ERR_CUDA;
    if (!aligned16(base) || (ld * elem_bytes) % 16 != 0) return QUAFF_ERR_ALIGNMENT;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {ld * (uint64_t)elem_bytes};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapDataType dt = elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    const CUresult rc = fn(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS ? QUAFF_OK : QUAFF_ERR_CUDA;
}

static cudaEvent_t g_time_start[2] = {nullptr, nullptr};
static cudaEvent_t g_time_stop[2] = {nullptr, nullptr};

template <int EPI>
static quaff_status_t launch_gemm(const GemmParams& p, cudaStream_t st) {
    static bool configured[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        if (cudaFuncSetAttribute(umma_gemm_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kGemmSmemBytes) != cudaSuccess)
            return QUAFF_ERR_CUDA;
        configured[dev] = true;
    }
    const int ntiles = p.tiles_m * p.tiles_n;
    if (ntiles == 0) return QUAFF_OK;
    const int grid = min(ntiles, sm_count());
    const bool timed = g_time_start[EPI] && g_time_stop[EPI];
    if (timed) cudaEventRecord(g_time_start[EPI], st);
    umma_gemm_kernel<EPI><<<grid, kGemmThreads, kGemmSmemBytes, st>>>(p);
    const quaff_status_t rc = launch_status();
    if (timed) {
        cudaEventRecord(g_time_stop[EPI], st);
        g_time_start[EPI] = g_time_stop[EPI] = nullptr;
    }
    return rc;
}

// ------------------------------------------------------------------ small kernels
// Bt[n][j] = B[j][n] for j < r, 0 for r <= j < rp  (K-major LoRA-up operand for the fused MMA)
__global__ void transpose_pad_kernel(const uint16_t* __restrict__ B, int r, int N, uint16_t* __restrict__ Bt, int rp) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= N * rp) return;
    const int n = idx / rp, j = idx % rp;
    Bt[idx] = j < r ? B[(int64_t)j * N + n] : (uint16_t)0;
}

// out[m][j] = bf16(scale * sum_c Big[m][c] * S(c, j)), one warp per row m, fp32 accumulation.
// S_IS_CJ: S stored [C][r] (LoRA A: T = X A); otherwise S stored [r][C] (LoRA B: G = dY B^T).
template <int R, bool S_IS_CJ>
__global__ void __launch_bounds__(256) row_times_small_kernel(const uint16_t* __restrict__ Big, int64_t ldb, int M, int C,
                                                             const uint16_t* __restrict__ S, int r, float scale,
                                                             uint16_t* __restrict__ out) {
    const int m = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (m >= M) return;
    float acc[R];
#pragma unroll
    for (int j = 0; j < R; ++j) acc[j] = 0.0f;
    const uint16_t* row = Big + (int64_t)m * ldb;
    for (int c0 = lane * 8; c0 < C; c0 += 256) {
        float x[8];
        if (c0 + 8 <= C) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(row + c0));
            x[0] = bf16_lo(v.x); x[1] = bf16_hi(v.x); x[2] = bf16_lo(v.y); x[3] = bf16_hi(v.y);
            x[4] = bf16_lo(v.z); x[5] = bf16_hi(v.z); x[6] = bf16_lo(v.w); x[7] = bf16_hi(v.w);
        } else {
            for (int e = 0; e < 8; ++e) x[e] = c0 + e < C ? bf16_bits_to_f32(row[c0 + e]) : 0.0f;
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int c = min(c0 + e, C - 1);
#pragma unroll
            for (int j = 0; j < R; ++j) {
                if (j < r) {
                    const float s = bf16_bits_to_f32(S_IS_CJ ? __ldg(S + (int64_t)c * r + j) : __ldg(S + (int64_t)j * C + c));
                    acc[j] = fmaf(x[e], s, acc[j]);
                }
            }
        }
    }
#pragma unroll
    for (int j = 0; j < R; ++j) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], o);
    }
    if (lane == 0)
        for (int j = 0; j < r; ++j) out[(int64_t)m * r + j] = (uint16_t)f32_to_bf16_bits(scale * acc[j]);
}

// part[s][c][j] = sum over the s-th slice of rows m of Big[m][c] * Small[m][j]   (fp32)
template <int R>
__global__ void __launch_bounds__(128) cols_times_small_kernel(const uint16_t* __restrict__ Big, int64_t ldb, int M, int C,
                                                              const uint16_t* __restrict__ Small, int r,
                                                              float* __restrict__ part, int rows_per_split) {
    __shared__ float sm_small[32][R];
    const int c = (blockIdx.x * 128 + threadIdx.x) * 2;
    const int m_begin = blockIdx.y * rows_per_split;
    const int m_end = min(M, m_begin + rows_per_split);
    float acc0[R], acc1[R];
#pragma unroll
    for (int j = 0; j < R; ++j) { acc0[j] = 0.0f; acc1[j] = 0.0f; }
    for (int mb = m_begin; mb < m_end; mb += 32) {
        __syncthreads();
        for (int i = threadIdx.x; i < 32 * R; i += 128) {
            const int mm = i / R, j = i % R;
            sm_small[mm][j] = (mb + mm < m_end && j < r) ? bf16_bits_to_f32(Small[(int64_t)(mb + mm) * r + j]) : 0.0f;
        }
        __syncthreads();
        if (c < C) {
            const int rows = min(32, m_end - mb);
            for (int mm = 0; mm < rows; ++mm) {
                const uint16_t* row = Big + (int64_t)(mb + mm) * ldb;
                float x0, x1;
                if (c + 1 < C && (ldb % 2 == 0)) {
                    const uint32_t v = __ldg(reinterpret_cast<const uint32_t*>(row + c));
                    x0 = bf16_lo(v); x1 = bf16_hi(v);
                } else {
                    x0 = bf16_bits_to_f32(row[c]);
                    x1 = c + 1 < C ? bf16_bits_to_f32(row[c + 1]) : 0.0f;
                }
#pragma unroll
                for (int j = 0; j < R; ++j) {
                    const float s = sm_small[mm][j];
                    acc0[j] = fmaf(x0, s, acc0[j]);
                    acc1[j] = fmaf(x1, s, acc1[j]);
                }
            }
        }
    }
    if (c < C) {
        float* o = part + ((int64_t)blockIdx.y * C + c) * r;
        for (int j = 0; j < r; ++j) o[j] = acc0[j];
        if (c + 1 < C) for (int j = 0; j < r; ++j) o[r + j] = acc1[j];
    }
}

// dst = (accumulate ? dst : 0) + scale * sum_s part[s][c][j];  dst index c*r + j, or j*C + c when transposed
__global__ void reduce_parts_kernel(const float* __restrict__ part, int S, int C, int r, float scale, int transposed,
                                    int accumulate, float* __restrict__ dst) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= C * r) return;
    int c, j;
    if (transposed) { j = idx / C; c = idx % C; } else { c = idx / r; j = idx % r; }
    float sum = 0.0f;
    for (int s = 0; s < S; ++s) sum += part[((int64_t)s * C + c) * r + j];
    sum *= scale;
    dst[idx] = accumulate ? dst[idx] + sum : sum;
}

// Dequantized, transposed weight for the grad-input GEMM (contraction over n must be contiguous):
//   rows 0..K-1              : Wext[k][n]          = bf16(Wq[n][k]   * dW[n])
//   rows K..Kpad-1           : 0   (Kpad = K rounded up to the tile width, so the rows below start a tile)
//   rows Kpad..Kpad+nOp-1    : Wext[Kpad+i][n]     = bf16(Wq[n][O_i] * dW[n])   (i < nO, else 0)
//   rows Kpad+nOp..Kpad+2nOp : Wext[Kpad+nOp+i][n] = bf16(wq_O[n][i] * dw_O[n])
__global__ void __launch_bounds__(256) expand_weight_kernel(const int8_t* __restrict__ Wq, int64_t ldwq_main,
                                                           const float* __restrict__ dW,
                                                           const int8_t* __restrict__ wq_O, int64_t ldwq,
                                                           const float* __restrict__ dw_O,
                                                           const int32_t* __restrict__ O_idx, int nO, int nOp, int K,
                                                           int Kpad, int N, uint16_t* __restrict__ Wext, int64_t ldw) {
    __shared__ uint16_t tile[32][33];
    const int e0 = blockIdx.x * 32, n0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 x 8
    const int Kext = Kpad + 2 * nOp;
    // load: thread (tx = ext row offset, ty.. = n offset)
    const int e = e0 + tx;
    const int8_t* src = nullptr;
    int64_t lds = 0;
    const float* sc = nullptr;
    if (e < K) { src = Wq + e; lds = ldwq_main; sc = dW; }
    else if (e >= Kpad && e < Kpad + nOp) { const int i = e - Kpad; if (i < nO) { src = Wq + O_idx[i]; lds = ldwq_main; sc = dW; } }
    else if (e >= Kpad + nOp && e < Kext) { src = wq_O + (e - Kpad - nOp); lds = ldwq; sc = dw_O; }
    for (int yy = ty; yy < 32; yy += 8) {
        const int n = n0 + yy;
        uint16_t v = 0;
        if (src && n < N) v = (uint16_t)f32_to_bf16_bits(__fmul_rn((float)src[(int64_t)n * lds], sc[n]));
        tile[tx][yy] = v;
    }
    __syncthreads();
    for (int yy = ty; yy < 32; yy += 8) {
        const int er = e0 + yy, n = n0 + tx;
        if (er < Kext && n < N) Wext[(int64_t)er * ldw + n] = tile[yy][tx];
    }
}

// dX[m][O_i] = bf16((P[m][i] + P[m][nOp+i]) / s_i + sum_j G[m][j] A[O_i][j])
__global__ void bwd_fixup_kernel(const float* __restrict__ P, int64_t ldp, int M, int nO, int nOp,
                                 const int32_t* __restrict__ O_idx, const float* __restrict__ s_O,
                                 const uint16_t* __restrict__ G, const uint16_t* __restrict__ A, int r,
                                 uint16_t* __restrict__ dX, int64_t lddx) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= M * nO) return;
    const int m = idx / nO, i = idx % nO;
    const int k = O_idx[i];
    float v = (P[(int64_t)m * ldp + i] + P[(int64_t)m * ldp + nOp + i]) / s_O[i];
    float l = 0.0f;
    for (int j = 0; j < r; ++j) l = fmaf(bf16_bits_to_f32(G[(int64_t)m * r + j]), bf16_bits_to_f32(A[(int64_t)k * r + j]), l);
    dX[(int64_t)m * lddx + k] = (uint16_t)f32_to_bf16_bits(v + l);
}

template <bool S_IS_CJ>
static quaff_status_t launch_row_times_small(const uint16_t* Big, int64_t ldb, int M, int C, const uint16_t* S, int r,
                                             float scale, uint16_t* out, cudaStream_t st) {
    const int grid = ceil_div(M, 8);
    if (r <= 16) row_times_small_kernel<16, S_IS_CJ><<<grid, 256, 0, st>>>(Big, ldb, M, C, S, r, scale, out);
    else if (r <= 32) row_times_small_kernel<32, S_IS_CJ><<<grid, 256, 0, st>>>(Big, ldb, M, C, S, r, scale, out);
    else row_times_small_kernel<64, S_IS_CJ><<<grid, 256, 0, st>>>(Big, ldb, M, C, S, r, scale, out);
    return launch_status();
}

static int split_count(int M, int C) {
    const int blocks_c = ceil_div(C, 256);
    int S = ceil_div(2 * sm_count(), blocks_c);
    S = max(1, min(S, ceil_div(M, 64)));
    return S;
}

static quaff_status_t launch_cols_times_small(const uint16_t* Big, int64_t ldb, int M, int C, const uint16_t* Small, int r,
                                              float scale, int transposed, int accumulate, float* part, float* dst,
                                              cudaStream_t st) {
    const int S = split_count(M, C);
    const int rows_per_split = ceil_div(ceil_div(M, S), 32) * 32;
    const dim3 grid(ceil_div(C, 256), S);
    if (r <= 16) cols_times_small_kernel<16><<<grid, 128, 0, st>>>(Big, ldb, M, C, Small, r, part, rows_per_split);
    else if (r <= 32) cols_times_small_kernel<32><<<grid, 128, 0, st>>>(Big, ldb, M, C, Small, r, part, rows_per_split);
    else cols_times_small_kernel<64><<<grid, 128, 0, st>>>(Big, ldb, M, C, Small, r, part, rows_per_split);
    if (launch_status() != QUAFF_OK) return QUAFF_ERR_CUDA;
    reduce_parts_kernel<<<ceil_div(C * r, 256), 256, 0, st>>>(part, S, C, r, scale, transposed, accumulate, dst);
    return launch_status();
}

static int pad16(int r) { return (r + 15) / 16 * 16; }

struct BwdWorkspace {
    size_t off_wext, off_g, off_p, off_part, total;
    int64_t ldw;  // row pitch of Wext in elements
};

static BwdWorkspace bwd_workspace(int M, int K, int N, int nOp, int r) {
    BwdWorkspace w;
    w.ldw = (int64_t)round_up((size_t)N, 8);
    size_t off = 0;
    const size_t kpad = round_up((size_t)K, kTileN);
    w.off_wext = off; off += round_up((kpad + 2 * (size_t)nOp) * w.ldw * 2, 256);
    w.off_g = off;    off += round_up((size_t)M * (size_t)max(r, 1) * 2, 256);
    w.off_p = off;    off += round_up((size_t)M * (size_t)max(2 * nOp, 1) * 4, 256);
    w.off_part = off;
    const size_t pa = (size_t)split_count(M, K) * K * max(r, 1) * 4;
    const size_t pb = (size_t)split_count(M, N) * N * max(r, 1) * 4;
    off += round_up(pa > pb ? pa : pb, 256);
    w.total = off;
    return w;
}

}  // namespace quaff

using namespace quaff;

extern "C" uint64_t quaff_debug_launch_count(void) { return g_launch_count; }

extern "C" void quaff_debug_time_gemm(int which, void* start_event, void* stop_event) {
    if (which < 0 || which > 1) return;
    g_time_start[which] = (cudaEvent_t)start_event;
    g_time_stop[which] = (cudaEvent_t)stop_event;
}

extern "C" const char* quaff_status_string(quaff_status_t s) {
    switch (s) {
        case QUAFF_OK: return "ok";
        case QUAFF_ERR_INVALID_ARG: return "invalid argument";
        case QUAFF_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case QUAFF_ERR_ALIGNMENT: return "pointer or leading dimension not 16-byte aligned";
        case QUAFF_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case QUAFF_ERR_CUDA: return "CUDA call failed";
        case QUAFF_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

extern "C" size_t quaff_workspace_bytes(int which, int M, int K, int N, int nOp, int r) {
    switch (which) {
        case QUAFF_WS_PREPARE: return 0;
        case QUAFF_WS_MOMENTUM: return round_up((size_t)(nOp + 1) * 4, 256);
        case QUAFF_WS_FWD: return round_up((size_t)N * (size_t)pad16(max(r, 1)) * 2, 256);
        case QUAFF_WS_BWD: return bwd_workspace(M, K, N, nOp, r).total;
    }
    return 0;
}

extern "C" quaff_status_t quaff_qlinear_fwd(int M, int K, int N, const int8_t* Xq, int64_t ldxq, const int8_t* xq_O,
                                            int64_t ldxo, int nOp, const float* dx, const int8_t* Wq, int64_t ldwq_main,
                                            const float* dW, const int8_t* wq_O, int64_t ldwq, const float* dw_O,
                                            const quaff_bf16* X, int64_t ldx, const quaff_bf16* A, const quaff_bf16* B,
                                            int r, float lora_scale, quaff_bf16* T_out, void* Y, int y_dtype, int64_t ldy,
                                            int32_t* dbg_acc_main, int32_t* dbg_acc_out, int32_t* status_opt, void* ws,
                                            size_t ws_bytes, quaff_stream_t stream) {
    QUAFF_RETURN_IF(M < 0 || K <= 0 || N <= 0 || nOp < 0 || r < 0, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(!Xq || !dx || !Wq || !dW || !Y || ldxq < K || ldwq_main < K || ldy < N, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(nOp > 0 && (!xq_O || !wq_O || !dw_O || ldxo < nOp || ldwq < nOp), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(r > 0 && (!X || !A || !B || !T_out || ldx < K), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(y_dtype != QUAFF_BF16 && y_dtype != QUAFF_F32, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF((nOp % 32) || (r % 8) || r > 64, QUAFF_ERR_UNSUPPORTED_SHAPE);
    QUAFF_RETURN_IF(!aligned16(Xq) || !aligned16(Wq) || (ldxq % 16) || (ldwq_main % 16), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(nOp > 0 && (!aligned16(xq_O) || !aligned16(wq_O) || (ldxo % 16) || (ldwq % 16)), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(r > 0 && (!aligned16(X) || !aligned16(T_out) || (ldx % 8)), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(!aligned16(Y), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(r > 0 && (!ws || !aligned16(ws) || ws_bytes < quaff_workspace_bytes(QUAFF_WS_FWD, M, K, N, nOp, r)),
                    QUAFF_ERR_WORKSPACE_TOO_SMALL);
    if (M == 0) return QUAFF_OK;
    cudaStream_t st = (cudaStream_t)stream;
    const int rp = pad16(r);
    uint16_t* Bt = reinterpret_cast<uint16_t*>(ws);

    GemmParams p;
    memset(&p, 0, sizeof(p));
    quaff_status_t rc;
    int np = 0;
    {   // main: acc1 = Xq Wq^T over K
        GemmPhase& ph = p.ph[np++];
        if ((rc = make_tmap_2d(&ph.map_a, Xq, 1, M, K, ldxq, kTileM, 128)) != QUAFF_OK) return rc;
        if ((rc = make_tmap_2d(&ph.map_b, Wq, 1, N, K, ldwq_main, kTileN, 128)) != QUAFF_OK) return rc;
        ph.nblk = ceil_div(K, 128); ph.is_i8 = 1; ph.kext = K; ph.acc_slot = 0; ph.fresh = 1; ph.tn_limit = 1 << 30;
    }
    if (nOp > 0) {   // outlier: acc2 = xq_O wq_O^T over nOp
        GemmPhase& ph = p.ph[np++];
        if ((rc = make_tmap_2d(&ph.map_a, xq_O, 1, M, nOp, ldxo, kTileM, 128)) != QUAFF_OK) return rc;
        if ((rc = make_tmap_2d(&ph.map_b, wq_O, 1, N, nOp, ldwq, kTileN, 128)) != QUAFF_OK) return rc;
        ph.nblk = ceil_div(nOp, 128); ph.is_i8 = 1; ph.kext = nOp; ph.acc_slot = 1; ph.fresh = 1; ph.tn_limit = 1 << 30;
    }
    if (r > 0) {     // LoRA up: acc3 = T Bt^T over r
        transpose_pad_kernel<<<ceil_div(N * rp, 256), 256, 0, st>>>(B, r, N, Bt, rp);
        if ((rc = launch_status()) != QUAFF_OK) return rc;
        if ((rc = launch_row_times_small<true>(X, ldx, M, K, A, r, 1.0f, T_out, st)) != QUAFF_OK) return rc;
        GemmPhase& ph = p.ph[np++];
        if ((rc = make_tmap_2d(&ph.map_a, T_out, 2, M, r, r, kTileM, 64)) != QUAFF_OK) return rc;
        if ((rc = make_tmap_2d(&ph.map_b, Bt, 2, N, rp, rp, kTileN, 64)) != QUAFF_OK) return rc;
        ph.nblk = ceil_div(rp, 64); ph.is_i8 = 0; ph.kext = rp; ph.acc_slot = 2; ph.fresh = 1; ph.tn_limit = 1 << 30;
    }
    p.nphases = np;
    p.M = M; p.N = N;
    p.tiles_m = ceil_div(M, kTileM); p.tiles_n = ceil_div(N, kTileN);
    p.status = status_opt;
    p.dx = dx; p.dW = dW; p.dw_O = dw_O; p.lora_scale = lora_scale;
    p.has_outlier = nOp > 0; p.has_lora = r > 0;
    p.Y = Y; p.ldy = ldy; p.y_f32 = (y_dtype == QUAFF_F32);
    p.dbg_main = dbg_acc_main; p.dbg_out = dbg_acc_out;
    return launch_gemm<EPI_FWD>(p, st);
}

extern "C" quaff_status_t quaff_qlinear_bwd(int M, int K, int N, const quaff_bf16* dY, int64_t lddy, const int8_t* Wq,
                                            int64_t ldwq_main, const float* dW, const int8_t* wq_O, int64_t ldwq,
                                            const float* dw_O, int nOp, const int32_t* O_idx, int nO, const float* s_O,
                                            const quaff_bf16* X, int64_t ldx, const quaff_bf16* T, const quaff_bf16* A,
                                            const quaff_bf16* B, int r, float lora_scale, quaff_bf16* dX, int64_t lddx,
                                            float* dA, float* dB, int accumulate, int32_t* status_opt, void* ws,
                                            size_t ws_bytes, quaff_stream_t stream) {
    QUAFF_RETURN_IF(M < 0 || K <= 0 || N <= 0 || nOp < 0 || nO < 0 || nO > nOp || r < 0, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(!dY || lddy < N || !Wq || !dW || ldwq_main < K, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(nOp > 0 && (!wq_O || !dw_O || ldwq < nOp), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(nO > 0 && (!O_idx || !s_O), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(r > 0 && (!A || !B), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(r > 0 && (dA || dB) && (!dA || !dB || !X || !T || ldx < K), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(dX && lddx < K, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF((nOp % 32) || (r % 8) || r > 64, QUAFF_ERR_UNSUPPORTED_SHAPE);
    QUAFF_RETURN_IF(!aligned16(dY) || (lddy % 8), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(dX && (!aligned16(dX) || (lddx % 8)), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(r > 0 && !aligned16(A), QUAFF_ERR_ALIGNMENT);
    const BwdWorkspace w = bwd_workspace(M, K, N, nOp, r);
    QUAFF_RETURN_IF(!ws || !aligned16(ws) || ws_bytes < w.total, QUAFF_ERR_WORKSPACE_TOO_SMALL);
    if (M == 0) return QUAFF_OK;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned char* base = reinterpret_cast<unsigned char*>(ws);
    uint16_t* Wext = reinterpret_cast<uint16_t*>(base + w.off_wext);
    uint16_t* G = reinterpret_cast<uint16_t*>(base + w.off_g);
    float* P = reinterpret_cast<float*>(base + w.off_p);
    float* part = reinterpret_cast<float*>(base + w.off_part);
    quaff_status_t rc;

    if (r > 0) {   // G = bf16(lora_scale * dY B^T)
        if ((rc = launch_row_times_small<false>(dY, lddy, M, N, B, r, lora_scale, G, st)) != QUAFF_OK) return rc;
    }
    if (dX) {
        const int Kpad = ceil_div(K, kTileN) * kTileN;
        const int Kext = nOp > 0 ? Kpad + 2 * nOp : K;
        expand_weight_kernel<<<dim3(ceil_div(Kext, 32), ceil_div(N, 32)), 256, 0, st>>>(Wq, ldwq_main, dW, wq_O, ldwq, dw_O,
                                                                                      O_idx, nO, nOp, K, Kpad, N, Wext, w.ldw);
        if ((rc = launch_status()) != QUAFF_OK) return rc;
        GemmParams p;
        memset(&p, 0, sizeof(p));
        int np = 0;
        {   // main: dY Wext^T over N
            GemmPhase& ph = p.ph[np++];
            if ((rc = make_tmap_2d(&ph.map_a, dY, 2, M, N, lddy, kTileM, 64)) != QUAFF_OK) return rc;
            if ((rc = make_tmap_2d(&ph.map_b, Wext, 2, Kext, N, w.ldw, kTileN, 64)) != QUAFF_OK) return rc;
            ph.nblk = ceil_div(N, 64); ph.is_i8 = 0; ph.kext = N; ph.acc_slot = 0; ph.fresh = 1; ph.tn_limit = 1 << 30;
        }
        if (r > 0) {   // + G A^T over r, only for the real dX columns
            GemmPhase& ph = p.ph[np++];
            if ((rc = make_tmap_2d(&ph.map_a, G, 2, M, r, r, kTileM, 64)) != QUAFF_OK) return rc;
            if ((rc = make_tmap_2d(&ph.map_b, A, 2, K, r, r, kTileN, 64)) != QUAFF_OK) return rc;
            ph.nblk = ceil_div(r, 64); ph.is_i8 = 0; ph.kext = pad16(r); ph.acc_slot = 0; ph.fresh = 0;
            ph.tn_limit = ceil_div(K, kTileN);
        }
        p.nphases = np;
        p.M = M;
        // columns [0,K) -> dX; the outlier partial products start at the next tile boundary Kpad
        p.n_split = K;
        p.p_col0 = Kpad;
        p.N = Kext;
        p.tiles_m = ceil_div(M, kTileM);
        p.tiles_n = ceil_div(p.N, kTileN);
        p.status = status_opt;
        p.dX = dX; p.lddx = lddx; p.P = P; p.ldp = 2 * nOp;
        if ((rc = launch_gemm<EPI_BWD>(p, st)) != QUAFF_OK) return rc;
        if (nO > 0) {
            bwd_fixup_kernel<<<ceil_div(M * nO, 256), 256, 0, st>>>(P, 2 * nOp, M, nO, nOp, O_idx, s_O, G, A, r, dX, lddx);
            if ((rc = launch_status()) != QUAFF_OK) return rc;
        }
    }
    if (r > 0 && dA && dB) {
        if ((rc = launch_cols_times_small(X, ldx, M, K, G, r, 1.0f, 0, accumulate, part, dA, st)) != QUAFF_OK) return rc;
        if ((rc = launch_cols_times_small(dY, lddy, M, N, T, r, lora_scale, 1, accumulate, part, dB, st)) != QUAFF_OK) return rc;
    }
    return QUAFF_OK;
}
