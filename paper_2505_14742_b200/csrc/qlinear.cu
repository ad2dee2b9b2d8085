// quaff_qlinear_fwd / quaff_qlinear_bwd: host side (validation, tensor maps, workspace carving,
// launches) and the small kernels around the two tcgen05 GEMMs (LoRA projections, weight
// dequantization for the backward, outlier-column fix-up, LoRA gradients).
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>

#include "bwd_expand.cuh"
#include "fwd256.cuh"

namespace quaff {

// ------------------------------------------------------------------ tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static const EncodeTiledFn fn = [] {      // initialised once, whichever thread comes first
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            return reinterpret_cast<EncodeTiledFn>(sym);
        return static_cast<EncodeTiledFn>(nullptr);
    }();
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

// Side streams of the backward: work that does not depend on each other (the dequantization of the weight,
// G = dY B^T, dB = T^T dY; later the outlier fix-up and dA = X^T G) is forked from the caller's stream onto
// these and joined back with events, so the small kernels overlap instead of queueing.  Each device has a small
// pool of SETS (two streams and their events), created by the first backward call on that device.  A call takes
// a set for the time it enqueues its work, under the device's mutex: outside stream capture any set will do (an
// event may be re-recorded once the wait that refers to it has been enqueued); a set whose streams have been drawn
// into a capture stays with that capture until it ends.  Calls from several host threads are therefore safe; they
// are enqueued one after the other.
constexpr int kSideSets = 4;
struct SideSet {
    cudaStream_t s[2];
    cudaEvent_t fork[2], join[2], g_ready;
};
struct DeviceSide {
    std::once_flag once;
    std::mutex mu;          // held while a backward call enqueues its work
    bool ok = false;
    SideSet set[kSideSets];
};
static DeviceSide* device_side() {
    static DeviceSide per_dev[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    DeviceSide& ds = per_dev[dev];
    std::call_once(ds.once, [&ds] {
        bool ok = true;
        // lowest priority, so that the side work never outranks the caller's stream (a default stream has the same
        // priority: there the launch order decides, which is why the backward enqueues dA and dB behind its GEMM)
        int least = 0, greatest = 0;
        cudaDeviceGetStreamPriorityRange(&least, &greatest);
        for (int k = 0; k < kSideSets; ++k) {
            SideSet& ss = ds.set[k];
            ok = ok && cudaEventCreateWithFlags(&ss.g_ready, cudaEventDisableTiming) == cudaSuccess;
            for (int i = 0; i < 2; ++i) {
                ok = ok && cudaStreamCreateWithPriority(&ss.s[i], cudaStreamNonBlocking, least) == cudaSuccess;
                ok = ok && cudaEventCreateWithFlags(&ss.fork[i], cudaEventDisableTiming) == cudaSuccess;
                ok = ok && cudaEventCreateWithFlags(&ss.join[i], cudaEventDisableTiming) == cudaSuccess;
            }
        }
        if (!ok) cudaGetLastError();
        ds.ok = ok;
    });
    return ds.ok ? &ds : nullptr;
}
// A set this call on stream `st` may use (the device's mutex is held): one whose streams belong to the capture `st`
// is part of, else one that is in no capture; null if every set is tied to some other capture.
static SideSet* pick_side_set(DeviceSide* ds, cudaStream_t st) {
    cudaStreamCaptureStatus mine = cudaStreamCaptureStatusNone;
    unsigned long long my_id = 0;
    if (cudaStreamGetCaptureInfo(st, &mine, &my_id) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    SideSet* free_set = nullptr;
    for (int k = 0; k < kSideSets; ++k) {
        SideSet* ss = &ds->set[k];
        bool in_capture = false, same = true;
        for (int i = 0; i < 2; ++i) {
            cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
            unsigned long long id = 0;
            if (cudaStreamGetCaptureInfo(ss->s[i], &cs, &id) != cudaSuccess) { cudaGetLastError(); in_capture = true; same = false; continue; }
            if (cs != cudaStreamCaptureStatusNone) {
                in_capture = true;
                if (cs != cudaStreamCaptureStatusActive || mine != cudaStreamCaptureStatusActive || id != my_id) same = false;
            }
        }
        if (in_capture && same) return ss;              // already part of this capture
        if (!in_capture && !free_set) free_set = ss;
    }
    return free_set;
}
// side stream i continues from the current end of `st` / `st` continues after side stream i
static bool fork_to(SideSet* ss, int i, cudaStream_t st) {
    return cudaEventRecord(ss->fork[i], st) == cudaSuccess && cudaStreamWaitEvent(ss->s[i], ss->fork[i], 0) == cudaSuccess;
}
static bool join_from(SideSet* ss, int i, cudaStream_t st) {
    return cudaEventRecord(ss->join[i], ss->s[i]) == cudaSuccess && cudaStreamWaitEvent(st, ss->join[i], 0) == cudaSuccess;
}

// Measurement aids: per host thread, one-shot (see quaff.h)
static thread_local cudaEvent_t g_time_start[2] = {nullptr, nullptr};
static thread_local cudaEvent_t g_time_stop[2] = {nullptr, nullptr};

// Tile-processing units (CTAs, or CTA pairs) that can be resident at once.
template <int EPI, int CTAS, int TN>
static int gemm_units(int dev) {
    static std::atomic<int> cached[64];
    if (cached[dev].load()) return cached[dev].load();
    int units = sm_count() / CTAS;
    if (CTAS == 2) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(sm_count() / 2 * 2);
        cfg.blockDim = dim3(kGemmThreads);
        cfg.dynamicSmemBytes = GemmCfg<EPI, CTAS, TN>::kSmemBytes;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        int nclusters = 0;
        if (cudaOccupancyMaxActiveClusters(&nclusters, umma_gemm_kernel<EPI, CTAS, TN>, &cfg) == cudaSuccess && nclusters > 0)
            units = min(units, nclusters);
        else
            cudaGetLastError();
    }
    cached[dev].store(max(units, 1));     // every thread computes the same value
    return cached[dev].load();
}

template <int EPI, int CTAS, int TN>
static quaff_status_t launch_gemm(const GemmParams& p, cudaStream_t st) {
    using Cfg = GemmCfg<EPI, CTAS, TN>;
    static std::atomic<bool> configured[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) return QUAFF_ERR_CUDA;
    if (!configured[dev].load()) {     // setting the attribute twice (two threads at once) is harmless
        if (cudaFuncSetAttribute(umma_gemm_kernel<EPI, CTAS, TN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::kSmemBytes) != cudaSuccess)
            return QUAFF_ERR_CUDA;
        configured[dev].store(true);
    }
    const int ntiles = p.tiles_m * p.tiles_n;
    if (ntiles == 0) return QUAFF_OK;
    const int units = min(ntiles, gemm_units<EPI, CTAS, TN>(dev));
    const bool timed = EPI < 2 && g_time_start[EPI % 2] && g_time_stop[EPI % 2];
    // while the stream is being captured into a CUDA graph, the events become event-record nodes of the
    // graph (every replay records them again); otherwise they are recorded once, now
    unsigned int ev_flags = cudaEventRecordDefault;
    if (timed) {
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusActive) ev_flags = cudaEventRecordExternal;
        cudaEventRecordWithFlags(g_time_start[EPI % 2], st, ev_flags);
    }
    launch_pdl(umma_gemm_kernel<EPI, CTAS, TN>, dim3(units * CTAS), dim3(kGemmThreads), Cfg::kSmemBytes, st, CTAS, p);
    const quaff_status_t rc = launch_status();
    if (timed) {
        cudaEventRecordWithFlags(g_time_stop[EPI % 2], st, ev_flags);
        g_time_start[EPI % 2] = g_time_stop[EPI % 2] = nullptr;
    }
    return rc;
}

// The wide forward kernels (fwd192.cuh, fwd256.cuh): which = 0 / 1
static quaff_status_t launch_fwd_wide(int which, const FwdWideParams& p, cudaStream_t st, int time_slot = 0) {
    static std::atomic<bool> configured[2][64];
    static std::atomic<int> units_of[2][64];
    void (*const kernel)(const FwdWideParams) = which ? fwd256_kernel : fwd192_kernel;
    const int threads = which ? kF256Threads : kF192Threads;
    const size_t smem = which ? kF256SmemBytes : kF192SmemBytes;
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) return QUAFF_ERR_CUDA;
    if (!configured[which][dev].load()) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return QUAFF_ERR_CUDA;
        int units = sm_count() / 2;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(units * 2);
        cfg.blockDim = dim3(threads);
        cfg.dynamicSmemBytes = smem;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        int nclusters = 0;
        if (cudaOccupancyMaxActiveClusters(&nclusters, kernel, &cfg) == cudaSuccess && nclusters > 0) units = min(units, nclusters);
        else cudaGetLastError();
        units_of[which][dev].store(max(units, 1));
        configured[which][dev].store(true);
    }
    const int ntiles = p.tiles_m * p.tiles_n;
    if (ntiles == 0) return QUAFF_OK;
    const int units = min(ntiles, units_of[which][dev].load());
    const bool timed = g_time_start[time_slot] && g_time_stop[time_slot];
    unsigned int ev_flags = cudaEventRecordDefault;
    if (timed) {
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusActive) ev_flags = cudaEventRecordExternal;
        cudaEventRecordWithFlags(g_time_start[time_slot], st, ev_flags);
    }
    launch_pdl(kernel, dim3(units * 2), dim3(threads), smem, st, 2, p);
    const quaff_status_t rc = launch_status();
    if (timed) {
        cudaEventRecordWithFlags(g_time_stop[time_slot], st, ev_flags);
        g_time_start[time_slot] = g_time_stop[time_slot] = nullptr;
    }
    return rc;
}

// The grad-input GEMM with in-kernel expansion of the INT8 weight (bwd_expand.cuh)
static size_t bx_fixed_bytes(int mask_words) {     // alignment slack, B ring, barriers, outlier mask
    return 1024 + (size_t)kBxBSlots * kBxBBytes + kBxBarrierBytes + round_up((size_t)2 * mask_words * 4, 16);
}
static size_t bx_smem_bytes(int nstages, int mask_words) {     // ... plus the IN ring with its row-scale ring
    return bx_fixed_bytes(mask_words) + (size_t)nstages * (kBxInBytes + 256);
}
static int bx_stages(int mask_words) {
    const int fit = (int)((kSmemLimit - bx_fixed_bytes(mask_words)) / (kBxInBytes + 256));
    return max(2, min(fit, kMaxStages));
}
static quaff_status_t launch_bwd_expand(const BxParams& p, cudaStream_t st) {
    static std::atomic<bool> configured[64];
    static std::atomic<int> units_of[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) return QUAFF_ERR_CUDA;
    if (!configured[dev].load()) {
        if (cudaFuncSetAttribute(bwd_expand_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) != cudaSuccess) return QUAFF_ERR_CUDA;
        int units = sm_count() / 2;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(units * 2);
        cfg.blockDim = dim3(kBxThreads);
        cfg.dynamicSmemBytes = kSmemLimit;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        int nclusters = 0;
        if (cudaOccupancyMaxActiveClusters(&nclusters, bwd_expand_kernel, &cfg) == cudaSuccess && nclusters > 0) units = min(units, nclusters);
        else cudaGetLastError();
        units_of[dev].store(max(units, 1));
        configured[dev].store(true);
    }
    const int ntiles = p.tiles_m * (p.tiles_main + p.tiles_p);
    if (ntiles == 0) return QUAFF_OK;
    const int units = min(ntiles, units_of[dev].load());
    const bool timed = g_time_start[1] && g_time_stop[1];
    unsigned int ev_flags = cudaEventRecordDefault;
    if (timed) {
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusActive) ev_flags = cudaEventRecordExternal;
        cudaEventRecordWithFlags(g_time_start[1], st, ev_flags);
    }
    launch_pdl(bwd_expand_kernel, dim3(units * 2), dim3(kBxThreads), bx_smem_bytes(p.nstages, p.mask_words), st, 2, p);
    const quaff_status_t rc = launch_status();
    if (timed) {
        cudaEventRecordWithFlags(g_time_stop[1], st, ev_flags);
        g_time_start[1] = g_time_stop[1] = nullptr;
    }
    return rc;
}

// ------------------------------------------------------------------ small kernels
// dst[c][j] = src[j][c] for j < rows, 0 for rows <= j < rows_pad   (src is [rows][cols], dst is [cols][rows_pad])
__global__ void transpose_pad_kernel(const uint16_t* __restrict__ src, int rows, int cols, uint16_t* __restrict__ dst, int rows_pad) {
    pdl_launch_dependents();
    pdl_wait();
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= cols * rows_pad) return;
    const int c = idx / rows_pad, j = idx % rows_pad;
    dst[idx] = j < rows ? src[(int64_t)j * cols + c] : (uint16_t)0;
}

// out[m][j] = bf16(scale * sum_s part[s][m][j]);  a thread sums 8 consecutive j (r is a multiple of 8)
__global__ void reduce_parts_bf16_kernel(const float* __restrict__ part, int S, int rows, int r, float scale,
                                         uint16_t* __restrict__ out) {
    pdl_launch_dependents();
    pdl_wait();
    const int64_t idx = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 8;
    const int64_t total = (int64_t)rows * r;
    if (idx >= total) return;
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    for (int s = 0; s < S; ++s) {
        const float4* src = reinterpret_cast<const float4*>(part + s * total + idx);
        const float4 a = __ldg(src), b = __ldg(src + 1);
        acc[0] += a.x; acc[1] += a.y; acc[2] += a.z; acc[3] += a.w;
        acc[4] += b.x; acc[5] += b.y; acc[6] += b.z; acc[7] += b.w;
    }
    *reinterpret_cast<uint4*>(out + idx) = make_uint4(pack_bf16x2(scale * acc[0], scale * acc[1]), pack_bf16x2(scale * acc[2], scale * acc[3]),
                                                      pack_bf16x2(scale * acc[4], scale * acc[5]), pack_bf16x2(scale * acc[6], scale * acc[7]));
}

// dst = (accumulate ? dst : 0) + scale * sum_s part[s][c][j];  dst index c*r + j, or j*C + c when transposed.
// A thread sums 4 consecutive j of one c (r is a multiple of 8); consecutive threads take consecutive c when the
// output is transposed (coalesced stores along c) and consecutive j-quads otherwise.
__global__ void reduce_parts_kernel(const float* __restrict__ part, int S, int C, int r, float scale, int transposed,
                                    int accumulate, float* __restrict__ dst) {
    pdl_launch_dependents();
    pdl_wait();
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    const int rq = r >> 2;
    if (idx >= C * rq) return;
    int c, jq;
    if (transposed) { jq = idx / C; c = idx % C; } else { c = idx / rq; jq = idx % rq; }
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < S; ++s) {
        const float4 a = __ldg(reinterpret_cast<const float4*>(part + ((int64_t)s * C + c) * r + 4 * jq));
        acc.x += a.x; acc.y += a.y; acc.z += a.z; acc.w += a.w;
    }
    const float v[4] = {acc.x * scale, acc.y * scale, acc.z * scale, acc.w * scale};
    if (!transposed) {
        float4* d = reinterpret_cast<float4*>(dst + (int64_t)c * r + 4 * jq);
        float4 o = make_float4(v[0], v[1], v[2], v[3]);
        if (accumulate) { const float4 old = *d; o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w; }
        *d = o;
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float* d = dst + (int64_t)(4 * jq + e) * C + c;
            *d = accumulate ? *d + v[e] : v[e];
        }
    }
}

// Dequantized weight for the grad-input GEMM, in the stored orientation [N][.] (the contraction index n
// is the row, so the GEMM reads it as an MN-major operand; nothing is transposed):
//   columns 0..K-1              : Wd[n][k]          = bf16(Wq[n][k]   * dW[n])
//   columns K..Kpad-1           : 0   (Kpad = K rounded up to 32: the epilogue tells dX from P columns per chunk)
//   columns Kpad..Kpad+nOp-1    : Wd[n][Kpad+i]     = bf16(Wq[n][O_i] * dW[n])   (i < nO, else 0)
//   columns Kpad+nOp..Kpad+2nOp : Wd[n][Kpad+nOp+i] = bf16(wq_O[n][i] * dw_O[n])
// One thread converts 16 consecutive columns of one row (one 128-bit load of codes, two 128-bit stores).
__global__ void __launch_bounds__(256) dequant_weight_kernel(const int8_t* __restrict__ Wq, int64_t ldwq_main,
                                                            const float* __restrict__ dW,
                                                            const int8_t* __restrict__ wq_O, int64_t ldwq,
                                                            const float* __restrict__ dw_O,
                                                            const int32_t* __restrict__ O_idx, int nO, int nOp, int K,
                                                            int Kpad, uint16_t* __restrict__ Wd, int64_t ldwd) {
    pdl_launch_dependents();
    pdl_wait();
    const int n = blockIdx.x;
    const int c = blockIdx.y * blockDim.x + threadIdx.x;
    const int k0 = c * 16;
    if (k0 >= Kpad + 2 * nOp) return;
    float v[16];
    if (k0 < Kpad) {
        const float sc = __ldg(dW + n);
        const int8_t* src = Wq + (int64_t)n * ldwq_main + k0;
        if (k0 + 16 <= K) {
            const uint4 raw = __ldg(reinterpret_cast<const uint4*>(src));
            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
            for (int e = 0; e < 16; ++e) v[e] = __fmul_rn((float)(int8_t)((w[e >> 2] >> ((e & 3) * 8)) & 0xFFu), sc);
        } else {
#pragma unroll
            for (int e = 0; e < 16; ++e) v[e] = (k0 + e < K) ? __fmul_rn((float)src[e], sc) : 0.0f;
        }
    } else if (k0 < Kpad + nOp) {
        const float sc = __ldg(dW + n);
        const int i0 = k0 - Kpad;
#pragma unroll
        for (int e = 0; e < 16; ++e)
            v[e] = (i0 + e < nO) ? __fmul_rn((float)Wq[(int64_t)n * ldwq_main + O_idx[i0 + e]], sc) : 0.0f;
    } else {
        const float sc = __ldg(dw_O + n);
        const uint4 raw = __ldg(reinterpret_cast<const uint4*>(wq_O + (int64_t)n * ldwq + (k0 - Kpad - nOp)));
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int e = 0; e < 16; ++e) v[e] = __fmul_rn((float)(int8_t)((w[e >> 2] >> ((e & 3) * 8)) & 0xFFu), sc);
    }
    uint4* out = reinterpret_cast<uint4*>(Wd + (int64_t)n * ldwd + k0);
    out[0] = make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
    out[1] = make_uint4(pack_bf16x2(v[8], v[9]), pack_bf16x2(v[10], v[11]), pack_bf16x2(v[12], v[13]), pack_bf16x2(v[14], v[15]));
}

// Outlier columns of the grad-input (Eq. 5: Xhat = X s^-1, so dX[:, O_i] = dXhat[:, O_i] / s_i), tolerance class (plain fp32):
//   dX[m][O_i] = bf16(((P1 - l) + P2) / s_i + l),   l = sum_j G[m][j] A[O_i][j]
// with P2 = P[m][nOp + i] = (dY wd)[m][i] and P1 = P[m][i] = (dY Wd)[m][O_i] + (lora_in_p1 ? the tensor cores' G A^T : 0).
// r is a multiple of 8: the rows of G and A are read as 128-bit words of 8 bf16
__global__ void bwd_fixup_kernel(const float* __restrict__ P, int64_t ldp, int M, int nO, int nOp,
                                 const int32_t* __restrict__ O_idx, const float* __restrict__ s_O,
                                 const uint16_t* __restrict__ G, const uint16_t* __restrict__ A, int r,
                                 uint16_t* __restrict__ dX, int64_t lddx, int lora_in_p1) {
    pdl_launch_dependents();
    pdl_wait();
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= M * nO) return;
    const int m = idx / nO, i = idx % nO;
    const int k = O_idx[i];
    float l = 0.0f;
    const uint4* g = reinterpret_cast<const uint4*>(G + (int64_t)m * r);
    const uint4* a = reinterpret_cast<const uint4*>(A + (int64_t)k * r);
    for (int j = 0; j < (r >> 3); ++j) {
        const uint4 gv = __ldg(g + j), av = __ldg(a + j);
        const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w}, aw[4] = {av.x, av.y, av.z, av.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            l = fmaf(bf16_lo(gw[e]), bf16_lo(aw[e]), l);
            l = fmaf(bf16_hi(gw[e]), bf16_hi(aw[e]), l);
        }
    }
    const float p1 = P[(int64_t)m * ldp + i] - (lora_in_p1 ? l : 0.0f);
    const float v = (p1 + P[(int64_t)m * ldp + nOp + i]) / s_O[i];
    dX[(int64_t)m * lddx + k] = (uint16_t)f32_to_bf16_bits(v + l);
}

static int pad16(int r) { return (r + 15) / 16 * 16; }

// Row tiles per band of the tile order: a band of the A operand (band x rows_per_tile rows of a_row_bytes) should
// stay in L2 while the column tiles sweep over it; at least enough row tiles to keep every CTA pair busy.
static int band_rows(int tiles_m, int tiles_n, int rows_per_tile, size_t a_row_bytes) {
    const size_t budget = 40u << 20;
    int b = (int)max((size_t)1, budget / max((size_t)1, (size_t)rows_per_tile * a_row_bytes));
    b = max(b, ceil_div(148 / 2, max(tiles_n, 1)));
    return min(b, max(tiles_m, 1));
}

constexpr int kPlanSMs = 148;   // split-K plans (and so workspace sizes) are fixed for the B200's 148 SMs

// Split-K plan of a skinny GEMM with `rows_out` output rows and a contraction of `kc` elements (bf16,
// 64 per k-block): as many splits as still run in ONE wave (a second, partial wave of split tiles costs more
// than shorter splits save), at least two k-blocks per split.
struct SplitPlan { int S, kblk; };
static SplitPlan split_plan(int rows_out, int kc) {
    const int tiles = max(1, ceil_div(rows_out, kTileM));   // an empty batch still gets a (never launched) plan
    const int nblk = max(1, ceil_div(kc, 64));
    int S = max(1, min(max(1, kPlanSMs / tiles), ceil_div(nblk, 2)));
    SplitPlan p;
    p.kblk = ceil_div(nblk, S);
    p.S = ceil_div(nblk, p.kblk);
    return p;
}
static size_t split_part_bytes(int rows_out, int kc, int r) {
    return (size_t)split_plan(rows_out, kc).S * rows_out * max(r, 1) * 4;
}

// One phase of a tile's contraction.  kext = contraction length in elements; box_k = contraction rows
// of an MN-major box (64 for a full k-block, less for a short LoRA contraction); ctas = CTAs per tile.
static void fill_phase(GemmPhase& ph, int is_i8, int kext, int acc_slot, int fresh, int tn_limit, int n_mma, int ctas,
                       int a_mn, int b_mn, int box_k, int b_per_tn) {
    const int kbox = is_i8 ? 128 : 64, kins = is_i8 ? 32 : 16;
    ph.nblk = ceil_div(kext, kbox);
    ph.is_i8 = is_i8;
    ph.nmma_last = ceil_div(kext - (ph.nblk - 1) * kbox, kins);
    ph.acc_slot = acc_slot;
    ph.fresh = fresh;
    ph.tn_limit = tn_limit;
    ph.a_mn = a_mn;
    ph.b_mn = b_mn;
    ph.n_mma = n_mma;
    const int b_cols = n_mma / ctas;                       // B extent per CTA
    ph.b_boxes = b_mn ? ceil_div(b_cols, 64) : 1;
    const uint32_t a_bytes = a_mn ? 2u * box_k * 128u : (uint32_t)kABytes;
    const uint32_t b_bytes = b_mn ? (uint32_t)ph.b_boxes * box_k * 128u : (uint32_t)b_cols * 128u;
    ph.tx_bytes = a_bytes + b_bytes;
    ph.kblk_per_tn = 0;
    ph.b_per_tn = b_per_tn;
}

// part[s][row][j] (f32, row pitch r) = sum over the s-th slice of the contraction of A(row, :) * B(j, :).
//   K-major  (mn_major = 0): A is [rows_out][kc] with pitch lda, B is [r][kc] with pitch ldb.
//   MN-major (mn_major = 1): A is [kc][rows_out] with pitch lda, B is [kc][r] with pitch ldb.
// skinny_prepare builds the launch parameters (tensor maps included; nothing is enqueued), skinny_launch enqueues.
struct SkinnyGemm { GemmParams p; int S; };
static quaff_status_t skinny_prepare(SkinnyGemm& g, int mn_major, const void* A, int64_t lda, const void* B, int64_t ldb, int rows_out,
                                     int kc, int r, float* part, int32_t* status) {
    const SplitPlan sp = split_plan(rows_out, kc);
    const int rp = pad16(r);
    GemmParams& p = g.p;
    memset(&p, 0, sizeof(p));
    GemmPhase& ph = p.ph[0];
    quaff_status_t rc;
    if (!mn_major) {
        if ((rc = make_tmap_2d(&ph.map_a, A, 2, rows_out, kc, lda, kTileM, 64)) != QUAFF_OK) return rc;
        if ((rc = make_tmap_2d(&ph.map_b, B, 2, r, kc, ldb, rp, 64)) != QUAFF_OK) return rc;
    } else {
        if ((rc = make_tmap_2d(&ph.map_a, A, 2, kc, rows_out, lda, 64, 64)) != QUAFF_OK) return rc;
        if ((rc = make_tmap_2d(&ph.map_b, B, 2, kc, r, ldb, 64, 64)) != QUAFF_OK) return rc;
    }
    fill_phase(ph, 0, 64, 0, 1, 1 << 30, rp, 1, mn_major, mn_major, 64, 0);
    ph.nblk = sp.kblk; ph.nmma_last = 4; ph.kblk_per_tn = sp.kblk;
    p.nphases = 1;
    p.M = rows_out; p.N = rp;
    p.tiles_m = ceil_div(rows_out, kTileM); p.tiles_n = sp.S;
    p.band_m = p.tiles_m;
    p.status = status;
    p.part = part; p.part_ld = r; p.part_cols = r;
    g.S = sp.S;
    return QUAFF_OK;
}
static quaff_status_t skinny_launch(const SkinnyGemm& g, cudaStream_t st) { return launch_gemm<EPI_PART, 1, 128>(g.p, st); }

static thread_local int g_force_fwd_tile = 0;   // quaff_debug_force_fwd_tile (per host thread): 0 = the cost model decides

// Cost model of the three forward kernels, fitted to sweeps of the number of waves at fixed shapes (B200, clocks of
// 1965 MHz): a tile of width W takes about  max(MMAs x kFwdMmaClk + kFwdTileOvh, kFwdTileMin)  clocks; the floor is
// the epilogue of a tile (stores of 16 bytes per row and instruction), which short contractions cannot hide.
constexpr int kFwdWidths[3] = {128, 192, 256};
constexpr double kFwdMmaClk[3] = {125.0, 157.0, 190.0};
constexpr double kFwdTileOvh[3] = {4100.0, 1500.0, 5000.0};
constexpr double kFwdTileMin[3] = {10900.0, 22500.0, 18700.0};
constexpr double kFwdTransposeClk = 7000.0;

struct FwdWorkspace { size_t off_bt, off_at, off_part, total; };
static FwdWorkspace fwd_workspace(int M, int K, int N, int r) {
    FwdWorkspace w;
    const int rp = pad16(max(r, 1));
    size_t off = 0;
    w.off_bt = off;   off += round_up((size_t)max(N, 1) * rp * 2, 256);  // B^T, K-major LoRA-up operand of the 192-column forward
    w.off_at = off;   off += round_up((size_t)rp * K * 2, 256);          // A^T, K-major LoRA-down operand
    w.off_part = off; off += round_up(split_part_bytes(M, K, r), 256);   // split-K partials of T = X A
    w.total = off;
    return w;
}

// ---- grad-input through a dequantized copy of the weight in the workspace (the faster of the two ways; see quaff.h)
static int round_up32(int k) { return (k + 31) / 32 * 32; }
static int bwd_tile_n_wd(int M, int K, int nOp) {
    const int units = kPlanSMs / 2;
    const int tm = ceil_div(M, 2 * kTileM);
    const int kext = nOp > 0 ? round_up32(K) + 2 * nOp : K;
    int best = 256;
    double best_cost = 0.0;
    for (int tn = 256; tn >= 128; tn -= 64) {
        const int tiles = tm * ceil_div(kext, tn);
        const double cost = (double)ceil_div(tiles, units) * (60.0 + 0.5 * tn);
        if (tn == 256 || cost < best_cost) { best = tn; best_cost = cost; }
    }
    return best;
}

struct BwdWdWorkspace {
    size_t off_wd, off_g, off_p, off_part, off_part_a, off_part_b, total;
    int tile_n;       // output-column tile of the grad-input GEMM
    int Kpad;         // K rounded up to 32: where the outlier columns start
    int64_t ldwd;     // row pitch of Wd in elements
};

static BwdWdWorkspace bwd_wd_workspace(int M, int K, int N, int nOp, int r) {
    BwdWdWorkspace w;
    w.tile_n = bwd_tile_n_wd(M, K, nOp);
    w.Kpad = round_up32(K);
    w.ldwd = (int64_t)w.Kpad + 2 * nOp;
    size_t off = 0;
    w.off_wd = off;   off += round_up((size_t)N * (size_t)w.ldwd * 2, 256);
    w.off_g = off;    off += round_up((size_t)M * (size_t)max(r, 1) * 2, 256);
    w.off_p = off;    off += round_up((size_t)M * (size_t)max(2 * nOp, 1) * 4, 256);
    // split-K partials: one buffer per skinny GEMM (they run concurrently)
    w.off_part = off;   off += round_up(split_part_bytes(M, N, r), 256);   // G = dY B^T
    w.off_part_a = off; off += round_up(split_part_bytes(K, M, r), 256);   // dA = X^T G
    w.off_part_b = off; off += round_up(split_part_bytes(N, M, r), 256);   // dB^T = dY^T T
    w.total = off;
    return w;
}


// ---- grad-input with the codes expanded inside the kernel (no copy of the weight)
// Output-column tile of the grad-input GEMM: 128, 192 or 256.  A tcgen05.mma of a CTA pair costs about 60 + N/2
// clocks (measured: N = 128: 125, 192: 165, 256: 190), so wide tiles are cheaper per column, while the width also
// decides how full the last wave is.  Cost model: waves on the CTA pairs x cost of one MMA of that width; among equals
// the wider tile (fewer tiles, fewer epilogues).  (Widths that are not a multiple of 64 run far below this model -
// measured: 176 columns 208 clocks per MMA, 240 columns 215 - so they are not candidates.)
static int bwd_tile_n(int M, int K, int nOp) {
    const int units = kPlanSMs / 2;
    const int tm = ceil_div(M, 2 * kTileM);
    int best = 256;
    double best_cost = 0.0;
    for (int tn = 256; tn >= 128; tn -= 64) {
        const int tiles = tm * (ceil_div(K, tn) + (nOp > 0 ? ceil_div(nOp, tn) : 0));      // main tiles + the tiles over the outlier rows
        const double cost = (double)ceil_div(tiles, units) * (60.0 + 0.5 * tn);
        if (tn == 256 || cost < best_cost) { best = tn; best_cost = cost; }
    }
    return best;
}

struct BwdLeanWorkspace {
    size_t off_g, off_p, off_part, off_part_a, off_part_b, total;
    int tile_n;       // output-column tile of the grad-input GEMM
};

static BwdLeanWorkspace bwd_lean_workspace(int M, int K, int N, int nOp, int r) {
    BwdLeanWorkspace w;
    w.tile_n = bwd_tile_n(M, K, nOp);
    size_t off = 0;
    // (no dequantized weight data: the grad-input GEMM expands the codes inside the kernel)
    w.off_g = off;    off += round_up((size_t)M * (size_t)max(r, 1) * 2, 256);
    w.off_p = off;    off += round_up((size_t)M * (size_t)max(2 * nOp, 1) * 4, 256);
    // split-K partials: one buffer per skinny GEMM (they run concurrently)
    w.off_part = off;   off += round_up(split_part_bytes(M, N, r), 256);   // G = dY B^T
    w.off_part_a = off; off += round_up(split_part_bytes(K, M, r), 256);   // dA = X^T G
    w.off_part_b = off; off += round_up(split_part_bytes(N, M, r), 256);   // dB^T = dY^T T
    w.total = off;
    return w;
}

// INT8 grad-input variant: the quantized gradient Zq [M][N], its step sizes, the dequantized outlier columns
// Wd_O [N][2 nOp] (the only bf16 weight data: the outlier columns stay on the floating-point path), G, P, split-K partials.
struct BwdInt8Workspace { size_t off_zq, off_dz, off_wdo, off_g, off_p, off_part, off_part_a, off_part_b, total; };
static BwdInt8Workspace bwd_int8_workspace(int M, int K, int N, int nOp, int r) {
    BwdInt8Workspace w;
    size_t off = 0;
    w.off_zq = off;   off += round_up((size_t)M * (size_t)N, 256);
    w.off_dz = off;   off += round_up((size_t)M * 4, 256);
    w.off_wdo = off;  off += round_up((size_t)N * (size_t)max(2 * nOp, 1) * 2, 256);
    w.off_g = off;    off += round_up((size_t)M * (size_t)max(r, 1) * 2, 256);
    w.off_p = off;    off += round_up((size_t)M * (size_t)max(2 * nOp, 1) * 4, 256);
    w.off_part = off;   off += round_up(split_part_bytes(M, N, r), 256);
    w.off_part_a = off; off += round_up(split_part_bytes(K, M, r), 256);
    w.off_part_b = off; off += round_up(split_part_bytes(N, M, r), 256);
    w.total = off;
    return w;
}

// T = bf16(X A): At = A^T (K-major operand), split-K tensor-core GEMM over K, reduction to bf16
static quaff_status_t lora_down(const quaff_bf16* X, int64_t ldx, int M, int K, const quaff_bf16* A, int r, quaff_bf16* T_out,
                                const FwdWorkspace& w, void* ws, int32_t* status_opt, cudaStream_t st) {
    unsigned char* base = reinterpret_cast<unsigned char*>(ws);
    uint16_t* At = reinterpret_cast<uint16_t*>(base + w.off_at);
    float* part = reinterpret_cast<float*>(base + w.off_part);
    const int rp = pad16(r);
    quaff_status_t rc;
    SkinnyGemm g;
    if ((rc = skinny_prepare(g, 0, X, ldx, At, K, M, K, r, part, status_opt)) != QUAFF_OK) return rc;
    launch_pdl(transpose_pad_kernel, dim3(ceil_div(K * rp, 256)), dim3(256), 0, st, 1, A, K, r, At, K);   // At[j][k] = A[k][j]
    if ((rc = launch_status()) != QUAFF_OK) return rc;
    if ((rc = skinny_launch(g, st)) != QUAFF_OK) return rc;
    launch_pdl(reduce_parts_bf16_kernel, dim3(ceil_div(M * r / 8, 256)), dim3(256), 0, st, 1, part, g.S, M, r, 1.0f, T_out);
    return launch_status();
}

// The backward of an empty batch: nothing to write to dX; the sums dA = X^T G and dB = T^T dY over no tokens are zero,
// which a call that does not accumulate has to store.
static quaff_status_t empty_batch_grads(int K, int N, int r, float* dA, float* dB, int accumulate, cudaStream_t st) {
    if (r <= 0 || !dA || accumulate) return QUAFF_OK;
    if (cudaMemsetAsync(dA, 0, (size_t)K * r * 4, st) != cudaSuccess) return QUAFF_ERR_CUDA;
    if (cudaMemsetAsync(dB, 0, (size_t)r * N * 4, st) != cudaSuccess) return QUAFF_ERR_CUDA;
    return QUAFF_OK;
}

}  // namespace quaff

using namespace quaff;

extern "C" quaff_status_t quaff_lora_down(const quaff_bf16* X, int64_t ldx, int M, int K, const quaff_bf16* A, int r,
                                          quaff_bf16* T_out, int32_t* status_opt, void* ws, size_t ws_bytes,
                                          quaff_stream_t stream) {
    QUAFF_RETURN_IF(M < 0 || K <= 0 || r <= 0 || !X || !A || !T_out || ldx < K, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF((r % 8) || r > 64 || (K % 8), QUAFF_ERR_UNSUPPORTED_SHAPE);
    QUAFF_RETURN_IF(!aligned16(X) || !aligned16(T_out) || (ldx % 8), QUAFF_ERR_ALIGNMENT);
    const FwdWorkspace w = fwd_workspace(M, K, 0, r);
    QUAFF_RETURN_IF(!ws || !aligned16(ws) || ws_bytes < w.total, QUAFF_ERR_WORKSPACE_TOO_SMALL);
    if (M == 0) return QUAFF_OK;
    return lora_down(X, ldx, M, K, A, r, T_out, w, ws, status_opt, (cudaStream_t)stream);
}

extern "C" uint64_t quaff_debug_launch_count(void) { return g_launch_count; }

extern "C" void quaff_debug_force_fwd_tile(int tile_n) { g_force_fwd_tile = tile_n; }

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
        case QUAFF_WS_FWD: return fwd_workspace(M, K, N, r).total;
        case QUAFF_WS_BWD: return max(bwd_wd_workspace(M, K, N, nOp, r).total, bwd_lean_workspace(M, K, N, nOp, r).total);
        case QUAFF_WS_BWD_LEAN: return bwd_lean_workspace(M, K, N, nOp, r).total;
        case QUAFF_WS_BWD_INT8: return bwd_int8_workspace(M, K, N, nOp, r).total;
        case QUAFF_WS_CALIBRATE: return round_up((size_t)max(K, 0) * 4, 256) + 256;   // column maxima / flags, sum, ticket
        case QUAFF_WS_HITS: return 2 * round_up((size_t)max(K, 0) * 4, 256) + 256;    // the same, then this batch's indicator
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
    const bool have_T = r > 0 && !X;      // T_out already holds T = bf16(X A) (quaff_lora_down)
    QUAFF_RETURN_IF(r > 0 && (!B || !T_out), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(r > 0 && !have_T && (!A || ldx < K), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(y_dtype != QUAFF_BF16 && y_dtype != QUAFF_F32, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF((nOp % 32) || (r % 8) || r > 64, QUAFF_ERR_UNSUPPORTED_SHAPE);
    QUAFF_RETURN_IF(r > 0 && ((K % 8) || (N % 8)), QUAFF_ERR_UNSUPPORTED_SHAPE);
    QUAFF_RETURN_IF(!aligned16(Xq) || !aligned16(Wq) || (ldxq % 16) || (ldwq_main % 16), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(nOp > 0 && (!aligned16(xq_O) || !aligned16(wq_O) || (ldxo % 16) || (ldwq % 16)), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(r > 0 && (!aligned16(T_out) || !aligned16(B)), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(r > 0 && !have_T && (!aligned16(X) || (ldx % 8)), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(!aligned16(Y), QUAFF_ERR_ALIGNMENT);
    const FwdWorkspace w = fwd_workspace(M, K, N, r);
    QUAFF_RETURN_IF(r > 0 && (!ws || !aligned16(ws) || ws_bytes < w.total), QUAFF_ERR_WORKSPACE_TOO_SMALL);
    if (M == 0) return QUAFF_OK;
    cudaStream_t st = (cudaStream_t)stream;
    const int rp = pad16(r);
    constexpr int CTAS = 2;
    // Eq. 2 alone (no outlier set, no LoRA) takes 256-column tiles.  With the two short contractions there are
    // three kernels: 128-column tiles with all three accumulators resident in TMEM (umma_gemm.cuh), 192-column
    // tiles with the short accumulators in rounds of 64 columns (fwd192.cuh), 256-column tiles with a single main
    // accumulator that the epilogue copies out at once and rounds of 128 columns (fwd256.cuh).  A tcgen05.mma
    // costs about 60 + N/2 clocks, so the wide tiles are cheaper per column; each kernel has its own overhead per
    // tile (ring stages of the rounds, hand-shakes, the wait for the accumulator).  The host takes the variant with
    // the smallest  waves x time per tile  (cost model above).  The rounds need an outlier round to be one k-block
    // (nOp <= 128).
    const int tiles_m2 = ceil_div(M, 2 * kTileM), pairs = kPlanSMs / 2;
    int wide = 0;     // 0: 128-column tiles, else the tile width of the wide kernel
    if ((nOp > 0 || r > 0) && nOp <= 128) {
        const double nmma = ceil_div(K, 32);
        double best = 0.0;
        for (int i = 0; i < 3; ++i) {
            const double tile = fmax(nmma * kFwdMmaClk[i] + kFwdTileOvh[i], kFwdTileMin[i]);
            // (the 192-column kernel wants LoRA B transposed: one more small kernel in front of it)
            const double cost = (double)ceil_div(tiles_m2 * ceil_div(N, kFwdWidths[i]), pairs) * tile + ((i == 1 && r > 0) ? kFwdTransposeClk : 0.0);
            if (i == 0 || cost < best) { best = cost; wide = i == 0 ? 0 : kFwdWidths[i]; }
        }
        if (g_force_fwd_tile == 128) wide = 0;
        if (g_force_fwd_tile == 192 || g_force_fwd_tile == 256) wide = g_force_fwd_tile;
    }
    if (wide) {
        const int WTN = wide, WR = wide == 256 ? kF256Round : kF192Round;
        FwdWideParams q;
        memset(&q, 0, sizeof(q));
        quaff_status_t rc;
        if ((rc = make_tmap_2d(&q.map_xq, Xq, 1, M, K, ldxq, kTileM, 128)) != QUAFF_OK) return rc;
        if ((rc = make_tmap_2d(&q.map_wq, Wq, 1, N, K, ldwq_main, WTN / 2, 128)) != QUAFF_OK) return rc;
        q.nblk = ceil_div(K, 128);
        q.nmma_last = ceil_div(K - (q.nblk - 1) * 128, 32);
        if (nOp > 0) {
            if ((rc = make_tmap_2d(&q.map_xo, xq_O, 1, M, nOp, ldxo, kTileM, 128)) != QUAFF_OK) return rc;
            if ((rc = make_tmap_2d(&q.map_wo, wq_O, 1, N, nOp, ldwq, WR / 2, 128)) != QUAFF_OK) return rc;
            q.nmma_o = nOp / 32;
        }
        if (r > 0) {
            if (!have_T && (rc = lora_down(X, ldx, M, K, A, r, T_out, w, ws, status_opt, st)) != QUAFF_OK) return rc;
            if ((rc = make_tmap_2d(&q.map_t, T_out, 2, M, r, r, kTileM, 64)) != QUAFF_OK) return rc;
            if (wide == 256) {   // B [r][N] is read in place as an MN-major operand (rows = contraction)
                if ((rc = make_tmap_2d(&q.map_bt, B, 2, r, N, N, rp, 64)) != QUAFF_OK) return rc;
            } else {             // rounds of 64 columns, 32 per CTA: K-major copy Bt[n][j] = B[j][n]
                uint16_t* Bt = reinterpret_cast<uint16_t*>(reinterpret_cast<unsigned char*>(ws) + w.off_bt);
                launch_pdl(transpose_pad_kernel, dim3(ceil_div(N * rp, 256)), dim3(256), 0, st, 1, B, r, N, Bt, rp);
                if ((rc = launch_status()) != QUAFF_OK) return rc;
                if ((rc = make_tmap_2d(&q.map_bt, Bt, 2, N, rp, rp, WR / 2, 64)) != QUAFF_OK) return rc;
            }
            q.nmma_l = rp / 16;
        }
        q.M = M; q.N = N;
        q.tiles_m = ceil_div(M, 2 * kTileM); q.tiles_n = ceil_div(N, WTN);
        q.band_m = band_rows(q.tiles_m, q.tiles_n, 2 * kTileM, (size_t)K);
        q.status = status_opt;
        q.dx = dx; q.dW = dW; q.dw_O = dw_O; q.lora_scale = lora_scale;
        q.Y = Y; q.ldy = ldy; q.y_f32 = (y_dtype == QUAFF_F32);
        q.dbg_main = dbg_acc_main; q.dbg_out = dbg_acc_out;
        return launch_fwd_wide(wide == 256 ? 1 : 0, q, st);
    }
    const int TN = (nOp == 0 && r == 0) ? 256 : 128;

    GemmParams p;
    memset(&p, 0, sizeof(p));
    quaff_status_t rc;
    int np = 0;
    {   // main: acc1 = Xq Wq^T over K
        GemmPhase& ph = p.ph[np++];
        if ((rc = make_tmap_2d(&ph.map_a, Xq, 1, M, K, ldxq, kTileM, 128)) != QUAFF_OK) return rc;
        if ((rc = make_tmap_2d(&ph.map_b, Wq, 1, N, K, ldwq_main, TN / CTAS, 128)) != QUAFF_OK) return rc;
        fill_phase(ph, 1, K, 0, 1, 1 << 30, TN, CTAS, 0, 0, 64, TN);
    }
    if (nOp > 0) {   // outlier: acc2 = xq_O wq_O^T over nOp
        GemmPhase& ph = p.ph[np++];
        if ((rc = make_tmap_2d(&ph.map_a, xq_O, 1, M, nOp, ldxo, kTileM, 128)) != QUAFF_OK) return rc;
        if ((rc = make_tmap_2d(&ph.map_b, wq_O, 1, N, nOp, ldwq, TN / CTAS, 128)) != QUAFF_OK) return rc;
        fill_phase(ph, 1, nOp, 1, 1, 1 << 30, TN, CTAS, 0, 0, 64, TN);
    }
    if (r > 0) {
        // LoRA down-projection T = bf16(X A), unless the caller has run it already
        if (!have_T && (rc = lora_down(X, ldx, M, K, A, r, T_out, w, ws, status_opt, st)) != QUAFF_OK) return rc;
        // LoRA up: acc3 = T B over r; B [r][N] is read in place as an MN-major operand (rows = contraction)
        GemmPhase& ph = p.ph[np++];
        if ((rc = make_tmap_2d(&ph.map_a, T_out, 2, M, r, r, kTileM, 64)) != QUAFF_OK) return rc;
        if ((rc = make_tmap_2d(&ph.map_b, B, 2, r, N, N, rp, 64)) != QUAFF_OK) return rc;
        fill_phase(ph, 0, rp, 2, 1, 1 << 30, TN, CTAS, 0, 1, rp, TN);
    }
    p.nphases = np;
    p.M = M; p.N = N;
    p.tiles_m = ceil_div(M, kTileM * CTAS); p.tiles_n = ceil_div(N, TN);
    p.band_m = band_rows(p.tiles_m, p.tiles_n, kTileM * CTAS, (size_t)K);
    p.status = status_opt;
    p.dx = dx; p.dW = dW; p.dw_O = dw_O; p.lora_scale = lora_scale;
    p.has_outlier = nOp > 0; p.has_lora = r > 0;
    p.Y = Y; p.ldy = ldy; p.y_f32 = (y_dtype == QUAFF_F32);
    p.dbg_main = dbg_acc_main; p.dbg_out = dbg_acc_out;
    return TN == 256 ? launch_gemm<EPI_FWD, CTAS, 256>(p, st) : launch_gemm<EPI_FWD, CTAS, 128>(p, st);
}

// quaff_qlinear_bwd with a dequantized copy of the weight in the workspace (arguments validated by the caller)
static quaff_status_t bwd_through_copy(int M, int K, int N, const quaff_bf16* dY, int64_t lddy, const int8_t* Wq,
                                       int64_t ldwq_main, const float* dW, const int8_t* wq_O, int64_t ldwq,
                                       const float* dw_O, int nOp, const int32_t* O_idx, int nO, const float* s_O,
                                       const quaff_bf16* X, int64_t ldx, const quaff_bf16* T, const quaff_bf16* A,
                                       const quaff_bf16* B, int r, float lora_scale, quaff_bf16* dX, int64_t lddx,
                                       float* dA, float* dB, int accumulate, quaff_bf16* G_out_opt,
                                       int32_t* status_opt, void* ws, cudaStream_t st) {
    const BwdWdWorkspace w = bwd_wd_workspace(M, K, N, nOp, r);
    unsigned char* base = reinterpret_cast<unsigned char*>(ws);
    uint16_t* Wd = reinterpret_cast<uint16_t*>(base + w.off_wd);
    uint16_t* G = (r > 0 && G_out_opt) ? G_out_opt : reinterpret_cast<uint16_t*>(base + w.off_g);
    float* P = reinterpret_cast<float*>(base + w.off_p);
    float* part = reinterpret_cast<float*>(base + w.off_part);
    float* part_a = reinterpret_cast<float*>(base + w.off_part_a);
    float* part_b = reinterpret_cast<float*>(base + w.off_part_b);
    quaff_status_t rc;
    const bool want_dAB = r > 0 && dA && dB;
    constexpr int CTAS = 2;
    const int TN = w.tile_n, Kpad = w.Kpad;
    const int Kext = nOp > 0 ? Kpad + 2 * nOp : K;

    // ---- every tensor map and launch parameter first: nothing has been enqueued when one of them fails
    SkinnyGemm gemm_g, gemm_db, gemm_da;
    GemmParams p;
    if (r > 0) {   // G = bf16(lora_scale * dY B^T): B [r][N] is already K-major for this contraction over N
        if ((rc = skinny_prepare(gemm_g, 0, dY, lddy, B, N, M, N, r, part, status_opt)) != QUAFF_OK) return rc;
    }
    if (dX) {
        memset(&p, 0, sizeof(p));
        int np = 0;
        {   // main: dY Wd over N; Wd [N][Kext] is MN-major for this contraction (rows = n)
            GemmPhase& ph = p.ph[np++];
            if ((rc = make_tmap_2d(&ph.map_a, dY, 2, M, N, lddy, kTileM, 64)) != QUAFF_OK) return rc;
            if ((rc = make_tmap_2d(&ph.map_b, Wd, 2, N, Kext, w.ldwd, 64, 64)) != QUAFF_OK) return rc;
            fill_phase(ph, 0, N, 0, 1, 1 << 30, TN, CTAS, 0, 1, 64, TN);
        }
        if (r > 0) {   // + G A^T over r, only for the real dX columns
            GemmPhase& ph = p.ph[np++];
            if ((rc = make_tmap_2d(&ph.map_a, G, 2, M, r, r, kTileM, 64)) != QUAFF_OK) return rc;
            if ((rc = make_tmap_2d(&ph.map_b, A, 2, K, r, r, TN / CTAS, 64)) != QUAFF_OK) return rc;
            fill_phase(ph, 0, pad16(r), 0, 0, ceil_div(K, TN), TN, CTAS, 0, 0, 64, TN);
        }
        p.nphases = np;
        p.M = M;
        // columns [0,K) -> dX; the outlier partial products start at Kpad (K rounded up to 32), inside whatever tile that is:
        // the LoRA phase of that tile adds nothing to them (rows of A beyond K read as zeros)
        p.n_split = K;
        p.p_col0 = Kpad;
        p.N = Kext;
        p.tiles_m = ceil_div(M, kTileM * CTAS);
        p.tiles_n = ceil_div(p.N, TN);
        p.band_m = band_rows(p.tiles_m, p.tiles_n, kTileM * CTAS, (size_t)N * 2);
        p.status = status_opt;
        p.dX = dX; p.lddx = lddx; p.P = P; p.ldp = 2 * nOp;
        p.tile_n = TN;      // the 256-column instance serves every width above 128
    }
    if (want_dAB) {
        // dB^T = dY^T T and dA = X^T G: the contraction runs over the tokens, the slow axis of all four matrices: MN-major operands
        if ((rc = skinny_prepare(gemm_db, 1, dY, lddy, T, r, N, M, r, part_b, status_opt)) != QUAFF_OK) return rc;
        if ((rc = skinny_prepare(gemm_da, 1, X, ldx, G, r, K, M, r, part_a, status_opt)) != QUAFF_OK) return rc;
    }

    // Dependencies:  dB = T^T dY needs nothing computed here;  the weight dequantization neither;
    // G = dY B^T feeds the grad-input GEMM and dA = X^T G;  the outlier fix-up follows the GEMM.
    DeviceSide* ds = device_side();
    std::unique_lock<std::mutex> lock;
    SideSet* ss = nullptr;
    if (ds) {
        lock = std::unique_lock<std::mutex>(ds->mu);
        ss = pick_side_set(ds, st);
    }
    cudaStream_t s_deq = ss ? ss->s[0] : st;       // dequantization, later dA
    cudaStream_t s_db = ss ? ss->s[1] : st;        // dB
    bool forked0 = false, forked1 = false;
    // From the first fork on, an error leaves through `leave`: whatever has been forked is joined back into the
    // caller's stream, so that no branch stays open (a stream capture would otherwise be invalid, and a caller could
    // reuse the workspace while a side stream still writes it).
    auto leave = [&](quaff_status_t code) {
        if (forked0 && !join_from(ss, 0, st) && code == QUAFF_OK) code = QUAFF_ERR_CUDA;
        if (forked1 && !join_from(ss, 1, st) && code == QUAFF_OK) code = QUAFF_ERR_CUDA;
        return code;
    };

    // Launch order = the order in which the block scheduler hands out SM slots while everything below runs at once:
    // the chain the grad-input GEMM waits for longest (G) first, then the bulk dequantization; dB and dA come behind
    // the GEMM.  The side streams fork off before any of it, so that they depend on nothing launched here.
    if (ss && want_dAB && !(forked1 = fork_to(ss, 1, st))) return leave(QUAFF_ERR_CUDA);
    if (ss && dX && !(forked0 = fork_to(ss, 0, st))) return leave(QUAFF_ERR_CUDA);
    if (r > 0) {
        if ((rc = skinny_launch(gemm_g, st)) != QUAFF_OK) return leave(rc);
        launch_pdl(reduce_parts_bf16_kernel, dim3(ceil_div(M * r / 8, 256)), dim3(256), 0, st, 1, part, gemm_g.S, M, r, lora_scale, G);
        if ((rc = launch_status()) != QUAFF_OK) return leave(rc);
        if (ss && cudaEventRecord(ss->g_ready, st) != cudaSuccess) return leave(QUAFF_ERR_CUDA);
    }
    if (dX) {
        const int chunks = (Kpad + 2 * nOp) / 16;
        launch_pdl(dequant_weight_kernel, dim3(N, ceil_div(chunks, 256)), dim3(256), 0, s_deq, 1, Wq, ldwq_main, dW, wq_O, ldwq, dw_O, O_idx,
                   nO, nOp, K, Kpad, Wd, w.ldwd);
        if ((rc = launch_status()) != QUAFF_OK) return leave(rc);
        if (forked0) {     // the dequantized weight is ready
            forked0 = false;
            if (!join_from(ss, 0, st)) return leave(QUAFF_ERR_CUDA);
        }
        rc = TN > 128 ? launch_gemm<EPI_BWD, CTAS, 256>(p, st) : launch_gemm<EPI_BWD, CTAS, 128>(p, st);
        if (rc != QUAFF_OK) return leave(rc);
    }
    if (want_dAB) {
        // dB needs nothing computed here, but it is held back (side stream 1 waits for the end of the dequantization) until the
        // grad-input GEMM is ready too and enqueued behind it: with the lowest priority it then runs in the SMs the GEMM
        // leaves free instead of competing with G and the dequantization for HBM in front of the GEMM.
        if (ss && dX && cudaStreamWaitEvent(ss->s[1], ss->join[0], 0) != cudaSuccess) return leave(QUAFF_ERR_CUDA);
        if ((rc = skinny_launch(gemm_db, s_db)) != QUAFF_OK) return leave(rc);
        launch_pdl(reduce_parts_kernel, dim3(ceil_div(N * r / 4, 256)), dim3(256), 0, s_db, 1, part_b, gemm_db.S, N, r, lora_scale, 1, accumulate, dB);
        if ((rc = launch_status()) != QUAFF_OK) return leave(rc);
        // dA needs G, not the grad-input GEMM: on side stream 0 it follows the weight dequantization and waits for G
        // only.  It is enqueued BEHIND the GEMM, so the persistent GEMM gets every SM first and the split-K CTAs of dA
        // move in as the pairs that have no tile left in the last wave retire.
        cudaStream_t s_da = st;
        if (ss && dX) {
            if (cudaStreamWaitEvent(ss->s[0], ss->g_ready, 0) != cudaSuccess) return leave(QUAFF_ERR_CUDA);
            forked0 = true;
            s_da = ss->s[0];
        }
        if ((rc = skinny_launch(gemm_da, s_da)) != QUAFF_OK) return leave(rc);
        launch_pdl(reduce_parts_kernel, dim3(ceil_div(K * r / 4, 256)), dim3(256), 0, s_da, 1, part_a, gemm_da.S, K, r, 1.0f, 0, accumulate, dA);
        if ((rc = launch_status()) != QUAFF_OK) return leave(rc);
    }
    if (dX && nO > 0) {
        launch_pdl(bwd_fixup_kernel, dim3(ceil_div(M * nO, 256)), dim3(256), 0, st, 1, P, (int64_t)(2 * nOp), M, nO, nOp, O_idx, s_O, G, A, r,
                   dX, lddx, 0);
        if ((rc = launch_status()) != QUAFF_OK) return leave(rc);
    }
    return leave(QUAFF_OK);
}


extern "C" quaff_status_t quaff_qlinear_bwd(int M, int K, int N, const quaff_bf16* dY, int64_t lddy, const int8_t* Wq,
                                            int64_t ldwq_main, const float* dW, const int8_t* wq_O, int64_t ldwq,
                                            const float* dw_O, int nOp, const int32_t* O_idx, int nO, const float* s_O,
                                            const quaff_bf16* X, int64_t ldx, const quaff_bf16* T, const quaff_bf16* A,
                                            const quaff_bf16* B, int r, float lora_scale, quaff_bf16* dX, int64_t lddx,
                                            float* dA, float* dB, int accumulate, quaff_bf16* G_out_opt,
                                            int32_t* status_opt, void* ws, size_t ws_bytes, quaff_stream_t stream) {
    QUAFF_RETURN_IF(M < 0 || K <= 0 || N <= 0 || nOp < 0 || nO < 0 || nO > nOp || r < 0, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(!dY || lddy < N || !Wq || !dW || ldwq_main < K, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(nOp > 0 && (!wq_O || !dw_O || ldwq < nOp), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(nO > 0 && (!O_idx || !s_O), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(r > 0 && (!A || !B), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(r > 0 && (dA || dB) && (!dA || !dB || !X || !T || ldx < K), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(dX && lddx < K, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF((nOp % 32) || (r % 8) || r > 64, QUAFF_ERR_UNSUPPORTED_SHAPE);
    QUAFF_RETURN_IF(r > 0 && (N % 8), QUAFF_ERR_UNSUPPORTED_SHAPE);
    QUAFF_RETURN_IF(!aligned16(dY) || (lddy % 8), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(!aligned16(Wq) || (ldwq_main % 16), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(nOp > 0 && (!aligned16(wq_O) || (ldwq % 16)), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(dX && (!aligned16(dX) || (lddx % 8)), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(r > 0 && (!aligned16(A) || !aligned16(B) || (G_out_opt && !aligned16(G_out_opt))), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(r > 0 && dA && (!aligned16(X) || !aligned16(T) || !aligned16(dA) || !aligned16(dB) || (ldx % 8)), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(nO > 0 && K > 32768, QUAFF_ERR_UNSUPPORTED_SHAPE);      // the per-column outlier mask lives in shared memory
    QUAFF_RETURN_IF(!aligned16(dW) || (nOp > 0 && !aligned16(dw_O)), QUAFF_ERR_ALIGNMENT);
    const BwdLeanWorkspace w = bwd_lean_workspace(M, K, N, nOp, r);
    QUAFF_RETURN_IF(!ws || !aligned16(ws) || ws_bytes < w.total, QUAFF_ERR_WORKSPACE_TOO_SMALL);
    if (M == 0) return empty_batch_grads(K, N, r, dA, dB, accumulate, (cudaStream_t)stream);
    cudaStream_t st = (cudaStream_t)stream;
    // Two ways through the frozen INT8 weight, the same products in the same order either way (dX is bit-identical off the
    // outlier columns): with room for a transient bf16 copy of the weight in the workspace (QUAFF_WS_BWD bytes) the copy is
    // made and read by TMA, which is the faster way; with QUAFF_WS_BWD_LEAN bytes the codes are expanded inside the GEMM.
    if (dX && ws_bytes >= bwd_wd_workspace(M, K, N, nOp, r).total)
        return bwd_through_copy(M, K, N, dY, lddy, Wq, ldwq_main, dW, wq_O, ldwq, dw_O, nOp, O_idx, nO, s_O, X, ldx, T, A, B, r, lora_scale, dX,
                                lddx, dA, dB, accumulate, G_out_opt, status_opt, ws, st);
    unsigned char* base = reinterpret_cast<unsigned char*>(ws);
    uint16_t* G = (r > 0 && G_out_opt) ? G_out_opt : reinterpret_cast<uint16_t*>(base + w.off_g);
    float* P = reinterpret_cast<float*>(base + w.off_p);
    float* part = reinterpret_cast<float*>(base + w.off_part);
    float* part_a = reinterpret_cast<float*>(base + w.off_part_a);
    float* part_b = reinterpret_cast<float*>(base + w.off_part_b);
    quaff_status_t rc;
    const bool want_dAB = r > 0 && dA && dB;
    const int TN = w.tile_n;

    // ---- every tensor map and launch parameter first: nothing has been enqueued when one of them fails
    SkinnyGemm gemm_g, gemm_db, gemm_da;
    BxParams p;
    if (r > 0) {   // G = bf16(lora_scale * dY B^T): B [r][N] is already K-major for this contraction over N
        if ((rc = skinny_prepare(gemm_g, 0, dY, lddy, B, N, M, N, r, part, status_opt)) != QUAFF_OK) return rc;
    }
    if (dX) {
        memset(&p, 0, sizeof(p));
        if ((rc = make_tmap_2d(&p.map_dy, dY, 2, M, N, lddy, kTileM, 64)) != QUAFF_OK) return rc;
        // the codes in their stored orientation, the contraction index n as the row: boxes of 64 rows x 128 codes
        if ((rc = make_tmap_2d(&p.map_wq, Wq, 1, N, K, ldwq_main, 64, 128)) != QUAFF_OK) return rc;
        if (nO > 0) {   // the re-quantized outlier rows, likewise: wd = bf16(wq_O dw_O) is formed inside the kernel
            if ((rc = make_tmap_2d(&p.map_wo, wq_O, 1, N, nOp, ldwq, 64, 128)) != QUAFF_OK) return rc;
        }
        if (r > 0) {
            if ((rc = make_tmap_2d(&p.map_g, G, 2, M, r, r, kTileM, 64)) != QUAFF_OK) return rc;
            if ((rc = make_tmap_2d(&p.map_a, A, 2, K, r, r, TN / 2, 64)) != QUAFF_OK) return rc;
            p.nmma_l = pad16(r) / 16;
        }
        p.M = M; p.N = N; p.K = K;
        p.nblk = ceil_div(N, 64);
        p.nmma_last = ceil_div(N - (p.nblk - 1) * 64, 16);
        p.tile_n = TN;
        p.tile_np = (nO > 0 && nOp > 128) ? 256 : 128;    // each CTA supplies whole boxes of 64 columns
        p.tiles_m = ceil_div(M, 2 * kTileM);
        p.tiles_main = ceil_div(K, TN);
        p.tiles_p = nO > 0 ? ceil_div(nOp, p.tile_np) : 0;
        p.band_m = band_rows(p.tiles_m, p.tiles_main + p.tiles_p, 2 * kTileM, (size_t)N * 2);
        p.nO = nO; p.nOp = nOp;
        p.mask_words = nO > 0 ? ceil_div(K, 32) : 0;
        p.nstages = bx_stages(p.mask_words);
        p.dW = dW; p.dw_O = dw_O; p.O_idx = O_idx;
        p.dX = dX; p.lddx = lddx; p.P = P;
        p.status = status_opt;
    }
    if (want_dAB) {
        // dB^T = dY^T T and dA = X^T G: the contraction runs over the tokens, the slow axis of all four matrices: MN-major operands
        if ((rc = skinny_prepare(gemm_db, 1, dY, lddy, T, r, N, M, r, part_b, status_opt)) != QUAFF_OK) return rc;
        if ((rc = skinny_prepare(gemm_da, 1, X, ldx, G, r, K, M, r, part_a, status_opt)) != QUAFF_OK) return rc;
    }

    // Dependencies:  G = dY B^T feeds the grad-input GEMM and dA = X^T G;  dB = T^T dY needs nothing computed here;
    // the outlier fix-up follows the GEMM.
    DeviceSide* ds = device_side();
    std::unique_lock<std::mutex> lock;
    SideSet* ss = nullptr;
    if (ds) {
        lock = std::unique_lock<std::mutex>(ds->mu);
        ss = pick_side_set(ds, st);
    }
    bool forked0 = false, forked1 = false;
    // From the first fork on, an error leaves through `leave`: whatever has been forked is joined back into the
    // caller's stream, so that no branch stays open (a stream capture would otherwise be invalid, and a caller could
    // reuse the workspace while a side stream still writes it).
    auto leave = [&](quaff_status_t code) {
        if (forked0 && !join_from(ss, 0, st) && code == QUAFF_OK) code = QUAFF_ERR_CUDA;
        if (forked1 && !join_from(ss, 1, st) && code == QUAFF_OK) code = QUAFF_ERR_CUDA;
        return code;
    };

    if (r > 0) {
        if ((rc = skinny_launch(gemm_g, st)) != QUAFF_OK) return leave(rc);
        launch_pdl(reduce_parts_bf16_kernel, dim3(ceil_div(M * r / 8, 256)), dim3(256), 0, st, 1, part, gemm_g.S, M, r, lora_scale, G);
        if ((rc = launch_status()) != QUAFF_OK) return leave(rc);
        if (ss && cudaEventRecord(ss->g_ready, st) != cudaSuccess) return leave(QUAFF_ERR_CUDA);
    }
    if (dX && (rc = launch_bwd_expand(p, st)) != QUAFF_OK) return leave(rc);
    if (want_dAB) {
        // dB and dA go to the side streams, behind G (dA needs it; dB needs nothing, but is held back as long, so that it does
        // not compete with G for HBM in front of the GEMM).  Launch order = the order in which the block scheduler hands out
        // SM slots: both are enqueued BEHIND the grad-input GEMM, which they do not depend on, so the persistent GEMM gets every
        // SM first and the split-K CTAs of dB and dA (lowest priority) move in as the pairs that have no tile left in the last
        // wave retire.
        cudaStream_t s_db = st, s_da = st;
        if (ss) {
            if (cudaStreamWaitEvent(ss->s[1], ss->g_ready, 0) != cudaSuccess) return leave(QUAFF_ERR_CUDA);
            forked1 = true;
            s_db = ss->s[1];
        }
        if ((rc = skinny_launch(gemm_db, s_db)) != QUAFF_OK) return leave(rc);
        launch_pdl(reduce_parts_kernel, dim3(ceil_div(N * r / 4, 256)), dim3(256), 0, s_db, 1, part_b, gemm_db.S, N, r, lora_scale, 1, accumulate, dB);
        if ((rc = launch_status()) != QUAFF_OK) return leave(rc);
        if (ss) {
            if (cudaStreamWaitEvent(ss->s[0], ss->g_ready, 0) != cudaSuccess) return leave(QUAFF_ERR_CUDA);
            forked0 = true;
            s_da = ss->s[0];
        }
        if ((rc = skinny_launch(gemm_da, s_da)) != QUAFF_OK) return leave(rc);
        launch_pdl(reduce_parts_kernel, dim3(ceil_div(K * r / 4, 256)), dim3(256), 0, s_da, 1, part_a, gemm_da.S, K, r, 1.0f, 0, accumulate, dA);
        if ((rc = launch_status()) != QUAFF_OK) return leave(rc);
    }
    if (dX && nO > 0) {
        launch_pdl(bwd_fixup_kernel, dim3(ceil_div(M * nO, 256)), dim3(256), 0, st, 1, P, (int64_t)(2 * nOp), M, nO, nOp, O_idx, s_O, G, A, r,
                   dX, lddx, 1);     // P1 was copied out of the accumulator: it contains G A^T
        if ((rc = launch_status()) != QUAFF_OK) return leave(rc);
    }
    return leave(QUAFF_OK);
}

// The INT8 grad-input variant (not the paper's method; see quaff.h).  Kernels: quant_grad (Z = dY Delta_W quantized per
// token), the 256-column INT8 kernel of the forward with the frozen codes Wq [N][K] read in place as an MN-major operand
// (contraction over N) and G A^T in its LoRA rounds, and - for the nO outlier columns only - the floating-point path of
// quaff_qlinear_bwd on the dequantized outlier columns (a grad-input GEMM with 2 nOp output columns, then the fix-up).
extern "C" quaff_status_t quaff_qlinear_bwd_int8(int M, int K, int N, const quaff_bf16* dY, int64_t lddy, const int8_t* Wq,
                                                 int64_t ldwq_main, const float* dW, const int8_t* wq_O, int64_t ldwq,
                                                 const float* dw_O, int nOp, const int32_t* O_idx, int nO, const float* s_O,
                                                 const quaff_bf16* X, int64_t ldx, const quaff_bf16* T, const quaff_bf16* A,
                                                 const quaff_bf16* B, int r, float lora_scale, quaff_bf16* dX, int64_t lddx,
                                                 float* dA, float* dB, int accumulate, quaff_bf16* G_out_opt,
                                                 int32_t* dbg_acc_opt, int32_t* status_opt, void* ws, size_t ws_bytes,
                                                 quaff_stream_t stream) {
    QUAFF_RETURN_IF(M < 0 || K <= 0 || N <= 0 || nOp < 0 || nO < 0 || nO > nOp || r < 0, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(!dY || lddy < N || !Wq || !dW || ldwq_main < K || !dX || lddx < K, QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(nOp > 0 && (!wq_O || !dw_O || ldwq < nOp), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(nO > 0 && (!O_idx || !s_O), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(r > 0 && (!A || !B), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF(r > 0 && (dA || dB) && (!dA || !dB || !X || !T || ldx < K), QUAFF_ERR_INVALID_ARG);
    QUAFF_RETURN_IF((nOp % 32) || (r % 8) || r > 64 || (N % 16) || N > 16384, QUAFF_ERR_UNSUPPORTED_SHAPE);
    QUAFF_RETURN_IF(!aligned16(dY) || (lddy % 8) || !aligned16(dW), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(!aligned16(Wq) || (ldwq_main % 16), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(nOp > 0 && (!aligned16(wq_O) || (ldwq % 16)), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(!aligned16(dX) || (lddx % 8), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(r > 0 && (!aligned16(A) || !aligned16(B) || (G_out_opt && !aligned16(G_out_opt))), QUAFF_ERR_ALIGNMENT);
    QUAFF_RETURN_IF(r > 0 && dA && (!aligned16(X) || !aligned16(T) || !aligned16(dA) || !aligned16(dB) || (ldx % 8)), QUAFF_ERR_ALIGNMENT);
    const BwdInt8Workspace w = bwd_int8_workspace(M, K, N, nOp, r);
    QUAFF_RETURN_IF(!ws || !aligned16(ws) || ws_bytes < w.total, QUAFF_ERR_WORKSPACE_TOO_SMALL);
    if (M == 0) return empty_batch_grads(K, N, r, dA, dB, accumulate, (cudaStream_t)stream);
    cudaStream_t st = (cudaStream_t)stream;
    unsigned char* base = reinterpret_cast<unsigned char*>(ws);
    int8_t* Zq = reinterpret_cast<int8_t*>(base + w.off_zq);
    float* dz = reinterpret_cast<float*>(base + w.off_dz);
    uint16_t* WdO = reinterpret_cast<uint16_t*>(base + w.off_wdo);
    uint16_t* G = (r > 0 && G_out_opt) ? G_out_opt : reinterpret_cast<uint16_t*>(base + w.off_g);
    float* P = reinterpret_cast<float*>(base + w.off_p);
    float* part = reinterpret_cast<float*>(base + w.off_part);
    float* part_a = reinterpret_cast<float*>(base + w.off_part_a);
    float* part_b = reinterpret_cast<float*>(base + w.off_part_b);
    quaff_status_t rc;
    const bool want_dAB = r > 0 && dA && dB;
    constexpr int CTAS = 2;

    // ---- every tensor map and launch parameter first
    SkinnyGemm gemm_g, gemm_db, gemm_da;
    if (r > 0 && (rc = skinny_prepare(gemm_g, 0, dY, lddy, B, N, M, N, r, part, status_opt)) != QUAFF_OK) return rc;
    FwdWideParams q;                                  // main: acc = Zq Wq over N; epilogue dX = dz[m] acc + G A^T
    memset(&q, 0, sizeof(q));
    if ((rc = make_tmap_2d(&q.map_xq, Zq, 1, M, N, N, kTileM, 128)) != QUAFF_OK) return rc;
    if ((rc = make_tmap_2d(&q.map_wq, Wq, 1, N, K, ldwq_main, 128, 128)) != QUAFF_OK) return rc;     // rows = contraction index n
    q.wq_mn = 1;
    q.nblk = ceil_div(N, 128);
    q.nmma_last = ceil_div(N - (q.nblk - 1) * 128, 32);
    if (r > 0) {
        if ((rc = make_tmap_2d(&q.map_t, G, 2, M, r, r, kTileM, 64)) != QUAFF_OK) return rc;
        if ((rc = make_tmap_2d(&q.map_bt, A, 2, K, r, r, kF256Round / 2, 64)) != QUAFF_OK) return rc;
        q.lora_kmajor = 1;
        q.nmma_l = pad16(r) / 16;
    }
    q.M = M; q.N = K;
    q.tiles_m = ceil_div(M, 2 * kTileM); q.tiles_n = ceil_div(K, kF256TN);
    q.band_m = band_rows(q.tiles_m, q.tiles_n, 2 * kTileM, (size_t)N);
    q.status = status_opt;
    q.dx = dz; q.dW = nullptr; q.dw_O = nullptr; q.lora_scale = 1.0f;
    q.Y = dX; q.ldy = lddx; q.y_f32 = 0;
    q.dbg_main = dbg_acc_opt; q.dbg_out = nullptr;
    GemmParams p;                                     // outlier columns: P = dY [Wd[:,O] | wd] over N, floating point
    const int TNP = 2 * nOp > 128 ? 256 : 128;
    if (nO > 0) {
        memset(&p, 0, sizeof(p));
        GemmPhase& ph = p.ph[0];
        if ((rc = make_tmap_2d(&ph.map_a, dY, 2, M, N, lddy, kTileM, 64)) != QUAFF_OK) return rc;
        if ((rc = make_tmap_2d(&ph.map_b, WdO, 2, N, 2 * nOp, 2 * nOp, 64, 64)) != QUAFF_OK) return rc;
        fill_phase(ph, 0, N, 0, 1, 1 << 30, TNP, CTAS, 0, 1, 64, TNP);
        p.nphases = 1;
        p.M = M; p.N = 2 * nOp;
        p.n_split = 0; p.p_col0 = 0;                  // every column is an outlier partial product
        p.tiles_m = ceil_div(M, kTileM * CTAS); p.tiles_n = ceil_div(p.N, TNP);
        p.band_m = p.tiles_m;
        p.status = status_opt;
        p.dX = nullptr; p.lddx = 0; p.P = P; p.ldp = 2 * nOp;
        p.tile_n = TNP;
    }
    if (want_dAB) {
        if ((rc = skinny_prepare(gemm_db, 1, dY, lddy, T, r, N, M, r, part_b, status_opt)) != QUAFF_OK) return rc;
        if ((rc = skinny_prepare(gemm_da, 1, X, ldx, G, r, K, M, r, part_a, status_opt)) != QUAFF_OK) return rc;
    }

    DeviceSide* ds = device_side();
    std::unique_lock<std::mutex> lock;
    SideSet* ss = nullptr;
    if (ds) {
        lock = std::unique_lock<std::mutex>(ds->mu);
        ss = pick_side_set(ds, st);
    }
    bool forked0 = false, forked1 = false;
    auto leave = [&](quaff_status_t code) {
        if (forked0 && !join_from(ss, 0, st) && code == QUAFF_OK) code = QUAFF_ERR_CUDA;
        if (forked1 && !join_from(ss, 1, st) && code == QUAFF_OK) code = QUAFF_ERR_CUDA;
        return code;
    };
    // side stream 0: the gradient quantization (beside G); later dA.  side stream 1: dB, enqueued behind the GEMMs.
    if (ss && want_dAB && !(forked1 = fork_to(ss, 1, st))) return leave(QUAFF_ERR_CUDA);
    if (ss && !(forked0 = fork_to(ss, 0, st))) return leave(QUAFF_ERR_CUDA);
    cudaStream_t s_q = ss ? ss->s[0] : st;
    if (r > 0) {
        if ((rc = skinny_launch(gemm_g, st)) != QUAFF_OK) return leave(rc);
        launch_pdl(reduce_parts_bf16_kernel, dim3(ceil_div(M * r / 8, 256)), dim3(256), 0, st, 1, part, gemm_g.S, M, r, lora_scale, G);
        if ((rc = launch_status()) != QUAFF_OK) return leave(rc);
        if (ss && cudaEventRecord(ss->g_ready, st) != cudaSuccess) return leave(QUAFF_ERR_CUDA);
    }
    if ((rc = quant_grad_dispatch(dY, lddy, M, N, dW, Zq, N, dz, s_q)) != QUAFF_OK) return leave(rc);
    if (nO > 0) {
        launch_pdl(dequant_weight_kernel, dim3(N, ceil_div(2 * nOp / 16, 256)), dim3(256), 0, s_q, 1, Wq, ldwq_main, dW, wq_O, ldwq, dw_O, O_idx,
                   nO, nOp, 0, 0, WdO, (int64_t)(2 * nOp));
        if ((rc = launch_status()) != QUAFF_OK) return leave(rc);
    }
    if (forked0) {
        forked0 = false;
        if (!join_from(ss, 0, st)) return leave(QUAFF_ERR_CUDA);
    }
    if ((rc = launch_fwd_wide(1, q, st, 1)) != QUAFF_OK) return leave(rc);      // timed as the grad-input GEMM
    if (nO > 0) {
        rc = TNP > 128 ? launch_gemm<EPI_BWD, CTAS, 256>(p, st) : launch_gemm<EPI_BWD, CTAS, 128>(p, st);
        if (rc != QUAFF_OK) return leave(rc);
    }
    if (want_dAB) {
        if (ss && cudaStreamWaitEvent(ss->s[1], ss->join[0], 0) != cudaSuccess) return leave(QUAFF_ERR_CUDA);
        cudaStream_t s_db = ss ? ss->s[1] : st;
        if ((rc = skinny_launch(gemm_db, s_db)) != QUAFF_OK) return leave(rc);
        launch_pdl(reduce_parts_kernel, dim3(ceil_div(N * r / 4, 256)), dim3(256), 0, s_db, 1, part_b, gemm_db.S, N, r, lora_scale, 1, accumulate, dB);
        if ((rc = launch_status()) != QUAFF_OK) return leave(rc);
        cudaStream_t s_da = st;
        if (ss) {
            if (cudaStreamWaitEvent(ss->s[0], ss->g_ready, 0) != cudaSuccess) return leave(QUAFF_ERR_CUDA);
            forked0 = true;
            s_da = ss->s[0];
        }
        if ((rc = skinny_launch(gemm_da, s_da)) != QUAFF_OK) return leave(rc);
        launch_pdl(reduce_parts_kernel, dim3(ceil_div(K * r / 4, 256)), dim3(256), 0, s_da, 1, part_a, gemm_da.S, K, r, 1.0f, 0, accumulate, dA);
        if ((rc = launch_status()) != QUAFF_OK) return leave(rc);
    }
    if (nO > 0) {
        launch_pdl(bwd_fixup_kernel, dim3(ceil_div(M * nO, 256)), dim3(256), 0, st, 1, P, (int64_t)(2 * nOp), M, nO, nOp, O_idx, s_O, G, A, r,
                   dX, lddx, 0);
        if ((rc = launch_status()) != QUAFF_OK) return leave(rc);
    }
    return leave(QUAFF_OK);
}
