// Persistent, warp-specialised tcgen05 GEMM pipeline shared by the forward (Eq. 9 + LoRA) and the
// grad-input kernels.
//
//   warp 0      : TMA producer (one elected lane) - 128-byte-swizzled operand tiles into a ring of stages
//   warp 1      : TMEM allocation + MMA issue (one elected lane) - tcgen05.mma, accumulators in TMEM
//   warps 2..5  : epilogue - tcgen05.ld of the finished accumulators, dequantization / conversion, stores
//
// An output tile is 128 x 128.  Its contraction is a list of up to three PHASES, each a run of
// k-blocks with its own pair of tensor maps, operand type and accumulator:
//   forward : main INT8 (over K) -> acc slot 0 | outlier INT8 (over nOp) -> slot 1 | LoRA bf16 (over r) -> slot 2
//   backward: main bf16 (over N) -> slot 0     | LoRA bf16 (over r) -> slot 0 (accumulating)
// Every k-block is one stage: an A tile and a B tile of 128 rows x 128 bytes each, both K-major.
// Tails need no special case: TMA zero-fills out-of-range rows and columns, and the epilogue masks stores.
//
// TMEM (512 columns): slot 0 is double-buffered at columns [0,128) and [128,256) so the main
// contraction of tile t+1 overlaps the epilogue of tile t; slots 1 and 2 live at [256,384) and
// [384,512) and are written only after the epilogue of the previous tile has drained them.
//
// Every wait is bounded (see mbar_wait); on expiry all roles fall through to the common exit, TMEM is
// freed, and QUAFF_ERR_TIMEOUT is written to the status word.
#pragma once

#include "common.cuh"

namespace quaff {

constexpr int kTileM = 128;
constexpr int kTileN = 128;
constexpr int kStages = 6;
constexpr int kOperandBytes = 128 * 128;          // one operand tile: 128 rows x 128 bytes
constexpr int kStageBytes = 2 * kOperandBytes;
constexpr int kGemmThreads = 192;
constexpr int kMaxPhases = 3;

struct GemmPhase {
    CUtensorMap map_a;   // rows = output rows (M side), columns = contraction
    CUtensorMap map_b;   // rows = output columns (N side), columns = contraction
    int nblk;            // k-blocks in this phase
    int is_i8;           // 1: kind::i8 (128 elements per block, 32 per MMA); 0: kind::f16 bf16 (64 per block, 16 per MMA)
    int kext;            // contraction extent in elements
    int acc_slot;        // 0 main (double-buffered), 1, 2 auxiliary
    int fresh;           // 1: first MMA of the phase overwrites the accumulator
    int tn_limit;        // the phase runs only for column tiles tn < tn_limit
};

enum { EPI_FWD = 0, EPI_BWD = 1 };

struct GemmParams {
    GemmPhase ph[kMaxPhases];
    int nphases;
    int M, N;            // output extent (rows, columns)
    int tiles_m, tiles_n;
    int32_t* status;
    // forward epilogue (Eq. 9 + LoRA)
    const float* dx;     // [M]
    const float* dW;     // [N]
    const float* dw_O;   // [N]
    float lora_scale;
    int has_outlier, has_lora;
    void* Y;
    int64_t ldy;
    int y_f32;
    int32_t* dbg_main;   // dense [M][N] or null
    int32_t* dbg_out;
    // backward epilogue: columns < n_split go to dX (bf16); columns >= p_col0 (a tile boundary) go to
    // P (f32, column index minus p_col0); columns in between are padding and are dropped
    int n_split;
    int p_col0;
    uint16_t* dX;
    int64_t lddx;
    float* P;
    int64_t ldp;
};

struct GemmSmem {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t tmem_full;
    uint64_t tmem_empty;
    uint32_t tmem_base;
    int abort_flag;
    float scale_w[2][kTileN];
    float scale_o[2][kTileN];
};

constexpr size_t kGemmSmemBytes = 1024 + (size_t)kStages * kStageBytes + sizeof(GemmSmem);

template <int EPI>
__global__ void __launch_bounds__(kGemmThreads, 1) umma_gemm_kernel(const __grid_constant__ GemmParams p) {
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t raw = smem_u32(smem_dyn);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;
    unsigned char* aligned = smem_dyn + (tiles_base - raw);
    GemmSmem* sm = reinterpret_cast<GemmSmem*>(aligned + (size_t)kStages * kStageBytes);
    volatile int* abort_flag = &sm->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int ntiles = p.tiles_m * p.tiles_n;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&sm->full[s]), 1);
            mbar_init(smem_u32(&sm->empty[s]), 1);
        }
        mbar_init(smem_u32(&sm->tmem_full), 1);
        mbar_init(smem_u32(&sm->tmem_empty), 4);
        sm->abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&sm->tmem_base), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sm->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (elect_one()) {
            for (int i = 0; i < p.nphases; ++i) {
                prefetch_tmap(&p.ph[i].map_a);
                prefetch_tmap(&p.ph[i].map_b);
            }
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
                const int tm = tile % p.tiles_m, tn = tile / p.tiles_m;
                const int m0 = tm * kTileM, n0 = tn * kTileN;
                for (int i = 0; i < p.nphases && ok; ++i) {
                    const GemmPhase& ph = p.ph[i];
                    if (tn >= ph.tn_limit) continue;
                    const int kbox = ph.is_i8 ? 128 : 64;
                    for (int b = 0; b < ph.nblk; ++b) {
                        if (!mbar_wait(smem_u32(&sm->empty[stage]), phase ^ 1u, abort_flag)) { ok = false; break; }
                        const uint32_t bar = smem_u32(&sm->full[stage]);
                        const uint32_t dst = tiles_base + stage * kStageBytes;
                        mbar_arrive_expect_tx(bar, kStageBytes);
                        tma_load_2d(dst, &ph.map_a, b * kbox, m0, bar);
                        tma_load_2d(dst + kOperandBytes, &ph.map_b, b * kbox, n0, bar);
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            const uint32_t idesc_i8 = umma_idesc(kCFmtS32, kFmtS8, kTileM, kTileN);
            const uint32_t idesc_bf = umma_idesc(kCFmtF32, kFmtBF16, kTileM, kTileN);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int t = 0;
            for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++t) {
                const int tn = tile / p.tiles_m;
                for (int i = 0; i < p.nphases && ok; ++i) {
                    const GemmPhase& ph = p.ph[i];
                    if (tn < ph.tn_limit) {
                        const uint32_t acc = tmem_base + (ph.acc_slot == 0 ? (uint32_t)((t & 1) * kTileN) : (uint32_t)((ph.acc_slot + 1) * kTileN));
                        const int kbox = ph.is_i8 ? 128 : 64;
                        const int kins = ph.is_i8 ? 32 : 16;
                        for (int b = 0; b < ph.nblk; ++b) {
                            if (!mbar_wait(smem_u32(&sm->full[stage]), phase, abort_flag)) { ok = false; break; }
                            tc_fence_after();
                            const uint32_t a_addr = tiles_base + stage * kStageBytes;
                            const uint64_t da = smem_desc_k_sw128(a_addr);
                            const uint64_t db = smem_desc_k_sw128(a_addr + kOperandBytes);
                            const int left = ph.kext - b * kbox;
                            const int nmma = (min(kbox, left) + kins - 1) / kins;
                            for (int k = 0; k < nmma; ++k) {
                                const uint32_t accumulate = (ph.fresh && b == 0 && k == 0) ? 0u : 1u;
                                if (ph.is_i8) umma_i8(acc, da + 2u * k, db + 2u * k, idesc_i8, accumulate);
                                else          umma_f16(acc, da + 2u * k, db + 2u * k, idesc_bf, accumulate);
                            }
                            umma_commit(smem_u32(&sm->empty[stage]));
                            if (++stage == kStages) { stage = 0; phase ^= 1u; }
                        }
                    }
                    // After the main phase: the auxiliary accumulators of this tile, and the main buffer of
                    // the next tile, may be written only once the epilogue has drained the previous tile.
                    if (ok && i == 0 && t > 0 && !mbar_wait(smem_u32(&sm->tmem_empty), (uint32_t)((t - 1) & 1), abort_flag)) ok = false;
                }
                if (!ok) break;
                umma_commit(smem_u32(&sm->tmem_full));
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (128 threads)
        const int q = warp & 3;                  // TMEM lane quarter this warp may read
        const int row = q * 32 + lane;
        const int et = threadIdx.x - 64;         // 0..127
        bool ok = true;
        int t = 0;
        for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++t) {
            const int tm = tile % p.tiles_m, tn = tile / p.tiles_m;
            const int m0 = tm * kTileM, n0 = tn * kTileN;
            const int buf = t & 1;
            if (EPI == EPI_FWD) {
                const int n = n0 + et;
                sm->scale_w[buf][et] = n < p.N ? p.dW[n] : 0.0f;
                sm->scale_o[buf][et] = (n < p.N && p.has_outlier) ? p.dw_O[n] : 0.0f;
                named_bar_sync(1, 128);
            }
            if (!mbar_wait(smem_u32(&sm->tmem_full), (uint32_t)(t & 1), abort_flag)) { ok = false; break; }
            tc_fence_after();
            const int m = m0 + row;
            const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
            for (int c = 0; c < kTileN / 32; ++c) {
                const int nc = n0 + c * 32;
                if (nc >= p.N) break;            // uniform across the warp
                uint32_t r0[32];
                tmem_ld_32x32(lane_addr + (uint32_t)(buf * kTileN + c * 32), r0);
                if (EPI == EPI_FWD) {
                    uint32_t r1[32], r2[32];
                    if (p.has_outlier) tmem_ld_32x32(lane_addr + (uint32_t)(2 * kTileN + c * 32), r1);
                    if (p.has_lora) tmem_ld_32x32(lane_addr + (uint32_t)(3 * kTileN + c * 32), r2);
                    tmem_ld_wait();
                    if (m < p.M) {
                        const float dxm = p.dx[m];
                        float y[32];
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            float w = (float)(int)r0[j] * sm->scale_w[buf][c * 32 + j];
                            if (p.has_outlier) w += (float)(int)r1[j] * sm->scale_o[buf][c * 32 + j];
                            float v = dxm * w;
                            if (p.has_lora) v += p.lora_scale * __uint_as_float(r2[j]);
                            y[j] = v;
                        }
                        const bool full = (nc + 32 <= p.N);
                        if (p.y_f32) {
                            float* out = reinterpret_cast<float*>(p.Y) + (int64_t)m * p.ldy + nc;
                            if (full && (p.ldy % 4 == 0)) {
#pragma unroll
                                for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4*>(out + j) = make_float4(y[j], y[j + 1], y[j + 2], y[j + 3]);
                            } else {
                                for (int j = 0; j < 32; ++j) if (nc + j < p.N) out[j] = y[j];
                            }
                        } else {
                            uint16_t* out = reinterpret_cast<uint16_t*>(p.Y) + (int64_t)m * p.ldy + nc;
                            if (full && (p.ldy % 8 == 0)) {
#pragma unroll
                                for (int j = 0; j < 32; j += 8)
                                    *reinterpret_cast<uint4*>(out + j) = make_uint4(pack_bf16x2(y[j], y[j + 1]), pack_bf16x2(y[j + 2], y[j + 3]),
                                                                                    pack_bf16x2(y[j + 4], y[j + 5]), pack_bf16x2(y[j + 6], y[j + 7]));
                            } else {
                                for (int j = 0; j < 32; ++j) if (nc + j < p.N) out[j] = (uint16_t)f32_to_bf16_bits(y[j]);
                            }
                        }
                        if (p.dbg_main) {
                            int32_t* d = p.dbg_main + (int64_t)m * p.N + nc;
                            for (int j = 0; j < 32; ++j) if (nc + j < p.N) d[j] = (int32_t)r0[j];
                        }
                        if (p.dbg_out) {
                            int32_t* d = p.dbg_out + (int64_t)m * p.N + nc;
                            for (int j = 0; j < 32; ++j) if (nc + j < p.N) d[j] = p.has_outlier ? (int32_t)r1[j] : 0;
                        }
                    }
                } else {
                    tmem_ld_wait();
                    if (m < p.M) {
                        if (nc < p.p_col0) {
                            uint16_t* out = p.dX + (int64_t)m * p.lddx + nc;
                            if (nc + 32 <= p.n_split && (p.lddx % 8 == 0)) {
#pragma unroll
                                for (int j = 0; j < 32; j += 8)
                                    *reinterpret_cast<uint4*>(out + j) =
                                        make_uint4(pack_bf16x2(__uint_as_float(r0[j]), __uint_as_float(r0[j + 1])),
                                                   pack_bf16x2(__uint_as_float(r0[j + 2]), __uint_as_float(r0[j + 3])),
                                                   pack_bf16x2(__uint_as_float(r0[j + 4]), __uint_as_float(r0[j + 5])),
                                                   pack_bf16x2(__uint_as_float(r0[j + 6]), __uint_as_float(r0[j + 7])));
                            } else {
                                for (int j = 0; j < 32; ++j) if (nc + j < p.n_split) out[j] = (uint16_t)f32_to_bf16_bits(__uint_as_float(r0[j]));
                            }
                        } else {
                            float* out = p.P + (int64_t)m * p.ldp + (nc - p.p_col0);
                            for (int j = 0; j < 32; ++j) if (nc + j < p.N) out[j] = __uint_as_float(r0[j]);
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm->tmem_empty));
        }
    }

    // ---------------------------------------------------------------------- common exit
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // let copies in flight land before the CTA retires
        if (threadIdx.x == 0 && p.status) atomicExch(p.status, (int)QUAFF_ERR_TIMEOUT);
        __syncthreads();
    }
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace quaff
