// Forward (Eq. 9 + LoRA) with 192-column tiles on CTA pairs.
//
// A tcgen05.mma of a CTA pair costs about 60 + N/2 clocks (measured), so the main INT8 contraction wants
// wide tiles; but the forward has three
// accumulators (main INT32, outlier INT32, LoRA fp32) and TMEM has 512 columns.  This kernel keeps the
// main accumulator 192 columns wide and double-buffered (2 x 192 columns) and gives the two SHORT
// contractions (over nOp <= 128 outlier codes and r <= 64 LoRA ranks) the remaining 128 columns, 64 each,
// by computing them in three ROUNDS of 64 output columns per tile:
//
//   TMEM columns   [0,192) main, even tiles   [192,384) main, odd tiles   [384,448) outlier round   [448,512) LoRA round
//
// The rounds travel through the same TMA/mbarrier ring as the main k-blocks, as extra stages, in a fixed
// interleaving known to the producer and to the MMA issuer alike (both run `for_each_item` below):
//
//   main(t) block 0 .. c1 | round (t-1, 1) | main(t) .. c2 | round (t-1, 2) | main(t) .. last | round (t, 0) | main(t+1) ...
//
// so that the epilogue drains round j of tile t (64 columns of all three accumulators) while the tensor
// pipe is a third of the way further into the main contraction of tile t+1.  Barriers beside the ring:
//   tmem_full / tmem_empty : main accumulator of a tile complete / drained (as in umma_gemm.cuh)
//   aux_ready / aux_free   : the two short accumulators of a round complete / drained
// Roles, CTA-pair protocol, bounded waits and the exit path are those of umma_gemm.cuh, with EIGHT epilogue
// warps (two per TMEM lane quarter) so that a round is drained well within a third of a main contraction.
#pragma once

#include "umma_gemm.cuh"

namespace quaff {

constexpr int kF192TN = 192;
constexpr int kF192Round = 64;                               // output columns per round
constexpr int kF192Threads = 64 + 8 * 32;                    // producer warp, MMA warp, eight epilogue warps
constexpr int kF192StageBytes = kABytes + (kF192TN / 2) * 128;   // A: 128 rows, B: this CTA's 96 rows (a round uses 32 of them)
constexpr int kF192ScaleBytes = 2 * 2 * kF192TN * 4;

struct Fwd192Smem {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full, tmem_empty, aux_ready, aux_free;
    uint32_t tmem_base;
    AbortCtl abort;
};

constexpr int kF192Fixed = 1024 + 256 + kF192ScaleBytes;      // alignment slack, barrier block (padded), scales
constexpr int kF192Stages = (kSmemLimit - kF192Fixed) / kF192StageBytes < kMaxStages ? (kSmemLimit - kF192Fixed) / kF192StageBytes : kMaxStages;
constexpr size_t kF192SmemBytes = (size_t)kF192Fixed + (size_t)kF192Stages * kF192StageBytes;
static_assert(sizeof(Fwd192Smem) <= 256, "barrier block");

// Parameters of the wide forward kernels (this one and fwd256.cuh, which states its own box sizes).
struct FwdWideParams {
    CUtensorMap map_xq, map_wq;      // main: Xq [M][K] (box 128 rows), Wq [N][K] (box 96 rows), 128-byte boxes
    CUtensorMap map_xo, map_wo;      // outlier: xq_O [M][nOp] (box 128 rows), wq_O [N][nOp] (box 32 rows)
    CUtensorMap map_t, map_bt;       // LoRA: T [M][r] bf16 (box 128 rows), B^T [N][rp] bf16 (box 32 rows), 64-element boxes
    int nblk, nmma_last;             // main k-blocks per tile; MMAs of the last one (1..4)
    int nmma_o, nmma_l;              // MMAs of an outlier round (nOp / 32, 0 = no outliers) / of a LoRA round (rp / 16, 0 = no LoRA)
    int M, N, tiles_m, tiles_n;
    int band_m;                      // row tiles per band of the tile order (see tile_coords)
    int32_t* status;
    const float* dx;
    const float* dW;
    const float* dw_O;
    float lora_scale;
    void* Y;
    int64_t ldy;
    int y_f32;
    int32_t* dbg_main;
    int32_t* dbg_out;
    // fwd256_kernel only (the INT8 grad-input variant runs through it with the roles of the matrices exchanged):
    int wq_mn;                       // 1: map_wq is [contraction][output columns] (MN-major B operand), boxes of 128 x 128 bytes
    int lora_kmajor;                 // 1: map_bt is [output columns][contraction] bf16 (K-major), boxes of 64 rows x 64 elements
};

// The ring schedule of one CTA pair: calls main_fn(t, tile, b) for every main k-block and aux_fn(t, tile, j)
// for every round, in ring order; both return false to stop (a wait gave up).
template <typename MainFn, typename AuxFn>
__device__ __forceinline__ void for_each_item(int unit, int nunits, int ntiles, int nblk, MainFn main_fn, AuxFn aux_fn) {
    const int c1 = (nblk - 1) / 3, c2 = (2 * (nblk - 1)) / 3;
    int t = 0, prev = -1;
    for (int tile = unit; tile < ntiles; tile += nunits, ++t) {
        for (int b = 0; b < nblk; ++b) {
            if (!main_fn(t, tile, b)) return;
            if (prev >= 0 && b == c1 && !aux_fn(t - 1, prev, 1)) return;
            if (prev >= 0 && b == c2 && !aux_fn(t - 1, prev, 2)) return;
        }
        if (!aux_fn(t, tile, 0)) return;
        prev = tile;
    }
    if (prev >= 0) {
        if (!aux_fn(t - 1, prev, 1)) return;
        aux_fn(t - 1, prev, 2);
    }
}

__global__ void __launch_bounds__(kF192Threads, 1) fwd192_kernel(const __grid_constant__ FwdWideParams p) {
    constexpr int TN = kF192TN;
    constexpr int kStages = kF192Stages;
    constexpr int kStageBytes = kF192StageBytes;
    constexpr uint32_t kColAuxO = 2 * TN, kColAuxL = 2 * TN + kF192Round;

    extern __shared__ unsigned char smem_dyn[];
    const uint32_t raw = smem_u32(smem_dyn);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;
    unsigned char* aligned = smem_dyn + (tiles_base - raw);
    Fwd192Smem* sm = reinterpret_cast<Fwd192Smem*>(aligned + (size_t)kStages * kStageBytes);
    float* scales = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(sm) + 256);   // [2][dW | dw_O][TN]
    volatile AbortCtl* abort_flag = &sm->abort;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int unit = (int)(blockIdx.x >> 1), nunits = (int)(gridDim.x >> 1);
    const int ntiles = p.tiles_m * p.tiles_n;
    const uint32_t full0 = smem_u32(&sm->full[0]), empty0 = smem_u32(&sm->empty[0]);
    const uint32_t tmem_full_bar = smem_u32(&sm->tmem_full), tmem_empty_bar = smem_u32(&sm->tmem_empty);
    const uint32_t aux_ready_bar = smem_u32(&sm->aux_ready), aux_free_bar = smem_u32(&sm->aux_free);
    const uint32_t lead_full0 = mapa_shared(full0, 0);
    const uint32_t lead_tmem_empty = mapa_shared(tmem_empty_bar, 0);
    const uint32_t lead_aux_free = mapa_shared(aux_free_bar, 0);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full0 + 8u * s, 1);
            mbar_init(empty0 + 8u * s, 1);
        }
        mbar_init(tmem_full_bar, 1);
        mbar_init(tmem_empty_bar, 8 * 2);       // eight epilogue warps in each CTA of the pair
        mbar_init(aux_ready_bar, 1);
        mbar_init(aux_free_bar, 8 * 2);
        sm->abort.flag = 0;
        sm->abort.peer = mapa_shared(smem_u32(&sm->abort.flag), rank ^ 1u);
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc<2>(smem_u32(&sm->tmem_base), 512);
        tmem_relinquish<2>();
    }
    pdl_launch_dependents();
    tc_fence_before();
    __syncthreads();
    cluster_sync();
    tc_fence_after();
    const uint32_t tmem_base = sm->tmem_base;
    pdl_wait();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs of the pair)
        if (elect_one()) {
            prefetch_tmap(&p.map_xq); prefetch_tmap(&p.map_wq);
            if (p.nmma_o) { prefetch_tmap(&p.map_xo); prefetch_tmap(&p.map_wo); }
            if (p.nmma_l) { prefetch_tmap(&p.map_t); prefetch_tmap(&p.map_bt); }
            uint32_t stage = 0, phase = 0;
            // one ring stage: A box at (x, ya), B box at (x, yb)
            auto load_stage = [&](const CUtensorMap* ma, const CUtensorMap* mb, int x, int ya, int yb, uint32_t tx) -> bool {
                if (!mbar_wait(empty0 + 8u * stage, phase ^ 1u, abort_flag)) return false;
                const uint32_t bar = lead_full0 + 8u * stage;
                const uint32_t dst = tiles_base + stage * kStageBytes;
                if (rank == 0) mbar_arrive_expect_tx(full0 + 8u * stage, tx * 2);
                tma_load_2d<2>(dst, ma, x, ya, bar);
                tma_load_2d<2>(dst + kABytes, mb, x, yb, bar);
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
                return true;
            };
            const uint32_t tx_main = kABytes + (TN / 2) * 128, tx_aux = kABytes + (kF192Round / 2) * 128;
            int tm = 0, tn = 0;
            for_each_item(unit, nunits, ntiles, p.nblk,
                [&](int, int tile, int b) -> bool {
                    if (b == 0) tile_coords(tile, p.tiles_m, p.tiles_n, p.band_m, tm, tn);   // once per tile: this loop is the issue path
                    return load_stage(&p.map_xq, &p.map_wq, b * 128, tm * 256 + (int)rank * kTileM, tn * TN + (int)rank * (TN / 2), tx_main);
                },
                [&](int, int tile, int j) -> bool {
                    int tm, tn;
                    tile_coords(tile, p.tiles_m, p.tiles_n, p.band_m, tm, tn);
                    const int m0 = tm * 256 + (int)rank * kTileM;
                    const int nr = tn * TN + j * kF192Round + (int)rank * (kF192Round / 2);
                    if (p.nmma_o && !load_stage(&p.map_xo, &p.map_wo, 0, m0, nr, tx_aux)) return false;
                    if (p.nmma_l && !load_stage(&p.map_t, &p.map_bt, 0, m0, nr, tx_aux)) return false;
                    return true;
                });
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (the leader's, for the pair)
        if (rank == 0 && elect_one()) {
            uint32_t stage = 0, phase = 0;
            int rounds = 0;                    // rounds issued so far
            const uint32_t idesc_main = umma_idesc(kCFmtS32, kFmtS8, 256, TN);
            const uint32_t idesc_o = umma_idesc(kCFmtS32, kFmtS8, 256, kF192Round);
            const uint32_t idesc_l = umma_idesc(kCFmtF32, kFmtBF16, 256, kF192Round);
            // consume one ring stage with `nmma` MMAs of 32 contraction bytes each
            auto mma_stage = [&](uint32_t acc, uint32_t idesc, bool i8, int nmma, uint32_t& accumulate) -> bool {
                if (!mbar_wait(full0 + 8u * stage, phase, abort_flag)) return false;
                tc_fence_after();
                const uint32_t a_lo = (((tiles_base + stage * kStageBytes) & 0x3FFFFu) >> 4) | (1u << 16);
                const uint32_t b_lo = a_lo + (kABytes >> 4);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (k < nmma) {
                        if (i8) umma_i8<2>(acc, make_desc(a_lo + 2 * k, kDescHi), make_desc(b_lo + 2 * k, kDescHi), idesc, accumulate);
                        else umma_f16<2>(acc, make_desc(a_lo + 2 * k, kDescHi), make_desc(b_lo + 2 * k, kDescHi), idesc, accumulate);
                        accumulate = 1u;
                    }
                }
                umma_commit<2>(empty0 + 8u * stage);
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
                return true;
            };
            uint32_t acc_main = 0;
            for_each_item(unit, nunits, ntiles, p.nblk,
                [&](int t, int, int b) -> bool {
                    if (b == 0) acc_main = 0u;
                    return mma_stage(tmem_base + (uint32_t)((t & 1) * TN), idesc_main, true, b == p.nblk - 1 ? p.nmma_last : 4, acc_main);
                },
                [&](int t, int, int j) -> bool {
                    if (j == 0) {
                        // Round 0 directly follows the tile's last main block (and the last rounds of the previous
                        // tile): the main accumulator is complete; the main buffer of the NEXT tile is the one the
                        // epilogue of the previous tile drains, so that epilogue must be through.
                        if (t > 0 && !mbar_wait(tmem_empty_bar, (uint32_t)((t - 1) & 1), abort_flag)) return false;
                        umma_commit<2>(tmem_full_bar);
                    }
                    // the two short accumulators are free once the epilogues have drained the previous round
                    if (rounds > 0 && !mbar_wait(aux_free_bar, (uint32_t)((rounds - 1) & 1), abort_flag)) return false;
                    uint32_t acc = 0u;
                    if (p.nmma_o && !mma_stage(tmem_base + kColAuxO, idesc_o, true, p.nmma_o, acc)) return false;
                    acc = 0u;
                    if (p.nmma_l && !mma_stage(tmem_base + kColAuxL, idesc_l, false, p.nmma_l, acc)) return false;
                    umma_commit<2>(aux_ready_bar);
                    ++rounds;
                    return true;
                });
        }
    } else {
        // ------------------------------------------------------------------ epilogue (8 warps = 256 threads per CTA)
        // Warps w and w + 4 share a TMEM lane quarter; of the 64 columns of a round, the first four warps take
        // columns [0,32) and the other four [32,64): a round is drained by all eight warps at once.
        const int q = warp & 3;
        const int g = (warp - 2) >> 2;           // which half of a round's columns
        const int row = q * 32 + lane;
        const int et = threadIdx.x - 64;         // 0..255
        const bool has_o = p.nmma_o != 0, has_l = p.nmma_l != 0;
        bool ok = true;
        int t = 0, rounds = 0;
        for (int tile = unit; tile < ntiles && ok; tile += nunits, ++t) {
            int tm, tn;
            tile_coords(tile, p.tiles_m, p.tiles_n, p.band_m, tm, tn);
            const int m0 = tm * 256 + (int)rank * kTileM, n0 = tn * TN;
            const int buf = t & 1;
            float* scale_w = scales + buf * 2 * TN;
            float* scale_o = scale_w + TN;
            if (et < TN) {
                const int n = n0 + et;
                scale_w[et] = n < p.N ? p.dW[n] : 0.0f;
                scale_o[et] = (n < p.N && has_o) ? p.dw_O[n] : 0.0f;
            }
            const int m = m0 + row;
            const float dxm = m < p.M ? __ldg(p.dx + m) : 0.0f;
            named_bar_sync(1, kF192Threads - 64);
            if (!mbar_wait(tmem_full_bar, (uint32_t)(t & 1), abort_flag)) { ok = false; break; }
            const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
            for (int j = 0; j < TN / kF192Round; ++j, ++rounds) {
                if (!mbar_wait(aux_ready_bar, (uint32_t)(rounds & 1), abort_flag)) { ok = false; break; }
                tc_fence_after();
                const int cl = j * kF192Round + g * 32;      // first of this warp's 32 columns inside the tile
#pragma unroll
                for (int h = 0; h < 2; ++h) {                // 16 columns at a time (register budget)
                    const int c0 = cl + 16 * h;
                    const int nc = n0 + c0;
                    uint32_t r0[16], r1[16], r2[16];
                    tmem_ld_32x16(lane_addr + (uint32_t)(buf * TN + c0), r0);
                    if (has_o) tmem_ld_32x16(lane_addr + kColAuxO + (uint32_t)(g * 32 + 16 * h), r1);
                    if (has_l) tmem_ld_32x16(lane_addr + kColAuxL + (uint32_t)(g * 32 + 16 * h), r2);
                    tmem_ld_wait();
                    if (m < p.M && nc < p.N) {
                        float y[16], sw[16], so[16];     // the 16 column scales by 128-bit shared loads
#pragma unroll
                        for (int i = 0; i < 16; i += 4) {
                            const float4 a = *reinterpret_cast<const float4*>(scale_w + c0 + i);
                            sw[i] = a.x; sw[i + 1] = a.y; sw[i + 2] = a.z; sw[i + 3] = a.w;
                            const float4 b = has_o ? *reinterpret_cast<const float4*>(scale_o + c0 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                            so[i] = b.x; so[i + 1] = b.y; so[i + 2] = b.z; so[i + 3] = b.w;
                        }
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            float w = (float)(int)r0[i] * sw[i];
                            if (has_o) w += (float)(int)r1[i] * so[i];
                            float v = dxm * w;
                            if (has_l) v += p.lora_scale * __uint_as_float(r2[i]);
                            y[i] = v;
                        }
                        const bool full = (nc + 16 <= p.N);
                        if (p.y_f32) {
                            float* out = reinterpret_cast<float*>(p.Y) + (int64_t)m * p.ldy + nc;
                            if (full && (p.ldy % 4 == 0)) {
#pragma unroll
                                for (int i = 0; i < 16; i += 4) *reinterpret_cast<float4*>(out + i) = make_float4(y[i], y[i + 1], y[i + 2], y[i + 3]);
                            } else {
                                for (int i = 0; i < 16; ++i) if (nc + i < p.N) out[i] = y[i];
                            }
                        } else {
                            uint16_t* out = reinterpret_cast<uint16_t*>(p.Y) + (int64_t)m * p.ldy + nc;
                            if (full && (p.ldy % 8 == 0)) {
#pragma unroll
                                for (int i = 0; i < 16; i += 8)
                                    *reinterpret_cast<uint4*>(out + i) = make_uint4(pack_bf16x2(y[i], y[i + 1]), pack_bf16x2(y[i + 2], y[i + 3]),
                                                                                    pack_bf16x2(y[i + 4], y[i + 5]), pack_bf16x2(y[i + 6], y[i + 7]));
                            } else {
                                for (int i = 0; i < 16; ++i) if (nc + i < p.N) out[i] = (uint16_t)f32_to_bf16_bits(y[i]);
                            }
                        }
                        if (p.dbg_main) {
                            int32_t* d = p.dbg_main + (int64_t)m * p.N + nc;
                            for (int i = 0; i < 16; ++i) if (nc + i < p.N) d[i] = (int32_t)r0[i];
                        }
                        if (p.dbg_out) {
                            int32_t* d = p.dbg_out + (int64_t)m * p.N + nc;
                            for (int i = 0; i < 16; ++i) if (nc + i < p.N) d[i] = has_o ? (int32_t)r1[i] : 0;
                        }
                    }
                }
                // this warp's share of the round is drained (also when its columns lie past N)
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (rank != 0) mbar_arrive_cluster(lead_aux_free);
                    else mbar_arrive(aux_free_bar);
                }
            }
            if (!ok) break;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (rank != 0) mbar_arrive_cluster(lead_tmem_empty);
                else mbar_arrive(tmem_empty_bar);
            }
        }
    }

    // ---------------------------------------------------------------------- common exit
    tc_fence_before();
    __syncthreads();
    if (abort_flag->flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // let copies in flight land before the CTA retires
        if (threadIdx.x == 0 && p.status) atomicExch(p.status, (int)QUAFF_ERR_TIMEOUT);
        __syncthreads();
    }
    cluster_sync();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc<2>(tmem_base, 512);
    }
}

}  // namespace quaff
