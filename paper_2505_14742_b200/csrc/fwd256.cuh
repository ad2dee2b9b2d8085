// Forward (Eq. 9 + LoRA) with 256-column tiles on CTA pairs.
//
// A tcgen05.mma of a CTA pair costs about 60 + N/2 clocks (measured), so the widest tile (N = 256) is the cheapest per
// output column: 0.74 clocks against 0.86 (N = 192) and 0.98 (N = 128).  Three accumulators of 256 columns do not fit
// TMEM's 512 columns, and neither does a double-buffered main one beside anything else.  This kernel keeps ONE main
// accumulator and frees it early.  The two SHORT contractions (over nOp <= 128 outlier codes and r <= 64 LoRA
// ranks) share the other 256 columns, 128 each, and are computed in two ROUNDS of 128 output columns per tile:
//
//   TMEM columns   [0,256) main   [256,384) outlier round   [384,512) LoRA round
//
// The rounds travel through the same TMA/mbarrier ring as the main k-blocks, as extra stages, in a fixed
// interleaving known to the producer and to the MMA issuer alike (both run `for_each_item256` below):
//
//   round (t-1, 1) | main(t) block 0 .. last | round (t, 0) | round (t, 1) | main(t+1) ...
//
// When the main accumulator of tile t and its round 0 are complete (tmem_full), the sixteen epilogue warps
//   1. finish columns [0,128) straight from TMEM (main + round 0); half of a bf16 result is stored at once, the other
//      half waits packed in registers and is stored after the hand-over,
//   2. copy columns [128,256) of the main accumulator into registers (32 per thread),
// and hand main accumulator and round accumulators back (tmem_empty): the tensor pipe waits only for that.  It then
// runs round 1 of tile t and starts the main contraction of tile t+1, during which the warps combine their registers
// with round 1 (aux_ready) and store columns [128,256) (aux_free, awaited before round 0 of tile t+1).
// Barriers beside the ring:
//   tmem_full / tmem_empty : main accumulator and round 0 complete / first half stored, second half copied out
//   aux_ready / aux_free   : round 1 complete / consumed
// Roles, CTA-pair protocol, bounded waits and the exit path are those of umma_gemm.cuh.
#pragma once

#include "fwd192.cuh"

namespace quaff {

constexpr int kF256TN = 256;
constexpr int kF256Round = 128;                              // output columns per round
constexpr int kF256EpiWarps = 16;
constexpr int kF256Threads = 64 + kF256EpiWarps * 32;        // producer warp, MMA warp, sixteen epilogue warps
constexpr int kF256StageBytes = kABytes + (kF256TN / 2) * 128;   // A: 128 rows, B: this CTA's 128 rows (a round uses 64 of them)
constexpr int kF256ScaleBytes = kF256EpiWarps * 2 * 64 * 4;  // per epilogue warp: dW and dw_O of its 2 x 32 columns

struct Fwd256Smem {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full, tmem_empty, aux_ready, aux_free;
    uint32_t tmem_base;
    AbortCtl abort;
};

constexpr int kF256Fixed = 1024 + 256 + kF256ScaleBytes;    // alignment slack, barrier block (padded), scales
constexpr int kF256Stages = (kSmemLimit - kF256Fixed) / kF256StageBytes < kMaxStages ? (kSmemLimit - kF256Fixed) / kF256StageBytes : kMaxStages;
constexpr size_t kF256SmemBytes = (size_t)kF256Fixed + (size_t)kF256Stages * kF256StageBytes;
static_assert(sizeof(Fwd256Smem) <= 256, "barrier block");

// The ring schedule of one CTA pair: calls main_fn(t, tile, b) for every main k-block and aux_fn(t, tile, j)
// for every round, in ring order; both return false to stop (a wait gave up).
template <typename MainFn, typename AuxFn>
__device__ __forceinline__ void for_each_item256(int unit, int nunits, int ntiles, int nblk, MainFn main_fn, AuxFn aux_fn) {
    int t = 0, prev = -1;
    for (int tile = unit; tile < ntiles; tile += nunits, ++t) {
        if (prev >= 0 && !aux_fn(t - 1, prev, 1)) return;
        for (int b = 0; b < nblk; ++b)
            if (!main_fn(t, tile, b)) return;
        if (!aux_fn(t, tile, 0)) return;
        prev = tile;
    }
    if (prev >= 0) aux_fn(t - 1, prev, 1);
}

// Parameters: FwdWideParams with the boxes of map_wq 128 rows and of map_wo 64 rows high;
// map_bt is LoRA B [r][N] itself, boxes of rp contraction rows x 64 columns.
// The INT8 grad-input variant uses the same kernel with the matrices in other roles (A operand = the quantized
// gradient Zq [M][N], contraction over N): its weight operand is Wq [N][K] read IN PLACE with the contraction index as
// the row (p.wq_mn: an MN-major INT8 operand, one box = 128 contraction rows x 128 output columns, so a CTA's half of
// the tile is exactly one box), its LoRA operand is A [K][r] (p.lora_kmajor), and a null p.dW means column scale 1.
__global__ void __launch_bounds__(kF256Threads, 1) fwd256_kernel(const __grid_constant__ FwdWideParams p) {
    constexpr int TN = kF256TN;
    constexpr int kStages = kF256Stages;
    constexpr int kStageBytes = kF256StageBytes;
    constexpr uint32_t kColAuxO = TN, kColAuxL = TN + kF256Round;

    extern __shared__ unsigned char smem_dyn[];
    const uint32_t raw = smem_u32(smem_dyn);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;
    unsigned char* aligned = smem_dyn + (tiles_base - raw);
    Fwd256Smem* sm = reinterpret_cast<Fwd256Smem*>(aligned + (size_t)kStages * kStageBytes);
    float* scales = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(sm) + 256);   // [epilogue warp][dW | dw_O][round][32]
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
        mbar_init(tmem_empty_bar, kF256EpiWarps * 2);       // every epilogue warp of both CTAs
        mbar_init(aux_ready_bar, 1);
        mbar_init(aux_free_bar, kF256EpiWarps * 2);
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
            auto load_stage = [&](const CUtensorMap* ma, const CUtensorMap* mb, int x, int ya, int yb, uint32_t tx, int xb = -1) -> bool {
                if (!mbar_wait(empty0 + 8u * stage, phase ^ 1u, abort_flag)) return false;
                const uint32_t bar = lead_full0 + 8u * stage;
                const uint32_t dst = tiles_base + stage * kStageBytes;
                if (rank == 0) mbar_arrive_expect_tx(full0 + 8u * stage, tx * 2);
                tma_load_2d<2>(dst, ma, x, ya, bar);
                tma_load_2d<2>(dst + kABytes, mb, xb < 0 ? x : xb, yb, bar);
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
                return true;
            };
            const uint32_t tx_main = kABytes + (TN / 2) * 128, tx_aux = kABytes + (kF256Round / 2) * 128;
            // LoRA B: one box of 64 columns x rp contraction rows (MN-major), or of 64 output columns x 64 elements (K-major)
            const uint32_t tx_lora = kABytes + (p.lora_kmajor ? 64u * 128u : (uint32_t)p.nmma_l * 16u * 128u);
            int tm = 0, tn = 0;
            for_each_item256(unit, nunits, ntiles, p.nblk,
                [&](int, int tile, int b) -> bool {
                    if (b == 0) tile_coords(tile, p.tiles_m, p.tiles_n, p.band_m, tm, tn);   // once per tile: this loop is the issue path
                    const int nb0 = tn * TN + (int)rank * (TN / 2);
                    if (p.wq_mn) return load_stage(&p.map_xq, &p.map_wq, b * 128, tm * 256 + (int)rank * kTileM, b * 128, tx_main, nb0);
                    return load_stage(&p.map_xq, &p.map_wq, b * 128, tm * 256 + (int)rank * kTileM, nb0, tx_main);
                },
                [&](int, int tile, int j) -> bool {
                    int tm, tn;
                    tile_coords(tile, p.tiles_m, p.tiles_n, p.band_m, tm, tn);
                    const int m0 = tm * 256 + (int)rank * kTileM;
                    const int nr = tn * TN + j * kF256Round + (int)rank * (kF256Round / 2);
                    if (p.nmma_o && !load_stage(&p.map_xo, &p.map_wo, 0, m0, nr, tx_aux)) return false;
                    // LoRA B [r][N] is read in place: MN-major, coordinates (column, contraction row)
                    if (p.nmma_l && !(p.lora_kmajor ? load_stage(&p.map_t, &p.map_bt, 0, m0, nr, tx_lora)
                                                    : load_stage(&p.map_t, &p.map_bt, 0, m0, 0, tx_lora, nr))) return false;
                    return true;
                });
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (the leader's, for the pair)
        if (rank == 0 && elect_one()) {
            uint32_t stage = 0, phase = 0;
            const uint32_t idesc_main = umma_idesc(kCFmtS32, kFmtS8, 256, TN) | (p.wq_mn ? (1u << 16) : 0u);
            const uint32_t idesc_o = umma_idesc(kCFmtS32, kFmtS8, 256, kF256Round);
            const uint32_t idesc_l = umma_idesc(kCFmtF32, kFmtBF16, 256, kF256Round) | (p.lora_kmajor ? 0u : (1u << 16));   // bit 16: B is MN-major
            // consume one ring stage with `nmma` MMAs of 32 contraction bytes each
            // (K-major operands advance 32 bytes inside the swizzled row per MMA; the MN-major B of the LoRA round
            // advances 16 contraction rows = 2048 bytes, its leading byte offset - the distance between boxes of 64
            // columns - is not used with a single box)
            // b_mn: the B operand of this stage is MN-major.  One MMA then consumes 32 bytes of contraction = 16 rows of
            // bf16 or 32 rows of INT8, rows being 128 bytes apart: an advance of 2048 resp. 4096 bytes.
            auto mma_stage = [&](uint32_t acc, uint32_t idesc, bool i8, bool b_mn, int nmma, uint32_t& accumulate) -> bool {
                if (!mbar_wait(full0 + 8u * stage, phase, abort_flag)) return false;
                tc_fence_after();
                const uint32_t s_lo = ((tiles_base + stage * kStageBytes) & 0x3FFFFu) >> 4;
                const uint32_t a_lo = s_lo | (1u << 16);
                const uint32_t b_lo = !b_mn ? a_lo + (kABytes >> 4) : ((s_lo + (kABytes >> 4)) | ((uint32_t)(kAtomBytes >> 4) << 16));
                const uint32_t b_adv = !b_mn ? 2u : (i8 ? (4096u >> 4) : (2048u >> 4));
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (k < nmma) {
                        if (i8) umma_i8<2>(acc, make_desc(a_lo + 2 * k, kDescHi), make_desc(b_lo + b_adv * k, kDescHi), idesc, accumulate);
                        else umma_f16<2>(acc, make_desc(a_lo + 2 * k, kDescHi), make_desc(b_lo + b_adv * k, kDescHi), idesc, accumulate);
                        accumulate = 1u;
                    }
                }
                umma_commit<2>(empty0 + 8u * stage);
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
                return true;
            };
            uint32_t acc_main = 0;
            for_each_item256(unit, nunits, ntiles, p.nblk,
                [&](int, int, int b) -> bool {
                    if (b == 0) acc_main = 0u;
                    return mma_stage(tmem_base, idesc_main, true, p.wq_mn != 0, b == p.nblk - 1 ? p.nmma_last : 4, acc_main);
                },
                [&](int t, int, int j) -> bool {
                    if (j == 0) {
                        // round 0 of tile t follows its main contraction; the round accumulators must have been
                        // consumed by round 1 of the previous tile
                        if (t > 0 && !mbar_wait(aux_free_bar, (uint32_t)((t - 1) & 1), abort_flag)) return false;
                    } else {
                        // round 1 of tile t opens the work on tile t+1 (or ends the kernel): the epilogue has taken
                        // what it needs of tile t out of the main and the round accumulators
                        if (!mbar_wait(tmem_empty_bar, (uint32_t)(t & 1), abort_flag)) return false;
                    }
                    tc_fence_after();
                    uint32_t acc = 0u;
                    if (p.nmma_o && !mma_stage(tmem_base + kColAuxO, idesc_o, true, false, p.nmma_o, acc)) return false;
                    acc = 0u;
                    if (p.nmma_l && !mma_stage(tmem_base + kColAuxL, idesc_l, false, !p.lora_kmajor, p.nmma_l, acc)) return false;
                    umma_commit<2>(j == 0 ? tmem_full_bar : aux_ready_bar);
                    return true;
                });
        }
    } else {
        // ------------------------------------------------------------------ epilogue (16 warps = 512 threads per CTA)
        // Warps w, w + 4, w + 8, w + 12 share a TMEM lane quarter; warp group cq = (w - 2) / 4 owns columns
        // [32 cq, 32 cq + 32) of each round, i.e. tile columns 128 j + 32 cq + [0, 32) for j = 0, 1.
        const int q = warp & 3;
        const int cq = (warp - 2) >> 2;
        const int row = q * 32 + lane;
        const bool has_o = p.nmma_o != 0, has_l = p.nmma_l != 0;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t aux_o = lane_addr + kColAuxO + (uint32_t)(cq * 32), aux_l = lane_addr + kColAuxL + (uint32_t)(cq * 32);
        // the scales of this warp's 2 x 32 columns live in the warp's own slice of shared memory (no barrier across
        // warps; with the shared-memory carve-out at its maximum there is hardly any L1 left for global loads)
        float* scale_w = scales + (warp - 2) * 128;      // [round][32]
        float* scale_o = scale_w + 64;

        // A lane stores its own row: 32 rows per store instruction, so the LSU spends one transaction per row whatever
        // the width.  Where Y's base and row pitch allow it, a store is 32 bytes (a whole sector) instead of 16.
        const bool wide = ((reinterpret_cast<uintptr_t>(p.Y) | (uintptr_t)(p.ldy * (p.y_f32 ? 4 : 2))) & 31u) == 0;
        // y = dx (acc dW + acc_o dw_O) + lora_scale acc_l for 8 consecutive columns (h = which 8 of the warp's 32 in round jj)
        auto compute8 = [&](float dxm, int h, int jj, const uint32_t (&a0)[8], const uint32_t (&a1)[8], const uint32_t (&a2)[8], float (&y)[8]) {
#pragma unroll
            for (int i = 0; i < 8; i += 4) {
                const float4 a = *reinterpret_cast<const float4*>(scale_w + jj * 32 + 8 * h + i);
                const float4 b = *reinterpret_cast<const float4*>(scale_o + jj * 32 + 8 * h + i);
                const float fw[4] = {a.x, a.y, a.z, a.w}, fo[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    float w = (float)(int)a0[i + u] * fw[u];
                    if (has_o) w += (float)(int)a1[i + u] * fo[u];
                    float v = dxm * w;
                    if (has_l) v += p.lora_scale * __uint_as_float(a2[i + u]);
                    y[i + u] = v;
                }
            }
        };
        auto store8_f32 = [&](int m, int nc, const float (&y)[8]) {
            float* out = reinterpret_cast<float*>(p.Y) + (int64_t)m * p.ldy + nc;
            if (nc + 8 <= p.N && wide) {
                st_global_v8(out, __float_as_uint(y[0]), __float_as_uint(y[1]), __float_as_uint(y[2]), __float_as_uint(y[3]),
                             __float_as_uint(y[4]), __float_as_uint(y[5]), __float_as_uint(y[6]), __float_as_uint(y[7]));
            } else if (nc + 8 <= p.N && (p.ldy % 4 == 0)) {
                *reinterpret_cast<float4*>(out) = make_float4(y[0], y[1], y[2], y[3]);
                *reinterpret_cast<float4*>(out + 4) = make_float4(y[4], y[5], y[6], y[7]);
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) if (nc + i < p.N) out[i] = y[i];
            }
        };
        // 16 consecutive bf16 columns of row m from column nc, packed two to a word
        auto store16_bf16 = [&](int m, int nc, uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3, uint32_t w4, uint32_t w5, uint32_t w6,
                                uint32_t w7) {
            uint16_t* out = reinterpret_cast<uint16_t*>(p.Y) + (int64_t)m * p.ldy + nc;
            if (nc + 16 <= p.N && wide) {
                st_global_v8(out, w0, w1, w2, w3, w4, w5, w6, w7);
            } else if (nc + 16 <= p.N && (p.ldy % 8 == 0)) {
                *reinterpret_cast<uint4*>(out) = make_uint4(w0, w1, w2, w3);
                *reinterpret_cast<uint4*>(out + 8) = make_uint4(w4, w5, w6, w7);
            } else {
                const uint32_t w[8] = {w0, w1, w2, w3, w4, w5, w6, w7};
#pragma unroll
                for (int i = 0; i < 16; ++i) if (nc + i < p.N) out[i] = (uint16_t)((w[i >> 1] >> ((i & 1) * 16)) & 0xFFFFu);
            }
        };
        auto dbg8 = [&](int m, int nc, const uint32_t (&a0)[8], const uint32_t (&a1)[8]) {     // test aids: the raw integer accumulators
            if (p.dbg_main) {
                int32_t* d = p.dbg_main + (int64_t)m * p.N + nc;
#pragma unroll
                for (int i = 0; i < 8; ++i) if (nc + i < p.N) d[i] = (int32_t)a0[i];
            }
            if (p.dbg_out) {
                int32_t* d = p.dbg_out + (int64_t)m * p.N + nc;
#pragma unroll
                for (int i = 0; i < 8; ++i) if (nc + i < p.N) d[i] = has_o ? (int32_t)a1[i] : 0;
            }
        };
        bool ok = true;
        int t = 0;
        for (int tile = unit; tile < ntiles && ok; tile += nunits, ++t) {
            int tm, tn;
            tile_coords(tile, p.tiles_m, p.tiles_n, p.band_m, tm, tn);
            const int m0 = tm * 256 + (int)rank * kTileM, n0 = tn * TN;
            __syncwarp();
#pragma unroll
            for (int jj = 0; jj < 2; ++jj) {
                const int n = n0 + jj * kF256Round + cq * 32 + lane;
                scale_w[jj * 32 + lane] = n < p.N ? (p.dW ? __ldg(p.dW + n) : 1.0f) : 0.0f;
                scale_o[jj * 32 + lane] = (n < p.N && has_o) ? __ldg(p.dw_O + n) : 0.0f;
            }
            __syncwarp();
            const int m = m0 + row;
            const float dxm = m < p.M ? __ldg(p.dx + m) : 0.0f;
            if (!mbar_wait(tmem_full_bar, (uint32_t)(t & 1), abort_flag)) { ok = false; break; }
            tc_fence_after();
            // columns [0,128) of the tile: main accumulator and round 0, straight from TMEM.  Half of a bf16 result
            // (8 packed words of this thread's 32 columns; more would spill) stays in registers and is stored after the
            // hand-over below: those stores overlap the next tile's main contraction instead of keeping the tensor pipe waiting.
            uint32_t ypk[16];
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                const int nc = n0 + cq * 32 + 8 * h;
                uint32_t a0[8], a1[8], a2[8];
                tmem_ld_32x8(lane_addr + (uint32_t)(cq * 32 + 8 * h), a0);
                if (has_o) tmem_ld_32x8(aux_o + (uint32_t)(8 * h), a1);
                if (has_l) tmem_ld_32x8(aux_l + (uint32_t)(8 * h), a2);
                tmem_ld_wait();
                float y[8];
                compute8(dxm, h, 0, a0, a1, a2, y);
#pragma unroll
                for (int i = 0; i < 4; ++i) ypk[4 * h + i] = pack_bf16x2(y[2 * i], y[2 * i + 1]);
                if (m < p.M && nc < p.N) {
                    if (p.y_f32) store8_f32(m, nc, y);
                    dbg8(m, nc, a0, a1);
                }
                if (h == 1 && !p.y_f32 && m < p.M)
                    store16_bf16(m, n0 + cq * 32, ypk[0], ypk[1], ypk[2], ypk[3], ypk[4], ypk[5], ypk[6], ypk[7]);
            }
            // columns [128,256): the main accumulator goes into registers until round 1 is there
            uint32_t acc[32];
            tmem_ld_32x32(lane_addr + (uint32_t)(kF256Round + cq * 32), acc);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (rank != 0) mbar_arrive_cluster(lead_tmem_empty);
                else mbar_arrive(tmem_empty_bar);
            }
            if (!p.y_f32 && m < p.M) {
                store16_bf16(m, n0 + cq * 32 + 16, ypk[8], ypk[9], ypk[10], ypk[11], ypk[12], ypk[13], ypk[14], ypk[15]);
            }
            if (!mbar_wait(aux_ready_bar, (uint32_t)(t & 1), abort_flag)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                const int nc = n0 + kF256Round + cq * 32 + 8 * h;
                uint32_t a0[8], a1[8], a2[8];
                if (has_o) tmem_ld_32x8(aux_o + (uint32_t)(8 * h), a1);
                if (has_l) tmem_ld_32x8(aux_l + (uint32_t)(8 * h), a2);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 8; ++i) a0[i] = acc[8 * h + i];
                float y[8];
                compute8(dxm, h, 1, a0, a1, a2, y);
#pragma unroll
                for (int i = 0; i < 4; ++i) ypk[4 * h + i] = pack_bf16x2(y[2 * i], y[2 * i + 1]);
                if (m < p.M && nc < p.N) {
                    if (p.y_f32) store8_f32(m, nc, y);
                    dbg8(m, nc, a0, a1);
                }
                if ((h & 1) && !p.y_f32 && m < p.M)
                    store16_bf16(m, nc - 8, ypk[4 * h - 4], ypk[4 * h - 3], ypk[4 * h - 2], ypk[4 * h - 1], ypk[4 * h], ypk[4 * h + 1], ypk[4 * h + 2],
                                 ypk[4 * h + 3]);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (rank != 0) mbar_arrive_cluster(lead_aux_free);
                else mbar_arrive(aux_free_bar);
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
