// Grad-input GEMM of the backward with the frozen INT8 weight expanded to bf16 INSIDE the kernel:
//   dXhat = dY Wd,  Wd[n][k] = bf16(Wq[n][k] * dW[n])      (one fp32 product, one rounding to bf16 per element)
// No dequantized copy of the weight exists in global memory: only the codes Wq [N][K] are read (half the bytes of a
// bf16 copy), in place, with the contraction index n as the row.
//
//   warp 0        : TMA producer - dY tiles (K-major A operand) and RAW INT8 weight tiles into a ring of stages
//   warp 1        : TMEM allocation + tcgen05.mma issue (the leader's, for the CTA pair)
//   warps 2..5    : epilogue - tcgen05.ld, bf16 stores of dX, fp32 stores of the outlier partial products
//   warps 6..21   : converters - raw INT8 tile -> bf16 B operand tile in the layout the MMA reads
//
// Two rings per CTA.  The IN ring (as many slots as fit, 7 on the benchmark shapes) receives what TMA brings: A = 128 rows
// of dY x 64 contraction elements (16 KB) and RAW = 64 contraction rows x 128 INT8 codes (8 KB, 128-byte swizzle, as TMA
// wrote it), plus the 64 step sizes dW[n] of those rows.  It is deep because it has to cover the latency of HBM.  The B
// ring (4 slots of 16 KB) holds this CTA's half of the tile's output columns x 64 contraction rows as bf16 in the MN-major
// 128-byte-swizzled layout the MMA reads (two boxes of 64 rows x 128 bytes); it is short because a slot lives only from
// its conversion to the completion of the MMAs that read it.  Every k-block takes the next slot of both rings.
// Barriers: full (leader, per IN slot: the A-region tiles of both CTAs have landed), rawfull (own CTA, per IN slot: its
// raw tile and step sizes have landed), conv (leader, per B slot: the two converter warps of the slot's group, in both
// CTAs, have written B), empty / bfree (both CTAs, per IN / B slot: the MMAs that read the slot have completed).
//
// The sixteen converter warps form four groups of four; group g converts every fourth k-block (block u with u % 4 = g)
// into B slot g, so four blocks are being converted at any time: what bounds a group is the LATENCY of one block (loads,
// a dependent chain of conversions, stores, the proxy fence, the arrival), not the instruction rate.  Inside a group a
// thread owns half of one contraction row of the block (row = 16 * warp of the group + lane % 16; 64 codes): four times
// a 16-byte shared-memory load, 16 x (byte -> fp32 -> * dW[n] -> bf16), two 16-byte stores.  Eight consecutive lanes touch
// eight consecutive rows, whose 16-byte chunks the swizzle spreads over all banks: loads and stores are conflict-free.  The bytes become floats without a conversion
// instruction: (code + 128) is placed in the low mantissa byte of 2^23, and subtracting 2^23 + 128 is exact.
// The writes are made visible to the tensor pipe with fence.proxy.async before the arrival on conv.
//
// Column tiles: tiles_main tiles of tile_n columns over the K columns of dX, then (with an outlier set) tiles_p tiles
// over the nOp columns of wd = bf16(wq_O * dw_O), expanded by the same converters from the codes wq_O [N][nOp] and the
// step sizes dw_O.  Eq. 5 needs, for the columns of O, the partial products separately: P2 = dY wd comes from those tiles;
// P1 = (dY Wd + G A^T)[:, O] is copied out of the main tiles' accumulators by the epilogue (a bit mask over the
// columns, built once per CTA in shared memory, says which columns of a 32-column chunk belong to O).  The fix-up
// kernel then forms dX[:, O_i] = ((P1 - G A^T) + P2) / s_i + G A^T.
// LoRA: + G A^T as one more block per main tile, accumulating into the same accumulator; both operands come by TMA, each
// into the A region of an IN slot of its own (the B ring belongs to the converters alone, so that everybody who waits
// on one of its barriers sees every one of its phases).
// CTA-pair protocol, accumulator double-buffering, tile order, bounded waits and the exit path: as in umma_gemm.cuh.
#pragma once

#include "umma_gemm.cuh"

namespace quaff {

constexpr int kBxConvWarps = 16;
constexpr int kBxThreads = 64 + 128 + kBxConvWarps * 32;            // producer, MMA, four epilogue warps, sixteen converter warps
constexpr int kBxRawBytes = 64 * 128;
constexpr int kBxBBytes = 2 * kAtomBytes;
constexpr int kBxInBytes = kABytes + kBxRawBytes;                   // one slot of the IN ring: 24 KB
constexpr int kBxBSlots = 4;                                       // = converter groups: group g writes B slot g
constexpr int kBxBarrierBytes = 512;

struct BxSmem {
    uint64_t full[kMaxStages];
    uint64_t rawfull[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t conv[kBxBSlots];
    uint64_t bfree[kBxBSlots];
    uint64_t tmem_full, tmem_empty;
    uint32_t tmem_base;
    AbortCtl abort;
};
static_assert(sizeof(BxSmem) <= kBxBarrierBytes, "barrier block");

struct BxParams {
    CUtensorMap map_dy;      // dY [M][N] bf16: boxes of 128 rows x 64 elements
    CUtensorMap map_wq;      // Wq [N][K] INT8, rows = contraction index: boxes of 64 rows x 128 bytes
    CUtensorMap map_wo;      // wq_O [N][nOp] INT8, rows = contraction index: boxes of 64 rows x 128 bytes
    CUtensorMap map_g;       // G [M][r] bf16: boxes of 128 rows x 64 elements
    CUtensorMap map_a;       // LoRA A [K][r] bf16: boxes of tile_n / 2 rows x 64 elements
    int M, N, K;             // tokens, contraction length (c_out), output columns (c_in)
    int nblk, nmma_last;     // k-blocks of 64 contraction rows per tile; MMAs of the last one (1..4)
    int nmma_l;              // MMAs of the LoRA stage (rp / 16), 0 = no LoRA
    int tiles_m, tiles_main, tiles_p;
    int band_m;
    int tile_n;              // output columns per main tile: 128, 192 or 256
    int tile_np;             // output columns per tile over wd: 128 or 256 (each CTA supplies whole 64-column boxes)
    int nO, nOp;
    int nstages;             // slots of the IN ring
    int mask_words;          // ceil(K / 32)
    const float* dW;         // [N]
    const float* dw_O;       // [N]
    const int32_t* O_idx;    // [nO] sorted
    uint16_t* dX;
    int64_t lddx;
    float* P;                // [M][2 nOp]: P1 in columns [0, nOp), P2 in [nOp, 2 nOp)
    int32_t* status;
};

// 16 INT8 codes (one 16-byte word) times `scale` -> 16 bf16 (two 16-byte words)
__device__ __forceinline__ void expand16(const uint4& raw, float scale, uint4& lo, uint4& hi) {
    const uint32_t w[4] = {raw.x ^ 0x80808080u, raw.y ^ 0x80808080u, raw.z ^ 0x80808080u, raw.w ^ 0x80808080u};   // code + 128
    uint32_t o[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        // byte b of w[i] into the low mantissa byte of 2^23: the float 2^23 + (code + 128); minus (2^23 + 128) is the code, exactly
        const float c0 = __fsub_rn(__uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7650)), 8388736.0f);
        const float c1 = __fsub_rn(__uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7651)), 8388736.0f);
        const float c2 = __fsub_rn(__uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7652)), 8388736.0f);
        const float c3 = __fsub_rn(__uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7653)), 8388736.0f);
        o[2 * i] = pack_bf16x2(__fmul_rn(c0, scale), __fmul_rn(c1, scale));
        o[2 * i + 1] = pack_bf16x2(__fmul_rn(c2, scale), __fmul_rn(c3, scale));
    }
    lo = make_uint4(o[0], o[1], o[2], o[3]);
    hi = make_uint4(o[4], o[5], o[6], o[7]);
}

__global__ void __launch_bounds__(kBxThreads, 1) bwd_expand_kernel(const __grid_constant__ BxParams p) {
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t raw_addr = smem_u32(smem_dyn);
    const uint32_t in_base = (raw_addr + 1023u) & ~1023u;                     // IN ring: nstages slots of [A | RAW]
    unsigned char* aligned = smem_dyn + (in_base - raw_addr);
    const int nstages = p.nstages;
    const uint32_t b_base = in_base + (uint32_t)nstages * kBxInBytes;         // B ring: kBxBSlots slots
    unsigned char* b_ptr = aligned + (size_t)nstages * kBxInBytes;
    BxSmem* sm = reinterpret_cast<BxSmem*>(b_ptr + (size_t)kBxBSlots * kBxBBytes);
    uint32_t* omask = reinterpret_cast<uint32_t*>(reinterpret_cast<unsigned char*>(sm) + kBxBarrierBytes);   // [mask_words]
    uint32_t* obase = omask + p.mask_words;                                                                 // [mask_words]
    float* sc_ring = reinterpret_cast<float*>(obase + p.mask_words + ((4 - ((2 * p.mask_words) & 3)) & 3)); // [nstages][64], 16-byte aligned
    volatile AbortCtl* abort_flag = &sm->abort;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int unit = (int)(blockIdx.x >> 1), nunits = (int)(gridDim.x >> 1);
    const int tiles_n = p.tiles_main + p.tiles_p;
    const int ntiles = p.tiles_m * tiles_n;
    const int half_n = p.tile_n >> 1;                    // output columns of a main tile that this CTA supplies
    const int half_np = p.tile_np >> 1;                  // ... of a tile over wd
    const uint32_t full0 = smem_u32(&sm->full[0]), rawfull0 = smem_u32(&sm->rawfull[0]), empty0 = smem_u32(&sm->empty[0]);
    const uint32_t conv0 = smem_u32(&sm->conv[0]), bfree0 = smem_u32(&sm->bfree[0]);
    const uint32_t tmem_full_bar = smem_u32(&sm->tmem_full), tmem_empty_bar = smem_u32(&sm->tmem_empty);
    const uint32_t lead_full0 = mapa_shared(full0, 0);
    const uint32_t lead_conv0 = mapa_shared(conv0, 0);
    static_assert(kBxConvWarps == 4 * kBxBSlots, "four converter warps per group, one group per B slot");
    const uint32_t lead_tmem_empty = mapa_shared(tmem_empty_bar, 0);

    if (threadIdx.x == 0) {
        for (int s = 0; s < nstages; ++s) {
            mbar_init(full0 + 8u * s, 1);
            mbar_init(rawfull0 + 8u * s, 1);
            mbar_init(empty0 + 8u * s, 1);
        }
        for (int s = 0; s < kBxBSlots; ++s) {
            mbar_init(conv0 + 8u * s, 8);                      // the four warps of the slot's converter group, in both CTAs
            mbar_init(bfree0 + 8u * s, 1);
        }
        mbar_init(tmem_full_bar, 1);
        mbar_init(tmem_empty_bar, 4 * 2);
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

    // Every role walks the same sequence of blocks: per tile nblk converted k-blocks (one IN slot and one B slot each),
    // plus, per main tile with LoRA, one block that takes two IN slots (G, then the rows of A) and no B slot.
    struct Ring {
        uint32_t i = 0, iph = 0, j = 0, jph = 0;
        int n;
        __device__ explicit Ring(int n_) : n(n_) {}
        __device__ void next_in() { if (++i == (uint32_t)n) { i = 0; iph ^= 1u; } }
        __device__ void next_b() { if (++j == (uint32_t)kBxBSlots) { j = 0; jph ^= 1u; } }
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs of the pair)
        if (elect_one()) {
            prefetch_tmap(&p.map_dy); prefetch_tmap(&p.map_wq);
            if (p.tiles_p) prefetch_tmap(&p.map_wo);
            if (p.nmma_l) { prefetch_tmap(&p.map_g); prefetch_tmap(&p.map_a); }
            Ring ring(nstages);
            bool ok = true;
            for (int tile = unit; tile < ntiles && ok; tile += nunits) {
                int tm, tn;
                tile_coords(tile, p.tiles_m, tiles_n, p.band_m, tm, tn);
                const int m0 = tm * 256 + (int)rank * kTileM;
                const bool main_tile = tn < p.tiles_main;
                // first output column of this CTA; the codes and their step sizes
                const int c0 = main_tile ? tn * p.tile_n + (int)rank * half_n : (tn - p.tiles_main) * p.tile_np + (int)rank * half_np;
                const CUtensorMap* map_raw = main_tile ? &p.map_wq : &p.map_wo;
                const float* scales = main_tile ? p.dW : p.dw_O;
                for (int b = 0; b < p.nblk; ++b) {
                    if (!mbar_wait(empty0 + 8u * ring.i, ring.iph ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t dst = in_base + ring.i * kBxInBytes;
                    if (rank == 0) mbar_arrive_expect_tx(full0 + 8u * ring.i, 2u * kABytes);
                    tma_load_2d<2>(dst, &p.map_dy, b * 64, m0, lead_full0 + 8u * ring.i);
                    // this CTA's raw tile and the step sizes of its 64 contraction rows (whole 16-byte pieces of the array
                    // only; the up to three floats of a ragged end are read by the converter threads themselves)
                    const uint32_t sc_bytes = (uint32_t)(min(64, p.N - b * 64) * 4) & ~15u;
                    mbar_arrive_expect_tx(rawfull0 + 8u * ring.i, kBxRawBytes + sc_bytes);
                    tma_load_2d<1>(dst + kABytes, map_raw, c0, b * 64, rawfull0 + 8u * ring.i);
                    if (sc_bytes) bulk_load_1d(smem_u32(sc_ring + ring.i * 64), scales + b * 64, sc_bytes, rawfull0 + 8u * ring.i);
                    ring.next_in();
                }
                if (ok && main_tile && p.nmma_l) {     // LoRA block: G [128 rows][r], then the rows c0.. of A [K][r], an IN slot each
                    if (!mbar_wait(empty0 + 8u * ring.i, ring.iph ^ 1u, abort_flag)) { ok = false; break; }
                    if (rank == 0) mbar_arrive_expect_tx(full0 + 8u * ring.i, 2u * kABytes);
                    tma_load_2d<2>(in_base + ring.i * kBxInBytes, &p.map_g, 0, m0, lead_full0 + 8u * ring.i);
                    ring.next_in();
                    if (!mbar_wait(empty0 + 8u * ring.i, ring.iph ^ 1u, abort_flag)) { ok = false; break; }
                    if (rank == 0) mbar_arrive_expect_tx(full0 + 8u * ring.i, 2u * (uint32_t)half_n * 128u);
                    tma_load_2d<2>(in_base + ring.i * kBxInBytes, &p.map_a, 0, c0, lead_full0 + 8u * ring.i);
                    ring.next_in();
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (the leader's, for the pair)
        if (rank == 0 && elect_one()) {
            Ring ring(nstages);
            bool ok = true;
            int t = 0;
            const uint32_t idesc_mn = umma_idesc(kCFmtF32, kFmtBF16, 256, 0) | ((uint32_t)(p.tile_n >> 3) << 17) | (1u << 16);   // B MN-major
            const uint32_t idesc_k = umma_idesc(kCFmtF32, kFmtBF16, 256, 0) | ((uint32_t)(p.tile_n >> 3) << 17);                 // both K-major
            const uint32_t idesc_p = umma_idesc(kCFmtF32, kFmtBF16, 256, 0) | ((uint32_t)(p.tile_np >> 3) << 17) | (1u << 16);  // tiles over wd
            for (int tile = unit; tile < ntiles && ok; tile += nunits, ++t) {
                int tm, tn;
                tile_coords(tile, p.tiles_m, tiles_n, p.band_m, tm, tn);
                const bool main_tile = tn < p.tiles_main;
                const uint32_t acc = tmem_base + (uint32_t)((t & 1) * 256);
                uint32_t accumulate = 0u;
                for (int b = 0; b < p.nblk; ++b) {
                    if (!mbar_wait(full0 + 8u * ring.i, ring.iph, abort_flag)) { ok = false; break; }
                    if (!mbar_wait(conv0 + 8u * ring.j, ring.jph, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_lo = (((in_base + ring.i * kBxInBytes) & 0x3FFFFu) >> 4) | (1u << 16);
                    const uint32_t b_lo = (((b_base + ring.j * kBxBBytes) & 0x3FFFFu) >> 4) | ((uint32_t)(kAtomBytes >> 4) << 16);
                    const int nmma = (b == p.nblk - 1) ? p.nmma_last : 4;
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (k < nmma) {
                            umma_f16<2>(acc, make_desc(a_lo + 2u * k, kDescHi), make_desc(b_lo + (2048u >> 4) * k, kDescHi), main_tile ? idesc_mn : idesc_p, accumulate);
                            accumulate = 1u;
                        }
                    umma_commit<2>(empty0 + 8u * ring.i);
                    umma_commit<2>(bfree0 + 8u * ring.j);
                    ring.next_in();
                    ring.next_b();
                }
                if (!ok) break;
                // this tile's buffer was last used by tile t - 2 and has been drained (awaited while tile t - 1 was issued);
                // before the next tile may start, the epilogue must be done with tile t - 1
                if (t > 0 && !mbar_wait(tmem_empty_bar, (uint32_t)((t - 1) & 1), abort_flag)) { ok = false; break; }
                if (main_tile && p.nmma_l) {
                    const uint32_t ig = ring.i;
                    if (!mbar_wait(full0 + 8u * ring.i, ring.iph, abort_flag)) { ok = false; break; }
                    ring.next_in();
                    if (!mbar_wait(full0 + 8u * ring.i, ring.iph, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_lo = (((in_base + ig * kBxInBytes) & 0x3FFFFu) >> 4) | (1u << 16);
                    const uint32_t b_lo = (((in_base + ring.i * kBxInBytes) & 0x3FFFFu) >> 4) | (1u << 16);
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (k < p.nmma_l) umma_f16<2>(acc, make_desc(a_lo + 2u * k, kDescHi), make_desc(b_lo + 2u * k, kDescHi), idesc_k, 1u);
                    umma_commit<2>(empty0 + 8u * ig);
                    umma_commit<2>(empty0 + 8u * ring.i);
                    ring.next_in();
                }
                umma_commit<2>(tmem_full_bar);
            }
        }
    } else if (warp < 6) {
        // ------------------------------------------------------------------ epilogue (128 threads per CTA)
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const int et = threadIdx.x - 64;
        // which columns of dX belong to O: one bit per column, and per 32-column word the index in O of its first member
        if (p.nO > 0) {
            for (int w = et; w < p.mask_words; w += 128) { omask[w] = 0u; obase[w] = 0u; }
            named_bar_sync(1, 128);
            for (int i = et; i < p.nO; i += 128) {
                const int k = __ldg(p.O_idx + i);
                atomicOr(&omask[k >> 5], 1u << (k & 31));
                if (i == 0 || (__ldg(p.O_idx + i - 1) >> 5) != (k >> 5)) obase[k >> 5] = (uint32_t)i;
            }
            named_bar_sync(1, 128);
        }
        bool ok = true;
        int t = 0;
        for (int tile = unit; tile < ntiles && ok; tile += nunits, ++t) {
            int tm, tn;
            tile_coords(tile, p.tiles_m, tiles_n, p.band_m, tm, tn);
            const bool main_tile = tn < p.tiles_main;
            const int m = tm * 256 + (int)rank * kTileM + row;
            const int n0 = main_tile ? tn * p.tile_n : (tn - p.tiles_main) * p.tile_np;
            const int ncols = main_tile ? p.K : p.nOp;
            const int width = main_tile ? p.tile_n : p.tile_np;
            if (!mbar_wait(tmem_full_bar, (uint32_t)(t & 1), abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)((t & 1) * 256);
#pragma unroll 1
            for (int c = 0; c < width; c += 32) {
                const int nc = n0 + c;
                if (nc >= ncols) break;              // uniform across the warp
                uint32_t r0[32];
                tmem_ld_32x32(lane_addr + (uint32_t)c, r0);
                tmem_ld_wait();
                if (m >= p.M) continue;
                if (main_tile) {
                    uint16_t* out = p.dX + (int64_t)m * p.lddx + nc;
                    if (nc + 32 <= p.K && (p.lddx % 8 == 0)) {
#pragma unroll
                        for (int j = 0; j < 32; j += 8)
                            *reinterpret_cast<uint4*>(out + j) =
                                make_uint4(pack_bf16x2(__uint_as_float(r0[j]), __uint_as_float(r0[j + 1])),
                                           pack_bf16x2(__uint_as_float(r0[j + 2]), __uint_as_float(r0[j + 3])),
                                           pack_bf16x2(__uint_as_float(r0[j + 4]), __uint_as_float(r0[j + 5])),
                                           pack_bf16x2(__uint_as_float(r0[j + 6]), __uint_as_float(r0[j + 7])));
                    } else {
                        for (int j = 0; j < 32; ++j) if (nc + j < p.K) out[j] = (uint16_t)f32_to_bf16_bits(__uint_as_float(r0[j]));
                    }
                    const uint32_t mask = p.nO > 0 ? omask[nc >> 5] : 0u;
                    if (mask) {                      // uniform across the warp: copy the columns of O out in fp32
                        float* pout = p.P + (int64_t)m * (2 * p.nOp) + obase[nc >> 5];
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if ((mask >> j) & 1u) pout[__popc(mask & ((1u << j) - 1u))] = __uint_as_float(r0[j]);
                    }
                } else {
                    float* pout = p.P + (int64_t)m * (2 * p.nOp) + p.nOp + nc;
                    for (int j = 0; j < 32; ++j) if (nc + j < p.nOp) pout[j] = __uint_as_float(r0[j]);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (rank != 0) mbar_arrive_cluster(lead_tmem_empty);
                else mbar_arrive(tmem_empty_bar);
            }
        }
    } else {
        // ------------------------------------------------------------------ converters (16 warps per CTA, 4 groups of 4)
        const int cw = warp - 6;
        const uint32_t grp = (uint32_t)(cw >> 2);        // this warp's group = the B slot it writes
        const int crow = (cw & 3) * 16 + (lane & 15);    // contraction row of the block this thread owns half of
        const int ghalf = lane >> 4;                     // which half of the row: 16-code groups 4 ghalf .. 4 ghalf + 3
        const uint32_t sw = (uint32_t)(crow & 7);
        Ring ring(nstages);
        uint32_t raw_parity = 0u;                        // per IN slot: parity of the next completion of its rawfull barrier (LoRA blocks
                                                         // take IN slots without using it, so it does not follow the ring's wraps)
        bool ok = true;
        for (int tile = unit; tile < ntiles && ok; tile += nunits) {
            int tm, tn;
            tile_coords(tile, p.tiles_m, tiles_n, p.band_m, tm, tn);
            const bool main_tile = tn < p.tiles_main;
            const int ngroups16 = (main_tile ? half_n : half_np) >> 4;      // 16-code groups of a row that the tile uses (4, 6 or 8)
            const float* scales = main_tile ? p.dW : p.dw_O;
            for (int b = 0; b < p.nblk; ++b) {
                const uint32_t in_slot = ring.i;
                const uint32_t par = (raw_parity >> in_slot) & 1u;
                raw_parity ^= 1u << in_slot;
                if (ring.j == grp) {
                    if (!mbar_wait(rawfull0 + 8u * in_slot, par, abort_flag)) { ok = false; break; }
                    if (!mbar_wait(bfree0 + 8u * grp, ring.jph ^ 1u, abort_flag)) { ok = false; break; }
                    // the step size of this thread's row: from the ring (no global load may be in flight when the proxy
                    // fence below is reached: it waits for every outstanding memory operation of the thread)
                    const int nrow = b * 64 + crow;
                    const int staged = b * 64 + ((min(64, p.N - b * 64) * 4) >> 4) * 4;     // rows below this index have their step size in the ring
                    const float scale = nrow < staged ? sc_ring[in_slot * 64 + crow] : (nrow < p.N ? __ldg(scales + nrow) : 0.0f);
                    const unsigned char* rawt = aligned + (size_t)in_slot * kBxInBytes + kABytes + crow * 128;
                    unsigned char* brow = b_ptr + (size_t)grp * kBxBBytes + crow * 128;
#pragma unroll
                    for (int gg = 0; gg < 4; ++gg) {
                        const int g = 4 * ghalf + gg;
                        if (g >= ngroups16) break;
                        const uint4 codes = *reinterpret_cast<const uint4*>(rawt + (((uint32_t)g ^ sw) << 4));
                        uint4 lo, hi;
                        expand16(codes, scale, lo, hi);
                        unsigned char* box = brow + (g >> 2) * kAtomBytes;
                        *reinterpret_cast<uint4*>(box + (((uint32_t)(2 * (g & 3)) ^ sw) << 4)) = lo;
                        *reinterpret_cast<uint4*>(box + (((uint32_t)(2 * (g & 3) + 1) ^ sw) << 4)) = hi;
                    }
                    fence_proxy_async();                 // generic-proxy writes -> visible to the tensor pipe's reads
                    __syncwarp();
                    if (lane == 0) {
                        if (rank != 0) mbar_arrive_cluster(lead_conv0 + 8u * grp);
                        else mbar_arrive(conv0 + 8u * grp);
                    }
                }
                ring.next_in();
                ring.next_b();
            }
            if (ok && main_tile && p.nmma_l) { ring.next_in(); ring.next_in(); }     // the LoRA block of the tile
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
