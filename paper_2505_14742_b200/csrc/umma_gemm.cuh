// Persistent, warp-specialised tcgen05 GEMM pipeline shared by the forward (Eq. 9 + LoRA), the
// grad-input GEMM and the skinny LoRA GEMMs (T = X A, G = dY B^T, dA = X^T G, dB = T^T dY).
//
//   warp 0      : TMA producer (one elected lane) - 128-byte-swizzled operand tiles into a ring of stages
//   warp 1      : TMEM allocation + MMA issue (one elected lane) - tcgen05.mma, accumulators in TMEM
//   warps 2..5  : epilogue - tcgen05.ld of the finished accumulators, dequantization / conversion, stores
//
// Template parameters: EPI (which epilogue), CTAS (1, or 2 = a CTA pair on two SMs that shares one
// 256-row output tile through tcgen05 cta_group::2) and TN (output columns per tile: 128, 256, and 192 for
// the grad-input GEMM).
//
// CTA pair (CTAS = 2, a cluster of two): each CTA loads its own 128 rows of A and its own half
// (TN / 2 output columns) of B into its own shared memory, at the same offsets in both CTAs.  The
// TMA loads of both CTAs signal the "full" barrier of the leader (cluster rank 0), whose MMA warp
// issues every tcgen05.mma for the pair; the accumulator rows 0..127 land in the leader's TMEM and
// rows 128..255 in its peer's.  tcgen05.commit multicasts the "stage free" and "accumulator ready"
// arrivals to both CTAs; the peer's epilogue warps report "accumulator drained" to the leader with a
// remote mbarrier arrive.  Per output element each SM reads half as many operand bytes as it would
// alone, which is what lets the stage ring cover the latency of the loads.  No TMA multicast anywhere.
//
// An output tile is (128 * CTAS) rows x TN columns.  Its contraction is a list of up to three PHASES,
// each a run of k-blocks with its own pair of tensor maps, operand type and accumulator:
//   forward : main INT8 (over K) -> slot 0 | outlier INT8 (over nOp) -> slot 1 | LoRA bf16 (over r) -> slot 2
//   backward: main bf16 (over N) -> slot 0 | LoRA bf16 (over r) -> slot 0 (accumulating)
//   skinny  : one bf16 phase over a slice of the contraction (split-K); partial sums go to a workspace
// Every k-block is one stage: 128 bytes of contraction per row (128 INT8 or 64 bf16 elements).
// Each operand is either K-major (rows = output index, the 128 bytes run along the contraction) or
// MN-major (rows = contraction index, the 128 bytes run along 64 output indices; used where the
// contraction is the slow axis of the caller's matrix: the dequantized weight and LoRA B in their
// stored orientation, X^T G and T^T dY).
// Tails need no special case: TMA zero-fills out-of-range rows and columns, and the epilogue masks stores.
//
// TMEM (512 columns): slot 0 is double-buffered at columns [0,TN) and [TN,2TN) so the main
// contraction of tile t+1 overlaps the epilogue of tile t; with TN = 128, slots 1 and 2 live at
// [256,384) and [384,512) and are written only after the epilogue of the previous tile has drained them.
// Measured on B200, a tcgen05.mma of a CTA pair (M = 256, 32 bytes of contraction) costs about 60 + N/2
// clocks (N = 128: 125, 192: 165, 256: 190): the wider the tile, the cheaper the column.  Two 256-column
// buffers fill TMEM, so TN = 256 is for contractions with a single accumulator (grad-input; forward
// without outliers and LoRA); the forward with its three accumulators runs TN = 128 here or the
// 192-column kernel of fwd192.cuh.
//
// The producer and the MMA issuer are single threads; their per-k-block instruction count bounds the
// tensor-pipe utilisation, so everything that does not change inside a phase is hoisted out of the
// k-block loops.
//
// Every wait is bounded (see mbar_wait); on expiry all roles fall through to the common exit, TMEM is
// freed, and QUAFF_ERR_TIMEOUT is written to the status word.
#pragma once

#include "common.cuh"

namespace quaff {

constexpr int kTileM = 128;                       // accumulator rows per CTA
constexpr int kABytes = 128 * 128;                // A region of a stage: 128 rows x 128 bytes
constexpr int kAtomBytes = 64 * 128;              // one MN-major box: 64 contraction rows x 128 bytes
constexpr int kGemmThreads = 192;
constexpr int kMaxPhases = 3;
constexpr int kMaxStages = 12;
constexpr int kSmemLimit = 232448;                // opt-in dynamic shared memory per CTA on sm_100

struct GemmPhase {
    CUtensorMap map_a;   // K-major: [rows = output rows][cols = contraction]; MN-major: [rows = contraction][cols = output rows]
    CUtensorMap map_b;   // same, for the output columns
    int nblk;            // k-blocks per tile in this phase
    int is_i8;           // 1: kind::i8 (128 elements per block, 32 per MMA); 0: kind::f16 bf16 (64 per block, 16 per MMA)
    int nmma_last;       // MMAs issued for the last k-block (1..4); every other block issues 4
    int acc_slot;        // 0 main (double-buffered), 1, 2 auxiliary
    int fresh;           // 1: the first MMA of the phase overwrites the accumulator
    int tn_limit;        // the phase runs only for column tiles tn < tn_limit
    int a_mn, b_mn;      // operand is MN-major (1) or K-major (0)
    int n_mma;           // N of the MMA instruction (multiple of 16, <= 256); each CTA of a pair supplies n_mma / CTAS columns of B
    int b_boxes;         // MN-major B: boxes of 64 output columns per CTA
    uint32_t tx_bytes;   // bytes that land in one stage of ONE CTA
    int kblk_per_tn;     // split-K: first k-block of a tile is tn * kblk_per_tn (0 otherwise)
    int b_per_tn;        // B offset (rows if K-major, columns if MN-major) per tn: the tile width, or 0 for split-K
};

enum { EPI_FWD = 0, EPI_BWD = 1, EPI_PART = 2 };

// Tile order.  The tiles that run at the same time should share operands in L2: the row tiles are cut into
// BANDS of band_m row tiles; inside a band the order is column tile by column tile, row tiles fastest, so that the
// ~74 concurrent tiles cover one band of A (sized by the host to stay L2-resident) and a few column panels of B.
__device__ __forceinline__ void tile_coords(int tile, int tiles_m, int tiles_n, int band_m, int& tm, int& tn) {
    const int per_band = band_m * tiles_n;
    const int band = tile / per_band, rem = tile - band * per_band;
    const int rows = min(band_m, tiles_m - band * band_m);     // the last band may be shorter
    tn = rem / rows;
    tm = band * band_m + (rem - tn * rows);
}

struct GemmParams {
    GemmPhase ph[kMaxPhases];
    int nphases;
    int M, N;            // output extent (rows, columns)
    int tiles_m, tiles_n;
    int band_m;          // row tiles per band of the tile order (tiles_m: one band)
    int tile_n;          // EPI_BWD: output columns per tile, a multiple of 64 up to TN (0: TN); other epilogues: TN
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
    // partial-sum epilogue (split-K): part[(tn * M + m) * part_ld + j] = accumulator[m][j], j < part_cols
    float* part;
    int part_ld;
    int part_cols;
};

struct GemmSmem {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full;
    uint64_t tmem_empty;
    uint32_t tmem_base;
    AbortCtl abort;
};

template <int EPI, int CTAS, int TN>
struct GemmCfg {
    // B region of a stage, per CTA: whole boxes of 64 output columns (an MN-major operand is loaded box by box;
    // the grad-input GEMM may use part of the last box)
    static constexpr int kBBytes = ((TN / CTAS + 63) / 64) * 64 * 128;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kScaleBytes = (EPI == EPI_FWD) ? 2 * 2 * TN * 4 : 0;   // [2 buffers][dW | dw_O][TN]
    static constexpr int kFixed = 1024 + (int)sizeof(GemmSmem) + kScaleBytes;
    // The skinny split-K GEMMs stream one operand from HBM and are bound by the latency of those loads: six stages
    // (measured: 4 -> 6 stages takes T = X A at 8192 x 11008 from 50 to 46 us, more gives nothing); half of TMEM, so that
    // a kernel that follows can allocate its own while this one drains.
    static constexpr int kStageCap = (EPI == EPI_PART) ? 6 : kMaxStages;
    static constexpr int kTmemCols = (EPI == EPI_PART) ? 2 * TN : 512;
    static constexpr int kStagesFit = (kSmemLimit - kFixed) / kStageBytes;
    static constexpr int kStages = kStagesFit < kStageCap ? kStagesFit : kStageCap;
    static constexpr size_t kSmemBytes = (size_t)kFixed + (size_t)kStages * kStageBytes;
};

// high word of the shared-memory matrix descriptor: stride byte offset 1024 (8 rows x 128 bytes),
// descriptor version 1, SWIZZLE_128B
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);

__device__ __forceinline__ uint64_t make_desc(uint32_t lo, uint32_t hi) {
    return (static_cast<uint64_t>(hi) << 32) | lo;
}

// Grad-input epilogue: W accumulator columns of row m, starting at column nc.  Columns below n_split go to dX (bf16);
// columns from p_col0 on (a multiple of 32) are outlier partial products and go to P (f32); in between: padding.
template <int W>
__device__ __forceinline__ void bwd_store_chunk(const GemmParams& p, int m, int nc, const uint32_t (&r0)[W]) {
    if (nc < p.p_col0) {
        uint16_t* out = p.dX + (int64_t)m * p.lddx + nc;
        if (nc + W <= p.n_split && (p.lddx % 8 == 0)) {
#pragma unroll
            for (int j = 0; j < W; j += 8)
                *reinterpret_cast<uint4*>(out + j) =
                    make_uint4(pack_bf16x2(__uint_as_float(r0[j]), __uint_as_float(r0[j + 1])),
                               pack_bf16x2(__uint_as_float(r0[j + 2]), __uint_as_float(r0[j + 3])),
                               pack_bf16x2(__uint_as_float(r0[j + 4]), __uint_as_float(r0[j + 5])),
                               pack_bf16x2(__uint_as_float(r0[j + 6]), __uint_as_float(r0[j + 7])));
        } else {
            for (int j = 0; j < W; ++j) if (nc + j < p.n_split) out[j] = (uint16_t)f32_to_bf16_bits(__uint_as_float(r0[j]));
        }
    } else {
        float* out = p.P + (int64_t)m * p.ldp + (nc - p.p_col0);
        for (int j = 0; j < W; ++j) if (nc + j < p.N) out[j] = __uint_as_float(r0[j]);
    }
}

template <int EPI, int CTAS, int TN>
__global__ void __launch_bounds__(kGemmThreads, 1) umma_gemm_kernel(const __grid_constant__ GemmParams p) {
    using Cfg = GemmCfg<EPI, CTAS, TN>;
    constexpr int kStages = Cfg::kStages;
    constexpr int kStageBytes = Cfg::kStageBytes;
    static_assert(CTAS == 1 || CTAS == 2, "one CTA or a CTA pair");
    static_assert(TN == 128 || TN == 256, "output-column tile");   // TN = 256: slot 0 only (no room for auxiliary accumulators)
    // The grad-input epilogue takes its tile width at run time (p.tile_n <= TN): the two buffers of its accumulator
    // then sit at columns 0 and TN.
    constexpr int kAccStride = TN;

    extern __shared__ unsigned char smem_dyn[];
    const uint32_t raw = smem_u32(smem_dyn);
    const uint32_t tiles_base = (raw + 1023u) & ~1023u;
    unsigned char* aligned = smem_dyn + (tiles_base - raw);
    GemmSmem* sm = reinterpret_cast<GemmSmem*>(aligned + (size_t)kStages * kStageBytes);
    float* scales = reinterpret_cast<float*>(sm + 1);                 // EPI_FWD only: [2][2][TN]
    volatile AbortCtl* abort_flag = &sm->abort;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = CTAS == 2 ? cluster_ctarank() : 0u;        // 0 = leader of the pair
    const int unit = CTAS == 2 ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;           // tile-processing unit (CTA or pair)
    const int nunits = CTAS == 2 ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    const int ntiles = p.tiles_m * p.tiles_n;
    const uint32_t full0 = smem_u32(&sm->full[0]);
    const uint32_t empty0 = smem_u32(&sm->empty[0]);
    const uint32_t tmem_full_bar = smem_u32(&sm->tmem_full);
    const uint32_t tmem_empty_bar = smem_u32(&sm->tmem_empty);
    // barriers of the leader as seen from this CTA (its own, when it is the leader)
    const uint32_t lead_full0 = CTAS == 2 ? mapa_shared(full0, 0) : full0;
    const uint32_t lead_tmem_empty = CTAS == 2 ? mapa_shared(tmem_empty_bar, 0) : tmem_empty_bar;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full0 + 8u * s, 1);
            mbar_init(empty0 + 8u * s, 1);
        }
        mbar_init(tmem_full_bar, 1);
        mbar_init(tmem_empty_bar, 4 * CTAS);
        sm->abort.flag = 0;
        sm->abort.peer = CTAS == 2 ? mapa_shared(smem_u32(&sm->abort.flag), rank ^ 1u) : 0u;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc<CTAS>(smem_u32(&sm->tmem_base), Cfg::kTmemCols);
        tmem_relinquish<CTAS>();
    }
    pdl_launch_dependents();
    tc_fence_before();
    __syncthreads();
    if (CTAS == 2) cluster_sync();      // the peer's barriers exist before anything can signal them
    tc_fence_after();
    const uint32_t tmem_base = sm->tmem_base;
    pdl_wait();                         // everything above overlapped the previous kernel; global memory only from here on

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs of a pair)
        if (elect_one()) {
            for (int i = 0; i < p.nphases; ++i) {
                prefetch_tmap(&p.ph[i].map_a);
                prefetch_tmap(&p.ph[i].map_b);
            }
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            for (int tile = unit; tile < ntiles && ok; tile += nunits) {
                int tm, tn;
                tile_coords(tile, p.tiles_m, p.tiles_n, p.band_m, tm, tn);
                const int m0 = tm * (kTileM * CTAS) + (int)rank * kTileM;
                for (int i = 0; i < p.nphases && ok; ++i) {
                    const GemmPhase& ph = p.ph[i];
                    if (tn >= ph.tn_limit) continue;
                    const CUtensorMap* map_a = &ph.map_a;
                    const CUtensorMap* map_b = &ph.map_b;
                    const int nblk = ph.nblk;
                    const uint32_t tx = ph.tx_bytes * CTAS;
                    const int n0 = tn * ph.b_per_tn + (int)rank * (ph.n_mma / CTAS);
                    const int kstep = ph.is_i8 ? 128 : 64;
                    int kc = tn * ph.kblk_per_tn * kstep;      // contraction coordinate of the next block
                    const bool a_mn = ph.a_mn != 0, b_mn = ph.b_mn != 0;
                    const int b_boxes = ph.b_boxes;
                    for (int b = 0; b < nblk; ++b, kc += kstep) {
                        if (!mbar_wait(empty0 + 8u * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                        const uint32_t bar = lead_full0 + 8u * stage;
                        const uint32_t dst = tiles_base + stage * kStageBytes;
                        if (rank == 0) mbar_arrive_expect_tx(full0 + 8u * stage, tx);
                        if (!a_mn) {
                            tma_load_2d<CTAS>(dst, map_a, kc, m0, bar);
                        } else {   // two boxes of 64 output rows x 64 contraction rows
                            tma_load_2d<CTAS>(dst, map_a, m0, kc, bar);
                            tma_load_2d<CTAS>(dst + kAtomBytes, map_a, m0 + 64, kc, bar);
                        }
                        if (!b_mn) {
                            tma_load_2d<CTAS>(dst + kABytes, map_b, kc, n0, bar);
                        } else {
                            for (int x = 0; x < b_boxes; ++x)
                                tma_load_2d<CTAS>(dst + kABytes + x * kAtomBytes, map_b, n0 + 64 * x, kc, bar);
                        }
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (the leader's, for the pair)
        if (rank == 0 && elect_one()) {
            uint32_t stage = 0, phase = 0;
            bool ok = true;
            int t = 0;
            for (int tile = unit; tile < ntiles && ok; tile += nunits, ++t) {
                int tm, tn;
                tile_coords(tile, p.tiles_m, p.tiles_n, p.band_m, tm, tn);
                for (int i = 0; i < p.nphases && ok; ++i) {
                    const GemmPhase& ph = p.ph[i];
                    if (tn < ph.tn_limit) {
                        const uint32_t acc = tmem_base + (ph.acc_slot == 0 ? (uint32_t)((t & 1) * kAccStride) : (uint32_t)((ph.acc_slot + 1) * TN));
                        const int nblk = ph.nblk;
                        const int nmma_last = ph.nmma_last;
                        const bool i8 = ph.is_i8 != 0;
                        // K-major: the leading byte offset is unused (encoded 1), one MMA advances 32 bytes inside the
                        // swizzled row.  MN-major: boxes of 64 output indices are kAtomBytes apart (leading byte
                        // offset); one MMA consumes 16 contraction rows = 2048 bytes.
                        const uint32_t a_lbo = ph.a_mn ? ((uint32_t)(kAtomBytes >> 4) << 16) : (1u << 16);
                        const uint32_t b_lbo = ph.b_mn ? ((uint32_t)(kAtomBytes >> 4) << 16) : (1u << 16);
                        const uint32_t a_kadv = ph.a_mn ? (2048u >> 4) : (32u >> 4);
                        const uint32_t b_kadv = ph.b_mn ? (2048u >> 4) : (32u >> 4);
                        const uint32_t idesc = (i8 ? umma_idesc(kCFmtS32, kFmtS8, kTileM * CTAS, 0) : umma_idesc(kCFmtF32, kFmtBF16, kTileM * CTAS, 0)) |
                                               ((uint32_t)(ph.n_mma >> 3) << 17) | (ph.a_mn ? (1u << 15) : 0u) | (ph.b_mn ? (1u << 16) : 0u);
                        uint32_t accumulate = ph.fresh ? 0u : 1u;
                        for (int b = 0; b < nblk; ++b) {
                            if (!mbar_wait(full0 + 8u * stage, phase, abort_flag)) { ok = false; break; }
                            tc_fence_after();
                            const uint32_t s_lo = ((tiles_base + stage * kStageBytes) & 0x3FFFFu) >> 4;
                            const uint32_t a_lo = s_lo | a_lbo;
                            const uint32_t b_lo = (s_lo + (kABytes >> 4)) | b_lbo;
                            const int nmma = (b == nblk - 1) ? nmma_last : 4;
                            if (i8) {
#pragma unroll
                                for (int k = 0; k < 4; ++k)
                                    if (k < nmma) { umma_i8<CTAS>(acc, make_desc(a_lo + k * a_kadv, kDescHi), make_desc(b_lo + k * b_kadv, kDescHi), idesc, accumulate); accumulate = 1u; }
                            } else {
#pragma unroll
                                for (int k = 0; k < 4; ++k)
                                    if (k < nmma) { umma_f16<CTAS>(acc, make_desc(a_lo + k * a_kadv, kDescHi), make_desc(b_lo + k * b_kadv, kDescHi), idesc, accumulate); accumulate = 1u; }
                            }
                            umma_commit<CTAS>(empty0 + 8u * stage);
                            if (++stage == kStages) { stage = 0; phase ^= 1u; }
                        }
                    }
                    // After the main phase: the auxiliary accumulators of this tile, and the main buffer of
                    // the next tile, may be written only once the epilogue has drained the previous tile.
                    if (ok && i == 0 && t > 0 && !mbar_wait(tmem_empty_bar, (uint32_t)((t - 1) & 1), abort_flag)) ok = false;
                }
                if (!ok) break;
                umma_commit<CTAS>(tmem_full_bar);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (128 threads per CTA)
        const int q = warp & 3;                  // TMEM lane quarter this warp may read
        const int row = q * 32 + lane;
        const int et = threadIdx.x - 64;         // 0..127
        bool ok = true;
        int t = 0;
        for (int tile = unit; tile < ntiles && ok; tile += nunits, ++t) {
            int tm, tn;
            tile_coords(tile, p.tiles_m, p.tiles_n, p.band_m, tm, tn);
            const int tn_cols = (EPI == EPI_BWD && p.tile_n) ? p.tile_n : TN;
            const int m0 = tm * (kTileM * CTAS) + (int)rank * kTileM, n0 = tn * tn_cols;
            const int buf = t & 1;
            float* scale_w = scales + buf * 2 * TN;
            float* scale_o = scale_w + TN;
            if (EPI == EPI_FWD) {
                for (int c = et; c < TN; c += 128) {
                    const int n = n0 + c;
                    scale_w[c] = n < p.N ? p.dW[n] : 0.0f;
                    scale_o[c] = (n < p.N && p.has_outlier) ? p.dw_O[n] : 0.0f;
                }
                named_bar_sync(1, 128);
            }
            if (!mbar_wait(tmem_full_bar, (uint32_t)(t & 1), abort_flag)) { ok = false; break; }
            tc_fence_after();
            const int m = m0 + row;
            const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
            if (EPI == EPI_PART) {
                // accumulator columns [0, part_cols) of this split -> workspace
#pragma unroll 1
                for (int c = 0; c * 32 < p.part_cols; ++c) {
                    uint32_t r0[32];
                    tmem_ld_32x32(lane_addr + (uint32_t)(buf * TN + c * 32), r0);
                    tmem_ld_wait();
                    if (m < p.M) {
                        float* out = p.part + ((int64_t)tn * p.M + m) * p.part_ld + c * 32;
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            if (c * 32 + j < p.part_cols)
                                *reinterpret_cast<float4*>(out + j) = make_float4(__uint_as_float(r0[j]), __uint_as_float(r0[j + 1]),
                                                                                 __uint_as_float(r0[j + 2]), __uint_as_float(r0[j + 3]));
                    }
                }
            } else if (EPI == EPI_BWD) {
#pragma unroll 1
                for (int c = 0; c < tn_cols; c += 32) {
                    const int nc = n0 + c;
                    if (nc >= p.N) break;            // uniform across the warp
                    uint32_t r0[32];
                    tmem_ld_32x32(lane_addr + (uint32_t)(buf * kAccStride + c), r0);
                    tmem_ld_wait();
                    if (m < p.M) bwd_store_chunk<32>(p, m, nc, r0);
                }
            } else {
#pragma unroll 1
                for (int c = 0; c < TN / 32; ++c) {
                    const int nc = n0 + c * 32;
                    if (nc >= p.N) break;            // uniform across the warp
                    uint32_t r0[32];
                    tmem_ld_32x32(lane_addr + (uint32_t)(buf * TN + c * 32), r0);
                    if (EPI == EPI_FWD) {
                        uint32_t r1[32], r2[32];
                        if (p.has_outlier) tmem_ld_32x32(lane_addr + (uint32_t)(2 * TN + c * 32), r1);
                        if (p.has_lora) tmem_ld_32x32(lane_addr + (uint32_t)(3 * TN + c * 32), r2);
                        tmem_ld_wait();
                        if (m < p.M) {
                            const float dxm = p.dx[m];
                            float y[32];
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                float w = (float)(int)r0[j] * scale_w[c * 32 + j];
                                if (p.has_outlier) w += (float)(int)r1[j] * scale_o[c * 32 + j];
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
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (CTAS == 2 && rank != 0) mbar_arrive_cluster(lead_tmem_empty);
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
    // neither CTA of a pair may retire (or free TMEM) while its partner can still read its shared
    // memory, write its TMEM or signal its barriers
    if (CTAS == 2) cluster_sync();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc<CTAS>(tmem_base, Cfg::kTmemCols);
    }
}

}  // namespace quaff
