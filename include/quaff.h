/*
 * quaff.h — C ABI of the B200 (sm_100a) library for the Quaff quantized linear layer:
 * INT8 weight-activation quantization with targeted momentum scaling on a fixed set of
 * outlier input channels, plus the adjacent LoRA branch, forward and backward.
 *
 * Notation follows the paper (Sec. 2.2): t -> M tokens, c_in -> K, c_out -> N, Y = X W with
 * W in R^{c_in x c_out}.  The frozen weight is stored in the nn.Linear layout [N][K]
 * (Wt[n][k] = W[k][n]), so both INT8 GEMM operands are contiguous along the contraction.
 * O is the fixed, sorted, duplicate-free set of outlier input channels, nO = |O|; nOp is nO
 * padded up to a multiple of 32 (the padding columns hold zero codes).
 *
 * Conventions
 *  - Every pointer is a DEVICE pointer unless its comment says "host".  The caller owns every
 *    buffer; the library allocates no memory and keeps no numerical state between calls.
 *  - All work is enqueued on the given stream; no call synchronises the device.
 *  - Matrices are row-major with leading dimensions given in ELEMENTS.
 *  - bf16 data are raw 16-bit patterns (quaff_bf16); INT8 codes are symmetric in [-127, 127].
 *  - Scratch memory comes from the caller (`ws`, `ws_bytes`); quaff_workspace_bytes() gives
 *    the size each entry point needs.  A workspace may be shared by calls on one stream.
 *  - Return value: QUAFF_OK or an error code.  Arguments are checked, and every tensor map is built, before the
 *    first launch: an argument error (codes 1-4) means nothing has been launched.  QUAFF_ERR_CUDA may come from a
 *    launch in the middle of a call; what was enqueued before it stays enqueued, every stream the call forked is
 *    joined back into `stream`, and the outputs are undefined.
 *    A device-side wait that gave up (after about two seconds) is reported through the optional `status` word
 *    (QUAFF_ERR_TIMEOUT) after the stream has been synchronised; outputs are then undefined.
 *  - Inputs must be finite.  Results are deterministic (no floating-point atomics).
 *  - An empty batch (M = 0) is valid wherever M is a token count (the calibration calls need M >= 1): nothing is
 *    launched, and a backward call that does not accumulate stores the empty sums dA = 0 and dB = 0.
 *  - The outlier set: 0 <= nO <= K and nO <= 4096 in every entry point that takes one (more: QUAFF_ERR_UNSUPPORTED_SHAPE).
 *  - Threads: every entry point may be called from several host threads at once, on the same or on different
 *    devices and streams (lazily created per-device resources are guarded; quaff_qlinear_bwd calls on one device are
 *    enqueued one after the other).  The usual CUDA rule remains: calls that share an output, a workspace or the
 *    built-in scratch of quaff_momentum_update_static must be ordered by the caller.  The library keeps no state
 *    that changes results between calls; the only switches are the per-thread measurement aids at the end of this file.
 */
#ifndef QUAFF_H_
#define QUAFF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef uint16_t quaff_bf16;
typedef void* quaff_stream_t; /* a cudaStream_t */

typedef enum {
    QUAFF_OK = 0,
    QUAFF_ERR_INVALID_ARG = 1,       /* null pointer, negative size, nO > K, gamma outside [0,1], ... */
    QUAFF_ERR_UNSUPPORTED_SHAPE = 2, /* a size outside what the kernels are built for */
    QUAFF_ERR_ALIGNMENT = 3,         /* base pointer or leading dimension not 16-byte aligned */
    QUAFF_ERR_WORKSPACE_TOO_SMALL = 4,
    QUAFF_ERR_CUDA = 5,              /* a CUDA runtime / driver call failed (launch, tensor map) */
    QUAFF_ERR_TIMEOUT = 6            /* only ever written to the device `status` word */
} quaff_status_t;

enum { QUAFF_BF16 = 0, QUAFF_F32 = 1 }; /* y_dtype of quaff_qlinear_fwd */

enum { /* `which` of quaff_workspace_bytes */
    QUAFF_WS_PREPARE = 0,
    QUAFF_WS_MOMENTUM = 1,
    QUAFF_WS_FWD = 2,
    QUAFF_WS_BWD = 3,
    QUAFF_WS_CALIBRATE = 4,  /* quaff_outlier_count and quaff_select_outliers (depends on K only) */
    QUAFF_WS_HITS = 5,       /* quaff_outlier_hits (depends on K only) */
    QUAFF_WS_BWD_INT8 = 6,   /* quaff_qlinear_bwd_int8 */
    QUAFF_WS_BWD_LEAN = 7    /* quaff_qlinear_bwd without a transient bf16 copy of the weight (see there) */
};

const char* quaff_status_string(quaff_status_t s);

/* Bytes of scratch that entry point `which` needs for these sizes (a multiple of 256; may be 0). */
size_t quaff_workspace_bytes(int which, int M, int K, int N, int nOp, int r);

/*
 * Calibration before fine-tuning (Sec. 3.3, Eq. 6), one call per calibration sample X^i [M][K]:
 *   xi[o] += 1   if   max_m |X[m][o]| > thr * mean(|X|)          (the paper uses thr = 100)
 * The indicator is one exact integer decision: |x| is taken in units of 2^-16, truncated and saturating
 * at 2^32 - 1, a(x) = min(floor(|x| 2^16), 2^32 - 1), and the test is a(max_o) * (M K) > thr * sum a(X).
 *   X [M][K] bf16, ldx (ldx % 8 == 0);  thr >= 0;  xi [K] int32 (in/out: the caller zeroes it before the first sample)
 *   ws: QUAFF_WS_CALIBRATE bytes
 */
quaff_status_t quaff_outlier_count(const quaff_bf16* X, int64_t ldx, int M, int K, int thr, int32_t* xi,
                                   void* ws, size_t ws_bytes, quaff_stream_t stream);

/*
 * The outlier set O from the counts of Eq. 6 (Sec. 3.3, weight preprocessing): the nO channels
 * with the largest xi, ties going to the lower channel index, written as a sorted index set.
 *   xi [K] int32 (in);  O_idx [nO] int32 (out, ascending);  nO <= K is the layer's budget;  ws: QUAFF_WS_CALIBRATE bytes
 */
quaff_status_t quaff_select_outliers(const int32_t* xi, int K, int nO, int32_t* O_idx, void* ws, size_t ws_bytes,
                                     quaff_stream_t stream);

/*
 * Hit-rate monitor during fine-tuning (Sec. 3.2, the hit-rate figures): of the channels that are outliers of the
 * CURRENT batch X by the criterion of Eq. 6 (the "real-time" outliers R, same integer decision as quaff_outlier_count),
 * how many lie in the predefined set O.
 *   hits[0] = |R and O|,  hits[1] = |R|   (device int32[2], overwritten);  hit rate = hits[0] / hits[1], undefined
 *   when the batch has no outlier channel.  The caller averages over iterations and layers.
 *   X [M][K] bf16, ldx (ldx % 8 == 0);  O_idx [nO] distinct channel indices (an index outside [0,K) is ignored);
 *   ws: QUAFF_WS_HITS bytes
 */
quaff_status_t quaff_outlier_hits(const quaff_bf16* X, int64_t ldx, int M, int K, int thr, const int32_t* O_idx, int nO,
                                  int32_t* hits, void* ws, size_t ws_bytes, quaff_stream_t stream);

/*
 * One-time weight preprocessing (Sec. 3.3, "weights preprocessing"; Eq. 1 per output channel).
 *   Wt   [N][K] bf16, ldw      frozen weight (in)
 *   Wq   [N][K] int8, ldwq     codes, Wq[n][k] = [Wt[n][k] / dW[n]]   (out)
 *   dW   [N] f32               step sizes max_k|Wt[n][k]| / 127       (out)
 *   W_O  [nO][N] bf16, ldwo    W_O[i][n] = Wt[n][O_i], the only full-precision rows kept (out)
 *   wmax_O [nO] f32            max_n |W_O[i][n]|, the max|W_i| of Eq. 8 (out)
 * nO may be 0 (W_O, wmax_O, O_idx may then be null).
 */
quaff_status_t quaff_prepare_weight(const quaff_bf16* Wt, int64_t ldw, int N, int K,
                                    const int32_t* O_idx, int nO,
                                    int8_t* Wq, int64_t ldwq, float* dW,
                                    quaff_bf16* W_O, int64_t ldwo, float* wmax_O,
                                    quaff_stream_t stream);

/*
 * Targeted momentum scaling (Eq. 8 then Eq. 7), only on the channels of O:
 *   colmax_i = max_m |X[m][O_i]| ;  beta_i = max(1, sqrt(colmax_i / wmax_O[i]))  (1 if wmax_O[i] = 0)
 *   s_O[i]  <- gamma * s_O[i] + (1 - gamma) * beta_i
 *   X [M][K] bf16, ldx (in);  O_idx [nO] int32 (in);  wmax_O [nO] f32 (in);  gamma in [0,1]
 *   s_O [nO] f32 (in: s_{t-1}, out: s_t; the caller initialises it, 1 = no scaling)
 *   colmax_O_opt, beta_O_opt [nO] f32: optional diagnostics, may be null
 *   ws: QUAFF_WS_MOMENTUM bytes.  nO = 0 is a no-op.  fp32, one rounding per operation.
 */
quaff_status_t quaff_momentum_update(const quaff_bf16* X, int64_t ldx, int M, int K,
                                     const int32_t* O_idx, int nO, const float* wmax_O, float gamma,
                                     float* s_O, float* colmax_O_opt, float* beta_O_opt,
                                     void* ws, size_t ws_bytes, quaff_stream_t stream);

/*
 * The same update in two halves, for a batch whose tokens are spread over several GPUs (the paper runs on one):
 * each GPU takes the column maxima of its own rows, the trainer combines them with an elementwise MAX all-reduce
 * (the maximum over all rows is the maximum of the per-shard maxima, so s_O comes out bit-identical to the
 * single-GPU update), and every GPU applies Eq. 8 and Eq. 7 to the combined maxima.
 *   quaff_outlier_colmax:  colmax_O[i] = max_m |X[m][O_i]|   ([nO] f32, out);  ws: QUAFF_WS_MOMENTUM bytes
 *   quaff_momentum_apply:  beta_i = max(1, sqrt(colmax_O[i] / wmax_O[i]))  (1 if wmax_O[i] = 0);
 *                          s_O[i] <- gamma * s_O[i] + (1 - gamma) * beta_i;  beta_O_opt [nO] optional
 * nO = 0 is a no-op in both.
 */
quaff_status_t quaff_outlier_colmax(const quaff_bf16* X, int64_t ldx, int M, int K, const int32_t* O_idx, int nO,
                                    float* colmax_O, void* ws, size_t ws_bytes, quaff_stream_t stream);
quaff_status_t quaff_momentum_apply(const float* colmax_O, const float* wmax_O, int nO, float gamma, float* s_O,
                                    float* beta_O_opt, quaff_stream_t stream);

/*
 * Scale and quantize the activations (Eq. 5: Xhat = X s^-1, s_i = 1 off O; Eq. 1 per token).
 *   Xhat[m][O_i] = X[m][O_i] / s_O[i];  dx[m] = max_k|Xhat[m][k]| / 127;
 *   Xq[m][k] = round_to_nearest_even(Xhat[m][k] * (127 / max_k|Xhat[m][k]|)), clamped to +-127
 *   xq_O[m][i] = Xq[m][O_i] for i < nO, 0 for nO <= i < nOp      (Eq. 9: xhat_int = [Xhat_int]_{:,O})
 *   X [M][K] bf16, ldx (in; ldx % 8 == 0);  Xq [M][K] int8, ldxq (out; ldxq % 16 == 0)
 *   xq_O [M][nOp] int8, ldxo (out; may be null when nOp == 0);  dx [M] f32 (out)
 * An all-zero row gives dx = 0 and zero codes.  One pass over X.
 */
quaff_status_t quaff_quant_act(const quaff_bf16* X, int64_t ldx, int M, int K,
                               const int32_t* O_idx, int nO, const float* s_O,
                               int8_t* Xq, int64_t ldxq,
                               int8_t* xq_O, int64_t ldxo, int nOp,
                               float* dx, quaff_stream_t stream);

/*
 * Re-quantize the scaled outlier rows of the weight, every step (Eq. 5: what = (s_O - 1) W_O; Eq. 1 per
 * output channel; Sec. 3.1):
 *   what[i][n] = (s_O[i] - 1) * W_O[i][n];  dw_O[n] = max_i|what[i][n]| / 127;
 *   wq_O[n][i] = round_to_nearest_even(what[i][n] * (127 / max_i|what[i][n]|)), 0 for i >= nO
 *   W_O [nO][N] bf16, ldwo (in);  s_O [nO] f32 (in)
 *   wq_O [N][nOp] int8, ldwq (out; same orientation as Wq; ldwq % 16 == 0);  dw_O [N] f32 (out)
 */
quaff_status_t quaff_requant_weight_rows(const quaff_bf16* W_O, int64_t ldwo, int nO, int N,
                                         const float* s_O,
                                         int8_t* wq_O, int64_t ldwq, int nOp,
                                         float* dw_O, quaff_stream_t stream);

/*
 * LoRA down-projection on its own: T_out [M][r] bf16 (dense) = bf16(X A), fp32 accumulation.  The paper's
 * LoRA adapter reads the unquantized X, so this step depends on nothing the other entry points compute: a
 * caller may run it on a second stream beside quaff_momentum_update / quaff_quant_act and hand the result to
 * quaff_qlinear_fwd (X = NULL there).   X [M][K] bf16, ldx (ldx % 8 == 0);  A [K][r] bf16 dense;
 * r a multiple of 8, <= 64; K a multiple of 8;  ws: QUAFF_WS_FWD bytes (its own, not shared with a call
 * that runs concurrently);  status_opt as in the forward.
 */
quaff_status_t quaff_lora_down(const quaff_bf16* X, int64_t ldx, int M, int K, const quaff_bf16* A, int r,
                               quaff_bf16* T_out, int32_t* status_opt, void* ws, size_t ws_bytes,
                               quaff_stream_t stream);

/*
 * Forward (Eq. 9) with the LoRA branch fused into the epilogue:
 *   acc1 = Xq Wq^T  (INT8 x INT8 -> INT32 over K),  acc2 = xq_O wq_O^T  (over nOp)
 *   T    = bf16(X A)                                                     [M][r], LoRA down-projection
 *   Y[m][n] = dx[m] * (acc1[m][n] * dW[n] + acc2[m][n] * dw_O[n]) + lora_scale * (T B)[m][n]
 *   Xq [M][K], ldxq;  xq_O [M][nOp], ldxo;  dx [M]           from quaff_quant_act
 *   Wq [N][K], ldwq_main;  dW [N]                             frozen (quaff_prepare_weight)
 *   wq_O [N][nOp], ldwq;  dw_O [N]                            from quaff_requant_weight_rows
 *   X [M][K] bf16, ldx;  A [K][r] bf16;  B [r][N] bf16        LoRA (dense, ld = r and N); r == 0 disables
 *   T_out [M][r] bf16 (out, dense; kept for the backward).  With X = NULL (and r > 0), T_out is an INPUT:
 *   T from an earlier quaff_lora_down on the same X and A; A may then be NULL (ws is still needed)
 *   Y [M][N], ldy, y_dtype QUAFF_BF16 or QUAFF_F32 (out)
 *   dbg_acc_main, dbg_acc_out: optional dense [M][N] int32 dumps of acc1 / acc2 (parity checks)
 *   status_opt: optional int32[4] device word, must be zero on entry; see QUAFF_ERR_TIMEOUT
 *   ws: QUAFF_WS_FWD bytes
 * Alignment: all matrix bases 16-byte aligned; ldxq, ldxo, ldwq_main, ldwq multiples of 16;
 * ldx multiple of 8; r multiple of 8, r <= 64; nOp multiple of 32 (0 allowed); with r > 0, K and N
 * multiples of 8 (A and B are read in place by TMA).
 */
quaff_status_t quaff_qlinear_fwd(int M, int K, int N,
                                 const int8_t* Xq, int64_t ldxq, const int8_t* xq_O, int64_t ldxo, int nOp,
                                 const float* dx,
                                 const int8_t* Wq, int64_t ldwq_main, const float* dW,
                                 const int8_t* wq_O, int64_t ldwq, const float* dw_O,
                                 const quaff_bf16* X, int64_t ldx, const quaff_bf16* A, const quaff_bf16* B,
                                 int r, float lora_scale,
                                 quaff_bf16* T_out,
                                 void* Y, int y_dtype, int64_t ldy,
                                 int32_t* dbg_acc_main, int32_t* dbg_acc_out,
                                 int32_t* status_opt, void* ws, size_t ws_bytes, quaff_stream_t stream);

/*
 * Backward.  The paper states no backward; this is the straight-through derivative of Eq. 9
 * with s and every step size held constant.  Gradients are not quantized (the paper keeps the
 * model in floating point and applies INT8 to the linear layers' forward operands only); the
 * frozen weight is used through its INT8 codes, dequantized to bf16 on the fly:
 *   Wd[n][k] = bf16(Wq[n][k] * dW[n]),  wd[n][i] = bf16(wq_O[n][i] * dw_O[n])
 *   dXhat = dY Wd ;  dXhat[:,O_i] += dY wd[:,i] ;  dXhat[:,O_i] /= s_O[i]
 *   G  = bf16(lora_scale * dY B^T)                                   [M][r]
 *   dX = dXhat + G A^T                                               [M][K] bf16, lddx (nullable: skipped)
 *   dA = X^T G  [K][r] f32 ;  dB = lora_scale * T^T dY  [r][N] f32   (nullable pair; accumulate != 0 adds)
 *   dY [M][N] bf16, lddy (lddy % 8 == 0);  T [M][r] bf16 from the forward
 *   Wq, wq_O: 16-byte aligned, ldwq_main and ldwq multiples of 16 (as in the forward)
 *   G_out_opt [M][r] bf16 (dense, 16-byte aligned), optional: receives G (otherwise G lives in the workspace only)
 *   dW, dw_O: 16-byte aligned;  with an outlier set, K <= 32768
 *   status_opt as in the forward.
 *   ws: QUAFF_WS_BWD bytes, or QUAFF_WS_BWD_LEAN bytes.  With QUAFF_WS_BWD bytes (2 N K bytes more) the call builds a
 *   transient bf16 copy Wd of the weight in the workspace and the grad-input GEMM reads it by TMA: the faster way (the
 *   copy lives only inside the call; nothing full-precision is kept between steps, Sec. 3.1).  With QUAFF_WS_BWD_LEAN
 *   bytes no copy is made at all: the GEMM reads the codes Wq and wq_O in place and expands them to bf16 in shared
 *   memory (about 1.4 times the GEMM time, bound by shared-memory bandwidth).  The products and their order are the same:
 *   dX is bit-identical between the two off the outlier columns.
 * Independent parts of the backward are forked onto two library-owned side streams (lowest priority) and
 * joined back into `stream` before the call returns: for the caller everything is still ordered on
 * `stream`.  The weight dequantization runs beside G in front of the grad-input GEMM; dA and dB are enqueued behind the
 * GEMM without depending on it, so that their split-K CTAs run in the SMs the GEMM's last wave leaves idle.  Each device
 * has four sets of side streams, created by the first backward call on that device (make that call outside any stream
 * capture).  Under capture the forks become parallel branches of the captured graph, and a set stays with its capture
 * until the capture ends; with more than four captures open at once on one device, further calls run unforked.
 */
quaff_status_t quaff_qlinear_bwd(int M, int K, int N,
                                 const quaff_bf16* dY, int64_t lddy,
                                 const int8_t* Wq, int64_t ldwq_main, const float* dW,
                                 const int8_t* wq_O, int64_t ldwq, const float* dw_O, int nOp,
                                 const int32_t* O_idx, int nO, const float* s_O,
                                 const quaff_bf16* X, int64_t ldx, const quaff_bf16* T,
                                 const quaff_bf16* A, const quaff_bf16* B, int r, float lora_scale,
                                 quaff_bf16* dX, int64_t lddx,
                                 float* dA, float* dB, int accumulate, quaff_bf16* G_out_opt,
                                 int32_t* status_opt, void* ws, size_t ws_bytes, quaff_stream_t stream);

/*
 * INT8 grad-input variant of the backward.  NOT the paper's method: the paper quantizes no gradient (Sec. 4.1 keeps the
 * model in floating point, Sec. 3.3 states a forward only), so this entry point is never what quaff_qlinear_bwd does
 * and its results are reported separately.  It puts the grad-input GEMM, the largest cost of a step, on the INT8
 * tensor path: the per-output-channel step sizes lie on the backward's contraction axis, so they are folded into dY
 * before a per-token quantization,
 *   Z[m][n] = dY[m][n] * dW[n] ;  dz[m] = max_n |Z[m][n]| / 127 ;  Zq[m][n] = round_to_nearest_even(Z[m][n] * (127 / max_n|Z[m][n]|))
 *   dXhat[m][k] = dz[m] * sum_n Zq[m][n] * Wq[n][k]                      (INT8 x INT8 -> INT32, Wq read in place)
 * for every k outside O; the nO outlier columns keep the floating-point path of quaff_qlinear_bwd,
 *   dXhat[m][O_i] = (sum_n dY[m][n] (Wd[n][O_i] + wd[n][i])) / s_O[i].
 * G, dX = dXhat + G A^T, dA, dB and all other arguments are those of quaff_qlinear_bwd; dX is required; N must be a
 * multiple of 16, at most 16384 (more: QUAFF_ERR_UNSUPPORTED_SHAPE); dbg_acc_opt: optional dense [M][K] int32 dump of sum_n Zq Wq (parity checks);  ws: QUAFF_WS_BWD_INT8 bytes.
 * quaff_quant_grad is the quantization step on its own (Zq [M][N] int8 with ldz % 16 == 0, dz [M] f32).
 */
quaff_status_t quaff_quant_grad(const quaff_bf16* dY, int64_t lddy, int M, int N, const float* dW, int8_t* Zq, int64_t ldz,
                                float* dz, quaff_stream_t stream);
quaff_status_t quaff_qlinear_bwd_int8(int M, int K, int N,
                                      const quaff_bf16* dY, int64_t lddy,
                                      const int8_t* Wq, int64_t ldwq_main, const float* dW,
                                      const int8_t* wq_O, int64_t ldwq, const float* dw_O, int nOp,
                                      const int32_t* O_idx, int nO, const float* s_O,
                                      const quaff_bf16* X, int64_t ldx, const quaff_bf16* T,
                                      const quaff_bf16* A, const quaff_bf16* B, int r, float lora_scale,
                                      quaff_bf16* dX, int64_t lddx,
                                      float* dA, float* dB, int accumulate, quaff_bf16* G_out_opt, int32_t* dbg_acc_opt,
                                      int32_t* status_opt, void* ws, size_t ws_bytes, quaff_stream_t stream);

/*
 * quaff_momentum_update without a caller-supplied workspace (the paper has no counterpart: this
 * is a packaging variant of the call above, same arithmetic, same outputs).
 *
 * For callers that cannot hand the library device scratch because they cannot allocate any: code
 * running where cudaMalloc is off limits - a plug-in inside a host framework that owns the whole
 * device-memory budget and forbids allocations outside its own pool, or a step on a latency-critical
 * path where the implicit device-wide synchronisation of cudaMalloc/cudaFree is unacceptable.  The
 * scratch (column maxima and a block counter) lives in a fixed array compiled into the library, so
 * this entry point calls no cudaMalloc, cudaFree or allocating library routine.
 *
 *  - Limit: nO <= 4096 outlier channels, the limit of every entry point (16 KB + 4 B of device memory,
 *    held by every GPU that loads the library until the process exits).  A larger nO returns
 *    QUAFF_ERR_UNSUPPORTED_SHAPE here as in quaff_momentum_update.
 *  - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *    that device current) and caches it.  Make that first call outside any stream capture.
 *  - All calls on a device share the one array.  Each call clears what must start at zero, but two
 *    calls whose kernels overlap on the GPU (different streams) race on it: serialise them.
 * Arguments and results are exactly those of quaff_momentum_update, minus `ws` / `ws_bytes`.
 */
quaff_status_t quaff_momentum_update_static(const quaff_bf16* X, int64_t ldx, int M, int K,
                                            const int32_t* O_idx, int nO, const float* wmax_O, float gamma,
                                            float* s_O, float* colmax_O_opt, float* beta_O_opt,
                                            quaff_stream_t stream);

/*
 * Measurement aids (no counterpart in the paper).  The two switches are PER HOST THREAD: they affect only later calls
 * made by the thread that set them, so no other caller's kernel choice or stream contents can change under it.
 *
 * quaff_debug_launch_count: number of kernels this library has launched since it was loaded (all threads).
 *
 * quaff_debug_force_fwd_tile: quaff_qlinear_fwd picks the output-column tile of its kernel (128, 192 or 256) by a
 * cost model; tile_n = 128 / 192 / 256 forces that kernel for the calling thread where the shape allows it (outlier set
 * or LoRA present, nOp <= 128), 0 gives the choice back to the cost model.  For tests and timing of each kernel on
 * the same shape.
 *
 * quaff_debug_time_gemm: arm a one-shot pair of CUDA events (cudaEvent_t, created by the caller
 * with timing enabled) around the calling thread's next launch of the forward (which = 0) or grad-input
 * (which = 1) tensor-core GEMM kernel: `start` is recorded on the launch stream right before the
 * kernel, `stop` right after, then the pair is disarmed.  Null events disarm.  If the stream is being
 * captured into a CUDA graph, the pair becomes two event-record nodes of that graph: every replay records
 * them again, and the elapsed time between them is that of the latest replay.
 */
uint64_t quaff_debug_launch_count(void);
void quaff_debug_force_fwd_tile(int tile_n);
void quaff_debug_time_gemm(int which, void* start_event, void* stop_event);

#ifdef __cplusplus
}
#endif
#endif /* QUAFF_H_ */
