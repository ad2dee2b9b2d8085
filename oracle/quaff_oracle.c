/*
 * CPU oracle for the Quaff quantized linear layer (test infrastructure, NOT a product path).
 *
 * Plain, slow and meant to be checked against the paper by eye.  It shares no code with
 * the CUDA library: own bf16 helpers, own loops, no blocking, no fusion.  Only the tests,
 * the smoke check and the benchmark's cpu_baseline / reference legs may call it.
 *
 * Arithmetic contract: every quantity that ends in an integer decision (INT8 codes, step
 * sizes, scale factors) is computed in IEEE fp32 with one rounding per listed operation
 * and no fused multiply-add (compile with -ffp-contract=off); integer GEMMs accumulate in
 * int64; everything after the integer accumulators (dequantization, LoRA, all gradients)
 * is computed in double.  bf16 values travel as uint16_t bit patterns.
 *
 * Notation (paper Sec. 2.2): t -> M tokens, c_in -> K, c_out -> N, Y = X W with
 * W in R^{c_in x c_out}.  The frozen weight is held in the nn.Linear layout
 * Wt[n][k] = W[k][n].  O is the fixed, sorted set of outlier input channels, nO = |O|;
 * nOp >= nO is the padded width of the outlier operands (padding is zero).
 *
 * Pinned by tests/test_oracle_pins.py (hand-computed codes, closed forms, brute force in
 * Python integers, the scaling identity, finite differences, numpy float64 products).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ---------------------------------------------------------------- bf16 helpers */

static float bf2f(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* fp32 -> bf16, round to nearest even (finite inputs) */
static uint16_t f2bf(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

/* double -> bf16 in ONE rounding (nearest even); avoids the double rounding of going through fp32 */
static uint16_t d2bf(double d) {
    uint64_t u;
    memcpy(&u, &d, 8);
    uint64_t sign = u >> 63;
    int64_t e = (int64_t)((u >> 52) & 0x7FF);
    uint64_t man = u & ((1ull << 52) - 1);
    int64_t eb = e - 1023 + 127;
    if (e == 0 || eb <= 0) return f2bf((float)d); /* zero / tiny: bf16 subnormal range, fp32 path is exact enough */
    if (eb >= 255) return (uint16_t)((sign << 15) | 0x7F80u);
    uint64_t keep = man >> 45;
    uint64_t rem = man & ((1ull << 45) - 1);
    uint64_t half = 1ull << 44;
    uint32_t bits = (uint32_t)((eb << 7) | (int64_t)keep);
    if (rem > half || (rem == half && (keep & 1))) bits += 1; /* a carry into the exponent is the right result */
    return (uint16_t)((sign << 15) | bits);
}

/* Eq. 1 with N = 8: code = [x / Delta], Delta = amax / 127, evaluated as x * (127 / amax)
 * (one division per row or column; the step size reported is amax / 127).  Ties to even. */
static int8_t quant_code(float x, float rinv) {
    float q = nearbyintf(x * rinv); /* default rounding mode: nearest even */
    if (q > 127.0f) q = 127.0f;
    if (q < -127.0f) q = -127.0f;
    return (int8_t)q;
}

int qo_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---------------------------------------------------------------- one-time weight preprocessing
 * Sec. 3.3, "weights preprocessing": quantize the frozen W per output channel (Eq. 1),
 * keep the rows of W that belong to outlier input channels in full precision (W_O), and
 * the per-row maximum max|W_i| that Eq. 8 divides by.
 *   Wt   [N][K] bf16   frozen weight, nn.Linear layout
 *   Wq   [N][K] int8   codes,  dW[N] step sizes
 *   W_O  [nO][N] bf16  W_O[i][n] = W[O_i][n] = Wt[n][O_i]
 *   wmax_O[nO]         max_n |W_O[i][n]|
 */
void qo_prepare_weight(const uint16_t* Wt, int N, int K, const int32_t* O_idx, int nO,
                       int8_t* Wq, float* dW, uint16_t* W_O, float* wmax_O) {
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        float amax = 0.0f;
        for (int k = 0; k < K; ++k) {
            float a = fabsf(bf2f(Wt[(int64_t)n * K + k]));
            if (a > amax) amax = a;
        }
        dW[n] = amax / 127.0f;
        float rinv = amax > 0.0f ? 127.0f / amax : 0.0f;
        for (int k = 0; k < K; ++k) Wq[(int64_t)n * K + k] = quant_code(bf2f(Wt[(int64_t)n * K + k]), rinv);
    }
    for (int i = 0; i < nO; ++i) {
        float amax = 0.0f;
        for (int n = 0; n < N; ++n) {
            uint16_t w = Wt[(int64_t)n * K + O_idx[i]];
            W_O[(int64_t)i * N + n] = w;
            float a = fabsf(bf2f(w));
            if (a > amax) amax = a;
        }
        wmax_O[i] = amax;
    }
}

/* ---------------------------------------------------------------- Eq. 8 then Eq. 7, only for i in O
 *   beta_i = max(1, sqrt(max_m |X[m][O_i]| / max|W_i|))         (Eq. 8; beta_i = 1 off O, never stored)
 *   s_i   <- gamma * s_i + (1 - gamma) * beta_i                 (Eq. 7)
 * A zero weight row gives beta_i = 1.
 */
void qo_momentum_update(const uint16_t* X, int64_t ldx, int M, int K, const int32_t* O_idx, int nO,
                        const float* wmax_O, float gamma, float* s_O, float* colmax_O, float* beta_O) {
    (void)K;
    float one_minus_gamma = 1.0f - gamma;
    for (int i = 0; i < nO; ++i) {
        float cmax = 0.0f;
        for (int m = 0; m < M; ++m) {
            float a = fabsf(bf2f(X[(int64_t)m * ldx + O_idx[i]]));
            if (a > cmax) cmax = a;
        }
        float beta = 1.0f;
        if (wmax_O[i] > 0.0f) {
            float q = cmax / wmax_O[i];
            beta = fmaxf(1.0f, sqrtf(q));
        }
        float hist = gamma * s_O[i];
        float cur = one_minus_gamma * beta;
        s_O[i] = hist + cur;
        if (colmax_O) colmax_O[i] = cmax;
        if (beta_O) beta_O[i] = beta;
    }
}

/* The same update in two halves, for a batch whose tokens are spread over several workers: the column maxima of
 * Eq. 8 are taken per shard (qo_outlier_colmax), combined by an elementwise maximum (max over a union of rows is the
 * maximum of the per-shard maxima), and Eq. 8 / Eq. 7 are then applied to the combined maxima. */
void qo_outlier_colmax(const uint16_t* X, int64_t ldx, int M, const int32_t* O_idx, int nO, float* colmax_O) {
    for (int i = 0; i < nO; ++i) {
        float cmax = 0.0f;
        for (int m = 0; m < M; ++m) {
            float a = fabsf(bf2f(X[(int64_t)m * ldx + O_idx[i]]));
            if (a > cmax) cmax = a;
        }
        colmax_O[i] = cmax;
    }
}

void qo_momentum_apply(const float* colmax_O, const float* wmax_O, int nO, float gamma, float* s_O, float* beta_O) {
    float one_minus_gamma = 1.0f - gamma;
    for (int i = 0; i < nO; ++i) {
        float beta = 1.0f;
        if (wmax_O[i] > 0.0f) {
            float q = colmax_O[i] / wmax_O[i];
            beta = fmaxf(1.0f, sqrtf(q));
        }
        float hist = gamma * s_O[i];
        float cur = one_minus_gamma * beta;
        s_O[i] = hist + cur;
        if (beta_O) beta_O[i] = beta;
    }
}

/* ---------------------------------------------------------------- Eq. 5 scaling + Eq. 1 per token
 *   Xhat[m][k] = X[m][k] / s_i   if k = O_i,  X[m][k] otherwise      (Xhat = X s^-1, s_i = 1 off O)
 *   Delta[m]   = max_k |Xhat[m][k]| / 127 ;  Xq[m][k] = [Xhat[m][k] / Delta[m]]
 *   xq_O[m][i] = Xq[m][O_i]  (Eq. 9: the outlier operand inherits the activation quantization)
 * n_literal_diff (nullable): number of codes that differ from the literal x / Delta form.
 */
void qo_quant_act(const uint16_t* X, int64_t ldx, int M, int K, const int32_t* O_idx, int nO, const float* s_O,
                  int8_t* Xq, int64_t ldxq, int8_t* xq_O, int64_t ldxo, int nOp, float* dx,
                  int64_t* n_literal_diff) {
    int64_t ndiff = 0;
#pragma omp parallel for schedule(static) reduction(+ : ndiff)
    for (int m = 0; m < M; ++m) {
        float* xh = (float*)malloc(sizeof(float) * (size_t)(K > 0 ? K : 1));
        for (int k = 0; k < K; ++k) xh[k] = bf2f(X[(int64_t)m * ldx + k]);
        for (int i = 0; i < nO; ++i) xh[O_idx[i]] = xh[O_idx[i]] / s_O[i];
        float amax = 0.0f;
        for (int k = 0; k < K; ++k) {
            float a = fabsf(xh[k]);
            if (a > amax) amax = a;
        }
        float delta = amax / 127.0f;
        float rinv = amax > 0.0f ? 127.0f / amax : 0.0f;
        dx[m] = delta;
        for (int k = 0; k < K; ++k) {
            int8_t c = quant_code(xh[k], rinv);
            Xq[(int64_t)m * ldxq + k] = c;
            if (n_literal_diff && delta > 0.0f) {
                float q = nearbyintf(xh[k] / delta);
                if (q > 127.0f) q = 127.0f;
                if (q < -127.0f) q = -127.0f;
                if ((int8_t)q != c) ndiff++;
            }
        }
        for (int i = 0; i < nOp; ++i) xq_O[(int64_t)m * ldxo + i] = i < nO ? Xq[(int64_t)m * ldxq + O_idx[i]] : 0;
        free(xh);
    }
    if (n_literal_diff) *n_literal_diff = ndiff;
}

/* ---------------------------------------------------------------- what = (s_O - 1) W_O, Eq. 1 per output channel
 *   what[i][n]  = (s_i - 1) * W_O[i][n]
 *   Dw[n]       = max_i |what[i][n]| / 127 ;  wq_O[n][i] = [what[i][n] / Dw[n]]   (stored [N][nOp], like Wq)
 */
void qo_requant_weight_rows(const uint16_t* W_O, int64_t ldwo, int nO, int N, const float* s_O,
                            int8_t* wq_O, int64_t ldwq, int nOp, float* dw_O) {
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        float amax = 0.0f;
        for (int i = 0; i < nO; ++i) {
            float sm1 = s_O[i] - 1.0f;
            float w = sm1 * bf2f(W_O[(int64_t)i * ldwo + n]);
            float a = fabsf(w);
            if (a > amax) amax = a;
        }
        dw_O[n] = amax / 127.0f;
        float rinv = amax > 0.0f ? 127.0f / amax : 0.0f;
        for (int i = 0; i < nOp; ++i) {
            int8_t c = 0;
            if (i < nO) {
                float sm1 = s_O[i] - 1.0f;
                float w = sm1 * bf2f(W_O[(int64_t)i * ldwo + n]);
                c = quant_code(w, rinv);
            }
            wq_O[(int64_t)n * ldwq + i] = c;
        }
    }
}

/* ---------------------------------------------------------------- integer GEMM, C[m][n] = sum_k A[m][k] B[n][k]
 * int64 accumulation; returns the number of results that do not fit int32 (must be 0). */
int64_t qo_int_gemm(const int8_t* A, int64_t lda, const int8_t* B, int64_t ldb, int M, int N, int K,
                    int32_t* C, int64_t ldc) {
    int64_t overflow = 0;
#pragma omp parallel for schedule(static) reduction(+ : overflow)
    for (int m = 0; m < M; ++m) {
        for (int n = 0; n < N; ++n) {
            int64_t acc = 0;
            for (int k = 0; k < K; ++k) acc += (int64_t)A[(int64_t)m * lda + k] * (int64_t)B[(int64_t)n * ldb + k];
            if (acc > INT32_MAX || acc < INT32_MIN) overflow++;
            C[(int64_t)m * ldc + n] = (int32_t)acc;
        }
    }
    return overflow;
}

/* ---------------------------------------------------------------- forward, Eq. 9 plus the LoRA branch
 *   acc1 = Xq Wq^T (over K), acc2 = xq_O wq_O^T (over nOp)                       integers
 *   Y[m][n] = dx[m] * (acc1 * dW[n] + acc2 * dw_O[n])                             Eq. 9, double
 *           + lora_scale * sum_j T[m][j] B[j][n],  T = bf16(X A)                  LoRA on the unquantized X
 * T_out [M][r] bf16, Y [M][N] double, acc1/acc2 [M][N] int32 (nullable).  r = 0 disables LoRA.
 * t_given != 0: T_out is an INPUT (the bf16 down-projection as somebody else rounded it; a sum taken in another
 * order may round one unit in the last place differently) and the LoRA up-projection is evaluated on those bits.
 * Returns the number of accumulators outside int32 (must be 0).
 */
int64_t qo_qlinear_fwd(int M, int K, int N,
                       const int8_t* Xq, int64_t ldxq, const int8_t* xq_O, int64_t ldxo, int nOp, const float* dx,
                       const int8_t* Wq, int64_t ldwq_main, const float* dW,
                       const int8_t* wq_O, int64_t ldwq, const float* dw_O,
                       const uint16_t* X, int64_t ldx, const uint16_t* A, const uint16_t* B, int r, float lora_scale,
                       uint16_t* T_out, int t_given, double* Y, int32_t* acc1_out, int32_t* acc2_out) {
    int64_t overflow = 0;
    if (r > 0 && !t_given) {
#pragma omp parallel for schedule(static)
        for (int m = 0; m < M; ++m)
            for (int j = 0; j < r; ++j) {
                double t = 0.0;
                for (int k = 0; k < K; ++k) t += (double)bf2f(X[(int64_t)m * ldx + k]) * (double)bf2f(A[(int64_t)k * r + j]);
                T_out[(int64_t)m * r + j] = d2bf(t);
            }
    }
#pragma omp parallel for schedule(static) reduction(+ : overflow)
    for (int m = 0; m < M; ++m) {
        for (int n = 0; n < N; ++n) {
            int64_t a1 = 0, a2 = 0;
            for (int k = 0; k < K; ++k) a1 += (int64_t)Xq[(int64_t)m * ldxq + k] * (int64_t)Wq[(int64_t)n * ldwq_main + k];
            for (int i = 0; i < nOp; ++i) a2 += (int64_t)xq_O[(int64_t)m * ldxo + i] * (int64_t)wq_O[(int64_t)n * ldwq + i];
            if (a1 > INT32_MAX || a1 < INT32_MIN || a2 > INT32_MAX || a2 < INT32_MIN) overflow++;
            if (acc1_out) acc1_out[(int64_t)m * N + n] = (int32_t)a1;
            if (acc2_out) acc2_out[(int64_t)m * N + n] = (int32_t)a2;
            double wsum = (double)a1 * (double)dW[n];
            if (nOp > 0) wsum += (double)a2 * (double)dw_O[n];
            double y = (double)dx[m] * wsum;
            if (r > 0) {
                double l = 0.0;
                for (int j = 0; j < r; ++j) l += (double)bf2f(T_out[(int64_t)m * r + j]) * (double)bf2f(B[(int64_t)j * N + n]);
                y += (double)lora_scale * l;
            }
            Y[(int64_t)m * N + n] = y;
        }
    }
    return overflow;
}

/* ---------------------------------------------------------------- backward
 * The paper gives no backward.  Reading: straight-through derivative of Eq. 9 with s and all
 * step sizes held constant, gradients NOT quantized, the frozen weight used through its INT8
 * codes dequantized to bf16 (no full-precision weight exists during fine-tuning):
 *   Wd[n][k] = bf16(Wq[n][k] * dW[n]),   wd[n][i] = bf16(wq_O[n][i] * dw_O[n])        (fp32 product, one bf16 rounding)
 *   dXhat[m][k]    = sum_n dY[m][n] Wd[n][k]
 *   dXhat[m][O_i] += sum_n dY[m][n] wd[n][i] ;  dXhat[m][O_i] /= s_i                  (Xhat = X s^-1)
 *   G = bf16(lora_scale * dY B^T)  [M][r]
 *   dX = dXhat + G A^T ;  dA = X^T G  [K][r] ;  dB = lora_scale * T^T dY  [r][N]
 * dX [M][K], dA, dB in double (nullable each); G_out [M][r] bf16 (nullable).
 * G_in (nullable): use these bf16 bits for G instead of rounding the sum here (see t_given of the forward).
 */
void qo_qlinear_bwd(int M, int K, int N,
                    const uint16_t* dY, int64_t lddy,
                    const int8_t* Wq, int64_t ldwq_main, const float* dW,
                    const int8_t* wq_O, int64_t ldwq, const float* dw_O, int nOp,
                    const int32_t* O_idx, int nO, const float* s_O,
                    const uint16_t* X, int64_t ldx, const uint16_t* T, const uint16_t* A, const uint16_t* B,
                    int r, float lora_scale,
                    double* dX, double* dA, double* dB, uint16_t* G_out, const uint16_t* G_in) {
    (void)nOp;
    uint16_t* G = NULL;
    if (r > 0) {
        G = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)M * (size_t)r);
        if (G_in) {
            memcpy(G, G_in, sizeof(uint16_t) * (size_t)M * (size_t)r);
        } else {
#pragma omp parallel for schedule(static)
            for (int m = 0; m < M; ++m)
                for (int j = 0; j < r; ++j) {
                    double g = 0.0;
                    for (int n = 0; n < N; ++n) g += (double)bf2f(dY[(int64_t)m * lddy + n]) * (double)bf2f(B[(int64_t)j * N + n]);
                    G[(int64_t)m * r + j] = d2bf((double)lora_scale * g);
                }
        }
        if (G_out) memcpy(G_out, G, sizeof(uint16_t) * (size_t)M * (size_t)r);
    }
    if (dX) {
        /* dequantized weights, each rounded once to bf16 */
        float* Wd = (float*)malloc(sizeof(float) * (size_t)N * (size_t)K);
        float* wd = (float*)malloc(sizeof(float) * (size_t)N * (size_t)(nO > 0 ? nO : 1));
        for (int n = 0; n < N; ++n) {
            for (int k = 0; k < K; ++k) Wd[(int64_t)n * K + k] = bf2f(f2bf((float)Wq[(int64_t)n * ldwq_main + k] * dW[n]));
            for (int i = 0; i < nO; ++i) wd[(int64_t)n * nO + i] = bf2f(f2bf((float)wq_O[(int64_t)n * ldwq + i] * dw_O[n]));
        }
#pragma omp parallel for schedule(static)
        for (int m = 0; m < M; ++m) {
            double* row = dX + (int64_t)m * K;
            for (int k = 0; k < K; ++k) row[k] = 0.0;
            for (int n = 0; n < N; ++n) {
                double g = (double)bf2f(dY[(int64_t)m * lddy + n]);
                const float* w = Wd + (int64_t)n * K;
                for (int k = 0; k < K; ++k) row[k] += g * (double)w[k];
            }
            for (int i = 0; i < nO; ++i) {
                double o = 0.0;
                for (int n = 0; n < N; ++n) o += (double)bf2f(dY[(int64_t)m * lddy + n]) * (double)wd[(int64_t)n * nO + i];
                row[O_idx[i]] = (row[O_idx[i]] + o) / (double)s_O[i];
            }
            if (r > 0)
                for (int k = 0; k < K; ++k) {
                    double l = 0.0;
                    for (int j = 0; j < r; ++j) l += (double)bf2f(G[(int64_t)m * r + j]) * (double)bf2f(A[(int64_t)k * r + j]);
                    row[k] += l;
                }
        }
        free(Wd);
        free(wd);
    }
    if (dA && r > 0) {
#pragma omp parallel for schedule(static)
        for (int k = 0; k < K; ++k)
            for (int j = 0; j < r; ++j) {
                double a = 0.0;
                for (int m = 0; m < M; ++m) a += (double)bf2f(X[(int64_t)m * ldx + k]) * (double)bf2f(G[(int64_t)m * r + j]);
                dA[(int64_t)k * r + j] = a;
            }
    }
    if (dB && r > 0) {
#pragma omp parallel for schedule(static)
        for (int j = 0; j < r; ++j)
            for (int n = 0; n < N; ++n) {
                double b = 0.0;
                for (int m = 0; m < M; ++m) b += (double)bf2f(T[(int64_t)m * r + j]) * (double)bf2f(dY[(int64_t)m * lddy + n]);
                dB[(int64_t)j * N + n] = (double)lora_scale * b;
            }
    }
    free(G);
}

/* ---------------------------------------------------------------- INT8 grad-input variant (NOT the paper's method)
 * The paper quantizes no gradient (Sec. 4.1 keeps the model in floating point; Sec. 3.3 gives a forward only).  This
 * variant exists to put the largest GEMM of the step on the INT8 tensor path; it is selected by its own entry point
 * and reported separately.  Per-output-channel step sizes Delta_W[n] lie on the contraction axis of the backward, so
 * they are folded into dY before a per-token quantization (Eq. 1 applied to the rows of Z):
 *   Z[m][n]   = dY[m][n] * Delta_W[n]                       (fp32, one rounding)
 *   Dz[m]     = max_n |Z[m][n]| / 127 ;  Zq[m][n] = [Z[m][n] / Dz[m]]          (ties to even, as everywhere)
 *   acc[m][k] = sum_n Zq[m][n] * Wq[n][k]                   (integers)
 *   dXhat[m][k] = Dz[m] * acc[m][k]                         for k outside O
 * The nO outlier columns stay on the floating-point path of qo_qlinear_bwd (they are few, and they are the ones
 * divided by s):  dXhat[m][O_i] = (sum_n dY[m][n] Wd[n][O_i] + sum_n dY[m][n] wd[n][i]) / s_i.
 * G, dX = dXhat + G A^T, dA and dB are those of qo_qlinear_bwd.
 */
void qo_quant_grad(const uint16_t* dY, int64_t lddy, int M, int N, const float* dW, int8_t* Zq, int64_t ldz, float* dz) {
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        float* z = (float*)malloc(sizeof(float) * (size_t)(N > 0 ? N : 1));
        float amax = 0.0f;
        for (int n = 0; n < N; ++n) {
            z[n] = bf2f(dY[(int64_t)m * lddy + n]) * dW[n];
            float a = fabsf(z[n]);
            if (a > amax) amax = a;
        }
        dz[m] = amax / 127.0f;
        float rinv = amax > 0.0f ? 127.0f / amax : 0.0f;
        for (int n = 0; n < N; ++n) Zq[(int64_t)m * ldz + n] = quant_code(z[n], rinv);
        free(z);
    }
}

/* dX [M][K] double (required); dA, dB, G_out, G_in as in qo_qlinear_bwd; Zq_out [M][N], dz_out [M], acc_out [M][K] int32
 * (nullable dumps).  Returns the number of accumulators outside int32 (must be 0). */
int64_t qo_qlinear_bwd_int8(int M, int K, int N,
                            const uint16_t* dY, int64_t lddy,
                            const int8_t* Wq, int64_t ldwq_main, const float* dW,
                            const int8_t* wq_O, int64_t ldwq, const float* dw_O, int nOp,
                            const int32_t* O_idx, int nO, const float* s_O,
                            const uint16_t* X, int64_t ldx, const uint16_t* T, const uint16_t* A, const uint16_t* B,
                            int r, float lora_scale,
                            double* dX, double* dA, double* dB, uint16_t* G_out, const uint16_t* G_in,
                            int8_t* Zq_out, float* dz_out, int32_t* acc_out) {
    /* G, dA, dB: exactly the floating-point routine with the grad-input switched off */
    uint16_t* G = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)M * (size_t)(r > 0 ? r : 1));
    qo_qlinear_bwd(M, K, N, dY, lddy, Wq, ldwq_main, dW, wq_O, ldwq, dw_O, nOp, O_idx, nO, s_O, X, ldx, T, A, B, r, lora_scale,
                   NULL, dA, dB, G, G_in);
    if (G_out && r > 0) memcpy(G_out, G, sizeof(uint16_t) * (size_t)M * (size_t)r);
    int8_t* Zq = (int8_t*)malloc((size_t)M * (size_t)N);
    float* dz = (float*)malloc(sizeof(float) * (size_t)M);
    qo_quant_grad(dY, lddy, M, N, dW, Zq, N, dz);
    if (Zq_out) memcpy(Zq_out, Zq, (size_t)M * (size_t)N);
    if (dz_out) memcpy(dz_out, dz, sizeof(float) * (size_t)M);
    int64_t overflow = 0;
#pragma omp parallel for schedule(static) reduction(+ : overflow)
    for (int m = 0; m < M; ++m) {
        double* row = dX + (int64_t)m * K;
        int64_t* acc = (int64_t*)calloc((size_t)K, sizeof(int64_t));
        for (int n = 0; n < N; ++n) {
            int64_t z = (int64_t)Zq[(int64_t)m * N + n];
            const int8_t* w = Wq + (int64_t)n * ldwq_main;
            for (int k = 0; k < K; ++k) acc[k] += z * (int64_t)w[k];
        }
        for (int k = 0; k < K; ++k) {
            if (acc[k] > INT32_MAX || acc[k] < INT32_MIN) overflow++;
            if (acc_out) acc_out[(int64_t)m * K + k] = (int32_t)acc[k];
            row[k] = (double)dz[m] * (double)acc[k];
        }
        free(acc);
        /* outlier columns: floating-point path, through the bf16-dequantized codes */
        for (int i = 0; i < nO; ++i) {
            double o = 0.0;
            for (int n = 0; n < N; ++n) {
                double g = (double)bf2f(dY[(int64_t)m * lddy + n]);
                double wd_main = (double)bf2f(f2bf((float)Wq[(int64_t)n * ldwq_main + O_idx[i]] * dW[n]));
                double wd_out = (double)bf2f(f2bf((float)wq_O[(int64_t)n * ldwq + i] * dw_O[n]));
                o += g * wd_main + g * wd_out;
            }
            row[O_idx[i]] = o / (double)s_O[i];
        }
        if (r > 0)
            for (int k = 0; k < K; ++k) {
                double l = 0.0;
                for (int j = 0; j < r; ++j) l += (double)bf2f(G[(int64_t)m * r + j]) * (double)bf2f(A[(int64_t)k * r + j]);
                row[k] += l;
            }
    }
    free(Zq);
    free(dz);
    free(G);
    return overflow;
}

/* ---------------------------------------------------------------- calibration, Eq. 6
 * One calibration sample X^i [M][K]:  xi[o] += 1  if  max_m |X[m][o]| > thr * mean(|X|).
 * So that the indicator is one well-defined integer decision, |x| is taken in units of 2^-16,
 * truncated (anything below 2^-16 counts as 0) and saturating at 2^32 - 1:
 *     a(x) = min(floor(|x| * 65536), 2^32 - 1)
 * and the comparison is made without any division:  a(max_o) * (M * K)  >  thr * sum_{m,k} a(X[m][k]).
 */
static uint64_t abs_fix16(uint16_t b) {
    double f = floor(fabs((double)bf2f(b)) * 65536.0); /* exact: bf16 -> double, scaling by a power of two */
    return f >= 4294967295.0 ? 4294967295ull : (uint64_t)f;
}

void qo_outlier_count(const uint16_t* X, int64_t ldx, int M, int K, int thr, int32_t* xi) {
    unsigned __int128 sum = 0;
    for (int m = 0; m < M; ++m)
        for (int k = 0; k < K; ++k) sum += abs_fix16(X[(int64_t)m * ldx + k]);
    const unsigned __int128 count = (unsigned __int128)M * (unsigned __int128)K;
    for (int k = 0; k < K; ++k) {
        uint64_t mx = 0;
        for (int m = 0; m < M; ++m) {
            uint64_t a = abs_fix16(X[(int64_t)m * ldx + k]);
            if (a > mx) mx = a;
        }
        if ((unsigned __int128)mx * count > (unsigned __int128)thr * sum) xi[k] += 1;
    }
}

/* Hit rate of the predefined outlier set during fine-tuning (Sec. 3.2, the hit-rate figures): of the channels that are
 * outliers of the current batch X by the criterion of Eq. 6 (the "real-time" outliers R), how many lie in O.
 *   hits[0] = |R and O|,  hits[1] = |R|;  the hit rate is hits[0] / hits[1] (undefined when the batch has no outlier).
 * O_idx holds distinct channel indices. */
void qo_outlier_hits(const uint16_t* X, int64_t ldx, int M, int K, int thr, const int32_t* O_idx, int nO, int32_t* hits) {
    int32_t* ind = (int32_t*)calloc((size_t)(K > 0 ? K : 1), sizeof(int32_t));
    qo_outlier_count(X, ldx, M, K, thr, ind); /* ind[k] = 1 for a real-time outlier channel */
    int32_t in_set = 0, all = 0;
    for (int k = 0; k < K; ++k) all += ind[k];
    for (int i = 0; i < nO; ++i) in_set += ind[O_idx[i]];
    hits[0] = in_set;
    hits[1] = all;
    free(ind);
}

/* The nO channels with the largest xi (ties: the lower channel index first), as a sorted index set. */
void qo_select_outliers(const int32_t* xi, int K, int nO, int32_t* O_idx) {
    char* taken = (char*)calloc((size_t)(K > 0 ? K : 1), 1);
    for (int i = 0; i < nO; ++i) {
        int best = -1;
        for (int k = 0; k < K; ++k)
            if (!taken[k] && (best < 0 || xi[k] > xi[best])) best = k; /* strict >: the first (lowest) index wins ties */
        taken[best] = 1;
    }
    int n = 0;
    for (int k = 0; k < K; ++k)
        if (taken[k]) O_idx[n++] = k;
    free(taken);
}

