"""Mutation audit of the oracle's pins (CPU only).

Each entry plants ONE plausible mistake (a dropped term, a wrong sign, scale, index, rounding or loop bound) in a COPY
of ``oracle/quaff_oracle.c``, builds the copy and runs ``tests/test_oracle_pins.py`` against it in a child process.
Every planted mistake has to make at least one pin fail: a survivor is a hole in the pins.  The product library is
never involved; the mistakes exist only in a temporary directory."""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "quaff_oracle.c")
PINS = os.path.join(ROOT, "tests", "test_oracle_pins.py")

MUTANTS = []


def m(name, old, new, occ=0):
    """Replace occurrence number `occ` of `old` by `new`."""
    MUTANTS.append((name, old, new, occ))


m("f2bf_trunc", "u += 0x7FFFu + lsb;", "u += 0;")
m("f2bf_half_up", "u += 0x7FFFu + lsb;", "u += 0x8000u;")
m("d2bf_tie_up", "(rem == half && (keep & 1))", "(rem == half)")
m("d2bf_via_f32", "if (e == 0 || eb <= 0) return", "if (1) return")
m("quant_round_half_away", "float q = nearbyintf(x * rinv);", "float q = roundf(x * rinv);")
m("quant_trunc", "float q = nearbyintf(x * rinv);", "float q = truncf(x * rinv);")
m("prep_delta_128", "dW[n] = amax / 127.0f;", "dW[n] = amax / 128.0f;")
m("prep_rinv_128", "float rinv = amax > 0.0f ? 127.0f / amax : 0.0f;\n        for (int k = 0; k < K; ++k) Wq", "float rinv = amax > 0.0f ? 128.0f / amax : 0.0f;\n        for (int k = 0; k < K; ++k) Wq")
m("prep_amax_signed", "float a = fabsf(bf2f(Wt[(int64_t)n * K + k]));", "float a = bf2f(Wt[(int64_t)n * K + k]);")
m("prep_WO_transposed", "uint16_t w = Wt[(int64_t)n * K + O_idx[i]];", "uint16_t w = Wt[(int64_t)O_idx[i] * K + (n % K)];")
m("prep_wmax_signed", "float a = fabsf(bf2f(w));", "float a = bf2f(w);")
m("prep_wmax_skip_last", "for (int n = 0; n < N; ++n) {\n            uint16_t w", "for (int n = 0; n < N - 1; ++n) {\n            uint16_t w")
m("mom_no_sqrt", "beta = fmaxf(1.0f, sqrtf(q));", "beta = fmaxf(1.0f, q);", 0)
m("mom_no_max1", "beta = fmaxf(1.0f, sqrtf(q));", "beta = sqrtf(q);", 0)
m("mom_inverted_ratio", "float q = cmax / wmax_O[i];", "float q = wmax_O[i] / cmax;")
m("mom_gamma_swapped", "float hist = gamma * s_O[i];\n        float cur = one_minus_gamma * beta;", "float hist = one_minus_gamma * s_O[i];\n        float cur = gamma * beta;", 0)
m("mom_colmax_signed", "float a = fabsf(bf2f(X[(int64_t)m * ldx + O_idx[i]]));\n            if (a > cmax) cmax = a;\n        }\n        float beta", "float a = bf2f(X[(int64_t)m * ldx + O_idx[i]]);\n            if (a > cmax) cmax = a;\n        }\n        float beta")
m("mom_colmax_wrong_col", "float a = fabsf(bf2f(X[(int64_t)m * ldx + O_idx[i]]));\n            if (a > cmax) cmax = a;\n        }\n        float beta", "float a = fabsf(bf2f(X[(int64_t)m * ldx + i]));\n            if (a > cmax) cmax = a;\n        }\n        float beta")
m("colmax_skip_row0", "void qo_outlier_colmax(const uint16_t* X, int64_t ldx, int M, const int32_t* O_idx, int nO, float* colmax_O) {\n    for (int i = 0; i < nO; ++i) {\n        float cmax = 0.0f;\n        for (int m = 0; m < M; ++m) {",
  "void qo_outlier_colmax(const uint16_t* X, int64_t ldx, int M, const int32_t* O_idx, int nO, float* colmax_O) {\n    for (int i = 0; i < nO; ++i) {\n        float cmax = 0.0f;\n        for (int m = 1; m < M; ++m) {")
m("apply_no_sqrt", "beta = fmaxf(1.0f, sqrtf(q));", "beta = fmaxf(1.0f, q);", 1)
m("apply_gamma_swapped", "float hist = gamma * s_O[i];\n        float cur = one_minus_gamma * beta;", "float hist = one_minus_gamma * s_O[i];\n        float cur = gamma * beta;", 1)
m("qa_multiply_s", "xh[O_idx[i]] = xh[O_idx[i]] / s_O[i];", "xh[O_idx[i]] = xh[O_idx[i]] * s_O[i];")
m("qa_no_scale", "xh[O_idx[i]] = xh[O_idx[i]] / s_O[i];", ";")
m("qa_amax_before_scale", "for (int i = 0; i < nO; ++i) xh[O_idx[i]] = xh[O_idx[i]] / s_O[i];\n        float amax = 0.0f;\n        for (int k = 0; k < K; ++k) {\n            float a = fabsf(xh[k]);\n            if (a > amax) amax = a;\n        }",
  "float amax = 0.0f;\n        for (int k = 0; k < K; ++k) {\n            float a = fabsf(xh[k]);\n            if (a > amax) amax = a;\n        }\n        for (int i = 0; i < nO; ++i) xh[O_idx[i]] = xh[O_idx[i]] / s_O[i];")
m("qa_delta_128", "float delta = amax / 127.0f;", "float delta = amax / 128.0f;")
m("qa_xqO_unscaled_idx", "i < nO ? Xq[(int64_t)m * ldxq + O_idx[i]] : 0;", "i < nO ? Xq[(int64_t)m * ldxq + i] : 0;")
m("rq_s_not_minus1", "float sm1 = s_O[i] - 1.0f;\n            float w = sm1 * bf2f(W_O[(int64_t)i * ldwo + n]);\n            float a", "float sm1 = s_O[i];\n            float w = sm1 * bf2f(W_O[(int64_t)i * ldwo + n]);\n            float a")
m("rq_s_not_minus1_codes", "float sm1 = s_O[i] - 1.0f;\n                float w", "float sm1 = s_O[i];\n                float w")
m("rq_amax_signed", "float a = fabsf(w);", "float a = w;")
m("rq_delta_128", "dw_O[n] = amax / 127.0f;", "dw_O[n] = amax / 128.0f;")
m("rq_transposed_read", "float w = sm1 * bf2f(W_O[(int64_t)i * ldwo + n]);\n                c =", "float w = sm1 * bf2f(W_O[(int64_t)(n % nO) * ldwo + (i % N)]);\n                c =")
m("igemm_B_transposed", "(int64_t)B[(int64_t)n * ldb + k];", "(int64_t)B[(int64_t)(k % N) * ldb + (n % K)];")
m("fwd_T_A_transposed", "(double)bf2f(A[(int64_t)k * r + j]);\n                T_out", "(double)bf2f(A[(int64_t)(j * K + k) % ((int64_t)K * r)]);\n                T_out")
m("fwd_T_via_f32", "T_out[(int64_t)m * r + j] = d2bf(t);", "T_out[(int64_t)m * r + j] = f2bf((float)t);")
m("fwd_drop_outlier_term", "if (nOp > 0) wsum += (double)a2 * (double)dw_O[n];", ";")
m("fwd_outlier_minus", "if (nOp > 0) wsum += (double)a2 * (double)dw_O[n];", "if (nOp > 0) wsum -= (double)a2 * (double)dw_O[n];")
m("fwd_outlier_wrong_scale", "if (nOp > 0) wsum += (double)a2 * (double)dw_O[n];", "if (nOp > 0) wsum += (double)a2 * (double)dW[n];")
m("fwd_drop_dx", "double y = (double)dx[m] * wsum;", "double y = wsum;")
m("fwd_drop_lora_scale", "y += (double)lora_scale * l;", "y += l;")
m("fwd_lora_B_transposed", "(double)bf2f(B[(int64_t)j * N + n]);\n                y +=", "(double)bf2f(B[((int64_t)n * r + j) % ((int64_t)r * N)]);\n                y +=")
m("fwd_a2_uses_Wq", "(int64_t)wq_O[(int64_t)n * ldwq + i];\n            if (a1", "(int64_t)Wq[(int64_t)n * ldwq_main + i];\n            if (a1")
m("bwd_G_no_scale", "G[(int64_t)m * r + j] = d2bf((double)lora_scale * g);", "G[(int64_t)m * r + j] = d2bf(g);")
m("bwd_G_via_f32", "G[(int64_t)m * r + j] = d2bf((double)lora_scale * g);", "G[(int64_t)m * r + j] = f2bf((float)((double)lora_scale * g));")
m("bwd_Wd_no_round", "Wd[(int64_t)n * K + k] = bf2f(f2bf((float)Wq[(int64_t)n * ldwq_main + k] * dW[n]));", "Wd[(int64_t)n * K + k] = (float)Wq[(int64_t)n * ldwq_main + k] * dW[n];")
m("bwd_wd_no_round", "wd[(int64_t)n * nO + i] = bf2f(f2bf((float)wq_O[(int64_t)n * ldwq + i] * dw_O[n]));", "wd[(int64_t)n * nO + i] = (float)wq_O[(int64_t)n * ldwq + i] * dw_O[n];")
m("bwd_wd_wrong_scale", "wd[(int64_t)n * nO + i] = bf2f(f2bf((float)wq_O[(int64_t)n * ldwq + i] * dw_O[n]));", "wd[(int64_t)n * nO + i] = bf2f(f2bf((float)wq_O[(int64_t)n * ldwq + i] * dW[n]));")
m("bwd_no_div_s", "row[O_idx[i]] = (row[O_idx[i]] + o) / (double)s_O[i];", "row[O_idx[i]] = (row[O_idx[i]] + o);")
m("bwd_mul_s", "row[O_idx[i]] = (row[O_idx[i]] + o) / (double)s_O[i];", "row[O_idx[i]] = (row[O_idx[i]] + o) * (double)s_O[i];")
m("bwd_div_only_outlier_term", "row[O_idx[i]] = (row[O_idx[i]] + o) / (double)s_O[i];", "row[O_idx[i]] = row[O_idx[i]] + o / (double)s_O[i];")
m("bwd_drop_outlier_term", "row[O_idx[i]] = (row[O_idx[i]] + o) / (double)s_O[i];", "row[O_idx[i]] = (row[O_idx[i]]) / (double)s_O[i];")
m("bwd_lora_before_div", "            for (int i = 0; i < nO; ++i) {\n                double o = 0.0;\n                for (int n = 0; n < N; ++n) o += (double)bf2f(dY[(int64_t)m * lddy + n]) * (double)wd[(int64_t)n * nO + i];\n                row[O_idx[i]] = (row[O_idx[i]] + o) / (double)s_O[i];\n            }\n            if (r > 0)\n                for (int k = 0; k < K; ++k) {\n                    double l = 0.0;\n                    for (int j = 0; j < r; ++j) l += (double)bf2f(G[(int64_t)m * r + j]) * (double)bf2f(A[(int64_t)k * r + j]);\n                    row[k] += l;\n                }\n",
  "            if (r > 0)\n                for (int k = 0; k < K; ++k) {\n                    double l = 0.0;\n                    for (int j = 0; j < r; ++j) l += (double)bf2f(G[(int64_t)m * r + j]) * (double)bf2f(A[(int64_t)k * r + j]);\n                    row[k] += l;\n                }\n            for (int i = 0; i < nO; ++i) {\n                double o = 0.0;\n                for (int n = 0; n < N; ++n) o += (double)bf2f(dY[(int64_t)m * lddy + n]) * (double)wd[(int64_t)n * nO + i];\n                row[O_idx[i]] = (row[O_idx[i]] + o) / (double)s_O[i];\n            }\n")
m("bwd_dA_uses_T", "a += (double)bf2f(X[(int64_t)m * ldx + k]) * (double)bf2f(G[(int64_t)m * r + j]);", "a += (double)bf2f(X[(int64_t)m * ldx + k]) * (double)bf2f(T[(int64_t)m * r + j]);")
m("bwd_dB_no_scale", "dB[(int64_t)j * N + n] = (double)lora_scale * b;", "dB[(int64_t)j * N + n] = b;")
m("bwd_dB_uses_G", "b += (double)bf2f(T[(int64_t)m * r + j]) * (double)bf2f(dY[(int64_t)m * lddy + n]);", "b += (double)bf2f(G[(int64_t)m * r + j]) * (double)bf2f(dY[(int64_t)m * lddy + n]);")
m("qg_no_dW", "z[n] = bf2f(dY[(int64_t)m * lddy + n]) * dW[n];", "z[n] = bf2f(dY[(int64_t)m * lddy + n]);")
m("qg_div_dW", "z[n] = bf2f(dY[(int64_t)m * lddy + n]) * dW[n];", "z[n] = bf2f(dY[(int64_t)m * lddy + n]) / dW[n];")
m("qg_delta_128", "dz[m] = amax / 127.0f;", "dz[m] = amax / 128.0f;")
m("b8_drop_dz", "row[k] = (double)dz[m] * (double)acc[k];", "row[k] = (double)acc[k];")
m("b8_outlier_no_div", "row[O_idx[i]] = o / (double)s_O[i];", "row[O_idx[i]] = o;")
m("b8_outlier_drop_wd_out", "o += g * wd_main + g * wd_out;", "o += g * wd_main;")
m("b8_outlier_keeps_int_path", "row[O_idx[i]] = o / (double)s_O[i];", "row[O_idx[i]] = (row[O_idx[i]] + o) / (double)s_O[i];")
m("cnt_trunc_unit", "floor(fabs((double)bf2f(b)) * 65536.0)", "floor(fabs((double)bf2f(b)) * 256.0)")
m("cnt_ge", "if ((unsigned __int128)mx * count > (unsigned __int128)thr * sum) xi[k] += 1;", "if ((unsigned __int128)mx * count >= (unsigned __int128)thr * sum) xi[k] += 1;")
m("cnt_mean_per_column", "const unsigned __int128 count = (unsigned __int128)M * (unsigned __int128)K;", "const unsigned __int128 count = (unsigned __int128)M;")
m("cnt_set_not_add", ") xi[k] += 1;", ") xi[k] = 1;")
m("hits_swapped", "hits[0] = in_set;\n    hits[1] = all;", "hits[0] = all;\n    hits[1] = in_set;")
m("sel_tie_high_index", "xi[k] > xi[best]", "xi[k] >= xi[best]")
m("sel_smallest", "xi[k] > xi[best]", "xi[k] < xi[best]")
m("qa_xqO_pad_nonzero", "i < nO ? Xq[(int64_t)m * ldxq + O_idx[i]] : 0;", "i < nO ? Xq[(int64_t)m * ldxq + O_idx[i]] : 1;")
m("rq_pad_nonzero", "int8_t c = 0;\n            if (i < nO) {", "int8_t c = 1;\n            if (i < nO) {")
m("mom_zero_row_divides", "if (wmax_O[i] > 0.0f) {\n            float q = cmax / wmax_O[i];", "if (1) {\n            float q = cmax / wmax_O[i];")
m("fwd_T_given_ignored", "if (r > 0 && !t_given) {", "if (r > 0) {")
m("bwd_G_given_ignored", "if (G_in) {", "if (0) {")
m("cnt_no_saturation", "return f >= 4294967295.0 ? 4294967295ull : (uint64_t)f;", "return f >= 4294967295.0 ? 0ull : (uint64_t)f;")
m("bwd_dA_transposed", "dA[(int64_t)k * r + j] = a;", "dA[(int64_t)j * K + k] = a;")
m("bwd_dB_transposed", "dB[(int64_t)j * N + n] = (double)lora_scale * b;", "dB[(int64_t)n * r + j] = (double)lora_scale * b;")
m("qg_amax_signed", "float a = fabsf(z[n]);", "float a = z[n];")
m("bwd_lora_dropped", "row[k] += l;", ";", 0)
m("b8_lora_dropped", "row[k] += l;", ";", 1)
m("mom_beta_out_is_s", "if (beta_O) beta_O[i] = beta;\n    }\n}\n\n/* The same update", "if (beta_O) beta_O[i] = s_O[i];\n    }\n}\n\n/* The same update")
m("mom_colmax_out_is_beta", "if (colmax_O) colmax_O[i] = cmax;", "if (colmax_O) colmax_O[i] = beta;")
m("fwd_acc1_skips_last_k", "for (int k = 0; k < K; ++k) a1 +=", "for (int k = 0; k < K - 1; ++k) a1 +=")
m("bwd_main_skips_last_n", "for (int n = 0; n < N; ++n) {\n                double g = (double)bf2f(dY[(int64_t)m * lddy + n]);\n                const float* w", "for (int n = 0; n < N - 1; ++n) {\n                double g = (double)bf2f(dY[(int64_t)m * lddy + n]);\n                const float* w")
m("b8_acc_skips_last_n", "for (int n = 0; n < N; ++n) {\n            int64_t z", "for (int n = 0; n < N - 1; ++n) {\n            int64_t z")


# Not in the list because they change no result: (1) clamping the code at -128 instead of -127: |x * (127 / amax)| never
# exceeds 127 by more than rounding error, so neither clamp of Eq. 1's code is ever taken; (2) dropping the amax > 0
# guard of the per-token scale: an all-zero row then computes 0 * inf = NaN, whose conversion to an integer code is
# 0 with this compiler and CPU anyway (the guard keeps the result defined, it does not change it here).


def _plant(src, old, new, occ):
    idx = -1
    for _ in range(occ + 1):
        idx = src.find(old, idx + 1)
        if idx < 0:
            return None
    return src[:idx] + new + src[idx + len(old):]


def _run_one(args):
    name, c_path, so_path = args
    cc = subprocess.run(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
                         "-w", "-o", so_path, c_path, "-lm"], capture_output=True, text=True)
    if cc.returncode != 0:
        return name, "does not compile: " + cc.stderr[-300:]
    env = dict(os.environ, QUAFF_ORACLE_LIB=so_path, OMP_NUM_THREADS="1")
    r = subprocess.run([sys.executable, "-m", "pytest", PINS, "-x", "-q", "-p", "no:cacheprovider"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    if r.returncode == 1:
        return name, None                      # a pin failed: detected
    if r.returncode == 0:
        return name, "SURVIVED"
    return name, "pytest exit %d: %s" % (r.returncode, (r.stdout + r.stderr)[-300:])


def test_every_planted_mistake_fails_a_pin(tmp_path):
    src = open(SRC).read()
    jobs = []
    for name, old, new, occ in MUTANTS:
        mutated = _plant(src, old, new, occ)
        assert mutated is not None and mutated != src, "the oracle no longer contains the text of mutant " + name
        c_path = str(tmp_path / (name + ".c"))
        with open(c_path, "w") as f:
            f.write(mutated)
        jobs.append((name, c_path, str(tmp_path / (name + ".so"))))
    assert len({j[0] for j in jobs}) == len(jobs)
    with ThreadPoolExecutor(max_workers=max(1, min(16, os.cpu_count() or 2))) as pool:
        results = list(pool.map(_run_one, jobs))
    bad = [(n, why) for n, why in results if why is not None]
    assert not bad, bad
