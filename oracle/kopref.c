/*
 * kopref — float64 CPU oracle for the fused pointwise+reduction segments.
 *
 * TEST INFRASTRUCTURE ONLY. This file is the slow, plain definition of what each
 * segment computes. It is used by the tests, by the smoke check and by the
 * benchmark's cpu_baseline / reference legs; the product path (the CUDA library)
 * never links, loads or calls it, and it shares no code, header, table or
 * constant with that path.
 *
 * The paper names these segment classes (planner strategies 8-9, the codegen
 * agent's "beating Inductor" list and the fusion agent's technique list:
 * fused softmax, single-pass LayerNorm / RMSNorm, activation+bias fusion,
 * residual+norm, reduction+pointwise, LogSumExp reductions) but never prints
 * their formulas, so each function below writes out the textbook definition in
 * the most direct form: two passes where the definition has two passes, no
 * online recurrences, no blocking, no reordering. The fast methods the CUDA
 * path uses (row in registers, online max/sum) reach the same real number up
 * to rounding order, so the plain definition is the reference.
 *
 * Conventions
 *   - data tensors come in as fp32, bf16 bit patterns (uint16) or fp64, chosen
 *     by a dtype tag; they are widened exactly to double. Parameter vectors
 *     (bias, gamma, beta, scale, shift, weight) are fp32 and widened exactly.
 *   - every output is double, never rounded back.
 *   - strides are in elements; the innermost stride is 1.
 *   - `threads` > 1 splits the outer (row / plane) loop with OpenMP; each row is
 *     still computed by one thread in index order, so results do not depend on it.
 *   - return value 0 = ok, negative = bad argument.
 *
 * All parity pins live in tests/test_oracle_pins.py; every function is pinned.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { KOPREF_F32 = 0, KOPREF_BF16 = 1, KOPREF_F64 = 2, KOPREF_F16 = 3 };

/* ---- exact widening / narrowing helpers ------------------------------------ */

/* bf16 is the upper 16 bits of an IEEE binary32, so widening is exact. */
double kopref_bf16_to_f64(uint16_t bits)
{
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* IEEE binary16 (1 sign, 5 exponent, 10 fraction bits) widened exactly, from its fields:
 * exponent 0: (-1)^s * fraction * 2^-24 (zero and subnormals); exponent 31: infinity or NaN;
 * otherwise (-1)^s * (1024 + fraction) * 2^(exponent - 25). */
double kopref_f16_to_f64(uint16_t bits)
{
    int s = bits >> 15, e = (bits >> 10) & 0x1F, f = bits & 0x3FF;
    double v;
    if (e == 0) v = ldexp((double)f, -24);
    else if (e == 31) v = f ? NAN : INFINITY;
    else v = ldexp((double)(1024 + f), e - 25);
    return s ? -v : v;
}

/* Round a double directly to bf16 (round to nearest, ties to even) without
 * passing through fp32, so there is no double rounding. bf16 has 8 significant
 * bits (1 implicit + 7 stored) and the fp32 exponent range. */
uint16_t kopref_f64_to_bf16_rne(double v)
{
    if (v != v) return 0x7FC0u;                          /* quiet NaN */
    uint16_t sign = signbit(v) ? 0x8000u : 0u;
    double a = fabs(v);
    if (a == 0.0) return sign;
    if (isinf(a)) return (uint16_t)(sign | 0x7F80u);
    int e;
    (void)frexp(a, &e);                                  /* a = m * 2^e, m in [0.5, 1) */
    int exp_unbiased = e - 1;                            /* a = (2m) * 2^(e-1), 2m in [1,2) */
    if (exp_unbiased < -126) exp_unbiased = -126;        /* subnormal range: fixed quantum */
    /* quantum of the bf16 grid at this exponent: 2^(exp_unbiased - 7) */
    double q = ldexp(1.0, exp_unbiased - 7);
    double n = a / q;                                    /* exact: power-of-two division */
    double fl = floor(n);
    double frac = n - fl;
    if (frac > 0.5 || (frac == 0.5 && fmod(fl, 2.0) == 1.0)) fl += 1.0;
    double r = fl * q;                                   /* rounded magnitude */
    if (r >= ldexp(1.0, 128)) return (uint16_t)(sign | 0x7F80u);   /* overflow to inf */
    float rf = (float)r;                                 /* exact: r is on the bf16 grid */
    uint32_t u;
    memcpy(&u, &rf, sizeof u);
    return (uint16_t)(sign | (uint16_t)(u >> 16));
}

static inline double load_elem(const void* base, int64_t idx, int dtype)
{
    switch (dtype) {
    case KOPREF_F32:  return (double)((const float*)base)[idx];
    case KOPREF_BF16: return kopref_bf16_to_f64(((const uint16_t*)base)[idx]);
    case KOPREF_F16:  return kopref_f16_to_f64(((const uint16_t*)base)[idx]);
    default:          return ((const double*)base)[idx];
    }
}

static int bad_dtype(int dtype) { return dtype < KOPREF_F32 || dtype > KOPREF_F16; }

static int pick_threads(int threads)
{
#ifdef _OPENMP
    if (threads < 1) threads = 1;
    return threads;
#else
    (void)threads;
    return 1;
#endif
}

int kopref_has_openmp(void)
{
#ifdef _OPENMP
    return 1;
#else
    return 0;
#endif
}

/* ---- softmax(x * s + b) over each row ---------------------------------------
 * z_j = x_j * s + b_j ; m = max_j z_j ; e_j = exp(z_j - m) ; S = sum_j e_j ;
 * y_j = e_j / S.   ("fused softmax", planner strategy 9.)  bias may be NULL (= 0).
 * A row whose z are all -inf gives NaN, as the definition's 0/0 does. */
int kopref_softmax_scale_bias(const void* x, const float* bias, double* y,
                              int64_t rows, int64_t cols, int64_t x_row_stride,
                              int64_t y_row_stride, double scale, int dtype, int threads)
{
    if (!x || !y || rows < 0 || cols <= 0 || bad_dtype(dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
        double* yr = y + i * y_row_stride;
        double m = -INFINITY;
        for (int64_t j = 0; j < cols; ++j) {
            double z = load_elem(x, i * x_row_stride + j, dtype) * scale
                     + (bias ? (double)bias[j] : 0.0);
            yr[j] = z;
            if (z > m) m = z;
        }
        double S = 0.0;
        for (int64_t j = 0; j < cols; ++j) {
            double e = exp(yr[j] - m);
            yr[j] = e;
            S += e;
        }
        for (int64_t j = 0; j < cols; ++j) yr[j] = yr[j] / S;
    }
    return 0;
}

/* ---- tanh-form GELU --------------------------------------------------------
 * g(u) = 0.5 u (1 + tanh( sqrt(2/pi) (u + 0.044715 u^3) )). */
double kopref_gelu_tanh(double u)
{
    const double k = sqrt(2.0 / 3.14159265358979323846264338327950288);
    return 0.5 * u * (1.0 + tanh(k * (u + 0.044715 * u * u * u)));
}

/* ---- bias + GELU + residual + LayerNorm --------------------------------------
 * v_j = r_j + g(x_j + b_j) ; mu = (1/H) sum v ; var = (1/H) sum (v - mu)^2 (biased) ;
 * rstd = 1 / sqrt(var + eps) ; y_j = (v_j - mu) rstd gamma_j + beta_j.
 * ("residual + norm" and "normalization fusion" in the fusion agent's list,
 * "activation + bias fusion" for the prologue.)  v is never rounded.
 * mean / rstd may be NULL. */
/* The exact (error-function) GELU: 0.5 u (1 + erf(u / sqrt 2)), the form without the tanh approximation. */
double kopref_gelu_erf(double u) { return 0.5 * u * (1.0 + erf(u * 0.70710678118654752440)); }

static int bias_gelu_residual_layernorm_impl(const void* x, const void* residual,
        const float* bias, const float* gamma, const float* beta,
        double* y, double* mean, double* rstd,
        int64_t rows, int64_t hidden, int64_t x_row_stride, int64_t res_row_stride,
        int64_t y_row_stride, double eps, int dtype, int threads, int erf_form)
{
    if (!x || !residual || !bias || !gamma || !beta || !y) return -1;
    if (rows < 0 || hidden <= 0 || bad_dtype(dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
        double* yr = y + i * y_row_stride;
        double sum = 0.0;
        for (int64_t j = 0; j < hidden; ++j) {
            double u = load_elem(x, i * x_row_stride + j, dtype) + (double)bias[j];
            double v = load_elem(residual, i * res_row_stride + j, dtype)
                     + (erf_form ? kopref_gelu_erf(u) : kopref_gelu_tanh(u));
            yr[j] = v;
            sum += v;
        }
        double mu = sum / (double)hidden;
        double ss = 0.0;
        for (int64_t j = 0; j < hidden; ++j) {
            double d = yr[j] - mu;
            ss += d * d;
        }
        double var = ss / (double)hidden;
        double rs = 1.0 / sqrt(var + eps);
        for (int64_t j = 0; j < hidden; ++j)
            yr[j] = (yr[j] - mu) * rs * (double)gamma[j] + (double)beta[j];
        if (mean) mean[i] = mu;
        if (rstd) rstd[i] = rs;
    }
    return 0;
}

int kopref_bias_gelu_residual_layernorm(const void* x, const void* residual,
        const float* bias, const float* gamma, const float* beta,
        double* y, double* mean, double* rstd,
        int64_t rows, int64_t hidden, int64_t x_row_stride, int64_t res_row_stride,
        int64_t y_row_stride, double eps, int dtype, int threads)
{
    return bias_gelu_residual_layernorm_impl(x, residual, bias, gamma, beta, y, mean, rstd, rows, hidden,
                                             x_row_stride, res_row_stride, y_row_stride, eps, dtype, threads, 0);
}

/* The same segment with the error-function GELU in place of the tanh form. */
int kopref_bias_erfgelu_residual_layernorm(const void* x, const void* residual,
        const float* bias, const float* gamma, const float* beta,
        double* y, double* mean, double* rstd,
        int64_t rows, int64_t hidden, int64_t x_row_stride, int64_t res_row_stride,
        int64_t y_row_stride, double eps, int dtype, int threads)
{
    return bias_gelu_residual_layernorm_impl(x, residual, bias, gamma, beta, y, mean, rstd, rows, hidden,
                                             x_row_stride, res_row_stride, y_row_stride, eps, dtype, threads, 1);
}

/* ---- inference BatchNorm affine + ReLU + global average pool (NCHW) ----------
 * a[n,c,h,w] = relu(x[n,c,h,w] * scale[c] + shift[c]) ; p[n,c] = mean_{h,w} a.
 * relu(v) = v if v > 0, 0 otherwise, and NaN stays NaN.  ("reduction +
 * pointwise"; BN / pooling epilogues of the CNN models.)  x and y are
 * contiguous NCHW. y may be NULL (only the pooled output is produced). */
int kopref_bn_relu_avgpool(const void* x, const float* scale, const float* shift,
        double* y, double* pooled, int64_t N, int64_t C, int64_t H, int64_t W,
        int dtype, int threads)
{
    if (!x || !scale || !shift || !pooled) return -1;
    if (N < 0 || C <= 0 || H <= 0 || W <= 0 || bad_dtype(dtype)) return -1;
    int64_t plane = H * W;
    int64_t planes = N * C;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t p = 0; p < planes; ++p) {
        int64_t c = p % C;
        double sc = (double)scale[c], sh = (double)shift[c];
        double sum = 0.0;
        for (int64_t k = 0; k < plane; ++k) {
            double v = load_elem(x, p * plane + k, dtype) * sc + sh;
            double a = (v != v) ? v : (v > 0.0 ? v : 0.0);
            if (y) y[p * plane + k] = a;
            sum += a;
        }
        pooled[p] = sum / (double)plane;
    }
    return 0;
}

/* ---- row-wise cross-entropy ---------------------------------------------------
 * m = max_j z_j ; lse = m + ln sum_j exp(z_j - m) ; loss_i = lse - z[i, label_i] ;
 * mean = (1/M) sum_i loss_i (row order).  ("LogSumExp reductions"; the loss is
 * logsumexp minus the label logit.)  A label outside [0, V) gives loss NaN and
 * is counted in *bad_label_count. mean_loss / bad_label_count may be NULL. */
int kopref_ce_loss_rowwise(const void* logits, const int32_t* labels,
        double* loss, double* mean_loss, int64_t* bad_label_count,
        int64_t rows, int64_t vocab, int64_t row_stride, int dtype, int threads)
{
    if (!logits || !labels || !loss) return -1;
    if (rows < 0 || vocab <= 0 || bad_dtype(dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
        double m = -INFINITY;
        for (int64_t j = 0; j < vocab; ++j) {
            double z = load_elem(logits, i * row_stride + j, dtype);
            if (z > m) m = z;
        }
        double S = 0.0;
        for (int64_t j = 0; j < vocab; ++j)
            S += exp(load_elem(logits, i * row_stride + j, dtype) - m);
        double lse = m + log(S);
        int32_t lab = labels[i];
        if (lab < 0 || (int64_t)lab >= vocab) loss[i] = NAN;
        else loss[i] = lse - load_elem(logits, i * row_stride + lab, dtype);
    }
    int64_t bad = 0;
    double total = 0.0;
    for (int64_t i = 0; i < rows; ++i) {
        int32_t lab = labels[i];
        if (lab < 0 || (int64_t)lab >= vocab) ++bad;
        total += loss[i];
    }
    if (mean_loss) *mean_loss = rows > 0 ? total / (double)rows : NAN;
    if (bad_label_count) *bad_label_count = bad;
    return 0;
}

/* ---- RMSNorm -------------------------------------------------------------------
 * y_j = x_j / sqrt( (1/H) sum_k x_k^2 + eps ) * w_j.  ("RMSNorm sequences".) */
int kopref_rmsnorm(const void* x, const float* weight, double* y,
        int64_t rows, int64_t hidden, int64_t x_row_stride, int64_t y_row_stride,
        double eps, int dtype, int threads)
{
    if (!x || !weight || !y || rows < 0 || hidden <= 0 || bad_dtype(dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
        double ss = 0.0;
        for (int64_t j = 0; j < hidden; ++j) {
            double v = load_elem(x, i * x_row_stride + j, dtype);
            ss += v * v;
        }
        double r = 1.0 / sqrt(ss / (double)hidden + eps);
        for (int64_t j = 0; j < hidden; ++j)
            y[i * y_row_stride + j] =
                load_elem(x, i * x_row_stride + j, dtype) * r * (double)weight[j];
    }
    return 0;
}

/* ---- Lp normalisation of rows (p = 1 or 2) ---------------------------------------
 * n_i = sum_j |x_ij|  (p = 1)   or   sqrt(sum_j x_ij^2)  (p = 2);   y_ij = x_ij / max(n_i, eps).
 * norm_out (may be NULL) receives n_i. ("Normalization fusion": a reduction and the pointwise pass that
 * uses it, in one kernel.) */
int kopref_lp_normalize_rows(const void* x, double* y, double* norm_out, int64_t rows, int64_t cols,
        int64_t x_row_stride, int64_t y_row_stride, int p, double eps, int dtype, int threads)
{
    if (!x || !y || rows < 0 || cols <= 0 || (p != 1 && p != 2) || bad_dtype(dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
        double acc = 0.0;
        for (int64_t j = 0; j < cols; ++j) {
            double v = load_elem(x, i * x_row_stride + j, dtype);
            acc += p == 1 ? fabs(v) : v * v;
        }
        double n = p == 1 ? acc : sqrt(acc);
        if (norm_out) norm_out[i] = n;
        double d = n > eps ? n : eps;             /* a NaN norm fails the comparison: d = eps, y = x / eps ... */
        if (n != n) d = n;                        /* ... so keep the NaN: every output of that row is NaN */
        for (int64_t j = 0; j < cols; ++j) y[i * y_row_stride + j] = load_elem(x, i * x_row_stride + j, dtype) / d;
    }
    return 0;
}

/* ---- SiLU(gate) * up -------------------------------------------------------------
 * Row layout [gate(0..I) | up(I..2I)]; out_j = gate_j / (1 + exp(-gate_j)) * up_j.
 * ("activation fusion (GELU/SiLU/ReLU)"; only the epilogue is fused.) */
int kopref_silu_mul(const void* gate_up, double* out, int64_t rows, int64_t inter,
        int64_t in_row_stride, int64_t out_row_stride, int dtype, int threads)
{
    if (!gate_up || !out || rows < 0 || inter <= 0 || bad_dtype(dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
        for (int64_t j = 0; j < inter; ++j) {
            double g = load_elem(gate_up, i * in_row_stride + j, dtype);
            double u = load_elem(gate_up, i * in_row_stride + inter + j, dtype);
            out[i * out_row_stride + j] = g / (1.0 + exp(-g)) * u;
        }
    }
    return 0;
}

/* ---- residual add ---------------------------------------------------------------
 * out = a + b ("pointwise + pointwise: load once, store once"). */
int kopref_residual_add(const void* a, const void* b, double* out, int64_t rows, int64_t cols,
        int64_t a_row_stride, int64_t b_row_stride, int64_t out_row_stride,
        int dtype, int threads)
{
    if (!a || !b || !out || rows < 0 || cols <= 0 || bad_dtype(dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < rows; ++i)
        for (int64_t j = 0; j < cols; ++j)
            out[i * out_row_stride + j] = load_elem(a, i * a_row_stride + j, dtype)
                                        + load_elem(b, i * b_row_stride + j, dtype);
    return 0;
}

/* ---- C = A * W^T (the preserved vendor GEMM, written as the triple loop) -----------
 * A [M,K] and W [N,K] row-major with their own dtype tags, C [M,N] double.
 * Used only for the chained-segment check. */
int kopref_gemm_nt(const void* A, int a_dtype, const void* Wt, int w_dtype, double* Cout,
        int64_t M, int64_t N, int64_t K, int threads)
{
    if (!A || !Wt || !Cout || M < 0 || N <= 0 || K <= 0) return -1;
    if (bad_dtype(a_dtype) || bad_dtype(w_dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < M; ++i)
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k)
                acc += load_elem(A, i * K + k, a_dtype) * load_elem(Wt, n * K + k, w_dtype);
            Cout[i * N + n] = acc;
        }
    return 0;
}

/* ---- row scale ("diag(a) * B" written as the O(N^2) product the paper's L1-012 case study reaches) ----
 * out[i,j] = a[i] * B[i,j].  a has the data dtype of B. */
int kopref_row_scale(const void* a, const void* B, double* out, int64_t rows, int64_t cols,
        int64_t b_row_stride, int64_t out_row_stride, int dtype, int threads)
{
    if (!a || !B || !out || rows < 0 || cols <= 0 || bad_dtype(dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
        double ai = load_elem(a, i, dtype);
        for (int64_t j = 0; j < cols; ++j)
            out[i * out_row_stride + j] = ai * load_elem(B, i * b_row_stride + j, dtype);
    }
    return 0;
}

/* ---- mat-vec with a bias sum (the form the paper's L2-018 case study reduces Linear -> Sum to) ----------
 * out[i] = sum_k X[i,k] * w[k] + b_sum, with w[k] = sum_j W[j,k] and b_sum = sum_j b[j] precomputed by the
 * caller (w fp32).  The later max / mean / logsumexp of that chain act on a single element per row and
 * are identities. */
int kopref_matvec_bias(const void* X, const float* w, double b_sum, double* out, int64_t M, int64_t K,
        int64_t x_row_stride, int dtype, int threads)
{
    if (!X || !w || !out || M < 0 || K <= 0 || bad_dtype(dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < M; ++i) {
        double acc = 0.0;
        for (int64_t k = 0; k < K; ++k) acc += load_elem(X, i * x_row_stride + k, dtype) * (double)w[k];
        out[i] = acc + b_sum;
    }
    return 0;
}

/* ---- residual add + LayerNorm, and plain LayerNorm ----------------------------------------------------
 * v_j = x_j + r_j (r may be NULL: v = x) ; then LayerNorm exactly as above: biased variance, eps inside
 * the square root, y = (v - mu) rstd gamma + beta.  This is the fusion agent's "residual + norm" pattern
 * without the bias / activation prologue. */
int kopref_residual_layernorm(const void* x, const void* residual, const float* gamma, const float* beta,
        double* y, double* mean, double* rstd, int64_t rows, int64_t hidden, int64_t x_row_stride,
        int64_t res_row_stride, int64_t y_row_stride, double eps, int dtype, int threads)
{
    if (!x || !gamma || !beta || !y || rows < 0 || hidden <= 0 || bad_dtype(dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
        double* yr = y + i * y_row_stride;
        double sum = 0.0;
        for (int64_t j = 0; j < hidden; ++j) {
            double v = load_elem(x, i * x_row_stride + j, dtype);
            if (residual) v += load_elem(residual, i * res_row_stride + j, dtype);
            yr[j] = v;
            sum += v;
        }
        double mu = sum / (double)hidden;
        double ss = 0.0;
        for (int64_t j = 0; j < hidden; ++j) {
            double d = yr[j] - mu;
            ss += d * d;
        }
        double rs = 1.0 / sqrt(ss / (double)hidden + eps);
        for (int64_t j = 0; j < hidden; ++j)
            yr[j] = (yr[j] - mu) * rs * (double)gamma[j] + (double)beta[j];
        if (mean) mean[i] = mu;
        if (rstd) rstd[i] = rs;
    }
    return 0;
}

/* ---- SiLU(gate) * up with interleaved columns ---------------------------------------------------------------
 * Row layout [g0, u0, g1, u1, ...]; out_j = g_j / (1 + exp(-g_j)) * u_j. */
int kopref_silu_mul_interleaved(const void* gate_up, double* out, int64_t rows, int64_t inter,
        int64_t in_row_stride, int64_t out_row_stride, int dtype, int threads)
{
    if (!gate_up || !out || rows < 0 || inter <= 0 || bad_dtype(dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < rows; ++i)
        for (int64_t j = 0; j < inter; ++j) {
            double g = load_elem(gate_up, i * in_row_stride + 2 * j, dtype);
            double u = load_elem(gate_up, i * in_row_stride + 2 * j + 1, dtype);
            out[i * out_row_stride + j] = g / (1.0 + exp(-g)) * u;
        }
    return 0;
}

/* ---- cross-entropy with ignore_index and label smoothing --------------------------------------------------
 * lse_i = logsumexp_j z_ij.  With smoothing s in [0,1):
 *   loss_i = (1 - s) (lse_i - z[i, label_i]) + s (lse_i - (1/V) sum_j z_ij)
 * Rows whose label equals ignore_index give loss 0 and do not count; mean = sum of counted losses /
 * number of counted rows (NaN when none is counted).  A label outside [0, V) that is not ignore_index
 * gives NaN and is counted in *bad_label_count. */
int kopref_ce_loss_opts(const void* logits, const int32_t* labels, double* loss, double* mean_loss,
        int64_t* bad_label_count, int64_t* counted_rows, int64_t rows, int64_t vocab, int64_t row_stride,
        int32_t ignore_index, double smoothing, int dtype, int threads)
{
    if (!logits || !labels || !loss || rows < 0 || vocab <= 0 || bad_dtype(dtype)) return -1;
    if (!(smoothing >= 0.0 && smoothing < 1.0)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
        int32_t lab = labels[i];
        if (lab == ignore_index) { loss[i] = 0.0; continue; }
        double m = -INFINITY, zsum = 0.0;
        for (int64_t j = 0; j < vocab; ++j) {
            double z = load_elem(logits, i * row_stride + j, dtype);
            if (z > m) m = z;
            zsum += z;
        }
        double S = 0.0;
        for (int64_t j = 0; j < vocab; ++j) S += exp(load_elem(logits, i * row_stride + j, dtype) - m);
        double lse = m + log(S);
        if (lab < 0 || (int64_t)lab >= vocab) { loss[i] = NAN; continue; }
        double nll = lse - load_elem(logits, i * row_stride + lab, dtype);
        double smooth = lse - zsum / (double)vocab;
        loss[i] = (1.0 - smoothing) * nll + smoothing * smooth;
    }
    int64_t bad = 0, counted = 0;
    double total = 0.0;
    for (int64_t i = 0; i < rows; ++i) {
        int32_t lab = labels[i];
        if (lab == ignore_index) continue;
        if (lab < 0 || (int64_t)lab >= vocab) ++bad;
        ++counted;
        total += loss[i];
    }
    if (mean_loss) *mean_loss = counted > 0 ? total / (double)counted : NAN;
    if (bad_label_count) *bad_label_count = bad;
    if (counted_rows) *counted_rows = counted;
    return 0;
}

/* Cross-entropy with reduction "sum": the per-row losses of kopref_ce_loss_opts (same options) added up over
 * the rows that count, i.e. mean * counted_rows without the division. No counted row gives 0 (an empty sum). */
int kopref_ce_loss_sum(const void* logits, const int32_t* labels, double* loss, double* sum_loss,
        int64_t rows, int64_t vocab, int64_t row_stride, int32_t ignore_index, double smoothing, int dtype,
        int threads)
{
    if (!sum_loss) return -1;
    int rc = kopref_ce_loss_opts(logits, labels, loss, NULL, NULL, NULL, rows, vocab, row_stride, ignore_index,
                                 smoothing, dtype, threads);
    if (rc != 0) return rc;
    double total = 0.0;
    for (int64_t i = 0; i < rows; ++i)
        if (labels[i] != ignore_index) total += loss[i];
    *sum_loss = total;
    return 0;
}

/* ---- GroupNorm (InstanceNorm when groups == C) + activation, NCHW -------------------------------------------
 * For every image n and group g (C/groups consecutive channels): mu, var (biased) over the group's
 * (C/groups) * H * W elements; y = (x - mu) / sqrt(var + eps) * gamma[c] + beta[c] (gamma / beta may be NULL:
 * 1 and 0); then act: 0 = none, 1 = ReLU (NaN kept), 2 = SiLU.  mean / rstd: [N, groups], may be NULL. */
int kopref_groupnorm_act(const void* x, const float* gamma, const float* beta, double* y, double* mean,
        double* rstd, int64_t N, int64_t C, int64_t H, int64_t W, int64_t groups, double eps, int act,
        int dtype, int threads)
{
    if (!x || !y || N < 0 || C <= 0 || H <= 0 || W <= 0 || groups <= 0 || C % groups || bad_dtype(dtype)) return -1;
    if (act < 0 || act > 2) return -1;
    const int64_t cpg = C / groups, plane = H * W, chunk = cpg * plane;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t ng = 0; ng < N * groups; ++ng) {
        const int64_t g = ng % groups;
        const int64_t base = ng * chunk;
        double sum = 0.0;
        for (int64_t k = 0; k < chunk; ++k) sum += load_elem(x, base + k, dtype);
        const double mu = sum / (double)chunk;
        double ss = 0.0;
        for (int64_t k = 0; k < chunk; ++k) {
            double d = load_elem(x, base + k, dtype) - mu;
            ss += d * d;
        }
        const double rs = 1.0 / sqrt(ss / (double)chunk + eps);
        for (int64_t k = 0; k < chunk; ++k) {
            const int64_t c = g * cpg + k / plane;
            double v = (load_elem(x, base + k, dtype) - mu) * rs;
            v = v * (gamma ? (double)gamma[c] : 1.0) + (beta ? (double)beta[c] : 0.0);
            if (act == 1) v = (v != v) ? v : (v > 0.0 ? v : 0.0);
            else if (act == 2) v = v / (1.0 + exp(-v));
            y[base + k] = v;
        }
        if (mean) mean[ng] = mu;
        if (rstd) rstd[ng] = rs;
    }
    return 0;
}

/* ---- row-wise cumulative sum (the CumSum rows of the paper's per-kernel results table, L1-089..093: plain,
 * reverse, exclusive and masked running sums along the last dimension) ---------------------------------
 * m[i,k] = 1 when mask is NULL, else (mask[i,k] != 0).
 *   inclusive, forward : y[i,j] = sum_{k <= j} x[i,k] m[i,k]
 *   exclusive, forward : y[i,j] = sum_{k <  j} x[i,k] m[i,k]
 *   inclusive, reverse : y[i,j] = sum_{k >= j} x[i,k] m[i,k]
 *   exclusive, reverse : y[i,j] = sum_{k >  j} x[i,k] m[i,k]
 * The running sum is carried in double, in index order. */
int kopref_cumsum_rows(const void* x, const unsigned char* mask, double* y, int64_t rows, int64_t cols,
        int64_t x_row_stride, int64_t mask_row_stride, int64_t y_row_stride, int exclusive, int reverse,
        int dtype, int threads)
{
    if (!x || !y || rows < 0 || cols <= 0 || bad_dtype(dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
        double run = 0.0;
        for (int64_t s = 0; s < cols; ++s) {
            int64_t j = reverse ? cols - 1 - s : s;
            double v = load_elem(x, i * x_row_stride + j, dtype);
            if (mask && mask[i * mask_row_stride + j] == 0) v = 0.0;
            if (exclusive) {
                y[i * y_row_stride + j] = run;
                run += v;
            } else {
                run += v;
                y[i * y_row_stride + j] = run;
            }
        }
    }
    return 0;
}

/* ---- per-channel affine + ReLU + windowed 2-D pooling (NCHW): the BatchNorm -> ReLU -> Pool epilogues that
 * follow the preserved convolutions in the paper's CNN problems ("Pool" is the most frequent non-vendor
 * operation of its level-2 / level-3 tables). --------------------------------------------------------------
 *   a[n,c,i,j] = x[n,c,i,j] * scale[c] + shift[c]   (scale / shift NULL: a = x), then ReLU if relu != 0
 *                (ReLU keeps NaN)
 *   OH = floor((H + 2 ph - kh) / sh) + 1,  OW likewise
 *   window of output (oi, oj): rows oi*sh - ph + di, di in [0, kh); columns oj*sw - pw + dj, dj in [0, kw)
 *   mode 0 (max): y = max of a over the window positions inside the image (padding never wins);
 *                 a NaN inside the window gives NaN
 *   mode 1 (avg): y = (sum of a over the window positions inside the image) / (kh * kw)
 *                 (padding counts as zeros in the divisor)
 * Requires ph <= kh / 2 and pw <= kw / 2, so that every window touches the image. */
int kopref_affine_relu_pool2d(const void* x, const float* scale, const float* shift, double* y, int64_t N,
        int64_t C, int64_t H, int64_t W, int kh, int kw, int sh, int sw, int ph, int pw, int mode, int relu,
        int dtype, int threads)
{
    if (!x || !y || N < 0 || C <= 0 || H <= 0 || W <= 0 || bad_dtype(dtype)) return -1;
    if (kh <= 0 || kw <= 0 || sh <= 0 || sw <= 0 || ph < 0 || pw < 0 || ph > kh / 2 || pw > kw / 2) return -1;
    if (H + 2 * ph < kh || W + 2 * pw < kw || (mode != 0 && mode != 1)) return -1;
    if ((scale == NULL) != (shift == NULL)) return -1;
    int64_t OH = (H + 2 * ph - kh) / sh + 1, OW = (W + 2 * pw - kw) / sw + 1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t p = 0; p < N * C; ++p) {
        int64_t c = p % C;
        double sc = scale ? (double)scale[c] : 1.0, sf = shift ? (double)shift[c] : 0.0;
        for (int64_t oi = 0; oi < OH; ++oi)
            for (int64_t oj = 0; oj < OW; ++oj) {
                double best = -INFINITY, sum = 0.0;
                int saw_nan = 0;
                for (int di = 0; di < kh; ++di)
                    for (int dj = 0; dj < kw; ++dj) {
                        int64_t i = oi * sh - ph + di, j = oj * sw - pw + dj;
                        if (i < 0 || i >= H || j < 0 || j >= W) continue;
                        double a = load_elem(x, (p * H + i) * W + j, dtype);
                        if (scale) a = a * sc + sf;
                        if (relu) a = (a != a) ? a : (a > 0.0 ? a : 0.0);
                        if (a != a) saw_nan = 1;
                        if (a > best) best = a;
                        sum += a;
                    }
                double out = mode == 0 ? (saw_nan ? NAN : best) : sum / (double)(kh * kw);
                y[(p * OH + oi) * OW + oj] = out;
            }
    }
    return 0;
}

/* ---- row reductions (the "Reduction" rows of the paper's result tables: sum / mean / max / min / argmax /
 * argmin over the last dimension, and the LogSumExp reduction its planner names) ---------------------------
 * op 0 sum, 1 mean, 2 max, 3 min, 4 logsumexp = m + ln sum_j exp(x_j - m) with m = max_j x_j.
 * out[i] is the reduced value; index[i] (may be NULL; used for max / min only) is the position of the first
 * element equal to the result. NaN: a NaN anywhere in the row makes every result NaN, and for max / min
 * the index is that of the first NaN (a NaN ranks above every number, and below none, as in torch).
 * logsumexp of a row of -inf is -inf; a +inf element gives +inf. Sums run in index order in double. */
int kopref_reduce_rows(const void* x, double* out, int32_t* index, int64_t rows, int64_t cols,
        int64_t x_row_stride, int op, int dtype, int threads)
{
    if (!x || !out || rows < 0 || cols <= 0 || op < 0 || op > 4 || bad_dtype(dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
        double sum = 0.0, best = (op == 3) ? INFINITY : -INFINITY;
        int64_t where = -1, first_nan = -1;
        for (int64_t j = 0; j < cols; ++j) {
            double v = load_elem(x, i * x_row_stride + j, dtype);
            if (v != v) { if (first_nan < 0) first_nan = j; continue; }
            sum += v;
            if (where < 0 || (op == 3 ? v < best : v > best)) { best = v; where = j; }
        }
        double r;
        if (first_nan >= 0) { r = NAN; where = first_nan; }
        else if (op == 0) r = sum;
        else if (op == 1) r = sum / (double)cols;
        else if (op == 2 || op == 3) r = best;
        else {
            if (isinf(best)) r = best;                    /* all -inf, or a +inf present */
            else {
                double S = 0.0;
                for (int64_t j = 0; j < cols; ++j) S += exp(load_elem(x, i * x_row_stride + j, dtype) - best);
                r = best + log(S);
            }
        }
        out[i] = r;
        if (index && (op == 2 || op == 3)) index[i] = (int32_t)where;
    }
    return 0;
}

/* ---- bias + activation epilogue (the fusion agent's "activation + bias fusion": the pointwise tail of a
 * Linear / GEMM call written once) -----------------------------------------------------------------------
 *   u = x[i,j] + bias[j]  (bias NULL: u = x[i,j]);  y[i,j] = act(u)
 * act: 0 identity, 1 relu (NaN stays NaN), 2 leaky_relu: u > 0 ? u : alpha u, 3 gelu (tanh form),
 * 4 gelu (erf form), 5 silu: u / (1 + exp(-u)), 6 sigmoid: 1 / (1 + exp(-u)), 7 tanh,
 * 8 mish: u tanh(ln(1 + exp(u))), 9 hardswish: u min(max(u + 3, 0), 6) / 6, 10 elu: u > 0 ? u : alpha (exp(u) - 1). */
static double act_value(double u, int act, double alpha)
{
    switch (act) {
    case 0: return u;
    case 1: return (u != u) ? u : (u > 0.0 ? u : 0.0);
    case 2: return u > 0.0 ? u : alpha * u;
    case 3: return kopref_gelu_tanh(u);
    case 4: return kopref_gelu_erf(u);
    case 5: return u / (1.0 + exp(-u));
    case 6: return 1.0 / (1.0 + exp(-u));
    case 7: return tanh(u);
    case 8: return u * tanh(u > 30.0 ? u : log1p(exp(u)));
    case 9: { double r = u + 3.0; r = r < 0.0 ? 0.0 : (r > 6.0 ? 6.0 : r); return (u != u) ? u : u * r / 6.0; }
    default: return u > 0.0 ? u : alpha * expm1(u);
    }
}

double kopref_act_value(double u, int act, double alpha) { return act_value(u, act, alpha); }

int kopref_bias_act(const void* x, const float* bias, double* y, int64_t rows, int64_t cols,
        int64_t x_row_stride, int64_t y_row_stride, int act, double alpha, int dtype, int threads)
{
    if (!x || !y || rows < 0 || cols <= 0 || act < 0 || act > 10 || bad_dtype(dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < rows; ++i)
        for (int64_t j = 0; j < cols; ++j) {
            double u = load_elem(x, i * x_row_stride + j, dtype) + (bias ? (double)bias[j] : 0.0);
            y[i * y_row_stride + j] = act_value(u, act, alpha);
        }
    return 0;
}

/* ---- softmax variants ("fused softmax", "online softmax", LogSoftmax) -------------------------------------
 * z[i,j] = x[i,j] * scale + bias[j] (bias may be NULL). With period > 0 the rows are causal: row i keeps the
 * columns j <= (i mod period) + (cols - period) (period == cols is the square causal mask of attention scores,
 * a smaller period leaves a prefix of cols - period columns visible to every row) and the others count as
 * z = -inf. log_out == 0: y = exp(z - m) / sum_j exp(z_j - m), m = max_j z_j (masked columns give 0);
 * log_out != 0: y = z - m - ln sum_j exp(z_j - m) (masked columns give -inf). */
int kopref_softmax_opts(const void* x, const float* bias, double* y, int64_t rows, int64_t cols,
        int64_t x_row_stride, int64_t y_row_stride, double scale, int log_out, int64_t period, int dtype,
        int threads)
{
    if (!x || !y || rows < 0 || cols <= 0 || period < 0 || period > cols || bad_dtype(dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
        double* yr = y + i * y_row_stride;
        int64_t last = period > 0 ? (i % period) + (cols - period) : cols - 1;   /* last visible column */
        double m = -INFINITY;
        for (int64_t j = 0; j < cols; ++j) {
            double z = j <= last ? load_elem(x, i * x_row_stride + j, dtype) * scale + (bias ? (double)bias[j] : 0.0)
                                 : -INFINITY;
            yr[j] = z;
            if (z > m) m = z;
        }
        double S = 0.0;
        for (int64_t j = 0; j < cols; ++j) S += exp(yr[j] - m);
        double lnS = log(S);
        for (int64_t j = 0; j < cols; ++j) yr[j] = log_out ? (yr[j] - m) - lnS : exp(yr[j] - m) / S;
    }
    return 0;
}

/* ---- pointwise epilogue chain (the paper's L2-064 case: several pointwise operations after a vendor GEMM,
 * fused into one pass; its exact operations are not given, this is the general form of the class) ---------
 *   u = (x[i,j] + bias[j]) * scale + residual[i,j] * residual_scale     (bias / residual NULL: term absent)
 *   u = min(max(u, lo), hi)                                              (NaN stays NaN; lo = -inf, hi = +inf: none)
 *   y = act(u)                                                           (activations of kopref_bias_act) */
int kopref_epilogue_chain(const void* x, const float* bias, const void* residual, double* y, int64_t rows,
        int64_t cols, int64_t x_row_stride, int64_t res_row_stride, int64_t y_row_stride, double scale,
        double residual_scale, double lo, double hi, int act, double alpha, int dtype, int threads)
{
    if (!x || !y || rows < 0 || cols <= 0 || act < 0 || act > 10 || bad_dtype(dtype) || !(lo <= hi)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t i = 0; i < rows; ++i)
        for (int64_t j = 0; j < cols; ++j) {
            double u = (load_elem(x, i * x_row_stride + j, dtype) + (bias ? (double)bias[j] : 0.0)) * scale;
            if (residual) u += load_elem(residual, i * res_row_stride + j, dtype) * residual_scale;
            if (u == u) u = u < lo ? lo : (u > hi ? hi : u);
            y[i * y_row_stride + j] = act_value(u, act, alpha);
        }
    return 0;
}

/* ---- LSTM cell, pointwise part (the gate arithmetic that follows the two preserved GEMMs of an LSTM step; the
 * paper's level-3 table lists LSTM / GRU models) -------------------------------------------------------------
 * gates[b, 0:H] = i, [H:2H] = f, [2H:3H] = g, [3H:4H] = o (pre-activations; gates2 and bias, when given, are
 * added first: a = gates + gates2 + bias):
 *   c_out = sigmoid(f) * c_prev + sigmoid(i) * tanh(g);   h_out = sigmoid(o) * tanh(c_out)
 * h_out uses the unrounded c_out. */
int kopref_lstm_cell(const void* gates, const void* gates2, const float* bias, const void* c_prev, double* h_out,
        double* c_out, int64_t rows, int64_t hidden, int dtype, int threads)
{
    if (!gates || !c_prev || !h_out || !c_out || rows < 0 || hidden <= 0 || bad_dtype(dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t b = 0; b < rows; ++b)
        for (int64_t j = 0; j < hidden; ++j) {
            double a[4];
            for (int k = 0; k < 4; ++k) {
                int64_t idx = b * 4 * hidden + k * hidden + j;
                a[k] = load_elem(gates, idx, dtype) + (gates2 ? load_elem(gates2, idx, dtype) : 0.0)
                     + (bias ? (double)bias[k * hidden + j] : 0.0);
            }
            double ig = 1.0 / (1.0 + exp(-a[0])), fg = 1.0 / (1.0 + exp(-a[1])), gg = tanh(a[2]),
                   og = 1.0 / (1.0 + exp(-a[3]));
            double c = fg * load_elem(c_prev, b * hidden + j, dtype) + ig * gg;
            c_out[b * hidden + j] = c;
            h_out[b * hidden + j] = og * tanh(c);
        }
    return 0;
}

/* ---- GRU cell, pointwise part (what follows the two preserved GEMMs gi = x W_ih^T and gh = h W_hh^T of a GRU
 * step; the paper's level-3 table lists GRU models) ----------------------------------------------------------
 * gi, gh: [rows, 3H], blocks r (reset), z (update), n (candidate); bias_i, bias_h: [3H] or NULL, added to gi
 * and gh respectively (they cannot be merged: the candidate's hidden part is gated before the sum):
 *   r = sigmoid(gi_r + gh_r);  z = sigmoid(gi_z + gh_z);  n = tanh(gi_n + r * gh_n);
 *   h_out = (1 - z) * n + z * h_prev */
int kopref_gru_cell(const void* gi, const void* gh, const float* bias_i, const float* bias_h, const void* h_prev,
        double* h_out, int64_t rows, int64_t hidden, int dtype, int threads)
{
    if (!gi || !gh || !h_prev || !h_out || rows < 0 || hidden <= 0 || bad_dtype(dtype)) return -1;
    int nt = pick_threads(threads);
    (void)nt;
#pragma omp parallel for num_threads(nt) schedule(static)
    for (int64_t b = 0; b < rows; ++b)
        for (int64_t j = 0; j < hidden; ++j) {
            double xi[3], xh[3];
            for (int k = 0; k < 3; ++k) {
                int64_t idx = b * 3 * hidden + k * hidden + j;
                xi[k] = load_elem(gi, idx, dtype) + (bias_i ? (double)bias_i[k * hidden + j] : 0.0);
                xh[k] = load_elem(gh, idx, dtype) + (bias_h ? (double)bias_h[k * hidden + j] : 0.0);
            }
            double r = 1.0 / (1.0 + exp(-(xi[0] + xh[0])));
            double z = 1.0 / (1.0 + exp(-(xi[1] + xh[1])));
            double n = tanh(xi[2] + r * xh[2]);
            h_out[b * hidden + j] = (1.0 - z) * n + z * load_elem(h_prev, b * hidden + j, dtype);
        }
    return 0;
}
