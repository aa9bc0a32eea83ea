/*
 * CPU oracle for the FP8 transformer-block hot path (test infrastructure, NOT a product path).
 *
 * Plain, slow, double-accumulating C.  It shares no code with the CUDA library and must never be
 * called from it; only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * What it follows in the paper:
 *   - FP8 formats E4M3 / E5M2 and their roles (forward / backward tensors): Section 2 (Background).
 *   - per-tensor scaling s(x) = FP8Max / absmax(x): Appendix C (definition before Theorem 1);
 *     rho(X) = FP8Max / (2^m max H): Appendix E.
 *   - end-to-end GEMM(X,Y) = 1/(rho_X rho_Y) * FP8GEMM(cast(rho_X X), cast(rho_Y Y)): Appendix E.
 *   - linear operators Y = XW and which products run in FP8 (QK^T and PV included): Appendix E, Table
 *     "Comparison between FP8 methods".
 *   - attention P = Softmax(s QK^T + M), selfattn = PV, grouped-query heads: Appendix B, Eq. (P).
 * Where the paper is silent (rounding mode, saturation, where FP8 enters inside attention, the backward
 * pass) the reading taken is written at the function.
 *
 * Parity status: codec, amax, scale, cast, GEMM, attention forward and backward (un-quantised: finite
 * differences; quantised: rebuilt step by step in numpy with two query heads per key/value head and a
 * saturating dS scale) and the tie-band rule (hand-worked values) are pinned by tests.
 * The *placement* of the two FP8 encodes inside the attention backward is our reading of "FP8 in forward
 * and backward"; the paper prints no value for it, so that placement stays a reading; its arithmetic is pinned.
 */
#include <float.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_E4M3 0
#define ORACLE_E5M2 1

/* ------------------------------------------------------------------------------------------------
 * Codec (Section 2: E4M3 = 1 sign, 4 exponent, 3 mantissa bits; E5M2 = 1-5-2).
 * E4M3 has no infinities and a single NaN mantissa pattern (S.1111.111); E5M2 is IEEE-like.
 * ---------------------------------------------------------------------------------------------- */
static int fmt_mbits(int fmt) { return fmt == ORACLE_E4M3 ? 3 : 2; }
static int fmt_ebits(int fmt) { return fmt == ORACLE_E4M3 ? 4 : 5; }
static int fmt_bias(int fmt) { return fmt == ORACLE_E4M3 ? 7 : 15; }

double oracle_fp8_max(int fmt) { return fmt == ORACLE_E4M3 ? 448.0 : 57344.0; }

double oracle_fp8_decode(uint8_t code, int fmt)
{
    const int mb = fmt_mbits(fmt), eb = fmt_ebits(fmt), bias = fmt_bias(fmt);
    const int sign = code >> 7;
    const int E = (code >> mb) & ((1 << eb) - 1);
    const int M = code & ((1 << mb) - 1);
    double v;
    if (fmt == ORACLE_E4M3) {
        if (E == 15 && M == 7) return NAN;
    } else {
        if (E == 31) return M == 0 ? (sign ? -INFINITY : INFINITY) : NAN;
    }
    if (E == 0)
        v = ldexp((double)M, 1 - bias - mb);                       /* subnormal: M * 2^(1-bias-mbits) */
    else
        v = ldexp(1.0 + (double)M / (double)(1 << mb), E - bias);  /* normal */
    return sign ? -v : v;
}

/* binary32 -> FP8 code, round-to-nearest-even, saturating to the largest finite value.
 * Reading (paper silent on rounding/overflow): finite inputs never produce Inf/NaN; +-Inf saturates;
 * NaN gives the NaN pattern 0x7F; the sign of zero and of values that round to zero is kept. */
uint8_t oracle_fp8_encode(float v, int fmt)
{
    const int mb = fmt_mbits(fmt), bias = fmt_bias(fmt);
    const double maxv = oracle_fp8_max(fmt);
    const double min_normal = ldexp(1.0, 1 - bias);
    const double min_sub = ldexp(1.0, 1 - bias - mb);
    if (isnan(v)) return 0x7F;
    const uint8_t sign = signbit(v) ? 0x80 : 0x00;
    const double a = fabs((double)v);
    uint8_t code;
    if (a > maxv) {
        code = (fmt == ORACLE_E4M3) ? 0x7E : 0x7B;
    } else if (a < min_normal) {
        /* fixed-point grid of step min_sub; nearbyint rounds half to even in the default mode;
         * q == 2^mbits is the code of min_normal by continuity of the encoding */
        code = (uint8_t)nearbyint(a / min_sub);
    } else {
        int ex;
        (void)frexp(a, &ex);          /* a = f * 2^ex, f in [0.5,1) */
        int e = ex - 1;               /* a = (1+frac) * 2^e */
        double frac = a / ldexp(1.0, e) - 1.0;
        int q = (int)nearbyint(frac * (double)(1 << mb));
        if (q == (1 << mb)) { q = 0; e += 1; }
        code = (uint8_t)(((e + bias) << mb) | q);
    }
    return (uint8_t)(code | sign);
}

void oracle_fp8_decode_table(int fmt, double *out256)
{
    for (int c = 0; c < 256; ++c) out256[c] = oracle_fp8_decode((uint8_t)c, fmt);
}

void oracle_fp8_encode_array(const float *v, size_t n, int fmt, uint8_t *out)
{
    for (size_t i = 0; i < n; ++i) out[i] = oracle_fp8_encode(v[i], fmt);
}

static float bf16_bits_to_float(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* ------------------------------------------------------------------------------------------------
 * amax: absmax(x) of Appendix C / max|x| of Appendix E, over a BF16 tensor.
 * |x| ordering of finite BF16 values equals the ordering of (bits & 0x7FFF) as integers.
 * ---------------------------------------------------------------------------------------------- */
float oracle_amax_bf16(const uint16_t *x, size_t n)
{
    uint16_t best = 0;
    for (size_t i = 0; i < n; ++i) {
        uint16_t m = (uint16_t)(x[i] & 0x7FFF);
        if (m > best) best = m;
    }
    return bf16_bits_to_float(best);
}

/* ------------------------------------------------------------------------------------------------
 * scale: s = FP8Max / (2^margin * amax) (Appendix C with margin 0; Appendix E with H = {amax}).
 * One binary32 division, then an exact power-of-two factor; scale_inv is one more binary32 division.
 * Readings (paper silent): amax == 0 or non-finite -> scale 1; an overflowing quotient -> FLT_MAX.
 * ---------------------------------------------------------------------------------------------- */
void oracle_scale(float amax, int fmt, int margin, float *scale, float *scale_inv)
{
    volatile float s;
    if (!(amax > 0.0f) || isinf(amax)) {
        s = 1.0f;
    } else {
        volatile float q = (float)oracle_fp8_max(fmt) / amax;
        s = q * ldexpf(1.0f, -margin);
        if (isinf(s)) s = FLT_MAX;
    }
    volatile float inv = 1.0f / s;
    *scale = s;
    *scale_inv = inv;
}

/* ------------------------------------------------------------------------------------------------
 * Delayed scaling (Appendix E): H = {h_1..h_l} holds the last l abs-max values of a tensor,
 * rho = FP8Max / (2^m max H), and after a step H <- {amax(X)} u {h_t}_{t=2..l}; the updated history
 * serves the following step.  Reading of the set notation: a FIFO, the dropped h_1 is the oldest entry; the new scale is
 * computed from the history *after* the insertion and is the one the next step casts with.  `head` is
 * the position of the oldest entry.  Entries that were never written are 0 and an all-zero history
 * gives scale 1 (same guard as oracle_scale).
 * ---------------------------------------------------------------------------------------------- */
void oracle_scale_update(float *history, int len, int *head, float amax_new, int fmt, int margin,
                         float *scale, float *scale_inv)
{
    history[*head] = amax_new;
    *head = (*head + 1) % len;
    float mx = 0.0f;
    for (int i = 0; i < len; ++i)
        if (history[i] > mx || isnan(history[i])) mx = history[i];
    oracle_scale(mx, fmt, margin, scale, scale_inv);
}

/* ------------------------------------------------------------------------------------------------
 * cast: FP8cast(rho * X) of Appendix E.  Reading of the precision (paper silent): the BF16 value is
 * widened exactly to binary32, multiplied by the scale in binary32 (round-to-nearest), and the product
 * is rounded once more to FP8 by oracle_fp8_encode.  out_t, if not NULL, is the same codes laid out
 * [cols, rows].
 * ---------------------------------------------------------------------------------------------- */
void oracle_cast_bf16(const uint16_t *x, size_t rows, size_t cols, float scale, int fmt,
                      uint8_t *out, uint8_t *out_t)
{
#pragma omp parallel for schedule(static)
    for (long r = 0; r < (long)rows; ++r) {
        for (size_t c = 0; c < cols; ++c) {
            volatile float p = bf16_bits_to_float(x[(size_t)r * cols + c]) * scale;
            uint8_t code = oracle_fp8_encode(p, fmt);
            if (out) out[(size_t)r * cols + c] = code;
            if (out_t) out_t[c * rows + (size_t)r] = code;
        }
    }
}

/* ------------------------------------------------------------------------------------------------
 * Kurtosis monitor (Section 4, "Long-term outlier dynamics"): kurt(x) = mu[x^4] / sigma^2[x]^2 for one token
 * vector x, without centring, averaged over the tokens of the tensor.  Reading of the printed formula
 * (its denominator is typeset as the variance of x^2): the un-centred second moment of x, squared, i.e.
 * mu[x^4] / mu[x^2]^2 - the only reading under which the quantity peaks for a vector dominated by a handful of
 * outliers, as the section says it does (a one-hot vector of length D gives D, a constant vector 1, a Gaussian about 3).
 * A row of zeros contributes 0.
 * ---------------------------------------------------------------------------------------------- */
double oracle_kurtosis_bf16(const uint16_t *x, size_t rows, size_t cols)
{
    double total = 0.0;
#pragma omp parallel for reduction(+ : total) schedule(static)
    for (long r = 0; r < (long)rows; ++r) {
        double s2 = 0.0, s4 = 0.0;
        for (size_t c = 0; c < cols; ++c) {
            double v = (double)bf16_bits_to_float(x[(size_t)r * cols + c]);
            s2 += v * v;
            s4 += v * v * v * v;
        }
        if (s2 > 0.0) total += (s4 / (double)cols) / ((s2 / (double)cols) * (s2 / (double)cols));
    }
    return total / (double)rows;
}

static uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x40);   /* NaN stays NaN */
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

/* ------------------------------------------------------------------------------------------------
 * Gated activation feeding the second FFN projection (Appendix B: FFN with activation phi; the Llama-style
 * workloads use SwiGLU): h = silu(gate) * up, silu(g) = g / (1 + exp(-g)), gate = columns [0,F) and
 * up = columns [F,2F) of the fused first-projection output.  h is rounded to BF16 (what a BF16 framework
 * would hold) and that tensor is what amax and the cast see, so the rest equals oracle_cast_bf16.
 * ---------------------------------------------------------------------------------------------- */
void oracle_swiglu_bf16(const uint16_t *gate_up, size_t T, size_t F, uint16_t *h)
{
#pragma omp parallel for schedule(static)
    for (long t = 0; t < (long)T; ++t)
        for (size_t f = 0; f < F; ++f) {
            double g = (double)bf16_bits_to_float(gate_up[(size_t)t * 2 * F + f]);
            double u = (double)bf16_bits_to_float(gate_up[(size_t)t * 2 * F + F + f]);
            h[(size_t)t * F + f] = f32_to_bf16_rne((float)(g / (1.0 + exp(-g)) * u));
        }
}

/* ------------------------------------------------------------------------------------------------
 * Element-wise FFN activations of the other architecture families (Appendix B, architecture table):
 *   act 1  GeLU(x)  = x * Phi(x) = 0.5 x (1 + erf(x / sqrt 2))     (exact form; the paper names no approximation)
 *   act 2  xIELU(x) = alpha_p x^2 + 0.5 x                          for x > 0      (Appendix B, Eq. (xIELU))
 *                     alpha_n (e^x - 1) - alpha_n x + 0.5 x        for x <= 0
 * x is the [T,F] BF16 output of the first FFN projection; h is rounded to BF16 like oracle_swiglu_bf16.
 * ---------------------------------------------------------------------------------------------- */
void oracle_activation_bf16(const uint16_t *x, size_t n, int act, double alpha_p, double alpha_n, uint16_t *h)
{
#pragma omp parallel for schedule(static)
    for (long i = 0; i < (long)n; ++i) {
        double v = (double)bf16_bits_to_float(x[i]), r;
        if (act == 1) r = 0.5 * v * (1.0 + erf(v * 0.70710678118654752440));
        else r = v > 0.0 ? alpha_p * v * v + 0.5 * v : alpha_n * expm1(v) - alpha_n * v + 0.5 * v;
        h[i] = f32_to_bf16_rne((float)r);
    }
}

/* ------------------------------------------------------------------------------------------------
 * Post-normalisation + residual (Section 3; Appendix B: block(X) = X^ + (N_post o FFN)(X^), X^ = X + (N_post o GQA)(X)):
 *   mode 0  RMSNorm     out = x + gamma (.) y / rms(y),  rms(y) = sqrt(mean(y^2) + eps)   (the paper's N_gamma has eps = 0)
 *   mode 1  LayerScale  out = x + gamma (.) y
 * x (residual stream), y (branch output): [T,D] BF16; gamma: D binary32; out rounded to BF16.
 * ---------------------------------------------------------------------------------------------- */
/* x_scale multiplies the residual input: 1 inside the network, sigma_0^-1 on the first block's input (Section 3: the
 * input of the first block is scaled by the inverse of the initialisation standard deviation; Appendix B,
 * architecture table, column "input scaling"). */
void oracle_postnorm_residual_scaled_bf16(const uint16_t *x, const uint16_t *y, const float *gamma, size_t T, size_t D,
                                          int mode, double eps, double x_scale, uint16_t *out)
{
#pragma omp parallel for schedule(static)
    for (long t = 0; t < (long)T; ++t) {
        double ss = 0.0;
        for (size_t d = 0; d < D; ++d) {
            double v = (double)bf16_bits_to_float(y[(size_t)t * D + d]);
            ss += v * v;
        }
        double rinv = mode == 0 ? 1.0 / sqrt(ss / (double)D + eps) : 1.0;
        for (size_t d = 0; d < D; ++d) {
            double r = x_scale * (double)bf16_bits_to_float(x[(size_t)t * D + d]) +
                       (double)gamma[d] * (double)bf16_bits_to_float(y[(size_t)t * D + d]) * rinv;
            out[(size_t)t * D + d] = f32_to_bf16_rne((float)r);
        }
    }
}

void oracle_postnorm_residual_bf16(const uint16_t *x, const uint16_t *y, const float *gamma, size_t T, size_t D,
                                   int mode, double eps, uint16_t *out)
{
    oracle_postnorm_residual_scaled_bf16(x, y, gamma, T, D, mode, eps, 1.0, out);
}

/* ------------------------------------------------------------------------------------------------
 * QK entropy regulariser + rotary embedding on a [T, H, d] BF16 tensor of per-head vectors (Section 3, Appendix B:
 * attnhead = selfattn(N_QK(X W_Q), N_QK(X W_K), X W_V), "standard" GQA with rotary position embeddings):
 *   mode 0  N(v) = v / rms(v)  over the d entries of one head (frozen unit gain: the gain lives in the softmax scale)
 *   mode 1  tanh(alpha v) element-wise
 *   mode 2  identity
 * then rotation of the pairs (i, i + d/2) by the angle of position pos = t mod seq_len:
 *   out[i]       = v[i] cos[pos,i] - v[i+d/2] sin[pos,i]
 *   out[i+d/2]   = v[i+d/2] cos[pos,i] + v[i] sin[pos,i]         cos, sin: [seq_len, d/2] binary32 tables (inputs)
 * rounded to BF16.  cos == NULL skips the rotation.
 * ---------------------------------------------------------------------------------------------- */
void oracle_qk_norm_rope_bf16(const uint16_t *x, size_t T, size_t H, size_t d, int mode, double alpha, double eps,
                              const float *cos_t, const float *sin_t, size_t seq_len, uint16_t *out)
{
#pragma omp parallel for schedule(static)
    for (long t = 0; t < (long)T; ++t) {
        double v[1024];
        for (size_t h = 0; h < H; ++h) {
            const uint16_t *px = x + ((size_t)t * H + h) * d;
            uint16_t *po = out + ((size_t)t * H + h) * d;
            double ss = 0.0;
            for (size_t i = 0; i < d; ++i) {
                v[i] = (double)bf16_bits_to_float(px[i]);
                ss += v[i] * v[i];
            }
            if (mode == 0) {
                double rinv = 1.0 / sqrt(ss / (double)d + eps);
                for (size_t i = 0; i < d; ++i) v[i] *= rinv;
            } else if (mode == 1) {
                for (size_t i = 0; i < d; ++i) v[i] = tanh(alpha * v[i]);
            }
            if (cos_t) {
                size_t pos = (size_t)t % seq_len, hd = d / 2;
                for (size_t i = 0; i < hd; ++i) {
                    double c = (double)cos_t[pos * hd + i], sn = (double)sin_t[pos * hd + i];
                    double a = v[i], b = v[i + hd];
                    v[i] = a * c - b * sn;
                    v[i + hd] = b * c + a * sn;
                }
            }
            for (size_t i = 0; i < d; ++i) po[i] = f32_to_bf16_rne((float)v[i]);
        }
    }
}

/* ------------------------------------------------------------------------------------------------
 * FP8 GEMM with descale (Appendix E): ref[i,j] = sa_inv*sb_inv * sum_k dec(A[i,k]) * dec(B[j,k]),
 * accumulated in double, on a list of output rows and columns.  A and B are addressed through
 * (row stride, reduction stride) so that the three linear products are this one routine on three
 * index patterns (see the wrappers below).  mag is the same sum over absolute values.
 * ---------------------------------------------------------------------------------------------- */
void oracle_gemm_sampled(const uint8_t *A, int fmtA, int64_t a_rs, int64_t a_ks,
                         const uint8_t *B, int fmtB, int64_t b_rs, int64_t b_ks,
                         double sa_inv, double sb_inv, int64_t kred,
                         const int64_t *rows, int64_t nrows, const int64_t *cols, int64_t ncols,
                         const double *prev, double *ref, double *mag)
{
    double ta[256], tb[256];
    oracle_fp8_decode_table(fmtA, ta);
    oracle_fp8_decode_table(fmtB, tb);
#pragma omp parallel for collapse(2) schedule(dynamic, 16)
    for (int64_t ii = 0; ii < nrows; ++ii) {
        for (int64_t jj = 0; jj < ncols; ++jj) {
            const uint8_t *pa = A + rows[ii] * a_rs;
            const uint8_t *pb = B + cols[jj] * b_rs;
            double acc = 0.0, am = 0.0;
            for (int64_t k = 0; k < kred; ++k) {
                double a = ta[pa[k * a_ks]], b = tb[pb[k * b_ks]];
                acc += a * b;
                am += fabs(a) * fabs(b);
            }
            double r = sa_inv * sb_inv * acc;
            if (prev) r += prev[ii * ncols + jj];
            ref[ii * ncols + jj] = r;
            if (mag) mag[ii * ncols + jj] = sa_inv * sb_inv * am;
        }
    }
}

/* Y[t,n] = sum_k X8[t,k] W8[n,k]   (Linear_W(X) = XW with W stored [out,in]; X, W in E4M3) */
void oracle_linear_fwd(const uint8_t *X8, const uint8_t *W8, double sx_inv, double sw_inv,
                       int64_t T, int64_t N, int64_t K,
                       const int64_t *rows, int64_t nrows, const int64_t *cols, int64_t ncols,
                       double *ref, double *mag)
{
    (void)T; (void)N;
    oracle_gemm_sampled(X8, ORACLE_E4M3, K, 1, W8, ORACLE_E4M3, K, 1, sx_inv, sw_inv, K,
                        rows, nrows, cols, ncols, NULL, ref, mag);
}

/* dX[t,k] = sum_n dY8[t,n] W8[n,k]   (dY in E5M2, W in E4M3) */
void oracle_linear_dgrad(const uint8_t *dY8, const uint8_t *W8, double sdy_inv, double sw_inv,
                         int64_t T, int64_t N, int64_t K,
                         const int64_t *rows, int64_t nrows, const int64_t *cols, int64_t ncols,
                         double *ref, double *mag)
{
    (void)T;
    oracle_gemm_sampled(dY8, ORACLE_E5M2, N, 1, W8, ORACLE_E4M3, 1, K, sdy_inv, sw_inv, N,
                        rows, nrows, cols, ncols, NULL, ref, mag);
}

/* dW[n,k] = (prev[n,k]) + sum_t dY8[t,n] X8[t,k]   (dY in E5M2, X in E4M3) */
void oracle_linear_wgrad(const uint8_t *dY8, const uint8_t *X8, double sdy_inv, double sx_inv,
                         int64_t T, int64_t N, int64_t K,
                         const int64_t *rows, int64_t nrows, const int64_t *cols, int64_t ncols,
                         const double *prev, double *ref, double *mag)
{
    oracle_gemm_sampled(dY8, ORACLE_E5M2, 1, N, X8, ORACLE_E4M3, 1, K, sdy_inv, sx_inv, T,
                        rows, nrows, cols, ncols, prev, ref, mag);
}

/* ------------------------------------------------------------------------------------------------
 * Attention (Appendix B, Eq. (P): P = Softmax(s QK^T + M), output PV; grouped-query heads).
 * Tensors are [B, N, H, d]; query head h reads key/value head h / (Hq/Hkv).  M is the causal mask
 * (0 for key <= query, -inf otherwise) or absent.
 *
 * An operand is either FP8 codes (decoded through a table) or real values in double; the second form
 * exists so that the un-quantised arithmetic can be checked by finite differences.
 * ---------------------------------------------------------------------------------------------- */
typedef struct {
    int32_t B, N, Hq, Hkv, d;
    int32_t causal;
    int32_t quant;     /* 1: P -> E4M3 and dS -> E5M2 are applied; 0: both encodes dropped */
    int32_t kv_block;  /* forward: 0 = whole row at once, else keys are taken in blocks of this length */
    int32_t max_mode;  /* forward: 0 = exact running maximum; 1 = maximum of x*log2(e) rounded up to an integer */
    int32_t pad_;
    double s;          /* softmax scale */
    double c_P;        /* quantisation scale of P~ = exp(x - m) in (0,1]; 448 = FP8Max/amax with amax = 1 */
    double q_inv, k_inv, v_inv, do_inv;  /* descales of Q8, K8, V8, dO8 */
    double ds_scale;   /* backward: quantisation scale of dS */
    double flip_eps;   /* relative uncertainty of an FP32 evaluation (0 disables the slack outputs) */
    double max_slack;  /* forward: tau >= 0 in powers of two; the reference maximum m moves only when a block maximum
                        * exceeds it by more than 2^tau, i.e. by tau*ln2 in the exponent (0: whenever it grows) */
} oracle_attn_params;

typedef struct {
    const uint8_t *codes;   /* used when vals == NULL */
    const double *vals;
    double table[256];
} operand;

static void operand_init(operand *o, const uint8_t *codes, const double *vals, int fmt)
{
    o->codes = codes;
    o->vals = vals;
    oracle_fp8_decode_table(fmt, o->table);
}
static inline double ld(const operand *o, int64_t idx)
{
    return o->vals ? o->vals[idx] : o->table[o->codes[idx]];
}
static inline int64_t idx4(const oracle_attn_params *p, int H, int b, int n, int h, int dd)
{
    return (((int64_t)b * p->N + n) * H + h) * p->d + dd;
}

/* x_ij = s * q_inv * k_inv * sum_d Q[i,h,d] K[j,g,d] */
static double score(const oracle_attn_params *p, const operand *Q, const operand *K,
                    int b, int h, int g, int i, int j)
{
    double acc = 0.0;
    for (int dd = 0; dd < p->d; ++dd)
        acc += ld(Q, idx4(p, p->Hq, b, i, h, dd)) * ld(K, idx4(p, p->Hkv, b, j, g, dd));
    return p->s * p->q_inv * p->k_inv * acc;
}

/* same sum over absolute values: the size against which an FP32 evaluation of x_ij is accurate */
static double score_mag(const oracle_attn_params *p, const operand *Q, const operand *K,
                        int b, int h, int g, int i, int j)
{
    double acc = 0.0;
    for (int dd = 0; dd < p->d; ++dd)
        acc += fabs(ld(Q, idx4(p, p->Hq, b, i, h, dd)) * ld(K, idx4(p, p->Hkv, b, j, g, dd)));
    return p->s * p->q_inv * p->k_inv * acc;
}

/* Where a value about to be encoded lies within `band` of the rounding boundary between two neighbouring
 * codes, a kernel that evaluates it in binary32 may legitimately pick the other code.  Returns the distance
 * between the two candidate values in that case, else 0.  The sums of these distances (times the other
 * operand's magnitude) are the `slack` outputs: the amount by which a correct FP32 implementation may
 * differ from this double-precision one through such tie decisions alone. */
static double flip_step(double y, double band, int fmt)
{
    if (!(band > 0.0)) return 0.0;
    const double a = fabs(y);
    const int top = (fmt == ORACLE_E4M3) ? 0x7E : 0x7B;
    if (a > oracle_fp8_max(fmt) + band) return 0.0;
    const int c = oracle_fp8_encode((float)a, fmt) & 0x7F;
    const double v = oracle_fp8_decode((uint8_t)c, fmt);
    if (c < top) {
        const double up = oracle_fp8_decode((uint8_t)(c + 1), fmt);
        if (0.5 * (v + up) - a <= band) return up - v;
    }
    if (c > 0) {
        const double dn = oracle_fp8_decode((uint8_t)(c - 1), fmt);
        if (a - 0.5 * (v + dn) <= band) return v - dn;
    }
    return 0.0;
}

static double quant_p(const oracle_attn_params *p, double pt)
{
    /* P~ * c_P is formed as a binary32 product and rounded once to E4M3; returned still scaled by c_P */
    if (!p->quant) return pt;
    volatile float prod = (float)pt * (float)p->c_P;
    return oracle_fp8_decode(oracle_fp8_encode(prod, ORACLE_E4M3), ORACLE_E4M3);
}

/* Forward for the listed (batch, query head) pairs and query rows [r0, r1).
 * Reading of where FP8 enters (paper: "QK^T and PV in FP8", nothing more): Q, K, V arrive as E4M3 codes;
 * scores and the softmax are real-valued; P~ = exp(x - m) is re-quantised to E4M3 with scale c_P right
 * before the PV product; the row sum l uses the un-quantised P~, so LSE is the true log-sum-exp.
 * Outputs: O[pair][row][d], LSE[pair][row], mag (sum of |P8||V| with the same normalisation; may be NULL). */
static void attention_fwd_core(const operand *Q, const operand *K, const operand *V,
                               const oracle_attn_params *p, const int32_t *bh, int nbh, int r0, int r1,
                               double *O, double *LSE, double *mag, double *slack)
{
    const int d = p->d, nr = r1 - r0, G = p->Hq / p->Hkv;
    const int want_slack = slack != NULL && p->quant && p->flip_eps > 0.0;
    const double LOG2E = 1.4426950408889634074, LN2 = 0.69314718055994530942;
    const double cP = p->quant ? p->c_P : 1.0;
#pragma omp parallel for collapse(2) schedule(dynamic, 8)
    for (int pi = 0; pi < nbh; ++pi) {
        for (int i = r0; i < r1; ++i) {
            const int b = bh[2 * pi], h = bh[2 * pi + 1], g = h / G;
            const int jlast = p->causal ? i : p->N - 1;
            const int Bc = p->kv_block > 0 ? p->kv_block : p->N;
            double *x = (double *)malloc(sizeof(double) * (size_t)Bc);
            double *acc = (double *)calloc((size_t)d, sizeof(double));
            double *am = (double *)calloc((size_t)d, sizeof(double));
            double *sl = (double *)calloc((size_t)d, sizeof(double));
            double m = -INFINITY, l = 0.0;
            for (int j0 = 0; j0 <= jlast; j0 += Bc) {
                const int j1 = (j0 + Bc - 1 < jlast) ? j0 + Bc - 1 : jlast;
                double bm = -INFINITY;
                for (int j = j0; j <= j1; ++j) {
                    x[j - j0] = score(p, Q, K, b, h, g, i, j);
                    if (x[j - j0] > bm) bm = x[j - j0];
                }
                double cand = (p->max_mode == 1) ? ceil(bm * LOG2E) * LN2 : bm;
                if (cand > m + p->max_slack * LN2) {
                    double f = isinf(m) ? 0.0 : exp(m - cand);
                    l *= f;
                    for (int dd = 0; dd < d; ++dd) { acc[dd] *= f; am[dd] *= f; sl[dd] *= f; }
                    m = cand;
                }
                for (int j = j0; j <= j1; ++j) {
                    double pt = exp(x[j - j0] - m);
                    l += pt;
                    double w = quant_p(p, pt);
                    double step = 0.0;
                    if (want_slack) {
                        /* P~ inherits the absolute error of its exponent: eps * (1 + |terms of x|) */
                        const double y = pt * p->c_P;
                        step = flip_step(y, y * p->flip_eps * (1.0 + score_mag(p, Q, K, b, h, g, i, j)), ORACLE_E4M3);
                    }
                    for (int dd = 0; dd < d; ++dd) {
                        double v = ld(V, idx4(p, p->Hkv, b, j, g, dd));
                        acc[dd] += w * v;
                        am[dd] += w * fabs(v);
                        sl[dd] += step * fabs(v);
                    }
                }
            }
            int64_t o = ((int64_t)pi * nr + (i - r0));
            for (int dd = 0; dd < d; ++dd) {
                O[o * d + dd] = p->v_inv * acc[dd] / (cP * l);
                if (mag) mag[o * d + dd] = p->v_inv * am[dd] / (cP * l);
                if (slack) slack[o * d + dd] = p->v_inv * sl[dd] / (cP * l);
            }
            LSE[o] = m + log(l);
            free(x); free(acc); free(am); free(sl);
        }
    }
}

void oracle_attention_fwd(const uint8_t *Q8, const uint8_t *K8, const uint8_t *V8,
                          const oracle_attn_params *p, const int32_t *bh, int nbh, int r0, int r1,
                          double *O, double *LSE, double *mag, double *slack)
{
    operand Q, K, V;
    operand_init(&Q, Q8, NULL, ORACLE_E4M3);
    operand_init(&K, K8, NULL, ORACLE_E4M3);
    operand_init(&V, V8, NULL, ORACLE_E4M3);
    attention_fwd_core(&Q, &K, &V, p, bh, nbh, r0, r1, O, LSE, mag, slack);
}

/* Same arithmetic on real-valued operands (used with quant = 0 for the finite-difference pin). */
void oracle_attention_fwd_real(const double *Qd, const double *Kd, const double *Vd,
                               const oracle_attn_params *p, const int32_t *bh, int nbh, int r0, int r1,
                               double *O, double *LSE, double *mag, double *slack)
{
    operand Q, K, V;
    operand_init(&Q, NULL, Qd, ORACLE_E4M3);
    operand_init(&K, NULL, Kd, ORACLE_E4M3);
    operand_init(&V, NULL, Vd, ORACLE_E4M3);
    attention_fwd_core(&Q, &K, &V, p, bh, nbh, r0, r1, O, LSE, mag, slack);
}

/* Backward of O = PV through the softmax (the paper runs it in FP8 too but gives no formula; this is the
 * textbook derivative with the FP8 encodes placed where a GEMM operand is produced):
 *   D_i  = sum_d dO_id O_id                    P_ij = exp(x_ij - LSE_i)
 *   dV_j = sum_i P8_ij/c_P * dO_i              dP_ij = dO_i . V_j
 *   dS_ij = P_ij (dP_ij - D_i)                 dS8 = E5M2(dS * ds_scale)
 *   dQ_i = s sum_j dS8_ij/ds_scale * K_j       dK_j = s sum_i dS8_ij/ds_scale * Q_i
 * with dO = do_inv*dec(dO8), V = v_inv*dec(V8) and so on; dK, dV sum over the query heads of a group.
 * Covers query rows [q0,q1) x key rows [k0,k1) for the listed (batch, kv head) pairs: dQ is complete
 * when the key range holds every key the rows attend to, dK/dV when the query range holds every query
 * that attends to the keys.  O is [B,N,Hq,d] and LSE [B,Hq,N], given by the caller.
 * Outputs: dQ[pair][G][q1-q0][d], dK,dV[pair][k1-k0][d], amax of |dS|, and (nullable) the magnitude sums
 * that serve as error-metric denominators: for dV the sum of |P8||dO|; for dQ and dK the sums of
 * P(|dP| + |D|)|K| resp. P(|dP| + |D|)|Q|, i.e. the size of the terms *before* dP - D cancels (the
 * componentwise condition of the formula: where softmax is nearly one-hot, dP - D is a difference of two
 * nearly equal numbers and an FP32 evaluation is only accurate relative to those numbers). */
static void attention_bwd_core(const operand *Q, const operand *K, const operand *V, const operand *dO,
                               const double *O, const double *LSE, const oracle_attn_params *p,
                               const int32_t *bg, int nbg, int q0, int q1, int k0, int k1,
                               double *dQ, double *dK, double *dV,
                               double *mag_dQ, double *mag_dK, double *mag_dV, double *amax_dS,
                               double *slack_dQ, double *slack_dK, double *slack_dV,
                               double *mag8_dQ, double *mag8_dK)
{
    const int d = p->d, G = p->Hq / p->Hkv, nq = q1 - q0, nk = k1 - k0;
    const double cP = p->quant ? p->c_P : 1.0;
    const int want_slack = p->quant && p->flip_eps > 0.0 && slack_dQ && slack_dK && slack_dV;
    double amax = 0.0;
    /* D_i for every (pair, head in group, row), and the sum of the absolute terms of D_i */
    double *D = (double *)malloc(sizeof(double) * (size_t)nbg * G * nq);
    double *Dm = (double *)malloc(sizeof(double) * (size_t)nbg * G * nq);
#pragma omp parallel for collapse(2) schedule(static)
    for (int pi = 0; pi < nbg; ++pi)
        for (int r = 0; r < G * nq; ++r) {
            const int b = bg[2 * pi], g = bg[2 * pi + 1], h = g * G + r / nq, i = q0 + r % nq;
            double acc = 0.0, accm = 0.0;
            for (int dd = 0; dd < d; ++dd) {
                const double t = p->do_inv * ld(dO, idx4(p, p->Hq, b, i, h, dd)) * O[idx4(p, p->Hq, b, i, h, dd)];
                acc += t;
                accm += fabs(t);
            }
            D[((int64_t)pi * G + r / nq) * nq + r % nq] = acc;
            Dm[((int64_t)pi * G + r / nq) * nq + r % nq] = accm;
        }

    /* row-local pass: dQ_i, and amax|dS| */
#pragma omp parallel for collapse(2) schedule(dynamic, 8) reduction(max : amax)
    for (int pi = 0; pi < nbg; ++pi)
        for (int r = 0; r < G * nq; ++r) {
            const int b = bg[2 * pi], g = bg[2 * pi + 1], hg = r / nq, h = g * G + hg, i = q0 + r % nq;
            const double lse = LSE[((int64_t)b * p->Hq + h) * p->N + i];
            const double Di = D[((int64_t)pi * G + hg) * nq + (i - q0)];
            const double Dmi = Dm[((int64_t)pi * G + hg) * nq + (i - q0)];
            double *out = dQ + (((int64_t)pi * G + hg) * nq + (i - q0)) * d;
            double *mout = mag_dQ ? mag_dQ + (((int64_t)pi * G + hg) * nq + (i - q0)) * d : NULL;
            double *sout = want_slack ? slack_dQ + (((int64_t)pi * G + hg) * nq + (i - q0)) * d : NULL;
            double *m8out = mag8_dQ ? mag8_dQ + (((int64_t)pi * G + hg) * nq + (i - q0)) * d : NULL;
            for (int dd = 0; dd < d; ++dd) {
                out[dd] = 0.0;
                if (mout) mout[dd] = 0.0;
                if (sout) sout[dd] = 0.0;
                if (m8out) m8out[dd] = 0.0;
            }
            for (int j = k0; j < k1; ++j) {
                if (p->causal && j > i) break;
                double P = exp(score(p, Q, K, b, h, g, i, j) - lse);
                double dP = 0.0, dPm = 0.0;
                for (int dd = 0; dd < d; ++dd) {
                    const double t = ld(dO, idx4(p, p->Hq, b, i, h, dd)) * ld(V, idx4(p, p->Hkv, b, j, g, dd));
                    dP += t;
                    dPm += fabs(t);
                }
                dP *= p->do_inv * p->v_inv;
                dPm *= p->do_inv * p->v_inv;
                double dS = P * (dP - Di);
                const double m_ds = P * (fabs(dP) + fabs(Di));   /* size of dS before the subtraction cancels */
                if (fabs(dS) > amax) amax = fabs(dS);
                double u = dS, step = 0.0;
                if (p->quant) {
                    volatile float prod = (float)dS * (float)p->ds_scale;
                    u = oracle_fp8_decode(oracle_fp8_encode(prod, ORACLE_E5M2), ORACLE_E5M2) / p->ds_scale;
                }
                if (want_slack) {
                    /* uncertainty of dS: P * eps * (terms of dP and D) + |dS| * (relative uncertainty of P) */
                    const double band = p->flip_eps * (P * (dPm + Dmi) +
                                                       fabs(dS) * (1.0 + score_mag(p, Q, K, b, h, g, i, j)));
                    step = flip_step(dS * p->ds_scale, band * p->ds_scale, ORACLE_E5M2) / p->ds_scale;
                }
                for (int dd = 0; dd < d; ++dd) {
                    double kv = ld(K, idx4(p, p->Hkv, b, j, g, dd));
                    out[dd] += p->s * p->k_inv * u * kv;
                    if (mout) mout[dd] += p->s * p->k_inv * m_ds * fabs(kv);
                    if (sout) sout[dd] += p->s * p->k_inv * step * fabs(kv);
                    if (m8out) m8out[dd] += p->s * p->k_inv * fabs(u) * fabs(kv);
                }
            }
        }

    /* column-local pass: dK_j, dV_j (sum over the group's query heads and the query rows) */
#pragma omp parallel for collapse(2) schedule(dynamic, 8)
    for (int pi = 0; pi < nbg; ++pi)
        for (int j = k0; j < k1; ++j) {
            const int b = bg[2 * pi], g = bg[2 * pi + 1];
            double *oK = dK + ((int64_t)pi * nk + (j - k0)) * d;
            double *oV = dV + ((int64_t)pi * nk + (j - k0)) * d;
            double *mK = mag_dK ? mag_dK + ((int64_t)pi * nk + (j - k0)) * d : NULL;
            double *mV = mag_dV ? mag_dV + ((int64_t)pi * nk + (j - k0)) * d : NULL;
            double *sK = want_slack ? slack_dK + ((int64_t)pi * nk + (j - k0)) * d : NULL;
            double *sV = want_slack ? slack_dV + ((int64_t)pi * nk + (j - k0)) * d : NULL;
            double *m8K = mag8_dK ? mag8_dK + ((int64_t)pi * nk + (j - k0)) * d : NULL;
            for (int dd = 0; dd < d; ++dd) {
                oK[dd] = 0.0; oV[dd] = 0.0;
                if (m8K) m8K[dd] = 0.0;
                if (mK) mK[dd] = 0.0;
                if (mV) mV[dd] = 0.0;
                if (sK) { sK[dd] = 0.0; sV[dd] = 0.0; }
            }
            for (int hg = 0; hg < G; ++hg) {
                const int h = g * G + hg;
                for (int i = q0; i < q1; ++i) {
                    if (p->causal && j > i) continue;
                    const double lse = LSE[((int64_t)b * p->Hq + h) * p->N + i];
                    const double Di = D[((int64_t)pi * G + hg) * nq + (i - q0)];
                    const double Dmi = Dm[((int64_t)pi * G + hg) * nq + (i - q0)];
                    double P = exp(score(p, Q, K, b, h, g, i, j) - lse);
                    double w = quant_p(p, P) / cP;
                    double dP = 0.0, dPm = 0.0;
                    for (int dd = 0; dd < d; ++dd) {
                        const double t = ld(dO, idx4(p, p->Hq, b, i, h, dd)) * ld(V, idx4(p, p->Hkv, b, j, g, dd));
                        dP += t;
                        dPm += fabs(t);
                    }
                    dP *= p->do_inv * p->v_inv;
                    dPm *= p->do_inv * p->v_inv;
                    double dS = P * (dP - Di);
                    const double m_ds = P * (fabs(dP) + fabs(Di));
                    double u = dS, stepS = 0.0, stepP = 0.0;
                    if (p->quant) {
                        volatile float prod = (float)dS * (float)p->ds_scale;
                        u = oracle_fp8_decode(oracle_fp8_encode(prod, ORACLE_E5M2), ORACLE_E5M2) / p->ds_scale;
                    }
                    if (want_slack) {
                        const double xm = 1.0 + score_mag(p, Q, K, b, h, g, i, j);
                        const double band = p->flip_eps * (P * (dPm + Dmi) + fabs(dS) * xm);
                        stepS = flip_step(dS * p->ds_scale, band * p->ds_scale, ORACLE_E5M2) / p->ds_scale;
                        stepP = flip_step(P * p->c_P, P * p->c_P * p->flip_eps * xm, ORACLE_E4M3) / p->c_P;
                    }
                    for (int dd = 0; dd < d; ++dd) {
                        double dov = ld(dO, idx4(p, p->Hq, b, i, h, dd));
                        double qv = ld(Q, idx4(p, p->Hq, b, i, h, dd));
                        oV[dd] += p->do_inv * w * dov;
                        oK[dd] += p->s * p->q_inv * u * qv;
                        if (mV) mV[dd] += p->do_inv * w * fabs(dov);
                        if (mK) mK[dd] += p->s * p->q_inv * m_ds * fabs(qv);
                        if (m8K) m8K[dd] += p->s * p->q_inv * fabs(u) * fabs(qv);
                        if (sK) {
                            sK[dd] += p->s * p->q_inv * stepS * fabs(qv);
                            sV[dd] += p->do_inv * stepP * fabs(dov);
                        }
                    }
                }
            }
        }
    free(D);
    free(Dm);
    if (amax_dS) *amax_dS = amax;
}

void oracle_attention_bwd(const uint8_t *Q8, const uint8_t *K8, const uint8_t *V8, const uint8_t *dO8,
                          const double *O, const double *LSE, const oracle_attn_params *p,
                          const int32_t *bg, int nbg, int q0, int q1, int k0, int k1,
                          double *dQ, double *dK, double *dV,
                          double *mag_dQ, double *mag_dK, double *mag_dV, double *amax_dS,
                          double *slack_dQ, double *slack_dK, double *slack_dV)
{
    operand Q, K, V, dO;
    operand_init(&Q, Q8, NULL, ORACLE_E4M3);
    operand_init(&K, K8, NULL, ORACLE_E4M3);
    operand_init(&V, V8, NULL, ORACLE_E4M3);
    operand_init(&dO, dO8, NULL, ORACLE_E5M2);
    attention_bwd_core(&Q, &K, &V, &dO, O, LSE, p, bg, nbg, q0, q1, k0, k1,
                       dQ, dK, dV, mag_dQ, mag_dK, mag_dV, amax_dS, slack_dQ, slack_dK, slack_dV, NULL, NULL);
}

void oracle_attention_bwd_real(const double *Qd, const double *Kd, const double *Vd, const double *dOd,
                               const double *O, const double *LSE, const oracle_attn_params *p,
                               const int32_t *bg, int nbg, int q0, int q1, int k0, int k1,
                               double *dQ, double *dK, double *dV,
                               double *mag_dQ, double *mag_dK, double *mag_dV, double *amax_dS,
                               double *slack_dQ, double *slack_dK, double *slack_dV)
{
    operand Q, K, V, dO;
    operand_init(&Q, NULL, Qd, ORACLE_E4M3);
    operand_init(&K, NULL, Kd, ORACLE_E4M3);
    operand_init(&V, NULL, Vd, ORACLE_E4M3);
    operand_init(&dO, NULL, dOd, ORACLE_E5M2);
    attention_bwd_core(&Q, &K, &V, &dO, O, LSE, p, bg, nbg, q0, q1, k0, k1,
                       dQ, dK, dV, mag_dQ, mag_dK, mag_dV, amax_dS, slack_dQ, slack_dK, slack_dV, NULL, NULL);
}

/* oracle_attention_bwd plus two more error-metric denominators: the sums of |dS8|/ds_scale * |K| (for dQ) and
 * |dS8|/ds_scale * |Q| (for dK), i.e. the magnitude of the product as the FP8 GEMM sees it, after dP - D has
 * cancelled.  Smaller than mag_dQ / mag_dK wherever the softmax row is nearly one-hot. */
void oracle_attention_bwd_mag8(const uint8_t *Q8, const uint8_t *K8, const uint8_t *V8, const uint8_t *dO8,
                               const double *O, const double *LSE, const oracle_attn_params *p,
                               const int32_t *bg, int nbg, int q0, int q1, int k0, int k1,
                               double *dQ, double *dK, double *dV,
                               double *mag_dQ, double *mag_dK, double *mag_dV, double *amax_dS,
                               double *slack_dQ, double *slack_dK, double *slack_dV,
                               double *mag8_dQ, double *mag8_dK)
{
    operand Q, K, V, dO;
    operand_init(&Q, Q8, NULL, ORACLE_E4M3);
    operand_init(&K, K8, NULL, ORACLE_E4M3);
    operand_init(&V, V8, NULL, ORACLE_E4M3);
    operand_init(&dO, dO8, NULL, ORACLE_E5M2);
    attention_bwd_core(&Q, &K, &V, &dO, O, LSE, p, bg, nbg, q0, q1, k0, k1,
                       dQ, dK, dV, mag_dQ, mag_dK, mag_dV, amax_dS, slack_dQ, slack_dK, slack_dV, mag8_dQ, mag8_dK);
}

/* The tie-band rule on its own, so that tests can pin it on hand-worked values. */
double oracle_flip_step(double y, double band, int fmt) { return flip_step(y, band, fmt); }

int oracle_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------------------------------
 * Fine-grained ("blockwise") scaling, the recipe the paper measures against (Section 2: several scaling factors per
 * tensor, different blocks with different factors; Appendix E, "Fine-grained scaling recipes"): a [R,C] tensor is cut
 * into blocks of br x bc elements (1 x 128 for activations, 128 x 128 for weights in the recipe measured there) and
 * every block is quantised like a tensor of its own: rho_b = FP8Max / amax(block), codes = FP8cast(rho_b * x).
 * scale_inv[rb * ncb + cb] = 1 / rho_b with ncb = ceil(C / bc).  Edge blocks are short.
 * ---------------------------------------------------------------------------------------------- */
void oracle_quantize_blockwise(const uint16_t *x, size_t R, size_t C, size_t br, size_t bc, int fmt, uint8_t *codes,
                               float *scale_inv)
{
    size_t nrb = (R + br - 1) / br, ncb = (C + bc - 1) / bc;
#pragma omp parallel for schedule(static)
    for (long b = 0; b < (long)(nrb * ncb); ++b) {
        size_t rb = (size_t)b / ncb, cb = (size_t)b % ncb;
        size_t r1 = (rb + 1) * br < R ? (rb + 1) * br : R, c1 = (cb + 1) * bc < C ? (cb + 1) * bc : C;
        float amax = 0.0f;
        for (size_t r = rb * br; r < r1; ++r)
            for (size_t c = cb * bc; c < c1; ++c) {
                float v = fabsf(bf16_bits_to_float(x[r * C + c]));
                if (v > amax) amax = v;            /* NaN never compares greater: same reading as oracle_amax_bf16 */
            }
        float s, si;
        oracle_scale(amax, fmt, 0, &s, &si);
        scale_inv[b] = si;
        for (size_t r = rb * br; r < r1; ++r)
            for (size_t c = cb * bc; c < c1; ++c) {
                volatile float p = bf16_bits_to_float(x[r * C + c]) * s;
                codes[r * C + c] = oracle_fp8_encode(p, fmt);
            }
    }
}

/* Y[t,n] = sum over K-blocks kb of sx_inv[t,kb] * sw_inv[n/bn,kb] * sum_{k in kb} dec(X8[t,k]) dec(W8[n,k]):
 * every K-block of 128 is an FP8 product of its own, descaled by its two factors and added in high precision
 * (the "promotion" that makes this recipe slower).  sx_inv: [T, K/bk]; sw_inv: [ceil(N/bn), K/bk].
 * mag is the same sum over absolute values. */
void oracle_linear_fwd_blockwise(const uint8_t *X8, const uint8_t *W8, const float *sx_inv, const float *sw_inv,
                                 int64_t T, int64_t N, int64_t K, int64_t bk, int64_t bn,
                                 const int64_t *rows, int64_t nrows, const int64_t *cols, int64_t ncols,
                                 double *ref, double *mag)
{
    double tab[256];
    oracle_fp8_decode_table(ORACLE_E4M3, tab);
    int64_t nkb = (K + bk - 1) / bk;
    (void)T; (void)N;
#pragma omp parallel for schedule(static)
    for (long i = 0; i < (long)nrows; ++i)
        for (int64_t j = 0; j < ncols; ++j) {
            int64_t t = rows[i], n = cols[j];
            double acc = 0.0, am = 0.0;
            for (int64_t kb = 0; kb < nkb; ++kb) {
                double part = 0.0, pm = 0.0;
                int64_t k1 = (kb + 1) * bk < K ? (kb + 1) * bk : K;
                for (int64_t k = kb * bk; k < k1; ++k) {
                    double a = tab[X8[t * K + k]], b = tab[W8[n * K + k]];
                    part += a * b;
                    pm += fabs(a * b);
                }
                double sc = (double)sx_inv[t * nkb + kb] * (double)sw_inv[(n / bn) * nkb + kb];
                acc += sc * part;
                am += sc * pm;
            }
            ref[i * ncols + j] = acc;
            mag[i * ncols + j] = am;
        }
}

/* Data gradient of the same recipe (Appendix E measures the recipe over whole training steps, forward and backward):
 * dX[t,k] = sum over N-blocks nb of sdy_inv[t,nb] * sw_inv[nb, k/bk] * sum_{n in nb} dec(dY8[t,n]) dec(W8[n,k]).
 * dY8: [T,N] E5M2 codes quantised in 1 x bn blocks, sdy_inv [T, N/bn]; W8: [N,K] E4M3 in bn x bk blocks, sw_inv
 * [N/bn, K/bk] (the forward's own weight blocks, now cut along the reduction index). */
void oracle_linear_dgrad_blockwise(const uint8_t *dY8, const uint8_t *W8, const float *sdy_inv, const float *sw_inv,
                                   int64_t T, int64_t N, int64_t K, int64_t bn, int64_t bk,
                                   const int64_t *rows, int64_t nrows, const int64_t *cols, int64_t ncols,
                                   double *ref, double *mag)
{
    double t5[256], t4[256];
    oracle_fp8_decode_table(ORACLE_E5M2, t5);
    oracle_fp8_decode_table(ORACLE_E4M3, t4);
    int64_t nnb = (N + bn - 1) / bn, nkb = (K + bk - 1) / bk;
    (void)T;
#pragma omp parallel for schedule(static)
    for (long i = 0; i < (long)nrows; ++i)
        for (int64_t j = 0; j < ncols; ++j) {
            int64_t t = rows[i], k = cols[j];
            double acc = 0.0, am = 0.0;
            for (int64_t nb = 0; nb < nnb; ++nb) {
                double part = 0.0, pm = 0.0;
                int64_t n1 = (nb + 1) * bn < N ? (nb + 1) * bn : N;
                for (int64_t n = nb * bn; n < n1; ++n) {
                    double a = t5[dY8[t * N + n]], b = t4[W8[n * K + k]];
                    part += a * b;
                    pm += fabs(a * b);
                }
                double sc = (double)sdy_inv[t * nnb + nb] * (double)sw_inv[nb * nkb + k / bk];
                acc += sc * part;
                am += sc * pm;
            }
            ref[i * ncols + j] = acc;
            mag[i * ncols + j] = am;
        }
}

/* Weight gradient: the reduction runs over tokens, so both operands are quantised in bt x 1 blocks (bt consecutive
 * tokens of one channel): dW[n,k] = sum over token blocks tb of sdy_inv_t[tb,n] * sx_inv_t[tb,k] *
 * sum_{t in tb} dec(dY8[t,n]) dec(X8[t,k]).  sdy_inv_t: [ceil(T/bt), N]; sx_inv_t: [ceil(T/bt), K]. */
void oracle_linear_wgrad_blockwise(const uint8_t *dY8, const uint8_t *X8, const float *sdy_inv_t, const float *sx_inv_t,
                                   int64_t T, int64_t N, int64_t K, int64_t bt,
                                   const int64_t *rows, int64_t nrows, const int64_t *cols, int64_t ncols,
                                   double *ref, double *mag)
{
    double t5[256], t4[256];
    oracle_fp8_decode_table(ORACLE_E5M2, t5);
    oracle_fp8_decode_table(ORACLE_E4M3, t4);
    int64_t ntb = (T + bt - 1) / bt;
#pragma omp parallel for schedule(static)
    for (long i = 0; i < (long)nrows; ++i)
        for (int64_t j = 0; j < ncols; ++j) {
            int64_t n = rows[i], k = cols[j];
            double acc = 0.0, am = 0.0;
            for (int64_t tb = 0; tb < ntb; ++tb) {
                double part = 0.0, pm = 0.0;
                int64_t t1 = (tb + 1) * bt < T ? (tb + 1) * bt : T;
                for (int64_t t = tb * bt; t < t1; ++t) {
                    double a = t5[dY8[t * N + n]], b = t4[X8[t * K + k]];
                    part += a * b;
                    pm += fabs(a * b);
                }
                double sc = (double)sdy_inv_t[tb * N + n] * (double)sx_inv_t[tb * K + k];
                acc += sc * part;
                am += sc * pm;
            }
            ref[i * ncols + j] = acc;
            mag[i * ncols + j] = am;
        }
}
