/*
 * fp8dpa — C ABI of the FP8 transformer-block hot path on one B200 (sm_100a).
 *
 * Every GEMM of the block runs on FP8 operands (forward and backward), fed by per-tensor scaling:
 *   amax -> scale -> saturating cast (BF16 -> E4M3 for activations/weights, E5M2 for gradients),
 *   linear forward / dgrad / wgrad, and attention forward / backward with QK^T and PV in FP8.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer owned by the caller unless it says "host".  The library
 *     allocates no device memory; scratch comes from the caller (`ws`, sized by the *_workspace_bytes
 *     functions, 256-byte aligned).
 *   - Tensor pointers must be 16-byte aligned and row pitches multiples of 16 bytes (128-bit access and
 *     TMA).  Violations return FP8_ERR_ALIGN / FP8_ERR_SHAPE before anything is launched.
 *   - `stream` is a cudaStream_t passed as void*; every call only enqueues work on it and returns.
 *     Scales and amax values are device scalars so that amax -> scale -> cast -> GEMM never syncs the host.
 *   - Return value: FP8_OK or a negative fp8_status.  fp8_last_error() gives a host string for the last
 *     failure on the calling thread.  Kernels never spin without bound: a wait that runs out records
 *     FP8_ERR_TIMEOUT in a device status word, read (and cleared) by fp8_device_status().
 *   - BF16 tensors are raw 16-bit words; FP8 tensors are raw bytes (codes).
 *   - There is no CPU fallback: on a device that is not compute capability 10.x every call returns
 *     FP8_ERR_ARCH.
 */
#ifndef FP8DPA_H
#define FP8DPA_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define FP8_API __attribute__((visibility("default")))
#else
#define FP8_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { FP8_E4M3 = 0, FP8_E5M2 = 1 } fp8_fmt;

typedef enum {
    FP8_OK = 0,
    FP8_ERR_NULL = -1,       /* a required pointer is NULL */
    FP8_ERR_ALIGN = -2,      /* pointer not 16-byte aligned */
    FP8_ERR_SHAPE = -3,      /* size zero, pitch not a multiple of 16 bytes, unsupported head_dim, Hq % Hkv != 0 */
    FP8_ERR_ENUM = -4,       /* bad fp8_fmt */
    FP8_ERR_WORKSPACE = -5,  /* ws NULL / too small / misaligned */
    FP8_ERR_CUDA = -6,       /* CUDA runtime or driver error; see fp8_last_error() */
    FP8_ERR_TIMEOUT = -7,    /* a bounded device-side wait expired (reported by fp8_device_status) */
    FP8_ERR_ARCH = -8        /* current device is not sm_100 */
} fp8_status;

/* Host string describing the last non-OK return on this thread (never NULL). */
FP8_API const char *fp8_last_error(void);

/* Synchronises `stream`, copies the device status word of the current device to *status_out (host; FP8_OK
 * or FP8_ERR_TIMEOUT) and clears it. */
FP8_API int fp8_device_status(int *status_out, void *stream);

/* Self-test of the bounded-wait path: one warp waits on a barrier that nothing ever completes, with a limit of
 * `limit_cycles` SM clocks (0 < limit_cycles <= 2^31).  At the limit it gives up the way every kernel of the library
 * does when a wait runs out: FP8_ERR_TIMEOUT goes into the device status word, *gave_up (device int) is set to 1 and
 * the kernel returns; the context stays usable.  Enqueues on `stream` and returns FP8_OK. */
FP8_API int fp8_selftest_wait_timeout(long long limit_cycles, int *gave_up, void *stream);

/* ---- per-tensor scaling ---------------------------------------------------------------------------
 * Appendix C (definition above Theorem 1): s(x) = MaxFP8Value / absmax(x); Appendix E: rho(X) =
 * FP8MaxValue / (2^m max H) and FP8cast(rho(X) X).  MaxFP8Value is 448 (E4M3) / 57344 (E5M2). */

/* *amax = max_i |x_i| over n BF16 values (overwritten; exact). */
FP8_API int fp8_amax(const void *x_bf16, size_t n, float *amax, void *stream);

/* *scale = FP8Max(fmt) / (2^margin * *amax) in binary32 (one IEEE division), *scale_inv = 1 / *scale.
 * amax == 0 or non-finite gives scale 1; an overflowing quotient gives FLT_MAX. */
FP8_API int fp8_scale(const float *amax, int fmt, int margin, float *scale, float *scale_inv, void *stream);

/* out[r,c] = sat_rne_fmt( float(x[r,c]) * *scale ): binary32 product, one round-to-nearest-even to FP8,
 * saturating at +-FP8Max (no Inf/NaN from finite input).  x is [rows, cols] row-major BF16.
 * out_t (nullable) receives the same codes as [cols, rows]; it needs rows % 16 == 0.
 * amax_out (nullable) is overwritten with amax(x) in the same pass (for delayed scaling).
 * cols % 16 == 0 unless rows == 1 (a flat tensor may have any length). */
FP8_API int fp8_cast(const void *x_bf16, size_t rows, size_t cols, const float *scale, int fmt,
             uint8_t *out, uint8_t *out_t, float *amax_out, void *stream);

/* Just-in-time scaling of one tensor: fp8_amax, fp8_scale (margin 0) and fp8_cast chained on `stream`
 * (two passes over x, as Section 2 notes for JIT scaling).  amax, scale, scale_inv are outputs. */
FP8_API int fp8_quantize(const void *x_bf16, size_t rows, size_t cols, int fmt, uint8_t *out, uint8_t *out_t,
                 float *amax, float *scale, float *scale_inv, void *stream);

/* fp8_quantize of up to 8 flat tensors (the operands of one layer) in two launches instead of two per tensor: one
 * reduction over all of them, one cast of all of them (the just-in-time recipe of Section 2, unchanged arithmetic: every
 * tensor has its own amax, scale and codes, bit-identical to fp8_quantize).  `items` is a HOST array; item i casts the
 * n BF16 values at x_bf16 to out (no transposed copy).  scalars: device array of 3 * n_items floats, overwritten with
 * (amax, scale, 1 / scale) of item i at scalars[3 i .. 3 i + 2]. */
typedef struct {
    const void *x_bf16;   /* device, 16-byte aligned */
    size_t n;             /* number of BF16 values, > 0 */
    int fmt;              /* FP8_E4M3 / FP8_E5M2 */
    uint8_t *out;         /* device, 16-byte aligned, n bytes */
} fp8_quant_item;
FP8_API int fp8_quantize_multi(const fp8_quant_item *items, int n_items, float *scalars, void *stream);

/* Delayed scaling (Appendix E): H holds the last `len` abs-max values of one tensor (the paper trains with
 * len = 1024, margin 0); rho = FP8Max / (2^margin * max H); after a step, H <- {amax} u H minus its oldest
 * entry, and the updated history serves the following step.  This call does that update on the device: history[*head] = *amax_new,
 * *head = (*head + 1) % len, then *scale / *scale_inv from the maximum of the updated history (guards as in
 * fp8_scale; an all-zero history gives 1).  history: `len` floats, zero-initialised by the caller; head: device
 * int, initially 0, the position of the oldest entry.  A training step then needs a single pass per tensor:
 * fp8_cast(x, scale, ..., amax_out = amax_new) followed by fp8_scale_update for the next step. */
FP8_API int fp8_scale_update(float *history, int len, int *head, const float *amax_new, int fmt, int margin,
                     float *scale, float *scale_inv, void *stream);

/* The whole delayed-scaling quantize (Appendix E) of up to 8 flat tensors in ONE launch.  Item i: *scale_next, as the
 * call finds it, is this step's scale (what the previous call left there from the history; before the first call the
 * caller sets it, e.g. to 1 or from fp8_amax + fp8_scale_update).  The n BF16 values are cast to out under it, the same
 * pass takes amax(x), *scale and *scale_inv receive this step's scale and its reciprocal (what the products of this
 * step read), and the last block to finish the tensor does its fp8_scale_update: history[*head] = amax, *head advances,
 * *scale_next = the scale of the next step from the maximum of the updated history; *amax = amax(x).  No pointer
 * changes between steps, so a step built on this call can be captured in a CUDA graph.  Codes, amax, history, head
 * and scales are bit-identical to fp8_cast(..., amax_out) followed by fp8_scale_update.  `items` is a HOST array;
 * every pointer inside it is a device pointer; scale and scale_inv must not alias scale_next.  sync: device array of
 * 2 * n_items 32-bit words, zero before the first call and left zero by every call (amax bits and a block counter
 * per tensor); calls that share `sync` must be ordered on one stream. */
typedef struct {
    const void *x_bf16;      /* device, 16-byte aligned */
    size_t n;                /* number of BF16 values, > 0 */
    int fmt;                 /* FP8_E4M3 / FP8_E5M2 */
    uint8_t *out;            /* device, 16-byte aligned, n bytes */
    float *history;          /* device ring of history_len floats (zero-initialised by the caller) */
    int *head;               /* device int, initially 0 */
    float *scale_next;       /* device, read then overwritten: this step's scale in, the next step's out */
    float *amax;             /* device, overwritten */
    float *scale;            /* device, overwritten: this step's scale */
    float *scale_inv;        /* device, overwritten: its reciprocal */
} fp8_delayed_item;
FP8_API int fp8_quantize_delayed_multi(const fp8_delayed_item *items, int n_items, int history_len, int margin,
                               uint32_t *sync, void *stream);

/* Gated activation fused with the cast (Appendix B: FFN with activation phi; SwiGLU in the Llama-style
 * workloads).  gate_up is the [T, 2F] BF16 output of the fused first FFN projection, gate = columns [0,F),
 * up = columns [F,2F).  h = silu(gate) * up is formed in FP32, rounded to BF16 (never written to memory), and
 * then treated exactly like the input of fp8_cast: out[t,f] = sat_rne_fmt(float(h) * *scale), out_t the same
 * codes as [F,T] (nullable), *amax_out = amax(h) (nullable).  out and out_t may both be NULL when only the amax
 * is wanted (first pass of just-in-time scaling).  F % 16 == 0, T % 16 == 0 when out_t is given.
 * The sigmoid uses the hardware exp2 / reciprocal approximations (relative error near 2^-22), so a code can
 * differ from a double-precision evaluation where h lies that close to a BF16 rounding boundary. */
FP8_API int fp8_swiglu_cast(const void *gate_up_bf16, size_t T, size_t F, const float *scale, int fmt,
                    uint8_t *out, uint8_t *out_t, float *amax_out, void *stream);

/* The un-gated FFN activations of the other architecture families (Appendix B, architecture table), fused with
 * the cast in the same way: x is the [T,F] BF16 output of the first FFN projection, h = act(x) rounded to BF16,
 * then out / out_t / amax_out as in fp8_swiglu_cast.
 *   FP8_ACT_GELU   h = 0.5 x (1 + erf(x / sqrt 2))                                   (exact form)
 *   FP8_ACT_XIELU  h = a_p x^2 + 0.5 x (x > 0);  a_n (e^x - 1) - a_n x + 0.5 x (x <= 0)   (Appendix B, Eq. (xIELU))
 * act_params: device pointer to {a_p, a_n} (the per-layer trainable scalars) for xIELU, ignored for GeLU. */
enum { FP8_ACT_GELU = 1, FP8_ACT_XIELU = 2 };
FP8_API int fp8_act_cast(const void *x_bf16, size_t T, size_t F, int act, const float *act_params, const float *scale,
                 int fmt, uint8_t *out, uint8_t *out_t, float *amax_out, void *stream);

/* Post-normalisation and residual connection of the block (Section 3; Appendix B: X^ = X + (N_post o GQA)(X),
 * block(X) = X^ + (N_post o FFN)(X^)), fused with the amax of the result, which is the operand of the next FP8
 * GEMM since these architectures have no pre-normalisation:
 *   FP8_NORM_RMS         out = x + gamma (.) y / sqrt(mean(y^2) + eps)      (eps = 0 is the paper's N_gamma)
 *   FP8_NORM_LAYERSCALE  out = x + gamma (.) y
 * x, y, out: [T,D] BF16 device tensors (out may alias x); gamma: D binary32 on the device; *amax_out (nullable) is
 * overwritten with amax(out).  D % 8 == 0, D <= 16384. */
enum { FP8_NORM_RMS = 0, FP8_NORM_LAYERSCALE = 1 };
FP8_API int fp8_postnorm_residual(const void *x_bf16, const void *y_bf16, const float *gamma, size_t T, size_t D,
                          int mode, float eps, void *out_bf16, float *amax_out, void *stream);

/* Producer form under delayed scaling (Appendix E: rho from the amax history; Section 3 / Appendix B: without a
 * pre-normalisation the post-norm output IS the operand of the next FP8 GEMM): the same result, and in the same
 * pass its FP8 codes out8[T,D] = FP8cast(*scale * out) of the BF16-rounded values (bit-identical to fp8_cast of
 * out_bf16) and *amax_out = amax(out) for fp8_scale_update.  x_scale multiplies the residual input x before the
 * sum: 1 inside the network; sigma_0^-1 for the first block, whose input is scaled by the inverse of the
 * initialisation standard deviation (Section 3; Appendix B, architecture table, column "input scaling").
 * out_bf16 is required (it is the residual stream), out8 and scale are required, amax_out may be NULL. */
FP8_API int fp8_postnorm_residual_q(const void *x_bf16, const void *y_bf16, const float *gamma, size_t T, size_t D,
                            int mode, float eps, float x_scale, const float *scale, int fmt, void *out_bf16,
                            uint8_t *out8, float *amax_out, void *stream);

/* QK entropy regulariser and rotary embedding of per-head query / key vectors (Section 3; Appendix B:
 * attnhead = selfattn(N_QK(X W_Q), N_QK(X W_K), X W_V) with rotary position embeddings), fused with the amax that
 * the FP8 cast of Q / K needs.  x, out: [T,H,d] BF16 (out may alias x), d in {64, 128}.
 *   FP8_QK_RMS   v / sqrt(mean(v^2) + eps) over the d entries of a head (unit gain: a frozen gain is folded into
 *                the softmax scale, Section 3.1)        FP8_QK_TANH  tanh(alpha v)        FP8_QK_NONE  v
 * then, if cos_table != NULL, the pairs (i, i + d/2) are rotated by the angle of position t mod seq_len:
 * out[i] = v[i] c - v[i+d/2] s, out[i+d/2] = v[i+d/2] c + v[i] s with c, s = cos/sin_table[pos, i]
 * ([seq_len, d/2] binary32 on the device, supplied by the caller).  *amax_out (nullable) = amax(out). */
enum { FP8_QK_RMS = 0, FP8_QK_TANH = 1, FP8_QK_NONE = 2 };
FP8_API int fp8_qk_norm_rope(const void *x_bf16, size_t T, size_t H, size_t d, int mode, float alpha, float eps,
                     const float *cos_table, const float *sin_table, size_t seq_len, void *out_bf16,
                     float *amax_out, void *stream);

/* Producer form under delayed scaling (Appendix E): the regularised, rotated vectors are the Q / K operands of the
 * FP8 attention (Appendix E, table "Comparison between FP8 methods": QK^T runs in FP8), so the same pass also
 * writes their FP8 codes out8[T,H,d] = FP8cast(*scale * out) of the BF16-rounded values (bit-identical to fp8_cast
 * of out_bf16) and *amax_out = amax(out).  out_bf16 may be NULL when only the codes are wanted. */
FP8_API int fp8_qk_norm_rope_q(const void *x_bf16, size_t T, size_t H, size_t d, int mode, float alpha, float eps,
                       const float *cos_table, const float *sin_table, size_t seq_len, const float *scale, int fmt,
                       void *out_bf16, uint8_t *out8, float *amax_out, void *stream);

/* Kurtosis monitor (Section 4): *out = mean over rows of mu[x^4] / mu[x^2]^2 of a [rows, cols] BF16 tensor
 * (un-centred; rows are token vectors).  *out is overwritten.  cols % 8 == 0. */
FP8_API int fp8_kurtosis(const void *x_bf16, size_t rows, size_t cols, float *out, void *stream);

/* The monitor folded into the amax pass of a just-in-time quantisation (Section 4 tracks the kurtosis of tensors
 * that are quantised anyway: FFN-2 input, QKV output, block output; Appendix C: s(x) = MaxFP8Value / absmax(x)):
 * one read of x gives *amax = max |x| (as fp8_amax, bit-exact) and *kurtosis (as fp8_kurtosis).  Both device
 * scalars are overwritten.  cols % 8 == 0. */
FP8_API int fp8_amax_kurtosis(const void *x_bf16, size_t rows, size_t cols, float *amax, float *kurtosis, void *stream);

/* ---- linear layers --------------------------------------------------------------------------------
 * Appendix E: GEMM(X,Y) = 1/(rho_X rho_Y) * FP8GEMM(FP8cast(rho_X X), FP8cast(rho_Y Y)), BF16 result;
 * Table "Comparison between FP8 methods": Linear_W(X) = XW for the FFN, QKV and output projections.
 * Weights are stored [out, in] = [N, K].  Operands are FP8 codes whose reduction index is contiguous;
 * where the stored tensor has the other orientation, pass the transposed copy fp8_cast produced.
 * sA_inv / sB_inv are device scalars (1/scale of each operand).  Accumulation is FP32 on the tensor
 * cores.  Output is BF16 (out_is_fp32 == 0) or FP32, row-major, fully overwritten unless `accumulate`.
 * Reduction lengths and output widths must be multiples of 16.  ws may be NULL (none needed today). */

/* Y[T,N] = sX_inv*sW_inv * X8[T,K] . W8[N,K]^T         (X8, W8: E4M3) */
FP8_API int fp8_linear_fwd(const uint8_t *X8, const uint8_t *W8, const float *sX_inv, const float *sW_inv,
                   void *Y, int out_is_fp32, int T, int N, int K, void *ws, size_t ws_bytes, void *stream);

/* dX[T,K] = sdY_inv*sW_inv * dY8[T,N] . W8t[K,N]^T     (dY8: E5M2; W8t = transposed copy of W8, E4M3) */
FP8_API int fp8_linear_dgrad(const uint8_t *dY8, const uint8_t *W8t, const float *sdY_inv, const float *sW_inv,
                     void *dX, int out_is_fp32, int T, int N, int K, void *ws, size_t ws_bytes, void *stream);

/* dW[N,K] (+)= sdY_inv*sX_inv * dY8t[N,T] . X8t[K,T]^T (dY8t: E5M2 [N,T]; X8t: E4M3 [K,T]) */
FP8_API int fp8_linear_wgrad(const uint8_t *dY8t, const uint8_t *X8t, const float *sdY_inv, const float *sX_inv,
                     void *dW, int out_is_fp32, int accumulate, int T, int N, int K,
                     void *ws, size_t ws_bytes, void *stream);

/* The two gradients with every operand read in place, exactly as the forward product stores it: W8 [N,K],
 * dY8 [T,N], X8 [T,K], row-major.  tcgen05 takes FP8 operands with either the reduction index or the output index
 * contiguous, so no transposed FP8 copy has to be written by the cast (fp8_cast / fp8_quantize with out_t = NULL).
 * Same arithmetic and outputs as fp8_linear_dgrad / fp8_linear_wgrad.  T, N, K multiples of 16. */
FP8_API int fp8_linear_dgrad_rm(const uint8_t *dY8, const uint8_t *W8, const float *sdY_inv, const float *sW_inv,
                        void *dX, int out_is_fp32, int T, int N, int K, void *stream);
FP8_API int fp8_linear_wgrad_rm(const uint8_t *dY8, const uint8_t *X8, const float *sdY_inv, const float *sX_inv,
                        void *dW, int out_is_fp32, int accumulate, int T, int N, int K, void *stream);

/* Grouped forward product for a mixture-of-experts FFN (Appendix D: sparse FFNs, 8 experts of which 2 are
 * active per token): X8 [T,K] holds the routed token copies sorted by expert; expert g owns the rows
 * [group_offsets[g], group_offsets[g+1]) (device int32 array of n_groups + 1 ascending entries, the router's output,
 * group_offsets[0] = 0, group_offsets[n_groups] <= T), the weights W8[g] ([N,K] each, stored back to back) and the
 * descale sW_inv[g].  Y[t, :] = sX_inv * sW_inv[g(t)] * X8[t, :] . W8[g(t)]^T, one launch for all experts; rows
 * past group_offsets[n_groups] are left untouched.  n_groups <= 256. */
FP8_API int fp8_grouped_linear_fwd(const uint8_t *X8, const uint8_t *W8, const float *sX_inv, const float *sW_inv,
                           const int *group_offsets, int n_groups, void *Y, int out_is_fp32, int T, int N, int K,
                           void *stream);

/* Its data gradient: dX[t, :] = sdY_inv * sW_inv[g(t)] * dY8[t, :] . W8[g(t)] with dY8 [T,N] in E5M2 (rows sorted by
 * expert like X8) and the weights read in place ([N,K] per expert, no transposed copies).  N % 128 == 0. */
FP8_API int fp8_grouped_linear_dgrad(const uint8_t *dY8, const uint8_t *W8, const float *sdY_inv, const float *sW_inv,
                             const int *group_offsets, int n_groups, void *dX, int out_is_fp32, int T, int N, int K,
                             void *stream);

/* Its weight gradients: dW[g] (+)= sdY_inv * sX_inv * dY8[rows of g]^T . X8[rows of g], dW [n_groups, N, K] (BF16 or
 * FP32), both operands read in place.  One launch of the weight-gradient product per expert on its slice of rows;
 * ragged and empty groups need no padding (an empty group gives zeros, or leaves dW[g] alone with `accumulate`).
 * Unlike the two calls above the offsets are a HOST array (n_groups + 1 entries): the per-expert launches are set up
 * on the host. */
FP8_API int fp8_grouped_linear_wgrad(const uint8_t *dY8, const uint8_t *X8, const float *sdY_inv, const float *sX_inv,
                             const int *group_offsets_host, int n_groups, void *dW, int out_is_fp32, int accumulate,
                             int T, int N, int K, void *stream);

/* The same weight gradients in one launch with the offsets on the DEVICE (group_offsets as in fp8_grouped_linear_fwd:
 * n_groups + 1 ascending int32 entries, clamped to [0, T] by the kernel), so that the router's output never has to reach
 * the host.  ws: device scratch of fp8_grouped_linear_wgrad_workspace_bytes(n_groups, N) = n_groups * 128 * N bytes,
 * 16-byte aligned, overwritten (it receives a zero-padded copy of the last, possibly ragged block of 128 rows of dY8 of
 * every expert; all other blocks are read in place).  Same arithmetic, outputs, `accumulate` and empty-group behaviour as
 * fp8_grouped_linear_wgrad (an empty group gives zeros, or leaves dW[g] unchanged in value with `accumulate`).
 * Errors: FP8_ERR_NULL, FP8_ERR_SHAPE, FP8_ERR_ALIGN, FP8_ERR_WORKSPACE before anything is launched. */
FP8_API size_t fp8_grouped_linear_wgrad_workspace_bytes(int n_groups, int N);
FP8_API int fp8_grouped_linear_wgrad_dev(const uint8_t *dY8, const uint8_t *X8, const float *sdY_inv, const float *sX_inv,
                                 const int *group_offsets, int n_groups, void *dW, int out_is_fp32, int accumulate,
                                 int T, int N, int K, void *ws, size_t ws_bytes, void *stream);

/* Producer forms for delayed scaling (Appendix E: rho comes from the amax history, so the producer of a tensor can
 * emit FP8 in its own epilogue, "a single pass on the data", Section 2).  Same products as fp8_linear_fwd /
 * fp8_linear_dgrad; the result is rounded to BF16 (the tensor an unfused chain would store), its amax is written to
 * *y_amax (nullable; overwritten; feed it to fp8_scale_update for the next step), and the codes
 * sat_rne_fmt(float(bf16 result) * *y_scale) go to Y8 [T,N] (dX8 [T,K]).  The codes and the amax are bit-identical
 * to fp8_linear_fwd (BF16 output) followed by fp8_cast with the same scale. */
FP8_API int fp8_linear_fwd_q(const uint8_t *X8, const uint8_t *W8, const float *sX_inv, const float *sW_inv,
                     const float *y_scale, int y_fmt, uint8_t *Y8, float *y_amax, int T, int N, int K,
                     void *stream);
FP8_API int fp8_linear_dgrad_q(const uint8_t *dY8, const uint8_t *W8t, const float *sdY_inv, const float *sW_inv,
                       const float *dx_scale, int dx_fmt, uint8_t *dX8, float *dx_amax, int T, int N, int K,
                       void *stream);

/* ---- fine-grained ("blockwise") scaling: the comparison recipe -------------------------------------
 * Section 2 (several scaling factors per tensor, one per block) and Appendix E ("Fine-grained scaling recipes",
 * throughput table): activations are quantised in 1 x 128 blocks, weights in 128 x 128 blocks, every block
 * just-in-time with its own rho_b = FP8Max / amax(block); the product then sums, over K-blocks of 128, FP8 partial
 * products that each carry their own descale.  Kept beside the tensor-wise path to measure what the finer recipe
 * costs on this hardware.
 *
 * fp8_quantize_blockwise: x [rows, cols] BF16 -> out [rows, cols] codes, one pass.  block_rows = 1: 1 x 128 blocks,
 * scale_inv laid out K-block-major, [cols/128][rows] (the order the product reads it in).  block_rows = 128:
 * 128 x 128 blocks, scale_inv [ceil(rows/128)][cols/128].  cols % 128 == 0.  Inputs are finite.
 * block_rows = FP8_BLOCK_128x1: blocks of 128 consecutive rows of one column (what the weight-gradient product needs,
 * whose reduction runs over the token rows), scale_inv [ceil(rows/128)][cols].
 * fp8_linear_fwd_blockwise: Y[t,n] = sum_kb sx_inv[kb][t] * sw_inv[n/128][kb] * sum_{k in kb} X8[t,k] W8[n,k], BF16
 * result; X8 [T,K], W8 [N,K] in E4M3; K % 128 == 0, N % 16 == 0.
 * fp8_linear_dgrad_blockwise: dX[t,k] = sum_nb sdy_inv[nb][t] * sw_inv[nb][k/128] * sum_{n in nb} dY8[t,n] W8[n,k];
 * dY8 [T,N] E5M2 quantised in 1 x 128 blocks (scales [N/128][T]), W8 [N,K] and its 128 x 128 scales exactly as the
 * forward uses them (read in place, no transposed copy); N % 128 == 0, K % 128 == 0.
 * fp8_linear_wgrad_blockwise: dW[n,k] = sum_tb sdy_inv_t[tb][n] * sx_inv_t[tb][k] * sum_{t in tb} dY8[t,n] X8[t,k];
 * dY8 [T,N] E5M2 and X8 [T,K] E4M3 both quantised in 128 x 1 blocks (FP8_BLOCK_128x1), read in place; BF16 result
 * [N,K]; N % 16 == 0, K % 16 == 0, T arbitrary (the last block of tokens may be short).
 * (Appendix E, throughput table: the recipe's cost is measured over a whole training step, forward and backward.) */
#define FP8_BLOCK_128x1 (-128)
FP8_API int fp8_quantize_blockwise(const void *x_bf16, size_t rows, size_t cols, int block_rows, int fmt,
                           uint8_t *out, float *scale_inv, void *stream);
FP8_API int fp8_linear_fwd_blockwise(const uint8_t *X8, const uint8_t *W8, const float *sx_inv, const float *sw_inv,
                             void *Y_bf16, int T, int N, int K, void *stream);
FP8_API int fp8_linear_dgrad_blockwise(const uint8_t *dY8, const uint8_t *W8, const float *sdy_inv, const float *sw_inv,
                               void *dX_bf16, int T, int N, int K, void *stream);
FP8_API int fp8_linear_wgrad_blockwise(const uint8_t *dY8, const uint8_t *X8, const float *sdy_inv_t,
                               const float *sx_inv_t, void *dW_bf16, int T, int N, int K, void *stream);

/* ---- attention ------------------------------------------------------------------------------------
 * Appendix B, Eq. (P): P = Softmax(s Q K^T + M), output P V, grouped-query heads; Appendix E table: both
 * products in FP8, forward and backward.  Tensors are [B, N, H, d] row-major; query head h reads KV head
 * h / (Hq/Hkv).  M is the causal mask when `causal` != 0.  d is 64 or 128; N % 16 == 0.
 *
 * Forward: scores and softmax in FP32; P~ = exp(x - running max) in (0,1] is re-quantised to E4M3 with
 * scale p_scale (448 = FP8Max / amax(P~)) before the PV product, keys taken in blocks of 128 in ascending
 * order; the row sum uses the un-quantised P~.  With max_slack = tau > 0 the reference maximum of a row is the
 * running maximum as of the last block that exceeded the previous reference by more than 2^tau (P~ in (0, 2^tau]).  O is BF16, LSE[b,h,i] the FP32 log-sum-exp (natural log).
 * Backward: recomputes P = exp(x - LSE); dV = P8^T dO, dP = dO V^T, dS = P o (dP - D) with
 * D = rowsum(dO o O), dS -> E5M2 with *ds_scale, dQ = s dS8 K, dK = s dS8^T Q; dK, dV summed over the
 * query heads of a group; *ds_amax (nullable) is overwritten with max|dS|. */
typedef struct {
    const float *q_inv, *k_inv, *v_inv; /* device scalars: 1/scale of Q8, K8, V8 */
    const float *do_inv;                /* device scalar: 1/scale of dO8 (backward only) */
    float softmax_scale;                /* host value s; 1/sqrt(d) for Llama-style blocks */
    float p_scale;                      /* host value c_P; 448 */
    const float *ds_scale;              /* device scalar: quantisation scale of dS (backward only) */
    float *ds_amax;                     /* device scalar out, nullable (backward only) */
    float max_slack;                    /* host value tau >= 0, in powers of two (forward only): a row keeps its reference
                                         * maximum until a block maximum exceeds it by more than 2^tau, so that
                                         * P~ <= 2^tau and O is rescaled rarely; pass p_scale = 448 / 2^tau (the scaling
                                         * rule of Appendix E with margin m = tau).  0 = exact running maximum */
} fp8_attn_scales;

/* Scratch bytes the attention calls need (op: 0 = forward, 1 = backward). */
FP8_API size_t fp8_attention_workspace_bytes(int op, int B, int N, int Hq, int Hkv, int d);

FP8_API int fp8_attention_fwd(const uint8_t *Q8, const uint8_t *K8, const uint8_t *V8, const fp8_attn_scales *sc,
                      int causal, int B, int N, int Hq, int Hkv, int d,
                      void *O_bf16, float *LSE, void *ws, size_t ws_bytes, void *stream);

/* Producer form of the forward for delayed scaling (Appendix E; "a single pass", Section 2): besides O (BF16, still
 * needed by the backward) and LSE it writes O8[B,N,Hq,d] = sat_rne_e4m3(float(O) * *o_scale), the operand of the
 * output projection, and *o_amax = amax(O) (nullable, overwritten).  Bit-identical to fp8_attention_fwd followed by
 * fp8_cast(O, o_scale, FP8_E4M3, amax_out). */
FP8_API int fp8_attention_fwd_q(const uint8_t *Q8, const uint8_t *K8, const uint8_t *V8, const fp8_attn_scales *sc,
                        int causal, int B, int N, int Hq, int Hkv, int d, void *O_bf16, float *LSE,
                        const float *o_scale, uint8_t *O8, float *o_amax, void *stream);

FP8_API int fp8_attention_bwd(const uint8_t *Q8, const uint8_t *K8, const uint8_t *V8, const uint8_t *dO8,
                      const void *O_bf16, const float *LSE, const fp8_attn_scales *sc,
                      int causal, int B, int N, int Hq, int Hkv, int d,
                      void *dQ_bf16, void *dK_bf16, void *dV_bf16, void *ws, size_t ws_bytes, void *stream);

/* ---- attention backward without caller scratch -------------------------------------------------------
 * (No counterpart in the paper: this is a packaging variant of fp8_attention_bwd, same arithmetic.)
 *
 * For callers that cannot allocate or pass device scratch - e.g. code that runs inside an already
 * committed memory pool, a plugin that only ever receives its input and output buffers, or a launch thread
 * that must not re-enter an allocator.  The scratch fp8_attention_bwd takes as `ws` is replaced by a fixed
 * array of FP8_STATIC_SCRATCH_BYTES inside the library's device image; every GPU that loads the library
 * holds that array until the process exits.  The call allocates nothing (no cudaMalloc / cudaFree, no
 * allocating library routine).
 *
 * Limit: fp8_attention_workspace_bytes(1, B, N, Hq, Hkv, d), about B*N*Hq*(d+1)*4 bytes for d = 64 and
 * B*N*Hq*(d+8)*4 for d = 128, must not exceed
 * FP8_STATIC_SCRATCH_BYTES; larger problems return FP8_ERR_WORKSPACE and launch nothing.
 * The first call on each device looks up the array's device address (with that device current); make that
 * first call before any stream capture begins.
 * All calls share the one array and it keeps the previous call's contents; each call clears what it needs
 * to start from zero.  Two calls that overlap on the GPU (different streams, or different host threads)
 * race on it: serialise them.  Inputs, outputs, scales and status codes are those of fp8_attention_bwd. */
#define FP8_STATIC_SCRATCH_BYTES (32u << 20)

FP8_API int fp8_attention_bwd_static(const uint8_t *Q8, const uint8_t *K8, const uint8_t *V8, const uint8_t *dO8,
                             const void *O_bf16, const float *LSE, const fp8_attn_scales *sc,
                             int causal, int B, int N, int Hq, int Hkv, int d,
                             void *dQ_bf16, void *dK_bf16, void *dV_bf16, void *stream);

/* ---- host-buffer forms ------------------------------------------------------------------------------
 * (No counterpart in the paper: packaging of the calls above for a caller whose tensors live in HOST memory.)
 *
 * fp8_linear_step_host: one linear layer's training step (Appendix E, throughput table) from BF16 HOST tensors
 * X[T,K], W[N,K], dY[T,N] to BF16 HOST tensors Y[T,N], dX[T,K], dW[N,K]: upload, fp8_quantize_multi of X and W
 * (E4M3) and dY (E5M2) with just-in-time scales, fp8_linear_fwd, fp8_linear_dgrad_rm, fp8_linear_wgrad_rm,
 * download.  T, N, K multiples of 16.
 * fp8_attention_step_host: one attention's training step (Appendix B, Eq. (P)) from BF16 HOST tensors
 * Q, dO [B,N,Hq,d] and K, V [B,N,Hkv,d] to HOST O, dQ [B,N,Hq,d] (BF16), LSE [B,Hq,N] (FP32) and
 * dK, dV [B,N,Hkv,d] (BF16): upload, fp8_quantize_multi of Q, K, V (E4M3) and dO (E5M2), fp8_attention_fwd with
 * p_scale = 448 and max_slack = 0, fp8_attention_bwd with the given ds_scale (a host value), download.
 * Results are bit-identical to the same chain of device-pointer calls.
 *
 * Pointers: every h* argument is HOST memory, owned by the caller; pinned (page-locked) memory is needed
 * for the copies to overlap anything, pageable memory is correct but serialises.  `ws` is DEVICE memory,
 * 256-byte aligned, of at least fp8_*_step_host_workspace_bytes(...) bytes (0 = unsupported shape); it
 * holds the uploaded tensors, their FP8 copies, the results and the scratch, and its contents are
 * unspecified afterwards.
 * Ordering: the calls enqueue on three streams owned by the library (uploads, kernels, downloads; one
 * set per device) and return without waiting, so that with two or more workspaces in rotation the
 * copies of one call run under the kernels of another.  A workspace may be reused at once: the library
 * orders the new call after the previous call on the same `ws` address.  Inputs must stay unchanged and
 * outputs are undefined until fp8_host_sync() has returned FP8_OK; it waits for every host-buffer call made
 * so far on the current device.  The calls are serialised by an internal lock and may come from any
 * host thread.  Errors: FP8_ERR_NULL, FP8_ERR_SHAPE, FP8_ERR_WORKSPACE before anything is enqueued; an
 * error of an inner call is returned as is, with the work enqueued before it left to finish. */
FP8_API size_t fp8_linear_step_host_workspace_bytes(int T, int N, int K);
FP8_API int fp8_linear_step_host(const void *hX_bf16, const void *hW_bf16, const void *hdY_bf16, int T, int N, int K,
                         void *hY_bf16, void *hdX_bf16, void *hdW_bf16, void *ws, size_t ws_bytes);
FP8_API size_t fp8_attention_step_host_workspace_bytes(int B, int N, int Hq, int Hkv, int d);
FP8_API int fp8_attention_step_host(const void *hQ_bf16, const void *hK_bf16, const void *hV_bf16, const void *hdO_bf16,
                            int B, int N, int Hq, int Hkv, int d, float softmax_scale, float ds_scale, int causal,
                            void *hO_bf16, float *hLSE, void *hdQ_bf16, void *hdK_bf16, void *hdV_bf16,
                            void *ws, size_t ws_bytes);
FP8_API int fp8_host_sync(void);

#ifdef __cplusplus
}
#endif
#endif /* FP8DPA_H */
