// Element-wise companions of the quantize path: the gated activation fused with the cast, and the kurtosis
// monitor.  Both are HBM streams (16-byte loads and stores).  The sigmoid uses the hardware exp2 and reciprocal
// approximations (relative error near 2^-22): h is rounded to BF16 straight after, so the approximation shows
// only where the exact value sits within that distance of a BF16 rounding boundary.
#include <math.h>

#include "common.cuh"

namespace fp8dpa {

__device__ __forceinline__ uint32_t absmax2e(uint32_t m, uint32_t w) { return __vmaxu2(m, w & 0x7FFF7FFFu); }

__device__ __forceinline__ void block_max_bf16_to(uint32_t m2, unsigned int *amax_bits)
{
    __shared__ uint32_t warp_max[32];
    uint32_t m = max(m2 & 0xFFFFu, m2 >> 16);
    m = __reduce_max_sync(0xffffffffu, m);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) warp_max[warp] = m;
    __syncthreads();
    if (warp == 0) {
        const int nwarps = (blockDim.x + 31) >> 5;
        m = lane < nwarps ? warp_max[lane] : 0u;
        m = __reduce_max_sync(0xffffffffu, m);
        if (lane == 0 && m != 0u) atomicMax(amax_bits, m << 16);
    }
}

__device__ __forceinline__ float silu_mul(float g, float u)
{
    float r;
    const float e = ex2_approx(-1.4426950408889634f * g);     // exp(-g); +inf for very negative g gives r = 0
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
    return g * r * u;
}

// The un-gated activations work on pairs of values with the packed binary32 instructions (one instruction, two
// lanes): they are bound by instruction issue, not by memory, and the packed forms halve the count.
__device__ __forceinline__ uint64_t splat2(float c) { return pack_f32x2(c, c); }
__device__ __forceinline__ float rcp_approx(float x)
{
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// GeLU (exact form) of two values: x * Phi(x), Phi(x) = erfc(-x / sqrt 2) / 2.
// With y = |x| / sqrt 2 and e = erfc(y) / 2 (taken from the tail side, so that the left tail keeps its relative
// accuracy): x * Phi(x) = -|x| e for x < 0 and x - |x| e for x > 0, i.e. (x + |x|) / 2 - |x| e for both.
// e = t * 2^(L Q(t) - 1 - L y^2), t = 1 / (1 + y/2), L = log2(e): Q is a degree-9 least-squares fit of
// log(erfcx(y) / t) on Chebyshev nodes of t in [0.2, 1] (y in [0, 8]); evaluated in binary32 the relative error of
// e stays below 2e-6 up to y = 4 and 6e-6 up to y = 8, past which e is below 1e-29.  The coefficients below are
// those of L Q (the constant one with the -1 folded in).
__device__ __forceinline__ uint64_t gelu2(float x0, float x1)
{
    constexpr float L = 1.4426950408889634f;
    const uint64_t x = pack_f32x2(x0, x1);
    const uint64_t nax = pack_f32x2(__uint_as_float(__float_as_uint(x0) | 0x80000000u),
                                    __uint_as_float(__float_as_uint(x1) | 0x80000000u));     // -|x|
    const uint64_t y = mul_f32x2(nax, splat2(-0.70710678118654752440f));
    float d0, d1;
    unpack_f32x2(fma_f32x2(y, splat2(0.5f), splat2(1.0f)), d0, d1);
    const uint64_t t = pack_f32x2(rcp_approx(d0), rcp_approx(d1));
    uint64_t q = splat2(1.227935892e-01f * L);
    q = fma_f32x2(q, t, splat2(-5.583772951e-01f * L));
    q = fma_f32x2(q, t, splat2(8.634607687e-01f * L));
    q = fma_f32x2(q, t, splat2(-2.980391946e-01f * L));
    q = fma_f32x2(q, t, splat2(-4.172309384e-01f * L));
    q = fma_f32x2(q, t, splat2(1.850209772e-01f * L));
    q = fma_f32x2(q, t, splat2(-2.980059381e-02f * L));
    q = fma_f32x2(q, t, splat2(4.005914557e-01f * L));
    q = fma_f32x2(q, t, splat2(9.969420963e-01f * L));
    q = fma_f32x2(q, t, splat2(-1.265360832e+00f * L - 1.0f));
    float z0, z1;
    unpack_f32x2(fma_f32x2(mul_f32x2(y, y), splat2(-L), q), z0, z1);
    const uint64_t e = mul_f32x2(t, pack_f32x2(ex2_approx(z0), ex2_approx(z1)));             // erfc(y) / 2
    const uint64_t relu2x = fma_f32x2(nax, splat2(-1.0f), x);                                 // x + |x|, exact
    return fma_f32x2(relu2x, splat2(0.5f), mul_f32x2(nax, e));
}

// xIELU of two values with (a_p, a_n): x > 0: a_p x^2 + x/2; x <= 0: a_n (e^x - 1 - x) + x/2, with e^x - 1 - x from
// its series near 0 (|x| < 1/4, next term below 2e-9 of the first) and from the hardware exp2 elsewhere.
__device__ __forceinline__ uint64_t xielu2(float x0, float x1, float a_p, float a_n)
{
    const uint64_t x = pack_f32x2(x0, x1);
    const uint64_t hx = mul_f32x2(x, splat2(0.5f));
    const uint64_t pos = fma_f32x2(mul_f32x2(x, splat2(a_p)), x, hx);
    uint64_t ser = splat2(1.0f / 5040.0f);
    ser = fma_f32x2(ser, x, splat2(1.0f / 720.0f));
    ser = fma_f32x2(ser, x, splat2(1.0f / 120.0f));
    ser = fma_f32x2(ser, x, splat2(1.0f / 24.0f));
    ser = fma_f32x2(ser, x, splat2(1.0f / 6.0f));
    ser = fma_f32x2(ser, x, splat2(0.5f));
    ser = mul_f32x2(ser, mul_f32x2(x, x));
    float a0, a1;
    unpack_f32x2(mul_f32x2(x, splat2(1.4426950408889634f)), a0, a1);
    const uint64_t big = add_f32x2(pack_f32x2(ex2_approx(a0), ex2_approx(a1)), fma_f32x2(x, splat2(-1.0f), splat2(-1.0f)));
    float s0, s1, b0, b1, p0, p1, n0, n1;
    unpack_f32x2(ser, s0, s1);
    unpack_f32x2(big, b0, b1);
    const uint64_t neg = fma_f32x2(splat2(a_n), pack_f32x2(x0 > -0.25f ? s0 : b0, x1 > -0.25f ? s1 : b1), hx);
    unpack_f32x2(pos, p0, p1);
    unpack_f32x2(neg, n0, n1);
    return pack_f32x2(x0 > 0.0f ? p0 : n0, x1 > 0.0f ? p1 : n1);
}

// activations: 0 = SiLU(gate) * up (two inputs), 1 = GeLU (exact form), 2 = xIELU with (a_p, a_n);
// two values in, one word of two BF16 values out
constexpr int ACT_SWIGLU = 0;
template <int ACT>
__device__ __forceinline__ uint32_t act2(float g0, float g1, float u0, float u1, float a_p, float a_n)
{
    if (ACT == ACT_SWIGLU) return pack_bf16x2(silu_mul(g0, u0), silu_mul(g1, u1));
    float r0, r1;
    unpack_f32x2(ACT == FP8_ACT_GELU ? gelu2(g0, g1) : xielu2(g0, g1, a_p, a_n), r0, r1);
    return pack_bf16x2(r0, r1);
}

// 8 inputs (+ 8 up values for the gated form) -> 8 BF16 values of h (packed two per word)
template <int ACT>
__device__ __forceinline__ uint4 act8(const uint4 g, const uint4 u, float a_p, float a_n)
{
    const uint32_t gw[4] = {g.x, g.y, g.z, g.w}, uw[4] = {u.x, u.y, u.z, u.w};
    uint32_t h[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
        h[i] = act2<ACT>(bf16_lo(gw[i]), bf16_hi(gw[i]), bf16_lo(uw[i]), bf16_hi(uw[i]), a_p, a_n);
    return make_uint4(h[0], h[1], h[2], h[3]);
}

template <int FMT>
__device__ __forceinline__ uint2 cast8e(const uint4 v, const float s)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint16_t h[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
        h[i] = cvt_f32x2_to_fp8x2<FMT>(__fmul_rn(bf16_lo(w[i]), s), __fmul_rn(bf16_hi(w[i]), s));
    return make_uint2((uint32_t)h[0] | ((uint32_t)h[1] << 16), (uint32_t)h[2] | ((uint32_t)h[3] << 16));
}

constexpr int ST = 128;          // tile edge
constexpr int SPITCH = ST + 4;   // padded row of the staging tile

// One CTA per 128 x 128 tile of h.  Phase 1 computes h, its amax, the codes (row-major store + staging tile);
// phase 2 writes the transposed copy from the staging tile.
template <int FMT, int ACT>
__global__ void __launch_bounds__(256) act_cast_kernel(const uint16_t *__restrict__ gate_up, int T, int F,
                                                       const float *__restrict__ act_params,
                                                       const float *__restrict__ scale_ptr,
                                                       uint8_t *__restrict__ out, uint8_t *__restrict__ out_t,
                                                       unsigned int *__restrict__ amax_bits)
{
    constexpr bool GATED = ACT == ACT_SWIGLU;
    const int pitch = GATED ? 2 * F : F;              // input row length
    const float a_p = ACT == FP8_ACT_XIELU ? __ldg(act_params) : 0.0f;
    const float a_n = ACT == FP8_ACT_XIELU ? __ldg(act_params + 1) : 0.0f;
    __shared__ __align__(16) uint8_t tile[ST * SPITCH];
    const bool want_codes = out != nullptr || out_t != nullptr;
    const float s = want_codes ? __ldg(scale_ptr) : 1.0f;
    const int r0 = blockIdx.y * ST, c0 = blockIdx.x * ST;
    uint32_t m = 0;
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int idx = it * 256 + threadIdx.x;
        const int r = idx >> 3, cg = idx & 7;
        const int gr = r0 + r, gc = c0 + cg * 16;
        if (gr < T && gc < F) {
            const uint4 *pg = reinterpret_cast<const uint4 *>(gate_up + (size_t)gr * pitch + gc);
            const uint4 *pu = reinterpret_cast<const uint4 *>(gate_up + (size_t)gr * pitch + F + gc);
            const uint4 g0 = __ldg(pg), g1 = __ldg(pg + 1);
            const uint4 u0 = GATED ? __ldg(pu) : g0, u1 = GATED ? __ldg(pu + 1) : g1;
            const uint4 h0 = act8<ACT>(g0, u0, a_p, a_n), h1 = act8<ACT>(g1, u1, a_p, a_n);
            if (amax_bits) {
                m = absmax2e(absmax2e(absmax2e(absmax2e(m, h0.x), h0.y), h0.z), h0.w);
                m = absmax2e(absmax2e(absmax2e(absmax2e(m, h1.x), h1.y), h1.z), h1.w);
            }
            if (want_codes) {
                const uint2 p0 = cast8e<FMT>(h0, s), p1 = cast8e<FMT>(h1, s);
                if (out) *reinterpret_cast<uint4 *>(out + (size_t)gr * F + gc) = make_uint4(p0.x, p0.y, p1.x, p1.y);
                if (out_t) {
                    uint32_t *t = reinterpret_cast<uint32_t *>(tile + r * SPITCH + cg * 16);
                    t[0] = p0.x; t[1] = p0.y; t[2] = p1.x; t[3] = p1.y;
                }
            }
        }
    }
    if (out_t) {
        __syncthreads();
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int idx = it * 256 + threadIdx.x;
            const int half = idx & 1, c = (idx >> 1) & 127, rp = idx >> 8;
            const int rg = rp * 2 + half;
            const int gc = c0 + c, gr = r0 + rg * 16;
            if (gc < F && gr < T) {
                uint32_t w[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint32_t v = 0;
#pragma unroll
                    for (int b = 0; b < 4; ++b) v |= (uint32_t)tile[(rg * 16 + q * 4 + b) * SPITCH + c] << (8 * b);
                    w[q] = v;
                }
                *reinterpret_cast<uint4 *>(out_t + (size_t)gc * T + gr) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
    }
    if (amax_bits) block_max_bf16_to(m, amax_bits);
}

// One CTA per row: sums of x^2 and x^4, then kurt = mean(x^4) / mean(x^2)^2 added (scaled by 1/rows) to *out.
// With amax_bits the same pass also takes the tensor's amax (the pass a just-in-time quantisation makes anyway).
__global__ void __launch_bounds__(256) kurtosis_kernel(const uint16_t *__restrict__ x, int cols, float inv_rows,
                                                       float *__restrict__ out, unsigned int *__restrict__ amax_bits)
{
    __shared__ float red2[8], red4[8];
    const uint4 *row = reinterpret_cast<const uint4 *>(x + (size_t)blockIdx.x * cols);
    float s2 = 0.0f, s4 = 0.0f;
    uint32_t m = 0;
    for (int i = threadIdx.x; i < cols / 8; i += blockDim.x) {
        const uint4 v = __ldg(row + i);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        m = absmax2e(absmax2e(absmax2e(absmax2e(m, v.x), v.y), v.z), v.w);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float a = bf16_lo(w[k]), b = bf16_hi(w[k]);
            const float a2 = a * a, b2 = b * b;
            s2 += a2 + b2;
            s4 += a2 * a2 + b2 * b2;
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        s2 += __shfl_xor_sync(0xffffffffu, s2, off);
        s4 += __shfl_xor_sync(0xffffffffu, s4, off);
    }
    if ((threadIdx.x & 31) == 0) {
        red2[threadIdx.x >> 5] = s2;
        red4[threadIdx.x >> 5] = s4;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float t2 = 0.0f, t4 = 0.0f;
        for (int w = 0; w < 8; ++w) { t2 += red2[w]; t4 += red4[w]; }
        if (t2 > 0.0f) {
            const float m2 = t2 / (float)cols, m4 = t4 / (float)cols;
            atomicAdd(out, m4 / (m2 * m2) * inv_rows);
        }
    }
    if (amax_bits) block_max_bf16_to(m, amax_bits);
}

// Post-norm + residual, one CTA per token row.  The row of y stays in registers between the sum of squares and the
// update: KG 16-byte groups per thread at 256 threads (KG = 1, 2, 4, 8 for up to 2048 ... 16384 columns, chosen at
// launch so that short rows do not pay for the registers of long ones).

// Eight BF16 values (four packed words) -> eight FP8 codes under `scale`: the codes fp8_cast gives for the same
// values (binary32 product, one rounding to FP8).  fmt: 0 = E4M3, 1 = E5M2.
__device__ __forceinline__ uint2 bf16x8_to_fp8x8(const uint32_t (&w)[4], float scale, int fmt)
{
    const float v0 = __fmul_rn(bf16_lo(w[0]), scale), v1 = __fmul_rn(bf16_hi(w[0]), scale);
    const float v2 = __fmul_rn(bf16_lo(w[1]), scale), v3 = __fmul_rn(bf16_hi(w[1]), scale);
    const float v4 = __fmul_rn(bf16_lo(w[2]), scale), v5 = __fmul_rn(bf16_hi(w[2]), scale);
    const float v6 = __fmul_rn(bf16_lo(w[3]), scale), v7 = __fmul_rn(bf16_hi(w[3]), scale);
    if (fmt == 0) return make_uint2(cvt_f32x4_to_fp8x4<0>(v0, v1, v2, v3), cvt_f32x4_to_fp8x4<0>(v4, v5, v6, v7));
    return make_uint2(cvt_f32x4_to_fp8x4<1>(v0, v1, v2, v3), cvt_f32x4_to_fp8x4<1>(v4, v5, v6, v7));
}

template <int MODE, int KG>
__global__ void __launch_bounds__(256) postnorm_residual_kernel(const uint16_t *__restrict__ x,
                                                                const uint16_t *__restrict__ y,
                                                                const float *__restrict__ gamma, int D, float eps,
                                                                uint16_t *__restrict__ out,
                                                                unsigned int *__restrict__ amax_bits, float x_scale,
                                                                const float *__restrict__ q_scale,
                                                                uint8_t *__restrict__ out8, int fmt)
{
    __shared__ float red[8];
    const float qs = out8 ? __ldg(q_scale) : 1.0f;
    const size_t base = (size_t)blockIdx.x * D;
    const uint4 *py = reinterpret_cast<const uint4 *>(y + base);
    const uint4 *px = reinterpret_cast<const uint4 *>(x + base);
    uint4 *po = reinterpret_cast<uint4 *>(out + base);
    const int n8 = D / 8;
    uint4 yv[KG], xv8[KG];
    float ss = 0.0f;
#pragma unroll
    for (int k = 0; k < KG; ++k) {
        const int i = k * 256 + threadIdx.x;
        if (i < n8) {
            yv[k] = __ldg(py + i);
            xv8[k] = __ldg(px + i);       // in flight during the reduction
            const uint32_t w[4] = {yv[k].x, yv[k].y, yv[k].z, yv[k].w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float a = bf16_lo(w[q]), b = bf16_hi(w[q]);
                ss = fmaf(a, a, fmaf(b, b, ss));
            }
        }
    }
    float rinv = 1.0f;
    if (MODE == FP8_NORM_RMS) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
        __syncthreads();
        float tot = 0.0f;
#pragma unroll
        for (int w = 0; w < 8; ++w) tot += red[w];
        rinv = 1.0f / sqrtf(tot / (float)D + eps);
    }
    uint32_t m = 0;
#pragma unroll
    for (int k = 0; k < KG; ++k) {
        const int i = k * 256 + threadIdx.x;
        if (i < n8) {
            const uint4 xv = xv8[k];
            const float4 g0 = __ldg(reinterpret_cast<const float4 *>(gamma) + 2 * i);
            const float4 g1 = __ldg(reinterpret_cast<const float4 *>(gamma) + 2 * i + 1);
            const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
            const uint32_t yw[4] = {yv[k].x, yv[k].y, yv[k].z, yv[k].w}, xw[4] = {xv.x, xv.y, xv.z, xv.w};
            uint32_t o[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float lo = fmaf(g[2 * q] * rinv, bf16_lo(yw[q]), x_scale * bf16_lo(xw[q]));
                const float hi = fmaf(g[2 * q + 1] * rinv, bf16_hi(yw[q]), x_scale * bf16_hi(xw[q]));
                o[q] = pack_bf16x2(lo, hi);
                m = absmax2e(m, o[q]);
            }
            po[i] = make_uint4(o[0], o[1], o[2], o[3]);
            if (out8) *reinterpret_cast<uint2 *>(out8 + base + (size_t)i * 8) = bf16x8_to_fp8x8(o, qs, fmt);
        }
    }
    if (amax_bits) block_max_bf16_to(m, amax_bits);
}

// QK regulariser + rotary embedding.  A (token, head) vector is handled by D/16 adjacent lanes: lane j of the group
// holds elements [8j, 8j+8) of the first half and the same of the second half (two 16-byte loads), so the rotation
// partner i + D/2 of every element lives in the same lane and the sum of squares needs log2(D/16) shuffles.
// A lane group takes QK_HC consecutive heads of one token, so the 16 cos/sin values of its position are read once
// per QK_HC vectors.
constexpr int QK_HC = 8;
template <int D, int MODE>
__global__ void __launch_bounds__(256) qk_norm_rope_kernel(const uint16_t *__restrict__ x, size_t n_tok, int H,
                                                           float alpha, float eps, const float *__restrict__ cos_t,
                                                           const float *__restrict__ sin_t, int seq_len,
                                                           uint16_t *__restrict__ out,
                                                           unsigned int *__restrict__ amax_bits,
                                                           const float *__restrict__ q_scale,
                                                           uint8_t *__restrict__ out8, int fmt)
{
    constexpr int LPV = D / 16;             // lanes per vector: 8 (d = 128) or 4 (d = 64)
    const float qs = out8 ? __ldg(q_scale) : 1.0f;
    constexpr int GPB = 256 / LPV;          // lane groups per CTA
    const int j = threadIdx.x % LPV;
    const int chunks = (H + QK_HC - 1) / QK_HC;
    const size_t n_items = n_tok * (size_t)chunks;            // (token, chunk of heads)
    uint32_t m = 0;
    // The trip counts are uniform over the CTA (the shuffles below name every lane of the warp): a lane group past
    // the end re-reads the last vector and stores nothing.
    for (size_t base = (size_t)blockIdx.x * GPB; base < n_items; base += (size_t)gridDim.x * GPB) {
        const size_t item_raw = base + threadIdx.x / LPV;
        const bool item_valid = item_raw < n_items;
        const size_t item = item_valid ? item_raw : n_items - 1;
        const size_t tok = item / (size_t)chunks;
        const int h0 = (int)(item % (size_t)chunks) * QK_HC;
        float c[8], sn[8];
        if (cos_t) {
            const size_t pos = tok % (size_t)seq_len;
            const float4 *pc = reinterpret_cast<const float4 *>(cos_t + pos * (D / 2) + j * 8);
            const float4 *ps = reinterpret_cast<const float4 *>(sin_t + pos * (D / 2) + j * 8);
            const float4 c0 = __ldg(pc), c1 = __ldg(pc + 1), s0 = __ldg(ps), s1 = __ldg(ps + 1);
            c[0] = c0.x; c[1] = c0.y; c[2] = c0.z; c[3] = c0.w; c[4] = c1.x; c[5] = c1.y; c[6] = c1.z; c[7] = c1.w;
            sn[0] = s0.x; sn[1] = s0.y; sn[2] = s0.z; sn[3] = s0.w; sn[4] = s1.x; sn[5] = s1.y; sn[6] = s1.z; sn[7] = s1.w;
        }
#pragma unroll 4
        for (int hh = 0; hh < QK_HC; ++hh) {
            const bool valid = item_valid && h0 + hh < H;
            const size_t v = tok * (size_t)H + (size_t)min(h0 + hh, H - 1);
            const uint16_t *px = x + v * D + j * 8;
            const uint4 wa = __ldg(reinterpret_cast<const uint4 *>(px));
            const uint4 wb = __ldg(reinterpret_cast<const uint4 *>(px + D / 2));
            const uint32_t ua[4] = {wa.x, wa.y, wa.z, wa.w}, ub[4] = {wb.x, wb.y, wb.z, wb.w};
            float a[8], b[8];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                a[2 * q] = bf16_lo(ua[q]); a[2 * q + 1] = bf16_hi(ua[q]);
                b[2 * q] = bf16_lo(ub[q]); b[2 * q + 1] = bf16_hi(ub[q]);
            }
            if (MODE == FP8_QK_RMS) {
                float ss = 0.0f;
#pragma unroll
                for (int e = 0; e < 8; ++e) ss = fmaf(a[e], a[e], fmaf(b[e], b[e], ss));
#pragma unroll
                for (int off = LPV / 2; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
                const float rinv = rsqrtf(fmaf(ss, 1.0f / (float)D, eps));
#pragma unroll
                for (int e = 0; e < 8; ++e) { a[e] *= rinv; b[e] *= rinv; }
            } else if (MODE == FP8_QK_TANH) {
#pragma unroll
                for (int e = 0; e < 8; ++e) { a[e] = tanhf(alpha * a[e]); b[e] = tanhf(alpha * b[e]); }
            }
            if (cos_t) {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float ra = a[e] * c[e] - b[e] * sn[e], rb = b[e] * c[e] + a[e] * sn[e];
                    a[e] = ra;
                    b[e] = rb;
                }
            }
            uint32_t oa[4], ob[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                oa[q] = pack_bf16x2(a[2 * q], a[2 * q + 1]);
                ob[q] = pack_bf16x2(b[2 * q], b[2 * q + 1]);
                if (valid) m = absmax2e(absmax2e(m, oa[q]), ob[q]);
            }
            if (valid && out) {
                uint16_t *po = out + v * D + j * 8;
                *reinterpret_cast<uint4 *>(po) = make_uint4(oa[0], oa[1], oa[2], oa[3]);
                *reinterpret_cast<uint4 *>(po + D / 2) = make_uint4(ob[0], ob[1], ob[2], ob[3]);
            }
            if (valid && out8) {
                uint8_t *p8 = out8 + v * D + j * 8;
                *reinterpret_cast<uint2 *>(p8) = bf16x8_to_fp8x8(oa, qs, fmt);
                *reinterpret_cast<uint2 *>(p8 + D / 2) = bf16x8_to_fp8x8(ob, qs, fmt);
            }
        }
    }
    if (amax_bits) block_max_bf16_to(m, amax_bits);
}

}  // namespace fp8dpa

using namespace fp8dpa;

static int act_cast(const char *who, const void *x, size_t T, size_t F, int act, const float *act_params,
                    const float *scale, int fmt, uint8_t *out, uint8_t *out_t, float *amax_out, void *stream)
{
    const bool want_codes = out || out_t;
    if (!x || (want_codes && !scale) || (!want_codes && !amax_out) || (act == FP8_ACT_XIELU && !act_params)) {
        set_error("%s: NULL pointer (need the input, either outputs with a scale or amax_out, and act_params for xIELU)", who);
        return FP8_ERR_NULL;
    }
    if ((fmt != FP8_E4M3 && fmt != FP8_E5M2) || act < 0 || act > FP8_ACT_XIELU) {
        set_error("%s: fmt %d / act %d is not a known enum value", who, fmt, act);
        return FP8_ERR_ENUM;
    }
    if (T == 0 || F == 0 || (F % 16) || (out_t && (T % 16)) || T > 0x7FFFFFFFull || F > 0x3FFFFFFFull) {
        set_error("%s: unsupported shape T=%zu F=%zu (F %% 16 == 0; T %% 16 == 0 with a transposed copy)", who, T, F);
        return FP8_ERR_SHAPE;
    }
    if (!aligned16(x) || !aligned16(out) || !aligned16(out_t)) {
        set_error("%s: tensor pointers must be 16-byte aligned", who);
        return FP8_ERR_ALIGN;
    }
    int rc = check_arch();
    if (rc != FP8_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (amax_out) FP8_CUDA_CHECK(cudaMemsetAsync(amax_out, 0, sizeof(float), st));
    dim3 grid((unsigned)((F + ST - 1) / ST), (unsigned)((T + ST - 1) / ST));
    const uint16_t *xp = static_cast<const uint16_t *>(x);
    unsigned int *ab = reinterpret_cast<unsigned int *>(amax_out);
#define FP8DPA_LAUNCH_ACT(FMT, ACT) \
    act_cast_kernel<FMT, ACT><<<grid, 256, 0, st>>>(xp, (int)T, (int)F, act_params, scale, out, out_t, ab)
    if (fmt == FP8_E4M3) {
        if (act == ACT_SWIGLU) FP8DPA_LAUNCH_ACT(0, ACT_SWIGLU);
        else if (act == FP8_ACT_GELU) FP8DPA_LAUNCH_ACT(0, FP8_ACT_GELU);
        else FP8DPA_LAUNCH_ACT(0, FP8_ACT_XIELU);
    } else {
        if (act == ACT_SWIGLU) FP8DPA_LAUNCH_ACT(1, ACT_SWIGLU);
        else if (act == FP8_ACT_GELU) FP8DPA_LAUNCH_ACT(1, FP8_ACT_GELU);
        else FP8DPA_LAUNCH_ACT(1, FP8_ACT_XIELU);
    }
#undef FP8DPA_LAUNCH_ACT
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

extern "C" int fp8_swiglu_cast(const void *gate_up_bf16, size_t T, size_t F, const float *scale, int fmt, uint8_t *out,
                               uint8_t *out_t, float *amax_out, void *stream)
{
    return act_cast("fp8_swiglu_cast", gate_up_bf16, T, F, ACT_SWIGLU, nullptr, scale, fmt, out, out_t, amax_out, stream);
}

extern "C" int fp8_act_cast(const void *x_bf16, size_t T, size_t F, int act, const float *act_params, const float *scale,
                            int fmt, uint8_t *out, uint8_t *out_t, float *amax_out, void *stream)
{
    if (act != FP8_ACT_GELU && act != FP8_ACT_XIELU) {
        set_error("fp8_act_cast: act %d is not FP8_ACT_GELU / FP8_ACT_XIELU", act);
        return FP8_ERR_ENUM;
    }
    return act_cast("fp8_act_cast", x_bf16, T, F, act, act_params, scale, fmt, out, out_t, amax_out, stream);
}

static int kurtosis_common(const void *x_bf16, size_t rows, size_t cols, float *out, float *amax_out, void *stream)
{
    if (!x_bf16 || !out) {
        set_error("fp8_kurtosis: NULL pointer");
        return FP8_ERR_NULL;
    }
    if (rows == 0 || cols == 0 || (cols % 8) || rows > 0x7FFFFFFFull || cols > 0x7FFFFFFFull) {
        set_error("fp8_kurtosis: unsupported shape rows=%zu cols=%zu (cols %% 8 == 0)", rows, cols);
        return FP8_ERR_SHAPE;
    }
    if (!aligned16(x_bf16)) {
        set_error("fp8_kurtosis: x must be 16-byte aligned");
        return FP8_ERR_ALIGN;
    }
    int rc = check_arch();
    if (rc != FP8_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    FP8_CUDA_CHECK(cudaMemsetAsync(out, 0, sizeof(float), st));
    if (amax_out) FP8_CUDA_CHECK(cudaMemsetAsync(amax_out, 0, sizeof(float), st));
    kurtosis_kernel<<<(unsigned)rows, 256, 0, st>>>(static_cast<const uint16_t *>(x_bf16), (int)cols,
                                                   1.0f / (float)rows, out, reinterpret_cast<unsigned int *>(amax_out));
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

extern "C" int fp8_kurtosis(const void *x_bf16, size_t rows, size_t cols, float *out, void *stream)
{
    return kurtosis_common(x_bf16, rows, cols, out, nullptr, stream);
}

extern "C" int fp8_amax_kurtosis(const void *x_bf16, size_t rows, size_t cols, float *amax, float *kurtosis, void *stream)
{
    if (!amax) {
        set_error("fp8_amax_kurtosis: NULL amax");
        return FP8_ERR_NULL;
    }
    return kurtosis_common(x_bf16, rows, cols, kurtosis, amax, stream);
}

static int postnorm_common(const void *x_bf16, const void *y_bf16, const float *gamma, size_t T, size_t D, int mode,
                           float eps, float x_scale, const float *q_scale, int fmt, void *out_bf16, uint8_t *out8,
                           float *amax_out, void *stream)
{
    if (!x_bf16 || !y_bf16 || !gamma || !out_bf16 || (out8 && !q_scale)) {
        set_error("fp8_postnorm_residual: NULL pointer");
        return FP8_ERR_NULL;
    }
    if (out8 && fmt != FP8_E4M3 && fmt != FP8_E5M2) {
        set_error("fp8_postnorm_residual_q: fmt %d is not FP8_E4M3 / FP8_E5M2", fmt);
        return FP8_ERR_ENUM;
    }
    if (!aligned16(out8) || !(x_scale == x_scale)) {
        set_error("fp8_postnorm_residual_q: out8 must be 16-byte aligned and x_scale a number");
        return FP8_ERR_ALIGN;
    }
    if (mode != FP8_NORM_RMS && mode != FP8_NORM_LAYERSCALE) {
        set_error("fp8_postnorm_residual: mode %d is not FP8_NORM_RMS / FP8_NORM_LAYERSCALE", mode);
        return FP8_ERR_ENUM;
    }
    if (T == 0 || D == 0 || (D % 8) || D > 16384 || T > 0x7FFFFFFFull || !(eps >= 0.0f)) {
        set_error("fp8_postnorm_residual: unsupported shape T=%zu D=%zu (D %% 8 == 0, D <= 16384) or eps < 0", T, D);
        return FP8_ERR_SHAPE;
    }
    if (!aligned16(x_bf16) || !aligned16(y_bf16) || !aligned16(gamma) || !aligned16(out_bf16)) {
        set_error("fp8_postnorm_residual: pointers must be 16-byte aligned");
        return FP8_ERR_ALIGN;
    }
    int rc = check_arch();
    if (rc != FP8_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (amax_out) FP8_CUDA_CHECK(cudaMemsetAsync(amax_out, 0, sizeof(float), st));
    const uint16_t *x = static_cast<const uint16_t *>(x_bf16), *y = static_cast<const uint16_t *>(y_bf16);
    uint16_t *o = static_cast<uint16_t *>(out_bf16);
    unsigned int *ab = reinterpret_cast<unsigned int *>(amax_out);
#define FP8DPA_LAUNCH_PN(MM, KG) \
    postnorm_residual_kernel<MM, KG><<<(unsigned)T, 256, 0, st>>>(x, y, gamma, (int)D, eps, o, ab, x_scale, q_scale, out8, fmt)
#define FP8DPA_LAUNCH_PN_KG(MM) \
    do { \
        if (D <= 2048) FP8DPA_LAUNCH_PN(MM, 1); \
        else if (D <= 4096) FP8DPA_LAUNCH_PN(MM, 2); \
        else if (D <= 8192) FP8DPA_LAUNCH_PN(MM, 4); \
        else FP8DPA_LAUNCH_PN(MM, 8); \
    } while (0)
    if (mode == FP8_NORM_RMS) FP8DPA_LAUNCH_PN_KG(FP8_NORM_RMS);
    else FP8DPA_LAUNCH_PN_KG(FP8_NORM_LAYERSCALE);
#undef FP8DPA_LAUNCH_PN_KG
#undef FP8DPA_LAUNCH_PN
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

extern "C" int fp8_postnorm_residual(const void *x_bf16, const void *y_bf16, const float *gamma, size_t T, size_t D,
                                     int mode, float eps, void *out_bf16, float *amax_out, void *stream)
{
    return postnorm_common(x_bf16, y_bf16, gamma, T, D, mode, eps, 1.0f, nullptr, 0, out_bf16, nullptr, amax_out, stream);
}

extern "C" int fp8_postnorm_residual_q(const void *x_bf16, const void *y_bf16, const float *gamma, size_t T, size_t D,
                                       int mode, float eps, float x_scale, const float *scale, int fmt, void *out_bf16,
                                       uint8_t *out8, float *amax_out, void *stream)
{
    if (!out8 || !scale) {
        set_error("fp8_postnorm_residual_q: NULL scale / out8");
        return FP8_ERR_NULL;
    }
    return postnorm_common(x_bf16, y_bf16, gamma, T, D, mode, eps, x_scale, scale, fmt, out_bf16, out8, amax_out, stream);
}

static int qk_common(const void *x_bf16, size_t T, size_t H, size_t d, int mode, float alpha, float eps,
                     const float *cos_table, const float *sin_table, size_t seq_len, const float *q_scale, int fmt,
                     void *out_bf16, uint8_t *out8, float *amax_out, void *stream)
{
    if (!x_bf16 || (!out_bf16 && !out8) || ((cos_table == nullptr) != (sin_table == nullptr)) || (out8 && !q_scale)) {
        set_error("fp8_qk_norm_rope: NULL pointer (cos and sin tables come together; FP8 output needs its scale)");
        return FP8_ERR_NULL;
    }
    if (out8 && fmt != FP8_E4M3 && fmt != FP8_E5M2) {
        set_error("fp8_qk_norm_rope_q: fmt %d is not FP8_E4M3 / FP8_E5M2", fmt);
        return FP8_ERR_ENUM;
    }
    if (!aligned16(out8)) {
        set_error("fp8_qk_norm_rope_q: out8 must be 16-byte aligned");
        return FP8_ERR_ALIGN;
    }
    if (mode < FP8_QK_RMS || mode > FP8_QK_NONE) {
        set_error("fp8_qk_norm_rope: mode %d is not FP8_QK_RMS / FP8_QK_TANH / FP8_QK_NONE", mode);
        return FP8_ERR_ENUM;
    }
    if (T == 0 || H == 0 || (d != 64 && d != 128) || (cos_table && seq_len == 0) || H > 65535 || !(eps >= 0.0f) ||
        seq_len > 0x7FFFFFFFull) {
        set_error("fp8_qk_norm_rope: unsupported shape T=%zu H=%zu d=%zu seq_len=%zu (d in {64,128})", T, H, d, seq_len);
        return FP8_ERR_SHAPE;
    }
    if (!aligned16(x_bf16) || !aligned16(out_bf16) || !aligned16(cos_table) || !aligned16(sin_table)) {
        set_error("fp8_qk_norm_rope: pointers must be 16-byte aligned");
        return FP8_ERR_ALIGN;
    }
    int rc = check_arch();
    if (rc != FP8_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (amax_out) FP8_CUDA_CHECK(cudaMemsetAsync(amax_out, 0, sizeof(float), st));
    const size_t gpb = 256 / (d / 16);          // lane groups per CTA, each taking QK_HC heads of one token
    const size_t n_items = T * ((H + QK_HC - 1) / QK_HC);
    size_t blocks = (n_items + gpb - 1) / gpb;
    const size_t cap = (size_t)sm_count() * 16;
    if (blocks > cap) blocks = cap;
    const uint16_t *x = static_cast<const uint16_t *>(x_bf16);
    uint16_t *o = static_cast<uint16_t *>(out_bf16);
    unsigned int *ab = reinterpret_cast<unsigned int *>(amax_out);
#define FP8DPA_LAUNCH_QK(DD, MM) \
    qk_norm_rope_kernel<DD, MM><<<(unsigned)blocks, 256, 0, st>>>(x, T, (int)H, alpha, eps, cos_table, sin_table, \
                                                                 (int)(seq_len ? seq_len : 1), o, ab, q_scale, out8, fmt)
    if (d == 128) {
        if (mode == FP8_QK_RMS) FP8DPA_LAUNCH_QK(128, FP8_QK_RMS);
        else if (mode == FP8_QK_TANH) FP8DPA_LAUNCH_QK(128, FP8_QK_TANH);
        else FP8DPA_LAUNCH_QK(128, FP8_QK_NONE);
    } else {
        if (mode == FP8_QK_RMS) FP8DPA_LAUNCH_QK(64, FP8_QK_RMS);
        else if (mode == FP8_QK_TANH) FP8DPA_LAUNCH_QK(64, FP8_QK_TANH);
        else FP8DPA_LAUNCH_QK(64, FP8_QK_NONE);
    }
#undef FP8DPA_LAUNCH_QK
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

extern "C" int fp8_qk_norm_rope(const void *x_bf16, size_t T, size_t H, size_t d, int mode, float alpha, float eps,
                                const float *cos_table, const float *sin_table, size_t seq_len, void *out_bf16,
                                float *amax_out, void *stream)
{
    if (!out_bf16) {
        set_error("fp8_qk_norm_rope: NULL output");
        return FP8_ERR_NULL;
    }
    return qk_common(x_bf16, T, H, d, mode, alpha, eps, cos_table, sin_table, seq_len, nullptr, 0, out_bf16, nullptr,
                     amax_out, stream);
}

extern "C" int fp8_qk_norm_rope_q(const void *x_bf16, size_t T, size_t H, size_t d, int mode, float alpha, float eps,
                                  const float *cos_table, const float *sin_table, size_t seq_len, const float *scale,
                                  int fmt, void *out_bf16, uint8_t *out8, float *amax_out, void *stream)
{
    if (!out8 || !scale) {
        set_error("fp8_qk_norm_rope_q: NULL scale / out8");
        return FP8_ERR_NULL;
    }
    return qk_common(x_bf16, T, H, d, mode, alpha, eps, cos_table, sin_table, seq_len, scale, fmt, out_bf16, out8,
                     amax_out, stream);
}
