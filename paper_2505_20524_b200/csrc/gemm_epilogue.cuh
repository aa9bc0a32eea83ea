// Pieces shared by the FP8 GEMM kernels: the tile order and the epilogue.
// Epilogue: 32 accumulator columns of one output row (binary32, straight from TMEM) ->
// descaled BF16 / FP32 values with 16-byte stores, or, for a producer under delayed scaling (Appendix E: the scale
// comes from the amax history, so a single pass suffices), FP8 codes of the BF16-rounded result plus its amax.
#pragma once
#include "common.cuh"

namespace fp8dpa {

// Tile order shared by the GEMM kernels: bands of GEMM_BAND tiles along the longer output dimension; inside a band the
// index along the shorter dimension advances slowest.  The CTAs that run at the same time then share one band of
// one operand (a few MB) and a handful of panels of the other, and both stay in L2 however long the matrix is.
constexpr int GEMM_BAND = 16;
__device__ __forceinline__ void band_coords_w(int tile, int n_long, int n_short, int band_w, int &i_long, int &i_short)
{
    const int per_band = band_w * n_short;
    const int band = tile / per_band, within = tile - band * per_band;
    const int len = min(band_w, n_long - band * band_w);     // the last band may be short
    i_short = within / len;
    i_long = band * band_w + (within - i_short * len);
}
__device__ __forceinline__ void band_coords(int tile, int n_long, int n_short, int &i_long, int &i_short)
{
    band_coords_w(tile, n_long, n_short, GEMM_BAND, i_long, i_short);
}

struct GemmOut {
    void *out;                 // BF16 / FP32 / FP8 [M,N] row-major
    int out_is_fp32;           // ignored when q_scale is set
    int accumulate;            // out += result (BF16 / FP32 only)
    const float *q_scale;      // non-NULL: emit FP8 codes of bf16(result) * *q_scale
    int q_fmt;                 // FP8_E4M3 / FP8_E5M2
    unsigned int *amax_bits;   // with q_scale: amax of the BF16-rounded result, as binary32 bits (atomicMax), nullable
};

// r: 32 accumulators of row `row`, columns col .. col+31 (ncols of them inside the matrix; N % 16 == 0 so ncols is
// 16 or 32).  amax2: per-thread running max of |BF16 bits| in both 16-bit halves (FP8 mode).
__device__ __forceinline__ void gemm_store_chunk(const uint32_t (&r)[32], float descale, const GemmOut &o, float q_scale,
                                                 int N, int row, int col, int ncols, uint32_t &amax2)
{
    if (o.q_scale) {
        uint8_t *dst = static_cast<uint8_t *>(o.out) + (size_t)row * N + col;
#pragma unroll
        for (int j = 0; j < 32; j += 16) {
            if (j < ncols) {
                uint32_t w[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    // BF16 first: these are the values an unfused chain would have stored and then cast
                    const uint32_t b0 = pack_bf16x2(__uint_as_float(r[j + 4 * q]) * descale,
                                                    __uint_as_float(r[j + 4 * q + 1]) * descale);
                    const uint32_t b1 = pack_bf16x2(__uint_as_float(r[j + 4 * q + 2]) * descale,
                                                    __uint_as_float(r[j + 4 * q + 3]) * descale);
                    amax2 = __vmaxu2(__vmaxu2(amax2, b0 & 0x7FFF7FFFu), b1 & 0x7FFF7FFFu);
                    const float f0 = __fmul_rn(bf16_lo(b0), q_scale), f1 = __fmul_rn(bf16_hi(b0), q_scale);
                    const float f2 = __fmul_rn(bf16_lo(b1), q_scale), f3 = __fmul_rn(bf16_hi(b1), q_scale);
                    w[q] = o.q_fmt == FP8_E4M3 ? cvt_f32x4_to_fp8x4<0>(f0, f1, f2, f3) : cvt_f32x4_to_fp8x4<1>(f0, f1, f2, f3);
                }
                *reinterpret_cast<uint4 *>(dst + j) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
    } else if (o.out_is_fp32) {
        float *dst = static_cast<float *>(o.out) + (size_t)row * N + col;
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
            if (j < ncols) {
                float4 v = make_float4(__uint_as_float(r[j]) * descale, __uint_as_float(r[j + 1]) * descale,
                                       __uint_as_float(r[j + 2]) * descale, __uint_as_float(r[j + 3]) * descale);
                if (o.accumulate) {
                    const float4 p = *reinterpret_cast<const float4 *>(dst + j);
                    v.x += p.x; v.y += p.y; v.z += p.z; v.w += p.w;
                }
                *reinterpret_cast<float4 *>(dst + j) = v;
            }
        }
    } else {
        uint16_t *dst = static_cast<uint16_t *>(o.out) + (size_t)row * N + col;
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
            if (j < ncols) {
                float v[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) v[q] = __uint_as_float(r[j + q]) * descale;
                if (o.accumulate) {
                    const uint4 p = *reinterpret_cast<const uint4 *>(dst + j);
                    v[0] += bf16_lo(p.x); v[1] += bf16_hi(p.x); v[2] += bf16_lo(p.y); v[3] += bf16_hi(p.y);
                    v[4] += bf16_lo(p.z); v[5] += bf16_hi(p.z); v[6] += bf16_lo(p.w); v[7] += bf16_hi(p.w);
                }
                *reinterpret_cast<uint4 *>(dst + j) = make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]),
                                                                  pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
            }
        }
    }
}

// After the last tile of an epilogue warp: publish its amax (FP8 mode).
__device__ __forceinline__ void gemm_publish_amax(const GemmOut &o, uint32_t amax2)
{
    if (!o.q_scale || !o.amax_bits) return;
    uint32_t m = max(amax2 & 0xFFFFu, amax2 >> 16);
    m = __reduce_max_sync(0xffffffffu, m);
    if ((threadIdx.x & 31) == 0 && m != 0u) atomicMax(o.amax_bits, m << 16);
}

}  // namespace fp8dpa
