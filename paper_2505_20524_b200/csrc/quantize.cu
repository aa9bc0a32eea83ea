// Per-tensor scaling kernels: amax reduction, scale computation, saturating BF16 -> FP8 cast
// (optionally with a transposed copy and a fused amax).  All are HBM streams: 128-bit loads and stores,
// warp-shuffle + one atomic per CTA for the reduction, scales read from device memory.
//
// No fast-math on this file: the binary32 division and product below define the bit-exact result.
#include <float.h>

#include "common.cuh"

namespace fp8dpa {

// ---------------------------------------------------------------- amax
__device__ __forceinline__ uint32_t absmax2(uint32_t m, uint32_t w) { return __vmaxu2(m, w & 0x7FFF7FFFu); }

__device__ __forceinline__ void block_atomic_max_bf16(uint32_t m2, unsigned int *amax_bits)
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
        // |x| as BF16 bits << 16 is the binary32 pattern of |x|; positive floats order like unsigned ints
        if (lane == 0 && m != 0u) atomicMax(amax_bits, m << 16);
    }
}

// The reduction over one tensor as seen by block `rank` of the `nblk` blocks that share it.
__device__ __forceinline__ void amax_body(const uint4 *__restrict__ x, size_t n_vec, const uint16_t *__restrict__ tail,
                                          int n_tail, unsigned int *__restrict__ amax_bits, unsigned rank, unsigned nblk)
{
    uint32_t m = 0;
    const size_t stride = (size_t)nblk * blockDim.x;
    size_t i = (size_t)rank * blockDim.x + threadIdx.x;
    // four independent 16-byte loads in flight per thread
    for (; i + 3 * stride < n_vec; i += 4 * stride) {
        const uint4 a = __ldg(x + i), b = __ldg(x + i + stride), c = __ldg(x + i + 2 * stride),
                    d = __ldg(x + i + 3 * stride);
        m = absmax2(absmax2(absmax2(absmax2(m, a.x), a.y), a.z), a.w);
        m = absmax2(absmax2(absmax2(absmax2(m, b.x), b.y), b.z), b.w);
        m = absmax2(absmax2(absmax2(absmax2(m, c.x), c.y), c.z), c.w);
        m = absmax2(absmax2(absmax2(absmax2(m, d.x), d.y), d.z), d.w);
    }
    for (; i < n_vec; i += stride) {
        const uint4 a = __ldg(x + i);
        m = absmax2(absmax2(absmax2(absmax2(m, a.x), a.y), a.z), a.w);
    }
    if (rank == 0 && (int)threadIdx.x < n_tail) m = absmax2(m, (uint32_t)tail[threadIdx.x]);
    block_atomic_max_bf16(m, amax_bits);
}

__global__ void __launch_bounds__(512) amax_kernel(const uint4 *__restrict__ x, size_t n_vec,
                                                   const uint16_t *__restrict__ tail, int n_tail,
                                                   unsigned int *__restrict__ amax_bits)
{
    amax_body(x, n_vec, tail, n_tail, amax_bits, blockIdx.x, gridDim.x);
}

// Several tensors in one launch (the operands of one layer): block b works on the tensor whose block range holds b.
constexpr int MULTI_MAX = 8;
struct MultiItem {
    const uint16_t *x;
    uint8_t *out;
    size_t n;
    int fmt;
    unsigned blk0;       // first block of this tensor
};
struct MultiArgs {
    MultiItem it[MULTI_MAX];
    int n_items;
    unsigned n_blocks;
    float *scalars;      // per tensor: amax, scale, 1 / scale
};

__global__ void __launch_bounds__(512) amax_multi_kernel(const MultiArgs a)
{
    int t = 0;
    while (t + 1 < a.n_items && blockIdx.x >= a.it[t + 1].blk0) ++t;
    const MultiItem &m = a.it[t];
    const unsigned nblk = (t + 1 < a.n_items ? a.it[t + 1].blk0 : a.n_blocks) - m.blk0;
    const size_t n_vec = m.n / 8;
    amax_body(reinterpret_cast<const uint4 *>(m.x), n_vec, m.x + n_vec * 8, (int)(m.n - n_vec * 8),
              reinterpret_cast<unsigned int *>(a.scalars + 3 * t), blockIdx.x - m.blk0, nblk);
}

// ---------------------------------------------------------------- scale
__device__ __forceinline__ float scale_from_amax(float a, float fp8_max, int margin)
{
    if (!(a > 0.0f) || isinf(a)) return 1.0f;
    const float s = __fmul_rn(__fdiv_rn(fp8_max, a), ldexpf(1.0f, -margin));   // power-of-two factor: exact
    return isinf(s) ? FLT_MAX : s;
}

__global__ void scale_kernel(const float *__restrict__ amax, float fp8_max, int margin, float *__restrict__ scale,
                             float *__restrict__ scale_inv)
{
    const float s = scale_from_amax(*amax, fp8_max, margin);
    *scale = s;
    *scale_inv = __fdiv_rn(1.0f, s);
}

// Where a cast takes its scale from.  Caller-supplied: `scale` is read.  Just-in-time (`amax` non-NULL): every
// thread derives the scale from the amax that the preceding pass left in memory (the arithmetic of scale_kernel)
// and the first thread of the grid publishes scale and 1/scale; no separate one-thread launch in between.
struct ScaleSrc {
    const float *scale;
    const float *amax;
    float fp8_max;
    float *scale_out, *scale_inv_out;
};
__device__ __forceinline__ float resolve_scale(const ScaleSrc &src, bool first_thread)
{
    if (!src.amax) return __ldg(src.scale);
    const float s = scale_from_amax(__ldg(src.amax), src.fp8_max, 0);
    if (first_thread) {
        *src.scale_out = s;
        *src.scale_inv_out = __fdiv_rn(1.0f, s);
    }
    return s;
}

// ---------------------------------------------------------------- delayed scaling: history ring update
// One CTA (256 threads): insert the new amax at the position of the oldest entry, then scale = FP8Max / (2^m max H).
__device__ __forceinline__ void ring_update_body(float *__restrict__ history, int len, int *__restrict__ head,
                                                 float amax_new, float fp8_max, int margin, float *__restrict__ scale,
                                                 float *__restrict__ scale_inv)
{
    __shared__ float warp_max[8];
    __shared__ int s_nan;
    if (threadIdx.x == 0) {
        const int h = *head;
        history[h] = amax_new;
        *head = (h + 1) % len;
        s_nan = 0;
    }
    __syncthreads();
    float m = 0.0f;
    for (int i = threadIdx.x; i < len; i += blockDim.x) {
        const float v = history[i];
        if (v != v) s_nan = 1;
        m = fmaxf(m, v);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w) m = fmaxf(m, warp_max[w]);
        float s;
        if (s_nan || !(m > 0.0f) || isinf(m)) {
            s = 1.0f;
        } else {
            s = __fmul_rn(__fdiv_rn(fp8_max, m), ldexpf(1.0f, -margin));
            if (isinf(s)) s = FLT_MAX;
        }
        *scale = s;
        *scale_inv = __fdiv_rn(1.0f, s);
    }
}

__global__ void __launch_bounds__(256) scale_update_kernel(float *__restrict__ history, int len, int *__restrict__ head,
                                                           const float *__restrict__ amax_new, float fp8_max,
                                                           int margin, float *__restrict__ scale,
                                                           float *__restrict__ scale_inv)
{
    ring_update_body(history, len, head, *amax_new, fp8_max, margin, scale, scale_inv);
}

// ---------------------------------------------------------------- cast
// 8 BF16 (one 16-byte word) -> 8 FP8 codes (two 32-bit words); each product is one binary32 multiply.
template <int FMT>
__device__ __forceinline__ uint2 cast8(const uint4 v, const float s)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint16_t h[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
        h[i] = cvt_f32x2_to_fp8x2<FMT>(__fmul_rn(bf16_lo(w[i]), s), __fmul_rn(bf16_hi(w[i]), s));
    return make_uint2((uint32_t)h[0] | ((uint32_t)h[1] << 16), (uint32_t)h[2] | ((uint32_t)h[3] << 16));
}

// The cast of one tensor as seen by block `rank` of the `nblk` blocks that share it.
template <int FMT, bool AMAX>
__device__ __forceinline__ void cast_flat_body(const uint4 *__restrict__ x, size_t n16, const uint16_t *__restrict__ tail_in,
                                               uint8_t *__restrict__ tail_out, int n_tail, const ScaleSrc &scale_src,
                                               uint4 *__restrict__ out, unsigned int *__restrict__ amax_bits, unsigned rank,
                                               unsigned nblk, float scale_value = -1.0f)
{
    // scale_value >= 0: the caller has the scale already (the delayed-scaling launch); scales are never negative
    const float s = scale_value >= 0.0f ? scale_value : resolve_scale(scale_src, rank == 0 && threadIdx.x == 0);
    uint32_t m = 0;
    const size_t stride = (size_t)nblk * blockDim.x;
    size_t i = (size_t)rank * blockDim.x + threadIdx.x;
    // Back to front: the amax pass that precedes a just-in-time cast walked the tensor front to back, so its
    // tail is what the L2 still holds.
    if (n16 > 0) {
        x += 2 * (n16 - 1);
        out += n16 - 1;
    }
    for (; i + stride < n16; i += 2 * stride) {
        const uint4 a0 = __ldg(x - 2 * i), a1 = __ldg(x - 2 * i + 1);
        const uint4 b0 = __ldg(x - 2 * (i + stride)), b1 = __ldg(x - 2 * (i + stride) + 1);
        if (AMAX) {
            m = absmax2(absmax2(absmax2(absmax2(m, a0.x), a0.y), a0.z), a0.w);
            m = absmax2(absmax2(absmax2(absmax2(m, a1.x), a1.y), a1.z), a1.w);
            m = absmax2(absmax2(absmax2(absmax2(m, b0.x), b0.y), b0.z), b0.w);
            m = absmax2(absmax2(absmax2(absmax2(m, b1.x), b1.y), b1.z), b1.w);
        }
        const uint2 p0 = cast8<FMT>(a0, s), p1 = cast8<FMT>(a1, s);
        const uint2 q0 = cast8<FMT>(b0, s), q1 = cast8<FMT>(b1, s);
        *(out - i) = make_uint4(p0.x, p0.y, p1.x, p1.y);
        *(out - (i + stride)) = make_uint4(q0.x, q0.y, q1.x, q1.y);
    }
    for (; i < n16; i += stride) {
        const uint4 a0 = __ldg(x - 2 * i), a1 = __ldg(x - 2 * i + 1);
        if (AMAX) {
            m = absmax2(absmax2(absmax2(absmax2(m, a0.x), a0.y), a0.z), a0.w);
            m = absmax2(absmax2(absmax2(absmax2(m, a1.x), a1.y), a1.z), a1.w);
        }
        const uint2 p0 = cast8<FMT>(a0, s), p1 = cast8<FMT>(a1, s);
        *(out - i) = make_uint4(p0.x, p0.y, p1.x, p1.y);
    }
    if (rank == 0 && (int)threadIdx.x < n_tail) {
        const uint32_t w = tail_in[threadIdx.x];
        if (AMAX) m = absmax2(m, w);
        const float p = __fmul_rn(bf16_lo(w), s);
        tail_out[threadIdx.x] = (uint8_t)(cvt_f32x2_to_fp8x2<FMT>(p, 0.0f) & 0xFF);
    }
    if (AMAX) block_atomic_max_bf16(m, amax_bits);
}

template <int FMT, bool AMAX>
__global__ void __launch_bounds__(256) cast_flat_kernel(const uint4 *__restrict__ x, size_t n16,
                                                        const uint16_t *__restrict__ tail_in,
                                                        uint8_t *__restrict__ tail_out, int n_tail,
                                                        const ScaleSrc scale_src,
                                                        uint4 *__restrict__ out, unsigned int *__restrict__ amax_bits)
{
    cast_flat_body<FMT, AMAX>(x, n16, tail_in, tail_out, n_tail, scale_src, out, amax_bits, blockIdx.x, gridDim.x);
}

// Just-in-time casts of several tensors in one launch: each takes its scale from the amax the reduction left in scalars.
__global__ void __launch_bounds__(256) cast_multi_kernel(const MultiArgs a)
{
    int t = 0;
    while (t + 1 < a.n_items && blockIdx.x >= a.it[t + 1].blk0) ++t;
    const MultiItem &m = a.it[t];
    const unsigned nblk = (t + 1 < a.n_items ? a.it[t + 1].blk0 : a.n_blocks) - m.blk0, rank = blockIdx.x - m.blk0;
    const size_t n16 = m.n / 16;
    const int n_tail = (int)(m.n - n16 * 16);
    float *sc = a.scalars + 3 * t;
    const ScaleSrc src{nullptr, sc, m.fmt == FP8_E4M3 ? 448.0f : 57344.0f, sc + 1, sc + 2};
    const uint4 *x = reinterpret_cast<const uint4 *>(m.x);
    if (m.fmt == FP8_E4M3)
        cast_flat_body<0, false>(x, n16, m.x + n16 * 16, m.out + n16 * 16, n_tail, src, reinterpret_cast<uint4 *>(m.out),
                                 nullptr, rank, nblk);
    else
        cast_flat_body<1, false>(x, n16, m.x + n16 * 16, m.out + n16 * 16, n_tail, src, reinterpret_cast<uint4 *>(m.out),
                                 nullptr, rank, nblk);
}

// Delayed scaling of several tensors in ONE launch: every tensor is cast under the scale its history gave after the
// previous step (*scale_next as the launch finds it; the first block also publishes it and its reciprocal for the
// products) while the same pass takes its amax; the last block of a tensor to finish (a counter per tensor) then does
// that tensor's ring update and leaves the scale of the next step in *scale_next.  sync[2 t] collects the amax bits, sync[2 t + 1]
// counts finished blocks; the last block leaves both at zero for the next call.
struct DelayedItem {
    const uint16_t *x;
    uint8_t *out;
    size_t n;
    int fmt;
    unsigned blk0;
    float *history;
    int *head;
    float *scale_next;                  // in: this step's scale; out (last block): the next step's
    float *amax, *scale, *scale_inv;    // out: amax(x); this step's scale and its reciprocal, for the products
};
struct DelayedArgs {
    DelayedItem it[MULTI_MAX];
    int n_items;
    unsigned n_blocks;
    int len, margin;
    unsigned int *sync;
};

__global__ void __launch_bounds__(256, 8) cast_delayed_multi_kernel(const DelayedArgs a)
{
    __shared__ int s_last;
    int t = 0;
    while (t + 1 < a.n_items && blockIdx.x >= a.it[t + 1].blk0) ++t;
    const DelayedItem &m = a.it[t];
    const unsigned nblk = (t + 1 < a.n_items ? a.it[t + 1].blk0 : a.n_blocks) - m.blk0, rank = blockIdx.x - m.blk0;
    const size_t n16 = m.n / 16;
    const int n_tail = (int)(m.n - n16 * 16);
    // A plain load, not the read-only path: the last block overwrites *scale_next at the end of this launch.  It does so
    // only after every block has counted in, and a block counts in after it has read the scale here.
    const float s = *reinterpret_cast<const volatile float *>(m.scale_next);
    if (rank == 0 && threadIdx.x == 0) {
        *m.scale = s;
        *m.scale_inv = __fdiv_rn(1.0f, s);
    }
    const ScaleSrc src{nullptr, nullptr, 0.0f, nullptr, nullptr};
    const uint4 *x = reinterpret_cast<const uint4 *>(m.x);
    unsigned int *acc = a.sync + 2 * t;
    if (m.fmt == FP8_E4M3)
        cast_flat_body<0, true>(x, n16, m.x + n16 * 16, m.out + n16 * 16, n_tail, src, reinterpret_cast<uint4 *>(m.out),
                                acc, rank, nblk, s);
    else
        cast_flat_body<1, true>(x, n16, m.x + n16 * 16, m.out + n16 * 16, n_tail, src, reinterpret_cast<uint4 *>(m.out),
                                acc, rank, nblk, s);
    // the block's atomic max was issued by thread 0 (if it had anything to add): make it visible, then count
    if (threadIdx.x == 0) {
        __threadfence();
        s_last = atomicAdd(acc + 1, 1u) == nblk - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __shared__ float s_amax;
    if (threadIdx.x == 0) {
        __threadfence();
        s_amax = __uint_as_float(atomicExch(acc, 0u));
        acc[1] = 0u;
        *m.amax = s_amax;
    }
    __syncthreads();
    __shared__ float s_unused_inv;
    ring_update_body(m.history, a.len, m.head, s_amax, m.fmt == FP8_E4M3 ? 448.0f : 57344.0f, a.margin, m.scale_next,
                     &s_unused_inv);
}

// Cast + transposed copy: one CTA per 128 x 128 tile.  Codes go straight to `out` (16-byte stores) and
// into a padded shared tile, which is then read column-wise so that `out_t` also gets 16-byte stores with
// two lanes covering each 32-byte sector.
constexpr int TT = 128;          // tile edge
constexpr int TPITCH = TT + 4;   // 33 words per row: column reads hit distinct banks

template <int FMT, bool AMAX>
__global__ void __launch_bounds__(256) cast_transpose_kernel(const uint16_t *__restrict__ x, int rows, int cols,
                                                             const ScaleSrc scale_src,
                                                             uint8_t *__restrict__ out, uint8_t *__restrict__ out_t,
                                                             unsigned int *__restrict__ amax_bits)
{
    __shared__ __align__(16) uint8_t tile[TT * TPITCH];
    const float s = resolve_scale(scale_src, blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0);
    // tiles are taken back to front (last rows first): after the amax pass of a just-in-time cast the tail of
    // the tensor is what the L2 still holds
    const int r0 = (int)(gridDim.y - 1 - blockIdx.y) * TT, c0 = (int)(gridDim.x - 1 - blockIdx.x) * TT;
    uint32_t m = 0;
    // phase 1: 128 rows x 8 groups of 16 columns
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int idx = it * 256 + threadIdx.x;
        const int r = idx >> 3, cg = idx & 7;
        const int gr = r0 + r, gc = c0 + cg * 16;
        if (gr < rows && gc < cols) {
            const uint4 *src = reinterpret_cast<const uint4 *>(x + (size_t)gr * cols + gc);
            const uint4 a0 = __ldg(src), a1 = __ldg(src + 1);
            if (AMAX) {
                m = absmax2(absmax2(absmax2(absmax2(m, a0.x), a0.y), a0.z), a0.w);
                m = absmax2(absmax2(absmax2(absmax2(m, a1.x), a1.y), a1.z), a1.w);
            }
            const uint2 p0 = cast8<FMT>(a0, s), p1 = cast8<FMT>(a1, s);
            if (out) *reinterpret_cast<uint4 *>(out + (size_t)gr * cols + gc) = make_uint4(p0.x, p0.y, p1.x, p1.y);
            uint32_t *t = reinterpret_cast<uint32_t *>(tile + r * TPITCH + cg * 16);
            t[0] = p0.x; t[1] = p0.y; t[2] = p1.x; t[3] = p1.y;
        }
    }
    __syncthreads();
    // phase 2: 128 columns x 8 groups of 16 rows; lanes (2k, 2k+1) write the two halves of one 32-byte sector
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int idx = it * 256 + threadIdx.x;
        const int half = idx & 1, c = (idx >> 1) & 127, rp = idx >> 8;   // rp: pair of row groups (0..3)
        const int rg = rp * 2 + half;
        const int gc = c0 + c, gr = r0 + rg * 16;
        if (gc < cols && gr < rows) {
            uint32_t w[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t v = 0;
#pragma unroll
                for (int b = 0; b < 4; ++b) v |= (uint32_t)tile[(rg * 16 + q * 4 + b) * TPITCH + c] << (8 * b);
                w[q] = v;
            }
            *reinterpret_cast<uint4 *>(out_t + (size_t)gc * rows + gr) = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
    if (AMAX) block_atomic_max_bf16(m, amax_bits);
}

static int validate_cast(const void *x, size_t rows, size_t cols, const float *scale, int fmt, uint8_t *out,
                         uint8_t *out_t)
{
    if (!x || !scale || (!out && !out_t)) {
        set_error("fp8_cast: NULL pointer (x=%p scale=%p out=%p out_t=%p)", x, (const void *)scale, (void *)out,
                  (void *)out_t);
        return FP8_ERR_NULL;
    }
    if (fmt != FP8_E4M3 && fmt != FP8_E5M2) {
        set_error("fp8_cast: fmt %d is not FP8_E4M3 / FP8_E5M2", fmt);
        return FP8_ERR_ENUM;
    }
    if (rows == 0 || cols == 0) {
        set_error("fp8_cast: empty tensor (rows=%zu cols=%zu)", rows, cols);
        return FP8_ERR_SHAPE;
    }
    if (!aligned16(x) || !aligned16(out) || !aligned16(out_t)) {
        set_error("fp8_cast: tensor pointers must be 16-byte aligned");
        return FP8_ERR_ALIGN;
    }
    if (out_t && (rows % 16 || cols % 16)) {
        set_error("fp8_cast: transposed copy needs rows %% 16 == 0 and cols %% 16 == 0 (rows=%zu cols=%zu)", rows, cols);
        return FP8_ERR_SHAPE;
    }
    if (!out_t && rows != 1 && cols % 16) {
        set_error("fp8_cast: cols %% 16 != 0 for a 2-D tensor (cols=%zu)", cols);
        return FP8_ERR_SHAPE;
    }
    if (rows > 0x7FFFFFFFull || cols > 0x7FFFFFFFull) {
        set_error("fp8_cast: rows/cols beyond 2^31-1");
        return FP8_ERR_SHAPE;
    }
    return FP8_OK;
}

template <int FMT, bool AMAX>
static void launch_cast(const void *x, size_t rows, size_t cols, const ScaleSrc &scale, uint8_t *out, uint8_t *out_t,
                        float *amax_out, cudaStream_t st)
{
    unsigned int *ab = reinterpret_cast<unsigned int *>(amax_out);
    if (out_t) {
        dim3 grid((unsigned)((cols + TT - 1) / TT), (unsigned)((rows + TT - 1) / TT));
        cast_transpose_kernel<FMT, AMAX><<<grid, 256, 0, st>>>(static_cast<const uint16_t *>(x), (int)rows, (int)cols,
                                                             scale, out, out_t, ab);
    } else {
        const size_t n = rows * cols, n16 = n / 16;
        const int n_tail = (int)(n - n16 * 16);
        size_t blocks = (n16 + 2 * 256 - 1) / (2 * 256);
        const size_t cap = (size_t)sm_count() * 8;
        if (blocks > cap) blocks = cap;
        if (blocks == 0) blocks = 1;
        cast_flat_kernel<FMT, AMAX><<<(unsigned)blocks, 256, 0, st>>>(
            static_cast<const uint4 *>(x), n16, static_cast<const uint16_t *>(x) + n16 * 16, out + n16 * 16, n_tail,
            scale, reinterpret_cast<uint4 *>(out), ab);
    }
}

static int do_amax(const void *x, size_t n, float *amax, cudaStream_t st)
{
    FP8_CUDA_CHECK(cudaMemsetAsync(amax, 0, sizeof(float), st));
    const size_t n_vec = n / 8;
    const int n_tail = (int)(n - n_vec * 8);
    size_t blocks = (n_vec + 4 * 512 - 1) / (4 * 512);
    const size_t cap = (size_t)sm_count() * 4;
    if (blocks > cap) blocks = cap;
    if (blocks == 0) blocks = 1;
    amax_kernel<<<(unsigned)blocks, 512, 0, st>>>(static_cast<const uint4 *>(x), n_vec,
                                                 static_cast<const uint16_t *>(x) + n_vec * 8, n_tail,
                                                 reinterpret_cast<unsigned int *>(amax));
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

static int do_cast(const void *x, size_t rows, size_t cols, const ScaleSrc &scale, int fmt, uint8_t *out,
                   uint8_t *out_t, float *amax_out, cudaStream_t st)
{
    if (amax_out) FP8_CUDA_CHECK(cudaMemsetAsync(amax_out, 0, sizeof(float), st));
    if (fmt == FP8_E4M3) {
        if (amax_out) launch_cast<0, true>(x, rows, cols, scale, out, out_t, amax_out, st);
        else launch_cast<0, false>(x, rows, cols, scale, out, out_t, amax_out, st);
    } else {
        if (amax_out) launch_cast<1, true>(x, rows, cols, scale, out, out_t, amax_out, st);
        else launch_cast<1, false>(x, rows, cols, scale, out, out_t, amax_out, st);
    }
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

}  // namespace fp8dpa

using namespace fp8dpa;

extern "C" int fp8_amax(const void *x_bf16, size_t n, float *amax, void *stream)
{
    if (!x_bf16 || !amax) {
        set_error("fp8_amax: NULL pointer");
        return FP8_ERR_NULL;
    }
    if (n == 0) {
        set_error("fp8_amax: n == 0");
        return FP8_ERR_SHAPE;
    }
    if (!aligned16(x_bf16)) {
        set_error("fp8_amax: x must be 16-byte aligned");
        return FP8_ERR_ALIGN;
    }
    int rc = check_arch();
    if (rc != FP8_OK) return rc;
    return do_amax(x_bf16, n, amax, static_cast<cudaStream_t>(stream));
}

extern "C" int fp8_scale(const float *amax, int fmt, int margin, float *scale, float *scale_inv, void *stream)
{
    if (!amax || !scale || !scale_inv) {
        set_error("fp8_scale: NULL pointer");
        return FP8_ERR_NULL;
    }
    if (fmt != FP8_E4M3 && fmt != FP8_E5M2) {
        set_error("fp8_scale: fmt %d is not FP8_E4M3 / FP8_E5M2", fmt);
        return FP8_ERR_ENUM;
    }
    if (margin < -64 || margin > 64) {
        set_error("fp8_scale: margin %d outside [-64, 64]", margin);
        return FP8_ERR_SHAPE;
    }
    int rc = check_arch();
    if (rc != FP8_OK) return rc;
    scale_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(amax, fmt == FP8_E4M3 ? 448.0f : 57344.0f, margin,
                                                                scale, scale_inv);
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

extern "C" int fp8_cast(const void *x_bf16, size_t rows, size_t cols, const float *scale, int fmt, uint8_t *out,
                        uint8_t *out_t, float *amax_out, void *stream)
{
    int rc = validate_cast(x_bf16, rows, cols, scale, fmt, out, out_t);
    if (rc != FP8_OK) return rc;
    rc = check_arch();
    if (rc != FP8_OK) return rc;
    const ScaleSrc src{scale, nullptr, 0.0f, nullptr, nullptr};
    return do_cast(x_bf16, rows, cols, src, fmt, out, out_t, amax_out, static_cast<cudaStream_t>(stream));
}

extern "C" int fp8_quantize(const void *x_bf16, size_t rows, size_t cols, int fmt, uint8_t *out, uint8_t *out_t,
                            float *amax, float *scale, float *scale_inv, void *stream)
{
    if (!amax || !scale || !scale_inv) {
        set_error("fp8_quantize: NULL amax/scale/scale_inv");
        return FP8_ERR_NULL;
    }
    int rc = validate_cast(x_bf16, rows, cols, scale, fmt, out, out_t);
    if (rc != FP8_OK) return rc;
    rc = check_arch();
    if (rc != FP8_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rc = do_amax(x_bf16, rows * cols, amax, st);
    if (rc != FP8_OK) return rc;
    const ScaleSrc src{nullptr, amax, fmt == FP8_E4M3 ? 448.0f : 57344.0f, scale, scale_inv};
    return do_cast(x_bf16, rows, cols, src, fmt, out, out_t, nullptr, st);
}

extern "C" int fp8_quantize_multi(const fp8_quant_item *items, int n_items, float *scalars, void *stream)
{
    if (!items || !scalars) {
        set_error("fp8_quantize_multi: NULL items / scalars");
        return FP8_ERR_NULL;
    }
    if (n_items < 1 || n_items > MULTI_MAX) {
        set_error("fp8_quantize_multi: n_items %d must be in [1, %d]", n_items, MULTI_MAX);
        return FP8_ERR_SHAPE;
    }
    MultiArgs am, ac;
    am.n_items = ac.n_items = n_items;
    am.scalars = ac.scalars = scalars;
    // the grids of the two passes: every tensor gets the blocks it would get alone, scaled down together at the cap
    size_t want_a[MULTI_MAX], want_c[MULTI_MAX], tot_a = 0, tot_c = 0;
    for (int t = 0; t < n_items; ++t) {
        const fp8_quant_item &q = items[t];
        if (!q.x_bf16 || !q.out) {
            set_error("fp8_quantize_multi: NULL pointer in item %d", t);
            return FP8_ERR_NULL;
        }
        if (q.fmt != FP8_E4M3 && q.fmt != FP8_E5M2) {
            set_error("fp8_quantize_multi: item %d: fmt %d is not FP8_E4M3 / FP8_E5M2", t, q.fmt);
            return FP8_ERR_ENUM;
        }
        if (q.n == 0) {
            set_error("fp8_quantize_multi: item %d is empty", t);
            return FP8_ERR_SHAPE;
        }
        if (!aligned16(q.x_bf16) || !aligned16(q.out)) {
            set_error("fp8_quantize_multi: tensor pointers must be 16-byte aligned (item %d)", t);
            return FP8_ERR_ALIGN;
        }
        am.it[t].x = ac.it[t].x = static_cast<const uint16_t *>(q.x_bf16);
        am.it[t].out = ac.it[t].out = q.out;
        am.it[t].n = ac.it[t].n = q.n;
        am.it[t].fmt = ac.it[t].fmt = q.fmt;
        want_a[t] = (q.n / 8 + 4 * 512 - 1) / (4 * 512);
        want_c[t] = (q.n / 16 + 2 * 256 - 1) / (2 * 256);
        if (want_a[t] == 0) want_a[t] = 1;
        if (want_c[t] == 0) want_c[t] = 1;
        tot_a += want_a[t];
        tot_c += want_c[t];
    }
    int rc = check_arch();
    if (rc != FP8_OK) return rc;
    const size_t cap_a = (size_t)sm_count() * 4, cap_c = (size_t)sm_count() * 8;
    unsigned ba = 0, bc = 0;
    for (int t = 0; t < n_items; ++t) {
        size_t na = tot_a > cap_a ? want_a[t] * cap_a / tot_a : want_a[t];
        size_t nc = tot_c > cap_c ? want_c[t] * cap_c / tot_c : want_c[t];
        if (na == 0) na = 1;
        if (nc == 0) nc = 1;
        am.it[t].blk0 = ba;
        ac.it[t].blk0 = bc;
        ba += (unsigned)na;
        bc += (unsigned)nc;
    }
    am.n_blocks = ba;
    ac.n_blocks = bc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    FP8_CUDA_CHECK(cudaMemsetAsync(scalars, 0, 3 * sizeof(float) * (size_t)n_items, st));
    amax_multi_kernel<<<ba, 512, 0, st>>>(am);
    FP8_CUDA_CHECK(cudaGetLastError());
    cast_multi_kernel<<<bc, 256, 0, st>>>(ac);
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

extern "C" int fp8_quantize_delayed_multi(const fp8_delayed_item *items, int n_items, int history_len, int margin,
                                          uint32_t *sync, void *stream)
{
    if (!items || !sync) {
        set_error("fp8_quantize_delayed_multi: NULL items / sync");
        return FP8_ERR_NULL;
    }
    if (n_items < 1 || n_items > MULTI_MAX) {
        set_error("fp8_quantize_delayed_multi: n_items %d must be in [1, %d]", n_items, MULTI_MAX);
        return FP8_ERR_SHAPE;
    }
    if (history_len <= 0 || history_len > (1 << 20) || margin < -64 || margin > 64) {
        set_error("fp8_quantize_delayed_multi: history_len %d must be in [1, 2^20] and margin %d in [-64, 64]",
                  history_len, margin);
        return FP8_ERR_SHAPE;
    }
    DelayedArgs a;
    a.n_items = n_items;
    a.len = history_len;
    a.margin = margin;
    a.sync = sync;
    size_t want[MULTI_MAX], tot = 0;
    for (int t = 0; t < n_items; ++t) {
        const fp8_delayed_item &q = items[t];
        if (!q.x_bf16 || !q.out || !q.history || !q.head || !q.scale_next || !q.amax || !q.scale || !q.scale_inv) {
            set_error("fp8_quantize_delayed_multi: NULL pointer in item %d", t);
            return FP8_ERR_NULL;
        }
        if (q.fmt != FP8_E4M3 && q.fmt != FP8_E5M2) {
            set_error("fp8_quantize_delayed_multi: item %d: fmt %d is not FP8_E4M3 / FP8_E5M2", t, q.fmt);
            return FP8_ERR_ENUM;
        }
        if (q.n == 0) {
            set_error("fp8_quantize_delayed_multi: item %d is empty", t);
            return FP8_ERR_SHAPE;
        }
        if (!aligned16(q.x_bf16) || !aligned16(q.out)) {
            set_error("fp8_quantize_delayed_multi: tensor pointers must be 16-byte aligned (item %d)", t);
            return FP8_ERR_ALIGN;
        }
        if (q.scale == q.scale_next || q.scale_inv == q.scale_next) {
            set_error("fp8_quantize_delayed_multi: item %d: scale / scale_inv must not alias scale_next", t);
            return FP8_ERR_SHAPE;
        }
        DelayedItem &d = a.it[t];
        d.x = static_cast<const uint16_t *>(q.x_bf16);
        d.out = q.out;
        d.n = q.n;
        d.fmt = q.fmt;
        d.history = q.history;
        d.head = q.head;
        d.scale_next = q.scale_next;
        d.amax = q.amax;
        d.scale = q.scale;
        d.scale_inv = q.scale_inv;
        want[t] = (q.n / 16 + 2 * 256 - 1) / (2 * 256);
        if (want[t] == 0) want[t] = 1;
        tot += want[t];
    }
    int rc = check_arch();
    if (rc != FP8_OK) return rc;
    const size_t cap = (size_t)sm_count() * 8;
    unsigned nb = 0;
    for (int t = 0; t < n_items; ++t) {
        size_t n = tot > cap ? want[t] * cap / tot : want[t];
        if (n == 0) n = 1;
        a.it[t].blk0 = nb;
        nb += (unsigned)n;
    }
    a.n_blocks = nb;
    cast_delayed_multi_kernel<<<nb, 256, 0, static_cast<cudaStream_t>(stream)>>>(a);
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

extern "C" int fp8_scale_update(float *history, int len, int *head, const float *amax_new, int fmt, int margin,
                                float *scale, float *scale_inv, void *stream)
{
    if (!history || !head || !amax_new || !scale || !scale_inv) {
        set_error("fp8_scale_update: NULL pointer");
        return FP8_ERR_NULL;
    }
    if (fmt != FP8_E4M3 && fmt != FP8_E5M2) {
        set_error("fp8_scale_update: fmt %d is not FP8_E4M3 / FP8_E5M2", fmt);
        return FP8_ERR_ENUM;
    }
    if (len <= 0 || len > (1 << 20) || margin < -64 || margin > 64) {
        set_error("fp8_scale_update: len %d must be in [1, 2^20] and margin %d in [-64, 64]", len, margin);
        return FP8_ERR_SHAPE;
    }
    int rc = check_arch();
    if (rc != FP8_OK) return rc;
    scale_update_kernel<<<1, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        history, len, head, amax_new, fmt == FP8_E4M3 ? 448.0f : 57344.0f, margin, scale, scale_inv);
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}
