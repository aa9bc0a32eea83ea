// Fine-grained ("blockwise") FP8 scaling: the recipe the paper measures its tensor-wise recipe against (Section 2;
// Appendix E, "Fine-grained scaling recipes").  Activations carry one scale per 1 x 128 block, weights one per
// 128 x 128 block; the GEMM is then a sum over K-blocks of 128 of FP8 products that each need their own descale, so
// every K-block's partial accumulator leaves the tensor core and is folded into an FP32 running sum on the CUDA
// cores ("promotion").  That extra work per K-block is the overhead the paper reports for this recipe.
//
// Kernels: two single-pass quantisers (a block is small enough to stay on chip between its amax and its cast) and
//   gemm_blockwise_kernel: persistent, one CTA per SM, tile 128 x 128, K-block = one 128-byte swizzle span
//     warp 0  TMA: A (128 rows x 128 B) and B (128 rows x 128 B) per K-block, 6 stages
//     warp 1  MMA: 4 x tcgen05.mma (M128 N128 K32) per K-block into one of two 128-column TMEM buffers, the first
//             one overwriting; commit frees the stage and publishes the partial
//     warps 2-9  promotion: two threads per output row (warps w and w+4 share a TMEM lane group and take 64 columns
//             each); acc[64] (registers) += partial[c] * sx_inv[kb,row] * sw_inv[tile,kb], the TMEM load of the next
//             32 columns in flight during the FMAs; after the last K-block the row is written as BF16
#include <float.h>
#include <stdlib.h>
#include <string.h>

#include "common.cuh"
#include "gemm_epilogue.cuh"

namespace fp8dpa {
namespace bw {

__device__ __forceinline__ float block_scale_from_amax(float a, float fp8_max)
{
    if (!(a > 0.0f) || isinf(a)) return 1.0f;
    const float s = __fdiv_rn(fp8_max, a);
    return isinf(s) ? FLT_MAX : s;
}

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
__device__ __forceinline__ uint32_t amax8(uint32_t m, const uint4 v)
{
    return __vmaxu2(__vmaxu2(__vmaxu2(__vmaxu2(m, v.x & 0x7FFF7FFFu), v.y & 0x7FFF7FFFu), v.z & 0x7FFF7FFFu),
                    v.w & 0x7FFF7FFFu);
}

// 1 x 128 blocks: 16 lanes per block (16-byte loads), two blocks per warp; every thread takes BU blocks per sweep so
// that BU loads are in flight before the first shuffle.  scale_inv is written K-block-major, [C/128][R], which is the
// order the GEMM's promotion warps read it in (one row per lane).
constexpr int BU = 4;
// IDX: the type the block index is split into (row, column block) with; 32-bit division is several times cheaper than
// 64-bit, and with 16 bytes loaded per division it decides the kernel's speed (3.0-3.7 -> TB/s with 64-bit indices).
template <int FMT, typename IDX>
__global__ void __launch_bounds__(256) quantize_1x128_kernel(const uint16_t *__restrict__ x, size_t R, int C,
                                                             uint8_t *__restrict__ out, float *__restrict__ scale_inv)
{
    const IDX ncb = (IDX)(C / 128);
    const IDX n_blocks = (IDX)(R * (size_t)ncb);
    const int j = threadIdx.x & 15;
    const IDX step = (IDX)gridDim.x * (IDX)(16 * BU);
    // uniform trip count: the shuffles name every lane
    for (IDX base = (IDX)blockIdx.x * (IDX)(16 * BU); base < n_blocks; base += step) {
        uint4 v[BU];
        size_t off[BU], sidx[BU];
        bool valid[BU];
#pragma unroll
        for (int u = 0; u < BU; ++u) {
            const IDX b_raw = base + (IDX)(u * 16 + (threadIdx.x >> 4));
            valid[u] = b_raw < n_blocks;
            const IDX b = valid[u] ? b_raw : n_blocks - 1;
            const IDX r = b / ncb;
            const IDX cb = b - r * ncb;
            off[u] = (size_t)r * (size_t)C + (size_t)cb * 128 + j * 8;
            sidx[u] = (size_t)cb * R + r;
            v[u] = __ldg(reinterpret_cast<const uint4 *>(x + off[u]));
        }
#pragma unroll
        for (int u = 0; u < BU; ++u) {
            const uint32_t m2 = amax8(0u, v[u]);
            uint32_t m = max(m2 & 0xFFFFu, m2 >> 16);
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
            const float s = block_scale_from_amax(__uint_as_float(m << 16), FMT == 0 ? 448.0f : 57344.0f);
            if (valid[u]) {
                *reinterpret_cast<uint2 *>(out + off[u]) = cast8<FMT>(v[u], s);
                if (j == 0) scale_inv[sidx[u]] = __fdiv_rn(1.0f, s);
            }
        }
    }
}

// 128 x 128 blocks: one CTA per block, 8 groups of 8 elements per thread held in registers.  scale_inv: [R/128][C/128].
template <int FMT>
__global__ void __launch_bounds__(256) quantize_128x128_kernel(const uint16_t *__restrict__ x, int R, int C,
                                                               uint8_t *__restrict__ out, float *__restrict__ scale_inv)
{
    __shared__ uint32_t warp_max[8];
    const int r0 = blockIdx.y * 128, c0 = blockIdx.x * 128;
    uint4 v[8];
    uint32_t m2 = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int idx = k * 256 + threadIdx.x;
        const int r = r0 + (idx >> 4), c = c0 + (idx & 15) * 8;
        v[k] = make_uint4(0, 0, 0, 0);
        if (r < R) v[k] = __ldg(reinterpret_cast<const uint4 *>(x + (size_t)r * C + c));
        m2 = amax8(m2, v[k]);
    }
    uint32_t m = max(m2 & 0xFFFFu, m2 >> 16);
    m = __reduce_max_sync(0xffffffffu, m);
    if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < 8; ++w) m = max(m, warp_max[w]);
    const float s = block_scale_from_amax(__uint_as_float(m << 16), FMT == 0 ? 448.0f : 57344.0f);
    if (threadIdx.x == 0) scale_inv[(size_t)blockIdx.y * gridDim.x + blockIdx.x] = __fdiv_rn(1.0f, s);
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int idx = k * 256 + threadIdx.x;
        const int r = r0 + (idx >> 4), c = c0 + (idx & 15) * 8;
        if (r < R) *reinterpret_cast<uint2 *>(out + (size_t)r * C + c) = cast8<FMT>(v[k], s);
    }
}

// 128 x 1 blocks (128 consecutive rows of one column; the layout the weight-gradient product needs, whose reduction
// runs over the rows): one CTA per 128 x 128 tile as above, column maxima combined through shared memory.
// scale_inv: [ceil(R/128)][C].
template <int FMT>
__global__ void __launch_bounds__(256) quantize_128x1_kernel(const uint16_t *__restrict__ x, int R, int C,
                                                             uint8_t *__restrict__ out, float *__restrict__ scale_inv)
{
    __shared__ uint4 col_max[16][16];                 // [row group][column group]: packed maxima of 8 columns
    const int r0 = blockIdx.y * 128, c0 = blockIdx.x * 128;
    const int rg = threadIdx.x >> 4, cg = threadIdx.x & 15;
    uint4 v[8];
    uint4 m = make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int r = r0 + k * 16 + rg, c = c0 + cg * 8;
        v[k] = make_uint4(0, 0, 0, 0);
        if (r < R) v[k] = __ldg(reinterpret_cast<const uint4 *>(x + (size_t)r * C + c));
        m.x = __vmaxu2(m.x, v[k].x & 0x7FFF7FFFu);
        m.y = __vmaxu2(m.y, v[k].y & 0x7FFF7FFFu);
        m.z = __vmaxu2(m.z, v[k].z & 0x7FFF7FFFu);
        m.w = __vmaxu2(m.w, v[k].w & 0x7FFF7FFFu);
    }
    col_max[rg][cg] = m;
    __syncthreads();
#pragma unroll
    for (int g = 0; g < 16; ++g) {
        const uint4 o = col_max[g][cg];
        m.x = __vmaxu2(m.x, o.x); m.y = __vmaxu2(m.y, o.y); m.z = __vmaxu2(m.z, o.z); m.w = __vmaxu2(m.w, o.w);
    }
    const uint32_t mw[4] = {m.x, m.y, m.z, m.w};
    float sc[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        sc[2 * i] = block_scale_from_amax(__uint_as_float((mw[i] & 0xFFFFu) << 16), FMT == 0 ? 448.0f : 57344.0f);
        sc[2 * i + 1] = block_scale_from_amax(__uint_as_float(mw[i] & 0xFFFF0000u), FMT == 0 ? 448.0f : 57344.0f);
    }
    if (rg == 0) {
        float *dst = scale_inv + (size_t)blockIdx.y * C + c0 + cg * 8;
#pragma unroll
        for (int i = 0; i < 8; ++i) dst[i] = __fdiv_rn(1.0f, sc[i]);
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int r = r0 + k * 16 + rg, c = c0 + cg * 8;
        if (r < R) {
            const uint32_t w[4] = {v[k].x, v[k].y, v[k].z, v[k].w};
            uint16_t h[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                h[i] = cvt_f32x2_to_fp8x2<FMT>(__fmul_rn(bf16_lo(w[i]), sc[2 * i]), __fmul_rn(bf16_hi(w[i]), sc[2 * i + 1]));
            *reinterpret_cast<uint2 *>(out + (size_t)r * C + c) =
                make_uint2((uint32_t)h[0] | ((uint32_t)h[1] << 16), (uint32_t)h[2] | ((uint32_t)h[3] << 16));
        }
    }
}

// ------------------------------------------------------------------------------------------------ GEMM
constexpr int BM = 128, BN = 128, BK = 128;
constexpr int STAGES = 6;
constexpr int A_BYTES = BM * BK, B_BYTES = BN * BK, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
// full[S], empty[S], part_full[2], part_empty[2], tmem slot, abort flag
constexpr int TOTAL = BAR_OFFSET + (2 * STAGES + 4) * 8 + 16;
constexpr int DYN_BYTES = TOTAL + 1024;
constexpr int THREADS = 320;
constexpr uint32_t TMEM_COLS = 256;

// MODE_FWD    Y[t,n]  = sum_kb sx[kb][t] sw[n/128][kb] sum_{k in kb} X8[t,k] W8[n,k]      A, B reduction-contiguous
// MODE_DGRAD  dX[t,k] = sum_nb sdy[nb][t] sw[nb][k/128] sum_{n in nb} dY8[t,n] W8[n,k]    B = W8 read in place (MN-major)
// MODE_WGRAD  dW[n,k] = sum_tb sdy[tb][n] sx[tb][k] sum_{t in tb} dY8[t,n] X8[t,k]        A and B read in place (MN-major),
//             one descale per output row and one per output column for every block of 128 tokens
enum { MODE_FWD = 0, MODE_DGRAD = 1, MODE_WGRAD = 2 };
struct Params {
    uint16_t *out;                 // [M,N] BF16
    const float *sx_inv;           // row descales, [reduction blocks][M]
    const float *sw_inv;           // fwd: [ceil(N/128)][K/128]; dgrad: [K/128][ceil(N/128)] (the same array, read across);
                                   // wgrad: column descales [reduction blocks][N]
    int M, N, K;                   // output rows, output columns, reduction length
    int *status;
};

template <int MODE>
__global__ void __launch_bounds__(THREADS, 1)
gemm_blockwise_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                      const Params p)
{
    constexpr int S = STAGES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar_base = sbase + BAR_OFFSET;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };
    auto pfull_bar = [&](int b) { return bar_base + 8u * (2 * S + b); };
    auto pempty_bar = [&](int b) { return bar_base + 8u * (2 * S + 2 + b); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + BAR_OFFSET + (2 * S + 4) * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_m = (p.M + BM - 1) / BM, tiles_n = (p.N + BN - 1) / BN;
    const int num_tiles = tiles_m * tiles_n;
    const int k_blocks = (p.K + BK - 1) / BK;      // (the weight-gradient reduction over tokens may end ragged: zero-filled)

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(pfull_bar(b), 1);
            mbar_init(pempty_bar(b), 8);              // one arrival per promotion warp
        }
        *abort_flag = 0;
        mbar_init_fence();
        tma_prefetch_desc(&tmap_a);
        tma_prefetch_desc(&tmap_b);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const WaitCtx ctx{p.status, abort_flag};
    auto coords = [&](int tile, int &tm, int &tn) {
        if (tiles_m >= tiles_n) band_coords(tile, tiles_m, tiles_n, tm, tn);
        else band_coords(tile, tiles_n, tiles_m, tn, tm);
    };

    if (warp == 0) {
        if (elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                int tm, tn;
                coords(tile, tm, tn);
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, ctx)) { ok = false; break; }
                    const uint32_t sa = sbase + stage * STAGE_BYTES, sb = sa + A_BYTES;
                    mbar_expect_tx(full_bar(stage), STAGE_BYTES);
                    // an operand read in place has the reduction index as its row index
                    if (MODE == MODE_WGRAD) tma_load_2d(sa, &tmap_a, full_bar(stage), tm * BM, kb * BK);
                    else tma_load_2d(sa, &tmap_a, full_bar(stage), kb * BK, tm * BM);
                    if (MODE == MODE_FWD) tma_load_2d(sb, &tmap_b, full_bar(stage), kb * BK, tn * BN);
                    else tma_load_2d(sb, &tmap_b, full_bar(stage), tn * BN, kb * BK);
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (elect_one()) {
            constexpr int A_MN = MODE == MODE_WGRAD, B_MN = MODE != MODE_FWD;
            constexpr uint32_t idesc = umma_idesc_f8(MODE == MODE_FWD ? 0 : 1, 0, BM, BN, A_MN, B_MN);   // gradients: E5M2
            constexpr uint32_t STEP_K = 2u, STEP_MN = (32u * 128u) >> 4;      // descriptor advance per 32 reduction steps
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            uint32_t n = 0;                           // K-blocks issued so far (over all tiles): partial buffer n & 1
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                for (int kb = 0; kb < k_blocks; ++kb, ++n) {
                    const int buf = (int)(n & 1u);
                    if (!mbar_wait(pempty_bar(buf), ((n >> 1) & 1u) ^ 1u, ctx)) { ok = false; break; }
                    if (!mbar_wait(full_bar(stage), phase, ctx)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = sbase + stage * STAGE_BYTES, sb = sa + A_BYTES;
                    const uint64_t da = A_MN ? umma_desc(sa, 128, 16) : umma_desc_k_sw128(sa);
                    const uint64_t db = B_MN ? umma_desc(sb, 128, 16) : umma_desc_k_sw128(sb);
#pragma unroll
                    for (int k = 0; k < BK / 32; ++k)
                        umma_f8_ss(tmem_base + (uint32_t)(buf * BN), da + (A_MN ? STEP_MN : STEP_K) * k,
                                   db + (B_MN ? STEP_MN : STEP_K) * k, idesc, k != 0 ? 1u : 0u);
                    umma_commit(empty_bar(stage));
                    umma_commit(pfull_bar(buf));
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else {
        const int quad = warp & 3;
        const int half = (warp - 2) >> 2;              // which 64 of the tile's 128 columns
        constexpr int HC = BN / 2;
        const uint32_t lane_addr = ((uint32_t)(quad * 32) << 16) + (uint32_t)(half * HC);
        bool ok = true;
        uint32_t n = 0;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
            int tm, tn;
            coords(tile, tm, tn);
            const int row = tm * BM + quad * 32 + lane;
            const int n0 = tn * BN + half * HC;
            const float *sx = p.sx_inv + (row < p.M ? row : 0);
            const int tiles_n_all = (p.N + BN - 1) / BN;
            // weight-block descale of (this output tile, reduction block kb): consecutive along kb in the forward,
            // one row of the [K/128][N/128] array apart in the data gradient
            const float *sw = MODE == MODE_DGRAD ? p.sw_inv + tn : p.sw_inv + (size_t)tn * k_blocks;
            const size_t sw_step = MODE == MODE_DGRAD ? (size_t)tiles_n_all : 1;
            // weight gradient: column descales of this thread's 64 output columns, [reduction blocks][N]
            const float *scol = p.sw_inv + (n0 < p.N ? n0 : 0);
            // accumulators as packed pairs: the promotion is one fma.rn.f32x2 per two outputs and K-block (per lane an
            // ordinary FP32 FMA, so the result is the scalar one bit for bit), which halves its issue slots
            uint64_t acc2[HC / 2];
#pragma unroll
            for (int c = 0; c < HC / 2; ++c) acc2[c] = 0ull;
            // the two descale factors of a K-block are fetched PF K-blocks ahead: a global load per K-block on the
            // critical path would cost more than the K-block's MMAs
            constexpr int PF = 4;
            float sxq[PF], swq[PF];
#pragma unroll
            for (int i = 0; i < PF; ++i) {
                sxq[i] = i < k_blocks ? __ldg(sx + (size_t)i * p.M) : 0.0f;
                swq[i] = (MODE != MODE_WGRAD && i < k_blocks) ? __ldg(sw + (size_t)i * sw_step) : 1.0f;
            }
            for (int kb = 0; kb < k_blocks; ++kb, ++n) {
                const int buf = (int)(n & 1u);
                const float sc = sxq[0] * swq[0];
                const uint64_t sc2 = pack_f32x2(sc, sc);
#pragma unroll
                for (int i = 0; i + 1 < PF; ++i) { sxq[i] = sxq[i + 1]; swq[i] = swq[i + 1]; }
                sxq[PF - 1] = kb + PF < k_blocks ? __ldg(sx + (size_t)(kb + PF) * p.M) : 0.0f;
                swq[PF - 1] = (MODE != MODE_WGRAD && kb + PF < k_blocks) ? __ldg(sw + (size_t)(kb + PF) * sw_step) : 1.0f;
                if (!mbar_wait_warp(pfull_bar(buf), (n >> 1) & 1u, ctx)) { ok = false; break; }
                tc_fence_after();
                const uint32_t taddr = tmem_base + lane_addr + (uint32_t)(buf * BN);
                uint32_t r0[32], r1[32];
                tmem_ld_32x32b_x32(taddr, r0);
                tmem_ld_wait();
                tmem_ld_32x32b_x32(taddr + 32u, r1);           // in flight during the first 32 FMAs
                if (MODE == MODE_WGRAD) {
                    // every column has its own descale for this block of tokens (the same 64 values for all lanes)
                    const float4 *pc = reinterpret_cast<const float4 *>(scol + (size_t)kb * p.N);
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        const float4 c4 = (n0 + i < p.N) ? __ldg(pc + (i >> 2)) : make_float4(0.f, 0.f, 0.f, 0.f);
                        acc2[i >> 1] = fma_f32x2(mul_f32x2(pack_u32x2(r0[i], r0[i + 1]), pack_f32x2(c4.x, c4.y)), sc2, acc2[i >> 1]);
                        acc2[(i >> 1) + 1] = fma_f32x2(mul_f32x2(pack_u32x2(r0[i + 2], r0[i + 3]), pack_f32x2(c4.z, c4.w)), sc2, acc2[(i >> 1) + 1]);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; i += 2) acc2[i >> 1] = fma_f32x2(pack_u32x2(r0[i], r0[i + 1]), sc2, acc2[i >> 1]);
                }
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(pempty_bar(buf));   // the partial is in registers: the buffer is free
                if (MODE == MODE_WGRAD) {
                    const float4 *pc = reinterpret_cast<const float4 *>(scol + (size_t)kb * p.N + 32);
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        const float4 c4 = (n0 + 32 + i < p.N) ? __ldg(pc + (i >> 2)) : make_float4(0.f, 0.f, 0.f, 0.f);
                        acc2[16 + (i >> 1)] = fma_f32x2(mul_f32x2(pack_u32x2(r1[i], r1[i + 1]), pack_f32x2(c4.x, c4.y)), sc2, acc2[16 + (i >> 1)]);
                        acc2[17 + (i >> 1)] = fma_f32x2(mul_f32x2(pack_u32x2(r1[i + 2], r1[i + 3]), pack_f32x2(c4.z, c4.w)), sc2, acc2[17 + (i >> 1)]);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; i += 2) acc2[16 + (i >> 1)] = fma_f32x2(pack_u32x2(r1[i], r1[i + 1]), sc2, acc2[16 + (i >> 1)]);
                }
            }
            if (ok && row < p.M) {
                float acc[HC];
#pragma unroll
                for (int c = 0; c < HC / 2; ++c) unpack_f32x2(acc2[c], acc[2 * c], acc[2 * c + 1]);
                uint16_t *dst = p.out + (size_t)row * p.N + n0;
#pragma unroll
                for (int c = 0; c < HC; c += 8) {
                    if (n0 + c < p.N)      // N % 16 == 0: groups of 8 are whole
                        *reinterpret_cast<uint4 *>(dst + c) =
                            make_uint4(pack_bf16x2(acc[c], acc[c + 1]), pack_bf16x2(acc[c + 2], acc[c + 3]),
                                       pack_bf16x2(acc[c + 4], acc[c + 5]), pack_bf16x2(acc[c + 6], acc[c + 7]));
                }
            }
        }
    }

    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(20000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace bw

// the CTA-pair form of the same products (blockwise_2cta_sm100.cu)
int launch_blockwise_pair(int mode, const CUtensorMap &ta, const CUtensorMap &tb, const float *sa_inv, const float *sb_inv,
                          uint16_t *out, int M, int N, int Kred, int *status, cudaStream_t st);
}  // namespace fp8dpa

using namespace fp8dpa;

extern "C" int fp8_quantize_blockwise(const void *x_bf16, size_t rows, size_t cols, int block_rows, int fmt,
                                      uint8_t *out, float *scale_inv, void *stream)
{
    if (!x_bf16 || !out || !scale_inv) {
        set_error("fp8_quantize_blockwise: NULL pointer");
        return FP8_ERR_NULL;
    }
    if ((fmt != FP8_E4M3 && fmt != FP8_E5M2) || (block_rows != 1 && block_rows != 128 && block_rows != FP8_BLOCK_128x1)) {
        set_error("fp8_quantize_blockwise: fmt %d / block_rows %d not supported (E4M3 or E5M2; 1, 128 or FP8_BLOCK_128x1)", fmt,
                  block_rows);
        return FP8_ERR_ENUM;
    }
    if (rows == 0 || cols == 0 || (cols % 128) || rows > 0x7FFFFFFFull || cols > 0x7FFFFFFFull) {
        set_error("fp8_quantize_blockwise: unsupported shape rows=%zu cols=%zu (cols %% 128 == 0)", rows, cols);
        return FP8_ERR_SHAPE;
    }
    if (!aligned16(x_bf16) || !aligned16(out)) {
        set_error("fp8_quantize_blockwise: tensor pointers must be 16-byte aligned");
        return FP8_ERR_ALIGN;
    }
    int rc = check_arch();
    if (rc != FP8_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint16_t *x = static_cast<const uint16_t *>(x_bf16);
    if (block_rows == 1) {
        const size_t n_blocks = rows * (cols / 128);
        size_t blocks = (n_blocks + 16 * bw::BU - 1) / (16 * bw::BU);
        const size_t cap = (size_t)sm_count() * 16;
        if (blocks > cap) blocks = cap;
        // 32-bit block indices while they cannot wrap (block count plus one grid stride below 2^32)
        const bool small = n_blocks + blocks * 16 * bw::BU < 0xFFFFFFFFull;
        if (fmt == FP8_E4M3) {
            if (small) bw::quantize_1x128_kernel<0, uint32_t><<<(unsigned)blocks, 256, 0, st>>>(x, rows, (int)cols, out, scale_inv);
            else bw::quantize_1x128_kernel<0, size_t><<<(unsigned)blocks, 256, 0, st>>>(x, rows, (int)cols, out, scale_inv);
        } else {
            if (small) bw::quantize_1x128_kernel<1, uint32_t><<<(unsigned)blocks, 256, 0, st>>>(x, rows, (int)cols, out, scale_inv);
            else bw::quantize_1x128_kernel<1, size_t><<<(unsigned)blocks, 256, 0, st>>>(x, rows, (int)cols, out, scale_inv);
        }
    } else if (block_rows == FP8_BLOCK_128x1) {
        dim3 grid((unsigned)(cols / 128), (unsigned)((rows + 127) / 128));
        if (fmt == FP8_E4M3) bw::quantize_128x1_kernel<0><<<grid, 256, 0, st>>>(x, (int)rows, (int)cols, out, scale_inv);
        else bw::quantize_128x1_kernel<1><<<grid, 256, 0, st>>>(x, (int)rows, (int)cols, out, scale_inv);
    } else {
        dim3 grid((unsigned)(cols / 128), (unsigned)((rows + 127) / 128));
        if (fmt == FP8_E4M3) bw::quantize_128x128_kernel<0><<<grid, 256, 0, st>>>(x, (int)rows, (int)cols, out, scale_inv);
        else bw::quantize_128x128_kernel<1><<<grid, 256, 0, st>>>(x, (int)rows, (int)cols, out, scale_inv);
    }
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

static int launch_blockwise(const char *who, int mode, const uint8_t *A8, const uint8_t *B8, const float *sa_inv,
                            const float *sb_inv, void *out_bf16, int M, int N, int Kred, uint64_t a_rows, uint64_t a_cols,
                            uint64_t b_rows, uint64_t b_cols, void *stream)
{
    if (!A8 || !B8 || !sa_inv || !sb_inv || !out_bf16) {
        set_error("%s: NULL pointer", who);
        return FP8_ERR_NULL;
    }
    if (!aligned16(A8) || !aligned16(B8) || !aligned16(out_bf16) || !aligned16(sb_inv)) {
        set_error("%s: tensor pointers must be 16-byte aligned", who);
        return FP8_ERR_ALIGN;
    }
    int rc = check_arch();
    if (rc != FP8_OK) return rc;
    CUtensorMap ta, tb;
    // every operand tile is 128 rows of 128 bytes, whichever index its rows count
    rc = make_tmap_2d_u8(&ta, A8, a_rows, a_cols, a_cols, 128, 128);
    if (rc != FP8_OK) return rc;
    rc = make_tmap_2d_u8(&tb, B8, b_rows, b_cols, b_cols, 128, 128);
    if (rc != FP8_OK) return rc;
    bw::Params p;
    p.out = static_cast<uint16_t *>(out_bf16);
    p.sx_inv = sa_inv; p.sw_inv = sb_inv;
    p.M = M; p.N = N; p.K = Kred;
    p.status = device_status_ptr();
    if (!p.status) return FP8_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // 256 x 256 tiles on CTA pairs wherever the output has more than one 128 x 128 tile in both directions; the
    // single-CTA kernel for narrow outputs (FP8DPA_BLOCKWISE=1cta forces it, for comparison)
    static const bool force_1cta = [] {
        const char *e = getenv("FP8DPA_BLOCKWISE");
        return e && !strcmp(e, "1cta");
    }();
    if (!force_1cta && M > bw::BM && N > bw::BN)
        return launch_blockwise_pair(mode, ta, tb, sa_inv, sb_inv, p.out, M, N, Kred, p.status, st);
    const int tiles = ((M + bw::BM - 1) / bw::BM) * ((N + bw::BN - 1) / bw::BN);
    const int grid = tiles < sm_count() ? tiles : sm_count();
#define FP8DPA_LAUNCH_BW(MODE) \
    do { \
        FP8_CUDA_CHECK(cudaFuncSetAttribute(bw::gemm_blockwise_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                            bw::DYN_BYTES)); \
        bw::gemm_blockwise_kernel<MODE><<<grid, bw::THREADS, bw::DYN_BYTES, st>>>(ta, tb, p); \
    } while (0)
    if (mode == bw::MODE_FWD) FP8DPA_LAUNCH_BW(bw::MODE_FWD);
    else if (mode == bw::MODE_DGRAD) FP8DPA_LAUNCH_BW(bw::MODE_DGRAD);
    else FP8DPA_LAUNCH_BW(bw::MODE_WGRAD);
#undef FP8DPA_LAUNCH_BW
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

extern "C" int fp8_linear_fwd_blockwise(const uint8_t *X8, const uint8_t *W8, const float *sx_inv, const float *sw_inv,
                                        void *Y_bf16, int T, int N, int K, void *stream)
{
    if (T <= 0 || N <= 0 || K <= 0 || (K % 128) || (N % 16)) {
        set_error("fp8_linear_fwd_blockwise: unsupported shape T=%d N=%d K=%d (K %% 128 == 0, N %% 16 == 0)", T, N, K);
        return FP8_ERR_SHAPE;
    }
    return launch_blockwise("fp8_linear_fwd_blockwise", bw::MODE_FWD, X8, W8, sx_inv, sw_inv, Y_bf16, T, N, K,
                            (uint64_t)T, (uint64_t)K, (uint64_t)N, (uint64_t)K, stream);
}

extern "C" int fp8_linear_dgrad_blockwise(const uint8_t *dY8, const uint8_t *W8, const float *sdy_inv,
                                          const float *sw_inv, void *dX_bf16, int T, int N, int K, void *stream)
{
    if (T <= 0 || N <= 0 || K <= 0 || (N % 128) || (K % 128)) {
        set_error("fp8_linear_dgrad_blockwise: unsupported shape T=%d N=%d K=%d (N %% 128 == 0, K %% 128 == 0)", T, N, K);
        return FP8_ERR_SHAPE;
    }
    // output [T, K], reduction over N: A = dY8 [T, N] as stored, B = W8 [N, K] read in place
    return launch_blockwise("fp8_linear_dgrad_blockwise", bw::MODE_DGRAD, dY8, W8, sdy_inv, sw_inv, dX_bf16, T, K, N,
                            (uint64_t)T, (uint64_t)N, (uint64_t)N, (uint64_t)K, stream);
}

extern "C" int fp8_linear_wgrad_blockwise(const uint8_t *dY8, const uint8_t *X8, const float *sdy_inv_t,
                                          const float *sx_inv_t, void *dW_bf16, int T, int N, int K, void *stream)
{
    if (T <= 0 || N <= 0 || K <= 0 || (N % 16) || (K % 16)) {
        set_error("fp8_linear_wgrad_blockwise: unsupported shape T=%d N=%d K=%d (N %% 16 == 0, K %% 16 == 0)", T, N, K);
        return FP8_ERR_SHAPE;
    }
    // output [N, K], reduction over T: A = dY8 [T, N] and B = X8 [T, K], both read in place
    return launch_blockwise("fp8_linear_wgrad_blockwise", bw::MODE_WGRAD, dY8, X8, sdy_inv_t, sx_inv_t, dW_bf16, N, K, T,
                            (uint64_t)T, (uint64_t)N, (uint64_t)T, (uint64_t)K, stream);
}
