// FP8 x FP8 -> FP32-accumulate GEMM on the 5th-generation tensor cores (tcgen05.mma.kind::f8f6f4).
//
//   C[M,N] (+)= sa_inv * sb_inv * A[M,K] . B[N,K]^T        A, B: FP8 codes, reduction index contiguous
//
// One persistent CTA per SM walks over (128*MT) x BN output tiles.  Warp roles:
//   warp 0    TMA producer: 128-byte-swizzled [128 x 128 B] / [BN x 128 B] boxes into a 3- or 4-stage ring
//   warp 1    MMA issuer (one elected lane): 4 x MT x (128 x BN x 32) MMAs per stage, accumulators in TMEM
//             (MT = 1: two accumulator buffers, so the epilogue of tile i overlaps the main loop of tile i+1)
//   warps 2.. epilogue (4 per accumulator): tcgen05.ld -> descale -> BF16/FP32 -> 16-byte global stores
// Every wait is bounded; on expiry the CTA records FP8_ERR_TIMEOUT and drains.
#include <stdlib.h>

#include "common.cuh"
#include "gemm_epilogue.cuh"

namespace fp8dpa {

constexpr int G_BM = 128;         // rows of one accumulator (one UMMA M)
constexpr int G_BK = 128;         // bytes = FP8 elements per stage row (one swizzle span)

// MT = number of 128-row accumulators per CTA tile.
//   MT = 1: tile 128 x BN, 4 stages of (16 + BN/8) KB, two TMEM buffers -> epilogue overlaps the next main loop.
//   MT = 2: tile 256 x 256, 3 stages of 64 KB, both accumulators fill TMEM (512 columns).  Each byte of B feeds two
//           MMAs, so the CTA pulls 64 B/clk from L2 instead of 96 B/clk; the main loop is feed-bound, so this is
//           faster whenever there are enough tiles to fill the SMs.
template <int BN, int MT>
struct GemmCfg {
    static constexpr int STAGES = MT == 1 ? 4 : 3;
    static constexpr int NBUF = MT == 1 ? 2 : 1;
    static constexpr int EPI_WARPS = 4 * MT;
    static constexpr int THREADS = 64 + 32 * EPI_WARPS;
    static constexpr int TILE_M = G_BM * MT;
    static constexpr int A_BYTES = G_BM * G_BK;           // one 128-row A sub-tile
    static constexpr int B_BYTES = BN * G_BK;
    static constexpr int STAGE_BYTES = MT * A_BYTES + B_BYTES;
    static constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
    // full[S], empty[S], tmem_full[2], tmem_empty[2], tmem base slot, abort flag
    static constexpr int TOTAL = BAR_OFFSET + (2 * STAGES + 4) * 8 + 16;
    static constexpr int DYN_BYTES = TOTAL + 1024;        // slack for manual 1024-byte alignment
    static constexpr uint32_t TMEM_COLS = NBUF * MT * BN; // 256 or 512: a power of two >= 32
};

struct GemmParams {
    GemmOut o;
    const float *sa_inv, *sb_inv;
    int M, N, K;
    int a_mn, b_mn;                // operand stored with the output index contiguous (BN = 128, MT = 1 only)
    uint32_t idesc;
    int *status;
};

template <int TILE_M, int BN>
__device__ __forceinline__ void tile_coords(int tile, int tiles_m, int tiles_n, int &tm, int &tn)
{
    if (tiles_m * TILE_M >= tiles_n * BN) band_coords(tile, tiles_m, tiles_n, tm, tn);
    else band_coords(tile, tiles_n, tiles_m, tn, tm);
}

template <int BN, int MT>
__global__ void __launch_bounds__(GemmCfg<BN, MT>::THREADS, 1)
gemm_fp8_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                const GemmParams p)
{
    using L = GemmCfg<BN, MT>;
    constexpr int S = L::STAGES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar_base = sbase + L::BAR_OFFSET;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };
    auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * S + b); };
    auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * S + 2 + b); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + L::BAR_OFFSET + (2 * S + 4) * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_m = (p.M + L::TILE_M - 1) / L::TILE_M, tiles_n = (p.N + BN - 1) / BN;
    const int num_tiles = tiles_m * tiles_n;
    const int k_blocks = (p.K + G_BK - 1) / G_BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), L::EPI_WARPS);   // one arrival per epilogue warp
        }
        *abort_flag = 0;
        mbar_init_fence();
        tma_prefetch_desc(&tmap_a);
        tma_prefetch_desc(&tmap_b);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), L::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const WaitCtx ctx{p.status, abort_flag};

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                int tm, tn;
                tile_coords<L::TILE_M, BN>(tile, tiles_m, tiles_n, tm, tn);
                const int m0 = tm * L::TILE_M, n0 = tn * BN;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, ctx)) { ok = false; break; }
                    const uint32_t sa = sbase + stage * L::STAGE_BYTES, sb = sa + MT * L::A_BYTES;
                    mbar_expect_tx(full_bar(stage), L::STAGE_BYTES);
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) {
                        if (p.a_mn) tma_load_2d(sa + mt * L::A_BYTES, &tmap_a, full_bar(stage), m0 + mt * G_BM, kb * G_BK);
                        else tma_load_2d(sa + mt * L::A_BYTES, &tmap_a, full_bar(stage), kb * G_BK, m0 + mt * G_BM);
                    }
                    if (p.b_mn) tma_load_2d(sb, &tmap_b, full_bar(stage), n0, kb * G_BK);
                    else tma_load_2d(sb, &tmap_b, full_bar(stage), kb * G_BK, n0);
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int it = 0;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
                const int buf = it % L::NBUF;
                const uint32_t acc_phase = (uint32_t)(it / L::NBUF) & 1u;
                if (!mbar_wait(tempty_bar(buf), acc_phase ^ 1u, ctx)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(buf * MT * BN);
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, ctx)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = sbase + stage * L::STAGE_BYTES, sb = sa + MT * L::A_BYTES;
                    const uint64_t db = p.b_mn ? umma_desc(sb, 128, 16) : umma_desc_k_sw128(sb);
                    // 32 reduction elements per MMA: +32 bytes inside the swizzle span (K-major: +2 in 16-byte units)
                    // or +32 rows of 128 bytes (MN-major)
                    const uint32_t step_a = p.a_mn ? (32u * 128u) >> 4 : 2u, step_b = p.b_mn ? (32u * 128u) >> 4 : 2u;
#pragma unroll
                    for (int k = 0; k < G_BK / 32; ++k) {
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt) {
                            const uint32_t sam = sa + mt * L::A_BYTES;
                            const uint64_t da = p.a_mn ? umma_desc(sam, 128, 16) : umma_desc_k_sw128(sam);
                            umma_f8_ss(tmem_d + (uint32_t)(mt * BN), da + step_a * k, db + step_b * k, p.idesc,
                                       (kb | k) != 0 ? 1u : 0u);
                        }
                    }
                    umma_commit(empty_bar(stage));   // frees the stage once these MMAs have read it
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(tfull_bar(buf));
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int e = warp - 2;                        // 0 .. EPI_WARPS-1
        const int quad = warp & 3;                     // TMEM lanes 32*quad .. 32*quad+31
        const int mt = e >> 2;                         // which 128-row accumulator (MT = 2 only)
        const float descale = __ldg(p.sa_inv) * __ldg(p.sb_inv);
        const float q_scale = p.o.q_scale ? __ldg(p.o.q_scale) : 1.0f;
        uint32_t amax2 = 0;
        bool ok = true;
        int it = 0;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
            const int buf = it % L::NBUF;
            const uint32_t acc_phase = (uint32_t)(it / L::NBUF) & 1u;
            int tm, tn;
            tile_coords<L::TILE_M, BN>(tile, tiles_m, tiles_n, tm, tn);
            const int m0 = tm * L::TILE_M + mt * G_BM, n0 = tn * BN;
            if (!mbar_wait_warp(tfull_bar(buf), acc_phase, ctx)) { ok = false; break; }
            tc_fence_after();
            const int row = m0 + quad * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)((buf * MT + mt) * BN);
#pragma unroll 1
            for (int c = 0; c < BN; c += 32) {
                uint32_t r[32];
                tmem_ld_32x32b_x32(taddr + (uint32_t)c, r);
                tmem_ld_wait();
                const int col = n0 + c;
                if (row < p.M && col < p.N) {
                    // N is a multiple of 16, so a 32-column chunk is either whole or half inside
                    gemm_store_chunk(r, descale, p.o, q_scale, p.N, row, col, min(32, p.N - col), amax2);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(buf));
        }
        gemm_publish_amax(p.o, amax2);
    }

    // ---------------------------------------------------------------- teardown (all roles fall through)
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // a wait gave up: let copies that may still be in flight land before the CTA's memory is released
        for (int i = 0; i < 64; ++i) __nanosleep(20000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, L::TMEM_COLS);
    }
}

int launch_gemm_2cta(const uint8_t *a, const uint8_t *b, const float *sa_inv, const float *sb_inv, const GemmOut &o,
                     int M, int N, int K, int a_mn, int b_mn, uint32_t idesc, int *status, cudaStream_t st);

int launch_gemm_2cta_grouped(const uint8_t *a, const uint8_t *b, const float *sa_inv, const float *sb_inv,
                             const int *group_offsets, int n_groups, const GemmOut &o, int M, int N, int K, int b_mn,
                             uint32_t idesc, int *status, cudaStream_t st);
int launch_gemm_2cta_grouped_red(const uint8_t *a, const uint8_t *b, const float *sa_inv, const float *sb_inv,
                                 const int *group_offsets, int n_groups, const GemmOut &o, int M, int N, int T,
                                 uint32_t idesc, uint8_t *tail, int *status, cudaStream_t st);

// FP8DPA_GEMM=1cta|2cta forces one kernel family (for A/B measurements); default: chosen per shape.
static int gemm_family_override()
{
    const char *e = getenv("FP8DPA_GEMM");
    return !e ? 0 : (e[0] == '1' ? 1 : (e[0] == '2' ? 2 : 0));
}

static int validate_gemm(const char *who, const void *a, const void *b, const float *sa, const float *sb, void *out,
                         int M, int N, int K, bool any_reduce = false)
{
    if (!a || !b || !sa || !sb || !out) {
        set_error("%s: NULL pointer", who);
        return FP8_ERR_NULL;
    }
    // (with both operands read in place the reduction index counts rows, which the tensor maps zero-fill past the end)
    if (M <= 0 || N <= 0 || K <= 0 || (!any_reduce && (K % 16)) || (N % 16)) {
        set_error("%s: unsupported shape (rows=%d cols=%d reduce=%d; cols and reduce must be positive multiples of 16)",
                  who, M, N, K);
        return FP8_ERR_SHAPE;
    }
    if (!aligned16(a) || !aligned16(b) || !aligned16(out)) {
        set_error("%s: tensor pointers must be 16-byte aligned", who);
        return FP8_ERR_ALIGN;
    }
    return FP8_OK;
}

template <int BN, int MT>
static int launch_gemm(const uint8_t *a, const uint8_t *b, const GemmParams &p, cudaStream_t st)
{
    using L = GemmCfg<BN, MT>;
    CUtensorMap ta, tb;
    // an MN-major operand is the [K, M] (or [K, N]) matrix as stored: box = 128 reduction rows x 128 bytes
    int rc = p.a_mn ? make_tmap_2d_u8(&ta, a, (uint64_t)p.K, (uint64_t)p.M, (uint64_t)p.M, G_BK, G_BM)
                    : make_tmap_2d_u8(&ta, a, (uint64_t)p.M, (uint64_t)p.K, (uint64_t)p.K, G_BM, G_BK);
    if (rc != FP8_OK) return rc;
    rc = p.b_mn ? make_tmap_2d_u8(&tb, b, (uint64_t)p.K, (uint64_t)p.N, (uint64_t)p.N, G_BK, BN)
                : make_tmap_2d_u8(&tb, b, (uint64_t)p.N, (uint64_t)p.K, (uint64_t)p.K, BN, G_BK);
    if (rc != FP8_OK) return rc;
    FP8_CUDA_CHECK(cudaFuncSetAttribute(gemm_fp8_kernel<BN, MT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        L::DYN_BYTES));
    const int tiles = ((p.M + L::TILE_M - 1) / L::TILE_M) * ((p.N + BN - 1) / BN);
    const int grid = tiles < sm_count() ? tiles : sm_count();
    gemm_fp8_kernel<BN, MT><<<grid, L::THREADS, L::DYN_BYTES, st>>>(ta, tb, p);
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

// C[M,N] (+)= sa_inv*sb_inv * A[M,K] . B[N,K]^T
// a_mn / b_mn: that operand is given as the [K, M] (or [K, N]) matrix, i.e. the way the other two products of a
// linear layer store it, and is read in place as an MN-major UMMA operand: no transposed copy exists anywhere.
int gemm_fp8(const char *who, const uint8_t *a, int fmt_a, const uint8_t *b, int fmt_b, const float *sa_inv,
             const float *sb_inv, const GemmOut &o, int M, int N, int K, cudaStream_t st, int a_mn = 0, int b_mn = 0)
{
    int rc = validate_gemm(who, a, b, sa_inv, sb_inv, o.out, M, N, K, a_mn && b_mn);
    if (rc != FP8_OK) return rc;
    if (o.q_scale && o.q_fmt != FP8_E4M3 && o.q_fmt != FP8_E5M2) {
        set_error("%s: output format %d is not FP8_E4M3 / FP8_E5M2", who, o.q_fmt);
        return FP8_ERR_ENUM;
    }
    rc = check_arch();
    if (rc != FP8_OK) return rc;
    if (o.q_scale && o.amax_bits) FP8_CUDA_CHECK(cudaMemsetAsync(o.amax_bits, 0, sizeof(float), st));
    if ((a_mn && (M % 16)) || (b_mn && (N % 16))) {
        set_error("%s: an operand read in place needs its contiguous extent to be a multiple of 16 (rows=%d cols=%d)", who,
                  M, N);
        return FP8_ERR_SHAPE;
    }
    GemmParams p;
    p.a_mn = a_mn; p.b_mn = b_mn;
    p.o = o;
    p.sa_inv = sa_inv;
    p.sb_inv = sb_inv;
    p.M = M; p.N = N; p.K = K;
    p.status = device_status_ptr();
    if (!p.status) return FP8_ERR_CUDA;
    // CTA pairs (256 x 256 per pair, 32 KB per CTA and stage) whenever the matrix gives most pairs a tile: two
    // thirds of the L2 traffic of 128 x 256 tiles on single CTAs, and the epilogue still overlaps the next main loop.
    {
        const long pair_tiles = (long)((M + 255) / 256) * ((N + 255) / 256);
        const int fam = gemm_family_override();
        // (measured: from about three quarters of a wave of pairs upwards the pair kernel wins, e.g. 2048 x 2048 x
        // 8192 with 64 pair tiles: 27 us against 36 us; below that the smaller single-CTA tiles fill more SMs)
        if (fam != 1 && M >= 256 && N >= 256 && (fam == 2 || pair_tiles >= (3 * (sm_count() / 2)) / 4)) {
            return launch_gemm_2cta(a, b, sa_inv, sb_inv, o, M, N, K, a_mn, b_mn,
                                    umma_idesc_f8(fmt_a, fmt_b, 256, 256, a_mn, b_mn), p.status, st);
        }
    }
    // Tile choice.  The 256 x 256 tile needs 2/3 of the L2 traffic of 128 x 256 but cannot overlap its epilogue
    // with the next main loop (its two accumulators fill TMEM), so it only wins for long reductions (measured:
    // +3% at K = 8192, -15% at K = 2048) and when it still fills the SMs in whole waves.
    const int sms = sm_count();
    auto waves = [&](long tiles) { return (double)((tiles + sms - 1) / sms); };
    const long t256 = (long)((M + 255) / 256) * ((N + 255) / 256);
    const long t128x256 = (long)((M + 127) / 128) * ((N + 255) / 256);
    if (a_mn || b_mn) {
        // operands read in place: one 128-byte swizzle span per operand tile, i.e. the 128 x 128 tile
        p.idesc = umma_idesc_f8(fmt_a, fmt_b, G_BM, 128, a_mn, b_mn);
        return launch_gemm<128, 1>(a, b, p, st);
    }
    if (N >= 256 && M >= 256 && K >= 8192 && 2.0 * waves(t256) <= 1.02 * waves(t128x256)) {
        p.idesc = umma_idesc_f8(fmt_a, fmt_b, G_BM, 256);
        return launch_gemm<256, 2>(a, b, p, st);
    }
    if (N >= 256 && t128x256 >= sms) {
        p.idesc = umma_idesc_f8(fmt_a, fmt_b, G_BM, 256);
        return launch_gemm<256, 1>(a, b, p, st);
    }
    p.idesc = umma_idesc_f8(fmt_a, fmt_b, G_BM, 128);
    return launch_gemm<128, 1>(a, b, p, st);
}

}  // namespace fp8dpa

using namespace fp8dpa;

extern "C" int fp8_linear_fwd(const uint8_t *X8, const uint8_t *W8, const float *sX_inv, const float *sW_inv, void *Y,
                              int out_is_fp32, int T, int N, int K, void *ws, size_t ws_bytes, void *stream)
{
    (void)ws; (void)ws_bytes;
    const GemmOut o{Y, out_is_fp32, 0, nullptr, 0, nullptr};
    return gemm_fp8("fp8_linear_fwd", X8, FP8_E4M3, W8, FP8_E4M3, sX_inv, sW_inv, o, T, N, K,
                    static_cast<cudaStream_t>(stream));
}

extern "C" int fp8_linear_dgrad(const uint8_t *dY8, const uint8_t *W8t, const float *sdY_inv, const float *sW_inv,
                                void *dX, int out_is_fp32, int T, int N, int K, void *ws, size_t ws_bytes,
                                void *stream)
{
    (void)ws; (void)ws_bytes;
    // dX[T,K] = dY8[T,N] . W8t[K,N]^T : rows T, cols K, reduce N
    const GemmOut o{dX, out_is_fp32, 0, nullptr, 0, nullptr};
    return gemm_fp8("fp8_linear_dgrad", dY8, FP8_E5M2, W8t, FP8_E4M3, sdY_inv, sW_inv, o, T, K, N,
                    static_cast<cudaStream_t>(stream));
}

extern "C" int fp8_linear_wgrad(const uint8_t *dY8t, const uint8_t *X8t, const float *sdY_inv, const float *sX_inv,
                                void *dW, int out_is_fp32, int accumulate, int T, int N, int K, void *ws,
                                size_t ws_bytes, void *stream)
{
    (void)ws; (void)ws_bytes;
    // dW[N,K] = dY8t[N,T] . X8t[K,T]^T : rows N, cols K, reduce T
    const GemmOut o{dW, out_is_fp32, accumulate, nullptr, 0, nullptr};
    return gemm_fp8("fp8_linear_wgrad", dY8t, FP8_E5M2, X8t, FP8_E4M3, sdY_inv, sX_inv, o, N, K, T,
                    static_cast<cudaStream_t>(stream));
}

extern "C" int fp8_linear_fwd_q(const uint8_t *X8, const uint8_t *W8, const float *sX_inv, const float *sW_inv,
                                const float *y_scale, int y_fmt, uint8_t *Y8, float *y_amax, int T, int N, int K,
                                void *stream)
{
    if (!y_scale) {
        set_error("fp8_linear_fwd_q: NULL y_scale");
        return FP8_ERR_NULL;
    }
    const GemmOut o{Y8, 0, 0, y_scale, y_fmt, reinterpret_cast<unsigned int *>(y_amax)};
    return gemm_fp8("fp8_linear_fwd_q", X8, FP8_E4M3, W8, FP8_E4M3, sX_inv, sW_inv, o, T, N, K,
                    static_cast<cudaStream_t>(stream));
}

extern "C" int fp8_linear_dgrad_q(const uint8_t *dY8, const uint8_t *W8t, const float *sdY_inv, const float *sW_inv,
                                  const float *dx_scale, int dx_fmt, uint8_t *dX8, float *dx_amax, int T, int N, int K,
                                  void *stream)
{
    if (!dx_scale) {
        set_error("fp8_linear_dgrad_q: NULL dx_scale");
        return FP8_ERR_NULL;
    }
    const GemmOut o{dX8, 0, 0, dx_scale, dx_fmt, reinterpret_cast<unsigned int *>(dx_amax)};
    return gemm_fp8("fp8_linear_dgrad_q", dY8, FP8_E5M2, W8t, FP8_E4M3, sdY_inv, sW_inv, o, T, K, N,
                    static_cast<cudaStream_t>(stream));
}

// The same two gradients with every operand read in place, as stored for the forward product: W8 [N,K], dY8 [T,N],
// X8 [T,K].  No transposed FP8 copies are needed (tcgen05 takes FP8 operands with either index contiguous).
extern "C" int fp8_linear_dgrad_rm(const uint8_t *dY8, const uint8_t *W8, const float *sdY_inv, const float *sW_inv,
                                   void *dX, int out_is_fp32, int T, int N, int K, void *stream)
{
    // dX[T,K] = dY8[T,N] . W8[N,K] : rows T, cols K, reduce N; B = W8 is [reduce, cols] in memory
    const GemmOut o{dX, out_is_fp32, 0, nullptr, 0, nullptr};
    return gemm_fp8("fp8_linear_dgrad_rm", dY8, FP8_E5M2, W8, FP8_E4M3, sdY_inv, sW_inv, o, T, K, N,
                    static_cast<cudaStream_t>(stream), 0, 1);
}

extern "C" int fp8_linear_wgrad_rm(const uint8_t *dY8, const uint8_t *X8, const float *sdY_inv, const float *sX_inv,
                                   void *dW, int out_is_fp32, int accumulate, int T, int N, int K, void *stream)
{
    // dW[N,K] = dY8[T,N]^T . X8[T,K] : rows N, cols K, reduce T; both operands are [reduce, output] in memory
    const GemmOut o{dW, out_is_fp32, accumulate, nullptr, 0, nullptr};
    return gemm_fp8("fp8_linear_wgrad_rm", dY8, FP8_E5M2, X8, FP8_E4M3, sdY_inv, sX_inv, o, N, K, T,
                    static_cast<cudaStream_t>(stream), 1, 1);
}

// Grouped forward product for a mixture-of-experts FFN (Appendix D: 8 experts, 2 active): the token rows of X8 are
// sorted by expert, expert g owns rows [group_offsets[g], group_offsets[g+1]) and the weight matrix W8[g] ([N,K]) with
// its own scale.
extern "C" int fp8_grouped_linear_fwd(const uint8_t *X8, const uint8_t *W8, const float *sX_inv, const float *sW_inv,
                                      const int *group_offsets, int n_groups, void *Y, int out_is_fp32, int T, int N,
                                      int K, void *stream)
{
    if (!group_offsets) {
        set_error("fp8_grouped_linear_fwd: NULL group_offsets");
        return FP8_ERR_NULL;
    }
    if (n_groups <= 0 || n_groups > 256) {
        set_error("fp8_grouped_linear_fwd: n_groups %d must be in [1, 256]", n_groups);
        return FP8_ERR_SHAPE;
    }
    int rc = validate_gemm("fp8_grouped_linear_fwd", X8, W8, sX_inv, sW_inv, Y, T, N, K);
    if (rc != FP8_OK) return rc;
    rc = check_arch();
    if (rc != FP8_OK) return rc;
    int *status = device_status_ptr();
    if (!status) return FP8_ERR_CUDA;
    const GemmOut o{Y, out_is_fp32, 0, nullptr, 0, nullptr};
    return launch_gemm_2cta_grouped(X8, W8, sX_inv, sW_inv, group_offsets, n_groups, o, T, N, K, 0,
                                    umma_idesc_f8(FP8_E4M3, FP8_E4M3, 256, 256), status,
                                    static_cast<cudaStream_t>(stream));
}

extern "C" int fp8_grouped_linear_dgrad(const uint8_t *dY8, const uint8_t *W8, const float *sdY_inv, const float *sW_inv,
                                        const int *group_offsets, int n_groups, void *dX, int out_is_fp32, int T, int N,
                                        int K, void *stream)
{
    if (!group_offsets) {
        set_error("fp8_grouped_linear_dgrad: NULL group_offsets");
        return FP8_ERR_NULL;
    }
    if (n_groups <= 0 || n_groups > 256) {
        set_error("fp8_grouped_linear_dgrad: n_groups %d must be in [1, 256]", n_groups);
        return FP8_ERR_SHAPE;
    }
    if (N % 128 != 0) {
        // a reduction block of 128 rows must not reach into the next expert's weight matrix
        set_error("fp8_grouped_linear_dgrad: N = %d must be a multiple of 128", N);
        return FP8_ERR_SHAPE;
    }
    // dX[T,K] = dY8[T,N] . W8_g[N,K]: reduction length N, output width K
    int rc = validate_gemm("fp8_grouped_linear_dgrad", dY8, W8, sdY_inv, sW_inv, dX, T, K, N);
    if (rc != FP8_OK) return rc;
    rc = check_arch();
    if (rc != FP8_OK) return rc;
    int *status = device_status_ptr();
    if (!status) return FP8_ERR_CUDA;
    const GemmOut o{dX, out_is_fp32, 0, nullptr, 0, nullptr};
    return launch_gemm_2cta_grouped(dY8, W8, sdY_inv, sW_inv, group_offsets, n_groups, o, T, K, N, 1,
                                    umma_idesc_f8(FP8_E5M2, FP8_E4M3, 256, 256, 0, 1), status,
                                    static_cast<cudaStream_t>(stream));
}

// Weight gradients of the grouped product, dW[g] (+)= dY8[rows of g]^T . X8[rows of g]: one launch of the in-place
// weight-gradient product per expert on that expert's slice of rows (the reduction runs over the slice; rows past its
// end are zero-filled by the slice's tensor maps, so ragged groups need no padding).  The offsets are read on the host.
extern "C" int fp8_grouped_linear_wgrad(const uint8_t *dY8, const uint8_t *X8, const float *sdY_inv, const float *sX_inv,
                                        const int *group_offsets_host, int n_groups, void *dW, int out_is_fp32,
                                        int accumulate, int T, int N, int K, void *stream)
{
    if (!group_offsets_host || !dY8 || !X8 || !dW) {
        set_error("fp8_grouped_linear_wgrad: NULL pointer");
        return FP8_ERR_NULL;
    }
    if (n_groups <= 0 || n_groups > 256 || N <= 0 || K <= 0 || (N % 16) || (K % 16)) {
        set_error("fp8_grouped_linear_wgrad: n_groups %d must be in [1, 256], N %d and K %d positive multiples of 16", n_groups,
                  N, K);
        return FP8_ERR_SHAPE;
    }
    for (int g = 0; g < n_groups; ++g) {
        if (group_offsets_host[g] < 0 || group_offsets_host[g + 1] < group_offsets_host[g] || group_offsets_host[g + 1] > T) {
            set_error("fp8_grouped_linear_wgrad: group_offsets must ascend from >= 0 to <= T (entry %d)", g);
            return FP8_ERR_SHAPE;
        }
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t elt = out_is_fp32 ? 4 : 2;
    for (int g = 0; g < n_groups; ++g) {
        const int r0 = group_offsets_host[g], rows = group_offsets_host[g + 1] - r0;
        uint8_t *dw_g = static_cast<uint8_t *>(dW) + (size_t)g * N * K * elt;
        if (rows == 0) {                      // an expert without tokens: a zero gradient
            if (!accumulate) FP8_CUDA_CHECK(cudaMemsetAsync(dw_g, 0, (size_t)N * K * elt, st));
            continue;
        }
        const GemmOut o{dw_g, out_is_fp32, accumulate, nullptr, 0, nullptr};
        const int rc = gemm_fp8("fp8_grouped_linear_wgrad", dY8 + (size_t)r0 * N, FP8_E5M2, X8 + (size_t)r0 * K, FP8_E4M3,
                                sdY_inv, sX_inv, o, N, K, rows, st, 1, 1);
        if (rc != FP8_OK) return rc;
    }
    return FP8_OK;
}

// The same weight gradients in ONE launch with the offsets on the device (the router's output, as in the forward and the
// data gradient): the CTA-pair kernel walks (expert, output tile) and reduces over that expert's rows; the last, possibly
// ragged block of 128 rows of every expert is read from a zero-padded copy in `ws` (made by a small kernel first), so the
// rows of the next expert that share the block contribute nothing.
extern "C" size_t fp8_grouped_linear_wgrad_workspace_bytes(int n_groups, int N)
{
    if (n_groups <= 0 || N <= 0) return 0;
    return (size_t)n_groups * 128 * (size_t)N;
}

extern "C" int fp8_grouped_linear_wgrad_dev(const uint8_t *dY8, const uint8_t *X8, const float *sdY_inv,
                                            const float *sX_inv, const int *group_offsets, int n_groups, void *dW,
                                            int out_is_fp32, int accumulate, int T, int N, int K, void *ws, size_t ws_bytes,
                                            void *stream)
{
    if (!group_offsets || !dY8 || !X8 || !dW || !sdY_inv || !sX_inv) {
        set_error("fp8_grouped_linear_wgrad_dev: NULL pointer");
        return FP8_ERR_NULL;
    }
    if (n_groups <= 0 || n_groups > 256 || T <= 0 || N <= 0 || K <= 0 || (N % 16) || (K % 16)) {
        set_error("fp8_grouped_linear_wgrad_dev: n_groups %d must be in [1, 256], T %d positive, N %d and K %d positive "
                  "multiples of 16", n_groups, T, N, K);
        return FP8_ERR_SHAPE;
    }
    if (!aligned16(dY8) || !aligned16(X8) || !aligned16(dW)) {
        set_error("fp8_grouped_linear_wgrad_dev: tensor pointers must be 16-byte aligned");
        return FP8_ERR_ALIGN;
    }
    const size_t need = fp8_grouped_linear_wgrad_workspace_bytes(n_groups, N);
    if (!ws || ws_bytes < need || !aligned16(ws)) {
        set_error("fp8_grouped_linear_wgrad_dev: workspace must be 16-byte aligned and hold %zu bytes (got %zu)", need,
                  ws_bytes);
        return FP8_ERR_WORKSPACE;
    }
    int rc = check_arch();
    if (rc != FP8_OK) return rc;
    int *status = device_status_ptr();
    if (!status) return FP8_ERR_CUDA;
    const GemmOut o{dW, out_is_fp32, accumulate, nullptr, 0, nullptr};
    return launch_gemm_2cta_grouped_red(dY8, X8, sdY_inv, sX_inv, group_offsets, n_groups, o, N, K, T,
                                        umma_idesc_f8(FP8_E5M2, FP8_E4M3, 256, 256, 1, 1), static_cast<uint8_t *>(ws), status,
                                        static_cast<cudaStream_t>(stream));
}
