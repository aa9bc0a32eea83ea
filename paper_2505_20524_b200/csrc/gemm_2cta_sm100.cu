// FP8 GEMM on CTA pairs (tcgen05.mma.cta_group::2): C[M,N] (+)= sa_inv*sb_inv * A[M,K] . B[N,K]^T
//
// Two CTAs of a cluster (ranks 0 and 1, neighbouring SMs) compute one 256 x 256 tile.  Each CTA loads its own
// 128 rows of A and its own 128 rows of B per stage (32 KB instead of the 48 KB a lone CTA needs for a
// 128 x 256 tile: the main loop is bound by the L2 -> shared-memory feed, so this is where the time goes); the
// MMA of shape 256 x 256 x 32 is issued by one thread of the even CTA, reads both CTAs' shared memory and writes
// 128 accumulator rows into each CTA's TMEM.  Accumulators are double-buffered (2 x 256 columns), so the epilogue
// of tile i overlaps the main loop of tile i+1.
//
// Barrier protocol (per CTA, same offsets in both):
//   full[s]   used in the even CTA only: its producer posts the byte count of both CTAs' loads; every load of the
//             pair credits the even CTA's barrier
//   empty[s]  one arrival per phase: the multicast commit of the MMAs that read stage s (lands in both CTAs)
//   tfull[b]  multicast commit after the last MMA of a tile (lands in both CTAs)
//   tempty[b] used in the even CTA only: 8 arrivals (4 epilogue warps of each CTA; the odd CTA arrives remotely)
// Every wait is bounded; a cluster barrier before exit keeps either CTA alive while its peer can still reach it.
#include <stdlib.h>
#include <string.h>

#include "common.cuh"
#include "gemm_epilogue.cuh"

namespace fp8dpa {

namespace g2 {

constexpr int BM = 128;            // rows per CTA (256 per pair)
constexpr int BN = 256;            // columns per pair; each CTA stages 128 rows of B
constexpr int BK = 128;
constexpr int STAGES = 6;
constexpr int THREADS = 192;
constexpr int A_BYTES = BM * BK, B_BYTES = (BN / 2) * BK;
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;              // 32 KB per CTA
constexpr int BAR_OFFSET = STAGES * STAGE_BYTES;
constexpr int N_BARS = 2 * STAGES + 4;
constexpr int DYN_BYTES = BAR_OFFSET + N_BARS * 8 + 16 + 1024;
constexpr uint32_t TMEM_COLS = 512;

struct Params {
    GemmOut o;
    const float *sa_inv, *sb_inv;
    int M, N, K;
    int a_mn, b_mn;                // operand stored with the output index contiguous ([K, M] / [K, N] in memory)
    uint32_t idesc;
    int num_pairs;
    int *status;
    // grouped form (mixture-of-experts FFN: the rows of A are sorted by expert, every expert has its own B):
    // group g owns rows [group_offsets[g], group_offsets[g+1]) of A and C, rows [g*N, (g+1)*N) of B and the
    // descale sb_inv[g]; the offsets live on the device (they come out of the router)
    const int *group_offsets;
    int n_groups;
    // Tile order of the plain form: bands of band_w tiles along the rows (band_on_m) or the columns of the output; inside
    // a band the other index advances slowest.  The operand of the banded dimension is then shared by consecutive
    // waves; where its band is sized to stay in L2 its loads carry evict_last and the other operand's evict_first
    // (hint_a / hint_b: 0 none, 1 evict_last, 2 evict_first).
    int band_w, band_on_m, hint_a, hint_b;
};
constexpr int MAX_GROUPS = 256;

__device__ __forceinline__ void tile_coords(const Params &p, int tile, int tiles_m, int tiles_n, int &tm, int &tn)
{
    if (p.band_on_m) band_coords_w(tile, tiles_m, tiles_n, p.band_w, tm, tn);
    else band_coords_w(tile, tiles_n, tiles_m, p.band_w, tn, tm);
}

// Tile -> (group, row offset of the group, rows of the group, tile coordinates inside the group) for the grouped form:
// tile_start[g] = first tile of group g (tiles of a group: ceil(rows / 256) x tiles_n, row tile fastest).
struct GroupTile { int g, row0, rows, tm, tn; };
__device__ __forceinline__ GroupTile group_tile(const int *tile_start, const int *offs, int n_groups, int tiles_n, int tile)
{
    int g = 0;
    while (g + 1 < n_groups && tile >= tile_start[g + 1]) ++g;
    const int local = tile - tile_start[g];
    const int rows = offs[g + 1] - offs[g];
    const int tiles_m = (rows + 2 * BM - 1) / (2 * BM);
    GroupTile t;
    t.g = g; t.row0 = offs[g]; t.rows = rows;
    t.tn = local / tiles_m;
    t.tm = local - t.tn * tiles_m;
    return t;
}

// MODE 0: one product.  MODE 1: grouped along the rows (forward / data gradient of the mixture-of-experts FFN).
// MODE 2: grouped along the reduction (its weight gradients): group g reduces over the rows [offs[g], offs[g+1]) of both
// operands (read in place, MN-major) into its own [M, N] output.  Every block of 128 reduction rows but a group's last comes
// from the operands themselves; the last one, which may be ragged, takes its A tile from a zero-padded copy of those rows
// (tmap_a_tail: [n_groups * 128, M], written by grouped_tail_kernel), so whatever rows of the next group the B tile
// carries meet zeros.  A group without rows reduces over one all-zero block.
template <int MODE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
gemm_fp8_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                     const __grid_constant__ CUtensorMap tmap_a_tail, const Params p)
{
    constexpr bool GROUPED = MODE == 1;
    constexpr bool GRED = MODE == 2;
    __shared__ int g_tile_start[GROUPED ? MAX_GROUPS + 1 : 1];
    __shared__ int g_offs[MODE != 0 ? MAX_GROUPS + 1 : 1];
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar_base = sbase + BAR_OFFSET;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
    auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + BAR_OFFSET + N_BARS * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();            // 0 = even CTA (issues the MMAs), 1 = its peer
    const int pair = blockIdx.x >> 1;
    const int tiles_m = (p.M + 2 * BM - 1) / (2 * BM), tiles_n = (p.N + BN - 1) / BN;
    int num_tiles = tiles_m * tiles_n;
    const int k_blocks = (p.K + BK - 1) / BK;
    if (GRED) {
        // the same clamping of the device-side offsets as below; the tiles do not depend on them
        if (threadIdx.x == 0) {
            int prev = min(max(__ldg(p.group_offsets), 0), p.K);
            for (int g = 0; g < p.n_groups; ++g) {
                g_offs[g] = prev;
                prev = min(max(__ldg(p.group_offsets + g + 1), prev), p.K);
            }
            g_offs[p.n_groups] = prev;
        }
        __syncthreads();
        num_tiles *= p.n_groups;
    }
    if (GROUPED) {
        // every CTA builds the same tile table from the device-side offsets
        if (threadIdx.x == 0) {
            // The offsets come from the router on the device and the host never sees them: force them into
            // 0 <= offs[0] <= offs[1] <= ... <= M, so that an array that breaks the contract gives wrong (clipped)
            // groups, never a store past the end of the output.
            int acc = 0, prev = min(max(__ldg(p.group_offsets), 0), p.M);
            for (int g = 0; g < p.n_groups; ++g) {
                const int o1 = min(max(__ldg(p.group_offsets + g + 1), prev), p.M);
                g_offs[g] = prev;
                g_tile_start[g] = acc;
                acc += ((o1 - prev + 2 * BM - 1) / (2 * BM)) * tiles_n;
                prev = o1;
            }
            g_offs[p.n_groups] = prev;
            g_tile_start[p.n_groups] = acc;
        }
        __syncthreads();
        num_tiles = g_tile_start[p.n_groups];
    }

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), 8);
        }
        *abort_flag = 0;
        mbar_init_fence();
        tma_prefetch_desc(&tmap_a);
        tma_prefetch_desc(&tmap_b);
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(tmem_slot), TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                  // both CTAs' barriers exist before anyone signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const WaitCtx ctx{p.status, abort_flag};

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (both CTAs)
        if (elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            const uint64_t pol_last = l2_policy_evict_last(), pol_first = l2_policy_evict_first();
            const uint64_t pol_a = p.hint_a == 1 ? pol_last : pol_first, pol_b = p.hint_b == 1 ? pol_last : pol_first;
            for (int tile = pair; tile < num_tiles && ok; tile += p.num_pairs) {
                int tm, tn, m_base = 0, n_base = 0, kb_base_b = 0, kbs = k_blocks, red0 = 0, g_red = 0;
                if (GRED) {
                    const int per = tiles_m * tiles_n, local = tile % per;
                    g_red = tile / per;
                    tn = local / tiles_m;
                    tm = local - tn * tiles_m;
                    red0 = g_offs[g_red];
                    kbs = max(1, (g_offs[g_red + 1] - red0 + BK - 1) / BK);
                } else if (GROUPED) {
                    const GroupTile gt = group_tile(g_tile_start, g_offs, p.n_groups, tiles_n, tile);
                    tm = gt.tm; tn = gt.tn;
                    m_base = gt.row0;              // rows of A: the group's slice of the sorted token matrix
                    // rows of B: the group's weight matrix -- its output rows (K-major B, forward) or its reduction
                    // rows (MN-major B: the stored [reduction, output] matrix of the data gradient)
                    if (p.b_mn) kb_base_b = gt.g * p.K;
                    else n_base = gt.g * p.N;
                } else {
                    tile_coords(p, tile, tiles_m, tiles_n, tm, tn);
                }
                const int m0 = m_base + tm * 2 * BM + (int)rank * BM, n0 = n_base + tn * BN + (int)rank * (BN / 2);
                for (int kb = 0; kb < kbs; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, ctx)) { ok = false; break; }
                    const uint32_t sa = sbase + stage * STAGE_BYTES, sb = sa + A_BYTES;
                    if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * STAGE_BYTES);
                    if (GRED) {
                        // both operands MN-major: [reduction rows, output index]
                        if (kb == kbs - 1) tma_load_2d_pair(sa, &tmap_a_tail, full_bar(stage), m0, g_red * BK);
                        else tma_load_2d_pair(sa, &tmap_a, full_bar(stage), m0, red0 + kb * BK);
                        tma_load_2d_pair(sb, &tmap_b, full_bar(stage), n0, red0 + kb * BK);
                        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                        continue;
                    }
                    // K-major tile: 128 rows of the output index x 128 reduction bytes; MN-major tile: 128 reduction
                    // rows x 128 bytes of the output index (the matrix as it lies in memory, no transposed copy)
                    const int a0 = p.a_mn ? m0 : kb * BK, a1 = p.a_mn ? kb * BK : m0;
                    const int b0 = p.b_mn ? n0 : kb * BK, b1 = p.b_mn ? kb_base_b + kb * BK : n0;
                    if (!GROUPED && p.hint_a) tma_load_2d_pair_hint(sa, &tmap_a, full_bar(stage), a0, a1, pol_a);
                    else tma_load_2d_pair(sa, &tmap_a, full_bar(stage), a0, a1);
                    if (!GROUPED && p.hint_b) tma_load_2d_pair_hint(sb, &tmap_b, full_bar(stage), b0, b1, pol_b);
                    else tma_load_2d_pair(sb, &tmap_b, full_bar(stage), b0, b1);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (even CTA only)
        if (rank == 0 && elect_one()) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int it = 0;
            for (int tile = pair; tile < num_tiles && ok; tile += p.num_pairs, ++it) {
                const int buf = it & 1;
                const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
                if (!mbar_wait(tempty_bar(buf), acc_phase ^ 1u, ctx)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(buf * BN);
                int kbs = k_blocks;
                if (GRED) {
                    const int g = tile / (tiles_m * tiles_n);
                    kbs = max(1, (g_offs[g + 1] - g_offs[g] + BK - 1) / BK);
                }
                for (int kb = 0; kb < kbs; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, ctx)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = sbase + stage * STAGE_BYTES, sb = sa + A_BYTES;
                    // 32 reduction elements per MMA: +32 bytes inside the swizzle span (K-major) or +32 rows of 128
                    // bytes (MN-major), in 16-byte units
                    const uint64_t da = p.a_mn ? umma_desc(sa, 128, 16) : umma_desc_k_sw128(sa);
                    const uint64_t db = p.b_mn ? umma_desc(sb, 128, 16) : umma_desc_k_sw128(sb);
                    const uint32_t step_a = p.a_mn ? (32u * 128u) >> 4 : 2u, step_b = p.b_mn ? (32u * 128u) >> 4 : 2u;
#pragma unroll
                    for (int k = 0; k < BK / 32; ++k)
                        umma_f8_ss_pair(tmem_d, da + step_a * k, db + step_b * k, p.idesc, (kb | k) != 0 ? 1u : 0u);
                    umma_commit_pair(empty_bar(stage), 3);      // frees the stage in both CTAs
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit_pair(tfull_bar(buf), 3);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5 of both CTAs)
        const int quad = warp & 3;
        const float descale = __ldg(p.sa_inv) * __ldg(p.sb_inv);
        const float q_scale = p.o.q_scale ? __ldg(p.o.q_scale) : 1.0f;
        uint32_t amax2 = 0;
        bool ok = true;
        int it = 0;
        for (int tile = pair; tile < num_tiles && ok; tile += p.num_pairs, ++it) {
            const int buf = it & 1;
            const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
            int tm, tn, m_base = 0, m_end = p.M, row_shift = 0;
            float descale_t = descale;
            if (GRED) {
                const int per = tiles_m * tiles_n, local = tile % per;
                tn = local / tiles_m;
                tm = local - tn * tiles_m;
                row_shift = (tile / per) * p.M;            // the group's [M, N] output follows the previous group's
            } else if (GROUPED) {
                const GroupTile gt = group_tile(g_tile_start, g_offs, p.n_groups, tiles_n, tile);
                tm = gt.tm; tn = gt.tn;
                m_base = gt.row0;
                m_end = gt.row0 + gt.rows;         // rows past the group's end belong to the next group: not stored
                descale_t = __ldg(p.sa_inv) * __ldg(p.sb_inv + gt.g);
            } else {
                tile_coords(p, tile, tiles_m, tiles_n, tm, tn);
            }
            const int m0 = m_base + tm * 2 * BM + (int)rank * BM, n0 = tn * BN;
            if (!mbar_wait_warp(tfull_bar(buf), acc_phase, ctx)) { ok = false; break; }
            tc_fence_after();
            const int row = m0 + quad * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * BN);
#pragma unroll 1
            for (int c = 0; c < BN; c += 32) {
                uint32_t r[32];
                tmem_ld_32x32b_x32(taddr + (uint32_t)c, r);
                tmem_ld_wait();
                const int col = n0 + c;
                if (row < m_end && col < p.N)
                    gemm_store_chunk(r, descale_t, p.o, q_scale, p.N, row_shift + row, col, min(32, p.N - col), amax2);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_pair_leader(tempty_bar(buf));   // the even CTA's barrier, from either CTA
        }
        gemm_publish_amax(p.o, amax2);
    }

    // ---------------------------------------------------------------- teardown
    __syncwarp();
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(20000);
        __syncthreads();
    }
    cluster_sync_all();             // neither CTA leaves (or frees TMEM) while its peer may still touch it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

}  // namespace g2

// Tile order and L2 priority of one product.  Every wave of 74 tiles streams its row panels and column panels
// (256 x K bytes each) once, in step along the reduction, so tiles of a wave share panels through L2 whatever their
// size; what matters is what the NEXT wave still finds.  One output dimension is cut into bands of w tiles, the other
// index advances slowest inside a band: consecutive waves then reuse the band's w panels and stream the others.
// w = as many panels as fit RESIDENT_BYTES (measured: the band survives a wave's streaming up to about 36 MB, well
// under the 126 MB of L2), but never under 8, since a wave of 8 x 9.25 tiles touches the fewest panels when nothing
// survives.  DRAM reads of the operands are then P * (n1 + ceil(n1 / w) * n2) for n1 banded tiles, n2 streamed ones
// and panel size P; the cheaper choice of the banded dimension wins.  The band's loads carry an evict_last policy
// (worth 0-10 % of the reads); evict_first on the streamed operand was measured and doubles the reads (tiles of a
// wave drift apart by more than such a line lives).  Measured on the 8B-class shapes (DRAM read MB, old order ->
// this one): 8192x28672x4096 350 -> 183, 8192x4096x28672 1217 -> 968, 28672x4096x8192 640 -> 328,
// 8192x4096x14336 583 -> 406, 4096x14336x8192 303 -> 172; durations equal within 2 % (the products are bound by the
// tensor pipe and board power, not by DRAM).  Small products (operands under FITS_BYTES) keep bands of 16 along the
// longer dimension.  FP8DPA_GEMM_ORDER=legacy keeps that form everywhere (for comparison; read per call).
static void choose_tile_order(g2::Params &p)
{
    using namespace g2;
    const int tiles_m = (p.M + 2 * BM - 1) / (2 * BM), tiles_n = (p.N + BN - 1) / BN;
    p.band_on_m = tiles_m >= tiles_n;
    p.band_w = GEMM_BAND;
    p.hint_a = p.hint_b = 0;
    const char *eo = getenv("FP8DPA_GEMM_ORDER");        // read per call: one process can compare the two orders
    const bool legacy = eo && !strcmp(eo, "legacy");
    const char *er = getenv("FP8DPA_GEMM_RESIDENT_MB");
    const double FITS_BYTES = 48e6, RESIDENT_BYTES = er ? atof(er) * 1e6 : 36e6;
    const double panel = 256.0 * p.K;
    if (legacy || ((double)p.M + p.N) * p.K <= FITS_BYTES) return;
    // at least 8 tiles wide: a wave of 74 tiles is then no longer than 8 x 9.25, the shape with the fewest panels
    const int wmax = (int)(RESIDENT_BYTES / panel) < 8 ? 8 : (int)(RESIDENT_BYTES / panel);
    double best = 0.0;
    for (int on_m = 0; on_m < 2; ++on_m) {
        const int n1 = on_m ? tiles_m : tiles_n, n2 = on_m ? tiles_n : tiles_m;
        const int w = wmax < n1 ? wmax : n1;
        const double reads = panel * (n1 + (double)((n1 + w - 1) / w) * n2);
        if (best == 0.0 || reads < best) {
            best = reads;
            p.band_on_m = on_m;
            p.band_w = w;
        }
    }
    const char *eh = getenv("FP8DPA_GEMM_HINTS");        // experiments: 0 none, 1 evict_last only, 2 both
    const int hint_mode = eh ? atoi(eh) : 1;
    const int resident = hint_mode >= 1 ? 1 : 0, streamed = hint_mode >= 2 ? 2 : 0;
    p.hint_a = p.band_on_m ? resident : streamed;
    p.hint_b = p.band_on_m ? streamed : resident;
}

// Returns FP8_OK after launching, or a negative status.  `max_pairs` = 0 lets the runtime size the grid.
int launch_gemm_2cta(const uint8_t *a, const uint8_t *b, const float *sa_inv, const float *sb_inv, const GemmOut &o,
                     int M, int N, int K, int a_mn, int b_mn, uint32_t idesc, int *status, cudaStream_t st)
{
    using namespace g2;
    CUtensorMap ta, tb;
    // an MN-major operand is the [K, M] (or [K, N]) matrix as stored: box = 128 reduction rows x 128 bytes
    int rc = a_mn ? make_tmap_2d_u8(&ta, a, (uint64_t)K, (uint64_t)M, (uint64_t)M, BK, BM)
                  : make_tmap_2d_u8(&ta, a, (uint64_t)M, (uint64_t)K, (uint64_t)K, BM, BK);
    if (rc != FP8_OK) return rc;
    rc = b_mn ? make_tmap_2d_u8(&tb, b, (uint64_t)K, (uint64_t)N, (uint64_t)N, BK, BN / 2)
              : make_tmap_2d_u8(&tb, b, (uint64_t)N, (uint64_t)K, (uint64_t)K, BN / 2, BK);
    if (rc != FP8_OK) return rc;
    FP8_CUDA_CHECK(cudaFuncSetAttribute(gemm_fp8_pair_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, DYN_BYTES));
    static int max_clusters = -1;
    if (max_clusters < 0) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * 74, 1, 1);
        cfg.blockDim = dim3(THREADS, 1, 1);
        cfg.dynamicSmemBytes = DYN_BYTES;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, gemm_fp8_pair_kernel<0>, &cfg) != cudaSuccess || n <= 0) {
            (void)cudaGetLastError();
            n = sm_count() / 2;
        }
        max_clusters = n;
    }
    const int tiles = ((M + 2 * BM - 1) / (2 * BM)) * ((N + BN - 1) / BN);
    Params p;
    p.o = o; p.sa_inv = sa_inv; p.sb_inv = sb_inv;
    p.M = M; p.N = N; p.K = K;
    p.a_mn = a_mn; p.b_mn = b_mn;
    p.idesc = idesc;
    p.num_pairs = tiles < max_clusters ? tiles : max_clusters;
    p.status = status;
    p.group_offsets = nullptr;
    p.n_groups = 0;
    choose_tile_order(p);
    gemm_fp8_pair_kernel<0><<<2 * p.num_pairs, THREADS, DYN_BYTES, st>>>(ta, tb, ta, p);
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

// Grouped form: Y[rows of group g] = sa_inv * sb_inv[g] * A[rows of group g] . B_g^T for every group, one launch.
int launch_gemm_2cta_grouped(const uint8_t *a, const uint8_t *b, const float *sa_inv, const float *sb_inv,
                             const int *group_offsets, int n_groups, const GemmOut &o, int M, int N, int K, int b_mn,
                             uint32_t idesc, int *status, cudaStream_t st)
{
    using namespace g2;
    CUtensorMap ta, tb;
    int rc = make_tmap_2d_u8(&ta, a, (uint64_t)M, (uint64_t)K, (uint64_t)K, BM, BK);
    if (rc != FP8_OK) return rc;
    // K-major B: the groups' [N, K] matrices back to back; MN-major B: their [K, N] matrices back to back (K here is the
    // reduction length of this product), 128 reduction rows x 128 bytes per box
    rc = b_mn ? make_tmap_2d_u8(&tb, b, (uint64_t)n_groups * K, (uint64_t)N, (uint64_t)N, BK, BN / 2)
              : make_tmap_2d_u8(&tb, b, (uint64_t)n_groups * N, (uint64_t)K, (uint64_t)K, BN / 2, BK);
    if (rc != FP8_OK) return rc;
    FP8_CUDA_CHECK(cudaFuncSetAttribute(gemm_fp8_pair_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, DYN_BYTES));
    // the host does not know the group sizes: at most ceil(M/256) + n_groups row tiles exist
    const long tiles_bound = ((long)(M + 2 * BM - 1) / (2 * BM) + n_groups) * ((N + BN - 1) / BN);
    const int pairs_max = sm_count() / 2;
    Params p;
    p.o = o; p.sa_inv = sa_inv; p.sb_inv = sb_inv;
    p.M = M; p.N = N; p.K = K;
    p.a_mn = 0; p.b_mn = b_mn;
    p.idesc = idesc;
    p.num_pairs = (int)(tiles_bound < pairs_max ? tiles_bound : pairs_max);
    p.status = status;
    p.group_offsets = group_offsets;
    p.n_groups = n_groups;
    p.band_w = GEMM_BAND; p.band_on_m = 1; p.hint_a = p.hint_b = 0;      // (the grouped form has its own tile table)
    gemm_fp8_pair_kernel<1><<<2 * p.num_pairs, THREADS, DYN_BYTES, st>>>(ta, tb, ta, p);
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

// Zero-padded copies of the last (possibly ragged) block of 128 reduction rows of every group: tail[g * 128 + i, :] =
// a[offs[g] + 128 * (blocks_g - 1) + i, :] for the rows of group g, zero beyond them (blocks_g = max(1, ceil(rows_g / 128))).
// The offsets are clamped like in the product kernel.  cols % 16 == 0.
__global__ void __launch_bounds__(256) grouped_tail_kernel(const uint8_t *__restrict__ a, const int *__restrict__ offs,
                                                           int n_rows, int cols, uint8_t *__restrict__ tail)
{
    const int g = blockIdx.x;
    int prev = min(max(__ldg(offs), 0), n_rows);
    for (int i = 0; i < g; ++i) prev = min(max(__ldg(offs + i + 1), prev), n_rows);
    const int r0 = prev, r1 = min(max(__ldg(offs + g + 1), prev), n_rows);
    const int rows = r1 - r0, blocks = max(1, (rows + 127) / 128);
    const int t0 = r0 + (blocks - 1) * 128, valid = rows - (blocks - 1) * 128;       // 0 .. 128 rows to copy
    const int vec = cols / 16;
    const long n = 128l * vec;
    for (long i = (long)blockIdx.y * blockDim.x + threadIdx.x; i < n; i += (long)gridDim.y * blockDim.x) {
        const int row = (int)(i / vec), cv = (int)(i - (long)row * vec);
        uint4 v = make_uint4(0, 0, 0, 0);
        if (row < valid) v = __ldg(reinterpret_cast<const uint4 *>(a + (size_t)(t0 + row) * cols) + cv);
        reinterpret_cast<uint4 *>(tail + ((size_t)g * 128 + row) * cols)[cv] = v;
    }
}

// Weight gradients of the grouped product in one launch: C[g] (+)= sa_inv * sb_inv * A[rows of g]^T . B[rows of g] for every
// group, A [T, M] and B [T, N] read in place, C [n_groups, M, N]; `tail` holds n_groups * 128 * M bytes of scratch.
int launch_gemm_2cta_grouped_red(const uint8_t *a, const uint8_t *b, const float *sa_inv, const float *sb_inv,
                                 const int *group_offsets, int n_groups, const GemmOut &o, int M, int N, int T,
                                 uint32_t idesc, uint8_t *tail, int *status, cudaStream_t st)
{
    using namespace g2;
    CUtensorMap ta, tb, tt;
    int rc = make_tmap_2d_u8(&ta, a, (uint64_t)T, (uint64_t)M, (uint64_t)M, BK, BM);
    if (rc != FP8_OK) return rc;
    rc = make_tmap_2d_u8(&tb, b, (uint64_t)T, (uint64_t)N, (uint64_t)N, BK, BN / 2);
    if (rc != FP8_OK) return rc;
    rc = make_tmap_2d_u8(&tt, tail, (uint64_t)n_groups * BK, (uint64_t)M, (uint64_t)M, BK, BM);
    if (rc != FP8_OK) return rc;
    dim3 tgrid((unsigned)n_groups, (unsigned)((128l * (M / 16) + 255) / 256 < 64 ? (128l * (M / 16) + 255) / 256 : 64));
    grouped_tail_kernel<<<tgrid, 256, 0, st>>>(a, group_offsets, T, M, tail);
    FP8_CUDA_CHECK(cudaGetLastError());
    FP8_CUDA_CHECK(cudaFuncSetAttribute(gemm_fp8_pair_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, DYN_BYTES));
    const long tiles = (long)n_groups * ((M + 2 * BM - 1) / (2 * BM)) * ((N + BN - 1) / BN);
    const int pairs_max = sm_count() / 2;
    Params p;
    p.o = o; p.sa_inv = sa_inv; p.sb_inv = sb_inv;
    p.M = M; p.N = N; p.K = T;
    p.a_mn = 1; p.b_mn = 1;
    p.idesc = idesc;
    p.num_pairs = (int)(tiles < pairs_max ? tiles : pairs_max);
    p.status = status;
    p.group_offsets = group_offsets;
    p.n_groups = n_groups;
    p.band_w = GEMM_BAND; p.band_on_m = 1; p.hint_a = p.hint_b = 0;
    gemm_fp8_pair_kernel<2><<<2 * p.num_pairs, THREADS, DYN_BYTES, st>>>(ta, tb, tt, p);
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

}  // namespace fp8dpa
