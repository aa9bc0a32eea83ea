// Blockwise-scaled FP8 products on CTA pairs (the comparison recipe of Section 2 / Appendix E, "Fine-grained scaling
// recipes"): the same arithmetic as the single-CTA kernel of blockwise_sm100.cu, on 256 x 256 tiles.
//
// A 128 x 128 tile with one 128-byte block of the reduction per stage needs 32 KB of operands for 4 MMAs: the lone CTA
// is bound by the L2 -> shared-memory feed long before the promotion costs anything.  Two CTAs of a cluster compute a
// 256 x 256 tile with tcgen05.mma.cta_group::2 (each loads its own 128 rows of A and 128 rows of B per stage: the same
// 32 KB, four times the work per pair).  Every block of the reduction is issued as two products of 128 output columns
// (64 rows of either CTA's B tile), each overwriting one of four 128-column TMEM buffers; sixteen promotion warps per
// CTA (four lane quads x four groups of 64 columns) fold a buffer into packed FP32 accumulators with that block's
// descale factors and release it while the tensor core fills the others.
//
//   warp 0      TMA (both CTAs): A box and B box per stage, credited to the even CTA's barrier
//   warp 1      MMA (even CTA): waits for the stage and, per half, for the buffer's release by the 16 promotion warps of the
//               pair that read it; 2 x 4 x M256 N128 K32, multicast commits publish each half and free the stage
//   warps 2-17  promotion: tcgen05.ld in chunks of 8 columns (the next one in flight under the FMAs of this one),
//               fma.rn.f32x2 into 32 packed accumulators, release of the buffer as soon as the partial is in
//               registers; BF16 stores after the last block
// Every wait is bounded; a cluster barrier before exit keeps either CTA alive while its peer can still reach it.
#include "common.cuh"
#include "gemm_epilogue.cuh"

namespace fp8dpa {
namespace bw2 {

constexpr int BM = 128;            // rows per CTA (256 per pair)
constexpr int BN = 256;            // columns per pair; each CTA stages 128 rows of B
constexpr int BK = 128;
constexpr int STAGES = 6;
constexpr int PROMO_WARPS = 16;
constexpr int THREADS = 64 + PROMO_WARPS * 32;
constexpr int QC = BN / 4;         // columns per promotion thread
constexpr int A_BYTES = BM * BK, B_BYTES = (BN / 2) * BK, STAGE_BYTES = A_BYTES + B_BYTES;
// weight gradient: the 256 column descales of every reduction block travel through a ring of their own (1 KB per
// slot).  A slot is rewritten SC_SLOTS blocks later; the producer runs at most STAGES blocks ahead of the MMAs and
// the MMAs at most two blocks ahead of the promotion warps' last read, so SC_SLOTS >= STAGES + 3 keeps a slot intact
// while it is read.
constexpr int SC_SLOTS = 12, SC_BYTES = BN * 4;
constexpr int SC_OFFSET = STAGES * STAGE_BYTES;
constexpr int BAR_OFFSET = SC_OFFSET + SC_SLOTS * SC_BYTES;
constexpr int N_BARS = 2 * STAGES + 8 + SC_SLOTS;      // full[S], empty[S], pfull[4], pempty[4], sfull[SC_SLOTS]
constexpr int DYN_BYTES = BAR_OFFSET + N_BARS * 8 + 16 + 1024;
constexpr uint32_t TMEM_COLS = 512;

enum { MODE_FWD = 0, MODE_DGRAD = 1, MODE_WGRAD = 2 };      // as in blockwise_sm100.cu
struct Params {
    uint16_t *out;                 // [M,N] BF16
    const float *sx_inv;           // row descales, [reduction blocks][M]
    const float *sw_inv;           // fwd: [ceil(N/128)][K/128]; dgrad: [K/128][ceil(N/128)]; wgrad: column descales [blocks][N]
    int M, N, K;                   // output rows, output columns, reduction length
    int num_pairs;
    int *status;
};

// acc2[C0/2 ..] += partial[C0 .. C0+8) * descale: one packed FMA per two outputs (per lane an ordinary binary32 FMA).
// Weight gradient: every output column has its own descale for this block of tokens (scol points at column 0's).
template <int MODE, int C0>
__device__ __forceinline__ void fold8(uint64_t (&acc2)[QC / 2], const uint32_t (&r)[8], uint64_t sc2, const float *scol,
                                      bool cols_valid)
{
    if (MODE == MODE_WGRAD) {
        if (!cols_valid) return;
#pragma unroll
        for (int i = 0; i < 8; i += 4) {
            const float4 c4 = *reinterpret_cast<const float4 *>(scol + C0 + i);      // shared memory, the same address in every lane
            acc2[(C0 + i) >> 1] = fma_f32x2(mul_f32x2(pack_u32x2(r[i], r[i + 1]), pack_f32x2(c4.x, c4.y)), sc2, acc2[(C0 + i) >> 1]);
            acc2[((C0 + i) >> 1) + 1] =
                fma_f32x2(mul_f32x2(pack_u32x2(r[i + 2], r[i + 3]), pack_f32x2(c4.z, c4.w)), sc2, acc2[((C0 + i) >> 1) + 1]);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; i += 2) acc2[(C0 + i) >> 1] = fma_f32x2(pack_u32x2(r[i], r[i + 1]), sc2, acc2[(C0 + i) >> 1]);
    }
}

template <int MODE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
gemm_blockwise_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                           const Params p)
{
    constexpr int S = STAGES;
    constexpr int A_MN = MODE == MODE_WGRAD, B_MN = MODE != MODE_FWD;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar_base = sbase + BAR_OFFSET;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (S + s); };
    // partial buffers: index 2 * (block parity) + column half
    auto pfull_bar = [&](int b) { return bar_base + 8u * (2 * S + b); };
    auto pempty_bar = [&](int b) { return bar_base + 8u * (2 * S + 4 + b); };
    auto sfull_bar = [&](int i) { return bar_base + 8u * (2 * S + 8 + i); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + BAR_OFFSET + N_BARS * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();            // 0 = even CTA (issues the MMAs), 1 = its peer
    const int pair = blockIdx.x >> 1;
    const int tiles_m = (p.M + 2 * BM - 1) / (2 * BM), tiles_n = (p.N + BN - 1) / BN;
    const int num_tiles = tiles_m * tiles_n;
    const int k_blocks = (p.K + BK - 1) / BK;           // the weight gradient's reduction over tokens may end ragged: zero-filled

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 4; ++b) {
            mbar_init(pfull_bar(b), 1);
            mbar_init(pempty_bar(b), PROMO_WARPS);         // used in the even CTA: the 8 + 8 promotion warps of that half
        }
        for (int i = 0; i < SC_SLOTS; ++i) mbar_init(sfull_bar(i), 1);
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
    auto coords = [&](int tile, int &tm, int &tn) {
        if (tiles_m >= tiles_n) band_coords(tile, tiles_m, tiles_n, tm, tn);
        else band_coords(tile, tiles_n, tiles_m, tn, tm);
    };

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (both CTAs)
        if (elect_one()) {
            int stage = 0, slot = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += p.num_pairs) {
                int tm, tn;
                coords(tile, tm, tn);
                const int m0 = tm * 2 * BM + (int)rank * BM, n0 = tn * BN + (int)rank * (BN / 2);
                const uint32_t sc_bytes = (uint32_t)min(BN, p.N - tn * BN) * 4u;     // N % 16 == 0: a multiple of 64 bytes
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, ctx)) { ok = false; break; }
                    if (MODE == MODE_WGRAD) {
                        // this CTA's copy of the tile's column descales for this block of tokens
                        mbar_expect_tx(sfull_bar(slot), sc_bytes);
                        bulk_load_1d(sbase + SC_OFFSET + slot * SC_BYTES, p.sw_inv + (size_t)kb * p.N + tn * BN, sc_bytes,
                                     sfull_bar(slot));
                        if (++slot == SC_SLOTS) slot = 0;
                    }
                    const uint32_t sa = sbase + stage * STAGE_BYTES, sb = sa + A_BYTES;
                    if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * STAGE_BYTES);
                    // an operand read in place has the reduction index as its row index
                    if (A_MN) tma_load_2d_pair(sa, &tmap_a, full_bar(stage), m0, kb * BK);
                    else tma_load_2d_pair(sa, &tmap_a, full_bar(stage), kb * BK, m0);
                    if (B_MN) tma_load_2d_pair(sb, &tmap_b, full_bar(stage), n0, kb * BK);
                    else tma_load_2d_pair(sb, &tmap_b, full_bar(stage), kb * BK, n0);
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (even CTA only)
        if (rank == 0 && elect_one()) {
            constexpr uint32_t idesc = umma_idesc_f8(MODE == MODE_FWD ? 0 : 1, 0, 2 * BM, BN / 2, A_MN, B_MN);   // gradients: E5M2
            constexpr uint32_t STEP_K = 2u, STEP_MN = (32u * 128u) >> 4;      // descriptor advance per 32 reduction steps
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            uint32_t n = 0;                           // reduction blocks issued so far (over all tiles): buffer n & 1
            for (int tile = pair; tile < num_tiles && ok; tile += p.num_pairs) {
                for (int kb = 0; kb < k_blocks; ++kb, ++n) {
                    const int buf = (int)(n & 1u);
                    if (!mbar_wait(full_bar(stage), phase, ctx)) { ok = false; break; }
                    const uint32_t sa = sbase + stage * STAGE_BYTES, sb = sa + A_BYTES;
                    const uint64_t da = A_MN ? umma_desc(sa, 128, 16) : umma_desc_k_sw128(sa);
                    const uint64_t db = B_MN ? umma_desc(sb, 128, 16) : umma_desc_k_sw128(sb);
                    // Two products of 128 output columns each (64 rows of either CTA's B tile), published and released
                    // separately: four partial buffers are in flight instead of two, which is what hides the
                    // MMA -> promotion -> MMA round trip of a buffer behind the tensor core's own time.
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (!mbar_wait(pempty_bar(2 * buf + h), ((n >> 1) & 1u) ^ 1u, ctx)) { ok = false; break; }
                        tc_fence_after();
                        // 64 rows of a K-major tile are 64 x 128 bytes on; 64 output columns of an MN-major tile are 64
                        // bytes on inside the swizzled row (16-byte units)
                        const uint64_t dbh = db + (uint64_t)(h * (B_MN ? (64 >> 4) : ((64 * 128) >> 4)));
#pragma unroll
                        for (int k = 0; k < BK / 32; ++k)
                            umma_f8_ss_pair(tmem_base + (uint32_t)(buf * BN + h * (BN / 2)), da + (A_MN ? STEP_MN : STEP_K) * k,
                                            dbh + (B_MN ? STEP_MN : STEP_K) * k, idesc, k != 0 ? 1u : 0u);
                        umma_commit_pair(pfull_bar(2 * buf + h), 3);    // this half of the partial is complete in both CTAs' TMEM
                    }
                    if (!ok) break;
                    umma_commit_pair(empty_bar(stage), 3);      // frees the stage in both CTAs
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else {
        // ------------------------------------------------------------ promotion (warps 2..17 of both CTAs)
        const int quad = warp & 3;                     // TMEM lanes 32*quad..: output rows of this warp
        const int cq = (warp - 2) >> 2;                // which 64 of the buffer's 256 TMEM columns
        const int half = cq >> 1;                      // the product (column half of the buffer) they belong to
        // a product of 128 columns takes 64 from either CTA's B tile: TMEM columns 128*half + 64*j hold the tile's columns
        // 128*j + 64*half
        const int col_in_tile = (cq & 1) * (BN / 2) + half * QC;
        const uint32_t lane_addr = ((uint32_t)(quad * 32) << 16) + (uint32_t)(cq * QC);
        const int wblocks = (p.N + 127) / 128;         // 128-wide weight blocks along the output columns
        bool ok = true;
        uint32_t n = 0;
        for (int tile = pair; tile < num_tiles && ok; tile += p.num_pairs) {
            int tm, tn;
            coords(tile, tm, tn);
            const int row = tm * 2 * BM + (int)rank * BM + quad * 32 + lane;
            const int n0 = tn * BN + col_in_tile;
            const float *sx = p.sx_inv + (row < p.M ? row : 0);
            // weight-block descale of (this thread's columns, reduction block kb): consecutive along kb in the forward,
            // one row of the [K/128][N/128] array apart in the data gradient
            const int wb = min(tn * 2 + (cq & 1), wblocks - 1);
            const float *sw = MODE == MODE_DGRAD ? p.sw_inv + wb : p.sw_inv + (size_t)wb * k_blocks;
            const size_t sw_step = MODE == MODE_DGRAD ? (size_t)wblocks : 1;
            uint64_t acc2[QC / 2];
#pragma unroll
            for (int c = 0; c < QC / 2; ++c) acc2[c] = 0ull;
            // the descale factors of a block are fetched PF blocks ahead: a global load per block on the critical
            // path would cost more than the block's MMAs
            constexpr int PF = 2;
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
                const int slot = (int)(n % (uint32_t)SC_SLOTS);
                const float *sck = reinterpret_cast<const float *>(smem + SC_OFFSET + slot * SC_BYTES) + col_in_tile;
                if (MODE == MODE_WGRAD && !mbar_wait_warp(sfull_bar(slot), (n / (uint32_t)SC_SLOTS) & 1u, ctx)) { ok = false; break; }
                if (!mbar_wait_warp(pfull_bar(2 * buf + half), (n >> 1) & 1u, ctx)) { ok = false; break; }
                tc_fence_after();
                const uint32_t taddr = tmem_base + lane_addr + (uint32_t)(buf * BN);
                // chunks of 8 columns, the next one in flight during the FMAs of this one (measured against 16-column
                // chunks, single or double: those need more than the 96 registers that 18 warps leave each thread)
                uint32_t ra[8], rb[8];
                const bool v0 = n0 < p.N, v1 = n0 + 16 < p.N, v2 = n0 + 32 < p.N, v3 = n0 + 48 < p.N;   // N % 16 == 0
                tmem_ld_32x32b_x8(taddr, ra);
                tmem_ld_wait();
                tmem_ld_32x32b_x8(taddr + 8u, rb);
                fold8<MODE, 0>(acc2, ra, sc2, sck, v0);
                tmem_ld_wait();
                tmem_ld_32x32b_x8(taddr + 16u, ra);
                fold8<MODE, 8>(acc2, rb, sc2, sck, v0);
                tmem_ld_wait();
                tmem_ld_32x32b_x8(taddr + 24u, rb);
                fold8<MODE, 16>(acc2, ra, sc2, sck, v1);
                tmem_ld_wait();
                tmem_ld_32x32b_x8(taddr + 32u, ra);
                fold8<MODE, 24>(acc2, rb, sc2, sck, v1);
                tmem_ld_wait();
                tmem_ld_32x32b_x8(taddr + 40u, rb);
                fold8<MODE, 32>(acc2, ra, sc2, sck, v2);
                tmem_ld_wait();
                tmem_ld_32x32b_x8(taddr + 48u, ra);
                fold8<MODE, 40>(acc2, rb, sc2, sck, v2);
                tmem_ld_wait();
                tmem_ld_32x32b_x8(taddr + 56u, rb);
                fold8<MODE, 48>(acc2, ra, sc2, sck, v3);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_pair_leader(pempty_bar(2 * buf + half));   // in registers: this half-buffer is free
                fold8<MODE, 56>(acc2, rb, sc2, sck, v3);
            }
            if (ok && row < p.M) {
                uint16_t *dst = p.out + (size_t)row * p.N + n0;
#pragma unroll
                for (int c = 0; c < QC; c += 8) {
                    if (n0 + c < p.N) {      // N % 16 == 0: groups of 8 are whole
                        float a[8];
#pragma unroll
                        for (int i = 0; i < 4; ++i) unpack_f32x2(acc2[(c >> 1) + i], a[2 * i], a[2 * i + 1]);
                        *reinterpret_cast<uint4 *>(dst + c) = make_uint4(pack_bf16x2(a[0], a[1]), pack_bf16x2(a[2], a[3]),
                                                                         pack_bf16x2(a[4], a[5]), pack_bf16x2(a[6], a[7]));
                    }
                }
            }
        }
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

}  // namespace bw2

// Launches the pair kernel; the tensor maps are the single-CTA kernel's (every box is 128 rows of 128 bytes).
int launch_blockwise_pair(int mode, const CUtensorMap &ta, const CUtensorMap &tb, const float *sa_inv, const float *sb_inv,
                          uint16_t *out, int M, int N, int Kred, int *status, cudaStream_t st)
{
    using namespace bw2;
    Params p;
    p.out = out;
    p.sx_inv = sa_inv; p.sw_inv = sb_inv;
    p.M = M; p.N = N; p.K = Kred;
    p.status = status;
    const int tiles = ((M + 2 * BM - 1) / (2 * BM)) * ((N + BN - 1) / BN);
    const int max_clusters = sm_count() / 2;
    p.num_pairs = tiles < max_clusters ? tiles : max_clusters;
#define FP8DPA_LAUNCH_BW2(MODE) \
    do { \
        FP8_CUDA_CHECK(cudaFuncSetAttribute(gemm_blockwise_pair_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                            DYN_BYTES)); \
        gemm_blockwise_pair_kernel<MODE><<<2 * p.num_pairs, THREADS, DYN_BYTES, st>>>(ta, tb, p); \
    } while (0)
    if (mode == MODE_FWD) FP8DPA_LAUNCH_BW2(MODE_FWD);
    else if (mode == MODE_DGRAD) FP8DPA_LAUNCH_BW2(MODE_DGRAD);
    else FP8DPA_LAUNCH_BW2(MODE_WGRAD);
#undef FP8DPA_LAUNCH_BW2
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

}  // namespace fp8dpa
