// FP8 attention backward for head_dim 128: software-pipelined, transposed formulation.
//
// One CTA per (128-key tile, KV head, batch) keeps K_j, V_j in shared memory and dK_j, dV_j in TMEM (256
// columns).  It walks over 64-query sub-tiles t (and the query heads of the group).  With rows = keys:
//   S^T  = K  Q_t^T   [128 x 64]     dP^T = V dO_t^T   [128 x 64]          (64 TMEM columns, one slot per group)
//   P~^T = 2^(c S^T - lse2_q),  P8^T = E4M3,  dS8^T = E5M2( P~^T o (a dP^T - db_q) )
//   dV  += P8^T dO_t      dK += dS8^T Q_t      dQ_t^T = K^T dS8^T  [128(d) x 64]  (64 TMEM columns, one slot)
// The per-query terms lse2_q and db_q never reach the element-wise threads as data: the prep kernel writes them,
// divided by c resp. a and split into three BF16 terms, as one row of 16 BF16 per query, and the tensor core adds them
// to the accumulators with one K = 16 BF16 product each (a tile of ones x that row), so that S^T and dP^T arrive as
// S^T - lse2_q / c and dP^T - db_q / a and one multiplication is left.  A shared-memory load in front of every pair
// of columns was what bounded these threads: while the tensor core streams operands out of shared memory, a
// dependent ld.shared takes several times its idle latency (measured: the exponential phase 1375 -> 650 clk).
// Two element-wise warpgroups take the sub-tiles in turn (even t / odd t), one thread per key row and all 64
// query columns, so the exponentials of one sub-tile overlap the dS arithmetic and the barrier round trips of
// the other.  Each group owns one 64-column TMEM slot that holds S^T_t and then dP^T_t (issued as soon as the
// group has S^T_t in registers), 2 x 16 TMEM columns for P8^T_t and dS8^T_t (rows = keys is exactly the layout of
// a left operand in TMEM: dV += P8^T dO and dK += dS8^T Q read them from there, four codes per column) and one
// dS8^T tile in shared memory (the right operand of dQ^T = K^T dS8^T).  dQ^T tiles have one TMEM slot and leave
// through two staging tiles in shared memory and one bulk reduce-add (binary32 add in L2) per sub-tile into the
// FP32 accumulator.
//
// Warpgroups: 0 = control (warp 0 TMA producer, warp 1 MMA issuer), 1-2 = element-wise, 3 = dQ drain; registers
// are moved from the control and drain groups to the element-wise groups (setmaxnreg).  Every wait is bounded.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <math.h>

#include "common.cuh"

namespace fp8dpa {

namespace bwd128 {

constexpr int D = 128;
constexpr int KT = 128;            // keys per CTA
constexpr int QT = 64;             // queries per sub-tile
constexpr int STAGES = 5;          // (Q, dO, lse2, db) stages: a TMA load takes several sub-tile periods to land
constexpr int THREADS = 16 * 32;     // four warpgroups: control (TMA, MMA), two element-wise groups, dQ drain
constexpr int DRAIN_WARPS = 4;
// per thread after setmaxnreg (splits of 56/176/104, 80/168/96, 96/160/96 measured the same within 0.5%; those that spill lose 2-4%)
constexpr int REGS_CTRL = 64, REGS_EW = 176, REGS_DRAIN = 88;
static_assert(REGS_CTRL + 2 * REGS_EW + REGS_DRAIN <= 4 * 128 && REGS_CTRL <= 128 && REGS_DRAIN <= 128 && REGS_EW >= 128,
              "register hand-over: releases must cover the increases inside the 512 x 128 of the launch");
constexpr int TMEM_COLS = 512;

struct Smem {
    static constexpr int K_OFF = 0;
    static constexpr int V_OFF = K_OFF + KT * D;
    static constexpr int QDO_OFF = V_OFF + KT * D;
    static constexpr int Q_BYTES = QT * D;                       // 8 KB
    static constexpr int VEC_BYTES = QT * 32;                    // 2 KB: per query 16 BF16 (shift of S^T, shift of dP^T)
    static constexpr int STAGE_BYTES = 2 * Q_BYTES + VEC_BYTES;  // Q, dO, the per-query shifts
    static constexpr int STAGE_TX = STAGE_BYTES;
    static constexpr int PDS_OFF = QDO_OFF + STAGES * STAGE_BYTES;
    static constexpr int PDS_TILE = KT * QT;                     // 8 KB: [128 key rows x 64 B]
    static constexpr int PDS_BUF = PDS_TILE;                     // dS8^T (P8^T lives in TMEM only)
    // left operands of the two rank-one products that add the per-query shifts: [128 keys x 16 BF16], ones in the
    // columns of the shift they pick (32-byte swizzle)
    static constexpr int ONES_OFF = PDS_OFF + 2 * PDS_BUF;
    static constexpr int ONES_BYTES = KT * 32;                   // 4 KB each
    static constexpr int DQ_OFF = ONES_OFF + 2 * ONES_BYTES;
    static constexpr int DQ_BYTES = QT * D * 4;                  // 32 KB: [64 q x 128 d] FP32
    static constexpr int BAR_OFF = DQ_OFF + 2 * DQ_BYTES;          // two staging tiles
    // kv_full, qdo_full[S], qdo_empty[S], then per group: s_full, dp_full, s_read, dp_read, pds_full, pds_free,
    // dq_full, dq_empty (of the two, index 0 serves the one dQ^T slot); all_done
    static constexpr int N_BARS = 1 + 2 * STAGES + 8 * 2 + 1;
    static constexpr int TOTAL = BAR_OFF + N_BARS * 8 + 16;
    static constexpr int DYN_BYTES = TOTAL + 1024;
};
// TMEM columns
// S^T/dP^T slot per group, one dQ^T slot, per group 16 columns of P8^T and 16 of dS8^T (A operands of the dV and dK
// products: lane = key, four codes per column), dV, dK
constexpr uint32_t T_SD0 = 0, T_SD1 = 64, T_DQ = 128, T_P0 = 192, T_DS0 = 208, T_P1 = 224, T_DS1 = 240, T_DV = 256, T_DK = 384;

struct Params {
    uint16_t *dK, *dV;     // [B,N,Hkv,D] BF16
    const float *q_inv, *k_inv, *v_inv, *do_inv, *ds_scale;
    float *ds_amax;
    float softmax_scale, p_scale;
    int causal;
    int B, N, Npad, Hq, Hkv;
    int *status;
};

__device__ __forceinline__ float e5m2_to_f32(uint32_t code)
{
    return __half2float(__ushort_as_half((unsigned short)(code << 8)));
}

// ---------------------------------------------------------------- prep
// Eight lanes per (b, i, h) with i < Npad (16-byte loads): D_i = do_inv * sum_d dec(dO8) * O, then the two per-query
// shifts of the main kernel, each already divided by the factor its accumulator is multiplied with afterwards:
//   L_i  = (log2(c_P) - LSE_i * log2(e)) / c      so that c * (S^T + L)  = c S^T - lse2        (exponent of c_P * P)
//   Db_i = (-D_i * ds_scale / c_P) / a            so that a * (dP^T + Db) = a dP^T - db        (factor of dS)
// Both go out as three BF16 terms (hi + mid + lo = the binary32 value exactly) in a row of 16 BF16: L in columns 0-2,
// Db in columns 8-10, zeros elsewhere.  The main kernel adds them to its accumulators with one K = 16 BF16 product each
// (ones x row), so its element-wise threads never load a per-query value.  Rows i >= N get L = -2^100 (P = 0) and
// Db = 0; the dQ accumulator row is zeroed.
__device__ __forceinline__ uint32_t bf16_rn_bits(float x) { return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(x)); }
__device__ __forceinline__ void split3_bf16(float x, uint32_t &hi, uint32_t &mid, uint32_t &lo)
{
    hi = bf16_rn_bits(x);
    const float r1 = x - __uint_as_float(hi << 16);
    mid = bf16_rn_bits(r1);
    const float r2 = r1 - __uint_as_float(mid << 16);
    lo = bf16_rn_bits(r2);
}
__global__ void __launch_bounds__(256) attn_bwd_d128_prep_kernel(const uint8_t *__restrict__ dO8, const uint16_t *__restrict__ O,
                                                   const float *__restrict__ LSE, const float *__restrict__ q_inv,
                                                   const float *__restrict__ k_inv, const float *__restrict__ v_inv,
                                                   const float *__restrict__ do_inv,
                                                   const float *__restrict__ ds_scale, float softmax_scale, float p_scale,
                                                   float log2_p_scale, uint4 *__restrict__ vec,
                                                   float *__restrict__ dQacc, int B, int N,
                                                   int Npad, int Hq)
{
    const long n_rows = (long)B * Npad * Hq;
    const int j = threadIdx.x & 7;
    const float scale = __ldg(do_inv) * __ldg(ds_scale) / p_scale;
    // the same expressions as in the main kernel
    const float c = softmax_scale * __ldg(q_inv) * __ldg(k_inv) * 1.4426950408889634f;
    const float a_dp = __ldg(do_inv) * __ldg(v_inv) * __ldg(ds_scale) / p_scale;
    // the trip count is uniform over the CTA: the shuffles below name every lane
    for (long base = (long)blockIdx.x * 32; base < n_rows; base += (long)gridDim.x * 32) {
        const long w_raw = base + (threadIdx.x >> 3);            // (b*Npad + i)*Hq + h
        const bool in_range = w_raw < n_rows;
        const long w = in_range ? w_raw : n_rows - 1;
        const int h = (int)(w % Hq);
        const long bi = w / Hq;
        const int i = (int)(bi % Npad), b = (int)(bi / Npad);
        const size_t vi = ((size_t)b * Hq + h) * Npad + i;
        const bool real = i < N;
        const size_t row = ((size_t)b * N + (real ? i : 0)) * Hq + h;
        float acc = 0.0f;
        if (real) {
            const uint4 cw4 = __ldg(reinterpret_cast<const uint4 *>(dO8 + row * D + j * 16));
            const uint4 o0 = __ldg(reinterpret_cast<const uint4 *>(O + row * D + j * 16));
            const uint4 o1 = __ldg(reinterpret_cast<const uint4 *>(O + row * D + j * 16 + 8));
            const uint32_t cw[4] = {cw4.x, cw4.y, cw4.z, cw4.w};
            const uint32_t ow[8] = {o0.x, o0.y, o0.z, o0.w, o1.x, o1.y, o1.z, o1.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                acc = fmaf(e5m2_to_f32(cw[q] & 0xFF), bf16_lo(ow[2 * q]), acc);
                acc = fmaf(e5m2_to_f32((cw[q] >> 8) & 0xFF), bf16_hi(ow[2 * q]), acc);
                acc = fmaf(e5m2_to_f32((cw[q] >> 16) & 0xFF), bf16_lo(ow[2 * q + 1]), acc);
                acc = fmaf(e5m2_to_f32(cw[q] >> 24), bf16_hi(ow[2 * q + 1]), acc);
            }
        }
#pragma unroll
        for (int off = 4; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (!in_range) continue;
        if (real) {
            float4 *z = reinterpret_cast<float4 *>(dQacc + row * D + j * 16);
            const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
            z[0] = zero; z[1] = zero; z[2] = zero; z[3] = zero;
        }
        if (j == 0) {
            uint32_t l0 = 0xF180u, l1 = 0, l2 = 0, d0 = 0, d1 = 0, d2 = 0;          // 0xF180 = -2^100 in BF16
            if (real) {
                const float nl = log2_p_scale - __ldg(LSE + ((size_t)b * Hq + h) * N + i) * 1.4426950408889634f;
                const float L = fminf(fmaxf(__fdiv_rn(nl, c), -1e30f), 1e30f);
                const float Db = fminf(fmaxf(__fdiv_rn(-acc * scale, a_dp), -1e30f), 1e30f);
                split3_bf16(L, l0, l1, l2);
                split3_bf16(Db, d0, d1, d2);
            }
            vec[2 * vi] = make_uint4(l0 | (l1 << 16), l2, 0u, 0u);
            vec[2 * vi + 1] = make_uint4(d0 | (d1 << 16), d2, 0u, 0u);
        }
    }
}

// dQ = s * k_inv / ds_scale * accumulator, BF16; four 16-byte loads in flight per thread
__global__ void __launch_bounds__(256) attn_bwd_d128_finish_kernel(const float4 *__restrict__ acc, uint2 *__restrict__ dQ, size_t n4,
                                                     const float *__restrict__ k_inv,
                                                     const float *__restrict__ ds_scale, float softmax_scale)
{
    const float f = softmax_scale * __ldg(k_inv) / __ldg(ds_scale);
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + 3 * stride < n4; i += 4 * stride) {
        const float4 v0 = __ldcs(acc + i), v1 = __ldcs(acc + i + stride), v2 = __ldcs(acc + i + 2 * stride),
                     v3 = __ldcs(acc + i + 3 * stride);
        dQ[i] = make_uint2(pack_bf16x2(v0.x * f, v0.y * f), pack_bf16x2(v0.z * f, v0.w * f));
        dQ[i + stride] = make_uint2(pack_bf16x2(v1.x * f, v1.y * f), pack_bf16x2(v1.z * f, v1.w * f));
        dQ[i + 2 * stride] = make_uint2(pack_bf16x2(v2.x * f, v2.y * f), pack_bf16x2(v2.z * f, v2.w * f));
        dQ[i + 3 * stride] = make_uint2(pack_bf16x2(v3.x * f, v3.y * f), pack_bf16x2(v3.z * f, v3.w * f));
    }
    for (; i < n4; i += stride) {
        const float4 v = acc[i];
        dQ[i] = make_uint2(pack_bf16x2(v.x * f, v.y * f), pack_bf16x2(v.z * f, v.w * f));
    }
}

// D[tmem] (+)= A[tmem] * B[smem]: A = 128 rows (lanes) x 32 FP8 values in 8 consecutive 32-bit columns.
__device__ __forceinline__ void umma_f8_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc,
                                           uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}

template <int N> __device__ __forceinline__ void reg_dec()
{
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N> __device__ __forceinline__ void reg_inc()
{
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}

// ---------------------------------------------------------------- main
__global__ void __launch_bounds__(THREADS, 1)
attn_bwd_d128_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
            const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
            const __grid_constant__ CUtensorMap tm_dq, const __grid_constant__ CUtensorMap tm_vec, const Params p)
{
    using L = Smem;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + L::BAR_OFF;
    const uint32_t kv_full = bar0;
    auto qdo_full = [&](int s) { return bar0 + 8u * (1 + s); };
    auto qdo_empty = [&](int s) { return bar0 + 8u * (1 + STAGES + s); };
    const uint32_t bar1 = bar0 + 8u * (1 + 2 * STAGES);
    // per element-wise group (= parity of the sub-tile index)
    auto s_full = [&](int g) { return bar1 + 8u * g; };
    auto dp_full = [&](int g) { return bar1 + 8u * (2 + g); };
    auto s_read = [&](int g) { return bar1 + 8u * (4 + g); };
    auto dp_read = [&](int g) { return bar1 + 8u * (6 + g); };
    auto pds_full = [&](int g) { return bar1 + 8u * (8 + g); };
    auto pds_free = [&](int g) { return bar1 + 8u * (10 + g); };
    auto dq_full = [&](int g) { return bar1 + 8u * (12 + g); };
    auto dq_empty = [&](int g) { return bar1 + 8u * (14 + g); };
    const uint32_t all_done = bar1 + 8u * 16;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + L::BAR_OFF + L::N_BARS * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int wg = warp >> 2;
    // KV head fastest: the CTAs that run at the same time then add their dQ tiles into different rows of a small,
    // L2-resident band of the accumulator instead of contending for the same rows
    // ... and key tiles in ascending order over the whole grid (batch folded into x): with a causal mask the first key
    // tiles see the most queries, so the longest CTAs of every batch start first
    const int g = (int)(blockIdx.x % (unsigned)p.Hkv), b = (int)(blockIdx.x / (unsigned)p.Hkv), k_tile = blockIdx.y;
    const int G = p.Hq / p.Hkv;
    const int k0 = k_tile * KT;
    const int n_sub = p.Npad / QT;
    const int i_first = p.causal ? (k0 / QT) : 0;         // first 64-query sub-tile that sees these keys
    const int per_head = n_sub - i_first;
    const int n_iter = per_head * G;
    auto head_of = [&](int t) { return g * G + t / per_head; };
    auto q0_of = [&](int t) { return (i_first + t % per_head) * QT; };

    if (threadIdx.x == 0) {
        mbar_init(kv_full, 1);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(qdo_full(s), 1);
            mbar_init(qdo_empty(s), 1);
        }
        for (int e = 0; e < 2; ++e) {
            mbar_init(s_full(e), 1);
            mbar_init(dp_full(e), 1);
            mbar_init(s_read(e), 4);
            mbar_init(dp_read(e), 4);
            mbar_init(pds_full(e), 4);
            mbar_init(pds_free(e), 1);
            mbar_init(dq_full(e), 1);
            mbar_init(dq_empty(e), DRAIN_WARPS);
        }
        mbar_init(all_done, 1);
        *abort_flag = 0;
        mbar_init_fence();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
        tma_prefetch_desc(&tm_do);
        tma_prefetch_desc(&tm_dq);
        tma_prefetch_desc(&tm_vec);
    }
    // the two ones-tiles: row r holds BF16 ones in columns 0-3 (picks L) resp. 8-11 (picks Db), zeros elsewhere; under
    // the 32-byte swizzle the 16-byte half c of row r lies at half c ^ ((r >> 2) & 1)
    if (threadIdx.x < 2 * KT) {
        const int which = threadIdx.x / KT, r = threadIdx.x % KT;
        uint4 *rowp = reinterpret_cast<uint4 *>(smem + L::ONES_OFF + which * L::ONES_BYTES + r * 32);
        const uint4 ones = make_uint4(0x3F803F80u, 0x3F803F80u, 0u, 0u), zero = make_uint4(0u, 0u, 0u, 0u);
        const int flip = (r >> 2) & 1;
        rowp[which ^ flip] = ones;
        rowp[(which ^ 1) ^ flip] = zero;
    }
    fence_proxy_async_smem();
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const WaitCtx ctx{p.status, abort_flag};

    if (wg == 0) {
        reg_dec<REGS_CTRL>();
        if (warp == 0) {
            // -------------------------------------------------------- TMA producer
            if (elect_one()) {
                mbar_expect_tx(kv_full, 2 * KT * D);
                tma_load_3d(sbase + L::K_OFF, &tm_k, kv_full, g * D, k0, b);
                tma_load_3d(sbase + L::V_OFF, &tm_v, kv_full, g * D, k0, b);
                for (int t = 0; t < n_iter; ++t) {
                    const int st = t % STAGES;
                    const uint32_t ph = (uint32_t)(t / STAGES) & 1u;
                    const int h = head_of(t), q0 = q0_of(t);
                    if (!mbar_wait(qdo_empty(st), ph ^ 1u, ctx)) break;
                    const uint32_t sq = sbase + L::QDO_OFF + st * L::STAGE_BYTES, sdo = sq + L::Q_BYTES;
                    const uint32_t sl = sdo + L::Q_BYTES;
                    const int vrow = (b * p.Hq + h) * p.Npad + q0;
                    mbar_expect_tx(qdo_full(st), L::STAGE_TX);
                    tma_load_3d(sq, &tm_q, qdo_full(st), h * D, q0, b);
                    tma_load_3d(sdo, &tm_do, qdo_full(st), h * D, q0, b);
                    tma_load_2d(sl, &tm_vec, qdo_full(st), 0, vrow);
                }
            }
        } else if (warp == 1) {
            // -------------------------------------------------------- MMA issuer
            if (elect_one()) {
                constexpr uint32_t E4 = 0, E5 = 1;
                constexpr uint32_t id_s = umma_idesc_f8(E4, E4, 128, QT, 0, 0);      // K (K-major) x Q (K-major)
                constexpr uint32_t id_dp = umma_idesc_f8(E4, E5, 128, QT, 0, 0);     // V x dO
                constexpr uint32_t id_dv = umma_idesc_f8(E4, E5, 128, D, 0, 1);      // P8^T (K-major) x dO (MN)
                constexpr uint32_t id_dk = umma_idesc_f8(E5, E4, 128, D, 0, 1);      // dS8^T (K-major) x Q (MN)
                constexpr uint32_t id_dq = umma_idesc_f8(E4, E5, 128, QT, 1, 1);     // K^T (MN) x dS8^T (MN)
                constexpr uint32_t id_vec = umma_idesc_f8(1, 1, 128, QT, 0, 0);      // kind::f16: BF16 ones x BF16 shifts
                const uint64_t d_ones_l = umma_desc_k_sw32(sbase + L::ONES_OFF);
                const uint64_t d_ones_d = umma_desc_k_sw32(sbase + L::ONES_OFF + L::ONES_BYTES);
                const uint64_t d_k = umma_desc(sbase + L::K_OFF, 128, 16);
                const uint64_t d_v = umma_desc(sbase + L::V_OFF, 128, 16);
                constexpr uint32_t ROWS32_128 = (32 * 128) >> 4;   // 32 rows of a 128-byte-row tile
                constexpr uint32_t ROWS32_64 = (32 * 64) >> 4;     // 32 rows of a 64-byte-row tile
                auto stage_q = [&](int t) { return sbase + L::QDO_OFF + (t % STAGES) * L::STAGE_BYTES; };
                auto wait_stage = [&](int t) {
                    return mbar_wait(qdo_full(t % STAGES), (uint32_t)(t / STAGES) & 1u, ctx);
                };
                auto issue_s = [&](int t) {     // S^T_t = K Q_t^T into the slot of group t & 1
                    const uint64_t d_q = umma_desc(stage_q(t), 128, 16);
                    const uint32_t dst = tmem_base + ((t & 1) ? T_SD1 : T_SD0);
#pragma unroll
                    for (int k = 0; k < D / 32; ++k) umma_f8_ss(dst, d_k + 2u * k, d_q + 2u * k, id_s, k != 0);
                    // + 1 x L_q: the accumulator leaves as S^T - lse2 / c
                    umma_bf16_ss(dst, d_ones_l, umma_desc_k_sw32(stage_q(t) + 2 * L::Q_BYTES), id_vec, 1u);
                    umma_commit(s_full(t & 1));
                };
                auto issue_dp = [&](int t) {    // dP^T_t = V dO_t^T into the same slot, once S^T_t is in registers
                    const uint64_t d_do = umma_desc(stage_q(t) + L::Q_BYTES, 128, 16);
                    const uint32_t dst = tmem_base + ((t & 1) ? T_SD1 : T_SD0);
#pragma unroll
                    for (int k = 0; k < D / 32; ++k) umma_f8_ss(dst, d_v + 2u * k, d_do + 2u * k, id_dp, k != 0);
                    // + 1 x Db_q: the accumulator leaves as dP^T - db / a
                    umma_bf16_ss(dst, d_ones_d, umma_desc_k_sw32(stage_q(t) + 2 * L::Q_BYTES), id_vec, 1u);
                    umma_commit(dp_full(t & 1));
                };
                // dQ^T_t, dV, dK of sub-tile t, once P8^T_t and dS8^T_t are in shared memory
                auto finish = [&](int t) {
                    const int e = t & 1;
                    const uint32_t u = (uint32_t)(t >> 1);
                    if (!mbar_wait(pds_full(e), u & 1u, ctx)) return false;
                    // one dQ^T slot: the drain must have taken sub-tile t-1 out of it
                    if (t > 0 && !mbar_wait(dq_empty(0), (uint32_t)(t - 1) & 1u, ctx)) return false;
                    tc_fence_after();
                    const uint32_t sds = sbase + L::PDS_OFF + e * L::PDS_BUF;
                    const uint64_t d_ds = umma_desc(sds, 64, 16);
                    const uint64_t d_q = umma_desc(stage_q(t), 128, 16), d_do = umma_desc(stage_q(t) + L::Q_BYTES, 128, 16);
                    // dQ^T_t = K^T dS8^T_t: reduction over the 128 keys, 32 rows of either tile per step
#pragma unroll
                    for (int k = 0; k < KT / 32; ++k)
                        umma_f8_ss(tmem_base + T_DQ, d_k + ROWS32_128 * k, d_ds + ROWS32_64 * k, id_dq, k != 0);
                    umma_commit(dq_full(0));
                    // dV += P8^T dO_t, dK += dS8^T Q_t: reduction over the 64 queries, 32 per step; the left operands
                    // come straight from TMEM (rows = keys is the layout the element-wise threads produce)
#pragma unroll
                    for (int k = 0; k < QT / 32; ++k)
                        umma_f8_ts(tmem_base + T_DV, tmem_base + (e ? T_P1 : T_P0) + 8u * k, d_do + ROWS32_128 * k, id_dv, (t | k) != 0);
#pragma unroll
                    for (int k = 0; k < QT / 32; ++k)
                        umma_f8_ts(tmem_base + T_DK, tmem_base + (e ? T_DS1 : T_DS0) + 8u * k, d_q + ROWS32_128 * k, id_dk, (t | k) != 0);
                    umma_commit(qdo_empty(t % STAGES));
                    umma_commit(pds_free(e));
                    return true;
                };
                bool ok = mbar_wait(kv_full, 0, ctx);
                if (ok) ok = wait_stage(0);
                if (ok) {
                    tc_fence_after();
                    issue_s(0);
                }
                if (ok && n_iter > 1) {
                    ok = wait_stage(1);
                    if (ok) {
                        tc_fence_after();
                        issue_s(1);
                    }
                }
                for (int t = 0; t < n_iter && ok; ++t) {
                    if (t >= 1 && t + 1 < n_iter) {
                        // the slot of sub-tile t+1 held dP_{t-1}: wait until the threads have read it
                        if (!mbar_wait(dp_read((t + 1) & 1), (uint32_t)((t - 1) >> 1) & 1u, ctx)) { ok = false; break; }
                        if (!wait_stage(t + 1)) { ok = false; break; }
                        tc_fence_after();
                        issue_s(t + 1);
                    }
                    if (!mbar_wait(s_read(t & 1), (uint32_t)(t >> 1) & 1u, ctx)) { ok = false; break; }
                    tc_fence_after();
                    issue_dp(t);
                    if (t >= 1 && !finish(t - 1)) { ok = false; break; }
                }
                if (ok) ok = finish(n_iter - 1);
                if (ok) umma_commit(all_done);
            }
        }
    } else if (wg <= 2) {
        reg_inc<REGS_EW>();
        // ------------------------------------------------------------ element-wise: P8^T, dS8^T
        // Group e takes the sub-tiles t = e, e+2, ...; each thread one key row and all 64 query columns.  The two
        // groups run half a period apart, so one group's exponentials overlap the other's dS arithmetic.
        const int e = wg - 1;
        const int quad = warp & 3;                      // TMEM lanes 32*quad..: rows (keys) of this warp
        const int r = quad * 32 + lane;                 // key row inside the tile
        const int key = k0 + r;
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        const uint32_t t_sd = tmem_base + (e ? T_SD1 : T_SD0) + lane_addr;
        const float c = p.softmax_scale * __ldg(p.q_inv) * __ldg(p.k_inv) * 1.4426950408889634f;
        const float dss = __ldg(p.ds_scale);
        const float a_dp = __ldg(p.do_inv) * __ldg(p.v_inv) * dss / p.p_scale;
        const uint64_t c2 = pack_f32x2(c, c), a2 = pack_f32x2(a_dp, a_dp);
        const int sw = (r >> 1) & 3;                    // 64-byte swizzle: 16-byte chunk index ^ ((row >> 1) & 3)
        uint8_t *dsrow = smem + L::PDS_OFF + e * L::PDS_BUF + r * 64;
        float amax = 0.0f;
        bool ok = true;
        for (int t = e; t < n_iter; t += 2) {
            const uint32_t u = (uint32_t)(t >> 1);
            const int q0 = q0_of(t);
            // valid iff key <= query (causal) and key < N; queries >= N carry -lse2 = -inf
            const bool need_mask = (p.causal && q0 < k0 + KT - 1) || (k0 + KT > p.N);
            const int first_ok = (key < p.N) ? (p.causal ? key - q0 : 0) : 64;   // columns >= first_ok are valid
            if (!mbar_wait_warp(s_full(e), u & 1u, ctx)) { ok = false; break; }
            tc_fence_after();
            float pe[64];
            {
                uint32_t sa[32], sb[32];
                tmem_ld_32x32b_x32(t_sd, sa);
                tmem_ld_32x32b_x32(t_sd + 32u, sb);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(s_read(e));   // the slot may take dP^T_t
#pragma unroll
                for (int i = 0; i < 64; i += 2) {
                    // the accumulator already carries the per-query shift (rank-one product): one multiply is left
                    const uint32_t *sx = i < 32 ? sa + i : sb + (i - 32);
                    float x0, x1;
                    unpack_f32x2(mul_f32x2(pack_u32x2(sx[0], sx[1]), c2), x0, x1);
                    pe[i] = ex2_approx(x0);             // c_P * P
                    pe[i + 1] = ex2_approx(x1);
                }
            }
            if (need_mask) {
#pragma unroll
                for (int i = 0; i < 64; ++i)
                    if (i < first_ok) pe[i] = 0.0f;
            }
            // the P8/dS8 buffer of this group was last read by the MMAs of sub-tile t-2
            if (u > 0 && !mbar_wait_warp(pds_free(e), (u - 1) & 1u, ctx)) { ok = false; break; }
            {
                uint32_t wp[16];                         // P8^T row of this key: 64 codes, four per word
#pragma unroll
                for (int q = 0; q < 16; ++q)
                    wp[q] = cvt_f32x4_to_fp8x4<0>(pe[4 * q], pe[4 * q + 1], pe[4 * q + 2], pe[4 * q + 3]);
                tmem_st_32x32b_x16(tmem_base + (e ? T_P1 : T_P0) + lane_addr, wp);
            }
            if (!mbar_wait_warp(dp_full(e), u & 1u, ctx)) { ok = false; break; }
            tc_fence_after();
            uint32_t wds[16];
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                uint32_t dv[32];
                tmem_ld_32x32b_x32(t_sd + (uint32_t)(32 * hf), dv);
                tmem_ld_wait();
                if (hf == 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(dp_read(e));   // the slot may take S^T_{t+2}
                }
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    float y0, y1;
                    unpack_f32x2(mul_f32x2(pack_f32x2(pe[32 * hf + i], pe[32 * hf + i + 1]),
                                           mul_f32x2(pack_u32x2(dv[i], dv[i + 1]), a2)), y0, y1);
                    pe[32 * hf + i] = y0;                // ds_scale * dS
                    pe[32 * hf + i + 1] = y1;
                    amax = fmaxf(amax, fmaxf(fabsf(y0), fabsf(y1)));
                }
#pragma unroll
                for (int ch = 2 * hf; ch < 2 * hf + 2; ++ch) {
                    uint4 w;
                    w.x = cvt_f32x4_to_fp8x4<1>(pe[16 * ch], pe[16 * ch + 1], pe[16 * ch + 2], pe[16 * ch + 3]);
                    w.y = cvt_f32x4_to_fp8x4<1>(pe[16 * ch + 4], pe[16 * ch + 5], pe[16 * ch + 6], pe[16 * ch + 7]);
                    w.z = cvt_f32x4_to_fp8x4<1>(pe[16 * ch + 8], pe[16 * ch + 9], pe[16 * ch + 10], pe[16 * ch + 11]);
                    w.w = cvt_f32x4_to_fp8x4<1>(pe[16 * ch + 12], pe[16 * ch + 13], pe[16 * ch + 14], pe[16 * ch + 15]);
                    *reinterpret_cast<uint4 *>(dsrow + ((ch ^ sw) << 4)) = w;       // right operand of dQ^T
                    wds[4 * ch] = w.x; wds[4 * ch + 1] = w.y; wds[4 * ch + 2] = w.z; wds[4 * ch + 3] = w.w;
                }
            }
            tmem_st_32x32b_x16(tmem_base + (e ? T_DS1 : T_DS0) + lane_addr, wds);      // left operand of dK
            tmem_st_wait();
            tc_fence_before();
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(pds_full(e));
        }
        // ---- epilogue: group 0 writes dV, group 1 dK (TMEM lane = key)
        if (ok && mbar_wait_warp(all_done, 0, ctx)) {
            tc_fence_after();
            const float f = e == 0 ? __ldg(p.do_inv) / p.p_scale : p.softmax_scale * __ldg(p.q_inv) / dss;
            uint16_t *dst = (e == 0 ? p.dV : p.dK) + (((size_t)b * p.N + key) * p.Hkv + g) * D;
            const uint32_t tcol = e == 0 ? T_DV : T_DK;
#pragma unroll 1
            for (int cc = 0; cc < D; cc += 32) {
                uint32_t v[32];
                tmem_ld_32x32b_x32(tmem_base + tcol + lane_addr + (uint32_t)cc, v);
                tmem_ld_wait();
                if (key < p.N) {
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        uint4 o;
                        o.x = pack_bf16x2(__uint_as_float(v[i]) * f, __uint_as_float(v[i + 1]) * f);
                        o.y = pack_bf16x2(__uint_as_float(v[i + 2]) * f, __uint_as_float(v[i + 3]) * f);
                        o.z = pack_bf16x2(__uint_as_float(v[i + 4]) * f, __uint_as_float(v[i + 5]) * f);
                        o.w = pack_bf16x2(__uint_as_float(v[i + 6]) * f, __uint_as_float(v[i + 7]) * f);
                        *reinterpret_cast<uint4 *>(dst + cc + i) = o;
                    }
                }
            }
            if (p.ds_amax) {
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
                // the kernel tracked ds_scale * |dS|; non-negative floats order like unsigned integers
                if (lane == 0) atomicMax(reinterpret_cast<unsigned int *>(p.ds_amax), __float_as_uint(amax / dss));
            }
        }
    } else {
        reg_dec<REGS_DRAIN>();
        // ------------------------------------------------------------ dQ drain (4 warps)
        const int quad = warp & 3;                      // TMEM lane = d index
        const int dd = quad * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        const bool issuer = (quad == 0) && lane == 0;
        for (int t = 0; t < n_iter; ++t) {
            const int h = head_of(t), q0 = q0_of(t), e = t & 1;
            float *dq_s = reinterpret_cast<float *>(smem + L::DQ_OFF + e * L::DQ_BYTES);
            const bool got = mbar_wait_warp(dq_full(0), (uint32_t)t & 1u, ctx);
            uint32_t va[32], vb[32];
            if (got) {
                tc_fence_after();
                const uint32_t src = tmem_base + T_DQ + lane_addr;
                tmem_ld_32x32b_x32(src, va);
                tmem_ld_32x32b_x32(src + 32u, vb);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(dq_empty(0));   // the dQ^T slot may be overwritten
            }
            // the reduce issued two sub-tiles ago must have finished reading this staging tile
            if (issuer) bulk_wait_group_read1();
            if (named_barrier_or(1, DRAIN_WARPS * 32, !got)) break;   // all four warps leave together
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                dq_s[i * D + dd] = __uint_as_float(va[i]);
                dq_s[(i + 32) * D + dd] = __uint_as_float(vb[i]);
            }
            fence_proxy_async_smem();
            named_barrier_sync(1, DRAIN_WARPS * 32);
            if (issuer) {
                tma_reduce_add_3d(&tm_dq, sbase + L::DQ_OFF + e * L::DQ_BYTES, h * D, q0, b);
                bulk_commit_group();
            }
        }
        if (issuer) bulk_wait_group0();                 // all reduce-adds complete before the CTA exits
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

}  // namespace bwd128

size_t attn_bwd_d128_ws_bytes(int B, int N, int Hq)
{
    // per (batch, head, padded query) one row of 16 BF16 (the two shifts), then the FP32 dQ accumulator
    const size_t Npad = ((size_t)N + bwd128::QT - 1) / bwd128::QT * bwd128::QT;
    const size_t vec = (((size_t)B * Hq * Npad * 32) + 255) & ~(size_t)255;
    return vec + (size_t)B * N * Hq * bwd128::D * sizeof(float);
}

int launch_attn_bwd_d128(const uint8_t *Q8, const uint8_t *K8, const uint8_t *V8, const uint8_t *dO8,
                         const uint16_t *O, const float *LSE, const fp8_attn_scales *sc, int causal, int B, int N,
                         int Hq, int Hkv, uint16_t *dQ, uint16_t *dK, uint16_t *dV, void *ws, int *status,
                         cudaStream_t st)
{
    using namespace bwd128;
    const int Npad = (N + QT - 1) / QT * QT;
    const size_t vec = (((size_t)B * Hq * Npad * 32) + 255) & ~(size_t)255;
    uint4 *shifts = static_cast<uint4 *>(ws);
    float *dQacc = reinterpret_cast<float *>(static_cast<uint8_t *>(ws) + vec);
    CUtensorMap tq, tk, tv, tdo, tdq, tvec;
    int rc = make_tmap_3d_u8(&tq, Q8, (uint64_t)Hq * D, (uint64_t)N, (uint64_t)B, D, QT);
    if (rc != FP8_OK) return rc;
    rc = make_tmap_3d_u8(&tk, K8, (uint64_t)Hkv * D, (uint64_t)N, (uint64_t)B, D, KT);
    if (rc != FP8_OK) return rc;
    rc = make_tmap_3d_u8(&tv, V8, (uint64_t)Hkv * D, (uint64_t)N, (uint64_t)B, D, KT);
    if (rc != FP8_OK) return rc;
    rc = make_tmap_3d_u8(&tdo, dO8, (uint64_t)Hq * D, (uint64_t)N, (uint64_t)B, D, QT);
    if (rc != FP8_OK) return rc;
    rc = make_tmap_3d_f32(&tdq, dQacc, (uint64_t)Hq * D, (uint64_t)N, (uint64_t)B, D, QT);
    if (rc != FP8_OK) return rc;
    rc = make_tmap_2d_bf16x16(&tvec, shifts, (uint64_t)B * Hq * Npad, QT);
    if (rc != FP8_OK) return rc;
    if (sc->ds_amax) FP8_CUDA_CHECK(cudaMemsetAsync(sc->ds_amax, 0, sizeof(float), st));
    const float log2_p = log2f(sc->p_scale);
    const long prep_rows = (long)B * Npad * Hq;
    long prep_blocks = (prep_rows + 31) / 32;                   // 32 rows per CTA and sweep
    if (prep_blocks > (long)sm_count() * 16) prep_blocks = (long)sm_count() * 16;
    attn_bwd_d128_prep_kernel<<<(unsigned)prep_blocks, 256, 0, st>>>(dO8, O, LSE, sc->q_inv, sc->k_inv, sc->v_inv, sc->do_inv,
                                                            sc->ds_scale, sc->softmax_scale, sc->p_scale, log2_p, shifts,
                                                            dQacc, B, N, Npad, Hq);
    FP8_CUDA_CHECK(cudaGetLastError());
    Params p;
    p.dK = dK; p.dV = dV;
    p.q_inv = sc->q_inv; p.k_inv = sc->k_inv; p.v_inv = sc->v_inv; p.do_inv = sc->do_inv;
    p.ds_scale = sc->ds_scale;
    p.ds_amax = sc->ds_amax;
    p.softmax_scale = sc->softmax_scale;
    p.p_scale = sc->p_scale;
    p.causal = causal ? 1 : 0;
    p.B = B; p.N = N; p.Npad = Npad; p.Hq = Hq; p.Hkv = Hkv;
    p.status = status;
    FP8_CUDA_CHECK(cudaFuncSetAttribute(attn_bwd_d128_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem::DYN_BYTES));
    dim3 grid((unsigned)(Hkv * B), (unsigned)((N + KT - 1) / KT), 1);
    {
        const int rc_regs = check_launch_registers(attn_bwd_d128_kernel, 128, "attn_bwd_d128_kernel");
        if (rc_regs != FP8_OK) return rc_regs;
    }
    attn_bwd_d128_kernel<<<grid, THREADS, Smem::DYN_BYTES, st>>>(tq, tk, tv, tdo, tdq, tvec, p);
    FP8_CUDA_CHECK(cudaGetLastError());
    const size_t n4 = (size_t)B * N * Hq * D / 4;
    size_t blocks = (n4 + 255) / 256;
    const size_t cap = (size_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    attn_bwd_d128_finish_kernel<<<(unsigned)blocks, 256, 0, st>>>(reinterpret_cast<const float4 *>(dQacc),
                                                   reinterpret_cast<uint2 *>(dQ), n4, sc->k_inv, sc->ds_scale,
                                                   sc->softmax_scale);
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

}  // namespace fp8dpa
