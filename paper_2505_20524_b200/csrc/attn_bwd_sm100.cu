// FP8 attention backward (gradient of Appendix B, Eq. (P) with every product on FP8 tensor cores).
//
//   D_i  = sum_d dO_id O_id                     P_ij  = exp(x_ij - LSE_i)        (recomputed, never stored)
//   dV_j = sum_i P8_ij dO_i                     dP_ij = dO_i . V_j
//   dS   = P o (dP - D)   -> E5M2 (dS8)         dQ_i  = s sum_j dS8_ij K_j       dK_j = s sum_i dS8_ij Q_i
//
// This file holds the simple (un-pipelined) form, used for head_dim 64; head_dim 128 runs the pipelined kernel
// of attn_bwd_d128_sm100.cu.  Three launches on the caller's stream:
//   1. prep:    D (FP32) from dO8 and O, and zeroing of the FP32 dQ accumulator (both live in the workspace)
//   2. main:    one CTA per (128-key tile, KV head, batch); it keeps K_j, V_j in shared memory, walks over
//               the query tiles (and the query heads of the group) that see these keys, and per tile pair runs
//                 S = Q K^T, dP = dO V^T                       (accumulators in TMEM columns 0..255)
//                 -> 128 threads, one query row each: P8, dS8 into shared memory (one swizzled tile each)
//                 dV += P8^T dO, dK += dS8^T Q                 (P8 / dS8 read as MN-major A operands)
//                 dQ_tile = dS8 K                              (same dS8 tile read as a K-major A operand)
//               dK, dV stay in TMEM for the whole walk; dQ tiles are added into the FP32 accumulator
//   3. finish:  dQ accumulator * s*k_inv/ds_scale -> BF16
#include <cuda_fp16.h>
#include <math.h>

#include "common.cuh"

namespace fp8dpa {

size_t attn_bwd_d128_ws_bytes(int B, int N, int Hq);
int launch_attn_bwd_d128(const uint8_t *Q8, const uint8_t *K8, const uint8_t *V8, const uint8_t *dO8,
                         const uint16_t *O, const float *LSE, const fp8_attn_scales *sc, int causal, int B, int N,
                         int Hq, int Hkv, uint16_t *dQ, uint16_t *dK, uint16_t *dV, void *ws, int *status,
                         cudaStream_t st);
int validate_attn(const char *who, const void *q, const void *k, const void *v, const fp8_attn_scales *sc, int B, int N,
                  int Hq, int Hkv, int d);

constexpr int B_BM = 128;   // queries per tile
constexpr int B_BN = 128;   // keys per CTA
constexpr int B_STAGES = 2;
constexpr int B_THREADS = 192;
constexpr int B_TMEM_COLS = 512;

template <int D>
struct AttnBwdSmem {
    static constexpr int TILE = 128 * D;                  // one [128 x D] operand tile
    static constexpr int K_OFF = 0;
    static constexpr int V_OFF = K_OFF + TILE;
    static constexpr int QDO_OFF = V_OFF + TILE;          // stages of (Q, dO)
    static constexpr int STAGE_BYTES = 2 * TILE;
    static constexpr int P_OFF = QDO_OFF + B_STAGES * STAGE_BYTES;
    static constexpr int DS_OFF = P_OFF + 128 * 128;
    static constexpr int BAR_OFF = DS_OFF + 128 * 128;
    // kv_full, qdo_full[2], qdo_empty[2], s_full, pds_full, dq_full, dq_empty
    static constexpr int N_BARS = 1 + 2 * B_STAGES + 4;
    static constexpr int TOTAL = BAR_OFF + N_BARS * 8 + 16;
    static constexpr int DYN_BYTES = TOTAL + 1024;
    // TMEM columns
    static constexpr int T_S = 0;       // S, later the dQ tile
    static constexpr int T_DP = 128;
    static constexpr int T_DV = 256;
    static constexpr int T_DK = 256 + D;
};

struct AttnBwdParams {
    const float *LSE;      // [B,Hq,N]
    const float *Dsum;     // [B,Hq,N]  (workspace)
    float *dQacc;          // [B,N,Hq,D] FP32 (workspace)
    uint16_t *dK, *dV;     // [B,N,Hkv,D] BF16
    const float *q_inv, *k_inv, *v_inv, *do_inv, *ds_scale;
    float *ds_amax;        // nullable
    float softmax_scale, p_scale, log2_p_scale;
    int causal;
    int B, N, Hq, Hkv;
    int *status;
};

__device__ __forceinline__ float e5m2_to_float(uint32_t code)
{
    // an E5M2 code is the high byte of the binary16 value it denotes
    return __half2float(__ushort_as_half((unsigned short)(code << 8)));
}

// ---------------------------------------------------------------- 1. prep
// One warp per (b, i, h) row: D = do_inv * sum_d dec(dO8) * O; zero the row of the dQ accumulator.
template <int D>
__global__ void __launch_bounds__(256) attn_bwd_prep_kernel(const uint8_t *__restrict__ dO8,
                                                            const uint16_t *__restrict__ O,
                                                            const float *__restrict__ do_inv, float *__restrict__ Dsum,
                                                            float *__restrict__ dQacc, int B, int N, int Hq)
{
    const int warps_per_block = blockDim.x >> 5;
    const long row = (long)blockIdx.x * warps_per_block + (threadIdx.x >> 5);   // (b*N + i)*Hq + h
    const int lane = threadIdx.x & 31;
    if (row >= (long)B * N * Hq) return;
    constexpr int PER = D / 32;   // elements per lane: 4 (D=128) or 2 (D=64)
    const uint8_t *pd = dO8 + row * D + lane * PER;
    const uint16_t *po = O + row * D + lane * PER;
    float acc = 0.0f;
#pragma unroll
    for (int e = 0; e < PER; ++e) acc += e5m2_to_float(pd[e]) * __uint_as_float((uint32_t)po[e] << 16);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    float *z = dQacc + row * D + lane * PER;
#pragma unroll
    for (int e = 0; e < PER; ++e) z[e] = 0.0f;
    if (lane == 0) {
        const int h = (int)(row % Hq);
        const long bi = row / Hq;
        const int i = (int)(bi % N), b = (int)(bi / N);
        Dsum[((size_t)b * Hq + h) * N + i] = acc * __ldg(do_inv);
    }
}

// ---------------------------------------------------------------- 3. finish
__global__ void __launch_bounds__(256) attn_bwd_finish_kernel(const float4 *__restrict__ acc, uint2 *__restrict__ dQ,
                                                              size_t n4, const float *__restrict__ k_inv,
                                                              const float *__restrict__ ds_scale, float softmax_scale)
{
    const float f = softmax_scale * __ldg(k_inv) / __ldg(ds_scale);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        const float4 v = acc[i];
        dQ[i] = make_uint2(pack_bf16x2(v.x * f, v.y * f), pack_bf16x2(v.z * f, v.w * f));
    }
}

// ---------------------------------------------------------------- 2. main
template <int D>
__global__ void __launch_bounds__(B_THREADS, 1)
attn_bwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                const AttnBwdParams p)
{
    using L = AttnBwdSmem<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + L::BAR_OFF;
    const uint32_t kv_full = bar0;
    auto qdo_full = [&](int s) { return bar0 + 8u * (1 + s); };
    auto qdo_empty = [&](int s) { return bar0 + 8u * (1 + B_STAGES + s); };
    const uint32_t s_full = bar0 + 8u * (1 + 2 * B_STAGES);
    const uint32_t pds_full = s_full + 8u, dq_full = s_full + 16u, dq_empty = s_full + 24u;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + L::BAR_OFF + L::N_BARS * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k_tile = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int G = p.Hq / p.Hkv;
    const int k0 = k_tile * B_BN;
    const int n_q_tiles = (p.N + B_BM - 1) / B_BM;
    const int i_first = p.causal ? k_tile : 0;            // query tiles that see this key tile
    const int per_head = n_q_tiles - i_first;
    const int n_iter = per_head * G;

    if (threadIdx.x == 0) {
        mbar_init(kv_full, 1);
        for (int s = 0; s < B_STAGES; ++s) {
            mbar_init(qdo_full(s), 1);
            mbar_init(qdo_empty(s), 1);
        }
        mbar_init(s_full, 1);
        mbar_init(pds_full, 4);
        mbar_init(dq_full, 1);
        mbar_init(dq_empty, 4);
        *abort_flag = 0;
        mbar_init_fence();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
        tma_prefetch_desc(&tm_do);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), B_TMEM_COLS);
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
            mbar_expect_tx(kv_full, 2 * L::TILE);
            tma_load_3d(sbase + L::K_OFF, &tm_k, kv_full, g * D, k0, b);
            tma_load_3d(sbase + L::V_OFF, &tm_v, kv_full, g * D, k0, b);
            for (int t = 0; t < n_iter; ++t) {
                const int st = t % B_STAGES;
                const uint32_t ph = (uint32_t)(t / B_STAGES) & 1u;
                const int h = g * G + t / per_head, q0 = (i_first + t % per_head) * B_BM;
                if (!mbar_wait(qdo_empty(st), ph ^ 1u, ctx)) break;
                const uint32_t sq = sbase + L::QDO_OFF + st * L::STAGE_BYTES, sdo = sq + L::TILE;
                mbar_expect_tx(qdo_full(st), L::STAGE_BYTES);
                tma_load_3d(sq, &tm_q, qdo_full(st), h * D, q0, b);
                tma_load_3d(sdo, &tm_do, qdo_full(st), h * D, q0, b);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            constexpr uint32_t E4 = 0, E5 = 1;
            constexpr uint32_t id_s = umma_idesc_f8(E4, E4, 128, 128, 0, 0);     // Q (K-major) x K (K-major)
            constexpr uint32_t id_dp = umma_idesc_f8(E5, E4, 128, 128, 0, 0);    // dO x V
            constexpr uint32_t id_dv = umma_idesc_f8(E4, E5, 128, D, 1, 1);      // P8^T (MN) x dO (MN)
            constexpr uint32_t id_dk = umma_idesc_f8(E5, E4, 128, D, 1, 1);      // dS8^T (MN) x Q (MN)
            constexpr uint32_t id_dq = umma_idesc_f8(E5, E4, 128, D, 0, 1);      // dS8 (K-major) x K (MN)
            const uint64_t d_k = umma_desc(sbase + L::K_OFF, D, 16);
            const uint64_t d_v = umma_desc(sbase + L::V_OFF, D, 16);
            const uint64_t d_p = umma_desc(sbase + L::P_OFF, 128, 16);
            const uint64_t d_ds = umma_desc(sbase + L::DS_OFF, 128, 16);
            constexpr uint32_t ROWS32_D = (32 * D) >> 4;        // 32 rows of a [.. x D] tile, 16-byte units
            constexpr uint32_t ROWS32_128 = (32 * 128) >> 4;    // 32 rows of a [.. x 128] tile
            bool ok = mbar_wait(kv_full, 0, ctx);
            for (int t = 0; t < n_iter && ok; ++t) {
                const int st = t % B_STAGES;
                const uint32_t ph = (uint32_t)(t / B_STAGES) & 1u;
                if (!mbar_wait(qdo_full(st), ph, ctx)) { ok = false; break; }
                if (t > 0 && !mbar_wait(dq_empty, (uint32_t)(t - 1) & 1u, ctx)) { ok = false; break; }
                tc_fence_after();
                const uint32_t sq = sbase + L::QDO_OFF + st * L::STAGE_BYTES, sdo = sq + L::TILE;
                const uint64_t d_q = umma_desc(sq, D, 16), d_do = umma_desc(sdo, D, 16);
#pragma unroll
                for (int k = 0; k < D / 32; ++k)
                    umma_f8_ss(tmem_base + L::T_S, d_q + 2u * k, d_k + 2u * k, id_s, k != 0);
#pragma unroll
                for (int k = 0; k < D / 32; ++k)
                    umma_f8_ss(tmem_base + L::T_DP, d_do + 2u * k, d_v + 2u * k, id_dp, k != 0);
                umma_commit(s_full);
                if (!mbar_wait(pds_full, (uint32_t)t & 1u, ctx)) { ok = false; break; }
                tc_fence_after();
                // reduction over the 128 queries of the tile, 32 at a time
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    umma_f8_ss(tmem_base + L::T_DV, d_p + ROWS32_128 * k, d_do + ROWS32_D * k, id_dv, (t | k) != 0);
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    umma_f8_ss(tmem_base + L::T_DK, d_ds + ROWS32_128 * k, d_q + ROWS32_D * k, id_dk, (t | k) != 0);
                // reduction over the 128 keys: 32 bytes along the dS8 rows, 32 rows of K
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    umma_f8_ss(tmem_base + L::T_S, d_ds + 2u * k, d_k + ROWS32_D * k, id_dq, k != 0);
                umma_commit(qdo_empty(st));
                umma_commit(dq_full);
            }
        }
    } else {
        // ------------------------------------------------------------ elementwise + dQ drain + epilogue
        const int quad = warp & 3;
        const int r = quad * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        const float LOG2E = 1.4426950408889634f;
        const float c = p.softmax_scale * __ldg(p.q_inv) * __ldg(p.k_inv) * LOG2E;
        const float dss = __ldg(p.ds_scale);
        const float a_dp = __ldg(p.do_inv) * __ldg(p.v_inv) * dss / p.p_scale;   // dP accumulator -> scaled dS factor
        const float b_d = dss / p.p_scale;
        uint8_t *prow = smem + L::P_OFF + r * 128;
        uint8_t *dsrow = smem + L::DS_OFF + r * 128;
        float amax = 0.0f;
        bool ok = true;
        for (int t = 0; t < n_iter; ++t) {
            const int h = g * G + t / per_head, q0 = (i_first + t % per_head) * B_BM;
            const int row = q0 + r;
            const bool row_ok = row < p.N;
            const size_t li = ((size_t)b * p.Hq + h) * p.N + (row_ok ? row : 0);
            // rows past N get P = 0 through an infinite LSE
            const float lse2 = row_ok ? __ldg(p.LSE + li) * LOG2E - p.log2_p_scale : INFINITY;
            const float db = row_ok ? __ldg(p.Dsum + li) * b_d : 0.0f;
            const int limit = min(p.causal ? row : 0x7FFFFFFF, p.N - 1) - k0;   // last valid local key
            const bool need_mask = (p.causal && k0 + B_BN - 1 > q0) || (k0 + B_BN > p.N);
            if (!mbar_wait_warp(s_full, (uint32_t)t & 1u, ctx)) { ok = false; break; }   // warp-uniform: .sync.aligned loads follow
            tc_fence_after();
#pragma unroll 1
            for (int cc = 0; cc < B_BN; cc += 32) {
                uint32_t sv[32], dv[32];
                tmem_ld_32x32b_x32(tmem_base + L::T_S + lane_addr + (uint32_t)cc, sv);
                tmem_ld_32x32b_x32(tmem_base + L::T_DP + lane_addr + (uint32_t)cc, dv);
                tmem_ld_wait();
                float pe[32], ds[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    float pv = ex2_approx(fmaf(__uint_as_float(sv[i]), c, -lse2));     // c_P * P
                    if (need_mask && cc + i > limit) pv = 0.0f;
                    pe[i] = pv;
                    ds[i] = pv * fmaf(__uint_as_float(dv[i]), a_dp, -db);              // ds_scale * dS
                    amax = fmaxf(amax, fabsf(ds[i]));
                }
                uint32_t w[8], u[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    w[i] = (uint32_t)cvt_f32x2_to_fp8x2<0>(pe[4 * i], pe[4 * i + 1]) |
                           ((uint32_t)cvt_f32x2_to_fp8x2<0>(pe[4 * i + 2], pe[4 * i + 3]) << 16);
                    u[i] = (uint32_t)cvt_f32x2_to_fp8x2<1>(ds[4 * i], ds[4 * i + 1]) |
                           ((uint32_t)cvt_f32x2_to_fp8x2<1>(ds[4 * i + 2], ds[4 * i + 3]) << 16);
                }
                const int ch = cc >> 4, sw = r & 7;
                *reinterpret_cast<uint4 *>(prow + ((ch ^ sw) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                *reinterpret_cast<uint4 *>(prow + (((ch + 1) ^ sw) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
                *reinterpret_cast<uint4 *>(dsrow + ((ch ^ sw) << 4)) = make_uint4(u[0], u[1], u[2], u[3]);
                *reinterpret_cast<uint4 *>(dsrow + (((ch + 1) ^ sw) << 4)) = make_uint4(u[4], u[5], u[6], u[7]);
            }
            tc_fence_before();
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(pds_full);
            // drain the dQ tile of this pair into the FP32 accumulator
            if (!mbar_wait_warp(dq_full, (uint32_t)t & 1u, ctx)) { ok = false; break; }
            tc_fence_after();
            float *qacc = p.dQacc + (((size_t)b * p.N + (row_ok ? row : 0)) * p.Hq + h) * D;
#pragma unroll 1
            for (int cc = 0; cc < D; cc += 32) {
                uint32_t v[32];
                tmem_ld_32x32b_x32(tmem_base + L::T_S + lane_addr + (uint32_t)cc, v);
                tmem_ld_wait();
                if (row_ok) {
#pragma unroll
                    for (int i = 0; i < 32; i += 4)
                        asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(qacc + cc + i),
                                     "f"(__uint_as_float(v[i])), "f"(__uint_as_float(v[i + 1])),
                                     "f"(__uint_as_float(v[i + 2])), "f"(__uint_as_float(v[i + 3]))
                                     : "memory");
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(dq_empty);
        }
        // ---- epilogue: dK, dV rows of this key tile (TMEM lane = key); the last dq_full covers every MMA
        if (ok) {
            const int key = k0 + r;
            const float f_dv = __ldg(p.do_inv) / p.p_scale;
            const float f_dk = p.softmax_scale * __ldg(p.q_inv) / dss;
            const size_t orow = (((size_t)b * p.N + key) * p.Hkv + g) * D;
#pragma unroll 1
            for (int which = 0; which < 2; ++which) {
                const uint32_t tcol = which == 0 ? L::T_DV : L::T_DK;
                const float f = which == 0 ? f_dv : f_dk;
                uint16_t *dst = (which == 0 ? p.dV : p.dK) + orow;
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
            }
            if (p.ds_amax) {
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 16));
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 8));
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 4));
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
                // the kernel tracked ds_scale * |dS|; non-negative floats order like unsigned integers
                if (lane == 0) atomicMax(reinterpret_cast<unsigned int *>(p.ds_amax), __float_as_uint(amax / dss));
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
        tmem_dealloc(tmem_base, B_TMEM_COLS);
    }
}

static size_t bwd_ws_bytes(int B, int N, int Hq, int d)
{
    if (d == 128) return attn_bwd_d128_ws_bytes(B, N, Hq);
    const size_t acc = (size_t)B * N * Hq * d * sizeof(float);
    const size_t dsum = (((size_t)B * Hq * N * sizeof(float)) + 255) & ~(size_t)255;
    return acc + dsum;
}

template <int D>
static int launch_attn_bwd(const uint8_t *Q8, const uint8_t *K8, const uint8_t *V8, const uint8_t *dO8,
                           const uint16_t *O, uint16_t *dQ, AttnBwdParams p, float *dsum, cudaStream_t st)
{
    CUtensorMap tq, tk, tv, tdo;
    int rc = make_tmap_3d_u8(&tq, Q8, (uint64_t)p.Hq * D, (uint64_t)p.N, (uint64_t)p.B, D, B_BM);
    if (rc != FP8_OK) return rc;
    rc = make_tmap_3d_u8(&tk, K8, (uint64_t)p.Hkv * D, (uint64_t)p.N, (uint64_t)p.B, D, B_BN);
    if (rc != FP8_OK) return rc;
    rc = make_tmap_3d_u8(&tv, V8, (uint64_t)p.Hkv * D, (uint64_t)p.N, (uint64_t)p.B, D, B_BN);
    if (rc != FP8_OK) return rc;
    rc = make_tmap_3d_u8(&tdo, dO8, (uint64_t)p.Hq * D, (uint64_t)p.N, (uint64_t)p.B, D, B_BM);
    if (rc != FP8_OK) return rc;
    if (p.ds_amax) FP8_CUDA_CHECK(cudaMemsetAsync(p.ds_amax, 0, sizeof(float), st));
    const long rows = (long)p.B * p.N * p.Hq;
    attn_bwd_prep_kernel<D><<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(dO8, O, p.do_inv, dsum, p.dQacc, p.B, p.N, p.Hq);
    FP8_CUDA_CHECK(cudaGetLastError());
    FP8_CUDA_CHECK(cudaFuncSetAttribute(attn_bwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        AttnBwdSmem<D>::DYN_BYTES));
    dim3 grid((unsigned)((p.N + B_BN - 1) / B_BN), (unsigned)p.Hkv, (unsigned)p.B);
    attn_bwd_kernel<D><<<grid, B_THREADS, AttnBwdSmem<D>::DYN_BYTES, st>>>(tq, tk, tv, tdo, p);
    FP8_CUDA_CHECK(cudaGetLastError());
    const size_t n4 = (size_t)rows * D / 4;
    size_t blocks = (n4 + 255) / 256;
    const size_t cap = (size_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    attn_bwd_finish_kernel<<<(unsigned)blocks, 256, 0, st>>>(reinterpret_cast<const float4 *>(p.dQacc),
                                                            reinterpret_cast<uint2 *>(dQ), n4, p.k_inv, p.ds_scale,
                                                            p.softmax_scale);
    FP8_CUDA_CHECK(cudaGetLastError());
    return FP8_OK;
}

}  // namespace fp8dpa

using namespace fp8dpa;

extern "C" size_t fp8_attention_workspace_bytes(int op, int B, int N, int Hq, int Hkv, int d)
{
    (void)Hkv;
    if (op == 0 || B <= 0 || N <= 0 || Hq <= 0 || d <= 0) return 0;
    return bwd_ws_bytes(B, N, Hq, d);
}

extern "C" int fp8_attention_bwd(const uint8_t *Q8, const uint8_t *K8, const uint8_t *V8, const uint8_t *dO8,
                                 const void *O_bf16, const float *LSE, const fp8_attn_scales *sc, int causal, int B,
                                 int N, int Hq, int Hkv, int d, void *dQ_bf16, void *dK_bf16, void *dV_bf16, void *ws,
                                 size_t ws_bytes, void *stream)
{
    int rc = validate_attn("fp8_attention_bwd", Q8, K8, V8, sc, B, N, Hq, Hkv, d);
    if (rc != FP8_OK) return rc;
    if (!dO8 || !O_bf16 || !LSE || !dQ_bf16 || !dK_bf16 || !dV_bf16 || !sc->do_inv || !sc->ds_scale) {
        set_error("fp8_attention_bwd: NULL pointer");
        return FP8_ERR_NULL;
    }
    if (!aligned16(dO8) || !aligned16(O_bf16) || !aligned16(dQ_bf16) || !aligned16(dK_bf16) || !aligned16(dV_bf16)) {
        set_error("fp8_attention_bwd: tensor pointers must be 16-byte aligned");
        return FP8_ERR_ALIGN;
    }
    const size_t need = bwd_ws_bytes(B, N, Hq, d);
    if (!ws || ws_bytes < need || (reinterpret_cast<uintptr_t>(ws) & 255u)) {
        set_error("fp8_attention_bwd: workspace must be 256-byte aligned and hold %zu bytes (got %p, %zu)", need, ws,
                  ws_bytes);
        return FP8_ERR_WORKSPACE;
    }
    rc = check_arch();
    if (rc != FP8_OK) return rc;
    AttnBwdParams p;
    float *dsum = static_cast<float *>(ws);
    const size_t dsum_bytes = (((size_t)B * Hq * N * sizeof(float)) + 255) & ~(size_t)255;
    p.LSE = LSE;
    p.Dsum = dsum;
    p.dQacc = reinterpret_cast<float *>(static_cast<uint8_t *>(ws) + dsum_bytes);
    p.dK = static_cast<uint16_t *>(dK_bf16);
    p.dV = static_cast<uint16_t *>(dV_bf16);
    p.q_inv = sc->q_inv; p.k_inv = sc->k_inv; p.v_inv = sc->v_inv; p.do_inv = sc->do_inv;
    p.ds_scale = sc->ds_scale;
    p.ds_amax = sc->ds_amax;
    p.softmax_scale = sc->softmax_scale;
    p.p_scale = sc->p_scale;
    p.log2_p_scale = log2f(sc->p_scale);
    p.causal = causal ? 1 : 0;
    p.B = B; p.N = N; p.Hq = Hq; p.Hkv = Hkv;
    p.status = device_status_ptr();
    if (!p.status) return FP8_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint16_t *O = static_cast<const uint16_t *>(O_bf16);
    uint16_t *dQ = static_cast<uint16_t *>(dQ_bf16);
    if (d == 128)
        return launch_attn_bwd_d128(Q8, K8, V8, dO8, O, LSE, sc, causal, B, N, Hq, Hkv, dQ, p.dK, p.dV, ws, p.status, st);
    return launch_attn_bwd<64>(Q8, K8, V8, dO8, O, dQ, p, dsum, st);
}
