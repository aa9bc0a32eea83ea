// Host-buffer forms of the hot path: one linear layer (quantize x 3, forward, data gradient, weight gradient) or one
// attention (quantize x 4, forward, backward) from BF16 tensors in pinned HOST memory to results in pinned HOST
// memory, through a device workspace the caller provides.  Nothing here computes: the calls below only move bytes and
// chain the device-pointer entry points of this library on three internal streams (uploads, kernels, downloads), so
// that the copies of one call run under the kernels of another and under the copies in the other direction.
//
// Ordering.  A call returns when its work is enqueued; fp8_host_sync() waits for everything.  A workspace may be
// handed to the next call at once: the library remembers, per workspace address, the event after which its previous
// results have left the device and its previous kernels have read their inputs, and makes the new uploads and kernels
// wait for it.  Host buffers must stay untouched until fp8_host_sync() returns.
#include <map>
#include <mutex>

#include "common.cuh"

namespace fp8dpa {
namespace {

struct HostCtx {
    cudaStream_t up = nullptr, main = nullptr, down = nullptr;
    std::map<const void *, cudaEvent_t> last_use;      // workspace -> downloads of its previous call have finished
    std::map<const void *, cudaEvent_t> last_main;     // workspace -> kernels of its previous call have finished
};
std::mutex g_mu;
HostCtx g_ctx[64];

__global__ void set_scalar_kernel(float *p, float v) { *p = v; }

int host_ctx(HostCtx **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        set_error("host step: no current CUDA device");
        return FP8_ERR_CUDA;
    }
    HostCtx &c = g_ctx[dev];
    if (!c.up) {
        FP8_CUDA_CHECK(cudaStreamCreateWithFlags(&c.up, cudaStreamNonBlocking));
        FP8_CUDA_CHECK(cudaStreamCreateWithFlags(&c.main, cudaStreamNonBlocking));
        FP8_CUDA_CHECK(cudaStreamCreateWithFlags(&c.down, cudaStreamNonBlocking));
    }
    *out = &c;
    return FP8_OK;
}

// the new call's uploads and kernels wait for the previous use of the same workspace
int begin_use(HostCtx &c, const void *ws)
{
    auto it = c.last_use.find(ws);
    if (it != c.last_use.end()) {
        FP8_CUDA_CHECK(cudaStreamWaitEvent(c.main, it->second, 0));       // results have been copied out
    }
    auto im = c.last_main.find(ws);
    if (im != c.last_main.end()) {
        FP8_CUDA_CHECK(cudaStreamWaitEvent(c.up, im->second, 0));         // inputs have been read
    }
    return FP8_OK;
}

int remember(std::map<const void *, cudaEvent_t> &m, const void *ws, cudaStream_t s)
{
    cudaEvent_t &e = m[ws];
    if (!e) FP8_CUDA_CHECK(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    FP8_CUDA_CHECK(cudaEventRecord(e, s));
    return FP8_OK;
}

struct Carve {
    uint8_t *p;
    size_t left;
    void *take(size_t bytes)
    {
        bytes = (bytes + 255) & ~(size_t)255;
        if (bytes > left) return nullptr;
        void *r = p;
        p += bytes;
        left -= bytes;
        return r;
    }
};

size_t up256(size_t b) { return (b + 255) & ~(size_t)255; }

}  // namespace
}  // namespace fp8dpa

using namespace fp8dpa;

extern "C" size_t fp8_linear_step_host_workspace_bytes(int T, int N, int K)
{
    if (T <= 0 || N <= 0 || K <= 0) return 0;
    const size_t tk = (size_t)T * K, nk = (size_t)N * K, tn = (size_t)T * N;
    // BF16 inputs, FP8 copies, BF16 outputs, 9 scalars
    return up256(2 * tk) + up256(2 * nk) + up256(2 * tn) + up256(tk) + up256(nk) + up256(tn) + up256(2 * tn) + up256(2 * tk) +
           up256(2 * nk) + 256;
}

extern "C" int fp8_linear_step_host(const void *hX, const void *hW, const void *hdY, int T, int N, int K, void *hY, void *hdX,
                                    void *hdW, void *ws, size_t ws_bytes)
{
    if (!hX || !hW || !hdY || !hY || !hdX || !hdW || !ws) {
        set_error("fp8_linear_step_host: NULL pointer");
        return FP8_ERR_NULL;
    }
    const size_t need = fp8_linear_step_host_workspace_bytes(T, N, K);
    if (need == 0 || (K % 16) || (N % 16) || (T % 16)) {
        set_error("fp8_linear_step_host: unsupported shape T=%d N=%d K=%d (multiples of 16)", T, N, K);
        return FP8_ERR_SHAPE;
    }
    if (ws_bytes < need || (reinterpret_cast<uintptr_t>(ws) & 255u)) {
        set_error("fp8_linear_step_host: workspace of %zu bytes (256-byte aligned) needed, %zu given", need, ws_bytes);
        return FP8_ERR_WORKSPACE;
    }
    std::lock_guard<std::mutex> lock(g_mu);
    HostCtx *c = nullptr;
    int rc = host_ctx(&c);
    if (rc != FP8_OK) return rc;
    const size_t tk = (size_t)T * K, nk = (size_t)N * K, tn = (size_t)T * N;
    Carve cv{static_cast<uint8_t *>(ws), ws_bytes};
    void *x = cv.take(2 * tk), *w = cv.take(2 * nk), *dy = cv.take(2 * tn);
    uint8_t *x8 = static_cast<uint8_t *>(cv.take(tk)), *w8 = static_cast<uint8_t *>(cv.take(nk)),
            *dy8 = static_cast<uint8_t *>(cv.take(tn));
    void *y = cv.take(2 * tn), *dx = cv.take(2 * tk), *dw = cv.take(2 * nk);
    float *sc = static_cast<float *>(cv.take(9 * sizeof(float)));
    if (!sc) {
        set_error("fp8_linear_step_host: workspace too small");
        return FP8_ERR_WORKSPACE;
    }
    rc = begin_use(*c, ws);
    if (rc != FP8_OK) return rc;
    cudaEvent_t up_done;
    FP8_CUDA_CHECK(cudaMemcpyAsync(x, hX, 2 * tk, cudaMemcpyHostToDevice, c->up));
    FP8_CUDA_CHECK(cudaMemcpyAsync(w, hW, 2 * nk, cudaMemcpyHostToDevice, c->up));
    FP8_CUDA_CHECK(cudaMemcpyAsync(dy, hdY, 2 * tn, cudaMemcpyHostToDevice, c->up));
    FP8_CUDA_CHECK(cudaEventCreateWithFlags(&up_done, cudaEventDisableTiming));
    FP8_CUDA_CHECK(cudaEventRecord(up_done, c->up));
    FP8_CUDA_CHECK(cudaStreamWaitEvent(c->main, up_done, 0));
    FP8_CUDA_CHECK(cudaEventDestroy(up_done));                  // released once the wait has consumed it
    // amax, scale, scale_inv of x, w, dy
    {
        const fp8_quant_item items[3] = {{x, tk, FP8_E4M3, x8}, {w, nk, FP8_E4M3, w8}, {dy, tn, FP8_E5M2, dy8}};
        rc = fp8_quantize_multi(items, 3, sc, c->main);
    }
    if (rc == FP8_OK) rc = fp8_linear_fwd(x8, w8, sc + 2, sc + 5, y, 0, T, N, K, nullptr, 0, c->main);
    if (rc == FP8_OK) rc = fp8_linear_dgrad_rm(dy8, w8, sc + 8, sc + 5, dx, 0, T, N, K, c->main);
    if (rc == FP8_OK) rc = fp8_linear_wgrad_rm(dy8, x8, sc + 8, sc + 2, dw, 0, 0, T, N, K, c->main);
    if (rc != FP8_OK) return rc;
    rc = remember(c->last_main, ws, c->main);
    if (rc != FP8_OK) return rc;
    FP8_CUDA_CHECK(cudaStreamWaitEvent(c->down, c->last_main[ws], 0));
    FP8_CUDA_CHECK(cudaMemcpyAsync(hY, y, 2 * tn, cudaMemcpyDeviceToHost, c->down));
    FP8_CUDA_CHECK(cudaMemcpyAsync(hdX, dx, 2 * tk, cudaMemcpyDeviceToHost, c->down));
    FP8_CUDA_CHECK(cudaMemcpyAsync(hdW, dw, 2 * nk, cudaMemcpyDeviceToHost, c->down));
    return remember(c->last_use, ws, c->down);
}

extern "C" size_t fp8_attention_step_host_workspace_bytes(int B, int N, int Hq, int Hkv, int d)
{
    if (B <= 0 || N <= 0 || (N % 16) || Hq <= 0 || Hkv <= 0 || (Hq % Hkv) || (d != 64 && d != 128)) return 0;
    const size_t bwd = fp8_attention_workspace_bytes(1, B, N, Hq, Hkv, d);
    if (bwd == 0) return 0;
    const size_t q = (size_t)B * N * Hq * d, kv = (size_t)B * N * Hkv * d;
    // BF16 q, k, v, do; FP8 copies; O, dQ, dK, dV BF16; LSE; backward scratch; scalars
    return 2 * up256(2 * q) + 2 * up256(2 * kv) + 2 * up256(q) + 2 * up256(kv) + 2 * up256(2 * q) + 2 * up256(2 * kv) +
           up256((size_t)B * Hq * N * 4) + up256(bwd) + 256;
}

extern "C" int fp8_attention_step_host(const void *hQ, const void *hK, const void *hV, const void *hdO, int B, int N, int Hq,
                                       int Hkv, int d, float softmax_scale, float ds_scale, int causal, void *hO, float *hLSE,
                                       void *hdQ, void *hdK, void *hdV, void *ws, size_t ws_bytes)
{
    if (!hQ || !hK || !hV || !hdO || !hO || !hLSE || !hdQ || !hdK || !hdV || !ws) {
        set_error("fp8_attention_step_host: NULL pointer");
        return FP8_ERR_NULL;
    }
    const size_t need = fp8_attention_step_host_workspace_bytes(B, N, Hq, Hkv, d);
    if (need == 0) {
        set_error("fp8_attention_step_host: unsupported shape B=%d N=%d Hq=%d Hkv=%d d=%d", B, N, Hq, Hkv, d);
        return FP8_ERR_SHAPE;
    }
    if (ws_bytes < need || (reinterpret_cast<uintptr_t>(ws) & 255u)) {
        set_error("fp8_attention_step_host: workspace of %zu bytes (256-byte aligned) needed, %zu given", need, ws_bytes);
        return FP8_ERR_WORKSPACE;
    }
    std::lock_guard<std::mutex> lock(g_mu);
    HostCtx *c = nullptr;
    int rc = host_ctx(&c);
    if (rc != FP8_OK) return rc;
    const size_t nq = (size_t)B * N * Hq * d, nkv = (size_t)B * N * Hkv * d, nl = (size_t)B * Hq * N;
    const size_t bwd = fp8_attention_workspace_bytes(1, B, N, Hq, Hkv, d);
    Carve cv{static_cast<uint8_t *>(ws), ws_bytes};
    void *q = cv.take(2 * nq), *dO = cv.take(2 * nq), *k = cv.take(2 * nkv), *v = cv.take(2 * nkv);
    uint8_t *q8 = static_cast<uint8_t *>(cv.take(nq)), *do8 = static_cast<uint8_t *>(cv.take(nq)),
            *k8 = static_cast<uint8_t *>(cv.take(nkv)), *v8 = static_cast<uint8_t *>(cv.take(nkv));
    void *o = cv.take(2 * nq), *dq = cv.take(2 * nq), *dk = cv.take(2 * nkv), *dv = cv.take(2 * nkv);
    float *lse = static_cast<float *>(cv.take(nl * 4));
    void *scratch = cv.take(bwd);
    float *sc = static_cast<float *>(cv.take(14 * sizeof(float)));
    if (!sc) {
        set_error("fp8_attention_step_host: workspace too small");
        return FP8_ERR_WORKSPACE;
    }
    rc = begin_use(*c, ws);
    if (rc != FP8_OK) return rc;
    cudaEvent_t up_done;
    FP8_CUDA_CHECK(cudaMemcpyAsync(q, hQ, 2 * nq, cudaMemcpyHostToDevice, c->up));
    FP8_CUDA_CHECK(cudaMemcpyAsync(k, hK, 2 * nkv, cudaMemcpyHostToDevice, c->up));
    FP8_CUDA_CHECK(cudaMemcpyAsync(v, hV, 2 * nkv, cudaMemcpyHostToDevice, c->up));
    FP8_CUDA_CHECK(cudaMemcpyAsync(dO, hdO, 2 * nq, cudaMemcpyHostToDevice, c->up));
    FP8_CUDA_CHECK(cudaEventCreateWithFlags(&up_done, cudaEventDisableTiming));
    FP8_CUDA_CHECK(cudaEventRecord(up_done, c->up));
    FP8_CUDA_CHECK(cudaStreamWaitEvent(c->main, up_done, 0));
    FP8_CUDA_CHECK(cudaEventDestroy(up_done));
    // scalars: (amax, scale, scale_inv) of q, k, v, do; then ds_scale and ds_amax
    {
        const fp8_quant_item items[4] = {{q, nq, FP8_E4M3, q8}, {k, nkv, FP8_E4M3, k8}, {v, nkv, FP8_E4M3, v8}, {dO, nq, FP8_E5M2, do8}};
        rc = fp8_quantize_multi(items, 4, sc, c->main);
    }
    if (rc != FP8_OK) return rc;
    set_scalar_kernel<<<1, 1, 0, c->main>>>(sc + 12, ds_scale);
    FP8_CUDA_CHECK(cudaGetLastError());
    fp8_attn_scales as;
    as.q_inv = sc + 2; as.k_inv = sc + 5; as.v_inv = sc + 8; as.do_inv = sc + 11;
    as.softmax_scale = softmax_scale;
    as.p_scale = 448.0f;
    as.ds_scale = sc + 12;
    as.ds_amax = sc + 13;
    as.max_slack = 0.0f;
    rc = fp8_attention_fwd(q8, k8, v8, &as, causal, B, N, Hq, Hkv, d, o, lse, nullptr, 0, c->main);
    if (rc == FP8_OK)
        rc = fp8_attention_bwd(q8, k8, v8, do8, o, lse, &as, causal, B, N, Hq, Hkv, d, dq, dk, dv, scratch, bwd, c->main);
    if (rc != FP8_OK) return rc;
    rc = remember(c->last_main, ws, c->main);
    if (rc != FP8_OK) return rc;
    FP8_CUDA_CHECK(cudaStreamWaitEvent(c->down, c->last_main[ws], 0));
    FP8_CUDA_CHECK(cudaMemcpyAsync(hO, o, 2 * nq, cudaMemcpyDeviceToHost, c->down));
    FP8_CUDA_CHECK(cudaMemcpyAsync(hLSE, lse, nl * 4, cudaMemcpyDeviceToHost, c->down));
    FP8_CUDA_CHECK(cudaMemcpyAsync(hdQ, dq, 2 * nq, cudaMemcpyDeviceToHost, c->down));
    FP8_CUDA_CHECK(cudaMemcpyAsync(hdK, dk, 2 * nkv, cudaMemcpyDeviceToHost, c->down));
    FP8_CUDA_CHECK(cudaMemcpyAsync(hdV, dv, 2 * nkv, cudaMemcpyDeviceToHost, c->down));
    return remember(c->last_use, ws, c->down);
}

extern "C" int fp8_host_sync(void)
{
    std::lock_guard<std::mutex> lock(g_mu);
    HostCtx *c = nullptr;
    int rc = host_ctx(&c);
    if (rc != FP8_OK) return rc;
    FP8_CUDA_CHECK(cudaStreamSynchronize(c->up));
    FP8_CUDA_CHECK(cudaStreamSynchronize(c->main));
    FP8_CUDA_CHECK(cudaStreamSynchronize(c->down));
    return FP8_OK;
}
