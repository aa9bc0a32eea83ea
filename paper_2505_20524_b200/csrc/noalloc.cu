// Attention backward for callers that cannot provide device scratch.
//
// fp8_attention_bwd needs scratch in global memory (the FP32 dQ accumulator and the row sums D).  Some
// callers have no way to hand it over: code running inside a memory pool that is already fully committed,
// a plugin that is only given its input and output buffers, a host process whose allocator must not be
// re-entered from the thread that launches work.  For them the scratch lives in a fixed array inside the
// library's device image.
#include "common.cuh"

namespace fp8dpa {

// Held by every GPU that loads the library, from module load until the process exits.
static __device__ __align__(256) unsigned char g_bwd_static_scratch[FP8_STATIC_SCRATCH_BYTES];

// In host code the array's name is only a handle for the runtime, not a device address; the address a
// kernel can use comes from cudaGetSymbolAddress, per device.
static const int kMaxDev = 64;
static void *g_scratch_ptr[kMaxDev] = {nullptr};

static int static_scratch(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) {
        set_error("fp8_attention_bwd_static: no current CUDA device");
        return FP8_ERR_CUDA;
    }
    if (!g_scratch_ptr[dev]) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_bwd_static_scratch);
        if (e != cudaSuccess || !p) {
            set_error("fp8_attention_bwd_static: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
            return FP8_ERR_CUDA;
        }
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return FP8_OK;
}

}  // namespace fp8dpa

using namespace fp8dpa;

extern "C" int fp8_attention_bwd_static(const uint8_t *Q8, const uint8_t *K8, const uint8_t *V8, const uint8_t *dO8,
                                        const void *O_bf16, const float *LSE, const fp8_attn_scales *sc, int causal,
                                        int B, int N, int Hq, int Hkv, int d, void *dQ_bf16, void *dK_bf16,
                                        void *dV_bf16, void *stream)
{
    const size_t need = fp8_attention_workspace_bytes(1, B, N, Hq, Hkv, d);
    if (need == 0) {
        set_error("fp8_attention_bwd_static: unsupported shape B=%d N=%d Hq=%d Hkv=%d d=%d", B, N, Hq, Hkv, d);
        return FP8_ERR_SHAPE;
    }
    if (need > (size_t)FP8_STATIC_SCRATCH_BYTES) {
        set_error("fp8_attention_bwd_static: this problem needs %zu bytes of scratch but the built-in array holds %zu "
                  "(about B*N*Hq*(d+8)*4 must not exceed it); use fp8_attention_bwd with a caller workspace",
                  need, (size_t)FP8_STATIC_SCRATCH_BYTES);
        return FP8_ERR_WORKSPACE;
    }
    void *scratch = nullptr;
    int rc = static_scratch(&scratch);
    if (rc != FP8_OK) return rc;
    // The first launch zeroes the accumulator part and overwrites the row sums, so whatever an earlier
    // call left in the array does not matter.
    return fp8_attention_bwd(Q8, K8, V8, dO8, O_bf16, LSE, sc, causal, B, N, Hq, Hkv, d, dQ_bf16, dK_bf16, dV_bf16,
                             scratch, need, stream);
}
