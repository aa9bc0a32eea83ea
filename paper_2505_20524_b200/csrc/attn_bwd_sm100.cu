// placeholder until the backward kernel lands
#include "common.cuh"
using namespace fp8dpa;
extern "C" size_t fp8_attention_workspace_bytes(int op, int B, int N, int Hq, int Hkv, int d)
{
    (void)Hkv;
    if (op == 0) return 0;
    return (size_t)B * N * Hq * d * 4 + (size_t)B * Hq * N * 4;
}
extern "C" int fp8_attention_bwd(const uint8_t *, const uint8_t *, const uint8_t *, const uint8_t *, const void *,
                                 const float *, const fp8_attn_scales *, int, int, int, int, int, int, void *, void *,
                                 void *, void *, size_t, void *)
{
    set_error("fp8_attention_bwd: not built yet");
    return FP8_ERR_CUDA;
}
