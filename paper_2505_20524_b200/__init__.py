"""FP8 transformer-block hot path for one B200 (sm_100a): per-tensor quantize, FP8 linear GEMMs and FP8
attention behind a C ABI (``include/fp8dpa.h``), with a thin Python binding of the same names.

``binding``  the C-ABI calls (ctypes; torch only supplies device memory and streams)
``synth``    seeded synthetic inputs shaped like the paper's workloads
``build``    compiles ``csrc/*.cu`` into ``csrc/libfp8dpa.so``
"""
from . import binding  # noqa: F401
from .binding import (ACT_GELU, ACT_XIELU, E4M3, E5M2, FP8_BLOCK_128x1, NORM_LAYERSCALE, NORM_RMS, QK_NONE, QK_RMS, QK_TANH,  # noqa: F401
                      Fp8Error, fp8_act_cast, fp8_amax, fp8_attention_bwd, fp8_attention_bwd_static,
                      fp8_attention_fwd, fp8_attention_fwd_q, fp8_attention_workspace_bytes, fp8_cast,
                      fp8_device_status, fp8_grouped_linear_dgrad, fp8_grouped_linear_fwd, fp8_grouped_linear_wgrad, fp8_grouped_linear_wgrad_dev, fp8_grouped_linear_wgrad_workspace_bytes, fp8_kurtosis, fp8_amax_kurtosis, fp8_last_error, fp8_linear_dgrad,
                      fp8_linear_dgrad_q, fp8_linear_dgrad_rm, fp8_linear_fwd, fp8_linear_fwd_blockwise,
                      fp8_linear_dgrad_blockwise, fp8_linear_wgrad_blockwise,
                      fp8_linear_fwd_q, fp8_linear_wgrad, fp8_linear_wgrad_rm, fp8_postnorm_residual, fp8_postnorm_residual_q,
                      fp8_qk_norm_rope, fp8_qk_norm_rope_q, fp8_quantize, fp8_quantize_multi, fp8_quantize_delayed_multi, fp8_quantize_blockwise, fp8_scale, fp8_scale_update,
                      fp8_selftest_wait_timeout, fp8_swiglu_cast, fp8_linear_step_host, fp8_linear_step_host_workspace_bytes,
                      fp8_attention_step_host, fp8_attention_step_host_workspace_bytes, fp8_host_sync)
