"""ctypes binding of ``libfp8dpa.so`` with the names of ``include/fp8dpa.h``.

Argument marshalling only: every function takes torch CUDA tensors (device memory and streams are torch's),
passes their addresses through the C ABI and raises ``Fp8Error`` on a non-zero status.  There is no
fallback of any kind: if the CUDA library is missing or fails to load, importing is fine but the first
call raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

E4M3 = 0
E5M2 = 1
FP8_BLOCK_128x1 = -128        # block_rows value of fp8_quantize_blockwise: 128 consecutive rows of one column

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "csrc", "libfp8dpa.so")
_lib = None

SYMBOLS = ["fp8_last_error", "fp8_device_status", "fp8_selftest_wait_timeout", "fp8_amax", "fp8_scale", "fp8_scale_update", "fp8_cast",
           "fp8_quantize", "fp8_quantize_multi", "fp8_quantize_delayed_multi", "fp8_swiglu_cast", "fp8_act_cast", "fp8_postnorm_residual", "fp8_postnorm_residual_q", "fp8_qk_norm_rope", "fp8_qk_norm_rope_q", "fp8_kurtosis", "fp8_amax_kurtosis",
           "fp8_linear_fwd", "fp8_linear_dgrad", "fp8_linear_wgrad", "fp8_linear_fwd_q", "fp8_linear_dgrad_q", "fp8_linear_dgrad_rm", "fp8_linear_wgrad_rm", "fp8_grouped_linear_fwd", "fp8_grouped_linear_dgrad", "fp8_grouped_linear_wgrad", "fp8_grouped_linear_wgrad_workspace_bytes", "fp8_grouped_linear_wgrad_dev", "fp8_quantize_blockwise", "fp8_linear_fwd_blockwise", "fp8_linear_dgrad_blockwise", "fp8_linear_wgrad_blockwise", "fp8_attention_workspace_bytes",
           "fp8_attention_fwd", "fp8_attention_fwd_q", "fp8_attention_bwd", "fp8_attention_bwd_static",
           "fp8_linear_step_host_workspace_bytes", "fp8_linear_step_host", "fp8_attention_step_host_workspace_bytes",
           "fp8_attention_step_host", "fp8_host_sync"]

STATIC_SCRATCH_BYTES = 32 << 20

STATUS_NAMES = {0: "FP8_OK", -1: "FP8_ERR_NULL", -2: "FP8_ERR_ALIGN", -3: "FP8_ERR_SHAPE", -4: "FP8_ERR_ENUM",
                -5: "FP8_ERR_WORKSPACE", -6: "FP8_ERR_CUDA", -7: "FP8_ERR_TIMEOUT", -8: "FP8_ERR_ARCH"}


class Fp8Error(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {msg}")
        self.status = status


class AttnScales(C.Structure):
    _fields_ = [("q_inv", C.c_void_p), ("k_inv", C.c_void_p), ("v_inv", C.c_void_p), ("do_inv", C.c_void_p),
                ("softmax_scale", C.c_float), ("p_scale", C.c_float),
                ("ds_scale", C.c_void_p), ("ds_amax", C.c_void_p), ("max_slack", C.c_float)]


def load() -> C.CDLL:
    """Loads the CUDA library; raises if it has not been built (there is nothing to fall back to)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2505_20524_b200.build`")
        lib = C.CDLL(LIB_PATH)
        lib.fp8_last_error.restype = C.c_char_p
        if hasattr(lib, "fp8_attention_workspace_bytes"):
            lib.fp8_attention_workspace_bytes.restype = C.c_size_t
            lib.fp8_attention_workspace_bytes.argtypes = [C.c_int] * 6
        if hasattr(lib, "fp8_grouped_linear_wgrad_workspace_bytes"):
            lib.fp8_grouped_linear_wgrad_workspace_bytes.restype = C.c_size_t
            lib.fp8_grouped_linear_wgrad_workspace_bytes.argtypes = [C.c_int] * 2
        if hasattr(lib, "fp8_linear_step_host_workspace_bytes"):
            lib.fp8_linear_step_host_workspace_bytes.restype = C.c_size_t
            lib.fp8_linear_step_host_workspace_bytes.argtypes = [C.c_int] * 3
            lib.fp8_attention_step_host_workspace_bytes.restype = C.c_size_t
            lib.fp8_attention_step_host_workspace_bytes.argtypes = [C.c_int] * 5
        _lib = lib
    return _lib


def _check(rc: int):
    if rc != 0:
        raise Fp8Error(rc, load().fp8_last_error().decode())


def _ptr(t):
    if t is None:
        return C.c_void_p(0)
    assert t.is_cuda and t.is_contiguous(), "expects contiguous CUDA tensors"
    return C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def fp8_last_error() -> str:
    return load().fp8_last_error().decode()


def fp8_device_status(stream=None) -> int:
    out = C.c_int(0)
    _check(load().fp8_device_status(C.byref(out), _stream(stream)))
    return out.value


def fp8_selftest_wait_timeout(limit_cycles, gave_up, stream=None):
    """One warp waits on a barrier nothing completes and gives up after limit_cycles: status word = FP8_ERR_TIMEOUT."""
    _check(load().fp8_selftest_wait_timeout(C.c_longlong(int(limit_cycles)), _ptr(gave_up), _stream(stream)))


def fp8_amax(x, amax, stream=None):
    _check(load().fp8_amax(_ptr(x), C.c_size_t(x.numel()), _ptr(amax), _stream(stream)))


def fp8_scale(amax, fmt, margin, scale, scale_inv, stream=None):
    _check(load().fp8_scale(_ptr(amax), C.c_int(fmt), C.c_int(margin), _ptr(scale), _ptr(scale_inv), _stream(stream)))


def fp8_scale_update(history, head, amax_new, fmt, margin, scale, scale_inv, stream=None):
    """Delayed scaling: push *amax_new into the FIFO `history` (float32 CUDA tensor, `head` an int32 CUDA scalar)
    and recompute scale / scale_inv from the updated history."""
    _check(load().fp8_scale_update(_ptr(history), C.c_int(history.numel()), _ptr(head), _ptr(amax_new), C.c_int(fmt),
                                   C.c_int(margin), _ptr(scale), _ptr(scale_inv), _stream(stream)))


def _rows_cols(x):
    if x.dim() == 1:
        return 1, x.numel()
    return x.numel() // x.shape[-1], x.shape[-1]


def fp8_cast(x, scale, fmt, out, out_t=None, amax_out=None, stream=None):
    rows, cols = _rows_cols(x)
    _check(load().fp8_cast(_ptr(x), C.c_size_t(rows), C.c_size_t(cols), _ptr(scale), C.c_int(fmt), _ptr(out),
                           _ptr(out_t), _ptr(amax_out), _stream(stream)))


def fp8_quantize(x, fmt, out, out_t, amax, scale, scale_inv, stream=None):
    rows, cols = _rows_cols(x)
    _check(load().fp8_quantize(_ptr(x), C.c_size_t(rows), C.c_size_t(cols), C.c_int(fmt), _ptr(out), _ptr(out_t),
                               _ptr(amax), _ptr(scale), _ptr(scale_inv), _stream(stream)))


class QuantItem(C.Structure):
    _fields_ = [("x_bf16", C.c_void_p), ("n", C.c_size_t), ("fmt", C.c_int), ("out", C.c_void_p)]


def fp8_quantize_multi(xs, fmts, outs, scalars, stream=None):
    """Just-in-time quantize of up to 8 tensors in two launches: xs BF16 CUDA tensors, outs uint8 CUDA tensors of the same
    sizes, scalars a float32 CUDA tensor of 3 * len(xs) entries receiving (amax, scale, 1 / scale) per tensor."""
    n = len(xs)
    assert len(fmts) == n and len(outs) == n and scalars.numel() >= 3 * n
    items = (QuantItem * n)()
    for i, (x, f, o) in enumerate(zip(xs, fmts, outs)):
        items[i] = QuantItem(_ptr(x).value, x.numel(), int(f), _ptr(o).value)
    _check(load().fp8_quantize_multi(items, C.c_int(n), _ptr(scalars), _stream(stream)))


class DelayedItem(C.Structure):
    _fields_ = [("x_bf16", C.c_void_p), ("n", C.c_size_t), ("fmt", C.c_int), ("out", C.c_void_p),
                ("history", C.c_void_p), ("head", C.c_void_p), ("scale_next", C.c_void_p), ("amax", C.c_void_p),
                ("scale", C.c_void_p), ("scale_inv", C.c_void_p)]


def fp8_quantize_delayed_multi(xs, fmts, outs, histories, heads, scales_next, amaxes, scales, scales_inv, margin,
                               sync, stream=None):
    """Delayed-scaling quantize of up to 8 tensors in one launch: cast under scales_next[i] as the call finds it (also
    written to scales[i] with its reciprocal in scales_inv[i]), amax, history update, and the next step's scale left in
    scales_next[i].  Lists of CUDA tensors, one entry per tensor; all histories have the same length; sync an int32 /
    uint32 CUDA tensor of 2 * len(xs) words that is zero before the first call."""
    n = len(xs)
    assert all(len(v) == n for v in (fmts, outs, histories, heads, scales_next, amaxes, scales, scales_inv))
    assert sync.numel() >= 2 * n and sync.element_size() == 4
    assert all(h.numel() == histories[0].numel() for h in histories)
    items = (DelayedItem * n)()
    for i in range(n):
        items[i] = DelayedItem(_ptr(xs[i]).value, xs[i].numel(), int(fmts[i]), _ptr(outs[i]).value,
                               _ptr(histories[i]).value, _ptr(heads[i]).value, _ptr(scales_next[i]).value,
                               _ptr(amaxes[i]).value, _ptr(scales[i]).value, _ptr(scales_inv[i]).value)
    _check(load().fp8_quantize_delayed_multi(items, C.c_int(n), C.c_int(histories[0].numel()), C.c_int(margin),
                                             _ptr(sync), _stream(stream)))


ACT_GELU, ACT_XIELU = 1, 2
NORM_RMS, NORM_LAYERSCALE = 0, 1
QK_RMS, QK_TANH, QK_NONE = 0, 1, 2


def fp8_postnorm_residual(x, y, gamma, mode, eps, out, amax_out=None, stream=None):
    """out = x + gamma * y / rms(y) (NORM_RMS) or x + gamma * y (NORM_LAYERSCALE); [T, D] BF16, amax of out optional."""
    T, D = x.shape
    _check(load().fp8_postnorm_residual(_ptr(x), _ptr(y), _ptr(gamma), C.c_size_t(T), C.c_size_t(D), C.c_int(mode),
                                        C.c_float(eps), _ptr(out), _ptr(amax_out), _stream(stream)))


def fp8_postnorm_residual_q(x, y, gamma, mode, eps, scale, fmt, out, out8, amax_out=None, x_scale=1.0, stream=None):
    """fp8_postnorm_residual that also writes the FP8 codes of its (BF16-rounded) result under the delayed `scale`;
    x_scale multiplies the residual input (sigma_0^-1 for the first block's input, else 1)."""
    T, D = x.shape
    _check(load().fp8_postnorm_residual_q(_ptr(x), _ptr(y), _ptr(gamma), C.c_size_t(T), C.c_size_t(D), C.c_int(mode),
                                          C.c_float(eps), C.c_float(x_scale), _ptr(scale), C.c_int(fmt), _ptr(out),
                                          _ptr(out8), _ptr(amax_out), _stream(stream)))


def fp8_qk_norm_rope_q(x, mode, alpha, eps, cos_table, sin_table, seq_len, scale, fmt, out, out8, amax_out=None,
                       stream=None):
    """fp8_qk_norm_rope that also writes the FP8 codes of its (BF16-rounded) result under the delayed `scale`
    (out may be None when only the codes are wanted)."""
    T, H, d = x.shape
    _check(load().fp8_qk_norm_rope_q(_ptr(x), C.c_size_t(T), C.c_size_t(H), C.c_size_t(d), C.c_int(mode),
                                     C.c_float(alpha), C.c_float(eps), _ptr(cos_table), _ptr(sin_table),
                                     C.c_size_t(seq_len), _ptr(scale), C.c_int(fmt), _ptr(out), _ptr(out8),
                                     _ptr(amax_out), _stream(stream)))


def fp8_qk_norm_rope(x, mode, alpha, eps, cos_table, sin_table, seq_len, out, amax_out=None, stream=None):
    """QK regulariser (per-head RMS norm / tanh(alpha x) / none) + rotary embedding on [T, H, d] BF16."""
    T, H, d = x.shape
    _check(load().fp8_qk_norm_rope(_ptr(x), C.c_size_t(T), C.c_size_t(H), C.c_size_t(d), C.c_int(mode),
                                   C.c_float(alpha), C.c_float(eps), _ptr(cos_table), _ptr(sin_table),
                                   C.c_size_t(seq_len), _ptr(out), _ptr(amax_out), _stream(stream)))


def fp8_act_cast(x, act, act_params, scale, fmt, out, out_t=None, amax_out=None, stream=None):
    """h = GeLU(x) or xIELU(x; a_p, a_n) fused with the cast; x is [T, F] BF16, act_params a device float[2] or None."""
    T, F = x.shape
    _check(load().fp8_act_cast(_ptr(x), C.c_size_t(T), C.c_size_t(F), C.c_int(act), _ptr(act_params), _ptr(scale),
                               C.c_int(fmt), _ptr(out), _ptr(out_t), _ptr(amax_out), _stream(stream)))


def fp8_swiglu_cast(gate_up, scale, fmt, out, out_t=None, amax_out=None, stream=None):
    """h = silu(gate) * up fused with the cast; gate_up is [T, 2F] BF16.  out / out_t may be None (amax only)."""
    T, F2 = gate_up.shape
    _check(load().fp8_swiglu_cast(_ptr(gate_up), C.c_size_t(T), C.c_size_t(F2 // 2), _ptr(scale), C.c_int(fmt),
                                  _ptr(out), _ptr(out_t), _ptr(amax_out), _stream(stream)))


def fp8_kurtosis(x, out, stream=None):
    rows, cols = _rows_cols(x)
    _check(load().fp8_kurtosis(_ptr(x), C.c_size_t(rows), C.c_size_t(cols), _ptr(out), _stream(stream)))


def fp8_amax_kurtosis(x, amax, kurtosis, stream=None):
    """amax and the kurtosis monitor of a [rows, cols] BF16 tensor from one read of it."""
    rows, cols = _rows_cols(x)
    _check(load().fp8_amax_kurtosis(_ptr(x), C.c_size_t(rows), C.c_size_t(cols), _ptr(amax), _ptr(kurtosis),
                                    _stream(stream)))


def _is_fp32(t):
    if t.dtype == torch.float32:
        return 1
    assert t.dtype in (torch.bfloat16, torch.int16, torch.uint16), "output must be BF16 or FP32"
    return 0


def fp8_linear_fwd(x8, w8, sx_inv, sw_inv, y, ws=None, stream=None):
    T, K = x8.shape
    N = w8.shape[0]
    _check(load().fp8_linear_fwd(_ptr(x8), _ptr(w8), _ptr(sx_inv), _ptr(sw_inv), _ptr(y), C.c_int(_is_fp32(y)),
                                 C.c_int(T), C.c_int(N), C.c_int(K), _ptr(ws),
                                 C.c_size_t(0 if ws is None else ws.numel() * ws.element_size()), _stream(stream)))


def fp8_linear_fwd_q(x8, w8, sx_inv, sw_inv, y_scale, y_fmt, y8, y_amax=None, stream=None):
    """Forward product emitting FP8 codes of the BF16-rounded result under a caller (delayed) scale, plus its amax."""
    T, K = x8.shape
    N = w8.shape[0]
    _check(load().fp8_linear_fwd_q(_ptr(x8), _ptr(w8), _ptr(sx_inv), _ptr(sw_inv), _ptr(y_scale), C.c_int(y_fmt),
                                   _ptr(y8), _ptr(y_amax), C.c_int(T), C.c_int(N), C.c_int(K), _stream(stream)))


def fp8_linear_dgrad_q(dy8, w8t, sdy_inv, sw_inv, dx_scale, dx_fmt, dx8, dx_amax=None, stream=None):
    """Data-gradient product emitting FP8 codes of the BF16-rounded result under a caller scale, plus its amax."""
    T, N = dy8.shape
    K = w8t.shape[0]
    _check(load().fp8_linear_dgrad_q(_ptr(dy8), _ptr(w8t), _ptr(sdy_inv), _ptr(sw_inv), _ptr(dx_scale),
                                     C.c_int(dx_fmt), _ptr(dx8), _ptr(dx_amax), C.c_int(T), C.c_int(N), C.c_int(K),
                                     _stream(stream)))


def fp8_linear_dgrad_rm(dy8, w8, sdy_inv, sw_inv, dx, stream=None):
    """dX = dY8 . W8 with W8 [N, K] read in place (no transposed copy)."""
    T, N = dy8.shape
    K = w8.shape[1]
    _check(load().fp8_linear_dgrad_rm(_ptr(dy8), _ptr(w8), _ptr(sdy_inv), _ptr(sw_inv), _ptr(dx),
                                      C.c_int(_is_fp32(dx)), C.c_int(T), C.c_int(N), C.c_int(K), _stream(stream)))


def fp8_linear_wgrad_rm(dy8, x8, sdy_inv, sx_inv, dw, accumulate=False, stream=None):
    """dW (+)= dY8^T . X8 with dY8 [T, N] and X8 [T, K] read in place (no transposed copies)."""
    T, N = dy8.shape
    K = x8.shape[1]
    _check(load().fp8_linear_wgrad_rm(_ptr(dy8), _ptr(x8), _ptr(sdy_inv), _ptr(sx_inv), _ptr(dw),
                                      C.c_int(_is_fp32(dw)), C.c_int(int(accumulate)), C.c_int(T), C.c_int(N),
                                      C.c_int(K), _stream(stream)))


def fp8_grouped_linear_fwd(x8, w8, sx_inv, sw_inv, group_offsets, y, stream=None):
    """Per-expert forward product: x8 [T, K] sorted by expert, w8 [E, N, K], sw_inv [E], group_offsets int32 [E + 1]."""
    T, K = x8.shape
    E, N = w8.shape[0], w8.shape[1]
    _check(load().fp8_grouped_linear_fwd(_ptr(x8), _ptr(w8), _ptr(sx_inv), _ptr(sw_inv), _ptr(group_offsets),
                                         C.c_int(E), _ptr(y), C.c_int(_is_fp32(y)), C.c_int(T), C.c_int(N), C.c_int(K),
                                         _stream(stream)))


def fp8_grouped_linear_dgrad(dy8, w8, sdy_inv, sw_inv, group_offsets, dx, stream=None):
    """Per-expert data gradient: dy8 [T, N] (E5M2) sorted by expert, w8 [E, N, K] read in place, dx [T, K]."""
    T, N = dy8.shape
    E, K = w8.shape[0], w8.shape[2]
    _check(load().fp8_grouped_linear_dgrad(_ptr(dy8), _ptr(w8), _ptr(sdy_inv), _ptr(sw_inv), _ptr(group_offsets),
                                           C.c_int(E), _ptr(dx), C.c_int(_is_fp32(dx)), C.c_int(T), C.c_int(N),
                                           C.c_int(K), _stream(stream)))


def fp8_grouped_linear_wgrad(dy8, x8, sdy_inv, sx_inv, group_offsets_host, dw, accumulate=False, stream=None):
    """Per-expert weight gradients: dy8 [T, N], x8 [T, K] sorted by expert, dw [E, N, K]; offsets are host integers."""
    T, N = dy8.shape
    K = x8.shape[1]
    offs = [int(v) for v in group_offsets_host]
    E = len(offs) - 1
    arr = (C.c_int * len(offs))(*offs)
    _check(load().fp8_grouped_linear_wgrad(_ptr(dy8), _ptr(x8), _ptr(sdy_inv), _ptr(sx_inv), arr, C.c_int(E), _ptr(dw),
                                           C.c_int(_is_fp32(dw)), C.c_int(int(accumulate)), C.c_int(T), C.c_int(N),
                                           C.c_int(K), _stream(stream)))


def fp8_grouped_linear_wgrad_workspace_bytes(n_groups, N) -> int:
    return int(load().fp8_grouped_linear_wgrad_workspace_bytes(n_groups, N))


def fp8_grouped_linear_wgrad_dev(dy8, x8, sdy_inv, sx_inv, group_offsets, dw, ws, accumulate=False, stream=None):
    """The same weight gradients in one launch; group_offsets is an int32 CUDA tensor (E + 1 entries), ws a uint8 CUDA tensor
    of fp8_grouped_linear_wgrad_workspace_bytes(E, N)."""
    T, N = dy8.shape
    K = x8.shape[1]
    E = group_offsets.numel() - 1
    _check(load().fp8_grouped_linear_wgrad_dev(_ptr(dy8), _ptr(x8), _ptr(sdy_inv), _ptr(sx_inv), _ptr(group_offsets),
                                               C.c_int(E), _ptr(dw), C.c_int(_is_fp32(dw)), C.c_int(int(accumulate)),
                                               C.c_int(T), C.c_int(N), C.c_int(K), _ptr(ws), C.c_size_t(ws.numel()),
                                               _stream(stream)))


def fp8_quantize_blockwise(x, block_rows, fmt, out, scale_inv, stream=None):
    """Block-by-block quantisation: 1 x 128 (scale_inv [cols/128, rows]), 128 x 128 (scale_inv [rows/128, cols/128])
    or, with block_rows = FP8_BLOCK_128x1, 128 x 1 (scale_inv [ceil(rows/128), cols])."""
    rows, cols = x.shape
    _check(load().fp8_quantize_blockwise(_ptr(x), C.c_size_t(rows), C.c_size_t(cols), C.c_int(block_rows), C.c_int(fmt),
                                         _ptr(out), _ptr(scale_inv), _stream(stream)))


def fp8_linear_fwd_blockwise(x8, w8, sx_inv, sw_inv, y, stream=None):
    T, K = x8.shape
    N = w8.shape[0]
    _check(load().fp8_linear_fwd_blockwise(_ptr(x8), _ptr(w8), _ptr(sx_inv), _ptr(sw_inv), _ptr(y), C.c_int(T),
                                           C.c_int(N), C.c_int(K), _stream(stream)))


def fp8_linear_dgrad_blockwise(dy8, w8, sdy_inv, sw_inv, dx, stream=None):
    """dX = dY W under the blockwise recipe: dy8 [T,N] in 1 x 128 blocks, w8 [N,K] in the forward's 128 x 128 blocks."""
    T, N = dy8.shape
    K = w8.shape[1]
    _check(load().fp8_linear_dgrad_blockwise(_ptr(dy8), _ptr(w8), _ptr(sdy_inv), _ptr(sw_inv), _ptr(dx), C.c_int(T),
                                             C.c_int(N), C.c_int(K), _stream(stream)))


def fp8_linear_wgrad_blockwise(dy8, x8, sdy_inv_t, sx_inv_t, dw, stream=None):
    """dW = dY^T X under the blockwise recipe: both operands in 128 x 1 blocks along the token axis."""
    T, N = dy8.shape
    K = x8.shape[1]
    _check(load().fp8_linear_wgrad_blockwise(_ptr(dy8), _ptr(x8), _ptr(sdy_inv_t), _ptr(sx_inv_t), _ptr(dw), C.c_int(T),
                                             C.c_int(N), C.c_int(K), _stream(stream)))


def fp8_linear_dgrad(dy8, w8t, sdy_inv, sw_inv, dx, ws=None, stream=None):
    T, N = dy8.shape
    K = w8t.shape[0]
    _check(load().fp8_linear_dgrad(_ptr(dy8), _ptr(w8t), _ptr(sdy_inv), _ptr(sw_inv), _ptr(dx),
                                   C.c_int(_is_fp32(dx)), C.c_int(T), C.c_int(N), C.c_int(K), _ptr(ws),
                                   C.c_size_t(0 if ws is None else ws.numel() * ws.element_size()), _stream(stream)))


def fp8_linear_wgrad(dy8t, x8t, sdy_inv, sx_inv, dw, accumulate=False, ws=None, stream=None):
    N, T = dy8t.shape
    K = x8t.shape[0]
    _check(load().fp8_linear_wgrad(_ptr(dy8t), _ptr(x8t), _ptr(sdy_inv), _ptr(sx_inv), _ptr(dw),
                                   C.c_int(_is_fp32(dw)), C.c_int(int(accumulate)), C.c_int(T), C.c_int(N),
                                   C.c_int(K), _ptr(ws),
                                   C.c_size_t(0 if ws is None else ws.numel() * ws.element_size()), _stream(stream)))


def fp8_attention_workspace_bytes(op, B, N, Hq, Hkv, d) -> int:
    return int(load().fp8_attention_workspace_bytes(op, B, N, Hq, Hkv, d))


def _scales(q_inv, k_inv, v_inv, do_inv, softmax_scale, p_scale, ds_scale, ds_amax, max_slack=0.0):
    return AttnScales(_ptr(q_inv).value, _ptr(k_inv).value, _ptr(v_inv).value, _ptr(do_inv).value,
                      float(softmax_scale), float(p_scale), _ptr(ds_scale).value, _ptr(ds_amax).value,
                      float(max_slack))


def fp8_attention_fwd(q8, k8, v8, q_inv, k_inv, v_inv, softmax_scale, causal, o, lse, ws, p_scale=448.0,
                      stream=None, max_slack=0.0):
    """max_slack = tau > 0: a row keeps its reference maximum until exceeded by more than 2^tau; p_scale <= 448 / 2^tau."""
    B, N, Hq, d = q8.shape
    Hkv = k8.shape[2]
    sc = _scales(q_inv, k_inv, v_inv, None, softmax_scale, p_scale, None, None, max_slack)
    _check(load().fp8_attention_fwd(_ptr(q8), _ptr(k8), _ptr(v8), C.byref(sc), C.c_int(int(causal)), C.c_int(B),
                                    C.c_int(N), C.c_int(Hq), C.c_int(Hkv), C.c_int(d), _ptr(o), _ptr(lse),
                                    _ptr(ws), C.c_size_t(0 if ws is None else ws.numel() * ws.element_size()),
                                    _stream(stream)))


def fp8_attention_fwd_q(q8, k8, v8, q_inv, k_inv, v_inv, softmax_scale, causal, o, lse, o_scale, o8, o_amax=None,
                        p_scale=448.0, stream=None, max_slack=0.0):
    """Forward that also emits E4M3 codes of O under a caller (delayed) scale and amax(O)."""
    B, N, Hq, d = q8.shape
    Hkv = k8.shape[2]
    sc = _scales(q_inv, k_inv, v_inv, None, softmax_scale, p_scale, None, None, max_slack)
    _check(load().fp8_attention_fwd_q(_ptr(q8), _ptr(k8), _ptr(v8), C.byref(sc), C.c_int(int(causal)), C.c_int(B),
                                      C.c_int(N), C.c_int(Hq), C.c_int(Hkv), C.c_int(d), _ptr(o), _ptr(lse),
                                      _ptr(o_scale), _ptr(o8), _ptr(o_amax), _stream(stream)))


def fp8_attention_bwd(q8, k8, v8, do8, o, lse, q_inv, k_inv, v_inv, do_inv, softmax_scale, ds_scale, causal,
                      dq, dk, dv, ws, ds_amax=None, p_scale=448.0, stream=None):
    B, N, Hq, d = q8.shape
    Hkv = k8.shape[2]
    sc = _scales(q_inv, k_inv, v_inv, do_inv, softmax_scale, p_scale, ds_scale, ds_amax)
    _check(load().fp8_attention_bwd(_ptr(q8), _ptr(k8), _ptr(v8), _ptr(do8), _ptr(o), _ptr(lse), C.byref(sc),
                                    C.c_int(int(causal)), C.c_int(B), C.c_int(N), C.c_int(Hq), C.c_int(Hkv),
                                    C.c_int(d), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(ws),
                                    C.c_size_t(0 if ws is None else ws.numel() * ws.element_size()),
                                    _stream(stream)))


def fp8_attention_bwd_static(q8, k8, v8, do8, o, lse, q_inv, k_inv, v_inv, do_inv, softmax_scale, ds_scale, causal,
                             dq, dk, dv, ds_amax=None, p_scale=448.0, stream=None):
    """fp8_attention_bwd for callers that cannot provide scratch: it uses the fixed array inside the library
    (problems up to STATIC_SCRATCH_BYTES of scratch; calls must not overlap on the GPU)."""
    B, N, Hq, d = q8.shape
    Hkv = k8.shape[2]
    sc = _scales(q_inv, k_inv, v_inv, do_inv, softmax_scale, p_scale, ds_scale, ds_amax)
    _check(load().fp8_attention_bwd_static(_ptr(q8), _ptr(k8), _ptr(v8), _ptr(do8), _ptr(o), _ptr(lse),
                                           C.byref(sc), C.c_int(int(causal)), C.c_int(B), C.c_int(N), C.c_int(Hq),
                                           C.c_int(Hkv), C.c_int(d), _ptr(dq), _ptr(dk), _ptr(dv), _stream(stream)))


def _hptr(t):
    assert not t.is_cuda and t.is_contiguous(), "expects contiguous HOST tensors"
    return C.c_void_p(t.data_ptr())


def fp8_linear_step_host_workspace_bytes(T, N, K) -> int:
    return int(load().fp8_linear_step_host_workspace_bytes(T, N, K))


def fp8_linear_step_host(hx, hw, hdy, hy, hdx, hdw, ws):
    """hx [T,K], hw [N,K], hdy [T,N] and the outputs hy, hdx, hdw: BF16 HOST tensors (pinned for overlap); ws: a uint8
    CUDA tensor of fp8_linear_step_host_workspace_bytes(T, N, K).  Returns once enqueued: see fp8_host_sync."""
    (T, K), N = hx.shape, hw.shape[0]
    _check(load().fp8_linear_step_host(_hptr(hx), _hptr(hw), _hptr(hdy), C.c_int(T), C.c_int(N), C.c_int(K), _hptr(hy),
                                       _hptr(hdx), _hptr(hdw), _ptr(ws), C.c_size_t(ws.numel())))


def fp8_attention_step_host_workspace_bytes(B, N, Hq, Hkv, d) -> int:
    return int(load().fp8_attention_step_host_workspace_bytes(B, N, Hq, Hkv, d))


def fp8_attention_step_host(hq, hk, hv, hdo, softmax_scale, ds_scale, causal, ho, hlse, hdq, hdk, hdv, ws):
    """hq, hdo, ho, hdq [B,N,Hq,d] and hk, hv, hdk, hdv [B,N,Hkv,d]: BF16 HOST tensors; hlse [B,Hq,N] FP32 HOST;
    softmax_scale and ds_scale host floats; ws: a uint8 CUDA tensor of fp8_attention_step_host_workspace_bytes(...)."""
    B, N, Hq, d = hq.shape
    Hkv = hk.shape[2]
    _check(load().fp8_attention_step_host(_hptr(hq), _hptr(hk), _hptr(hv), _hptr(hdo), C.c_int(B), C.c_int(N), C.c_int(Hq),
                                          C.c_int(Hkv), C.c_int(d), C.c_float(softmax_scale), C.c_float(ds_scale),
                                          C.c_int(int(causal)), _hptr(ho), _hptr(hlse), _hptr(hdq), _hptr(hdk), _hptr(hdv),
                                          _ptr(ws), C.c_size_t(ws.numel())))


def fp8_host_sync():
    """Waits for every host-buffer call made so far on the current device."""
    _check(load().fp8_host_sync())
