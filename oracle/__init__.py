"""CPU oracle of the FP8 transformer-block hot path: test infrastructure, not a product path.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package.  It is a
ctypes view of ``fp8_oracle.c`` (plain C, double accumulation) and shares nothing with the CUDA library.
FP8 tensors are ``uint8`` code arrays, BF16 tensors are ``uint16`` bit arrays, everything else is
float64/float32 numpy.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

E4M3 = 0
E5M2 = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fp8_oracle.c")
_LIB = os.path.join(_HERE, "libfp8_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile fp8_oracle.c with gcc (OpenMP, no FMA contraction, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared",
               "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class AttnParams(C.Structure):
    _fields_ = [("B", C.c_int32), ("N", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32), ("d", C.c_int32),
                ("causal", C.c_int32), ("quant", C.c_int32), ("kv_block", C.c_int32),
                ("max_mode", C.c_int32), ("pad_", C.c_int32),
                ("s", C.c_double), ("c_P", C.c_double),
                ("q_inv", C.c_double), ("k_inv", C.c_double), ("v_inv", C.c_double), ("do_inv", C.c_double),
                ("ds_scale", C.c_double), ("flip_eps", C.c_double), ("max_slack", C.c_double)]


def _L():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_fp8_decode.restype = C.c_double
        _lib.oracle_fp8_decode.argtypes = [C.c_uint8, C.c_int]
        _lib.oracle_fp8_encode.restype = C.c_uint8
        _lib.oracle_fp8_encode.argtypes = [C.c_float, C.c_int]
        _lib.oracle_fp8_max.restype = C.c_double
        _lib.oracle_fp8_max.argtypes = [C.c_int]
        _lib.oracle_amax_bf16.restype = C.c_float
        _lib.oracle_amax_bf16.argtypes = [C.c_void_p, C.c_size_t]
        _lib.oracle_scale.restype = None
        _lib.oracle_scale.argtypes = [C.c_float, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        _lib.oracle_cast_bf16.restype = None
        _lib.oracle_cast_bf16.argtypes = [C.c_void_p, C.c_size_t, C.c_size_t, C.c_float, C.c_int,
                                          C.c_void_p, C.c_void_p]
        _lib.oracle_fp8_encode_array.restype = None
        _lib.oracle_fp8_encode_array.argtypes = [C.c_void_p, C.c_size_t, C.c_int, C.c_void_p]
        _lib.oracle_num_threads.restype = C.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dt):
    a = np.ascontiguousarray(a, dtype=dt)
    return a


def num_threads() -> int:
    return int(_L().oracle_num_threads())


# ---------------------------------------------------------------- codec
def fp8_max(fmt: int) -> float:
    return float(_L().oracle_fp8_max(fmt))


def decode(code: int, fmt: int) -> float:
    return float(_L().oracle_fp8_decode(int(code) & 0xFF, fmt))


def encode(v: float, fmt: int) -> int:
    return int(_L().oracle_fp8_encode(np.float32(v), fmt))


def decode_table(fmt: int) -> np.ndarray:
    out = np.empty(256, dtype=np.float64)
    _L().oracle_fp8_decode_table(fmt, _p(out))
    return out


def decode_array(codes: np.ndarray, fmt: int) -> np.ndarray:
    return decode_table(fmt)[np.asarray(codes, dtype=np.uint8)]


def encode_array(v: np.ndarray, fmt: int) -> np.ndarray:
    v = _c(v, np.float32)
    out = np.empty(v.shape, dtype=np.uint8)
    _L().oracle_fp8_encode_array(_p(v), v.size, fmt, _p(out))
    return out


# ---------------------------------------------------------------- quantize
def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def amax(x_bf16: np.ndarray) -> np.float32:
    x = _c(x_bf16, np.uint16)
    return np.float32(_L().oracle_amax_bf16(_p(x), x.size))


def scale(amax_value, fmt: int, margin: int = 0):
    s = C.c_float()
    si = C.c_float()
    _L().oracle_scale(np.float32(amax_value), fmt, margin, C.byref(s), C.byref(si))
    return np.float32(s.value), np.float32(si.value)


def scale_update(history: np.ndarray, head: int, amax_new, fmt: int, margin: int = 0):
    """Delayed scaling: push amax_new into the FIFO `history` (float32, modified in place; `head` = position of
    the oldest entry) and return (new_head, scale, scale_inv) computed from the updated history."""
    assert history.dtype == np.float32 and history.flags["C_CONTIGUOUS"]
    h = C.c_int(int(head))
    s = C.c_float()
    si = C.c_float()
    f = _L().oracle_scale_update
    f.restype = None
    f(_p(history), C.c_int(history.size), C.byref(h), C.c_float(float(amax_new)), C.c_int(fmt), C.c_int(margin),
      C.byref(s), C.byref(si))
    return h.value, np.float32(s.value), np.float32(si.value)


def kurtosis(x_bf16: np.ndarray) -> float:
    """Mean over rows of mu[x^4] / mu[x^2]^2 (un-centred), x = rows of a [rows, cols] BF16 tensor."""
    x = _c(x_bf16, np.uint16)
    x2 = x.reshape(-1, x.shape[-1])
    f = _L().oracle_kurtosis_bf16
    f.restype = C.c_double
    return float(f(_p(x2), C.c_size_t(x2.shape[0]), C.c_size_t(x2.shape[1])))


def swiglu(gate_up_bf16: np.ndarray) -> np.ndarray:
    """h = silu(gate) * up as BF16 bits; gate / up are the first / second half of the last axis."""
    x = _c(gate_up_bf16, np.uint16)
    T, F2 = x.shape
    out = np.empty((T, F2 // 2), dtype=np.uint16)
    f = _L().oracle_swiglu_bf16
    f.restype = None
    f(_p(x), C.c_size_t(T), C.c_size_t(F2 // 2), _p(out))
    return out


GELU, XIELU = 1, 2
NORM_RMS, NORM_LAYERSCALE = 0, 1
QK_RMS, QK_TANH, QK_NONE = 0, 1, 2


def postnorm_residual(x_bf16, y_bf16, gamma, mode: int = NORM_RMS, eps: float = 0.0, x_scale: float = 1.0) -> np.ndarray:
    """x_scale * x + gamma * y / rms(y) (mode 0) or x_scale * x + gamma * y (mode 1), rounded to BF16 (Section 3,
    Appendix B); x_scale = sigma_0^-1 on the first block's input, 1 elsewhere."""
    x, y = _c(x_bf16, np.uint16), _c(y_bf16, np.uint16)
    g = _c(gamma, np.float32)
    T, D = x.shape
    out = np.empty_like(x)
    f = _L().oracle_postnorm_residual_scaled_bf16
    f.restype = None
    f(_p(x), _p(y), _p(g), C.c_size_t(T), C.c_size_t(D), C.c_int(mode), C.c_double(eps), C.c_double(x_scale), _p(out))
    return out


def qk_norm_rope(x_bf16, mode: int, alpha: float, eps: float, cos=None, sin=None, seq_len: int = 1) -> np.ndarray:
    """QK regulariser (per-head RMS norm / tanh(alpha x) / none) then rotary embedding on [T,H,d] BF16."""
    x = _c(x_bf16, np.uint16)
    T, H, d = x.shape
    out = np.empty_like(x)
    c = _c(cos, np.float32) if cos is not None else None
    s_ = _c(sin, np.float32) if sin is not None else None
    f = _L().oracle_qk_norm_rope_bf16
    f.restype = None
    f(_p(x), C.c_size_t(T), C.c_size_t(H), C.c_size_t(d), C.c_int(mode), C.c_double(alpha), C.c_double(eps),
      _p(c) if c is not None else None, _p(s_) if s_ is not None else None, C.c_size_t(seq_len), _p(out))
    return out


def activation(x_bf16: np.ndarray, act: int, alpha_p: float = 0.0, alpha_n: float = 0.0) -> np.ndarray:
    """GeLU (exact erf form) or xIELU of a BF16 tensor, rounded to BF16 (Appendix B)."""
    x = _c(x_bf16, np.uint16)
    out = np.empty_like(x)
    f = _L().oracle_activation_bf16
    f.restype = None
    f(_p(x), C.c_size_t(x.size), C.c_int(act), C.c_double(alpha_p), C.c_double(alpha_n), _p(out))
    return out


def cast(x_bf16: np.ndarray, scale_value, fmt: int, transpose: bool = False):
    x = _c(x_bf16, np.uint16)
    if x.ndim == 1:
        x = x.reshape(1, -1)
    x2 = x.reshape(-1, x.shape[-1])
    rows, cols = x2.shape
    out = np.empty((rows, cols), dtype=np.uint8)
    out_t = np.empty((cols, rows), dtype=np.uint8) if transpose else None
    _L().oracle_cast_bf16(_p(x2), rows, cols, np.float32(scale_value), fmt, _p(out), _p(out_t))
    out = out.reshape(x_bf16.shape)
    return (out, out_t) if transpose else out


def quantize(x_bf16: np.ndarray, fmt: int, transpose: bool = False):
    """amax -> scale -> cast of the same tensor (just-in-time scaling)."""
    a = amax(x_bf16)
    s, si = scale(a, fmt)
    q = cast(x_bf16, s, fmt, transpose)
    return q, a, s, si


# ---------------------------------------------------------------- linear
def _idx(sel, n):
    return _c(np.arange(n) if sel is None else sel, np.int64)


def _linear(fn, a8, b8, sa_inv, sb_inv, T, N, K, out_rows, out_cols, rows, cols, prev=None):
    rows = _idx(rows, out_rows)
    cols = _idx(cols, out_cols)
    a8 = _c(a8, np.uint8)
    b8 = _c(b8, np.uint8)
    ref = np.empty((rows.size, cols.size), dtype=np.float64)
    mag = np.empty_like(ref)
    args = [_p(a8), _p(b8), C.c_double(float(sa_inv)), C.c_double(float(sb_inv)),
            C.c_int64(T), C.c_int64(N), C.c_int64(K),
            _p(rows), C.c_int64(rows.size), _p(cols), C.c_int64(cols.size)]
    if prev is not None or fn == "oracle_linear_wgrad":
        pv = None if prev is None else _c(prev, np.float64)
        args.append(_p(pv))
    args += [_p(ref), _p(mag)]
    f = getattr(_L(), fn)
    f.restype = None
    f(*args)
    return ref, mag


def linear_fwd(x8, w8, sx_inv, sw_inv, rows=None, cols=None):
    """Y[t,n] = sx_inv*sw_inv * sum_k X8[t,k] W8[n,k]; returns (ref, mag) on rows x cols."""
    T, K = x8.shape
    N = w8.shape[0]
    assert w8.shape[1] == K
    return _linear("oracle_linear_fwd", x8, w8, sx_inv, sw_inv, T, N, K, T, N, rows, cols)


def linear_dgrad(dy8, w8, sdy_inv, sw_inv, rows=None, cols=None):
    """dX[t,k] = sdy_inv*sw_inv * sum_n dY8[t,n] W8[n,k]."""
    T, N = dy8.shape
    K = w8.shape[1]
    assert w8.shape[0] == N
    return _linear("oracle_linear_dgrad", dy8, w8, sdy_inv, sw_inv, T, N, K, T, K, rows, cols)


def linear_wgrad(dy8, x8, sdy_inv, sx_inv, rows=None, cols=None, prev=None):
    """dW[n,k] = prev[n,k] + sdy_inv*sx_inv * sum_t dY8[t,n] X8[t,k] (prev given on rows x cols)."""
    T, N = dy8.shape
    K = x8.shape[1]
    assert x8.shape[0] == T
    return _linear("oracle_linear_wgrad", dy8, x8, sdy_inv, sx_inv, T, N, K, N, K, rows, cols, prev)


def quantize_blockwise(x_bf16, br: int, bc: int, fmt: int):
    """Block-by-block just-in-time quantisation; returns (codes [R,C], scale_inv [ceil(R/br), ceil(C/bc)])."""
    x = _c(x_bf16, np.uint16)
    R, Cc = x.shape
    codes = np.empty((R, Cc), dtype=np.uint8)
    si = np.empty(((R + br - 1) // br, (Cc + bc - 1) // bc), dtype=np.float32)
    f = _L().oracle_quantize_blockwise
    f.restype = None
    f(_p(x), C.c_size_t(R), C.c_size_t(Cc), C.c_size_t(br), C.c_size_t(bc), C.c_int(fmt), _p(codes), _p(si))
    return codes, si


def linear_fwd_blockwise(x8, w8, sx_inv, sw_inv, bk=128, bn=128, rows=None, cols=None):
    """Y with one descale per (row, K-block) of X and per (bn x bk) block of W; returns (ref, mag) on rows x cols."""
    x8, w8 = _c(x8, np.uint8), _c(w8, np.uint8)
    T, K = x8.shape
    N = w8.shape[0]
    sx, sw = _c(sx_inv, np.float32), _c(sw_inv, np.float32)
    assert sx.shape == (T, (K + bk - 1) // bk) and sw.shape == ((N + bn - 1) // bn, (K + bk - 1) // bk)
    r = np.arange(T, dtype=np.int64) if rows is None else _c(rows, np.int64)
    c = np.arange(N, dtype=np.int64) if cols is None else _c(cols, np.int64)
    ref = np.empty((r.size, c.size), dtype=np.float64)
    mag = np.empty_like(ref)
    f = _L().oracle_linear_fwd_blockwise
    f.restype = None
    f(_p(x8), _p(w8), _p(sx), _p(sw), C.c_int64(T), C.c_int64(N), C.c_int64(K), C.c_int64(bk), C.c_int64(bn),
      _p(r), C.c_int64(r.size), _p(c), C.c_int64(c.size), _p(ref), _p(mag))
    return ref, mag


def linear_dgrad_blockwise(dy8, w8, sdy_inv, sw_inv, bn=128, bk=128, rows=None, cols=None):
    """dX with one descale per (row, N-block) of dY and per (bn x bk) block of W; returns (ref, mag) on rows x cols."""
    dy8, w8 = _c(dy8, np.uint8), _c(w8, np.uint8)
    T, N = dy8.shape
    K = w8.shape[1]
    sdy, sw = _c(sdy_inv, np.float32), _c(sw_inv, np.float32)
    assert sdy.shape == (T, (N + bn - 1) // bn) and sw.shape == ((N + bn - 1) // bn, (K + bk - 1) // bk)
    r = np.arange(T, dtype=np.int64) if rows is None else _c(rows, np.int64)
    c = np.arange(K, dtype=np.int64) if cols is None else _c(cols, np.int64)
    ref = np.empty((r.size, c.size), dtype=np.float64)
    mag = np.empty_like(ref)
    f = _L().oracle_linear_dgrad_blockwise
    f.restype = None
    f(_p(dy8), _p(w8), _p(sdy), _p(sw), C.c_int64(T), C.c_int64(N), C.c_int64(K), C.c_int64(bn), C.c_int64(bk),
      _p(r), C.c_int64(r.size), _p(c), C.c_int64(c.size), _p(ref), _p(mag))
    return ref, mag


def linear_wgrad_blockwise(dy8, x8, sdy_inv_t, sx_inv_t, bt=128, rows=None, cols=None):
    """dW with one descale per (token block, channel) of dY and of X; returns (ref, mag) on rows x cols of [N, K]."""
    dy8, x8 = _c(dy8, np.uint8), _c(x8, np.uint8)
    T, N = dy8.shape
    K = x8.shape[1]
    sdy, sx = _c(sdy_inv_t, np.float32), _c(sx_inv_t, np.float32)
    ntb = (T + bt - 1) // bt
    assert sdy.shape == (ntb, N) and sx.shape == (ntb, K)
    r = np.arange(N, dtype=np.int64) if rows is None else _c(rows, np.int64)
    c = np.arange(K, dtype=np.int64) if cols is None else _c(cols, np.int64)
    ref = np.empty((r.size, c.size), dtype=np.float64)
    mag = np.empty_like(ref)
    f = _L().oracle_linear_wgrad_blockwise
    f.restype = None
    f(_p(dy8), _p(x8), _p(sdy), _p(sx), C.c_int64(T), C.c_int64(N), C.c_int64(K), C.c_int64(bt),
      _p(r), C.c_int64(r.size), _p(c), C.c_int64(c.size), _p(ref), _p(mag))
    return ref, mag


# ---------------------------------------------------------------- attention
def attn_params(B, N, Hq, Hkv, d, causal=True, quant=True, kv_block=0, max_mode=0, s=None, c_P=448.0,
                q_inv=1.0, k_inv=1.0, v_inv=1.0, do_inv=1.0, ds_scale=1.0, flip_eps=0.0, max_slack=0.0) -> AttnParams:
    return AttnParams(B=B, N=N, Hq=Hq, Hkv=Hkv, d=d, causal=int(causal), quant=int(quant),
                      kv_block=kv_block, max_mode=max_mode, pad_=0,
                      s=float(d ** -0.5 if s is None else s), c_P=float(c_P),
                      q_inv=float(q_inv), k_inv=float(k_inv), v_inv=float(v_inv), do_inv=float(do_inv),
                      ds_scale=float(ds_scale), flip_eps=float(flip_eps), max_slack=float(max_slack))


def _pairs(sel, nb, nh):
    if sel is None:
        sel = [(b, h) for b in range(nb) for h in range(nh)]
    return _c(np.asarray(sel, dtype=np.int32).reshape(-1, 2), np.int32)


def attention_fwd(q, k, v, p: AttnParams, heads=None, rows=None, real=False, with_slack=False):
    """O[pair,row,d], LSE[pair,row], mag for the (batch, query head) pairs and the query-row range given.

    q, k, v: [B,N,H,d] uint8 E4M3 codes, or float64 values when real=True.  with_slack adds a fourth
    array: how far O may move through FP32-vs-double tie decisions of the P8 encode (needs p.flip_eps)."""
    dt = np.float64 if real else np.uint8
    q, k, v = _c(q, dt), _c(k, dt), _c(v, dt)
    bh = _pairs(heads, p.B, p.Hq)
    r0, r1 = (0, p.N) if rows is None else rows
    O = np.empty((bh.shape[0], r1 - r0, p.d), dtype=np.float64)
    LSE = np.empty((bh.shape[0], r1 - r0), dtype=np.float64)
    mag = np.empty_like(O)
    slack = np.zeros_like(O) if with_slack else None
    f = _L().oracle_attention_fwd_real if real else _L().oracle_attention_fwd
    f.restype = None
    f(_p(q), _p(k), _p(v), C.byref(p), _p(bh), C.c_int(bh.shape[0]), C.c_int(r0), C.c_int(r1),
      _p(O), _p(LSE), _p(mag), _p(slack))
    return (O, LSE, mag, slack) if with_slack else (O, LSE, mag)


def attention_bwd(q, k, v, do, O, LSE, p: AttnParams, kv_heads=None, q_rows=None, k_rows=None, real=False):
    """Gradients for the (batch, kv head) pairs given, over query rows x key rows.

    O: [B,N,Hq,d] float64 (the values handed to the backward, e.g. BF16-rounded), LSE: [B,Hq,N] float64.
    Returns dict with dQ[pair,G,nq,d], dK/dV[pair,nk,d], mag_* (error-metric denominators; for code operands also
    mag8_dQ / mag8_dK, the sums over the quantised |dS8|), slack_* (how far
    each output may move through FP32-vs-double tie decisions of the two encodes; zero unless p.flip_eps > 0)
    and amax_dS."""
    dt = np.float64 if real else np.uint8
    q, k, v, do = _c(q, dt), _c(k, dt), _c(v, dt), _c(do, dt)
    O = _c(O, np.float64)
    LSE = _c(LSE, np.float64)
    bg = _pairs(kv_heads, p.B, p.Hkv)
    q0, q1 = (0, p.N) if q_rows is None else q_rows
    k0, k1 = (0, p.N) if k_rows is None else k_rows
    G = p.Hq // p.Hkv
    n = bg.shape[0]
    out = {
        "dQ": np.empty((n, G, q1 - q0, p.d)), "dK": np.empty((n, k1 - k0, p.d)),
        "dV": np.empty((n, k1 - k0, p.d)),
    }
    for key in ("dQ", "dK", "dV"):
        out["mag_" + key] = np.empty_like(out[key])
        out["slack_" + key] = np.zeros_like(out[key])
    am = C.c_double()
    args = [_p(q), _p(k), _p(v), _p(do), _p(O), _p(LSE), C.byref(p), _p(bg), C.c_int(n),
            C.c_int(q0), C.c_int(q1), C.c_int(k0), C.c_int(k1),
            _p(out["dQ"]), _p(out["dK"]), _p(out["dV"]),
            _p(out["mag_dQ"]), _p(out["mag_dK"]), _p(out["mag_dV"]), C.byref(am),
            _p(out["slack_dQ"]), _p(out["slack_dK"]), _p(out["slack_dV"])]
    if real:
        f = _L().oracle_attention_bwd_real
    else:
        # also the denominators built from the quantised dS8 (sum of |dS8|/ds_scale |K| resp. |Q|)
        out["mag8_dQ"] = np.empty_like(out["dQ"])
        out["mag8_dK"] = np.empty_like(out["dK"])
        args += [_p(out["mag8_dQ"]), _p(out["mag8_dK"])]
        f = _L().oracle_attention_bwd_mag8
    f.restype = None
    f(*args)
    out["amax_dS"] = am.value
    return out


def flip_step(y: float, band: float, fmt: int) -> float:
    """Distance between the two candidate FP8 values when y lies within `band` of a rounding midpoint, else 0."""
    f = _L().oracle_flip_step
    f.restype = C.c_double
    return float(f(C.c_double(y), C.c_double(band), C.c_int(fmt)))
