"""GPU parity of the fused gated activation + cast and of the kurtosis monitor."""
import numpy as np
import pytest
import torch

import oracle as o
import paper_2505_20524_b200 as fp8
from paper_2505_20524_b200 import synth
from gpu_util import dev, host, scalar

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("rows,cols", [(256, 256), (8192, 4096), (100, 1024), (16, 14336)])
def test_kurtosis_matches_oracle(rows, cols):
    c = synth.choose_columns(cols, max(1, cols // 200), 1, 5)
    x = synth.normal_bf16((rows, cols), 4, 6, 1.0, c, 30.0)
    out = scalar(-5.0)
    fp8.fp8_kurtosis(dev(x), out)
    exp = o.kurtosis(x)
    assert abs(float(out.item()) - exp) <= 2e-5 * exp        # FP32 sums of x^4 over a row, FP32 atomics over rows


def neighbours(code, ref, fmt):
    """True where code == ref or the two codes are adjacent values of the format."""
    t = o.decode_table(fmt)
    order = np.argsort(np.where(np.isfinite(t), t, np.inf), kind="stable")
    rank = np.empty(256, dtype=np.int64)
    rank[order] = np.arange(256)
    return np.abs(rank[code] - rank[ref]) <= 2            # +0 and -0 sit next to each other in the ordering


def test_amax_and_kurtosis_from_one_pass():
    """The monitor folded into the amax pass: amax bit-exact as fp8_amax, kurtosis as fp8_kurtosis."""
    for rows, cols in ((64, 4096), (1000, 264), (8192, 2048)):
        c = synth.choose_columns(cols, max(1, cols // 100), 6, 1)
        xb = synth.normal_bf16((rows, cols), 14, 1, 1.0, c, 30.0)
        a, k, k0 = scalar(-1.0), scalar(-1.0), scalar(-1.0)
        fp8.fp8_amax_kurtosis(dev(xb), a, k)
        fp8.fp8_kurtosis(dev(xb), k0)
        torch.cuda.synchronize()
        assert float(a.item()) == float(o.amax(xb))
        ref = o.kurtosis(xb)
        assert abs(float(k.item()) - ref) <= 2e-5 * ref
        assert abs(float(k.item()) - float(k0.item())) <= 1e-5 * ref


@pytest.mark.parametrize("fmt", [o.E4M3, o.E5M2])
@pytest.mark.parametrize("T,F", [(256, 1024), (144, 272), (1024, 5632)])
def test_swiglu_cast_matches_oracle(fmt, T, F):
    c = synth.choose_columns(2 * F, max(2, F // 100), 2, 7)
    gu = synth.normal_bf16((T, 2 * F), 6, 8, 1.0, c, 8.0)
    h = o.swiglu(gu)
    x = dev(gu)
    a = scalar()
    fp8.fp8_swiglu_cast(x, None, fmt, None, None, a)                     # JIT pass 1: amax of h only
    ea = o.amax(h)
    assert abs(float(a.item()) - float(ea)) <= 2.0 ** -7 * float(ea)     # expf vs exp: at most one BF16 step
    s, si = scalar(), scalar()
    fp8.fp8_scale(a, fmt, 0, s, si)
    out = torch.empty((T, F), dtype=torch.uint8, device="cuda")
    out_t = torch.empty((F, T), dtype=torch.uint8, device="cuda")
    a2 = scalar(3.0)
    fp8.fp8_swiglu_cast(x, s, fmt, out, out_t, a2)                        # pass 2: cast (+ amax again)
    assert float(a2.item()) == float(a.item())
    got = host(out)
    exp = o.cast(h, float(s.item()), fmt)                                 # same scale on both sides
    diff = got != exp
    assert diff.mean() <= 2e-3, diff.mean()             # h differs by one BF16 ulp where expf and exp disagree
    assert neighbours(got[diff], exp[diff], fmt).all()
    assert np.array_equal(host(out_t), got.T)
    # and against the unfused chain on the GPU itself: identical h bits would give identical codes
    hd = dev(h)
    ref = torch.empty((T, F), dtype=torch.uint8, device="cuda")
    fp8.fp8_cast(hd, s, fmt, ref)
    assert (host(ref) != got).mean() <= 2e-3


def test_swiglu_argument_validation():
    x = dev(synth.normal_bf16((32, 64), 0, 0, 1.0))
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_swiglu_cast(x, None, 0, None, None, None)
    assert e.value.status == -1
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_swiglu_cast(x[:, :48].contiguous(), scalar(1), 0, torch.empty((32, 24), dtype=torch.uint8, device="cuda"))
    assert e.value.status == -3
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_kurtosis(x[:, :60].contiguous(), scalar())
    assert e.value.status == -3


@pytest.mark.parametrize("fmt", [o.E4M3, o.E5M2])
@pytest.mark.parametrize("act", [o.GELU, o.XIELU])
@pytest.mark.parametrize("T,F", [(256, 1024), (144, 272), (512, 8192)])
def test_act_cast_matches_oracle(fmt, act, T, F):
    c = synth.choose_columns(F, max(2, F // 100), 3, 9)
    xb = synth.normal_bf16((T, F), 9, 3, 1.0, c, 8.0)
    ap, an = 0.8125, 1.3125
    h = o.activation(xb, act, ap, an)
    x = dev(xb)
    params = torch.tensor([ap, an], dtype=torch.float32, device="cuda") if act == o.XIELU else None
    a = scalar()
    fp8.fp8_act_cast(x, act, params, None, fmt, None, None, a)                # amax of h only
    ea = o.amax(h)
    assert abs(float(a.item()) - float(ea)) <= 2.0 ** -7 * float(ea)
    s, si = scalar(), scalar()
    fp8.fp8_scale(a, fmt, 0, s, si)
    out = torch.empty((T, F), dtype=torch.uint8, device="cuda")
    out_t = torch.empty((F, T), dtype=torch.uint8, device="cuda")
    fp8.fp8_act_cast(x, act, params, s, fmt, out, out_t, None)
    got = host(out)
    exp = o.cast(h, float(s.item()), fmt)
    diff = got != exp
    assert diff.mean() <= 2e-3, diff.mean()            # FP32 erf / expm1 against double, seen through BF16 rounding
    assert neighbours(got[diff], exp[diff], fmt).all()
    assert np.array_equal(host(out_t), got.T)


def test_act_cast_argument_validation():
    x = dev(synth.normal_bf16((32, 64), 0, 0, 1.0))
    out = torch.empty((32, 64), dtype=torch.uint8, device="cuda")
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_act_cast(x, fp8.ACT_XIELU, None, scalar(1), 0, out)           # xIELU needs its two scalars
    assert e.value.status == -1
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_act_cast(x, 7, None, scalar(1), 0, out)
    assert e.value.status == -4


def bf16_close(got_bits, exp_bits, max_frac=2e-3):
    """Equal BF16 tensors except for at most `max_frac` of elements that differ by one BF16 step."""
    g = got_bits.astype(np.int32).ravel()
    e = exp_bits.astype(np.int32).ravel()
    diff = g != e
    assert diff.mean() <= max_frac, diff.mean()
    # sign-magnitude ordering: one step apart (or +0 / -0)
    key = lambda b: np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)
    assert np.all(np.abs(key(g[diff]) - key(e[diff])) <= 1)


@pytest.mark.parametrize("mode,eps", [(o.NORM_RMS, 0.0), (o.NORM_RMS, 1e-5), (o.NORM_LAYERSCALE, 0.0)])
@pytest.mark.parametrize("T,D", [(64, 2048), (100, 4096), (7, 264), (16, 16384)])
def test_postnorm_residual_matches_oracle(mode, eps, T, D):
    c = synth.choose_columns(D, max(1, D // 200), 4, 1)
    xb = synth.normal_bf16((T, D), 10, 1, 1.0, c, 20.0)
    yb = synth.normal_bf16((T, D), 10, 2, 0.02, c, 20.0)
    gamma = (np.full(D, 1.0 / np.sqrt(32.0)) * (1.0 + 0.01 * np.arange(D) / D)).astype(np.float32)
    exp = o.postnorm_residual(xb, yb, gamma, mode, eps)
    out = torch.empty((T, D), dtype=torch.int16, device="cuda")
    a = scalar(-1.0)
    fp8.fp8_postnorm_residual(dev(xb), dev(yb), torch.from_numpy(gamma).cuda(), mode, eps, out, a)
    got = host(out).view(np.uint16)
    bf16_close(got, exp)
    assert float(a.item()) == float(o.amax(got))            # amax of what was written
    # in place on the residual stream
    xio = dev(xb)
    fp8.fp8_postnorm_residual(xio, dev(yb), torch.from_numpy(gamma).cuda(), mode, eps, xio, None)
    assert np.array_equal(host(xio).view(np.uint16), got)


@pytest.mark.parametrize("mode", [o.QK_RMS, o.QK_TANH, o.QK_NONE])
@pytest.mark.parametrize("rope", [True, False])
@pytest.mark.parametrize("T,H,d,N", [(256, 8, 128, 64), (96, 4, 64, 32), (33, 3, 128, 11)])
def test_qk_norm_rope_matches_oracle(mode, rope, T, H, d, N):
    xb = synth.normal_bf16((T, H * d), 12, 3, 1.5).reshape(T, H, d)
    inv = 10000.0 ** (-np.arange(d // 2) * 2.0 / d)
    ang = np.arange(N)[:, None] * inv[None]
    cos, sin = np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)
    exp = o.qk_norm_rope(xb, mode, 0.5, 1e-6, cos if rope else None, sin if rope else None, N)
    out = torch.empty((T, H, d), dtype=torch.int16, device="cuda")
    a = scalar(-1.0)
    fp8.fp8_qk_norm_rope(dev(xb), mode, 0.5, 1e-6, torch.from_numpy(cos).cuda() if rope else None,
                         torch.from_numpy(sin).cuda() if rope else None, N, out, a)
    got = host(out).view(np.uint16)
    bf16_close(got, exp, 4e-3 if mode == o.QK_TANH else 2e-3)
    assert float(a.item()) == float(o.amax(got))


@pytest.mark.parametrize("mode,fmt,x_scale", [(o.NORM_RMS, o.E4M3, 1.0), (o.NORM_LAYERSCALE, o.E4M3, 1.0),
                                               (o.NORM_RMS, o.E5M2, 1.0), (o.NORM_RMS, o.E4M3, 50.0)])
@pytest.mark.parametrize("T,D", [(64, 2048), (100, 4096), (7, 264)])
def test_postnorm_residual_producer_form_equals_unfused_chain(mode, fmt, x_scale, T, D):
    """Delayed scaling: the same pass writes the FP8 codes of its result; they are the codes fp8_cast gives for the
    BF16 output, the amax is that of the BF16 output, and the BF16 output matches the oracle (with the input factor)."""
    c = synth.choose_columns(D, max(1, D // 200), 4, 1)
    xb = synth.normal_bf16((T, D), 11, 1, 1.0 / x_scale, c, 20.0)
    yb = synth.normal_bf16((T, D), 11, 2, 0.02, c, 20.0)
    gamma = (np.full(D, 1.0 / np.sqrt(32.0)) * (1.0 + 0.01 * np.arange(D) / D)).astype(np.float32)
    gd = torch.from_numpy(gamma).cuda()
    exp = o.postnorm_residual(xb, yb, gamma, mode, 1e-5, x_scale)
    sc = scalar(3.7)                                           # a "history" scale, not the tensor's own
    out = torch.empty((T, D), dtype=torch.int16, device="cuda")
    out8 = torch.full((T, D), 0x55, dtype=torch.uint8, device="cuda")
    a = scalar(-1.0)
    fp8.fp8_postnorm_residual_q(dev(xb), dev(yb), gd, mode, 1e-5, sc, fmt, out, out8, a, x_scale=x_scale)
    torch.cuda.synchronize()
    got = host(out).view(np.uint16)
    bf16_close(got, exp)
    assert float(a.item()) == float(o.amax(got))
    assert np.array_equal(host(out8), o.cast(got, np.float32(3.7), fmt))      # the oracle's cast of the same BF16 values
    if D % 16 == 0:                                                               # (fp8_cast wants whole 16-byte rows)
        ref8 = torch.empty_like(out8)
        fp8.fp8_cast(out.view(torch.bfloat16), sc, fmt, ref8)                    # and the library's own unfused chain
        assert torch.equal(out8, ref8)
    if x_scale == 1.0:
        plain = torch.empty_like(out)
        fp8.fp8_postnorm_residual(dev(xb), dev(yb), gd, mode, 1e-5, plain, None)
        assert torch.equal(plain, out)


@pytest.mark.parametrize("mode,fmt", [(o.QK_RMS, o.E4M3), (o.QK_TANH, o.E4M3), (o.QK_NONE, o.E5M2)])
@pytest.mark.parametrize("T,H,d,N", [(256, 8, 128, 64), (96, 4, 64, 32), (33, 3, 128, 11)])
def test_qk_norm_rope_producer_form_equals_unfused_chain(mode, fmt, T, H, d, N):
    xb = synth.normal_bf16((T, H * d), 13, 3, 1.5).reshape(T, H, d)
    inv = 10000.0 ** (-np.arange(d // 2) * 2.0 / d)
    ang = np.arange(N)[:, None] * inv[None]
    cos, sin = torch.from_numpy(np.cos(ang).astype(np.float32)).cuda(), torch.from_numpy(np.sin(ang).astype(np.float32)).cuda()
    plain = torch.empty((T, H, d), dtype=torch.int16, device="cuda")
    a0 = scalar(-1.0)
    fp8.fp8_qk_norm_rope(dev(xb), mode, 0.5, 1e-6, cos, sin, N, plain, a0)
    sc = scalar(100.0)
    out = torch.empty_like(plain)
    out8 = torch.full((T, H, d), 0x55, dtype=torch.uint8, device="cuda")
    a = scalar(-1.0)
    fp8.fp8_qk_norm_rope_q(dev(xb), mode, 0.5, 1e-6, cos, sin, N, sc, fmt, out, out8, a)
    torch.cuda.synchronize()
    assert torch.equal(out, plain) and float(a.item()) == float(a0.item())
    assert np.array_equal(host(out8), o.cast(host(out).view(np.uint16), np.float32(100.0), fmt))
    # codes only
    only8 = torch.full((T, H, d), 0x55, dtype=torch.uint8, device="cuda")
    fp8.fp8_qk_norm_rope_q(dev(xb), mode, 0.5, 1e-6, cos, sin, N, sc, fmt, None, only8, None)
    assert torch.equal(only8, out8)


def test_glue_argument_validation():
    x = dev(synth.normal_bf16((8, 64), 0, 0, 1.0))
    g = torch.ones(64, device="cuda")
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_postnorm_residual(x, x, g, 5, 0.0, x)
    assert e.value.status == -4
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_postnorm_residual(x[:, :60].contiguous(), x[:, :60].contiguous(), g, 0, 0.0, x)
    assert e.value.status == -3
    q = x.view(8, 1, 64)
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_qk_norm_rope(q, 0, 0.0, 0.0, g, None, 4, q)           # cos without sin
    assert e.value.status == -1
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_qk_norm_rope(x.view(8, 2, 32), 0, 0.0, 0.0, None, None, 1, x.view(8, 2, 32))
    assert e.value.status == -3
