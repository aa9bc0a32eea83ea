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
