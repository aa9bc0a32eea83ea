"""Pins of the kurtosis monitor (Section 4) and the gated activation (Appendix B) in the oracle."""
import numpy as np

import oracle as o
from paper_2505_20524_b200 import synth


def bf16(v):
    return synth.f32_to_bf16(np.asarray(v, dtype=np.float32))


def test_kurtosis_closed_forms():
    D = 64
    assert o.kurtosis(bf16(np.full((3, D), 0.5))) == 1.0                         # constant vector
    assert o.kurtosis(bf16(np.where(np.arange(D) % 2 == 0, 2.0, -2.0)[None])) == 1.0   # signs do not matter
    onehot = np.zeros((1, D)); onehot[0, 7] = 3.0
    assert o.kurtosis(bf16(onehot)) == float(D)                                    # a single outlier: maximal
    two = np.zeros((1, D)); two[0, :2] = 1.0
    assert o.kurtosis(bf16(two)) == D / 2.0
    # average over token vectors, scale invariance (powers of two are exact in BF16)
    x = np.stack([np.full(D, 0.25), onehot[0]])
    assert o.kurtosis(bf16(x)) == (1.0 + D) / 2.0
    g = synth.bf16_to_f32(synth.normal_bf16((64, 256), 1, 1, 1.0))
    assert abs(o.kurtosis(bf16(g)) - o.kurtosis(bf16(4.0 * g))) < 1e-12
    # against numpy moments of the same BF16 values
    exp = np.mean((g.astype(np.float64) ** 4).mean(axis=1) / (g.astype(np.float64) ** 2).mean(axis=1) ** 2)
    assert abs(o.kurtosis(bf16(g)) - exp) < 1e-12


def test_kurtosis_of_gaussian_is_three_and_grows_with_outliers():
    g = synth.normal_bf16((256, 4096), 2, 1, 1.0)
    k0 = o.kurtosis(g)
    assert abs(k0 - 3.0) < 0.05
    cols = synth.choose_columns(4096, 21, 4, 100)
    k1 = o.kurtosis(synth.normal_bf16((256, 4096), 2, 1, 1.0, cols, 30.0))
    assert k1 > 20 * k0                      # 0.5% of channels x30 dominate the fourth moment


def test_swiglu_values():
    g = np.array([[0.0, 1.0, -1.0, 8.0, -8.0, 2.0, 0.5, -0.5]])
    u = np.array([[3.0, 1.0, 1.0, 0.5, 2.0, -1.0, 4.0, 4.0]])
    x = np.concatenate([np.tile(g, (1, 2)), np.tile(u, (1, 2))], axis=1)            # F = 16
    h = synth.bf16_to_f32(o.swiglu(bf16(x)))[0, :8]
    exp = g[0] / (1.0 + np.exp(-g[0])) * u[0]                                         # silu(g) * u
    assert np.allclose(h, exp, rtol=2.0 ** -8)
    assert h[0] == 0.0 and abs(h[1] - 0.7310585786) < 3e-3 and abs(h[3] - 3.99866) < 2e-2
    # silu(g) -> g for large g, -> 0 for very negative g; up = 0 gives 0
    big = np.zeros((1, 32)); big[0, :16] = 30.0; big[0, 16:] = 1.5
    assert np.all(synth.bf16_to_f32(o.swiglu(bf16(big))) == 45.0)
    neg = np.zeros((1, 32)); neg[0, :16] = -30.0; neg[0, 16:] = 1.5
    assert np.all(np.abs(synth.bf16_to_f32(o.swiglu(bf16(neg)))) < 1e-11)


def test_gelu_values():
    x = np.array([[0.0, 1.0, -1.0, 3.0, -3.0, 0.5, -0.5, 8.0, -8.0, 2.0, -2.0, 0.25, 6.0, -6.0, 1.5, -1.5]])
    h = synth.bf16_to_f32(o.activation(bf16(x), o.GELU))[0]
    # x * Phi(x) with the standard normal CDF at the usual table points
    phi = {0.0: 0.5, 1.0: 0.8413447461, 3.0: 0.9986501020, 0.5: 0.6914624613, 2.0: 0.9772498681, 1.5: 0.9331927987}
    for i, v in enumerate(x[0]):
        p = phi.get(abs(v))
        if p is None:
            continue
        exp = v * (p if v >= 0 else 1.0 - p)
        assert abs(h[i] - exp) <= 2.0 ** -8 * abs(exp) + 1e-30, (v, h[i], exp)
    assert h[7] == 8.0 and abs(h[8]) < 1e-13                       # identity far right, zero far left
    # GeLU(x) - GeLU(-x) = x exactly in real arithmetic
    assert np.allclose(h[1] - h[2], 1.0, atol=2.0 ** -7) and np.allclose(h[9] - h[10], 2.0, atol=2.0 ** -6)


def test_xielu_values_and_limits():
    ap, an = 0.75, 1.25
    x = np.array([[0.0, 1.0, 2.0, -1.0, -2.0, 0.5, -0.5, 4.0, -16.0, 0.125, -0.125, 3.0, -3.0, 8.0, -8.0, 1.5]])
    h = synth.bf16_to_f32(o.activation(bf16(x), o.XIELU, ap, an))[0]
    assert h[0] == 0.0
    assert h[1] == ap + 0.5 and h[2] == 4 * ap + 1.0 and h[7] == 16 * ap + 2.0            # exact in BF16
    e = np.exp(-1.0)
    assert abs(h[3] - (an * (e - 1.0) + an - 0.5)) < 2.0 ** -8
    # far left the exponential dies: slope 0.5 - alpha_n, offset -alpha_n
    assert abs(h[8] - (-an - (0.5 - an) * 16.0)) < 2.0 ** -4
    # continuous with slope 0.5 through the origin on both sides
    assert abs(h[9] - 0.0625) < 0.02 and abs(h[10] + 0.0625) < 0.02
    # alpha_p = alpha_n = 0 is x / 2
    z = synth.bf16_to_f32(o.activation(bf16(x), o.XIELU, 0.0, 0.0))[0]
    assert np.array_equal(z, x[0] * 0.5)
