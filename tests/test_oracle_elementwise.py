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


def test_postnorm_residual_closed_forms():
    D = 64
    x = np.arange(D, dtype=np.float64)[None] * 0.25
    g = np.full(D, 0.5, dtype=np.float32)
    # constant branch output: y / rms(y) = sign(y)
    out = synth.bf16_to_f32(o.postnorm_residual(bf16(x), bf16(np.full((1, D), -3.0)), g))
    assert np.array_equal(out, x - 0.5)
    # one non-zero entry a: rms = |a| / sqrt(D), so that entry becomes sqrt(D) = 8
    y = np.zeros((1, D)); y[0, 5] = 0.75
    out = synth.bf16_to_f32(o.postnorm_residual(bf16(x), bf16(y), g))
    exp = x.copy(); exp[0, 5] += 0.5 * 8.0
    assert np.array_equal(out, exp)
    # scale invariance in y (powers of two are exact), and eps breaks it the right way
    yy = synth.normal_bf16((8, D), 3, 4, 1.0)
    xx = synth.normal_bf16((8, D), 3, 5, 1.0)
    y4 = bf16(4.0 * synth.bf16_to_f32(yy))
    assert np.array_equal(o.postnorm_residual(xx, yy, g), o.postnorm_residual(xx, y4, g))
    big_eps = synth.bf16_to_f32(o.postnorm_residual(xx, yy, g, o.NORM_RMS, 1e6))
    assert np.allclose(big_eps, synth.bf16_to_f32(xx), atol=0.01)          # y / sqrt(1e6) vanishes
    # LayerScale: x + gamma * y, exact on these values
    out = synth.bf16_to_f32(o.postnorm_residual(bf16(x), bf16(np.full((1, D), 2.0)), g, o.NORM_LAYERSCALE))
    assert np.array_equal(out, x + 1.0)
    # against numpy on random data
    xf, yf = synth.bf16_to_f32(xx).astype(np.float64), synth.bf16_to_f32(yy).astype(np.float64)
    ref = xf + 0.5 * yf / np.sqrt((yf ** 2).mean(axis=1, keepdims=True) + 1e-5)
    got = synth.bf16_to_f32(o.postnorm_residual(xx, yy, g, o.NORM_RMS, 1e-5))
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-30)


def test_postnorm_residual_input_scaling():
    """x_scale multiplies the residual input only (the first block's input is scaled by sigma_0^-1, Section 3)."""
    D = 64
    g = np.full(D, 0.5, dtype=np.float32)
    xx, yy = synth.normal_bf16((8, D), 3, 6, 1.0), synth.normal_bf16((8, D), 3, 7, 1.0)
    # factor 1 is the plain form
    assert np.array_equal(o.postnorm_residual(xx, yy, g, o.NORM_RMS, 1e-5, 1.0), o.postnorm_residual(xx, yy, g, o.NORM_RMS, 1e-5))
    # zero branch output: out = BF16(u x); a power of two is exact
    zero = bf16(np.zeros((8, D)))
    out = synth.bf16_to_f32(o.postnorm_residual(xx, zero, g, o.NORM_LAYERSCALE, 0.0, 4.0))
    assert np.array_equal(out, 4.0 * synth.bf16_to_f32(xx))
    out = synth.bf16_to_f32(o.postnorm_residual(xx, zero, g, o.NORM_LAYERSCALE, 0.0, 1.0 / 0.02))
    assert np.array_equal(out, synth.bf16_to_f32(bf16(synth.bf16_to_f32(xx).astype(np.float64) * 50.0)))
    # the factor does not touch the branch: u x + gamma y / rms(y) against numpy
    xf, yf = synth.bf16_to_f32(xx).astype(np.float64), synth.bf16_to_f32(yy).astype(np.float64)
    ref = 50.0 * xf + 0.5 * yf / np.sqrt((yf ** 2).mean(axis=1, keepdims=True))
    got = synth.bf16_to_f32(o.postnorm_residual(xx, yy, g, o.NORM_RMS, 0.0, 50.0))
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-30)


def test_qk_norm_rope_closed_forms():
    T, H, d, N = 6, 2, 64, 3
    q = synth.normal_bf16((T, H * d), 5, 6, 2.0).reshape(T, H, d)
    qf = synth.bf16_to_f32(q).astype(np.float64)
    # RMS norm without rotation: unit mean square per head
    out = synth.bf16_to_f32(o.qk_norm_rope(q, o.QK_RMS, 0.0, 0.0)).astype(np.float64)
    assert np.allclose((out ** 2).mean(axis=2), 1.0, atol=5e-3)
    assert np.all(np.abs(out - qf / np.sqrt((qf ** 2).mean(axis=2, keepdims=True))) <= 2.0 ** -8 * np.abs(out) + 1e-30)
    # tanh regulariser: values
    v = np.zeros((1, 1, d)); v[0, 0, :4] = [2.0, -2.0, 0.0, 1.0]
    out = synth.bf16_to_f32(o.qk_norm_rope(bf16(v), o.QK_TANH, 0.5, 0.0))[0, 0]
    assert abs(out[0] - 0.761594) < 3e-3 and out[1] == -out[0] and out[2] == 0.0 and abs(out[3] - 0.462117) < 2e-3
    # quarter turn at every frequency: (a, b) -> (-b, a); identity at angle 0; position = t mod seq_len
    cos = np.zeros((N, d // 2), dtype=np.float32); sin = np.zeros((N, d // 2), dtype=np.float32)
    cos[0] = 1.0                              # position 0: no rotation
    sin[1] = 1.0                              # position 1: 90 degrees
    cos[2] = -1.0                             # position 2: 180 degrees
    out = synth.bf16_to_f32(o.qk_norm_rope(q, o.QK_NONE, 0.0, 0.0, cos, sin, N))
    f = synth.bf16_to_f32(q)
    for t in range(T):
        a, b = f[t, :, :d // 2], f[t, :, d // 2:]
        exp = {0: (a, b), 1: (-b, a), 2: (-a, -b)}[t % N]
        assert np.array_equal(out[t, :, :d // 2], exp[0]) and np.array_equal(out[t, :, d // 2:], exp[1])
    # a rotation keeps the length of every pair
    th = np.linspace(0.1, 3.0, N * d // 2).reshape(N, d // 2)
    out = synth.bf16_to_f32(o.qk_norm_rope(q, o.QK_NONE, 0.0, 0.0, np.cos(th), np.sin(th), N)).astype(np.float64)
    n_in = qf[:, :, :d // 2] ** 2 + qf[:, :, d // 2:] ** 2
    n_out = out[:, :, :d // 2] ** 2 + out[:, :, d // 2:] ** 2
    assert np.allclose(n_in, n_out, rtol=2e-2, atol=1e-6)
