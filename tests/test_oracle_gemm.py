"""Pins of the oracle's FP8 GEMM (Appendix E: GEMM(X,Y) = 1/(rho_X rho_Y) FP8GEMM(cast(rho_X X), cast(rho_Y Y)))."""
import numpy as np

import oracle as o
from paper_2505_20524_b200 import synth


def codes(shape, seed, fmt):
    rng = np.random.default_rng(seed)
    table = o.decode_table(fmt)
    ok = np.flatnonzero(np.isfinite(table))
    return ok[rng.integers(0, ok.size, size=shape)].astype(np.uint8)


def test_brute_force_tiny_triple_loops():
    T, N, K = 5, 7, 8
    x8, w8, dy8 = codes((T, K), 1, o.E4M3), codes((N, K), 2, o.E4M3), codes((T, N), 3, o.E5M2)
    d4, d5 = o.decode_table(o.E4M3), o.decode_table(o.E5M2)
    sa, sb = 0.37, 2.5
    y, ymag = o.linear_fwd(x8, w8, sa, sb)
    dx, _ = o.linear_dgrad(dy8, w8, sa, sb)
    dw, _ = o.linear_wgrad(dy8, x8, sa, sb)
    for t in range(T):
        for n in range(N):
            acc = sum(d4[x8[t, k]] * d4[w8[n, k]] for k in range(K))
            mag = sum(abs(d4[x8[t, k]]) * abs(d4[w8[n, k]]) for k in range(K))
            assert abs(y[t, n] - sa * sb * acc) <= 1e-12 * max(1.0, sa * sb * mag)
            assert abs(ymag[t, n] - sa * sb * mag) <= 1e-12 * sa * sb * mag
        for k in range(K):
            acc = sum(d5[dy8[t, n]] * d4[w8[n, k]] for n in range(N))
            assert abs(dx[t, k] - sa * sb * acc) <= 1e-9 * max(1.0, abs(sa * sb * acc))
    for n in range(N):
        for k in range(K):
            acc = sum(d5[dy8[t, n]] * d4[x8[t, k]] for t in range(T))
            assert abs(dw[n, k] - sa * sb * acc) <= 1e-9 * max(1.0, abs(sa * sb * acc))


def test_against_float64_matmul_of_decoded_operands():
    T, N, K = 33, 21, 64
    x8, w8, dy8 = codes((T, K), 4, o.E4M3), codes((N, K), 5, o.E4M3), codes((T, N), 6, o.E5M2)
    X, W, dY = o.decode_array(x8, o.E4M3), o.decode_array(w8, o.E4M3), o.decode_array(dy8, o.E5M2)
    y, ymag = o.linear_fwd(x8, w8, 0.5, 0.25)
    dx, dxm = o.linear_dgrad(dy8, w8, 0.5, 0.25)
    dw, dwm = o.linear_wgrad(dy8, x8, 0.5, 0.25)
    for got, mag, exp in ((y, ymag, X @ W.T), (dx, dxm, dY @ W), (dw, dwm, dY.T @ X)):
        assert np.all(np.abs(got - 0.125 * exp) <= 1e-12 * mag + 1e-300)
    assert np.allclose(ymag, 0.125 * np.abs(X) @ np.abs(W).T, rtol=1e-12)


def test_sampled_rows_cols_and_accumulate():
    T, N, K = 16, 12, 32
    x8, dy8 = codes((T, K), 7, o.E4M3), codes((T, N), 8, o.E5M2)
    full, _ = o.linear_wgrad(dy8, x8, 1.0, 1.0)
    rows, cols = np.array([3, 0, 11]), np.array([31, 2])
    part, _ = o.linear_wgrad(dy8, x8, 1.0, 1.0, rows, cols)
    assert np.array_equal(part, full[np.ix_(rows, cols)])
    prev = np.arange(6, dtype=np.float64).reshape(3, 2)
    acc, _ = o.linear_wgrad(dy8, x8, 1.0, 1.0, rows, cols, prev=prev)
    assert np.array_equal(acc, part + prev)


def test_all_ones_and_identity():
    K = 48
    ones = np.full((4, K), 0x38, dtype=np.uint8)
    y, _ = o.linear_fwd(ones, ones, 0.5, 3.0)
    assert np.all(y == K * 1.5)
    eye = np.where(np.eye(K, dtype=bool), 0x38, 0x00).astype(np.uint8)
    x8 = codes((9, K), 9, o.E4M3)
    y, _ = o.linear_fwd(x8, eye, 1.0, 1.0)
    assert np.array_equal(y, o.decode_array(x8, o.E4M3))


def test_power_of_two_tensors_make_the_whole_pipeline_exact():
    """Values that are signed powers of two quantise exactly, so quantize + FP8 GEMM + descale equals the
    real product (the closed form of the Appendix E identity)."""
    rng = np.random.default_rng(10)
    T, N, K = 8, 6, 64
    X = np.ldexp(rng.choice([-1.0, 1.0], (T, K)), rng.integers(-3, 3, (T, K)))
    W = np.ldexp(rng.choice([-1.0, 1.0], (N, K)), rng.integers(-5, 1, (N, K)))
    X[0, 0], W[0, 0] = 7.0, -1.75                   # amax = 448 / 2^k -> scale and scale_inv powers of two
    xq, _, _, sxi = o.quantize(synth.f32_to_bf16(X), o.E4M3)
    wq, _, _, swi = o.quantize(synth.f32_to_bf16(W), o.E4M3)
    y, _ = o.linear_fwd(xq, wq, sxi, swi)
    assert np.array_equal(y, X @ W.T)


def test_constant_tensors_closed_form():
    T, N, K, a, b = 4, 3, 256, 0.3, -0.02
    xq, _, _, sxi = o.quantize(synth.f32_to_bf16(np.full((T, K), a)), o.E4M3)
    wq, _, _, swi = o.quantize(synth.f32_to_bf16(np.full((N, K), b)), o.E4M3)
    y, _ = o.linear_fwd(xq, wq, sxi, swi)
    a16 = float(synth.bf16_to_f32(synth.f32_to_bf16(np.float32([a])))[0])
    b16 = float(synth.bf16_to_f32(synth.f32_to_bf16(np.float32([b])))[0])
    # X == a everywhere -> every code is the format maximum and 448 * scale_inv returns a to 2 roundings
    assert np.all(np.abs(y - K * a16 * b16) <= abs(K * a16 * b16) * 2.0 ** -21)
