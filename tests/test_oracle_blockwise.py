"""Pins of the fine-grained (blockwise) scaling oracle (Section 2; Appendix E, "Fine-grained scaling recipes")."""
import numpy as np

import oracle as o
from paper_2505_20524_b200 import synth


def bf16(v):
    return synth.f32_to_bf16(np.asarray(v, dtype=np.float32))


def test_one_block_is_the_tensorwise_quantiser():
    x = synth.normal_bf16((128, 128), 31, 1, 1.0)
    codes, si = o.quantize_blockwise(x, 128, 128, o.E4M3)
    c2, amax, s, s_inv = o.quantize(x, o.E4M3)
    assert np.array_equal(codes, c2) and si.shape == (1, 1) and si[0, 0] == np.float32(s_inv)
    # 1 x 128 blocks of a [T,128] tensor: every row is a tensor of its own
    codes, si = o.quantize_blockwise(x, 1, 128, o.E5M2)
    for r in (0, 17, 127):
        cr, _, _, sir = o.quantize(x[r:r + 1], o.E5M2)
        assert np.array_equal(codes[r], cr[0]) and si[r, 0] == np.float32(sir)


def test_every_block_uses_its_own_range():
    # blocks with very different magnitudes: each block's largest element lands on the largest code
    R, C = 256, 384
    x = synth.bf16_to_f32(synth.normal_bf16((R, C), 32, 1, 1.0)).copy()
    x[:128, :128] *= 1000.0
    x[128:, 256:] *= 1e-3
    xb = bf16(x)
    for br, bc in ((128, 128), (1, 128)):
        codes, si = o.quantize_blockwise(xb, br, bc, o.E4M3)
        assert si.shape == (R // br, C // bc)
        dec = o.decode_array(codes, o.E4M3)
        for rb in range(R // br):
            for cb in range(C // bc):
                blk = np.abs(dec[rb * br:(rb + 1) * br, cb * bc:(cb + 1) * bc])
                assert blk.max() == 448.0
        # a tensor-wide scale would flush the small block to (almost) nothing; block scales keep 3 bits everywhere
        back = dec * np.repeat(np.repeat(si, br, axis=0), bc, axis=1)
        xf = synth.bf16_to_f32(xb)
        big = np.abs(xf) > 1e-2 * np.abs(xf).reshape(R // br, br, C // bc, bc).max(axis=(1, 3)).repeat(br, 0).repeat(bc, 1)
        assert np.all(np.abs(back - xf)[big] <= 2.0 ** -4 * np.abs(xf)[big] * 1.001)


def test_ragged_edges():
    x = synth.normal_bf16((130, 200), 33, 1, 1.0)
    codes, si = o.quantize_blockwise(x, 128, 128, o.E4M3)
    assert si.shape == (2, 2)
    c_edge, _, _, s_edge = o.quantize(np.ascontiguousarray(x[128:, 128:]), o.E4M3)
    assert np.array_equal(codes[128:, 128:], c_edge) and si[1, 1] == np.float32(s_edge)


def test_blockwise_gemm_reduces_to_the_tensorwise_one():
    T, N, K = 8, 256, 384
    x8 = o.quantize(synth.normal_bf16((T, K), 34, 1, 1.0), o.E4M3)[0]
    w8 = o.quantize(synth.normal_bf16((N, K), 34, 2, 0.02), o.E4M3)[0]
    sx = np.full((T, 3), 0.25, dtype=np.float32)
    sw = np.full((2, 3), 0.5, dtype=np.float32)
    ref, mag = o.linear_fwd_blockwise(x8, w8, sx, sw)
    ref2, mag2 = o.linear_fwd(x8, w8, 0.25, 0.5)
    assert np.allclose(ref, ref2, rtol=1e-13, atol=1e-300) and np.allclose(mag, mag2, rtol=1e-13)
    # one K-block switched off, one weight block doubled
    sx2 = sx.copy(); sx2[:, 1] = 0.0
    sw2 = sw.copy(); sw2[1, :] = 1.0
    ref3, _ = o.linear_fwd_blockwise(x8, w8, sx2, sw2)
    tab = o.decode_table(o.E4M3)
    a, b = tab[x8], tab[w8]
    keep = np.r_[0:128, 256:384]
    exp = a[:, keep] @ b[:, keep].T * 0.25 * np.where(np.arange(N) < 128, 0.5, 1.0)[None]
    assert np.allclose(ref3, exp, rtol=1e-12, atol=1e-300)


def test_blockwise_pipeline_is_exact_on_powers_of_two():
    # powers of two quantise exactly under any power-of-two block amax, so the whole pipeline is integer arithmetic
    T, N, K = 4, 128, 256
    rng = np.random.default_rng(5)
    x = np.ldexp(1.0, rng.integers(-3, 3, size=(T, K))) * rng.choice([-1.0, 1.0], size=(T, K))
    w = np.ldexp(1.0, rng.integers(-6, 0, size=(N, K))) * rng.choice([-1.0, 1.0], size=(N, K))
    x[:, 0] = 4.0; x[:, 128] = 4.0            # block amax 4 -> scale 112, a power of two times 7: products stay exact
    w[0, 0] = 1.0; w[0, 128] = 1.0
    x8, sx = o.quantize_blockwise(bf16(x), 1, 128, o.E4M3)
    w8, sw = o.quantize_blockwise(bf16(w), 128, 128, o.E4M3)
    ref, _ = o.linear_fwd_blockwise(x8, w8, sx, sw)
    # codes hold x*112 and w*448 exactly wherever those are representable; compare against the decoded operands
    tab = o.decode_table(o.E4M3)
    xd = tab[x8] * np.repeat(sx.astype(np.float64), 128, axis=1)
    wd = tab[w8] * np.repeat(np.repeat(sw.astype(np.float64), 128, axis=0), 128, axis=1)
    assert np.allclose(ref, xd @ wd.T, rtol=1e-6)


def test_column_block_quantiser_is_the_row_block_one_transposed():
    # 128 x 1 blocks of x are the 1 x 128 blocks of x^T: same codes, same descales, transposed
    x = synth.normal_bf16((300, 40), 61, 0, 3.0)
    codes, si = o.quantize_blockwise(x, 128, 1, o.E5M2)
    codes_t, si_t = o.quantize_blockwise(np.ascontiguousarray(x.T), 1, 128, o.E5M2)
    assert si.shape == (3, 40)
    assert np.array_equal(codes, codes_t.T) and np.array_equal(si.view(np.uint32), si_t.T.view(np.uint32))


def test_blockwise_gradients_reduce_to_plain_matrix_products():
    T, N, K = 200, 256, 384                      # T ragged against the 128-token blocks of the weight gradient
    tab4, tab5 = o.decode_table(o.E4M3), o.decode_table(o.E5M2)
    dy8 = o.quantize(synth.normal_bf16((T, N), 35, 1, 1.0), o.E5M2)[0]
    w8 = o.quantize(synth.normal_bf16((N, K), 35, 2, 0.02), o.E4M3)[0]
    x8 = o.quantize(synth.normal_bf16((T, K), 35, 3, 1.0), o.E4M3)[0]
    g, w, x = tab5[dy8], tab4[w8], tab4[x8]
    # constant scales: the plain products times the two factors
    ref, mag = o.linear_dgrad_blockwise(dy8, w8, np.full((T, 2), 0.25, np.float32), np.full((2, 3), 0.5, np.float32))
    assert np.allclose(ref, 0.125 * (g @ w), rtol=1e-12, atol=1e-300)
    assert np.allclose(mag, 0.125 * (np.abs(g) @ np.abs(w)), rtol=1e-12)
    ntb = 2
    ref, mag = o.linear_wgrad_blockwise(dy8, x8, np.full((ntb, N), 0.25, np.float32), np.full((ntb, K), 2.0, np.float32))
    assert np.allclose(ref, 0.5 * (g.T @ x), rtol=1e-12, atol=1e-300)
    assert np.allclose(mag, 0.5 * (np.abs(g).T @ np.abs(x)), rtol=1e-12)
    # distinct scales per block: every factor lands on its own block and nowhere else
    rng = np.random.default_rng(9)
    sdy = rng.uniform(0.5, 2.0, size=(T, 2)).astype(np.float32)
    sw = rng.uniform(0.5, 2.0, size=(2, 3)).astype(np.float32)
    gd = g * np.repeat(sdy.astype(np.float64), 128, axis=1)
    wd = w * np.repeat(np.repeat(sw.astype(np.float64), 128, axis=0), 128, axis=1)
    ref, mag = o.linear_dgrad_blockwise(dy8, w8, sdy, sw)
    assert np.max(np.abs(ref - gd @ wd) / mag) < 1e-13          # sums that cancel: measure against the magnitude
    assert np.max(np.abs(ref - (g * np.repeat(sdy[:, ::-1].astype(np.float64), 128, axis=1)) @ wd) / mag) > 1e-2
    sdt = rng.uniform(0.5, 2.0, size=(ntb, N)).astype(np.float32)
    sxt = rng.uniform(0.5, 2.0, size=(ntb, K)).astype(np.float32)
    gd = g * np.repeat(sdt.astype(np.float64), 128, axis=0)[:T]
    xd = x * np.repeat(sxt.astype(np.float64), 128, axis=0)[:T]
    ref, mag = o.linear_wgrad_blockwise(dy8, x8, sdt, sxt)
    assert np.max(np.abs(ref - gd.T @ xd) / mag) < 1e-13
    assert np.max(np.abs(ref - (g * np.repeat(sdt[::-1].astype(np.float64), 128, axis=0)[:T]).T @ xd) / mag) > 1e-2
    # sampled rows and columns pick the same entries
    rows, cols = np.array([3, 255]), np.array([0, 129, 383])
    sub, _ = o.linear_wgrad_blockwise(dy8, x8, sdt, sxt, rows=rows, cols=cols)
    assert np.array_equal(sub, ref[np.ix_(rows, cols)])


def test_blockwise_gradient_pipeline_recovers_the_unquantised_products():
    # quantise -> product -> descale reproduces the BF16 operands' product to the formats' precision
    T, N, K = 256, 128, 256
    dy = synth.normal_bf16((T, N), 36, 1, 1e-3)
    w = synth.normal_bf16((N, K), 36, 2, 0.02)
    x = synth.normal_bf16((T, K), 36, 3, 1.0)
    f = lambda a: (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    dy8, sdy = o.quantize_blockwise(dy, 1, 128, o.E5M2)
    w8, sw = o.quantize_blockwise(w, 128, 128, o.E4M3)
    ref, mag = o.linear_dgrad_blockwise(dy8, w8, sdy, sw)
    exact = f(dy) @ f(w)
    assert np.max(np.abs(ref - exact) / mag) < 0.07          # E5M2 half-ulp 2^-3 and E4M3 2^-4, averaged over a sum
    dy8t, sdt = o.quantize_blockwise(dy, 128, 1, o.E5M2)
    x8t, sxt = o.quantize_blockwise(x, 128, 1, o.E4M3)
    ref, mag = o.linear_wgrad_blockwise(dy8t, x8t, sdt, sxt)
    exact = f(dy).T @ f(x)
    assert np.max(np.abs(ref - exact) / mag) < 0.07
