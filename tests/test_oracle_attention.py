"""Pins of the oracle's attention (Appendix B, Eq. (P): P = Softmax(s QK^T + M), selfattn = PV)."""
import numpy as np
import pytest

import oracle as o

ONE = 0x38  # E4M3 code of 1.0


def rand_codes(shape, seed, lo=0x20, hi=0x48):
    """E4M3 codes of moderate magnitude with random signs."""
    rng = np.random.default_rng(seed)
    c = rng.integers(lo, hi, size=shape).astype(np.uint8)
    return c | (rng.integers(0, 2, size=shape).astype(np.uint8) << 7)


def dec(c, fmt=o.E4M3):
    return o.decode_array(c, fmt)


def softmax_reference(Q, K, V, s, causal):
    """Textbook float64 attention for one head: numpy only."""
    x = s * Q @ K.T
    if causal:
        x = np.where(np.tril(np.ones_like(x, dtype=bool)), x, -np.inf)
    x = x - x.max(axis=1, keepdims=True)
    P = np.exp(x)
    P /= P.sum(axis=1, keepdims=True)
    lse = None
    return P, P @ V


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("max_mode,kv_block", [(0, 0), (1, 0), (0, 3), (1, 4), (0, 1)])
def test_unquantised_forward_is_textbook_softmax_attention(causal, max_mode, kv_block):
    B, N, Hq, Hkv, d = 2, 11, 4, 2, 8
    q, k, v = rand_codes((B, N, Hq, d), 1), rand_codes((B, N, Hkv, d), 2), rand_codes((B, N, Hkv, d), 3)
    p = o.attn_params(B, N, Hq, Hkv, d, causal=causal, quant=False, kv_block=kv_block, max_mode=max_mode,
                      s=0.3, q_inv=0.5, k_inv=2.0, v_inv=0.25)
    O, LSE, _ = o.attention_fwd(q, k, v, p)
    Q, K, V = dec(q) * 0.5, dec(k) * 2.0, dec(v) * 0.25
    for b in range(B):
        for h in range(Hq):
            g = h // (Hq // Hkv)                        # grouped-query mapping
            P, ref = softmax_reference(Q[b, :, h], K[b, :, g], V[b, :, g], 0.3, causal)
            assert np.allclose(O[b * Hq + h], ref, rtol=1e-12, atol=1e-13)
            x = 0.3 * Q[b, :, h] @ K[b, :, g].T
            if causal:
                x = np.where(np.tril(np.ones_like(x, dtype=bool)), x, -np.inf)
            assert np.allclose(LSE[b * Hq + h], np.log(np.exp(x).sum(axis=1)), rtol=1e-12)


def test_rows_of_P_sum_to_one():
    """V = identity (d = N) makes O equal to P."""
    N = 16
    q, k = rand_codes((1, N, 1, N), 4), rand_codes((1, N, 1, N), 5)
    v = np.where(np.eye(N, dtype=bool), ONE, 0).astype(np.uint8).reshape(1, N, 1, N)
    for causal in (True, False):
        p = o.attn_params(1, N, 1, 1, N, causal=causal, quant=False, s=0.2)
        O, _, _ = o.attention_fwd(q, k, v, p)
        assert np.allclose(O[0].sum(axis=1), 1.0, atol=1e-12)
        if causal:
            assert np.all(np.triu(O[0], 1) == 0.0)


@pytest.mark.parametrize("quant", [True, False])
def test_closed_forms_single_key_zero_query_first_row(quant):
    B, N, H, d = 1, 9, 2, 8
    q, k, v = rand_codes((B, N, H, d), 6), rand_codes((B, N, H, d), 7), rand_codes((B, N, H, d), 8)
    V = dec(v) * 0.125
    # N = 1: O = V exactly (P~ = 1 -> code 0x7E = 448 = c_P)
    p1 = o.attn_params(1, 1, H, H, d, quant=quant, v_inv=0.125, max_mode=0)
    O, LSE, _ = o.attention_fwd(q[:, :1], k[:, :1], v[:, :1], p1)
    assert np.array_equal(O[:, 0], V[0, 0])
    # causal row 0 attends to key 0 only
    p = o.attn_params(B, N, H, H, d, quant=quant, v_inv=0.125, max_mode=0)
    O, LSE, _ = o.attention_fwd(q, k, v, p)
    assert np.array_equal(O[:, 0], V[0, 0])
    # Q == 0: uniform weights, O_i = mean of V_0..V_i, LSE_i = ln(i+1); exact in FP8 mode as well
    O, LSE, _ = o.attention_fwd(np.zeros_like(q), k, v, p)
    for h in range(H):
        pref = np.cumsum(V[0, :, h], axis=0) / np.arange(1, N + 1)[:, None]
        assert np.allclose(O[h], pref, rtol=1e-13, atol=0)
        assert np.allclose(LSE[h], np.log(np.arange(1, N + 1)), rtol=1e-13)


def test_key_permutation_invariance_non_causal():
    B, N, H, d = 1, 12, 1, 8
    q, k, v = rand_codes((B, N, H, d), 9), rand_codes((B, N, H, d), 10), rand_codes((B, N, H, d), 11)
    perm = np.random.default_rng(0).permutation(N)
    for quant in (False, True):
        p = o.attn_params(B, N, H, H, d, causal=False, quant=quant, kv_block=0)
        O1, L1, _ = o.attention_fwd(q, k, v, p)
        O2, L2, _ = o.attention_fwd(q, k[:, perm], v[:, perm], p)
        assert np.allclose(O1, O2, rtol=1e-12, atol=1e-14) and np.allclose(L1, L2, rtol=1e-13)


def test_quantised_forward_matches_stepwise_definition():
    """quant=on differs from the textbook form only by P8 = E4M3(P~ c_P) in the numerator."""
    B, N, H, d = 1, 10, 1, 8
    q, k, v = rand_codes((B, N, H, d), 12), rand_codes((B, N, H, d), 13), rand_codes((B, N, H, d), 14)
    for max_mode in (0, 1):
        p = o.attn_params(B, N, H, H, d, quant=True, s=0.4, max_mode=max_mode)
        O, LSE, mag = o.attention_fwd(q, k, v, p)
        Q, K, V = dec(q)[0, :, 0], dec(k)[0, :, 0], dec(v)[0, :, 0]
        x = np.where(np.tril(np.ones((N, N), dtype=bool)), 0.4 * Q @ K.T, -np.inf)
        m = x.max(axis=1, keepdims=True)
        if max_mode == 1:
            m = np.ceil(m * np.log2(np.e)) * np.log(2.0)
        Pt = np.exp(x - m)
        P8 = dec(o.encode_array((Pt.astype(np.float32) * np.float32(448.0)), o.E4M3))
        ref = (P8 @ V) / (448.0 * Pt.sum(axis=1, keepdims=True))
        assert np.allclose(O[0], ref, rtol=1e-12, atol=1e-14)
        assert np.allclose(LSE[0], (m + np.log(Pt.sum(axis=1, keepdims=True)))[:, 0], rtol=1e-13)
        assert np.allclose(mag[0], (P8 @ np.abs(V)) / (448.0 * Pt.sum(axis=1, keepdims=True)), rtol=1e-12)
        if max_mode == 1:   # reference maximum is an integer number of octaves above the true one
            assert np.all((Pt.max(axis=1) > 0.5) & (Pt.max(axis=1) <= 1.0))


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("kv_block,tau", [(3, 1.0), (4, 3.0), (1, 2.5)])
def test_reference_maximum_with_slack_leaves_unquantised_attention_unchanged(causal, kv_block, tau):
    """O and LSE do not depend on the reference maximum: with quant off the slack mode is the textbook result."""
    B, N, Hq, Hkv, d = 2, 13, 4, 2, 8
    q, k, v = rand_codes((B, N, Hq, d), 31), rand_codes((B, N, Hkv, d), 32), rand_codes((B, N, Hkv, d), 33)
    kw = dict(causal=causal, quant=False, kv_block=kv_block, s=0.3, q_inv=0.5, k_inv=2.0, v_inv=0.25)
    O0, L0, _ = o.attention_fwd(q, k, v, o.attn_params(B, N, Hq, Hkv, d, **kw))
    O1, L1, _ = o.attention_fwd(q, k, v, o.attn_params(B, N, Hq, Hkv, d, max_slack=tau, **kw))
    assert np.allclose(O0, O1, rtol=1e-12, atol=1e-13)
    assert np.allclose(L0, L1, rtol=1e-12)


def test_quantised_forward_with_slack_matches_stepwise_definition():
    """Slack tau: the reference maximum of a row moves only when a block maximum exceeds it by more than 2^tau, so
    P~ reaches at most 2^tau and is quantised with c_P = 448 / 2^tau.  Reference maximum rebuilt here block by block."""
    B, N, H, d, Bc, tau = 1, 12, 1, 8, 2, 2.0
    cP = 448.0 / 2.0 ** tau
    q, k, v = rand_codes((B, N, H, d), 42), rand_codes((B, N, H, d), 43), rand_codes((B, N, H, d), 44)
    p = o.attn_params(B, N, H, H, d, quant=True, s=0.9, kv_block=Bc, c_P=cP, max_slack=tau)
    O, LSE, _ = o.attention_fwd(q, k, v, p)
    Q, K, V = dec(q)[0, :, 0], dec(k)[0, :, 0], dec(v)[0, :, 0]
    x = np.where(np.tril(np.ones((N, N), dtype=bool)), 0.9 * Q @ K.T, -np.inf)
    moved_late = 0
    for i in range(N):
        m, num, l = -np.inf, np.zeros(d), 0.0
        for j0 in range(0, i + 1, Bc):
            blk = x[i, j0:min(j0 + Bc, i + 1)]
            if blk.max() > m + tau * np.log(2.0):
                f = 0.0 if np.isinf(m) else np.exp(m - blk.max())
                num, l, m = num * f, l * f, blk.max()
                moved_late += j0 > 0
            pt = np.exp(blk - m)
            assert pt.max() <= 2.0 ** tau * (1 + 1e-12)
            p8 = dec(o.encode_array(pt.astype(np.float32) * np.float32(cP), o.E4M3))
            num = num + p8 @ V[j0:j0 + len(blk)]
            l += pt.sum()
        assert np.allclose(O[0, i], num / (cP * l), rtol=1e-12, atol=1e-14)
        assert np.isclose(LSE[0, i], m + np.log(l), rtol=1e-13)
    assert moved_late > 0                      # the case does exercise a later move of the reference


def _fd_setup():
    rng = np.random.default_rng(21)
    B, N, Hq, Hkv, d = 1, 8, 2, 1, 4
    Q, K, V = rng.normal(size=(B, N, Hq, d)), rng.normal(size=(B, N, Hkv, d)), rng.normal(size=(B, N, Hkv, d))
    dO = rng.normal(size=(B, N, Hq, d))
    return B, N, Hq, Hkv, d, Q, K, V, dO


@pytest.mark.parametrize("causal", [True, False])
def test_unquantised_backward_matches_finite_differences(causal):
    B, N, Hq, Hkv, d, Q, K, V, dO = _fd_setup()
    s = 0.7
    p = o.attn_params(B, N, Hq, Hkv, d, causal=causal, quant=False, s=s, max_mode=0)

    def loss(Q_, K_, V_):
        O, _, _ = o.attention_fwd(Q_, K_, V_, p, real=True)       # [pair=(b,h), row, d]
        return float((O.reshape(B, Hq, N, d).transpose(0, 2, 1, 3) * dO).sum())

    O, LSE, _ = o.attention_fwd(Q, K, V, p, real=True)
    Ofull = O.reshape(B, Hq, N, d).transpose(0, 2, 1, 3)
    g = o.attention_bwd(Q, K, V, dO, Ofull, LSE.reshape(B, Hq, N), p, real=True)
    dQ = g["dQ"].reshape(B, Hkv, Hq // Hkv, N, d)
    h = 1e-5
    for name, T_, grad in (("Q", Q, None), ("K", K, g["dK"]), ("V", V, g["dV"])):
        for idx in np.ndindex(T_.shape):
            Tp, Tm = T_.copy(), T_.copy()
            Tp[idx] += h
            Tm[idx] -= h
            args_p = {"Q": (Tp, K, V), "K": (Q, Tp, V), "V": (Q, K, Tp)}[name]
            args_m = {"Q": (Tm, K, V), "K": (Q, Tm, V), "V": (Q, K, Tm)}[name]
            fd = (loss(*args_p) - loss(*args_m)) / (2 * h)
            b, n, hh, dd = idx
            if name == "Q":
                an = dQ[b, hh // (Hq // Hkv), hh % (Hq // Hkv), n, dd]
            else:
                an = grad[b * Hkv + hh, n, dd]
            assert abs(fd - an) <= 1e-6 * max(1.0, abs(an)), (name, idx, fd, an)


def test_backward_rows_of_dS_sum_to_zero():
    """K = identity (d = N) makes dQ_i = s * dS_i, and every row of dS sums to zero."""
    rng = np.random.default_rng(5)
    N = 8
    Q, V, dO = rng.normal(size=(1, N, 1, N)), rng.normal(size=(1, N, 1, N)), rng.normal(size=(1, N, 1, N))
    K = np.eye(N).reshape(1, N, 1, N)
    p = o.attn_params(1, N, 1, 1, N, causal=True, quant=False, s=0.9)
    O, LSE, _ = o.attention_fwd(Q, K, V, p, real=True)
    g = o.attention_bwd(Q, K, V, dO, O.reshape(1, N, 1, N), LSE.reshape(1, 1, N), p, real=True)
    assert np.allclose(g["dQ"][0, 0].sum(axis=1), 0.0, atol=1e-13)
    assert g["amax_dS"] == pytest.approx(np.abs(g["dQ"]).max() / 0.9, rel=1e-12)


@pytest.mark.parametrize("quant", [False, True])
def test_backward_zero_query_closed_form(quant):
    """Q == 0: P_ij = 1/(i+1); dV_j = sum_{i>=j} P8_ij/c_P dO_i with P8 = E4M3(448/(i+1))."""
    B, N, H, d = 1, 12, 1, 8
    k, v = rand_codes((B, N, H, d), 30), rand_codes((B, N, H, d), 31)
    do = rand_codes((B, N, H, d), 32, 0x10, 0x30)            # read as E5M2 codes
    q = np.zeros_like(k)
    p = o.attn_params(B, N, H, H, d, quant=quant, max_mode=0, do_inv=0.5, ds_scale=64.0)
    O, LSE, _ = o.attention_fwd(q, k, v, p)
    g = o.attention_bwd(q, k, v, do, O.reshape(B, N, H, d), LSE.reshape(B, H, N), p)
    dO = dec(do, o.E5M2)[0, :, 0] * 0.5
    w = 1.0 / np.arange(1, N + 1)
    if quant:
        w = dec(o.encode_array((w.astype(np.float32) * np.float32(448.0)), o.E4M3)) / 448.0
    exp = np.array([(w[j:, None] * dO[j:]).sum(axis=0) for j in range(N)])
    assert np.allclose(g["dV"][0], exp, rtol=1e-12, atol=1e-15)
    assert np.all(g["dK"] == 0.0)                            # dK_j = s sum_i dS_ij Q_i with Q = 0


def test_backward_ranges_compose():
    """Partial (query range x key range) results add up to the full backward."""
    B, N, Hq, Hkv, d = 1, 12, 2, 1, 8
    q, k, v = rand_codes((B, N, Hq, d), 40), rand_codes((B, N, Hkv, d), 41), rand_codes((B, N, Hkv, d), 42)
    do = rand_codes((B, N, Hq, d), 43, 0x10, 0x30)
    p = o.attn_params(B, N, Hq, Hkv, d, quant=True, ds_scale=16.0, do_inv=0.01)
    O, LSE, _ = o.attention_fwd(q, k, v, p)
    Of = O.reshape(B, Hq, N, d).transpose(0, 2, 1, 3)
    L = LSE.reshape(B, Hq, N)
    full = o.attention_bwd(q, k, v, do, Of, L, p)
    # causal: rows [0,6) see keys [0,6) only; keys [6,12) are seen by rows [6,12) only
    a = o.attention_bwd(q, k, v, do, Of, L, p, q_rows=(0, 6), k_rows=(0, 6))
    b = o.attention_bwd(q, k, v, do, Of, L, p, q_rows=(6, 12), k_rows=(6, 12))
    assert np.allclose(a["dQ"], full["dQ"][:, :, :6], rtol=1e-13, atol=1e-300)
    assert np.allclose(b["dK"], full["dK"][:, 6:], rtol=1e-13, atol=1e-300)
    assert np.allclose(b["dV"], full["dV"][:, 6:], rtol=1e-13, atol=1e-300)


def test_softmax_scale_fold_identity():
    """Section 3 (QK regularisation): a frozen gain g on normalised Q and K equals scaling s by g^2."""
    B, N, H, d = 1, 6, 1, 8
    q, k, v = rand_codes((B, N, H, d), 50), rand_codes((B, N, H, d), 51), rand_codes((B, N, H, d), 52)
    g2 = 2.0 ** 0.5                     # s = 0.125 at d = 128 corresponds to gamma^2 = sqrt(2)
    p1 = o.attn_params(B, N, H, H, d, quant=False, s=g2 / d ** 0.5)
    p2 = o.attn_params(B, N, H, H, d, quant=False, s=1 / d ** 0.5, q_inv=g2 ** 0.5, k_inv=g2 ** 0.5)
    O1, _, _ = o.attention_fwd(q, k, v, p1)
    O2, _, _ = o.attention_fwd(q, k, v, p2)
    assert np.allclose(O1, O2, rtol=1e-12)
    assert abs(0.125 * 128 ** 0.5 - g2) < 1e-12


def test_tie_slack_outputs():
    """slack_* bound the effect of FP32-vs-double tie decisions: zero without flip_eps, monotone in it, and
    with an absurdly large eps every term counts with the full gap between neighbouring codes."""
    B, N, H, d = 1, 10, 1, 8
    q, k, v = rand_codes((B, N, H, d), 60), rand_codes((B, N, H, d), 61), rand_codes((B, N, H, d), 62)
    do = rand_codes((B, N, H, d), 63, 0x10, 0x30)
    prev_f, prev_b = None, None
    for eps in (0.0, 1e-6, 1e-2, 1e3):
        p = o.attn_params(B, N, H, H, d, quant=True, s=0.4, ds_scale=64.0, flip_eps=eps)
        O, LSE, mag, slack = o.attention_fwd(q, k, v, p, with_slack=True)
        g = o.attention_bwd(q, k, v, do, O.reshape(B, N, H, d), LSE.reshape(B, H, N), p)
        tot_b = sum(g["slack_" + n].sum() for n in ("dQ", "dK", "dV"))
        if eps == 0.0:
            assert slack.sum() == 0.0 and tot_b == 0.0
        else:
            assert slack.sum() >= prev_f and tot_b >= prev_b
        prev_f, prev_b = slack.sum(), tot_b
    assert (slack > 0).all()
    # Q = 0: every P~ c_P is exactly 448 (the top code, no neighbour above, the one below is 32 away)
    p = o.attn_params(B, N, H, H, d, quant=True, flip_eps=1e-6)
    _, _, _, slack = o.attention_fwd(np.zeros_like(q), k, v, p, with_slack=True)
    assert slack.sum() == 0.0


def _stepwise_quantised_backward(q, k, v, do, O, LSE, s, q_inv, k_inv, v_inv, do_inv, ds_scale, causal, cP=448.0):
    """The quantised backward rebuilt in numpy, one (batch, head) at a time, in the order of the definition:
    P = exp(x - LSE); P8 = E4M3(fl32(P) fl32(c_P)); dV += P8^T dO / c_P; dP = dO V^T; D = rowsum(dO * O);
    dS = P (dP - D); dS8 = E5M2(fl32(dS) fl32(ds_scale)); dQ = s dS8 K / ds_scale; dK += s dS8^T Q / ds_scale."""
    B, N, Hq, d = q.shape
    Hkv = k.shape[2]
    G = Hq // Hkv
    Qc, Kc, Vc, dOc = dec(q), dec(k), dec(v), dec(do, o.E5M2)
    dQ = np.zeros((B, Hq, N, d))
    dK = np.zeros((B, Hkv, N, d))
    dV = np.zeros((B, Hkv, N, d))
    m8Q = np.zeros_like(dQ)
    m8K = np.zeros_like(dK)
    amax, nsat = 0.0, 0
    mask = np.tril(np.ones((N, N), dtype=bool)) if causal else np.ones((N, N), dtype=bool)
    for b in range(B):
        for h in range(Hq):
            g = h // G
            x = s * q_inv * k_inv * (Qc[b, :, h] @ Kc[b, :, g].T)
            P = np.where(mask, np.exp(x - LSE[b, h][:, None]), 0.0)
            P8 = dec(o.encode_array(P.astype(np.float32) * np.float32(cP), o.E4M3))
            dOr = do_inv * dOc[b, :, h]
            D = (dOr * O[b, :, h]).sum(axis=1)
            dV[b, g] += P8.T @ dOr / cP
            dP = do_inv * v_inv * (dOc[b, :, h] @ Vc[b, :, g].T)
            dS = np.where(mask, P * (dP - D[:, None]), 0.0)
            amax = max(amax, np.abs(dS).max())
            prod = dS.astype(np.float32) * np.float32(ds_scale)
            nsat += int((np.abs(prod) > 57344.0).sum())
            dS8 = dec(o.encode_array(prod, o.E5M2), o.E5M2) / ds_scale
            dQ[b, h] = s * k_inv * (dS8 @ Kc[b, :, g])
            dK[b, g] += s * q_inv * (dS8.T @ Qc[b, :, h])
            m8Q[b, h] = s * k_inv * (np.abs(dS8) @ np.abs(Kc[b, :, g]))
            m8K[b, g] += s * q_inv * (np.abs(dS8).T @ np.abs(Qc[b, :, h]))
    return dQ, dK, dV, m8Q, m8K, amax, nsat


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("ds_scale,expect_saturation", [(2048.0, False), (3.0e7, True)])
def test_quantised_backward_matches_stepwise_definition(causal, ds_scale, expect_saturation):
    """quant=on differs from the textbook gradient only by the two encodes, placed where a product's operand is
    formed: P8 feeds dV, dS8 feeds dQ and dK.  Two query heads per key/value head, so the group sum is covered;
    the large ds_scale pushes dS * ds_scale past 57344, where the cast saturates."""
    B, N, Hq, Hkv, d = 2, 10, 4, 2, 8
    q, k, v = rand_codes((B, N, Hq, d), 70), rand_codes((B, N, Hkv, d), 71), rand_codes((B, N, Hkv, d), 72)
    do = rand_codes((B, N, Hq, d), 73, 0x10, 0x30)           # read as E5M2 codes
    kw = dict(s=0.35, q_inv=0.5, k_inv=1.5, v_inv=0.25, do_inv=0.125)
    p = o.attn_params(B, N, Hq, Hkv, d, causal=causal, quant=True, ds_scale=ds_scale, **kw)
    # O and LSE are inputs of the backward: LSE is the log-sum-exp of the scores, O any tensor (here the textbook one)
    Qr, Kr, Vr = dec(q) * 0.5, dec(k) * 1.5, dec(v) * 0.25
    O = np.empty((B, N, Hq, d))
    LSE = np.empty((B, Hq, N))
    for b in range(B):
        for h in range(Hq):
            g = h // (Hq // Hkv)
            P, O[b, :, h] = softmax_reference(Qr[b, :, h], Kr[b, :, g], Vr[b, :, g], 0.35, causal)
            x = 0.35 * Qr[b, :, h] @ Kr[b, :, g].T
            if causal:
                x = np.where(np.tril(np.ones_like(x, dtype=bool)), x, -np.inf)
            LSE[b, h] = np.log(np.exp(x).sum(axis=1))
    g_ = o.attention_bwd(q, k, v, do, O, LSE, p)
    dQ, dK, dV, m8Q, m8K, amax, nsat = _stepwise_quantised_backward(q, k, v, do, O, LSE, ds_scale=ds_scale,
                                                                    causal=causal, **kw)
    assert (nsat > 0) == expect_saturation
    G = Hq // Hkv
    got_dQ = g_["dQ"].reshape(B, Hkv, G, N, d).reshape(B, Hq, N, d)
    assert np.allclose(got_dQ, dQ, rtol=1e-11, atol=1e-300)
    assert np.allclose(g_["dK"].reshape(B, Hkv, N, d), dK, rtol=1e-11, atol=1e-300)
    assert np.allclose(g_["dV"].reshape(B, Hkv, N, d), dV, rtol=1e-11, atol=1e-300)
    assert np.isclose(g_["amax_dS"], amax, rtol=1e-12)
    assert np.allclose(g_["mag8_dQ"].reshape(B, Hq, N, d), m8Q, rtol=1e-11)
    assert np.allclose(g_["mag8_dK"].reshape(B, Hkv, N, d), m8K, rtol=1e-11)
    assert np.all(np.abs(dK).max(axis=(0, 2, 3)) > 0) and np.abs(dQ).max() > 0
    if expect_saturation:
        # a saturated dS8 is +-57344 / ds_scale: the result differs from the un-saturated product
        unsat = o.attention_bwd(q, k, v, do, O, LSE, o.attn_params(B, N, Hq, Hkv, d, causal=causal, quant=False, **kw))
        assert not np.allclose(unsat["dQ"], g_["dQ"], rtol=0.2)


def test_quantised_backward_pin_catches_plausible_mistakes():
    """The step-wise rebuild separates the variants a mistaken oracle could implement: dS quantised in E4M3,
    P8 (not P) inside dS, a missing 1/ds_scale — each moves the result by far more than the pin's tolerance."""
    B, N, H, d = 1, 10, 1, 8
    q, k, v = rand_codes((B, N, H, d), 80), rand_codes((B, N, H, d), 81), rand_codes((B, N, H, d), 82)
    do = rand_codes((B, N, H, d), 83, 0x10, 0x30)
    p = o.attn_params(B, N, H, H, d, quant=True, s=0.4, ds_scale=512.0)
    O, LSE, _ = o.attention_fwd(q, k, v, p)
    g_ = o.attention_bwd(q, k, v, do, O.reshape(B, N, H, d), LSE.reshape(B, H, N), p)
    Qc, Kc, Vc, dOc = dec(q)[0, :, 0], dec(k)[0, :, 0], dec(v)[0, :, 0], dec(do, o.E5M2)[0, :, 0]
    mask = np.tril(np.ones((N, N), dtype=bool))
    P = np.where(mask, np.exp(0.4 * Qc @ Kc.T - LSE[0][:, None]), 0.0)
    P8 = dec(o.encode_array(P.astype(np.float32) * np.float32(448.0), o.E4M3)) / 448.0
    D = (dOc * O[0]).sum(axis=1)
    dP = dOc @ Vc.T
    right = P * (dP - D[:, None])
    variants = {
        "e4m3": dec(o.encode_array((right * 512.0).astype(np.float32), o.E4M3)) / 512.0,
        "p8_in_dS": dec(o.encode_array((P8 * (dP - D[:, None]) * 512.0).astype(np.float32), o.E5M2), o.E5M2) / 512.0,
        "no_descale": dec(o.encode_array((right * 512.0).astype(np.float32), o.E5M2), o.E5M2),
    }
    good = dec(o.encode_array((right * 512.0).astype(np.float32), o.E5M2), o.E5M2) / 512.0
    assert np.allclose(g_["dQ"][0, 0], 0.4 * good @ Kc, rtol=1e-11, atol=1e-300)
    for name, ds8 in variants.items():
        assert not np.allclose(g_["dQ"][0, 0], 0.4 * ds8 @ Kc, rtol=1e-6, atol=1e-300), name


def test_flip_step_hand_worked_values():
    """The tie band: a value within `band` of the midpoint between two neighbouring codes may go to either, and
    the function returns the gap between them; anywhere else it returns 0."""
    f = o.flip_step
    E4, E5 = o.E4M3, o.E5M2
    # E4M3 around 1: codes 0x38 = 1, 0x39 = 1.125, midpoint 1.0625, gap 0.125
    assert f(1.0625, 1e-9, E4) == 0.125
    assert f(-1.0625, 1e-9, E4) == 0.125                      # sign-symmetric
    assert f(1.0625 + 0.004, 0.005, E4) == 0.125              # inside the band, above the midpoint (code 0x39)
    assert f(1.0625 - 0.004, 0.005, E4) == 0.125              # inside the band, below it (code 0x38)
    assert f(1.0625 + 0.006, 0.005, E4) == 0.0                # just outside
    assert f(1.0625 - 0.006, 0.005, E4) == 0.0
    assert f(1.0, 0.01, E4) == 0.0                            # on a code, far from both midpoints
    assert f(1.0625, 0.0, E4) == 0.0                          # band 0 switches the rule off
    # binade boundary: 1.875 | 2.0 | 2.25 — the gap differs on the two sides of 2
    assert f(1.9375, 1e-9, E4) == 0.125
    assert f(2.125, 1e-9, E4) == 0.25
    # top of the range: 416 | 448, nothing above 448 (the cast saturates, so no flip there)
    assert f(432.0, 1e-6, E4) == 32.0
    assert f(448.0, 1.0, E4) == 0.0
    assert f(449.0, 2.0, E4) == 0.0
    assert f(1e4, 1.0, E4) == 0.0
    assert f(450.0, 20.0, E4) == 32.0                         # saturated, but the band reaches down to 432
    assert f(464.0, 20.0, E4) == 0.0                          # 32 above the midpoint: out of a band of 20
    # subnormal range of E4M3: grid of 2^-9 up to 2^-6
    u = 2.0 ** -9
    assert f(0.5 * u, 1e-12, E4) == u                         # between 0 and the smallest subnormal
    assert f(1.5 * u, 1e-12, E4) == u
    assert f(7.5 * u, 1e-12, E4) == u                         # last subnormal | first normal
    assert f(8.5 * u, 1e-12, E4) == u                         # first normal binade has the same spacing
    assert f(16.5 * u, 1e-12, E4) == 0.0                      # 2^-5 binade: spacing 2u, 16.5u is not a midpoint
    assert f(17.0 * u, 1e-12, E4) == 2 * u
    assert f(0.0, 1e-12, E4) == 0.0
    # E5M2: 1 | 1.25 (gap 0.25), top 49152 | 57344 (gap 8192), subnormal grid 2^-16
    assert f(1.125, 1e-9, E5) == 0.25
    assert f(1.125 + 0.02, 0.01, E5) == 0.0
    assert f(53248.0, 1e-3, E5) == 8192.0
    assert f(57344.0, 100.0, E5) == 0.0
    assert f(1.5 * 2.0 ** -16, 1e-15, E5) == 2.0 ** -16
    # consistency with the encoder on every pair of neighbouring finite codes
    for fmt, top in ((E4, 0x7E), (E5, 0x7B)):
        t = o.decode_table(fmt)
        for c in range(top):
            mid, gap = 0.5 * (t[c] + t[c + 1]), t[c + 1] - t[c]
            assert f(mid, gap * 1e-6, fmt) == gap
            assert f(mid + 0.26 * gap, 0.25 * gap, fmt) == 0.0
            assert f(mid - 0.26 * gap, 0.25 * gap, fmt) == 0.0
