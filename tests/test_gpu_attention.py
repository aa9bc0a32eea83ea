"""GPU parity: FP8 attention forward / backward against the oracle on identical FP8 codes."""
import numpy as np
import pytest
import torch

import oracle as o
import paper_2505_20524_b200 as fp8
from paper_2505_20524_b200 import synth
from gpu_util import (dev, host, scalar, gpu_quantize, rel_err, quantile_err, norm_ratios, report, BWD_FLOOR, FLIP_EPS,
                      FRO_FWD, FRO_BWD)

pytestmark = pytest.mark.gpu

TOL_FWD = 2e-2     # max |gpu - ref| / sum_j P8_ij |V_jd| (normalised like O)
TOL_BWD = 3e-2
KV_BLOCK = 128     # the kernel takes keys in blocks of 128 with an exact running maximum


def quantized_qkv(cfg, N, B, seed_shift=0):
    q, k, v, do = synth.attention_inputs(cfg, seq=N, batch=B)
    out = {}
    for name, t, fmt in (("q", q, o.E4M3), ("k", k, o.E4M3), ("v", v, o.E4M3), ("do", do, o.E5M2)):
        c, a, s, si = o.quantize(t, fmt)
        out[name] = (c, float(si))
    return out


def run_fwd(qd, B, N, Hq, Hkv, d, causal, s, p_scale=448.0, max_slack=0.0):
    q8, k8, v8 = dev(qd["q"][0]), dev(qd["k"][0]), dev(qd["v"][0])
    O = torch.empty((B, N, Hq, d), dtype=torch.bfloat16, device="cuda")
    LSE = torch.empty((B, Hq, N), dtype=torch.float32, device="cuda")
    fp8.fp8_attention_fwd(q8, k8, v8, scalar(qd["q"][1]), scalar(qd["k"][1]), scalar(qd["v"][1]), s, causal,
                          O, LSE, None, p_scale=p_scale, max_slack=max_slack)
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    return O, LSE


@pytest.mark.parametrize("name,B,N,causal", [("c1", 1, 256, True), ("c1", 2, 128, True), ("c1", 1, 400, True),
                                             ("c1", 1, 256, False), ("c1", 1, 16, True), ("c1", 1, 208, False),
                                             ("c3", 1, 384, True), ("c4", 1, 272, True), ("c4", 1, 256, False),
                                             ("c3", 2, 144, True), ("c4", 2, 112, False)])
def test_forward_matches_oracle(name, B, N, causal):
    cfg = synth.CONFIGS[name]
    Hq, Hkv, d = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    if name != "c1":
        Hq, Hkv = Hq // 4, Hkv // 4          # a few heads are enough at this size
        cfg = synth.BlockConfig(**{**cfg.__dict__, "n_q_heads": Hq, "n_kv_heads": Hkv})
    qd = quantized_qkv(cfg, N, B)
    s = d ** -0.5
    O, LSE = run_fwd(qd, B, N, Hq, Hkv, d, causal, s)
    p = o.attn_params(B, N, Hq, Hkv, d, causal=causal, quant=True, kv_block=KV_BLOCK, max_mode=0, s=s,
                      q_inv=qd["q"][1], k_inv=qd["k"][1], v_inv=qd["v"][1], flip_eps=FLIP_EPS)
    ref, lse, mag, slack = o.attention_fwd(qd["q"][0], qd["k"][0], qd["v"][0], p, with_slack=True)
    got = O.float().cpu().numpy().astype(np.float64).transpose(0, 2, 1, 3).reshape(B * Hq, N, d)
    err = rel_err(got, ref, mag, slack)
    assert err <= TOL_FWD, err
    assert slack.sum() <= 1e-2 * mag.sum()    # tie decisions are the exception, not a blanket excuse
    glse = LSE.cpu().numpy().astype(np.float64).reshape(B * Hq, N)
    assert np.max(np.abs(glse - lse)) <= 1e-3 * max(1.0, np.abs(lse).max())
    fro, inf = norm_ratios(got, ref)
    assert fro <= FRO_FWD, fro
    # information, not gates: how far the kernel is from the schedule-free oracle (whole row at once) and from
    # attention without the P8 encode; both differences are quantisation noise of P8, not kernel error
    kw = dict(causal=causal, max_mode=0, s=s, q_inv=qd["q"][1], k_inv=qd["k"][1], v_inv=qd["v"][1])
    ref0, _, mag0 = o.attention_fwd(qd["q"][0], qd["k"][0], qd["v"][0],
                                    o.attn_params(B, N, Hq, Hkv, d, quant=True, kv_block=0, **kw))
    refu, _, _ = o.attention_fwd(qd["q"][0], qd["k"][0], qd["v"][0],
                                 o.attn_params(B, N, Hq, Hkv, d, quant=False, kv_block=0, **kw))
    report("fwd %s B%d N%d causal=%d" % (name, B, N, causal), max_rel=err, raw_max_rel=rel_err(got, ref, mag),
           fro=fro, inf=inf, vs_whole_row_max=rel_err(got, ref0, mag0), vs_whole_row_fro=norm_ratios(got, ref0)[0],
           vs_unquantised_max=rel_err(got, refu, mag0), vs_unquantised_fro=norm_ratios(got, refu)[0],
           oracle_whole_row_vs_blocked_fro=norm_ratios(ref0, ref)[0])


@pytest.mark.parametrize("family", ["single", "pair", "stream2", "stream"])
@pytest.mark.parametrize("name,B,N,causal", [("c3", 1, 656, True), ("c4", 2, 400, True), ("c4", 1, 272, False),
                                             ("c3", 3, 128, True)])
def test_forward_kernel_families_at_head_dim_128(family, name, B, N, causal, monkeypatch):
    """FP8DPA_ATTN_FWD picks the d = 128 kernel: one tile per CTA, two tiles per CTA, or the persistent kernel whose CTAs
    walk several (tile, head, batch) items with two or three (the default) softmax warpgroups taking the key blocks in turn.
    All four must agree with the oracle; the shapes give CTAs of the persistent kernel items of different lengths, block
    counts of every residue (the warpgroups change roles from item to item), a ragged last tile and grouped heads."""
    monkeypatch.setenv("FP8DPA_ATTN_FWD", family)
    cfg = synth.CONFIGS[name]
    Hq, Hkv, d = cfg.n_q_heads // 4, cfg.n_kv_heads // 4, cfg.head_dim
    cfg = synth.BlockConfig(**{**cfg.__dict__, "n_q_heads": Hq, "n_kv_heads": Hkv})
    qd = quantized_qkv(cfg, N, B)
    s = d ** -0.5
    O, LSE = run_fwd(qd, B, N, Hq, Hkv, d, causal, s)
    p = o.attn_params(B, N, Hq, Hkv, d, causal=causal, quant=True, kv_block=KV_BLOCK, max_mode=0, s=s,
                      q_inv=qd["q"][1], k_inv=qd["k"][1], v_inv=qd["v"][1], flip_eps=FLIP_EPS)
    ref, lse, mag, slack = o.attention_fwd(qd["q"][0], qd["k"][0], qd["v"][0], p, with_slack=True)
    got = O.float().cpu().numpy().astype(np.float64).transpose(0, 2, 1, 3).reshape(B * Hq, N, d)
    assert rel_err(got, ref, mag, slack) <= TOL_FWD
    glse = LSE.cpu().numpy().astype(np.float64).reshape(B * Hq, N)
    assert np.max(np.abs(glse - lse)) <= 1e-3 * max(1.0, np.abs(lse).max())


@pytest.mark.parametrize("N,B,Hq,Hkv", [(16, 1, 1, 1), (112, 2, 4, 2), (128, 1, 8, 1), (144, 3, 2, 2), (272, 1, 40, 8),
                                        (400, 2, 4, 2), (784, 1, 8, 1), (1296, 1, 4, 2), (3088, 1, 8, 1)])
def test_forward_kernel_families_agree_over_many_item_layouts(N, B, Hq, Hkv, monkeypatch):
    """The persistent kernels give every CTA a different list of items (1 to 25 key blocks each, more or fewer items than
    CTAs, warpgroups changing roles at every item boundary).  Random codes, all four d = 128 kernels, causal and not, exact
    and slack reference maximum: the same codes must come out up to the BF16 rounding of O (the kernels differ only in the
    order of the row sum) and no bounded wait may expire."""
    d = 128
    g = torch.Generator(device="cuda").manual_seed(N * 131 + B * 17 + Hq)
    def codes(*shape):
        c = torch.randint(0x20, 0x50, shape, dtype=torch.uint8, device="cuda", generator=g)
        return c | (torch.randint(0, 2, shape, dtype=torch.uint8, device="cuda", generator=g) << 7)
    q8, k8, v8 = codes(B, N, Hq, d), codes(B, N, Hkv, d), codes(B, N, Hkv, d)
    s1 = scalar(0.04)
    def run(kind, causal, tau):
        monkeypatch.setenv("FP8DPA_ATTN_FWD", kind)
        O = torch.zeros((B, N, Hq, d), dtype=torch.bfloat16, device="cuda")
        LSE = torch.zeros((B, Hq, N), dtype=torch.float32, device="cuda")
        fp8.fp8_attention_fwd(q8, k8, v8, s1, s1, s1, d ** -0.5, causal, O, LSE, None, p_scale=448.0 / 2 ** tau, max_slack=tau)
        torch.cuda.synchronize()
        assert fp8.fp8_device_status() == 0, kind
        return O.float(), LSE
    for causal in (True, False):
        if not causal and N > 1300:
            continue
        for tau in (0.0, 2.0):
            ref = run("single", causal, tau)
            for kind in ("pair", "stream2", "stream"):
                O, LSE = run(kind, causal, tau)
                assert torch.isfinite(O).all()
                assert (O - ref[0]).abs().max() <= 2.0 ** -7 * ref[0].abs().max(), (kind, causal, tau)
                assert (LSE - ref[1]).abs().max() <= 1e-4, (kind, causal, tau)


@pytest.mark.parametrize("name,B,N,causal,tau", [("c1", 1, 400, True, 3.0), ("c3", 1, 384, True, 3.0),
                                                 ("c4", 1, 272, True, 2.0), ("c4", 1, 256, False, 3.0)])
def test_forward_with_reference_maximum_slack_matches_oracle(name, B, N, causal, tau):
    """The reference maximum of a row moves only when exceeded by more than 2^tau; P~ is scaled by 448 / 2^tau."""
    cfg = synth.CONFIGS[name]
    Hq, Hkv, d = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    if name != "c1":
        Hq, Hkv = Hq // 4, Hkv // 4
        cfg = synth.BlockConfig(**{**cfg.__dict__, "n_q_heads": Hq, "n_kv_heads": Hkv})
    qd = quantized_qkv(cfg, N, B)
    s = d ** -0.5
    c_P = 448.0 / 2.0 ** tau
    O, LSE = run_fwd(qd, B, N, Hq, Hkv, d, causal, s, p_scale=c_P, max_slack=tau)
    p = o.attn_params(B, N, Hq, Hkv, d, causal=causal, quant=True, kv_block=KV_BLOCK, max_mode=0, s=s, c_P=c_P,
                      max_slack=tau, q_inv=qd["q"][1], k_inv=qd["k"][1], v_inv=qd["v"][1], flip_eps=FLIP_EPS)
    ref, lse, mag, slack = o.attention_fwd(qd["q"][0], qd["k"][0], qd["v"][0], p, with_slack=True)
    got = O.float().cpu().numpy().astype(np.float64).transpose(0, 2, 1, 3).reshape(B * Hq, N, d)
    # a row whose block maximum sits within rounding of reference + 2^tau may move its reference on one side only:
    # both results are valid there (O does not depend on the reference), they differ by quantisation noise of P8
    err = np.maximum(np.abs(got - ref) - slack, 0.0) / np.maximum(mag, 1e-30)
    assert np.quantile(err, 0.999) <= TOL_FWD, np.quantile(err, 0.999)
    assert err.max() <= 4 * TOL_FWD, err.max()
    glse = LSE.cpu().numpy().astype(np.float64).reshape(B * Hq, N)
    assert np.max(np.abs(glse - lse)) <= 1e-3 * max(1.0, np.abs(lse).max())
    # and against the exact-maximum result of the same kernel: the same attention up to P8 quantisation noise
    O0, _ = run_fwd(qd, B, N, Hq, Hkv, d, causal, s)
    g0 = O0.float().cpu().numpy().astype(np.float64).transpose(0, 2, 1, 3).reshape(B * Hq, N, d)
    assert np.quantile(np.abs(got - g0) / np.maximum(mag, 1e-30), 0.999) <= 6e-2


def test_reference_maximum_slack_validation():
    cfg = synth.CONFIGS["c1"]
    qd = quantized_qkv(cfg, 128, 1)
    with pytest.raises(fp8.Fp8Error) as e:        # P~ would reach 8 * 448
        run_fwd(qd, 1, 128, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, True, 0.125, p_scale=448.0, max_slack=3.0)
    assert e.value.status == -3


def test_softmax_scale_parameter():
    """s = 0.125 at d = 128 (the frozen-gain QK-norm setting of Appendix A) instead of 1/sqrt(d)."""
    cfg = synth.BlockConfig(**{**synth.CONFIGS["c3"].__dict__, "n_q_heads": 2, "n_kv_heads": 2})
    B, N, d = 1, 256, 128
    qd = quantized_qkv(cfg, N, B)
    O, LSE = run_fwd(qd, B, N, 2, 2, d, True, 0.125)
    p = o.attn_params(B, N, 2, 2, d, causal=True, quant=True, kv_block=KV_BLOCK, s=0.125,
                      q_inv=qd["q"][1], k_inv=qd["k"][1], v_inv=qd["v"][1], flip_eps=FLIP_EPS)
    ref, lse, mag, slack = o.attention_fwd(qd["q"][0], qd["k"][0], qd["v"][0], p, with_slack=True)
    got = O.float().cpu().numpy().astype(np.float64).transpose(0, 2, 1, 3).reshape(B * 2, N, d)
    assert rel_err(got, ref, mag, slack) <= TOL_FWD


def mag8_stats(got, ref, name, tol=TOL_BWD):
    """|gpu - ref| (less the tie slack) over the sum of |dS8||K| (resp. |Q|), element by element: quantiles, the share
    of elements above the gate, and how strongly dS cancelled (mag / mag8) on the elements above it."""
    diff = np.maximum(np.abs(got - ref[name]) - ref["slack_" + name], 0.0).ravel()
    mag, mag8 = ref["mag_" + name].ravel(), ref["mag8_" + name].ravel()
    e8 = diff / np.maximum(mag8, max(1e-30, BWD_FLOOR * float(mag8.mean())))
    over = e8 > tol
    cancel = mag / np.maximum(mag8, 1e-300)
    keep = cancel <= 4.0                       # elements whose dS did not cancel by more than 4x
    out = {"q50": float(np.quantile(e8, 0.5)), "q99": float(np.quantile(e8, 0.99)),
           "q999": float(np.quantile(e8, 0.999)), "max": float(e8.max()), "share_over": float(over.mean()),
           "min_cancel_of_over": float(cancel[over].min()) if over.any() else 0.0,
           "share_uncancelled": float(keep.mean()),
           "max_uncancelled": float(e8[keep].max()) if keep.any() else 0.0}
    return out


def oracle_fwd_for_bwd(qd, p, B, N, Hq, d):
    """Oracle forward; returns O as BF16 bits [B,N,Hq,d] and LSE float32 [B,Hq,N] (what a framework saves)."""
    ref, lse, _ = o.attention_fwd(qd["q"][0], qd["k"][0], qd["v"][0], p)
    O = ref.reshape(B, Hq, N, d).transpose(0, 2, 1, 3)
    O_bits = synth.f32_to_bf16(O.astype(np.float32))
    return O_bits, lse.reshape(B, Hq, N).astype(np.float32)


def run_bwd(qd, O_bits, lse32, B, N, Hq, Hkv, d, causal, s, ds_scale):
    q8, k8, v8, do8 = dev(qd["q"][0]), dev(qd["k"][0]), dev(qd["v"][0]), dev(qd["do"][0])
    dQ = torch.empty((B, N, Hq, d), dtype=torch.bfloat16, device="cuda")
    dK = torch.empty((B, N, Hkv, d), dtype=torch.bfloat16, device="cuda")
    dV = torch.empty((B, N, Hkv, d), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(fp8.fp8_attention_workspace_bytes(1, B, N, Hq, Hkv, d), dtype=torch.uint8, device="cuda")
    amax = scalar(-1.0)
    fp8.fp8_attention_bwd(q8, k8, v8, do8, dev(O_bits), dev(lse32), scalar(qd["q"][1]), scalar(qd["k"][1]),
                          scalar(qd["v"][1]), scalar(qd["do"][1]), s, scalar(ds_scale), causal, dQ, dK, dV, ws,
                          ds_amax=amax)
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    return dQ, dK, dV, float(amax.item())


@pytest.mark.parametrize("name,B,N,causal", [("c1", 1, 256, True), ("c1", 2, 128, True), ("c1", 1, 400, True),
                                             ("c1", 1, 256, False), ("c1", 1, 16, True),
                                             ("c3", 1, 384, True), ("c4", 1, 272, True), ("c4", 1, 256, False),
                                             # d = 128 corner cases of the two-group kernel: a single sub-tile per CTA,
                                             # an odd number of sub-tiles, a ragged tail, grouped heads on one tile
                                             ("c3", 1, 64, True), ("c3", 2, 144, True), ("c3", 1, 192, False),
                                             ("c4", 1, 64, True), ("c4", 2, 112, False)])
def test_backward_matches_oracle(name, B, N, causal):
    cfg = synth.CONFIGS[name]
    Hq, Hkv, d = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    if name != "c1":
        Hq, Hkv = Hq // 4, Hkv // 4
        cfg = synth.BlockConfig(**{**cfg.__dict__, "n_q_heads": Hq, "n_kv_heads": Hkv})
    G = Hq // Hkv
    qd = quantized_qkv(cfg, N, B)
    s = d ** -0.5
    kw = dict(causal=causal, quant=True, kv_block=KV_BLOCK, max_mode=0, s=s, q_inv=qd["q"][1], k_inv=qd["k"][1],
              v_inv=qd["v"][1], do_inv=qd["do"][1])
    p = o.attn_params(B, N, Hq, Hkv, d, ds_scale=1.0, **kw)
    O_bits, lse32 = oracle_fwd_for_bwd(qd, p, B, N, Hq, d)
    Of = synth.bf16_to_f32(O_bits).astype(np.float64)
    args = (qd["q"][0], qd["k"][0], qd["v"][0], qd["do"][0], Of, lse32.astype(np.float64))
    # delayed-scaling style calibration of the dS scale: one oracle pass with scale 1 gives amax(dS)
    cal = o.attention_bwd(*args, p)
    ds_scale, _ = o.scale(np.float32(cal["amax_dS"]), o.E5M2)
    p = o.attn_params(B, N, Hq, Hkv, d, ds_scale=float(ds_scale), flip_eps=FLIP_EPS, **kw)
    ref = o.attention_bwd(*args, p)
    dQ, dK, dV, amax = run_bwd(qd, O_bits, lse32, B, N, Hq, Hkv, d, causal, s, float(ds_scale))
    assert abs(amax - ref["amax_dS"]) <= 1e-3 * ref["amax_dS"]
    gq = dQ.float().cpu().numpy().astype(np.float64).reshape(B, N, Hkv, G, d).transpose(0, 2, 3, 1, 4)
    gq = gq.reshape(B * Hkv, G, N, d)
    gk = dK.float().cpu().numpy().astype(np.float64).transpose(0, 2, 1, 3).reshape(B * Hkv, N, d)
    gv = dV.float().cpu().numpy().astype(np.float64).transpose(0, 2, 1, 3).reshape(B * Hkv, N, d)
    errs = {n_: rel_err(g_, ref[n_], ref["mag_" + n_], ref["slack_" + n_], BWD_FLOOR)
            for n_, g_ in (("dQ", gq), ("dK", gk), ("dV", gv))}
    assert max(errs.values()) <= TOL_BWD, errs
    for n_ in ("dQ", "dK", "dV"):
        assert ref["slack_" + n_].sum() <= 1e-2 * ref["mag_" + n_].sum()
    # the same differences against the denominators built from the quantised dS8 (sum |dS8||K| resp. |Q|): smaller than
    # mag wherever dP - D cancels (one-hot softmax rows, which the outlier channels produce)
    m = {}
    for n_, g_ in (("dQ", gq), ("dK", gk)):
        st = mag8_stats(g_, ref, n_)
        m.update({n_ + "_mag8_" + k: v for k, v in st.items()})
        # wherever dS did not cancel by more than 4x, the gate holds on this denominator too; an element above it
        # sits in a row whose dS cancelled by at least three orders of magnitude (there |dS8| is zero or a few
        # subnormal codes, and the difference is FP32 rounding of dP - D, which mag measures and mag8 does not)
        assert st["max_uncancelled"] <= TOL_BWD, (n_, st)
        assert st["share_over"] == 0.0 or st["min_cancel_of_over"] >= 1e3, (n_, st)
        if d == 128:            # the large configurations have no such rows at these sizes: plain maximum
            assert st["max"] <= TOL_BWD, (n_, st)
    for n_, g_ in (("dQ", gq), ("dK", gk), ("dV", gv)):
        fro, inf = norm_ratios(g_, ref[n_])
        assert fro <= FRO_BWD, (n_, fro)
        m[n_ + "_max_rel"], m[n_ + "_fro"], m[n_ + "_inf"] = errs[n_], fro, inf
    report("bwd %s B%d N%d causal=%d" % (name, B, N, causal), **m)


@pytest.mark.parametrize("name,B,N,causal", [("c1", 1, 400, True), ("c4", 1, 272, True), ("c1", 2, 128, False)])
def test_forward_fp8_output_equals_unfused_chain(name, B, N, causal):
    """Producer form: O and LSE unchanged, O8 and amax bit-identical to fp8_cast of the BF16 output."""
    cfg = synth.CONFIGS[name]
    Hq, Hkv, d = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    if name != "c1":
        Hq, Hkv = Hq // 4, Hkv // 4
        cfg = synth.BlockConfig(**{**cfg.__dict__, "n_q_heads": Hq, "n_kv_heads": Hkv})
    qd = quantized_qkv(cfg, N, B)
    s = d ** -0.5
    O, LSE = run_fwd(qd, B, N, Hq, Hkv, d, causal, s)
    a_now = scalar()
    fp8.fp8_amax(O, a_now)
    o_scale, o_inv = scalar(), scalar()
    fp8.fp8_scale(scalar(float(a_now.item()) * 1.5), o.E4M3, 0, o_scale, o_inv)      # a "history" scale
    ref8 = torch.empty((B, N, Hq, d), dtype=torch.uint8, device="cuda")
    fp8.fp8_cast(O.view(B * N, Hq * d), o_scale, o.E4M3, ref8.view(B * N, Hq * d))
    q8, k8, v8 = dev(qd["q"][0]), dev(qd["k"][0]), dev(qd["v"][0])
    O2 = torch.empty_like(O)
    LSE2 = torch.empty_like(LSE)
    O8 = torch.full((B, N, Hq, d), 0x55, dtype=torch.uint8, device="cuda")
    a = scalar(-2.0)
    fp8.fp8_attention_fwd_q(q8, k8, v8, scalar(qd["q"][1]), scalar(qd["k"][1]), scalar(qd["v"][1]), s, causal,
                            O2, LSE2, o_scale, O8, a)
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    assert torch.equal(O2.view(torch.int16), O.view(torch.int16)) and torch.equal(LSE2, LSE)
    assert torch.equal(O8, ref8)
    assert float(a.item()) == float(a_now.item())
