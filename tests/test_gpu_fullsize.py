"""GPU parity at the full workload sizes, in the launch configuration bench.py times (BlockHotPath.step).

The oracle cannot redo these sizes whole, so it computes sampled outputs one by one: output rows/columns of
each GEMM (each a complete reduction), and for attention the query rows / key rows whose results depend only
on data the oracle can afford (causality makes the first rows an N = rows problem, and the last key rows
depend only on the last query rows)."""
import numpy as np
import pytest
import torch

import oracle as o
import paper_2505_20524_b200 as fp8
from paper_2505_20524_b200 import synth
from paper_2505_20524_b200.hotpath import BlockHotPath
from gpu_util import (dev, host, scalar, rel_err, quantile_err, norm_ratios, report, BWD_FLOOR, FLIP_EPS, FRO_FWD,
                      FRO_BWD)

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("log2n,fmts", [(27, (o.E4M3, o.E5M2)), (29, (o.E4M3, o.E5M2))])
def test_quantize_sweep_sizes_bit_exact(log2n, fmts):
    n = 1 << log2n
    x = synth.flat_tensor(n)
    xd = dev(x)
    a, s, si = scalar(), scalar(), scalar()
    ea = o.amax(x)
    assert float(ea) == 200.0
    for fmt in fmts:
        q = torch.empty(n, dtype=torch.uint8, device="cuda")
        fp8.fp8_quantize(xd, fmt, q, None, a, s, si)
        es, esi = o.scale(ea, fmt)
        assert float(a.item()) == float(ea) and float(s.item()) == float(es) and float(si.item()) == float(esi)
        exp = o.cast(x.reshape(-1, 4096), es, fmt).reshape(-1)
        assert np.array_equal(host(q), exp)
        del q


def _sample(n, k, seed):
    """k indices of [0, n): tile edges, the ragged end and seeded picks."""
    fixed = [0, 1, 127, 128, 255, 256, n // 2 - 1, n // 2, n - 129, n - 128, n - 2, n - 1]
    rng = np.random.default_rng(seed)
    idx = sorted(set([i for i in fixed if 0 <= i < n] + rng.integers(0, n, size=k).tolist()))
    return np.array(idx[:max(k, len(fixed))], dtype=np.int64)


@pytest.mark.parametrize("name", ["c3", "c4"])
def test_block_gemms_sampled(name):
    cfg = synth.CONFIGS[name]
    hp = BlockHotPath(cfg, "cuda", with_attention=False)
    h = hp.generate_host_inputs()
    hp.allocate()
    hp.step()
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    for lin in hp.linears:
        x8, _, _, sx = o.quantize(h["x_" + lin.name], o.E4M3)
        w8, _, _, sw = o.quantize(h["w_" + lin.name], o.E4M3)
        dy8, _, _, sdy = o.quantize(h["dy_" + lin.name], o.E5M2)
        assert np.array_equal(host(lin.x.q), x8) and np.array_equal(host(lin.w.q), w8)
        assert np.array_equal(host(lin.dy.q), dy8)
        T, N, K = lin.T, lin.N, lin.K
        for out, fn, a8, b8, sa, sb, nr, nc in ((lin.y, o.linear_fwd, x8, w8, sx, sw, T, N),
                                                (lin.dx, o.linear_dgrad, dy8, w8, sdy, sw, T, K),
                                                (lin.dw, o.linear_wgrad, dy8, x8, sdy, sx, N, K)):
            rows, cols = _sample(nr, 16, 1), _sample(nc, 48, 2)
            ref, mag = fn(a8, b8, sa, sb, rows=rows, cols=cols)
            got = out[torch.from_numpy(rows).cuda()][:, torch.from_numpy(cols).cuda()].float().cpu().numpy()
            err = rel_err(got.astype(np.float64), ref, mag)
            assert err <= 2.0 ** -8, (lin.name, fn.__name__, err)


def _attention_case(name, kv_heads, head_rows):
    cfg = synth.CONFIGS[name]
    hp = BlockHotPath(cfg, "cuda", with_linears=False)
    h = hp.generate_host_inputs()
    hp.allocate()
    a = hp.attn
    B, N, Hq, Hkv, d = hp.B, hp.N, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    G = Hq // Hkv
    q8, _, _, qi = o.quantize(h["q"], o.E4M3)
    k8, _, _, ki = o.quantize(h["k"], o.E4M3)
    v8, _, _, vi = o.quantize(h["v"], o.E4M3)
    do8, _, _, doi = o.quantize(h["do"], o.E5M2)
    lo, hi = (0, head_rows), (N - head_rows, N)
    kw = dict(causal=True, quant=True, kv_block=128, max_mode=0, q_inv=qi, k_inv=ki, v_inv=vi, do_inv=doi,
              flip_eps=FLIP_EPS)
    p = o.attn_params(B, N, Hq, Hkv, d, ds_scale=1.0, **kw)
    heads = [(b, g * G + j) for (b, g) in kv_heads for j in range(G)]
    fwd = {}
    for rng in (lo, hi):
        fwd[rng] = o.attention_fwd(q8, k8, v8, p, heads=heads, rows=rng, with_slack=True)
    # a dS scale from the oracle alone: power of two, 4x headroom over the amax seen on the sampled pairs
    O_or = np.zeros((B, N, Hq, d))
    L_or = np.zeros((B, Hq, N))
    for rng in (lo, hi):
        O_, lse_, _, _ = fwd[rng]
        for n_, (b, hh) in enumerate(heads):
            O_or[b, rng[0]:rng[1], hh] = synth.bf16_to_f32(synth.f32_to_bf16(O_[n_].astype(np.float32)))
            L_or[b, hh, rng[0]:rng[1]] = lse_[n_].astype(np.float32)
    cal = o.attention_bwd(q8, k8, v8, do8, O_or, L_or, p, kv_heads=kv_heads, q_rows=hi, k_rows=hi)
    ds_scale = 2.0 ** np.floor(np.log2(57344.0 / (4.0 * cal["amax_dS"])))
    a["ds_scale"].fill_(float(ds_scale))

    hp.step()                                                 # the timed configuration: quantize + fwd + bwd
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    assert np.array_equal(host(a["q"].q), q8) and np.array_equal(host(a["do"].q), do8)
    gO = a["o"].float().cpu().numpy().astype(np.float64)
    gL = a["lse"].cpu().numpy().astype(np.float64)
    for rng in (lo, hi):
        O_, lse_, mag_, slack_ = fwd[rng]
        for n_, (b, hh) in enumerate(heads):
            e = rel_err(gO[b, rng[0]:rng[1], hh], O_[n_], mag_[n_], slack_[n_])
            assert e <= 2e-2, ("O", rng, b, hh, e)
            fro = norm_ratios(gO[b, rng[0]:rng[1], hh], O_[n_])[0]
            assert fro <= FRO_FWD, ("O", rng, b, hh, fro)
            report("fwd %s full size rows %d:%d b%d h%d" % (name, rng[0], rng[1], b, hh), max_rel=e, fro=fro)
            assert np.max(np.abs(gL[b, hh, rng[0]:rng[1]] - lse_[n_])) <= 1e-3 * max(1.0, np.abs(lse_[n_]).max())

    # backward again on the oracle's O / LSE for the sampled (head, row) ranges, so both sides see equal inputs
    Ot = a["o"].clone()
    Lt = a["lse"].clone()
    for rng in (lo, hi):
        for (b, hh) in heads:
            bits = synth.f32_to_bf16(O_or[b, rng[0]:rng[1], hh].astype(np.float32))
            Ot[b, rng[0]:rng[1], hh] = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()
            Lt[b, hh, rng[0]:rng[1]] = torch.from_numpy(L_or[b, hh, rng[0]:rng[1]].astype(np.float32)).cuda()
    fp8.fp8_attention_bwd(a["q"].q, a["k"].q, a["v"].q, a["do"].q, Ot, Lt, a["q"].scale_inv, a["k"].scale_inv,
                          a["v"].scale_inv, a["do"].scale_inv, a["softmax_scale"], a["ds_scale"], True, a["dq"],
                          a["dk"], a["dv"], a["ws"], ds_amax=a["ds_amax"])
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    p = o.attn_params(B, N, Hq, Hkv, d, ds_scale=float(ds_scale), **kw)
    first = o.attention_bwd(q8, k8, v8, do8, O_or, L_or, p, kv_heads=kv_heads, q_rows=lo, k_rows=lo)
    last = o.attention_bwd(q8, k8, v8, do8, O_or, L_or, p, kv_heads=kv_heads, q_rows=hi, k_rows=hi)
    assert float(a["ds_amax"].item()) >= 0.999 * max(first["amax_dS"], last["amax_dS"])
    gq = a["dq"].float().cpu().numpy().astype(np.float64)
    gk = a["dk"].float().cpu().numpy().astype(np.float64)
    gv = a["dv"].float().cpu().numpy().astype(np.float64)
    for n_, (b, g) in enumerate(kv_heads):
        for j in range(G):
            got = gq[b, lo[0]:lo[1], g * G + j]
            e = rel_err(got, first["dQ"][n_, j], first["mag_dQ"][n_, j], first["slack_dQ"][n_, j], BWD_FLOOR)
            assert e <= 3e-2, ("dQ", b, g, j, e)
            q999, mx = quantile_err(got, first["dQ"][n_, j], first["mag8_dQ"][n_, j], first["slack_dQ"][n_, j],
                                    0.999, BWD_FLOOR)
            fro = norm_ratios(got, first["dQ"][n_, j])[0]
            assert fro <= FRO_BWD and mx <= 3e-2, ("dQ", b, g, j, fro, mx)
            report("bwd %s full size dQ b%d h%d" % (name, b, g * G + j), max_rel=e, mag8_q999=q999, mag8_max=mx,
                   fro=fro)
        for nm, got in (("dK", gk), ("dV", gv)):
            gt = got[b, hi[0]:hi[1], g]
            e = rel_err(gt, last[nm][n_], last["mag_" + nm][n_], last["slack_" + nm][n_], BWD_FLOOR)
            assert e <= 3e-2, (nm, b, g, e)
            fro = norm_ratios(gt, last[nm][n_])[0]
            assert fro <= FRO_BWD, (nm, b, g, fro)
            m = dict(max_rel=e, fro=fro)
            if nm == "dK":
                q999, mx = quantile_err(gt, last[nm][n_], last["mag8_dK"][n_], last["slack_dK"][n_], 0.999, BWD_FLOOR)
                assert mx <= 3e-2, (nm, b, g, mx)
                m.update(mag8_q999=q999, mag8_max=mx)
            report("bwd %s full size %s b%d g%d" % (name, nm, b, g), **m)


def test_attention_1p5b_block_sampled():
    _attention_case("c3", kv_heads=[(0, 0), (3, 15)], head_rows=256)


def test_attention_8b_block_sampled():
    _attention_case("c4", kv_heads=[(0, 0), (1, 7)], head_rows=256)


def test_attention_long_context_sampled():
    _attention_case("c5", kv_heads=[(0, 13)], head_rows=1024)


def test_host_to_host_step_equals_device_step():
    """The pipelined host-to-host step (uploads / kernels / downloads on three streams) returns the bits of step()."""
    cfg = synth.CONFIGS["c1"]
    hp = BlockHotPath(cfg, "cuda")
    h = hp.generate_host_inputs()
    hp.allocate()
    hp.calibrate_ds_scale()
    hp.step()
    torch.cuda.synchronize()
    ref = {n: t.clone() for n, t in hp.output_tensors()}
    hin = {n: torch.from_numpy(h[n].view("int16")).view(torch.bfloat16).reshape(t.shape).pin_memory()
           for n, t in hp.input_tensors()}
    hout = {n: torch.empty(t.shape, dtype=t.dtype).pin_memory() for n, t in hp.output_tensors()}
    for n, t in hp.input_tensors():
        t.zero_()                                   # the device copies must come from the host buffers
    for _ in range(3):                              # back-to-back steps reuse the device buffers
        hp.step_host(hin, hout)
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    for n, t in ref.items():
        a, b = hout[n], t.cpu()
        assert torch.equal(a.view(torch.uint8), b.view(torch.uint8)), n
    # overlapped form: consecutive steps in flight, one wait at the end
    for n in hout:
        hout[n].zero_()
    for _ in range(4):
        hp.step_host(hin, hout, wait=False)
    hp.finish_host()
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    for n, t in ref.items():
        assert torch.equal(hout[n].view(torch.uint8), t.cpu().view(torch.uint8)), n


@pytest.mark.parametrize("name", ["c1", "c4"])
def test_host_buffer_entry_points_equal_device_step(name):
    """The step through fp8_linear_step_host / fp8_attention_step_host (the form bench.py times end to end), three
    steps in flight on the same workspaces, returns the bits of step(); dQ at head_dim 128 within its summation-order
    noise."""
    cfg = synth.CONFIGS[name]
    hp = BlockHotPath(cfg, "cuda")
    h = hp.generate_host_inputs()
    hp.allocate()
    hp.calibrate_ds_scale()
    hp.step()
    torch.cuda.synchronize()
    ref = {n: t.cpu() for n, t in hp.output_tensors()}
    hin = {n: torch.from_numpy(h[n].view("int16")).view(torch.bfloat16).reshape(t.shape).pin_memory()
           for n, t in hp.input_tensors()}
    hout = {n: torch.zeros(t.shape, dtype=t.dtype).pin_memory() for n, t in hp.output_tensors()}
    for _ in range(3):
        hp.step_host_abi(hin, hout)
    fp8.fp8_host_sync()
    assert fp8.fp8_device_status() == 0
    for n, t in ref.items():
        if n == "dq" and cfg.head_dim == 128:
            a, b = hout[n].float(), t.float()
            assert (a - b).abs().max() <= 2.0 ** -7 * b.abs().max()
        else:
            assert torch.equal(hout[n].view(torch.uint8), t.view(torch.uint8)), n


@pytest.mark.parametrize("multi", [True, False], ids=["one_launch_per_group", "two_launches_per_tensor"])
def test_delayed_scaling_step_equals_the_just_in_time_step_on_repeated_inputs(multi):
    """With the same inputs every step, the abs-max history holds one value: the delayed-scaling step (one cast pass per
    tensor under the history's scale, Appendix E) must return the bits of the just-in-time step; and when an input grows,
    the step that sees it still casts (saturating) under the old scale and the next one under the new."""
    cfg = synth.CONFIGS["c1"]
    jit = BlockHotPath(cfg, "cuda")
    h = jit.generate_host_inputs()
    jit.allocate()
    jit.calibrate_ds_scale()
    jit.step()
    torch.cuda.synchronize()
    ref = {n: t.clone() for n, t in jit.output_tensors()}
    dl = BlockHotPath(cfg, "cuda", scaling="delayed", multi_quantize=multi)
    dl.allocate(h)
    dl.attn["ds_scale"].copy_(jit.attn["ds_scale"])
    for _ in range(3):
        dl.step()
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    for n, t in dl.output_tensors():
        assert torch.equal(t.view(torch.uint8), ref[n].view(torch.uint8)), n
    assert dl.quantize_bytes() * 5 == jit.quantize_bytes() * 3            # 3 instead of 5 bytes per element
    # an input doubles: this step's codes are those of the old scale, the next step's those of the new one
    x = dl.linears[0].x
    old_scale = float(x.scale.item())
    x.x.copy_((x.x.float() * 2).to(torch.bfloat16))
    dl.step()
    torch.cuda.synchronize()
    assert float(x.scale.item()) == old_scale
    want = torch.empty_like(x.q)
    fp8.fp8_cast(x.x, x.scale, x.fmt, want)
    assert torch.equal(x.q, want)
    dl.step()
    torch.cuda.synchronize()
    assert float(x.scale.item()) == old_scale / 2
    assert fp8.fp8_device_status() == 0


def test_overlapped_step_equals_the_step():
    """Quantize calls on a side stream, products on the current one, ordered by events: the bits of step()."""
    for name in ("c1", "c3"):
        cfg = synth.CONFIGS[name]
        hp = BlockHotPath(cfg, "cuda")
        hp.generate_host_inputs()
        hp.allocate()
        hp.calibrate_ds_scale()
        hp.step()
        torch.cuda.synchronize()
        ref = {n: t.clone() for n, t in hp.output_tensors()}
        for _, t in hp.output_tensors():
            t.zero_()
        for _ in range(3):
            hp.step_overlapped()
        torch.cuda.synchronize()
        assert fp8.fp8_device_status() == 0
        for n, t in hp.output_tensors():
            if n == "dq" and cfg.head_dim == 128:
                # dQ is summed over key tiles by FP32 adds in L2 whose order follows the CTA schedule: equal up to that
                # rounding from run to run, whichever streams the step uses
                a, b = t.float(), ref[n].float()
                assert float((a - b).abs().max()) <= 2.0 ** -7 * float(b.abs().max()), (name, n)
            else:
                assert torch.equal(t.view(torch.uint8), ref[n].view(torch.uint8)), (name, n)
        del hp, ref
        torch.cuda.empty_cache()


def test_graph_replay_of_the_step_equals_the_step():
    """The step makes no host synchronisation: captured into a CUDA graph and replayed it returns the same bits."""
    cfg = synth.CONFIGS["c1"]
    hp = BlockHotPath(cfg, "cuda")
    hp.generate_host_inputs()
    hp.allocate()
    hp.calibrate_ds_scale()
    hp.step()
    torch.cuda.synchronize()
    ref = {n: t.clone() for n, t in hp.output_tensors()}
    g = hp.capture_graph()
    for _, t in hp.output_tensors():
        t.zero_()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    for n, t in hp.output_tensors():
        assert torch.equal(t.view(torch.uint8), ref[n].view(torch.uint8)), n
    # delayed scaling: the one-launch group quantize keeps its pointers from step to step, so three replays of one
    # captured step equal three eager steps (the history advances on the device); the per-tensor form swaps its scale
    # buffers on the host between steps and refuses capture
    eager = BlockHotPath(cfg, "cuda", scaling="delayed")
    eager.allocate(hp.host_inputs)
    eager.attn["ds_scale"].copy_(hp.attn["ds_scale"])
    for _ in range(4):
        eager.step()
    torch.cuda.synchronize()
    want = {n: t.clone() for n, t in eager.output_tensors()}
    dl = BlockHotPath(cfg, "cuda", scaling="delayed")
    dl.allocate(hp.host_inputs)
    dl.attn["ds_scale"].copy_(hp.attn["ds_scale"])
    g = dl.capture_graph()                       # runs one eager step itself
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    for n, t in dl.output_tensors():
        assert torch.equal(t.view(torch.uint8), want[n].view(torch.uint8)), n
    assert torch.equal(dl.linears[0].x.history, eager.linears[0].x.history)
    assert int(dl.linears[0].x.head.item()) == int(eager.linears[0].x.head.item())
    with pytest.raises(ValueError):
        BlockHotPath(cfg, "cuda", scaling="delayed", multi_quantize=False).capture_graph()


def test_glue_and_producer_forms_at_c4_sizes():
    """The (f)-row entry points at the 8B-class block's sizes, in the launch configurations bench.py --report times."""
    from gpu_util import dev, scalar
    cfg = synth.CONFIGS["c4"]
    T, H, F = cfg.tokens, cfg.hidden, cfg.ffn
    # gated activation + cast on the [T, 2F] output of the up projection: sampled rows against the oracle
    cols = synth.choose_columns(2 * F, cfg.n_outlier_cols(2 * F), 4, 77)
    gu = synth.normal_bf16((T, 2 * F), 4, 77, 1.0, cols, 8.0)
    a, s, si = scalar(), scalar(), scalar()
    x = dev(gu)
    fp8.fp8_swiglu_cast(x, None, o.E4M3, None, None, a)
    fp8.fp8_scale(a, o.E4M3, 0, s, si)
    out = torch.empty((T, F), dtype=torch.uint8, device="cuda")
    out_t = torch.empty((F, T), dtype=torch.uint8, device="cuda")
    fp8.fp8_swiglu_cast(x, s, o.E4M3, out, out_t, None)
    rows = _sample(T, 64, 5)
    h = o.swiglu(np.ascontiguousarray(gu[rows]))
    exp = o.cast(h, float(s.item()), o.E4M3)
    got = host(out)[rows]
    assert (got != exp).mean() <= 2e-3
    assert np.array_equal(host(out_t)[:, rows], got.T)
    assert abs(float(a.item()) - float(o.amax(o.swiglu(gu)))) <= 2.0 ** -7 * float(a.item())
    del x, out, out_t
    # post-norm + residual on the residual stream [T, H]
    xb, yb = synth.normal_bf16((T, H), 4, 78, 1.0), synth.normal_bf16((T, H), 4, 79, 0.05)
    g = np.full(H, 1.0 / np.sqrt(32.0), dtype=np.float32)
    res = torch.empty((T, H), dtype=torch.bfloat16, device="cuda")
    fp8.fp8_postnorm_residual(dev(xb), dev(yb), torch.from_numpy(g).cuda(), o.NORM_RMS, 1e-5, res, a)
    exp = o.postnorm_residual(xb[rows], yb[rows], g, o.NORM_RMS, 1e-5)
    got = host(res)[rows]
    d = got.astype(np.int32) != exp.astype(np.int32)
    assert d.mean() <= 2e-3
    assert float(a.item()) == float(o.amax(host(res)))
    # producer form of the largest GEMM (up projection): bit-identical to the unfused chain
    Tt, N, K = cfg.linear_shapes()["up"]
    x8 = torch.randint(0x20, 0x48, (Tt, K), dtype=torch.uint8, device="cuda")
    w8 = torch.randint(0x20, 0x48, (N, K), dtype=torch.uint8, device="cuda") | 0x80
    s1 = scalar(2.0 ** -7)
    ybf = torch.empty((Tt, N), dtype=torch.bfloat16, device="cuda")
    fp8.fp8_linear_fwd(x8, w8, s1, s1, ybf)
    fp8.fp8_amax(ybf, a)
    fp8.fp8_scale(scalar(float(a.item()) * 1.3), o.E4M3, 0, s, si)
    ref8 = torch.empty((Tt, N), dtype=torch.uint8, device="cuda")
    fp8.fp8_cast(ybf, s, o.E4M3, ref8)
    got8 = torch.empty_like(ref8)
    a2 = scalar()
    fp8.fp8_linear_fwd_q(x8, w8, s1, s1, s, o.E4M3, got8, a2)
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    assert torch.equal(got8, ref8) and float(a2.item()) == float(a.item())
    del ybf, ref8, got8
    # blockwise recipe at the QKV projection's size: sampled rows against the oracle
    Tt, N, K = cfg.linear_shapes()["qkv"]
    xq = synth.normal_bf16((Tt, K), 4, 80, 1.0, synth.choose_columns(K, 21, 4, 80), 30.0)
    wq = synth.normal_bf16((N, K), 4, 81, synth.W_STD)
    x8 = torch.empty((Tt, K), dtype=torch.uint8, device="cuda")
    w8 = torch.empty((N, K), dtype=torch.uint8, device="cuda")
    sx = torch.empty((K // 128, Tt), device="cuda")
    sw = torch.empty((N // 128, K // 128), device="cuda")
    fp8.fp8_quantize_blockwise(dev(xq), 1, o.E4M3, x8, sx)
    fp8.fp8_quantize_blockwise(dev(wq), 128, o.E4M3, w8, sw)
    y = torch.empty((Tt, N), dtype=torch.bfloat16, device="cuda")
    fp8.fp8_linear_fwd_blockwise(x8, w8, sx, sw, y)
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    rows = _sample(Tt, 16, 6)
    ox8, osx = o.quantize_blockwise(np.ascontiguousarray(xq[rows]), 1, 128, o.E4M3)
    ow8, osw = o.quantize_blockwise(wq, 128, 128, o.E4M3)
    assert np.array_equal(host(x8)[rows], ox8) and np.array_equal(host(w8), ow8)
    ref, mag = o.linear_fwd_blockwise(ox8, ow8, osx, osw)
    got = y.float().cpu().numpy().astype(np.float64)[rows]
    assert rel_err(got, ref, mag) <= 2.0 ** -8
    # its data gradient on sampled token rows, and its weight gradient on sampled entries
    dyq = synth.normal_bf16((Tt, N), 4, 82, 1e-3, synth.choose_columns(N, 8, 4, 82), 20.0)
    dy8 = torch.empty((Tt, N), dtype=torch.uint8, device="cuda")
    sdy = torch.empty((N // 128, Tt), device="cuda")
    fp8.fp8_quantize_blockwise(dev(dyq), 1, o.E5M2, dy8, sdy)
    dx = torch.empty((Tt, K), dtype=torch.bfloat16, device="cuda")
    fp8.fp8_linear_dgrad_blockwise(dy8, w8, sdy, sw, dx)
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    ody8, osdy = o.quantize_blockwise(np.ascontiguousarray(dyq[rows]), 1, 128, o.E5M2)
    assert np.array_equal(host(dy8)[rows], ody8)
    ref, mag = o.linear_dgrad_blockwise(ody8, ow8, osdy, osw)
    assert rel_err(dx.float().cpu().numpy().astype(np.float64)[rows], ref, mag) <= 2.0 ** -8
    del dx, y
    nb = (Tt + 127) // 128
    sdt, sxt = torch.empty((nb, N), device="cuda"), torch.empty((nb, K), device="cuda")
    fp8.fp8_quantize_blockwise(dev(dyq), fp8.FP8_BLOCK_128x1, o.E5M2, dy8, sdt)
    fp8.fp8_quantize_blockwise(dev(xq), fp8.FP8_BLOCK_128x1, o.E4M3, x8, sxt)
    dw = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
    fp8.fp8_linear_wgrad_blockwise(dy8, x8, sdt, sxt, dw)
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    ns, ks = _sample(N, 12, 7), _sample(K, 12, 8)
    ody8, osdt = o.quantize_blockwise(np.ascontiguousarray(dyq[:, ns]), 128, 1, o.E5M2)
    ox8, osxt = o.quantize_blockwise(np.ascontiguousarray(xq[:, ks]), 128, 1, o.E4M3)
    assert np.array_equal(host(dy8)[:, ns], ody8) and np.array_equal(host(x8)[:, ks], ox8)
    ref, mag = o.linear_wgrad_blockwise(ody8, ox8, osdt, osxt)
    assert rel_err(dw.float().cpu().numpy().astype(np.float64)[np.ix_(ns, ks)], ref, mag) <= 2.0 ** -8


def test_bench_line_carries_the_contract_keys():
    """`bench.py` on the small configuration: one JSON line with every key the measurement contract names."""
    import json
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--config", "c1", "--steps", "3", "--warmup", "3",
                          "--graph"], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
              "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline", "graph"):
        assert k in line, k
    assert line["n_gpus"] == 1 and line["steps"] == 3 and line["value"] > 0 and line["gpu_launches"] > 0
    assert "workload" in line["config"] and "model" not in line["config"]
    for k in ("value", "unit", "h2d_bytes_per_step", "d2h_bytes_per_step"):
        assert k in line["e2e"], k
    assert line["e2e"]["h2d_bytes_per_step"] > 0 and line["e2e"]["d2h_bytes_per_step"] > 0
    for k in ("bound", "achieved", "peak", "unit", "frac", "traffic"):
        assert k in line["roofline"], k
    for k in ("value", "unit", "cores", "kind", "sample"):
        assert k in line["cpu_baseline"], k
    assert line["cpu_baseline"]["kind"] == "oracle"
    for k in ("sm_mhz", "sm_max_mhz", "reasons"):
        assert k in line["clocks"], k
