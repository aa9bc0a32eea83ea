"""The scratch-free attention backward (fp8_attention_bwd_static) against fp8_attention_bwd.

Some callers cannot allocate device memory or hand a workspace to the library (a plugin that only gets its
inputs and outputs, code inside a fully committed memory pool), so this entry point keeps its scratch in a
fixed array inside the library.  The array is shared by all calls and keeps the last call's contents, hence
the check runs twice in a row on different inputs.  This file sorts last on purpose: a run that stops at the
first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle as o
import paper_2505_20524_b200 as fp8
from paper_2505_20524_b200 import synth
from gpu_util import dev, scalar, rel_err, BWD_FLOOR, FLIP_EPS

pytestmark = pytest.mark.gpu
TOL = 3e-2   # the attention-gradient tolerance of the other tests; the two paths should in fact agree far better


def _inputs(name, B, N, heads_div):
    cfg = synth.CONFIGS[name]
    Hq, Hkv, d = cfg.n_q_heads // heads_div, cfg.n_kv_heads // heads_div, cfg.head_dim
    cfg = synth.BlockConfig(**{**cfg.__dict__, "n_q_heads": Hq, "n_kv_heads": Hkv})
    q, k, v, do = synth.attention_inputs(cfg, seq=N, batch=B)
    t = {}
    for n_, x, fmt in (("q", q, o.E4M3), ("k", k, o.E4M3), ("v", v, o.E4M3), ("do", do, o.E5M2)):
        c, _, _, si = o.quantize(x, fmt)
        t[n_] = (dev(c), scalar(float(si)))
        t[n_ + "_host"] = (c, float(si))
    return t, B, N, Hq, Hkv, d


DS_SCALE = 4096.0


def _both(t, B, N, Hq, Hkv, d):
    s = d ** -0.5
    O = torch.empty((B, N, Hq, d), dtype=torch.bfloat16, device="cuda")
    LSE = torch.empty((B, Hq, N), dtype=torch.float32, device="cuda")
    fp8.fp8_attention_fwd(t["q"][0], t["k"][0], t["v"][0], t["q"][1], t["k"][1], t["v"][1], s, True, O, LSE, None)
    t["O"], t["LSE"] = O, LSE
    outs = []
    for static in (False, True):
        dq = torch.zeros((B, N, Hq, d), dtype=torch.bfloat16, device="cuda")
        dk = torch.zeros((B, N, Hkv, d), dtype=torch.bfloat16, device="cuda")
        dv = torch.zeros((B, N, Hkv, d), dtype=torch.bfloat16, device="cuda")
        args = (t["q"][0], t["k"][0], t["v"][0], t["do"][0], O, LSE, t["q"][1], t["k"][1], t["v"][1], t["do"][1], s,
                scalar(DS_SCALE), True, dq, dk, dv)
        if static:
            fp8.fp8_attention_bwd_static(*args)
        else:
            ws = torch.empty(fp8.fp8_attention_workspace_bytes(1, B, N, Hq, Hkv, d), dtype=torch.uint8, device="cuda")
            fp8.fp8_attention_bwd(*args, ws)
        torch.cuda.synchronize()
        outs.append([x.float().cpu().numpy().astype(np.float64) for x in (dq, dk, dv)])
    assert fp8.fp8_device_status() == 0
    return outs


def test_static_scratch_matches_workspace_version_twice_in_a_row():
    # second problem is smaller, so stale contents of the first call lie beyond what it clears
    for name, B, N, div in (("c3", 1, 384, 4), ("c1", 2, 144, 1)):
        t, B, N, Hq, Hkv, d = _inputs(name, B, N, div)
        (dq0, dk0, dv0), (dq1, dk1, dv1) = _both(t, B, N, Hq, Hkv, d)
        for a, b in ((dq0, dq1), (dk0, dk1), (dv0, dv1)):
            assert np.abs(a).max() > 0
            assert np.max(np.abs(a - b)) <= TOL * np.abs(a).max()
        # dK and dV do not go through atomics: identical bits
        assert np.array_equal(dk0, dk1) and np.array_equal(dv0, dv1)
        # and against the oracle, on the O and LSE the backward was given, with the gate of the other gradient tests
        G = Hq // Hkv
        p = o.attn_params(B, N, Hq, Hkv, d, causal=True, quant=True, s=d ** -0.5, q_inv=t["q_host"][1],
                          k_inv=t["k_host"][1], v_inv=t["v_host"][1], do_inv=t["do_host"][1], ds_scale=DS_SCALE,
                          flip_eps=FLIP_EPS)
        ref = o.attention_bwd(t["q_host"][0], t["k_host"][0], t["v_host"][0], t["do_host"][0],
                              t["O"].float().cpu().numpy().astype(np.float64),
                              t["LSE"].cpu().numpy().astype(np.float64), p)
        gq = dq1.reshape(B, N, Hkv, G, d).transpose(0, 2, 3, 1, 4).reshape(B * Hkv, G, N, d)
        gk = dk1.transpose(0, 2, 1, 3).reshape(B * Hkv, N, d)
        gv = dv1.transpose(0, 2, 1, 3).reshape(B * Hkv, N, d)
        for n_, g_ in (("dQ", gq), ("dK", gk), ("dV", gv)):
            e = rel_err(g_, ref[n_], ref["mag_" + n_], ref["slack_" + n_], BWD_FLOOR)
            assert e <= TOL, (name, n_, e)


def test_static_scratch_call_leaves_free_device_memory_unchanged():
    """The entry point promises to allocate nothing: after a first call (which looks up the array's address and sets
    kernel attributes) a further call must not change the amount of free device memory."""
    t, B, N, Hq, Hkv, d = _inputs("c1", 1, 256, 1)
    s = d ** -0.5
    O = torch.empty((B, N, Hq, d), dtype=torch.bfloat16, device="cuda")
    LSE = torch.empty((B, Hq, N), dtype=torch.float32, device="cuda")
    fp8.fp8_attention_fwd(t["q"][0], t["k"][0], t["v"][0], t["q"][1], t["k"][1], t["v"][1], s, True, O, LSE, None)
    dq = torch.zeros((B, N, Hq, d), dtype=torch.bfloat16, device="cuda")
    dk = torch.zeros((B, N, Hkv, d), dtype=torch.bfloat16, device="cuda")
    dv = torch.zeros((B, N, Hkv, d), dtype=torch.bfloat16, device="cuda")
    ds = scalar(DS_SCALE)
    args = (t["q"][0], t["k"][0], t["v"][0], t["do"][0], O, LSE, t["q"][1], t["k"][1], t["v"][1], t["do"][1], s,
            ds, True, dq, dk, dv)
    fp8.fp8_attention_bwd_static(*args)
    torch.cuda.synchronize()
    unchanged = False
    for _ in range(3):          # free memory is a device-wide figure: allow for another process moving it once
        free0 = torch.cuda.mem_get_info()[0]
        for _ in range(3):
            fp8.fp8_attention_bwd_static(*args)
        torch.cuda.synchronize()
        unchanged = unchanged or torch.cuda.mem_get_info()[0] == free0
    assert unchanged
    assert fp8.fp8_device_status() == 0


def test_static_scratch_rejects_problems_beyond_its_size():
    B, N, Hq, Hkv, d = 4, 4096, 32, 8, 128
    assert fp8.fp8_attention_workspace_bytes(1, B, N, Hq, Hkv, d) > fp8.binding.STATIC_SCRATCH_BYTES
    # operands of the real size, so that a regression of the size check gives wrong numbers, not an out-of-bounds launch
    z8 = torch.zeros(B * N * Hq * d, dtype=torch.uint8, device="cuda")
    zb = torch.zeros(B * N * Hq * d, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(B * Hq * N, dtype=torch.float32, device="cuda")
    sc = fp8.binding._scales(scalar(1), scalar(1), scalar(1), scalar(1), 0.1, 448.0, scalar(1), None)
    import ctypes as C
    rc = fp8.binding.load().fp8_attention_bwd_static(
        C.c_void_p(z8.data_ptr()), C.c_void_p(z8.data_ptr()), C.c_void_p(z8.data_ptr()), C.c_void_p(z8.data_ptr()),
        C.c_void_p(zb.data_ptr()), C.c_void_p(lse.data_ptr()), C.byref(sc), 1, B, N, Hq, Hkv, d,
        C.c_void_p(zb.data_ptr()), C.c_void_p(zb.data_ptr()), C.c_void_p(zb.data_ptr()), None)
    assert rc == -5 and "scratch" in fp8.fp8_last_error()
