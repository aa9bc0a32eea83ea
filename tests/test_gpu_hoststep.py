"""The host-buffer entry points (fp8_linear_step_host, fp8_attention_step_host) against the oracle and against the
same chain of device-pointer calls.

The host forms only move bytes and chain the device entry points, so their results must carry the oracle's
tolerances and be bit-identical to the device chain (dQ at head_dim 128 is summed by atomics in an order that
follows the block schedule, so there only the tolerance applies).  Two workspaces are used in rotation and one
of them is reused without a sync in between, to exercise the ordering the library promises.
"""
import numpy as np
import pytest
import torch

import oracle as o
import paper_2505_20524_b200 as fp8
from paper_2505_20524_b200 import synth
from gpu_util import dev, scalar, rel_err, FLIP_EPS

pytestmark = pytest.mark.gpu
DS_SCALE = 4096.0
KV_BLOCK = 128      # the forward takes keys in blocks of 128
TOL_FWD = 2e-2      # the forward tolerance of the attention tests


def pinned(bits: np.ndarray) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.pin_memory()


def pinned_out(shape, dtype=torch.bfloat16) -> torch.Tensor:
    return torch.zeros(shape, dtype=dtype).pin_memory()


def f64(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy().astype(np.float64)


def device_linear(x, w, dy):
    T, K = x.shape
    N = w.shape[0]
    xd, wd, dyd = dev(x), dev(w), dev(dy)
    q = {}
    for n_, t, fmt in (("x", xd, fp8.E4M3), ("w", wd, fp8.E4M3), ("dy", dyd, fp8.E5M2)):
        c = torch.empty(t.shape, dtype=torch.uint8, device="cuda")
        a, s, si = scalar(), scalar(), scalar()
        fp8.fp8_quantize(t, fmt, c, None, a, s, si)
        q[n_] = (c, si)
    y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    dx = torch.empty((T, K), dtype=torch.bfloat16, device="cuda")
    dw = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
    fp8.fp8_linear_fwd(q["x"][0], q["w"][0], q["x"][1], q["w"][1], y)
    fp8.fp8_linear_dgrad_rm(q["dy"][0], q["w"][0], q["dy"][1], q["w"][1], dx)
    fp8.fp8_linear_wgrad_rm(q["dy"][0], q["x"][0], q["dy"][1], q["x"][1], dw)
    torch.cuda.synchronize()
    return y, dx, dw


@pytest.mark.parametrize("T,N,K", [(256, 768, 256), (400, 272, 144), (1024, 2064, 528)])
def test_linear_step_from_host_buffers(T, N, K):
    seed = T + 3 * N + 7 * K
    problems = []
    for i in range(3):       # three calls on two workspaces: the third reuses the first without a sync
        x = synth.normal_bf16((T, K), seed + i, 0, 1.0, [1, K - 2], 50.0)
        w = synth.normal_bf16((N, K), seed + i, 1, synth.W_STD)
        dy = synth.normal_bf16((T, N), seed + i, 2, synth.GRAD_STD)
        problems.append((x, w, dy))
    nbytes = fp8.fp8_linear_step_host_workspace_bytes(T, N, K)
    assert nbytes > 0
    wss = [torch.empty(nbytes, dtype=torch.uint8, device="cuda") for _ in range(2)]
    outs = []
    for i, (x, w, dy) in enumerate(problems):
        hy, hdx, hdw = pinned_out((T, N)), pinned_out((T, K)), pinned_out((N, K))
        hin = (pinned(x), pinned(w), pinned(dy))
        fp8.fp8_linear_step_host(*hin, hy, hdx, hdw, wss[i % 2])
        outs.append((hin, hy, hdx, hdw))
    fp8.fp8_host_sync()
    assert fp8.fp8_device_status() == 0
    for (x, w, dy), (_, hy, hdx, hdw) in zip(problems, outs):
        x8, _, _, sx = o.quantize(x, o.E4M3)
        w8, _, _, sw = o.quantize(w, o.E4M3)
        dy8, _, _, sdy = o.quantize(dy, o.E5M2)
        for got, (ref, mag) in ((hy, o.linear_fwd(x8, w8, sx, sw)), (hdx, o.linear_dgrad(dy8, w8, sdy, sw)),
                                (hdw, o.linear_wgrad(dy8, x8, sdy, sx))):
            assert rel_err(f64(got), ref, mag) <= 2.0 ** -8
        y, dx, dw = device_linear(x, w, dy)
        for got, want in ((hy, y), (hdx, dx), (hdw, dw)):
            assert torch.equal(got.view(torch.int16), want.cpu().view(torch.int16))


def device_attention(q, k, v, do, causal):
    B, N, Hq, d = q.shape
    Hkv = k.shape[2]
    t = {}
    for n_, bits, fmt in (("q", q, fp8.E4M3), ("k", k, fp8.E4M3), ("v", v, fp8.E4M3), ("do", do, fp8.E5M2)):
        x = dev(bits)
        c = torch.empty(x.shape, dtype=torch.uint8, device="cuda")
        a, s, si = scalar(), scalar(), scalar()
        fp8.fp8_quantize(x, fmt, c, None, a, s, si)
        t[n_] = (c, si)
    s = d ** -0.5
    O = torch.empty((B, N, Hq, d), dtype=torch.bfloat16, device="cuda")
    LSE = torch.empty((B, Hq, N), dtype=torch.float32, device="cuda")
    fp8.fp8_attention_fwd(t["q"][0], t["k"][0], t["v"][0], t["q"][1], t["k"][1], t["v"][1], s, causal, O, LSE, None)
    dq = torch.zeros((B, N, Hq, d), dtype=torch.bfloat16, device="cuda")
    dk = torch.zeros((B, N, Hkv, d), dtype=torch.bfloat16, device="cuda")
    dv = torch.zeros((B, N, Hkv, d), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(fp8.fp8_attention_workspace_bytes(1, B, N, Hq, Hkv, d), dtype=torch.uint8, device="cuda")
    fp8.fp8_attention_bwd(t["q"][0], t["k"][0], t["v"][0], t["do"][0], O, LSE, t["q"][1], t["k"][1], t["v"][1],
                          t["do"][1], s, scalar(DS_SCALE), causal, dq, dk, dv, ws)
    torch.cuda.synchronize()
    return O, LSE, dq, dk, dv


@pytest.mark.parametrize("name,B,N,div", [("c1", 2, 144, 1), ("c3", 1, 400, 4), ("c4", 1, 272, 8)])
def test_attention_step_from_host_buffers(name, B, N, div):
    cfg = synth.CONFIGS[name]
    Hq, Hkv, d = cfg.n_q_heads // div, max(1, cfg.n_kv_heads // div), cfg.head_dim
    cfg = synth.BlockConfig(**{**cfg.__dict__, "n_q_heads": Hq, "n_kv_heads": Hkv})
    nbytes = fp8.fp8_attention_step_host_workspace_bytes(B, N, Hq, Hkv, d)
    assert nbytes > 0
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    runs = []
    for i in range(2):       # the same workspace twice, no sync in between
        q, k, v, do = synth.attention_inputs(synth.BlockConfig(**{**cfg.__dict__, "seed": cfg.seed + 11 * i}), seq=N, batch=B)
        hin = tuple(pinned(a) for a in (q, k, v, do))
        ho, hdq = pinned_out((B, N, Hq, d)), pinned_out((B, N, Hq, d))
        hdk, hdv = pinned_out((B, N, Hkv, d)), pinned_out((B, N, Hkv, d))
        hlse = pinned_out((B, Hq, N), torch.float32)
        fp8.fp8_attention_step_host(*hin, d ** -0.5, DS_SCALE, True, ho, hlse, hdq, hdk, hdv, ws)
        runs.append(((q, k, v, do), hin, (ho, hlse, hdq, hdk, hdv)))
    fp8.fp8_host_sync()
    assert fp8.fp8_device_status() == 0
    for (q, k, v, do), _, (ho, hlse, hdq, hdk, hdv) in runs:
        O, LSE, dq, dk, dv = device_attention(q, k, v, do, True)
        assert torch.equal(ho.view(torch.int16), O.cpu().view(torch.int16))
        assert torch.equal(hlse, LSE.cpu())
        assert torch.equal(hdk.view(torch.int16), dk.cpu().view(torch.int16))
        assert torch.equal(hdv.view(torch.int16), dv.cpu().view(torch.int16))
        a, b = f64(hdq), f64(dq)
        assert np.abs(b).max() > 0
        if d == 64:
            assert np.array_equal(a, b)
        else:
            assert np.max(np.abs(a - b)) <= 2.0 ** -7 * np.abs(b).max()
    # the oracle on the first problem: forward output and log-sum-exp (the gradients' parity is that of the device
    # chain, which the attention tests hold against the oracle; here they are bit-equal to it)
    (q, k, v, do), _, (ho, hlse, _, _, _) = runs[0]
    qq = {}
    for n_, bits, fmt in (("q", q, o.E4M3), ("k", k, o.E4M3), ("v", v, o.E4M3)):
        c, _, _, si = o.quantize(bits, fmt)
        qq[n_] = (c, float(si))
    p = o.attn_params(B, N, Hq, Hkv, d, causal=True, quant=True, kv_block=KV_BLOCK, max_mode=0, s=d ** -0.5,
                      q_inv=qq["q"][1], k_inv=qq["k"][1], v_inv=qq["v"][1], flip_eps=FLIP_EPS)
    ref, lse, mag, slack = o.attention_fwd(qq["q"][0], qq["k"][0], qq["v"][0], p, with_slack=True)
    got = f64(ho).transpose(0, 2, 1, 3).reshape(B * Hq, N, d)
    assert rel_err(got, ref, mag, slack) <= TOL_FWD
    glse = hlse.numpy().astype(np.float64).reshape(B * Hq, N)
    assert np.max(np.abs(glse - lse)) <= 1e-3 * max(1.0, np.abs(lse).max())


def test_host_step_rejects_bad_arguments():
    ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    h = pinned_out((16, 16))
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_linear_step_host(h, h, h, h, h, h, ws)
    assert e.value.status == -5
    assert fp8.fp8_attention_step_host_workspace_bytes(1, 128, 4, 4, 96) == 0      # head_dim 64 or 128 only
    assert fp8.fp8_attention_step_host_workspace_bytes(1, 128, 4, 3, 64) == 0      # Hq % Hkv
    big = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    hq = pinned_out((1, 16, 2, 96))
    hl = pinned_out((1, 2, 16), torch.float32)
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_attention_step_host(hq, hq, hq, hq, 0.1, 1.0, True, hq, hl, hq, hq, hq, big)
    assert e.value.status == -3
    fp8.fp8_host_sync()
