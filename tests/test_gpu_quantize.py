"""GPU parity: amax -> scale -> cast must match the oracle bit for bit (through the C ABI)."""
import numpy as np
import pytest
import torch

import oracle as o
import paper_2505_20524_b200 as fp8
from paper_2505_20524_b200 import synth
from gpu_util import dev, host, scalar, gpu_quantize

pytestmark = pytest.mark.gpu
FMTS = [o.E4M3, o.E5M2]


def bits(t):
    return int(t.cpu().view(torch.int32).item()) & 0xFFFFFFFF


@pytest.mark.parametrize("fmt", FMTS)
def test_all_65536_bf16_patterns_scale_one(fmt):
    x = np.arange(65536, dtype=np.uint16)
    out = torch.empty(65536, dtype=torch.uint8, device="cuda")
    fp8.fp8_cast(dev(x), scalar(1.0), fmt, out)
    got = host(out)
    exp = o.cast(x, 1.0, fmt)
    vals = o.bf16_to_f32(x)
    ok = ~np.isnan(vals)
    assert np.array_equal(got[ok], exp[ok])
    assert np.isnan(o.decode_array(got[~ok], fmt)).all()      # a NaN input gives a NaN code


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("n", [1, 7, 16, 1000, 4096 + 5, (1 << 20) + 3, 1 << 24])
def test_flat_quantize_bit_exact(fmt, n):
    x = synth.flat_tensor(n, seed=2 + n % 7)
    q, _, a, s, si = gpu_quantize(x, fmt)
    eq, ea, es, esi = o.quantize(x, fmt)
    assert bits(a) == int(np.float32(ea).view(np.uint32))
    assert bits(s) == int(np.float32(es).view(np.uint32))
    assert bits(si) == int(np.float32(esi).view(np.uint32))
    assert np.array_equal(host(q), eq)


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("shape", [(16, 16), (256, 256), (48, 272), (400, 144), (1024, 768), (2048, 5632)])
def test_cast_with_transposed_copy(fmt, shape):
    cols = synth.choose_columns(shape[1], 2, 0, 1)
    x = synth.normal_bf16(shape, 0, 3, 1.0, cols, 50.0)
    q, qt, a, s, si = gpu_quantize(x, fmt, transpose=True)
    eq, ea, es, esi = o.quantize(x, fmt)
    assert bits(a) == int(np.float32(ea).view(np.uint32))
    assert np.array_equal(host(q), eq)
    assert np.array_equal(host(qt), eq.T)


def test_amax_scale_cast_separately_and_fused_amax():
    x = synth.normal_bf16((512, 384), 1, 4, 3.0)
    xd = dev(x)
    a, s, si, a2 = scalar(), scalar(), scalar(), scalar(123.0)
    fp8.fp8_amax(xd, a)
    assert float(a.item()) == float(o.amax(x))
    for fmt in FMTS:
        for margin in (0, 1, 3):
            fp8.fp8_scale(a, fmt, margin, s, si)
            es, esi = o.scale(o.amax(x), fmt, margin)
            assert bits(s) == int(es.view(np.uint32)) and bits(si) == int(esi.view(np.uint32))
        fp8.fp8_scale(a, fmt, 0, s, si)
        out = torch.empty(x.shape, dtype=torch.uint8, device="cuda")
        out_t = torch.empty(x.shape[::-1], dtype=torch.uint8, device="cuda")
        fp8.fp8_cast(xd, s, fmt, out, None, a2)                       # delayed-scaling style: cast + amax
        assert float(a2.item()) == float(o.amax(x))
        es, _ = o.scale(o.amax(x), fmt)
        assert np.array_equal(host(out), o.cast(x, es, fmt))
        a2.fill_(7.0)
        fp8.fp8_cast(xd, s, fmt, out, out_t, a2)
        assert float(a2.item()) == float(o.amax(x))
        assert np.array_equal(host(out_t), o.cast(x, es, fmt).T)


def test_scale_guards():
    s, si = scalar(), scalar()
    for a, fmt in ((0.0, o.E4M3), (float("inf"), o.E5M2), (1e-40, o.E5M2), (200.0, o.E4M3)):
        fp8.fp8_scale(scalar(a), fmt, 0, s, si)
        es, esi = o.scale(np.float32(a), fmt)
        assert bits(s) == int(es.view(np.uint32)) and bits(si) == int(esi.view(np.uint32))


def test_saturating_cast_with_stale_scale():
    x = synth.normal_bf16((64, 64), 5, 5, 100.0)
    for fmt in FMTS:
        out = torch.empty(x.shape, dtype=torch.uint8, device="cuda")
        fp8.fp8_cast(dev(x), scalar(1000.0), fmt, out)
        got = host(out)
        assert np.array_equal(got, o.cast(x, 1000.0, fmt))
        assert np.isfinite(o.decode_array(got, fmt)).all()


def test_argument_validation_returns_errors_not_faults():
    x = dev(synth.normal_bf16((32, 32), 0, 0, 1.0))
    out = torch.empty((32, 32), dtype=torch.uint8, device="cuda")
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_cast(x, scalar(1.0), 5, out)
    assert e.value.status == -4
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_cast(x, None, 0, out)
    assert e.value.status == -1
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_cast(x.view(torch.int16).flatten()[1:].view(torch.bfloat16), scalar(1.0), 0, out)
    assert e.value.status == -2
    # empty inputs are refused, not launched
    empty = torch.empty(0, dtype=torch.bfloat16, device="cuda")
    for call in (lambda: fp8.fp8_amax(empty, scalar(0.0)),
                 lambda: fp8.fp8_cast(empty, scalar(1.0), 0, torch.empty(0, dtype=torch.uint8, device="cuda"))):
        with pytest.raises(fp8.Fp8Error) as e:
            call()
        assert e.value.status in (-1, -3)       # an empty torch tensor has a null data pointer
    assert fp8.fp8_device_status() == 0


def test_delayed_scaling_ring_matches_oracle():
    """fp8_scale_update against the oracle over more steps than the history holds (l = 1024 as in Appendix E)."""
    l, steps = 1024, 2200
    rng = np.random.default_rng(3)
    amaxes = np.abs(rng.normal(size=steps)).astype(np.float32) * np.where(rng.random(steps) < 0.01, 40.0, 1.0).astype(np.float32)
    hist_d = torch.zeros(l, dtype=torch.float32, device="cuda")
    head_d = torch.zeros(1, dtype=torch.int32, device="cuda")
    a_d = torch.from_numpy(amaxes).cuda()
    s, si = scalar(), scalar()
    hist = np.zeros(l, dtype=np.float32)
    head = 0
    for t in range(steps):
        fp8.fp8_scale_update(hist_d, head_d, a_d[t:t + 1], o.E4M3, 0, s, si)
        head, es, esi = o.scale_update(hist, head, amaxes[t], o.E4M3)
        if t % 97 == 0 or t == steps - 1:
            assert bits(s) == int(es.view(np.uint32)) and bits(si) == int(esi.view(np.uint32)), t
            assert int(head_d.item()) == head
            assert np.array_equal(hist_d.cpu().numpy(), hist)


def test_delayed_scaling_step_is_one_pass():
    """cast with last step's scale + fused amax, then the ring update: equals the oracle's chain bit for bit."""
    l = 16
    hist_d = torch.zeros(l, dtype=torch.float32, device="cuda")
    head_d = torch.zeros(1, dtype=torch.int32, device="cuda")
    s, si, a = scalar(1.0), scalar(1.0), scalar()
    hist = np.zeros(l, dtype=np.float32)
    head, es = 0, np.float32(1.0)
    for step in range(5):
        x = synth.normal_bf16((256, 128), 10 + step, 1, 1.0 + step)
        out = torch.empty(x.shape, dtype=torch.uint8, device="cuda")
        fp8.fp8_cast(dev(x), s, o.E4M3, out, None, a)                 # scale from the history so far
        assert np.array_equal(host(out), o.cast(x, es, o.E4M3))
        fp8.fp8_scale_update(hist_d, head_d, a, o.E4M3, 0, s, si)
        head, es, _ = o.scale_update(hist, head, o.amax(x), o.E4M3)
        assert bits(s) == int(es.view(np.uint32))


def test_bounded_wait_gives_up_and_reports():
    """A wait that nothing completes runs out at its limit: FP8_ERR_TIMEOUT in the status word, the kernel returns,
    and the context stays usable (the path every kernel of the library takes when a wait expires)."""
    import time
    assert fp8.fp8_device_status() == 0
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    t0 = time.time()
    fp8.fp8_selftest_wait_timeout(1 << 22, flag)          # about 2 ms of SM clocks
    torch.cuda.synchronize()
    assert time.time() - t0 < 5.0
    assert int(flag.item()) == 1
    assert fp8.fp8_device_status() == -7                   # FP8_ERR_TIMEOUT, cleared by the read
    assert fp8.fp8_device_status() == 0
    x = torch.arange(-8, 8, dtype=torch.float32, device="cuda").to(torch.bfloat16)
    a = torch.zeros(1, dtype=torch.float32, device="cuda")
    fp8.fp8_amax(x, a)                                      # the next kernel runs as usual
    torch.cuda.synchronize()
    assert float(a.item()) == 8.0 and fp8.fp8_device_status() == 0
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_selftest_wait_timeout(0, flag)
    assert e.value.status == -3


def test_quantize_multi_equals_per_tensor_quantize_and_oracle():
    """fp8_quantize_multi (one reduction launch and one cast launch for a group of tensors) gives every tensor the codes
    and the three scalars of its own fp8_quantize: sizes from 1 element to several blocks, ragged tails, both formats,
    an all-zero tensor (scale 1), eight tensors (the maximum) and a single one."""
    sizes = [1, 15, 16, 4096 + 7, 300_000, 1 << 20, (1 << 20) + 24, 2_500_000]
    fmts = [fp8.E4M3, fp8.E5M2, fp8.E4M3, fp8.E5M2, fp8.E4M3, fp8.E4M3, fp8.E5M2, fp8.E4M3]
    xs_host = [synth.flat_tensor(n, seed=40 + i) if n >= 16 else synth.normal_bf16((1, n), 40 + i, 0, 3.0).reshape(-1)
               for i, n in enumerate(sizes)]
    xs_host[4] = np.zeros(sizes[4], dtype=np.uint16)            # amax 0: scale 1
    for take in (slice(0, 8), slice(3, 4), slice(4, 7)):
        xs = [dev(x) for x in xs_host[take]]
        f = fmts[take]
        outs = [torch.full((x.numel(),), 0xAA, dtype=torch.uint8, device="cuda") for x in xs]
        scal = torch.full((3 * len(xs),), -1.0, dtype=torch.float32, device="cuda")
        fp8.fp8_quantize_multi(xs, f, outs, scal)
        torch.cuda.synchronize()
        sc = scal.cpu().numpy()
        for i, (x, xh, fmt, out) in enumerate(zip(xs, xs_host[take], f, outs)):
            q = torch.empty(x.numel(), dtype=torch.uint8, device="cuda")
            a, s_, si = scalar(), scalar(), scalar()
            fp8.fp8_quantize(x.reshape(1, -1), fmt, q, None, a, s_, si)
            assert torch.equal(out, q), i
            assert sc[3 * i] == a.item() and sc[3 * i + 1] == s_.item() and sc[3 * i + 2] == si.item(), i
            oc, oa, osc, osi = o.quantize(xh.reshape(1, -1), fmt)
            assert np.array_equal(out.cpu().numpy(), oc.reshape(-1)), i
            assert np.float32(sc[3 * i]) == np.float32(oa) and np.float32(sc[3 * i + 1]) == np.float32(osc), i
    with pytest.raises(fp8.Fp8Error):
        fp8.fp8_quantize_multi([dev(xs_host[2])] * 9, [fp8.E4M3] * 9, [torch.empty(16, dtype=torch.uint8, device="cuda")] * 9,
                               torch.empty(27, device="cuda"))


def test_delayed_multi_is_the_oracle_chain_in_one_launch():
    """fp8_quantize_delayed_multi over more steps than the history holds, with the same pointers every step: per tensor
    and step the codes equal the oracle's cast under the scale of the history so far, the published scale and reciprocal
    are that scale's, and amax, history, position and next scale equal the oracle's scale_update; sizes from 1 element
    to several blocks per tensor, both formats, an all-zero tensor, a ring of length 3 (wraps twice) with margin 1; the
    counter words are zero after every call."""
    l, margin, steps = 3, 1, 8
    sizes = [1, 15, 4096 + 7, 300_000, (1 << 20) + 24, 2_500_000]
    fmts = [fp8.E4M3, fp8.E5M2, fp8.E4M3, fp8.E5M2, fp8.E5M2, fp8.E4M3]
    n = len(sizes)
    hist_d = [torch.zeros(l, dtype=torch.float32, device="cuda") for _ in range(n)]
    head_d = [torch.zeros(1, dtype=torch.int32, device="cuda") for _ in range(n)]
    nxt = [scalar(1.0) for _ in range(n)]                     # the first step casts under scale 1
    cur, cur_inv = [scalar(-1.0) for _ in range(n)], [scalar(-1.0) for _ in range(n)]
    amax_d = [scalar(-1.0) for _ in range(n)]
    sync = torch.zeros(2 * n, dtype=torch.int32, device="cuda")
    hist = [np.zeros(l, dtype=np.float32) for _ in range(n)]
    head = [0] * n
    es = [np.float32(1.0)] * n
    for step in range(steps):
        xs_host = []
        for i, sz in enumerate(sizes):
            if i == 3 and step == 2:
                xs_host.append(np.zeros(sz, dtype=np.uint16))              # amax 0 enters the history
            elif sz >= 16:
                xs_host.append(synth.flat_tensor(sz, seed=100 + 10 * step + i))
            else:
                xs_host.append(synth.normal_bf16((1, sz), 100 + 10 * step + i, 0, 1.0 + step).reshape(-1))
        xs = [dev(x) for x in xs_host]
        outs = [torch.full((sz,), 0xAA, dtype=torch.uint8, device="cuda") for sz in sizes]
        fp8.fp8_quantize_delayed_multi(xs, fmts, outs, hist_d, head_d, nxt, amax_d, cur, cur_inv, margin, sync)
        torch.cuda.synchronize()
        assert int(sync.abs().sum().item()) == 0
        for i in range(n):
            assert np.array_equal(outs[i].cpu().numpy(), o.cast(xs_host[i].reshape(1, -1), es[i], fmts[i]).reshape(-1)), (step, i)
            assert np.float32(cur[i].item()) == es[i], (step, i)
            assert np.float32(cur_inv[i].item()) == np.float32(1.0) / es[i], (step, i)
            a = o.amax(xs_host[i])
            assert np.float32(amax_d[i].item()) == np.float32(a), (step, i)
            head[i], s_new, _ = o.scale_update(hist[i], head[i], a, fmts[i], margin)
            assert bits(nxt[i]) == int(s_new.view(np.uint32)), (step, i)
            assert int(head_d[i].item()) == head[i] and np.array_equal(hist_d[i].cpu().numpy(), hist[i]), (step, i)
            es[i] = s_new
    # a single tensor, and the argument checks
    one = dev(synth.flat_tensor(70_000, seed=7))
    out = torch.empty(70_000, dtype=torch.uint8, device="cuda")
    fp8.fp8_quantize_delayed_multi([one], [fp8.E4M3], [out], hist_d[:1], head_d[:1], nxt[:1], amax_d[:1], cur[:1],
                                   cur_inv[:1], 0, sync)
    assert np.array_equal(out.cpu().numpy(), o.cast(host(one).reshape(1, -1), es[0], fp8.E4M3).reshape(-1))
    with pytest.raises(fp8.Fp8Error):      # this step's scale may not be published over the state it is read from
        fp8.fp8_quantize_delayed_multi([one], [fp8.E4M3], [out], hist_d[:1], head_d[:1], nxt[:1], amax_d[:1], nxt[:1],
                                       cur_inv[:1], 0, sync)
    with pytest.raises(fp8.Fp8Error):
        fp8.fp8_quantize_delayed_multi([one] * 9, [fp8.E4M3] * 9, [out] * 9, hist_d[:1] * 9, head_d[:1] * 9,
                                       nxt[:1] * 9, amax_d[:1] * 9, cur[:1] * 9, cur_inv[:1] * 9, 0,
                                       torch.zeros(18, dtype=torch.int32, device="cuda"))
