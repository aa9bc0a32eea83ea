"""GPU parity: FP8 linear forward / dgrad / wgrad against the double-accumulating oracle on identical codes."""
import numpy as np
import pytest
import torch

import oracle as o
import paper_2505_20524_b200 as fp8
from paper_2505_20524_b200 import synth
from gpu_util import dev, host, scalar, gpu_quantize, bf16_host_to_f64, rel_err

pytestmark = pytest.mark.gpu

# max |gpu - ref| / sum_k |a_k||b_k| : FP32 accumulation (<= K * 2^-24) plus one BF16 rounding (2^-9 of |ref|)
TOL_BF16 = 2e-2      # the stated bar; observed values are near 2^-9
TOL_FP32 = 1e-4


def run_three(x, w, dy, out_dtype, rows=None):
    """Quantize on the GPU, run the three GEMMs, return GPU outputs and oracle inputs."""
    T, K = x.shape
    N = w.shape[0]
    x8, x8t, _, _, sx = gpu_quantize(x, o.E4M3, True)
    w8, w8t, _, _, sw = gpu_quantize(w, o.E4M3, True)
    dy8, dy8t, _, _, sdy = gpu_quantize(dy, o.E5M2, True)
    y = torch.empty((T, N), dtype=out_dtype, device="cuda")
    dx = torch.empty((T, K), dtype=out_dtype, device="cuda")
    dw = torch.empty((N, K), dtype=out_dtype, device="cuda")
    fp8.fp8_linear_fwd(x8, w8, sx, sw, y)
    fp8.fp8_linear_dgrad(dy8, w8t, sdy, sw, dx)
    fp8.fp8_linear_wgrad(dy8t, x8t, sdy, sx, dw)
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    # the oracle quantises the same BF16 bytes itself (bit-exactness of that step is tested elsewhere)
    ox8, _, _, osx = o.quantize(x, o.E4M3)
    ow8, _, _, osw = o.quantize(w, o.E4M3)
    ody8, _, _, osdy = o.quantize(dy, o.E5M2)
    assert np.array_equal(host(x8), ox8) and np.array_equal(host(dy8), ody8)
    return (y, dx, dw), (ox8, ow8, ody8, osx, osw, osdy)


def check(got_t, ref, mag, tol):
    got = got_t.float().cpu().numpy().astype(np.float64)
    err = rel_err(got, ref, mag)
    assert err <= tol, err
    return err


@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("T,N,K", [(256, 768, 256), (256, 256, 256), (256, 1024, 256), (256, 256, 1024),
                                   (128, 128, 128), (400, 272, 144), (16, 16, 16), (144, 528, 2064)])
def test_three_gemms_match_oracle(T, N, K, out_dtype):
    cfg_seed = T * 7 + N * 3 + K
    cols = synth.choose_columns(K, 2, cfg_seed, 1)
    x = synth.normal_bf16((T, K), cfg_seed, 0, 1.0, cols, 50.0)
    w = synth.normal_bf16((N, K), cfg_seed, 1, synth.W_STD)
    dy = synth.normal_bf16((T, N), cfg_seed, 2, synth.GRAD_STD)
    (y, dx, dw), (x8, w8, dy8, sx, sw, sdy) = run_three(x, w, dy, out_dtype)
    tol = TOL_BF16 if out_dtype == torch.bfloat16 else TOL_FP32
    ref, mag = o.linear_fwd(x8, w8, sx, sw)
    e1 = check(y, ref, mag, tol)
    ref, mag = o.linear_dgrad(dy8, w8, sdy, sw)
    e2 = check(dx, ref, mag, tol)
    ref, mag = o.linear_wgrad(dy8, x8, sdy, sx)
    e3 = check(dw, ref, mag, tol)
    if out_dtype == torch.bfloat16:
        assert max(e1, e2, e3) <= 2.0 ** -8          # what the arithmetic should give: one BF16 rounding


@pytest.mark.parametrize("family", ["1cta", "2cta"])
@pytest.mark.parametrize("T,N,K", [(256, 256, 128), (400, 528, 144), (1024, 768, 2064), (272, 1040, 256)])
def test_both_kernel_families_on_ragged_shapes(family, T, N, K, monkeypatch):
    """FP8DPA_GEMM forces the single-CTA or the CTA-pair kernel; both must agree with the oracle on tiles that
    hang over the matrix edge (the pair kernel is otherwise only chosen for large matrices)."""
    monkeypatch.setenv("FP8DPA_GEMM", family)
    x = synth.normal_bf16((T, K), T + N, 0, 1.0, [1, K - 2], 50.0)
    w = synth.normal_bf16((N, K), T + N, 1, synth.W_STD)
    dy = synth.normal_bf16((T, N), T + N, 2, synth.GRAD_STD)
    for out_dtype, tol in ((torch.bfloat16, 2.0 ** -8), (torch.float32, TOL_FP32)):
        (y, dx, dw), (x8, w8, dy8, sx, sw, sdy) = run_three(x, w, dy, out_dtype)
        check(y, *o.linear_fwd(x8, w8, sx, sw), tol)
        check(dx, *o.linear_dgrad(dy8, w8, sdy, sw), tol)
        check(dw, *o.linear_wgrad(dy8, x8, sdy, sx), tol)
    if family == "2cta":                       # accumulate path of the pair kernel's epilogue
        prev = np.random.default_rng(1).normal(size=(N, K)).astype(np.float32) * 1e-3
        dwa = dev(prev.copy())
        x8d, x8t, _, _, sxd = gpu_quantize(x, o.E4M3, True)
        dy8d, dy8t, _, _, sdyd = gpu_quantize(dy, o.E5M2, True)
        fp8.fp8_linear_wgrad(dy8t, x8t, sdyd, sxd, dwa, accumulate=True)
        ref, mag = o.linear_wgrad(host(dy8d), host(x8d), float(sdyd.item()), float(sxd.item()),
                                  prev=prev.astype(np.float64))
        assert rel_err(host(dwa).astype(np.float64), ref, mag + np.abs(prev)) <= TOL_FP32


def test_wgrad_accumulate_fp32():
    T, N, K = 256, 128, 384
    x = synth.normal_bf16((T, K), 1, 0, 1.0)
    dy = synth.normal_bf16((T, N), 1, 2, synth.GRAD_STD)
    x8, x8t, _, _, sx = gpu_quantize(x, o.E4M3, True)
    dy8, dy8t, _, _, sdy = gpu_quantize(dy, o.E5M2, True)
    prev = np.random.default_rng(0).normal(size=(N, K)).astype(np.float32) * 1e-3
    dw = dev(prev.copy())
    fp8.fp8_linear_wgrad(dy8t, x8t, sdy, sx, dw, accumulate=True)
    ref, mag = o.linear_wgrad(host(dy8), host(x8), float(sdy.item()), float(sx.item()), prev=prev.astype(np.float64))
    assert rel_err(host(dw).astype(np.float64), ref, mag + np.abs(prev)) <= TOL_FP32


def test_exact_cases():
    """All-ones operands and an identity weight give exactly representable results."""
    K = 256
    ones = torch.full((128, K), 0x38, dtype=torch.uint8, device="cuda")
    y = torch.empty((128, 128), dtype=torch.float32, device="cuda")
    fp8.fp8_linear_fwd(ones, ones[:128], scalar(0.5), scalar(3.0), y)
    assert torch.all(y == K * 1.5)
    eye = torch.where(torch.eye(K, device="cuda", dtype=torch.bool), 0x38, 0).to(torch.uint8)
    x8 = dev(np.random.default_rng(1).integers(0, 0x7F, size=(128, K)).astype(np.uint8))
    y = torch.empty((128, K), dtype=torch.float32, device="cuda")
    fp8.fp8_linear_fwd(x8, eye, scalar(1.0), scalar(1.0), y)
    assert np.array_equal(host(y).astype(np.float64), o.decode_array(host(x8), o.E4M3))


def test_argument_validation():
    a = torch.zeros((64, 64), dtype=torch.uint8, device="cuda")
    y = torch.empty((64, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_linear_fwd(a[:, :40].contiguous(), a[:, :40].contiguous(), scalar(1), scalar(1), y)
    assert e.value.status == -3
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_linear_fwd(a, a, None, scalar(1), y)
    assert e.value.status == -1


@pytest.mark.parametrize("family", ["1cta", "2cta"])
@pytest.mark.parametrize("T,N,K", [(256, 768, 256), (400, 528, 144), (1024, 1040, 2064), (16, 16, 16)])
def test_fp8_output_epilogue(family, T, N, K, monkeypatch):
    """Producer form (delayed scaling): codes and amax equal the unfused chain bit for bit, and decode close to the oracle."""
    monkeypatch.setenv("FP8DPA_GEMM", family)
    seed = T + N + K
    cols = synth.choose_columns(K, 2, seed, 1)
    x = synth.normal_bf16((T, K), seed, 0, 1.0, cols, 50.0)
    w = synth.normal_bf16((N, K), seed, 1, synth.W_STD)
    dy = synth.normal_bf16((T, N), seed, 2, synth.GRAD_STD)
    x8, _, _, _, sx = gpu_quantize(x, o.E4M3, True)
    w8, w8t, _, _, sw = gpu_quantize(w, o.E4M3, True)
    dy8, _, _, _, sdy = gpu_quantize(dy, o.E5M2, True)
    for name, fmt in (("fwd", o.E4M3), ("dgrad", o.E5M2)):
        rows, cols_out = (T, N) if name == "fwd" else (T, K)
        ybf = torch.empty((rows, cols_out), dtype=torch.bfloat16, device="cuda")
        if name == "fwd":
            fp8.fp8_linear_fwd(x8, w8, sx, sw, ybf)
        else:
            fp8.fp8_linear_dgrad(dy8, w8t, sdy, sw, ybf)
        # a "delayed" scale: from a slightly larger amax than this step's (history maximum), not from this tensor
        a_now = scalar()
        fp8.fp8_amax(ybf, a_now)
        hist = scalar(float(a_now.item()) * 1.25)
        s, si = scalar(), scalar()
        fp8.fp8_scale(hist, fmt, 0, s, si)
        ref8 = torch.empty((rows, cols_out), dtype=torch.uint8, device="cuda")
        fp8.fp8_cast(ybf, s, fmt, ref8)
        got8 = torch.full((rows, cols_out), 0x55, dtype=torch.uint8, device="cuda")
        a = scalar(-3.0)
        if name == "fwd":
            fp8.fp8_linear_fwd_q(x8, w8, sx, sw, s, fmt, got8, a)
        else:
            fp8.fp8_linear_dgrad_q(dy8, w8t, sdy, sw, s, fmt, got8, a)
        torch.cuda.synchronize()
        assert fp8.fp8_device_status() == 0
        assert torch.equal(got8, ref8)                                   # same accumulators, same roundings
        assert float(a.item()) == float(a_now.item())
        # against the oracle: decode / scale within the GEMM tolerance plus half a quantisation step of the format
        ox8, _, _, osx = o.quantize(x, o.E4M3)
        ow8, _, _, osw = o.quantize(w, o.E4M3)
        ody8, _, _, osdy = o.quantize(dy, o.E5M2)
        ref, mag = o.linear_fwd(ox8, ow8, osx, osw) if name == "fwd" else o.linear_dgrad(ody8, ow8, osdy, osw)
        dec = o.decode_array(host(got8), fmt).astype(np.float64) * float(si.item())
        step = np.maximum(np.abs(ref) * (2.0 ** -3 if fmt == o.E4M3 else 2.0 ** -2),
                          (2.0 ** -9 if fmt == o.E4M3 else 2.0 ** -16) * float(si.item()))
        assert np.all(np.abs(dec - ref) <= TOL_BF16 * mag + 0.5 * step + 2.0 ** -8 * np.abs(ref))


def test_fp8_output_argument_validation():
    x8 = torch.zeros((32, 32), dtype=torch.uint8, device="cuda")
    s = scalar(1.0)
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_linear_fwd_q(x8, x8, s, s, None, 0, x8)
    assert e.value.status == -1
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_linear_fwd_q(x8, x8, s, s, s, 3, x8)
    assert e.value.status == -4


@pytest.mark.parametrize("family", ["1cta", "2cta"])
@pytest.mark.parametrize("T,N,K", [(256, 768, 256), (400, 528, 144), (1024, 1040, 2064), (16, 16, 16), (512, 256, 1024)])
def test_gradients_with_operands_read_in_place(family, T, N, K, monkeypatch):
    """dgrad / wgrad on the row-major FP8 tensors of the forward (MN-major UMMA operands) against the oracle and
    against the transposed-copy path."""
    monkeypatch.setenv("FP8DPA_GEMM", family)
    seed = 3 * T + N + K
    cols = synth.choose_columns(K, 2, seed, 1)
    x = synth.normal_bf16((T, K), seed, 0, 1.0, cols, 50.0)
    w = synth.normal_bf16((N, K), seed, 1, synth.W_STD)
    dy = synth.normal_bf16((T, N), seed, 2, synth.GRAD_STD)
    x8, x8t, _, _, sx = gpu_quantize(x, o.E4M3, True)
    w8, w8t, _, _, sw = gpu_quantize(w, o.E4M3, True)
    dy8, dy8t, _, _, sdy = gpu_quantize(dy, o.E5M2, True)
    for dt, tol in ((torch.bfloat16, 2.0 ** -8), (torch.float32, TOL_FP32)):
        dx = torch.empty((T, K), dtype=dt, device="cuda")
        dw = torch.empty((N, K), dtype=dt, device="cuda")
        fp8.fp8_linear_dgrad_rm(dy8, w8, sdy, sw, dx)
        fp8.fp8_linear_wgrad_rm(dy8, x8, sdy, sx, dw)
        dx2, dw2 = torch.empty_like(dx), torch.empty_like(dw)
        fp8.fp8_linear_dgrad(dy8, w8t, sdy, sw, dx2)
        fp8.fp8_linear_wgrad(dy8t, x8t, sdy, sx, dw2)
        torch.cuda.synchronize()
        assert fp8.fp8_device_status() == 0
        ox8, _, _, osx = o.quantize(x, o.E4M3)
        ow8, _, _, osw = o.quantize(w, o.E4M3)
        ody8, _, _, osdy = o.quantize(dy, o.E5M2)
        ref, mag = o.linear_dgrad(ody8, ow8, osdy, osw)
        check(dx, ref, mag, tol)
        ref, mag = o.linear_wgrad(ody8, ox8, osdy, osx)
        check(dw, ref, mag, tol)
        # the same products in the same order of reduction: the two operand forms agree to FP32 accumulation noise
        assert (dx.float() - dx2.float()).abs().max().item() <= 2.0 ** -7 * dx2.float().abs().max().item() + 1e-30
        assert (dw.float() - dw2.float()).abs().max().item() <= 2.0 ** -7 * dw2.float().abs().max().item() + 1e-30
    # accumulate into FP32 weight gradients
    acc = torch.full((N, K), 0.5, dtype=torch.float32, device="cuda")
    fp8.fp8_linear_wgrad_rm(dy8, x8, sdy, sx, acc, accumulate=True)
    ref, mag = o.linear_wgrad(ody8, ox8, osdy, osx, prev=np.full((N, K), 0.5))
    check(acc, ref, mag + 0.5, TOL_FP32)


@pytest.mark.parametrize("sizes,N,K", [([300, 0, 129, 512, 83], 528, 144), ([256, 256], 256, 256),
                                        ([1000, 17, 2000, 1, 600, 0, 0, 350], 1024, 512), ([16], 16, 16)])
@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
def test_grouped_forward_matches_oracle_per_expert(sizes, N, K, out_dtype):
    """Mixture-of-experts FFN product: token rows sorted by expert, one weight matrix and one weight scale per expert."""
    E, T = len(sizes), sum(sizes)
    Tpad = T + 37                                               # rows past the last group stay untouched
    offs = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    x = synth.normal_bf16((Tpad, K), 90 + E, 0, 1.0, synth.choose_columns(K, 2, 90, 1), 40.0)
    x8, _, _, _, sx = gpu_quantize(x, o.E4M3, False)
    ox8, _, _, osx = o.quantize(x, o.E4M3)
    w8 = torch.empty((E, N, K), dtype=torch.uint8, device="cuda")
    sw = torch.empty(E, dtype=torch.float32, device="cuda")
    ow = []
    for e in range(E):
        w = synth.normal_bf16((N, K), 90 + E, 10 + e, synth.W_STD * (1 + e))      # a different range per expert
        c, _, _, _, si = gpu_quantize(w, o.E4M3, False)
        w8[e].copy_(c)
        sw[e:e + 1].copy_(si)
        ow.append(o.quantize(w, o.E4M3))
    y = torch.full((Tpad, N), 7.0, dtype=out_dtype, device="cuda")
    fp8.fp8_grouped_linear_fwd(x8, w8, sx, sw, torch.from_numpy(offs).cuda(), y)
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    got = y.float().cpu().numpy().astype(np.float64)
    tol = 2.0 ** -8 if out_dtype == torch.bfloat16 else TOL_FP32
    for e in range(E):
        r0, r1 = int(offs[e]), int(offs[e + 1])
        if r1 == r0:
            continue
        ref, mag = o.linear_fwd(ox8[r0:r1], ow[e][0], osx, ow[e][3])
        assert rel_err(got[r0:r1], ref, mag) <= tol, e
    assert np.all(got[T:] == 7.0)


def test_grouped_forward_with_offsets_that_break_the_contract_stays_inside_the_output():
    """The group offsets live on the device, so the host cannot validate them.  An array that is not ascending or
    runs past T must not make the kernel store outside the [T, N] output: the kernel clips every offset into
    [previous offset, T]."""
    T, N, K, E = 1024, 256, 128, 4
    guard = 64
    x8 = torch.randint(0x20, 0x48, (T + guard, K), dtype=torch.uint8, device="cuda")
    w8 = torch.randint(0x20, 0x48, (E, N, K), dtype=torch.uint8, device="cuda")
    sx, sw = scalar(2.0 ** -4), torch.full((E,), 2.0 ** -5, device="cuda")
    for bad in ([0, 300, 200, 900, 5000], [-7, 100, 100, 2000, 1500], [0, 1 << 30, 3, 4, 5]):
        y = torch.full((T + guard, N), 7.0, dtype=torch.bfloat16, device="cuda")
        offs = torch.tensor(bad, dtype=torch.int32, device="cuda")
        fp8.fp8_grouped_linear_fwd(x8[:T], w8, sx, sw, offs, y[:T])
        torch.cuda.synchronize()
        assert fp8.fp8_device_status() == 0
        assert torch.all(y[T:] == 7.0)
        assert torch.isfinite(y.float()).all()


@pytest.mark.parametrize("sizes,N,K", [([300, 0, 129, 512, 83], 512, 144), ([256, 256], 256, 256),
                                        ([1000, 17, 2000, 1, 600, 0, 0, 350], 1024, 528), ([16], 128, 16)])
@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
def test_grouped_data_gradient_matches_oracle_per_expert(sizes, N, K, out_dtype):
    """dX of the mixture-of-experts product: gradient rows sorted by expert, every expert's [N, K] weights read in place."""
    E, T = len(sizes), sum(sizes)
    Tpad = T + 21
    offs = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    dy = synth.normal_bf16((Tpad, N), 70 + E, 0, synth.GRAD_STD)
    dy8, _, _, _, sdy = gpu_quantize(dy, o.E5M2, False)
    ody8, _, _, osdy = o.quantize(dy, o.E5M2)
    w8 = torch.empty((E, N, K), dtype=torch.uint8, device="cuda")
    sw = torch.empty(E, dtype=torch.float32, device="cuda")
    ow = []
    for e in range(E):
        w = synth.normal_bf16((N, K), 70 + E, 10 + e, synth.W_STD * (1 + e))
        c, _, _, _, si = gpu_quantize(w, o.E4M3, False)
        w8[e].copy_(c)
        sw[e:e + 1].copy_(si)
        ow.append(o.quantize(w, o.E4M3))
    dx = torch.full((Tpad, K), 7.0, dtype=out_dtype, device="cuda")
    fp8.fp8_grouped_linear_dgrad(dy8, w8, sdy, sw, torch.from_numpy(offs).cuda(), dx)
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    got = dx.float().cpu().numpy().astype(np.float64)
    tol = 2.0 ** -8 if out_dtype == torch.bfloat16 else TOL_FP32
    for e in range(E):
        r0, r1 = int(offs[e]), int(offs[e + 1])
        if r1 == r0:
            continue
        ref, mag = o.linear_dgrad(ody8[r0:r1], ow[e][0], osdy, ow[e][3])
        assert rel_err(got[r0:r1], ref, mag) <= tol, e
    assert np.all(got[T:] == 7.0)
    with pytest.raises(fp8.Fp8Error) as err:                       # a reduction block must not span two experts
        fp8.fp8_grouped_linear_dgrad(dy8[:, :N - 16].contiguous(), w8[:, :N - 16].contiguous(), sdy, sw,
                                     torch.from_numpy(offs).cuda(), dx)
    assert err.value.status == -3


@pytest.mark.parametrize("sizes,N,K", [([300, 0, 129, 512, 83], 528, 144), ([256, 256], 256, 256),
                                        ([1000, 17, 2000, 1, 600, 0, 0, 350], 1024, 512), ([5], 16, 16)])
def test_grouped_weight_gradient_matches_oracle_per_expert(sizes, N, K):
    """dW of the mixture-of-experts product: per expert the reduction runs over its (ragged) slice of the sorted rows."""
    E, T = len(sizes), sum(sizes)
    Tpad = T + 9
    offs = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    dy = synth.normal_bf16((Tpad, N), 60 + E, 0, synth.GRAD_STD)
    x = synth.normal_bf16((Tpad, K), 60 + E, 1, 1.0, synth.choose_columns(K, 2, 60, 1), 40.0)
    dy8, _, _, _, sdy = gpu_quantize(dy, o.E5M2, False)
    x8, _, _, _, sx = gpu_quantize(x, o.E4M3, False)
    ody8, _, _, osdy = o.quantize(dy, o.E5M2)
    ox8, _, _, osx = o.quantize(x, o.E4M3)
    dw = torch.full((E, N, K), 7.0, dtype=torch.bfloat16, device="cuda")
    fp8.fp8_grouped_linear_wgrad(dy8, x8, sdy, sx, offs, dw)
    acc = torch.full((E, N, K), 0.25, dtype=torch.float32, device="cuda")
    fp8.fp8_grouped_linear_wgrad(dy8, x8, sdy, sx, offs, acc, accumulate=True)
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    got, gacc = dw.float().cpu().numpy().astype(np.float64), acc.cpu().numpy().astype(np.float64)
    for e in range(E):
        r0, r1 = int(offs[e]), int(offs[e + 1])
        if r1 == r0:
            assert np.all(got[e] == 0.0) and np.all(gacc[e] == 0.25)      # no tokens: zero gradient / untouched
            continue
        ref, mag = o.linear_wgrad(ody8[r0:r1], ox8[r0:r1], osdy, osx)
        assert rel_err(got[e], ref, mag) <= 2.0 ** -8, e
        assert rel_err(gacc[e], ref + 0.25, mag + 0.25) <= TOL_FP32, e
    with pytest.raises(fp8.Fp8Error) as err:
        fp8.fp8_grouped_linear_wgrad(dy8, x8, sdy, sx, [0, T + 100], dw[:1])
    assert err.value.status == -3


@pytest.mark.parametrize("sizes,N,K", [([300, 0, 129, 512, 83], 528, 144), ([256, 256], 256, 256),
                                        ([1000, 17, 2000, 1, 600, 0, 0, 350], 1024, 512), ([5], 16, 16),
                                        ([0, 0, 384], 272, 1040), ([127, 1, 128, 129], 256, 512)])
def test_grouped_weight_gradient_in_one_launch_with_device_offsets(sizes, N, K):
    """The same gradients from fp8_grouped_linear_wgrad_dev: one launch over (expert, output tile), the offsets read on
    the device, the ragged last block of every expert taken from a zero-padded copy.  Rows past the last offset and the
    rows of the neighbouring experts that share a block of 128 must not leak into a gradient; out-of-range offsets are
    clamped, not followed."""
    E, T = len(sizes), sum(sizes)
    Tpad = T + 9
    offs = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    dy = synth.normal_bf16((Tpad, N), 80 + E, 0, synth.GRAD_STD)
    x = synth.normal_bf16((Tpad, K), 80 + E, 1, 1.0, synth.choose_columns(K, 2, 80, 1), 40.0)
    dy8, _, _, _, sdy = gpu_quantize(dy, o.E5M2, False)
    x8, _, _, _, sx = gpu_quantize(x, o.E4M3, False)
    ody8, _, _, osdy = o.quantize(dy, o.E5M2)
    ox8, _, _, osx = o.quantize(x, o.E4M3)
    doffs = torch.from_numpy(offs).cuda()
    ws = torch.full((fp8.fp8_grouped_linear_wgrad_workspace_bytes(E, N),), 0x7B, dtype=torch.uint8, device="cuda")
    dw = torch.full((E, N, K), 7.0, dtype=torch.bfloat16, device="cuda")
    fp8.fp8_grouped_linear_wgrad_dev(dy8, x8, sdy, sx, doffs, dw, ws)
    acc = torch.full((E, N, K), 0.25, dtype=torch.float32, device="cuda")
    fp8.fp8_grouped_linear_wgrad_dev(dy8, x8, sdy, sx, doffs, acc, ws, accumulate=True)
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    got, gacc = dw.float().cpu().numpy().astype(np.float64), acc.cpu().numpy().astype(np.float64)
    for e in range(E):
        r0, r1 = int(offs[e]), int(offs[e + 1])
        if r1 == r0:
            assert np.all(got[e] == 0.0) and np.all(gacc[e] == 0.25)      # no tokens: zero gradient / unchanged
            continue
        ref, mag = o.linear_wgrad(ody8[r0:r1], ox8[r0:r1], osdy, osx)
        assert rel_err(got[e], ref, mag) <= 2.0 ** -8, e
        assert rel_err(gacc[e], ref + 0.25, mag + 0.25) <= TOL_FP32, e
    # bit-equal to the per-expert launches (same kernel arithmetic, same order of the reduction blocks)
    dw2 = torch.full((E, N, K), 7.0, dtype=torch.bfloat16, device="cuda")
    fp8.fp8_grouped_linear_wgrad(dy8, x8, sdy, sx, offs, dw2)
    if N >= 256 and K >= 256:
        assert torch.equal(dw.view(torch.int16), dw2.view(torch.int16))
    # offsets that break the contract are clamped to [0, T] and made ascending: no access past the tensors
    bad = torch.tensor([0, Tpad + 500] + [Tpad + 900] * (E - 1), dtype=torch.int32, device="cuda")
    fp8.fp8_grouped_linear_wgrad_dev(dy8, x8, sdy, sx, bad, dw, ws)
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    ref, mag = o.linear_wgrad(ody8, ox8, osdy, osx)
    assert rel_err(dw[0].float().cpu().numpy().astype(np.float64), ref, mag) <= 2.0 ** -8
    assert all(bool((dw[e] == 0).all()) for e in range(1, E))
    with pytest.raises(fp8.Fp8Error) as err:
        fp8.fp8_grouped_linear_wgrad_dev(dy8, x8, sdy, sx, doffs, dw, ws[:16])
    assert err.value.status == -5


def test_grouped_forward_argument_validation():
    x8 = torch.zeros((32, 32), dtype=torch.uint8, device="cuda")
    w8 = torch.zeros((2, 16, 32), dtype=torch.uint8, device="cuda")
    s = scalar(1.0)
    y = torch.empty((32, 16), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_grouped_linear_fwd(x8, w8, s, torch.ones(2, device="cuda"), None, y)
    assert e.value.status == -1
    big = torch.zeros((300, 16, 32), dtype=torch.uint8, device="cuda")
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_grouped_linear_fwd(x8, big, s, torch.ones(300, device="cuda"), torch.zeros(301, dtype=torch.int32, device="cuda"), y)
    assert e.value.status == -3
