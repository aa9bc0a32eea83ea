"""GPU parity of the fine-grained (blockwise) scaling path: block quantisers bit-exact, GEMM within the GEMM tolerance."""
import numpy as np
import pytest
import torch

import oracle as o
import paper_2505_20524_b200 as fp8
from paper_2505_20524_b200 import synth
from gpu_util import dev, host, rel_err

pytestmark = pytest.mark.gpu


def gpu_quantize_blockwise(xb, block_rows, fmt):
    R, C = xb.shape
    out = torch.empty((R, C), dtype=torch.uint8, device="cuda")
    shape = {1: (C // 128, R), 128: ((R + 127) // 128, C // 128), fp8.FP8_BLOCK_128x1: ((R + 127) // 128, C)}[block_rows]
    si = torch.full(shape, -1.0, dtype=torch.float32, device="cuda")
    fp8.fp8_quantize_blockwise(dev(xb), block_rows, fmt, out, si)
    return out, si


@pytest.mark.parametrize("fmt", [o.E4M3, o.E5M2])
@pytest.mark.parametrize("R,C", [(256, 384), (130, 256), (1000, 1024), (7, 128)])
def test_block_quantisers_bit_exact(fmt, R, C):
    cols = synth.choose_columns(C, 2, 5, 5)
    xb = synth.normal_bf16((R, C), 40, 1, 1.0, cols, 40.0)
    xb[0, :128] = 0                                        # an all-zero block: scale 1
    # 1 x 128
    out, si = gpu_quantize_blockwise(xb, 1, fmt)
    codes, osi = o.quantize_blockwise(xb, 1, 128, fmt)
    assert np.array_equal(host(out), codes)
    assert np.array_equal(host(si).T.view(np.uint32), osi.view(np.uint32))      # GPU layout is [C/128][R]
    # 128 x 128
    out, si = gpu_quantize_blockwise(xb, 128, fmt)
    codes, osi = o.quantize_blockwise(xb, 128, 128, fmt)
    assert np.array_equal(host(out), codes)
    assert np.array_equal(host(si).view(np.uint32), osi.view(np.uint32))
    # 128 x 1
    out, si = gpu_quantize_blockwise(xb, fp8.FP8_BLOCK_128x1, fmt)
    codes, osi = o.quantize_blockwise(xb, 128, 1, fmt)
    assert np.array_equal(host(out), codes)
    assert np.array_equal(host(si).view(np.uint32), osi.view(np.uint32))


@pytest.mark.parametrize("T,N,K", [(256, 256, 256), (400, 384, 640), (1000, 512, 2048), (16, 128, 128), (130, 1024, 256)])
def test_blockwise_dgrad_matches_oracle(T, N, K):
    seed = T + 5 * N + K
    dy = synth.normal_bf16((T, N), seed, 0, 1e-3, synth.choose_columns(N, 2, seed, 2), 30.0)
    w = synth.normal_bf16((N, K), seed, 1, synth.W_STD)
    dy8, sdy = gpu_quantize_blockwise(dy, 1, o.E5M2)
    w8, sw = gpu_quantize_blockwise(w, 128, o.E4M3)
    dx = torch.empty((T, K), dtype=torch.bfloat16, device="cuda")
    fp8.fp8_linear_dgrad_blockwise(dy8, w8, sdy, sw, dx)
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    ody8, osdy = o.quantize_blockwise(dy, 1, 128, o.E5M2)
    ow8, osw = o.quantize_blockwise(w, 128, 128, o.E4M3)
    assert np.array_equal(host(dy8), ody8) and np.array_equal(host(w8), ow8)
    ref, mag = o.linear_dgrad_blockwise(ody8, ow8, osdy, osw)
    err = rel_err(dx.float().cpu().numpy().astype(np.float64), ref, mag)
    assert err <= 2.0 ** -8, err


@pytest.mark.parametrize("T,N,K", [(256, 256, 256), (400, 384, 640), (1000, 512, 2048), (77, 128, 128), (2048, 1024, 256)])
def test_blockwise_wgrad_matches_oracle(T, N, K):
    seed = T + 7 * N + K
    dy = synth.normal_bf16((T, N), seed, 0, 1e-3, synth.choose_columns(N, 2, seed, 2), 30.0)
    x = synth.normal_bf16((T, K), seed, 1, 1.0, synth.choose_columns(K, 3, seed, 1), 50.0)
    dy8, sdy = gpu_quantize_blockwise(dy, fp8.FP8_BLOCK_128x1, o.E5M2)
    x8, sx = gpu_quantize_blockwise(x, fp8.FP8_BLOCK_128x1, o.E4M3)
    dw = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
    fp8.fp8_linear_wgrad_blockwise(dy8, x8, sdy, sx, dw)
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    ody8, osdy = o.quantize_blockwise(dy, 128, 1, o.E5M2)
    ox8, osx = o.quantize_blockwise(x, 128, 1, o.E4M3)
    assert np.array_equal(host(dy8), ody8) and np.array_equal(host(x8), ox8)
    ref, mag = o.linear_wgrad_blockwise(ody8, ox8, osdy, osx)
    err = rel_err(dw.float().cpu().numpy().astype(np.float64), ref, mag)
    assert err <= 2.0 ** -8, err


@pytest.mark.parametrize("T,N,K", [(256, 256, 256), (400, 272, 384), (128, 1040, 1024), (1000, 512, 2048), (16, 16, 128)])
def test_blockwise_gemm_matches_oracle(T, N, K):
    seed = T + 3 * N + K
    cols = synth.choose_columns(K, 3, seed, 1)
    x = synth.normal_bf16((T, K), seed, 0, 1.0, cols, 50.0)
    w = synth.normal_bf16((N, K), seed, 1, synth.W_STD)
    x8, sx = gpu_quantize_blockwise(x, 1, o.E4M3)
    w8, sw = gpu_quantize_blockwise(w, 128, o.E4M3)
    y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    fp8.fp8_linear_fwd_blockwise(x8, w8, sx, sw, y)
    torch.cuda.synchronize()
    assert fp8.fp8_device_status() == 0
    ox8, osx = o.quantize_blockwise(x, 1, 128, o.E4M3)
    ow8, osw = o.quantize_blockwise(w, 128, 128, o.E4M3)
    assert np.array_equal(host(x8), ox8) and np.array_equal(host(w8), ow8)
    ref, mag = o.linear_fwd_blockwise(ox8, ow8, osx, osw)
    got = y.float().cpu().numpy().astype(np.float64)
    err = rel_err(got, ref, mag)
    assert err <= 2.0 ** -8, err                 # FP32 accumulation + one BF16 rounding, as for the tensor-wise product


def test_blockwise_keeps_small_blocks_that_tensorwise_scaling_flushes():
    """The point of the finer recipe: with a x200000 outlier block elsewhere in the tensor, the tensor-wise cast loses
    the ordinary rows, the block-wise cast does not."""
    T, N, K = 256, 256, 512
    x = synth.bf16_to_f32(synth.normal_bf16((T, K), 77, 0, 1.0)).copy()
    x[:16, :128] *= 2.0e5
    xb = synth.f32_to_bf16(x.astype(np.float32))
    w = synth.normal_bf16((N, K), 77, 1, synth.W_STD)
    exact = synth.bf16_to_f32(xb).astype(np.float64) @ synth.bf16_to_f32(w).astype(np.float64).T
    rows = np.arange(64, 256)                                    # rows without the outlier block
    x8, sx = gpu_quantize_blockwise(xb, 1, o.E4M3)
    w8, sw = gpu_quantize_blockwise(w, 128, o.E4M3)
    y = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    fp8.fp8_linear_fwd_blockwise(x8, w8, sx, sw, y)
    yb = y.float().cpu().numpy().astype(np.float64)
    from gpu_util import gpu_quantize
    x8t, _, _, _, sxt = gpu_quantize(xb, o.E4M3, False)
    w8t, _, _, _, swt = gpu_quantize(w, o.E4M3, False)
    y2 = torch.empty((T, N), dtype=torch.bfloat16, device="cuda")
    fp8.fp8_linear_fwd(x8t, w8t, sxt, swt, y2)
    yt = y2.float().cpu().numpy().astype(np.float64)
    e_block = np.abs(yb - exact)[rows].mean() / np.abs(exact[rows]).mean()
    e_tensor = np.abs(yt - exact)[rows].mean() / np.abs(exact[rows]).mean()
    assert e_block < 0.06 and e_tensor > 5 * e_block, (e_block, e_tensor)


def test_blockwise_argument_validation():
    x = dev(synth.normal_bf16((32, 192), 0, 0, 1.0))
    out = torch.empty((32, 192), dtype=torch.uint8, device="cuda")
    si = torch.empty(64, device="cuda")
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_quantize_blockwise(x, 1, 0, out, si)            # 192 % 128 != 0
    assert e.value.status == -3
    x = dev(synth.normal_bf16((32, 128), 0, 0, 1.0))
    out = torch.empty((32, 128), dtype=torch.uint8, device="cuda")
    with pytest.raises(fp8.Fp8Error) as e:
        fp8.fp8_quantize_blockwise(x, 64, 0, out, si)
    assert e.value.status == -4
