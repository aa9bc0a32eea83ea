"""Helpers of the GPU parity tests: host arrays <-> device tensors, error metric."""
import numpy as np
import torch

import oracle as o
import paper_2505_20524_b200 as fp8


def dev(a: np.ndarray) -> torch.Tensor:
    """numpy (uint16 BF16 bits / uint8 codes / float32) -> CUDA tensor with the same bytes."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def host(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def bf16_host_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy().astype(np.float64)


def scalar(v=0.0) -> torch.Tensor:
    return torch.full((1,), float(v), dtype=torch.float32, device="cuda")


def gpu_quantize(x_bits: np.ndarray, fmt: int, transpose: bool = False):
    """fp8_quantize through the C ABI; returns device tensors (q, q_t, amax, scale, scale_inv)."""
    x = dev(x_bits)
    q = torch.empty(x.shape, dtype=torch.uint8, device="cuda")
    qt = None
    if transpose:
        rows, cols = x.numel() // x.shape[-1], x.shape[-1]
        qt = torch.empty((cols, rows), dtype=torch.uint8, device="cuda")
    a, s, si = scalar(), scalar(), scalar()
    fp8.fp8_quantize(x, fmt, q, qt, a, s, si)
    return q, qt, a, s, si


def rel_err(got: np.ndarray, ref: np.ndarray, mag: np.ndarray, floor_frac: float = 0.0) -> float:
    """max |got - ref| / mag, mag = the sum of |a||b| over the reduction (componentwise GEMM error).

    floor_frac > 0 floors the denominator at floor_frac * mean(mag).  The attention gradients need it:
    dS = P o (dP - D) cancels to an exact zero on rows whose softmax is one-hot (the oracle's double
    arithmetic gives 0, FP32 gives rounding noise ~1e-7 of the operands), so there mag is 0 and the plain
    ratio would divide noise by zero; the floor turns the check into an absolute one at 1% of the
    tensor's typical magnitude sum."""
    tiny = 1e-30
    den = np.maximum(mag, max(tiny, floor_frac * float(np.mean(mag))))
    return float(np.max(np.abs(got - ref) / den))


BWD_FLOOR = 1e-2
