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


def rel_err(got: np.ndarray, ref: np.ndarray, mag: np.ndarray, slack=None, floor_frac: float = 0.0) -> float:
    """max (|got - ref| - slack)+ / mag: componentwise error against the oracle's magnitude sums.

    mag: for GEMMs and the attention output, the sum of |a||b| over the reduction; for dQ and dK it is built
    from P(|dP| + |D|), the size of dS before dP - D cancels (an FP32 evaluation of that difference is only
    accurate relative to the two numbers being subtracted).
    slack: the oracle's bound on how far an output may move because a value that is re-quantised to FP8
    inside the kernel (P~, dS) lies within FP32 rounding noise of a tie between two codes; there both codes
    are correct results, and the jump between them (6-25% of that term) is not an error.
    floor_frac floors the denominator at floor_frac * mean(mag) so an output with all-zero operands cannot
    divide by zero."""
    tiny = 1e-30
    den = np.maximum(mag, max(tiny, floor_frac * float(np.mean(mag))))
    diff = np.abs(got - ref)
    if slack is not None:
        diff = np.maximum(diff - slack, 0.0)
    return float(np.max(diff / den))


BWD_FLOOR = 1e-6
# relative uncertainty of the kernel's FP32 evaluation of a length-128 dot product and an exp2:
# measured tcgen05 accumulation error is 2^-22 of the magnitude sum at K = 128; 8x margin
FLIP_EPS = 2.0 ** -19


def quantile_err(got, ref, mag, slack=None, q=0.999, floor_frac=0.0):
    """(q-quantile, maximum) of (|got - ref| - slack)+ / mag over all elements."""
    den = np.maximum(mag, max(1e-30, floor_frac * float(np.mean(mag))))
    diff = np.abs(got - ref)
    if slack is not None:
        diff = np.maximum(diff - slack, 0.0)
    e = (diff / den).ravel()
    return float(np.quantile(e, q)), float(e.max())


def norm_ratios(got, ref):
    """(Frobenius, max-norm) ratios ||got - ref|| / ||ref||."""
    d = got - ref
    return (float(np.linalg.norm(d.ravel()) / max(np.linalg.norm(ref.ravel()), 1e-300)),
            float(np.abs(d).max() / max(np.abs(ref).max(), 1e-300)))


def report(case: str, **metrics):
    """Print one line of parity figures (pytest -s shows it) and, when FP8DPA_PARITY_REPORT names a file, append
    it there as JSON so that the figures quoted in the design notes can be regenerated."""
    import json
    import os
    line = json.dumps({"case": case, **{k: (float("%.4g" % v) if isinstance(v, float) else v)
                                        for k, v in metrics.items()}})
    print("parity:", line)
    path = os.environ.get("FP8DPA_PARITY_REPORT")
    if path:
        with open(path, "a") as f:
            f.write(line + "\n")


# Frobenius-norm gates (||gpu - oracle||_F / ||oracle||_F).  O and the gradients are BF16 (2^-9 relative per element)
# and inherit the re-quantisation ties of P8 / dS8 on a small share of the terms.
FRO_FWD = 5e-3
FRO_BWD = 5e-3
