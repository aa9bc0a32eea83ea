"""Seeded synthetic inputs shaped like the paper's workloads (Appendix A model sizes; Section 5 setups).

This module only *draws inputs*: BF16 tensors as ``uint16`` bit arrays from a counter-based generator
(``synth.c``), with outlier channels / outlier entries injected so that per-tensor scaling is exercised.
It contains none of the method's arithmetic and is the one thing the CUDA path's tests and the CPU
oracle have in common.
"""
from __future__ import annotations

import ctypes as C
import math
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "synth.c")
_LIB = os.path.join(_HERE, "libsynth.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.run(["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"],
                       check=True)
    return _LIB


def _L():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.synth_hash.restype = C.c_uint64
        _lib.synth_hash.argtypes = [C.c_uint64]
        _lib.synth_fill_bf16.restype = None
        _lib.synth_fill_bf16.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_uint64, C.c_uint64, C.c_double,
                                         C.c_void_p, C.c_double, C.c_double, C.c_double]
        _lib.synth_f32_to_bf16.restype = None
        _lib.synth_f32_to_bf16.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
    return _lib


def choose_columns(ncols: int, k: int, seed: int, tid: int) -> np.ndarray:
    """k distinct column indices in [0, ncols): a partial Fisher-Yates shuffle driven by splitmix64."""
    idx = list(range(ncols))
    state = (seed * 1000003 + tid) & 0xFFFFFFFFFFFFFFFF
    for i in range(k):
        state = int(_L().synth_hash(state))
        j = i + state % (ncols - i)
        idx[i], idx[j] = idx[j], idx[i]
    return np.array(sorted(idx[:k]), dtype=np.int64)


def normal_bf16(shape, seed: int, tid: int, std: float, outlier_cols=None, col_factor: float = 1.0,
                elem_prob: float = 0.0, elem_value: float = 0.0) -> np.ndarray:
    """BF16 bits (uint16) of N(0, std) values; the last axis is the column axis for outlier channels."""
    shape = tuple(int(s) for s in shape)
    cols = shape[-1]
    rows = int(np.prod(shape[:-1])) if len(shape) > 1 else 1
    out = np.empty(rows * cols, dtype=np.uint16)
    mask = None
    if outlier_cols is not None and len(outlier_cols):
        mask = np.zeros(cols, dtype=np.uint8)
        mask[np.asarray(outlier_cols)] = 1
    _L().synth_fill_bf16(out.ctypes.data, rows, cols, seed, tid, float(std),
                         None if mask is None else mask.ctypes.data, float(col_factor),
                         float(elem_prob), float(elem_value))
    return out.reshape(shape)


def f32_to_bf16(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    _L().synth_f32_to_bf16(x.ctypes.data, x.size, out.ctypes.data)
    return out


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


# tensor ids (stable: they are part of the recipe)
TID = {"x_qkv": 0, "w_qkv": 1, "x_o": 2, "w_o": 3, "x_up": 4, "w_up": 5, "x_down": 6, "w_down": 7,
       "dy_qkv": 8, "dy_o": 9, "dy_up": 10, "dy_down": 11, "q": 12, "k": 13, "v": 14, "do": 15, "flat": 16}


@dataclass(frozen=True)
class BlockConfig:
    """One transformer block of the workload list (tokens T = batch * seq)."""
    name: str
    seed: int
    batch: int
    seq: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    gated: bool
    act_outlier_frac: float   # fraction of activation channels scaled up
    act_outlier_factor: float
    act_outlier_count: int = 0   # if > 0, overrides the fraction
    qkv_outlier_frac: float = 0.0
    qkv_outlier_factor: float = 1.0
    has_linears: bool = True

    @property
    def tokens(self) -> int:
        return self.batch * self.seq

    def linear_shapes(self):
        """name -> (T, N, K) with Y[T,N] = X[T,K] W[N,K]^T."""
        T, D = self.tokens, self.hidden
        return {
            "qkv": (T, (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim, D),
            "o": (T, D, self.n_q_heads * self.head_dim),
            "up": (T, self.ffn * (2 if self.gated else 1), D),
            "down": (T, D, self.ffn),
        }

    def n_outlier_cols(self, ncols: int, frac=None) -> int:
        if frac is None:
            if self.act_outlier_count:
                return self.act_outlier_count
            frac = self.act_outlier_frac
        return int(math.ceil(frac * ncols)) if frac > 0 else 0


CONFIGS = {
    # tiny single block: 2 of 256 channels x50
    "c1": BlockConfig("c1", 0, 1, 256, 256, 4, 4, 64, 1024, False, 0.0, 50.0, act_outlier_count=2,
                      qkv_outlier_frac=2 / 256, qkv_outlier_factor=50.0),
    # ~1.5B-class block: 0.5% outlier channels x30
    "c3": BlockConfig("c3", 3, 4, 2048, 2048, 16, 16, 128, 5632, True, 0.005, 30.0,
                      qkv_outlier_frac=0.005, qkv_outlier_factor=30.0),
    # ~8B-class block (Appendix A, 8B row: 32 query heads, 8 KV groups, FFN 14336)
    "c4": BlockConfig("c4", 4, 2, 4096, 4096, 32, 8, 128, 14336, True, 0.005, 30.0,
                      qkv_outlier_frac=0.005, qkv_outlier_factor=30.0),
    # long-context attention stress: 1% of head dims x40
    "c5": BlockConfig("c5", 5, 1, 16384, 4096, 32, 32, 128, 0, False, 0.0, 1.0,
                      qkv_outlier_frac=0.01, qkv_outlier_factor=40.0, has_linears=False),
}

W_STD = 0.02
GRAD_STD = 1e-3


def linear_inputs(cfg: BlockConfig, layer: str):
    """(X[T,K], W[N,K], dY[T,N]) as BF16 bits for one projection of the block."""
    T, N, K = cfg.linear_shapes()[layer]
    cols = choose_columns(K, cfg.n_outlier_cols(K), cfg.seed, 100 + TID["x_" + layer])
    x = normal_bf16((T, K), cfg.seed, TID["x_" + layer], 1.0, cols, cfg.act_outlier_factor)
    w = normal_bf16((N, K), cfg.seed, TID["w_" + layer], W_STD)
    dy = normal_bf16((T, N), cfg.seed, TID["dy_" + layer], GRAD_STD)
    return x, w, dy


def attention_inputs(cfg: BlockConfig, seq: int | None = None, batch: int | None = None):
    """(Q[B,N,Hq,d], K[B,N,Hkv,d], V[B,N,Hkv,d], dO[B,N,Hq,d]) as BF16 bits.

    Outlier (head, dim) columns are drawn independently for Q, K and V."""
    B = cfg.batch if batch is None else batch
    N = cfg.seq if seq is None else seq
    out = []
    for name, H in (("q", cfg.n_q_heads), ("k", cfg.n_kv_heads), ("v", cfg.n_kv_heads)):
        ncols = H * cfg.head_dim
        cols = choose_columns(ncols, cfg.n_outlier_cols(ncols, cfg.qkv_outlier_frac), cfg.seed, 100 + TID[name])
        t = normal_bf16((B * N, ncols), cfg.seed, TID[name], 1.0, cols, cfg.qkv_outlier_factor)
        out.append(t.reshape(B, N, H, cfg.head_dim))
    do = normal_bf16((B, N, cfg.n_q_heads, cfg.head_dim), cfg.seed, TID["do"], GRAD_STD)
    return out[0], out[1], out[2], do


FLAT_SIZES = (1 << 20, 1 << 24, 1 << 27, 1 << 29)


def flat_tensor(n: int, seed: int = 2) -> np.ndarray:
    """Quantize-sweep tensor: N(0,1), each entry replaced by +-200 with probability 1e-4."""
    return normal_bf16((n,), seed, TID["flat"], 1.0, None, 1.0, 1e-4, 200.0)
