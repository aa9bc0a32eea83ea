"""CPU-side checks: the C-ABI library loads and exports every declared symbol, host-side accounting, recipes."""
import ctypes as C
import json
import os
import re
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "fp8dpa.h")).read()
    return re.findall(r"FP8_API\s+[\w\s\*]+?\b(fp8_\w+)\s*\(", text)


def test_library_exports_every_declared_symbol():
    from paper_2505_20524_b200 import binding, build
    build.build()
    lib = C.CDLL(binding.LIB_PATH)
    names = declared_symbols()
    assert len(names) >= 13 and len(set(names)) == len(names)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(names) == sorted(binding.SYMBOLS)
    lib.fp8_last_error.restype = C.c_char_p
    assert isinstance(lib.fp8_last_error(), bytes)


def test_binding_mirrors_header_constants():
    from paper_2505_20524_b200 import binding
    text = open(os.path.join(ROOT, "include", "fp8dpa.h")).read()
    for name, val in re.findall(r"(FP8_(?:OK|ERR_\w+))\s*=\s*(-?\d+)", text):
        assert binding.STATUS_NAMES[int(val)] == name
    assert "FP8_E4M3 = 0" in text and "FP8_E5M2 = 1" in text and binding.E4M3 == 0 and binding.E5M2 == 1
    assert C.sizeof(binding.AttnScales) == 64          # 4 pointers, 2 floats, 2 pointers, 1 float (+ padding)
    m = re.search(r"FP8_STATIC_SCRATCH_BYTES\s*\((\d+)u\s*<<\s*(\d+)\)", text)
    assert int(m.group(1)) << int(m.group(2)) == binding.STATIC_SCRATCH_BYTES


def test_binding_structures_have_the_header_layout(tmp_path):
    """The ctypes structures that cross the boundary by pointer match the C compiler's layout of the header's structs:
    size and the offset of every field, from a program compiled against include/fp8dpa.h."""
    from paper_2505_20524_b200 import binding
    pairs = {"fp8_quant_item": binding.QuantItem, "fp8_delayed_item": binding.DelayedItem,
             "fp8_attn_scales": binding.AttnScales}
    text = open(os.path.join(ROOT, "include", "fp8dpa.h")).read()
    lines = ["#include <stdio.h>", "#include <stddef.h>", '#include "fp8dpa.h"', "int main(void) {"]
    for cname, st in pairs.items():
        body = re.search(r"typedef struct \{([^{}]*)\}\s*" + cname + r"\s*;", text, re.S).group(1)
        body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
        fields = [re.findall(r"\w+", part)[-1] for d in body.split(";") if d.strip() for part in d.split(",")]
        assert fields == [f[0] for f in st._fields_], (cname, fields)         # same names in the same order
        lines.append(f'printf("{cname} %zu", sizeof({cname}));')
        lines += [f'printf(" %zu", offsetof({cname}, {f}));' for f in fields]
        lines.append('printf("\\n");')
    lines.append("return 0; }")
    src = tmp_path / "layout.c"
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split("\n")
    for line in filter(None, out):
        name, size, *offs = line.split()
        st = pairs[name]
        assert C.sizeof(st) == int(size), name
        assert [getattr(st, f[0]).offset for f in st._fields_] == [int(v) for v in offs], name


def test_workspace_size_is_host_only_arithmetic():
    from paper_2505_20524_b200 import binding
    n = binding.fp8_attention_workspace_bytes(1, 2, 4096, 32, 8, 128)
    assert n >= 2 * 4096 * 32 * 128 * 4 + 2 * 32 * 4096 * 4 and n % 256 == 0
    assert binding.fp8_attention_workspace_bytes(0, 2, 4096, 32, 8, 128) == 0


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    from paper_2505_20524_b200 import binding
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    monkeypatch.setattr(binding, "_lib", None)
    with pytest.raises(RuntimeError):
        binding.load()


def test_generator_is_deterministic_and_shaped():
    from paper_2505_20524_b200 import synth
    a = synth.normal_bf16((64, 48), 3, 7, 1.0, [5, 9], 30.0)
    b = synth.normal_bf16((64, 48), 3, 7, 1.0, [5, 9], 30.0)
    assert np.array_equal(a, b) and a.dtype == np.uint16 and a.shape == (64, 48)
    f = synth.bf16_to_f32(a)
    assert f[:, 5].std() > 10 * f[:, 6].std()
    assert not np.array_equal(a, synth.normal_bf16((64, 48), 4, 7, 1.0, [5, 9], 30.0))
    cols = synth.choose_columns(4096, 21, 4, 100)
    assert len(set(cols.tolist())) == 21 and cols.min() >= 0 and cols.max() < 4096
    x = synth.flat_tensor(1 << 20)
    frac = (np.abs(synth.bf16_to_f32(x)) == 200).mean()
    assert 0.5e-4 < frac < 2e-4


def test_workload_shapes_and_flop_accounting():
    from paper_2505_20524_b200 import synth
    from paper_2505_20524_b200.hotpath import BlockHotPath
    c4 = synth.CONFIGS["c4"]
    sh = c4.linear_shapes()
    assert sh["qkv"] == (8192, 6144, 4096) and sh["up"] == (8192, 28672, 4096) and sh["down"] == (8192, 4096, 14336)
    fwd = sum(2.0 * t * n * k for t, n, k in sh.values())
    assert abs(fwd / 1e9 - 3573.4) < 0.1                      # forward GEMM FLOPs of the 8B-class block
    hp = BlockHotPath(c4, "cpu")
    hp.B, hp.N = c4.batch, c4.seq
    hp.attn = {}                                              # accounting only
    assert abs(hp.attention_flops() / 1e9 - 962.1) < 0.1
    assert c4.n_outlier_cols(4096) == 21 and c4.n_outlier_cols(14336) == 72
    c3 = synth.CONFIGS["c3"]
    assert sum(2.0 * t * n * k for t, n, k in c3.linear_shapes().values()) / 1e9 == pytest.approx(841.8, abs=0.1)


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--config", "c1"], capture_output=True, text=True, check=True)
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "TFLOP/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["higher_is_better"] is True


def test_bench_refuses_to_run_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "1"], capture_output=True,
                         text=True)
    assert out.returncode != 0 and "CUDA" in (out.stderr + out.stdout)
