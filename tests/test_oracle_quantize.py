"""Pins of amax -> scale -> cast (Appendix C: s(x) = MaxFP8Value/absmax(x); Appendix E: FP8cast(rho X))."""
import os

import numpy as np
import pytest

import oracle as o
from paper_2505_20524_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
FMT = {"e4m3": o.E4M3, "e5m2": o.E5M2}


def bits(f32):
    return int(np.float32(f32).view(np.uint32))


def bf16(vals):
    return synth.f32_to_bf16(np.asarray(vals, dtype=np.float32))


def test_amax_of_sweep_tensor_is_the_injected_outlier():
    x = synth.flat_tensor(1 << 20)
    assert o.amax(x) == np.float32(200.0)
    # independent route: numpy max of |float view|
    assert o.amax(x) == np.abs(synth.bf16_to_f32(x)).max()


def test_amax_invariances():
    x = synth.normal_bf16((4096,), 7, 1, 3.0)
    a = o.amax(x)
    rng = np.random.default_rng(0)
    assert o.amax(rng.permutation(x)) == a
    assert o.amax(x ^ np.uint16(0x8000)) == a
    assert o.amax(bf16([0.0, -0.0])) == 0.0
    assert o.amax(bf16([1.0, -3.5, 2.0])) == np.float32(3.5)


def test_scale_bit_patterns_file():
    for line in open(os.path.join(GOLD, "scale_bits.txt")):
        line = line.split("#")[0].split()
        if not line:
            continue
        s, si = o.scale(float(line[1]), FMT[line[0]])
        assert bits(s) == int(line[2], 16), line
        if line[3] != "-":
            assert bits(si) == int(line[3], 16), line


def test_scale_guards_and_margin():
    assert o.scale(0.0, o.E4M3) == (1.0, 1.0)
    assert o.scale(np.inf, o.E5M2) == (1.0, 1.0)
    assert o.scale(np.nan, o.E5M2) == (1.0, 1.0)
    s, _ = o.scale(np.float32(1e-40), o.E5M2)           # quotient overflows binary32
    assert bits(s) == 0x7F7FFFFF
    s0, _ = o.scale(3.0, o.E4M3, 0)
    s2, _ = o.scale(3.0, o.E4M3, 2)
    assert s2 == s0 / 4                                 # rho = FP8Max / (2^m max H)
    # scale * amax never exceeds the format maximum by more than one rounding
    for a in (0.37, 5.0, 200.0, 1234.5):
        for fmt in (o.E4M3, o.E5M2):
            s, _ = o.scale(a, fmt)
            assert abs(float(s) * a - o.fp8_max(fmt)) <= o.fp8_max(fmt) * 2.0 ** -23


def test_cast_worked_values():
    s4, _ = o.scale(200.0, o.E4M3)
    s5, _ = o.scale(200.0, o.E5M2)
    x = bf16([200.0, -200.0, 1.0, 3.0, 100.0])
    assert list(o.cast(x, s4, o.E4M3)) == [0x7E, 0xFE, 0x41, 0x4D, 0x76]
    assert list(o.cast(bf16([200.0, 1.0]), s5, o.E5M2)) == [0x7B, 0x5C]


def test_cast_equals_elementwise_definition_and_transpose():
    x = synth.normal_bf16((37, 53), 1, 2, 2.0)
    s, _ = o.scale(o.amax(x), o.E4M3)
    q, qt = o.cast(x, s, o.E4M3, transpose=True)
    prod = synth.bf16_to_f32(x) * np.float32(s)         # numpy binary32 multiply
    exp = o.encode_array(prod, o.E4M3)
    assert np.array_equal(q, exp)
    assert np.array_equal(qt, q.T)


def test_cast_idempotent_on_power_of_two_scale():
    x = synth.normal_bf16((2048,), 3, 4, 1.0)
    for fmt in (o.E4M3, o.E5M2):
        q = o.cast(x, 4.0, fmt)
        back = (o.decode_array(q, fmt) * 0.25).astype(np.float32)
        assert np.array_equal(o.cast(bf16(back), 4.0, fmt), q)   # decoded values are exact in BF16


def test_quantize_is_amax_scale_cast():
    x = synth.normal_bf16((64, 128), 9, 9, 1.0, outlier_cols=[5], col_factor=50.0)
    q, a, s, si = o.quantize(x, o.E5M2)
    assert a == o.amax(x) and (s, si) == o.scale(a, o.E5M2)
    assert np.array_equal(q, o.cast(x, s, o.E5M2))
    assert (q & 0x7F).max() == 0x7B                      # the amax element lands on the format maximum


@pytest.mark.parametrize("fmt", [o.E4M3, o.E5M2])
def test_larger_outlier_quantises_the_rest_less_accurately(fmt):
    """Theorem 1 (Appendix C): with a larger outlier the other entries use no more distinct codes and
    their mean absolute quantisation error does not shrink."""
    base = synth.bf16_to_f32(synth.normal_bf16((8192,), 11, 3, 1.0)).copy()
    prev_codes, prev_err = None, None
    for tau in (8.0, 32.0, 128.0, 512.0, 2048.0):
        v = base.copy()
        v[0] = tau
        x = bf16(v)
        q, a, s, si = o.quantize(x, fmt)
        rest = o.decode_array(q[1:], fmt) * float(si)
        err = np.abs(rest - synth.bf16_to_f32(x)[1:]).mean()
        ncodes = len(np.unique(q[1:]))
        if prev_codes is not None:
            assert ncodes <= prev_codes
            assert err >= prev_err * 0.999
        prev_codes, prev_err = ncodes, err


def test_delayed_scaling_history_is_a_fifo_of_the_last_l_amaxes():
    """Appendix E: rho = FP8Max / (2^m max H), H <- {amax} u {h_t}_{t=2..l} (the oldest entry leaves)."""
    l = 5
    hist = np.zeros(l, dtype=np.float32)
    head = 0
    seq = [3.0, 1.0, 7.0, 2.0, 2.0, 1.0, 1.0, 0.5, 0.5, 0.5, 0.25, 0.25]
    for t, a in enumerate(seq):
        head, s, si = o.scale_update(hist, head, a, o.E4M3)
        window = seq[max(0, t + 1 - l):t + 1]                     # the last l values, independent bookkeeping
        es, esi = o.scale(np.float32(max(window)), o.E4M3)
        assert (s, si) == (es, esi), (t, window)
        assert sorted(hist[hist > 0].tolist()) == sorted(window)
        assert head == (t + 1) % l
    # 7.0 dominated from step 2 until it left the window at step 7
    assert o.scale_update(np.zeros(4, dtype=np.float32), 0, 0.0, o.E5M2)[1:] == (1.0, 1.0)   # empty history
    h2 = np.zeros(3, dtype=np.float32)
    _, s2, _ = o.scale_update(h2, 0, 2.0, o.E5M2, margin=1)
    assert s2 == np.float32(57344.0 / 2.0 / 2.0)
