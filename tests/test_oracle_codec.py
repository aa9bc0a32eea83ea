"""Pins of the oracle's FP8 codec against the format definitions (Section 2: E4M3 / E5M2)."""
import math
import os

import numpy as np
import pytest

import oracle as o

GOLD = os.path.join(os.path.dirname(__file__), "golden")
FMT = {"e4m3": o.E4M3, "e5m2": o.E5M2}


def _finite_codes(fmt):
    t = o.decode_table(fmt)
    return [c for c in range(256) if math.isfinite(t[c])]


def test_decode_anchor_values():
    assert o.decode(0x38, o.E4M3) == 1.0 and o.decode(0x3C, o.E5M2) == 1.0
    assert o.decode(0x7E, o.E4M3) == 448.0 and o.decode(0x7B, o.E5M2) == 57344.0
    assert o.decode(0x08, o.E4M3) == 2.0 ** -6 and o.decode(0x01, o.E4M3) == 2.0 ** -9
    assert o.decode(0x04, o.E5M2) == 2.0 ** -14 and o.decode(0x01, o.E5M2) == 2.0 ** -16
    assert o.decode(0xB8, o.E4M3) == -1.0 and o.decode(0x80, o.E4M3) == 0.0
    assert o.fp8_max(o.E4M3) == 448.0 and o.fp8_max(o.E5M2) == 57344.0


def test_special_code_counts():
    t4, t5 = o.decode_table(o.E4M3), o.decode_table(o.E5M2)
    assert sorted(np.flatnonzero(np.isnan(t4))) == [0x7F, 0xFF]
    assert not np.isinf(t4).any()
    assert sorted(np.flatnonzero(np.isinf(t5))) == [0x7C, 0xFC]
    assert sorted(np.flatnonzero(np.isnan(t5))) == [0x7D, 0x7E, 0x7F, 0xFD, 0xFE, 0xFF]


@pytest.mark.parametrize("fmt", [o.E4M3, o.E5M2])
def test_decode_matches_bitfield_formula(fmt):
    """Independent closed form: value = (-1)^s 2^(E-bias) (1 + M/2^m), subnormals 2^(1-bias) M/2^m."""
    mb, bias = (3, 7) if fmt == o.E4M3 else (2, 15)
    for c in _finite_codes(fmt):
        s, E, M = c >> 7, (c & 0x7F) >> mb, c & ((1 << mb) - 1)
        v = (2.0 ** (1 - bias)) * M / (1 << mb) if E == 0 else (2.0 ** (E - bias)) * (1 + M / (1 << mb))
        assert o.decode(c, fmt) == (-v if s else v)


@pytest.mark.parametrize("fmt", [o.E4M3, o.E5M2])
def test_positive_codes_are_monotone(fmt):
    codes = [c for c in _finite_codes(fmt) if c < 0x80]
    vals = [o.decode(c, fmt) for c in codes]
    assert all(b > a for a, b in zip(vals, vals[1:]))


@pytest.mark.parametrize("fmt", [o.E4M3, o.E5M2])
def test_round_trip_every_finite_code(fmt):
    for c in _finite_codes(fmt):
        assert o.encode(o.decode(c, fmt), fmt) == c


@pytest.mark.parametrize("fmt", [o.E4M3, o.E5M2])
def test_midpoints_tie_to_even_and_neighbours(fmt):
    codes = [c for c in _finite_codes(fmt) if c < 0x80]
    for lo, hi in zip(codes, codes[1:]):
        a, b = o.decode(lo, fmt), o.decode(hi, fmt)
        mid = np.float32((a + b) / 2)          # exact: both have <= 4 significant bits
        assert float(mid) == (a + b) / 2
        even = lo if lo % 2 == 0 else hi
        assert o.encode(mid, fmt) == even
        assert o.encode(np.nextafter(mid, np.float32(0)), fmt) == lo
        assert o.encode(np.nextafter(mid, np.float32(np.inf)), fmt) == hi
        assert o.encode(-mid, fmt) == even | 0x80


def test_worked_values_file():
    n = 0
    for line in open(os.path.join(GOLD, "fp8_worked_values.txt")):
        line = line.split("#")[0].split()
        if not line:
            continue
        fmt, val, code = FMT[line[0]], float(line[1]), int(line[2], 16)
        assert o.encode(np.float32(val), fmt) == code, line
        n += 1
    assert n >= 25


def test_saturation_and_nan():
    for fmt, top in ((o.E4M3, 0x7E), (o.E5M2, 0x7B)):
        assert o.encode(np.float32(3.0e38), fmt) == top
        assert o.encode(np.float32(-3.0e38), fmt) == top | 0x80
        assert o.encode(np.float32(np.inf), fmt) == top
        assert math.isnan(o.decode(o.encode(np.float32(np.nan), fmt), fmt))
    # just above the last rounding boundary that still exists below the maximum
    assert o.encode(np.float32(464.0), o.E4M3) == 0x7E and o.encode(np.float32(432.0), o.E4M3) == 0x7E
    assert o.encode(np.float32(431.9), o.E4M3) == 0x7D
    assert o.encode(np.float32(-0.0), o.E4M3) == 0x80 and o.encode(np.float32(-1e-9), o.E5M2) == 0x80


@pytest.mark.parametrize("fmt", [o.E4M3, o.E5M2])
def test_brute_force_all_bf16_patterns(fmt):
    """Every BF16 bit pattern: encode == nearest finite table entry, ties to the even code, clamp above max."""
    bits = np.arange(65536, dtype=np.uint16)
    vals = o.bf16_to_f32(bits)
    got = o.encode_array(vals, fmt)
    table = o.decode_table(fmt)
    pos = np.array([c for c in range(128) if math.isfinite(table[c])])
    pv = table[pos]                                           # ascending
    finite = np.isfinite(vals)
    a = np.minimum(np.abs(vals[finite].astype(np.float64)), pv[-1])   # clamp above the maximum
    dist = np.abs(a[:, None] - pv[None, :])                   # linear search over the whole table
    best = dist.min(axis=1)
    cand = dist == best[:, None]                              # one or two candidates
    first = cand.argmax(axis=1)
    last = cand.shape[1] - 1 - cand[:, ::-1].argmax(axis=1)
    pick = np.where(pos[first] % 2 == 0, first, last)
    exp = pos[pick] | np.where(np.signbit(vals[finite]), 0x80, 0)
    assert np.array_equal(got[finite], exp.astype(np.uint8))
    inf = np.isinf(vals)
    assert np.array_equal(got[inf] & 0x7F, np.full(inf.sum(), pos[-1], dtype=np.uint8))
    assert np.isnan(table[got[np.isnan(vals)]]).all()
