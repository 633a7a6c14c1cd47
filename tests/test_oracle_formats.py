"""Pins for the oracle's number formats: decode tables, round-to-nearest-even encode, bf16
rounding.  Everything here is checked against the format definitions (Sec. 2.3 of the paper
names the formats), hand arithmetic or brute force -- never against the CUDA path."""
import math
import os

import numpy as np
import pytest

from oracle import snip_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")
FP8, FP4 = orc.FMT_FP8_E4M3, orc.FMT_FP4_E2M1


def _read_pairs(name):
    out = []
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split()
            out.append((k, float(v)))
    return out


def e4m3_value(code):
    """Independent closed form written out here (not the oracle's routine)."""
    s, e, m = code >> 7, (code >> 3) & 15, code & 7
    v = (m / 8.0) * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7)
    return -v if s else v


def e2m1_value(code):
    s, e, m = (code >> 3) & 1, (code >> 1) & 3, code & 1
    v = m * 0.5 if e == 0 else (1 + m / 2.0) * 2.0 ** (e - 1)
    return -v if s else v


def test_e2m1_table_matches_golden():
    for code, val in _read_pairs("e2m1_values.txt"):
        code = int(code)
        assert orc.decode_code(FP4, code) == val
        assert orc.decode_code(FP4, code | 8) == -val
    pos = sorted({orc.decode_code(FP4, c) for c in range(16) if orc.decode_code(FP4, c) > 0})
    assert pos == [0.5, 1, 1.5, 2, 3, 4, 6]
    assert sum(pos) == 18


def test_e4m3_enumeration_matches_golden_facts():
    facts = dict(_read_pairs("e4m3_facts.txt"))
    finite = [c for c in range(256) if (c & 0x7F) != 0x7F]
    assert len(finite) == facts["finite_codes"]
    vals = [orc.decode_code(FP8, c) for c in finite]
    for c, v in zip(finite, vals):
        assert v == e4m3_value(c)
    pos = sorted({v for v in vals if v > 0})
    assert len(pos) == facts["positive_values"]
    assert max(pos) == facts["max"] == orc.fpx_max(FP8)
    assert min(pos) == facts["min_subnorm"]
    assert sum(pos) == facts["sum_positive"]
    for key, v in facts.items():
        if key.startswith("code_"):
            assert orc.decode_code(FP8, int(key[5:], 16)) == v
    # strictly increasing in the code for positive codes
    assert all(orc.decode_code(FP8, c) < orc.decode_code(FP8, c + 1) for c in range(0x7E))
    assert orc.fpx_max(FP4) == 6.0


def _positive_table(fmt):
    ncodes = 0x7F if fmt == FP8 else 8
    return [(c, orc.decode_code(fmt, c)) for c in range(ncodes)]


def _brute_nearest(fmt, t):
    """Nearest representable magnitude by exhaustive search; ties to the even code;
    values beyond the maximum saturate."""
    tab = _positive_table(fmt)
    a = min(abs(t), tab[-1][1])  # saturation: nothing lies beyond the largest magnitude
    best = None
    for c, v in tab:
        d = abs(a - v)
        if best is None or d < best[0] or (d == best[0] and c % 2 == 0 and best[1] % 2 == 1):
            best = (d, c)
    sign = (0x80 if fmt == FP8 else 0x8) if math.copysign(1.0, t) < 0 else 0
    return best[1] | sign


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_encode_midpoints_go_to_even_and_neighbours_to_nearest(fmt):
    tab = _positive_table(fmt)
    for (c0, v0), (c1, v1) in zip(tab[:-1], tab[1:]):
        mid = (v0 + v1) / 2  # exactly representable in binary32
        even = c0 if c0 % 2 == 0 else c1
        assert orc.encode(fmt, mid) == even, (c0, c1)
        assert orc.encode(fmt, -mid) == even | (0x80 if fmt == FP8 else 8)
        below = np.nextafter(np.float32(mid), np.float32(0))
        above = np.nextafter(np.float32(mid), np.float32(np.inf))
        assert orc.encode(fmt, float(below)) == c0
        assert orc.encode(fmt, float(above)) == c1
        assert orc.encode(fmt, v0) == c0  # representable values are fixed points


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_encode_all_bf16_patterns_against_brute_force(fmt):
    # every finite bf16 value is a legal binary32 input to the encoder
    bits = np.arange(65536, dtype=np.uint16)
    vals = orc.bf16_to_float(bits)
    finite = np.isfinite(vals)
    for b in bits[finite]:
        t = float(vals[b])
        got = orc.encode(fmt, t)
        assert got == _brute_nearest(fmt, t), hex(int(b))
    # monotone: larger input never gives a smaller decoded value
    pos = np.sort(vals[finite & (vals >= 0)])
    dec = [orc.decode_code(fmt, orc.encode(fmt, float(t))) for t in pos]
    assert all(a <= b for a, b in zip(dec[:-1], dec[1:]))


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_encode_saturates_and_keeps_sign_of_zero(fmt):
    mx = orc.fpx_max(fmt)
    top = 0x7E if fmt == FP8 else 7
    sbit = 0x80 if fmt == FP8 else 8
    for t in (mx, mx * (1 + 2.0 ** -23), mx * 1.07, mx * 2, 1e30, 3.0e38):
        assert orc.encode(fmt, t) == top
        assert orc.encode(fmt, -t) == top | sbit
    assert orc.encode(fmt, 0.0) == 0
    assert orc.encode(fmt, -0.0) == sbit
    assert orc.encode(fmt, -1e-30) == sbit      # underflow keeps the sign
    assert orc.encode(fmt, 1e-45) == 0
    # no NaN code is ever produced for FP8
    if fmt == FP8:
        rng = np.random.default_rng(1)
        for t in rng.standard_normal(2000) * 300:
            assert (orc.encode(fmt, float(t)) & 0x7F) != 0x7F


def test_encode_random_float32_against_brute_force():
    rng = np.random.default_rng(7)
    for fmt, span in ((FP8, 500.0), (FP4, 7.0)):
        ts = np.concatenate([rng.uniform(-span, span, 3000), rng.standard_normal(3000) * 0.01])
        for t in ts.astype(np.float32):
            assert orc.encode(fmt, float(t)) == _brute_nearest(fmt, float(t))


def test_bf16_rounding_against_integer_rule():
    # reference rule written independently: add 0x7FFF + lsb to the binary32 word, truncate
    rng = np.random.default_rng(3)
    v = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-30, 30, 20000),
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895e38, 1e-40])])
    f32 = v.astype(np.float32)
    exact32 = f32.astype(np.float64)  # inputs chosen as float32 so one rounding is compared
    u = f32.view(np.uint32)
    want = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
    got = orc.round_to_bf16(exact32)
    assert np.array_equal(got, want)
    # ties: 1 + 2^-8 is halfway between 1 and 1 + 2^-7 -> even (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    assert orc.round_to_bf16(np.array([1 + 2.0 ** -8]))[0] == 0x3F80
    assert orc.round_to_bf16(np.array([1 + 3 * 2.0 ** -8]))[0] == 0x3F82
    # a double just above the tie must round up (double rounding through float32 would not)
    assert orc.round_to_bf16(np.array([1 + 2.0 ** -8 + 2.0 ** -40]))[0] == 0x3F81
    # round trip of every finite bf16 value
    bits = np.arange(65536, dtype=np.uint16)
    vals = orc.bf16_to_float(bits)
    fin = np.isfinite(vals)
    assert np.array_equal(orc.round_to_bf16(vals[fin]), bits[fin])
