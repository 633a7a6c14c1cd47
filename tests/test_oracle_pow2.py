"""Pins for the power-of-two scale option of the oracle (an added quantization option; the paper's
rule stays the default).  Checked with exact rational arithmetic and invariants."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

FP8, FP4 = orc.FMT_FP8_E4M3, orc.FMT_FP4_E2M1


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_scale_is_the_largest_power_of_two_that_fits(fmt):
    fmax = Fraction(orc.fpx_max(fmt))
    rng = np.random.default_rng(5)
    bits = np.concatenate([rng.integers(1, 0x7F80, 4000), [0x0001, 0x007F, 0x0080, 0x3F80, 0x7F7F, 0x43E0, 0x40C0]]).astype(np.uint16)
    for b in bits:
        amax = float(orc.bf16_to_float(np.array([b], dtype=np.uint16))[0])
        s = float(orc.tile_scale_pow2(fmt, amax))
        m, e = np.frexp(s)
        assert m == 0.5                                   # a power of two
        ex = int(e) - 1
        a = Fraction(amax)
        if -126 < ex < 127:
            assert a * Fraction(2) ** ex <= fmax < a * Fraction(2) ** (ex + 1)
        elif ex == 127:
            assert a * Fraction(2) ** 127 <= fmax         # clamped from above
    assert orc.tile_scale_pow2(fmt, 0.0) == 1.0
    # never larger than the paper's quotient, and within a factor of two of it
    for amax in (0.013, 1.0, 5.9, 6.0, 6.1, 447.0, 448.0, 449.0, 1e10):
        q = float(orc.tile_scale(fmt, amax)); p = float(orc.tile_scale_pow2(fmt, amax))
        assert q / 2 < p <= q * (1 + 1e-6)


@pytest.mark.parametrize("fmt", [FP8, FP4])
@pytest.mark.parametrize("block", [orc.BLOCK_ROW, orc.BLOCK_COL, orc.BLOCK_BLK])
def test_quantize_with_pow2_scales(fmt, block):
    rng = np.random.default_rng(8)
    x = wl.to_bf16_bits(rng.standard_normal((192, 320)).astype(np.float32) * np.float32(2.5))
    q = orc.quantize(x, fmt, block, pow2_scale=True)
    xf = orc.bf16_to_float(x)
    # products x*S are exact, so codes = RNE of the exact value and dequantization is exact too
    m, _ = np.frexp(q.scales.astype(np.float64))
    assert (m == 0.5).all()
    top = 0x7E if fmt == FP8 else 7
    mask = 0x7F if fmt == FP8 else 7
    assert ((q.codes & mask) <= top).all()
    # no tile saturates beyond FPX_MAX: |x| * S <= FPX_MAX everywhere
    xh = orc.dequantize(q.codes, q.scales, fmt, block)
    assert np.array_equal(xh, q.xhat)
    assert np.abs(q.xhat).max() <= np.abs(xf).max() * (1 + 2.0 ** -3)
    # error bound of RNE with at most half the dynamic range lost: relative to the paper's rule the
    # error sum grows by at most 4x
    q0 = orc.quantize(x, fmt, block)
    assert q.sumsq_err <= 4.0 * q0.sumsq_err + 1e-30 and q.sumsq_err > 0
    assert q.sumsq_x == q0.sumsq_x
    # a tile that the paper's rule already scales by a power of two gives identical results
    tile = np.zeros((1, 128), dtype=np.float32); tile[0, :8] = [6, 3, -1.5, 0.5, 4, -2, 1, 0]
    t = wl.to_bf16_bits(tile * np.float32(2.0 ** -5))
    a, b = orc.quantize(t, fmt, orc.BLOCK_ROW, pow2_scale=True), orc.quantize(t, fmt, orc.BLOCK_ROW)
    if fmt == FP4:
        assert np.array_equal(a.codes, b.codes) and np.array_equal(a.scales, b.scales)


def test_gemm_with_pow2_scales_matches_explicit_sum():
    rng = np.random.default_rng(2)
    x = wl.to_bf16_bits(rng.standard_normal((3, 256)).astype(np.float32))
    w = wl.to_bf16_bits(rng.standard_normal((2, 256)).astype(np.float32) * np.float32(0.02))
    y, qx, qw = orc.linear_fwd(x, w, FP8, FP4, pow2_scale=True)
    for m in range(3):
        for n in range(2):
            acc = 0.0
            for j in range(2):
                part = sum(orc.decode_code(FP8, int(qx.codes[m, k])) * orc.decode_code(FP4, int(qw.codes[n, k])) for k in range(128 * j, 128 * j + 128))
                acc += part / (float(qx.scales[j, m]) * float(qw.scales[0, j]))
            assert y[m, n] == acc                           # power-of-two scaling is exact in binary64
