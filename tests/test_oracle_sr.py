"""Pins of the oracle's stochastic rounding (paper Sec. 6.1: FP4 output gradients are rounded
probabilistically to one of the two nearest values): the generator against published known answers,
the rounding rule against exact rational arithmetic and exhaustive counting, unbiasedness over seeds."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

FP8, FP4 = orc.FMT_FP8_E4M3, orc.FMT_FP4_E2M1
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def magnitudes(fmt):
    """Ascending representable magnitudes with their codes, from the golden value tables' closed form."""
    n = 8 if fmt == FP4 else 127
    return [(orc.decode_code(fmt, m), m) for m in range(n)]


def test_philox_known_answers():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for f in rows:
        w = [int(v, 16) for v in f]
        assert [int(v) for v in orc.philox4x32_10(w[0:4], w[4:6])] == w[6:10]


def test_uniform16_layout_eight_elements_per_counter():
    seed = 0x0123456789ABCDEF
    for blk in (0, 1, 77, 2 ** 32 + 5):
        w = orc.philox4x32_10([blk & 0xFFFFFFFF, blk >> 32, 0, 0], [seed & 0xFFFFFFFF, seed >> 32])
        for j in range(8):
            assert orc.sr_uniform16(seed, 8 * blk + j) == (int(w[j // 2]) >> (16 * (j % 2))) & 0xFFFF


@pytest.mark.parametrize("fmt", [FP4, FP8])
def test_rule_against_exact_rationals(fmt):
    mags = magnitudes(fmt)
    rng = np.random.default_rng(5)
    sign_bit = 8 if fmt == FP4 else 128
    for (vlo, mlo), (vhi, mhi) in zip(mags[:-1], mags[1:]):
        for w in (0.0, 1e-4, 0.25, 0.5, 0.75, 1 - 1e-4):
            t = np.float32(vlo + w * (vhi - vlo))
            if not (vlo <= float(t) < vhi):
                continue
            frac = (Fraction(float(t)) - Fraction(vlo)) / (Fraction(vhi) - Fraction(vlo))
            for u in [0, 1, 32767, 32768, 65535] + [int(v) for v in rng.integers(0, 65536, 6)]:
                up = frac > Fraction(2 * u + 1, 131072)
                assert orc.encode_sr(fmt, t, u) == (mhi if up else mlo)
                assert orc.encode_sr(fmt, -t, u) == sign_bit | (mhi if up else mlo)


@pytest.mark.parametrize("fmt", [FP4, FP8])
def test_representable_values_never_move_and_saturation(fmt):
    mags = magnitudes(fmt)
    sign_bit = 8 if fmt == FP4 else 128
    for v, m in mags:
        for u in (0, 1, 65535):
            assert orc.encode_sr(fmt, v, u) == m
            assert orc.encode_sr(fmt, -v, u) == sign_bit | m       # includes -0 -> signed zero
    top_v, top_m = mags[-1]
    for t in (top_v * (1 + 2 ** -23), top_v * 2, 3e38):
        for u in (0, 65535):
            assert orc.encode_sr(fmt, t, u) == top_m and orc.encode_sr(fmt, -t, u) == sign_bit | top_m


@pytest.mark.parametrize("t", [0.3, 1.2, 2.9, 5.999, 0.0001, 4.0000005])
def test_probability_of_rounding_up_is_the_fraction_fp4(t):
    """Exhaustive over the 65536 uniforms: #up = number of u with (2u+1)/2^17 < frac, a closed form."""
    mags = magnitudes(FP4)
    t32 = float(np.float32(t))
    vlo, mlo = max((v, m) for v, m in mags if v <= t32)
    vhi = min(v for v, _ in mags if v > t32)
    frac = (Fraction(t32) - Fraction(vlo)) / (Fraction(vhi) - Fraction(vlo))
    ups = sum(orc.encode_sr(FP4, t32, u) != mlo for u in range(65536))
    expect = max(0, math.ceil(frac * 65536 - Fraction(1, 2)))
    assert ups == expect
    assert abs(ups / 65536 - float(frac)) <= 2 ** -17 + 1e-12


def test_quantize_sr_scales_neighbours_determinism():
    rng = np.random.default_rng(3)
    x = wl.make_dy(rng, 128, 256)
    q0 = orc.quantize(x, FP4, orc.BLOCK_ROW)
    q1 = orc.quantize(x, FP4, orc.BLOCK_ROW, sr_seed=11)
    q2 = orc.quantize(x, FP4, orc.BLOCK_ROW, sr_seed=11)
    q3 = orc.quantize(x, FP4, orc.BLOCK_ROW, sr_seed=12)
    assert np.array_equal(q0.scales, q1.scales)                    # scales depend on amax only
    assert np.array_equal(q1.codes, q2.codes) and not np.array_equal(q1.codes, q3.codes)
    # every stochastic code is the nearest-even code or its neighbour on the other side of x*S
    xf = orc.bf16_to_float(x)
    s = np.repeat(q1.scales.T, 128, axis=1)[:, :256]
    t = (xf.astype(np.float32) * s.astype(np.float32)).astype(np.float64)
    v1 = np.vectorize(lambda c: orc.decode_code(FP4, int(c)))(q1.codes)
    v0 = np.vectorize(lambda c: orc.decode_code(FP4, int(c)))(q0.codes)
    step = np.where(np.abs(t) < 2, 0.5, np.where(np.abs(t) < 4, 1.0, 2.0))
    assert np.all(np.abs(v1 - t) < step + 1e-12) and np.all(np.abs(v1 - v0) <= step + 1e-12)
    assert q1.sumsq_err >= q0.sumsq_err                             # nearest rounding minimises the error
    # the statistic is the squared distance to the stochastic values
    assert q1.sumsq_err == pytest.approx(float(((xf - q1.xhat) ** 2).sum()), rel=1e-12)


def test_unbiased_over_seeds():
    """E[xhat] = x: mean of the dequantized values over many seeds, against the binomial standard error."""
    rng = np.random.default_rng(8)
    x = wl.to_bf16_bits(rng.uniform(-6, 6, size=(1, 128)).astype(np.float32))
    x[0, 0] = wl.to_bf16_bits(np.array([6.0], dtype=np.float32))[0]    # pins S = 1
    xf = orc.bf16_to_float(x)[0]
    n = 3000
    acc = np.zeros(128)
    for seed in range(n):
        acc += orc.quantize(x, FP4, orc.BLOCK_ROW, sr_seed=1000 + seed).xhat[0]
    mean = acc / n
    step = np.where(np.abs(xf) < 2, 0.5, np.where(np.abs(xf) < 4, 1.0, 2.0))
    sigma = step * 0.5 / math.sqrt(n)                                   # worst case p = 1/2
    assert np.all(np.abs(mean - xf) <= 5 * sigma + 1e-9)
    # nearest rounding is biased on the same data (sanity of the test's power)
    q = orc.quantize(x, FP4, orc.BLOCK_ROW)
    assert np.any(np.abs(q.xhat[0] - xf) > 5 * sigma)
