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


def _hand_matrix(rows, cols):
    """A matrix with hand-chosen power-of-two tile maxima: element (r, c) = 2^-(r % 11) * 2^-(c % 7), so a 1x128
    tile of row r has amax 2^-(r % 11), a 128x1 tile of column c has amax 2^-(c % 7) (every tile holds an index
    with remainder 0 in the other direction) and every 128x128 block has amax 1."""
    r = np.arange(rows)[:, None] % 11
    c = np.arange(cols)[None, :] % 7
    return wl.to_bf16_bits((2.0 ** -(r + c)).astype(np.float32))


def _expected_atom(line_bytes):
    """512-byte atom written out from the sentence in include/snip.h: the byte of tile line r is stored four
    times at byte offsets (r % 32) * 16 + (r / 32) * 4 + {0,1,2,3}; lines beyond the matrix hold 127."""
    atom = bytearray([0]) * 512
    for r in range(128):
        b = line_bytes[r] if r < len(line_bytes) else 127
        off = (r % 32) * 16 + (r // 32) * 4
        for k in range(4):
            atom[off + k] = b
    assert all(v != 0 for v in atom)       # every byte of the atom is covered exactly by the rule
    return bytes(atom)


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_scale_factor_atoms_byte_by_byte(fmt):
    # 192 x 320: the second row tile and the third column tile are 64 wide (their missing lines must read 127)
    rows, cols = 192, 320
    x = _hand_matrix(rows, cols)
    fmax_e = 8 if fmt == FP8 else 2        # largest e with 2^e <= FPX_MAX (448 -> 2^8, 6 -> 2^2)
    tr, tc = 2, 3

    def byte_for(amax_log2):               # S = 2^e, e = fmax_e - amax_log2; the atom holds 127 - e
        return 127 - (fmax_e - amax_log2)

    # ROW tiles (as stored): atom [row tile i][chunk j], line = row inside the tile, amax = 2^-(row % 11)
    q = orc.quantize(x, fmt, orc.BLOCK_ROW, pow2_scale=True)
    got = orc.sf_atoms(q, False).tobytes()
    for i in range(tr):
        for j in range(tc):
            lines = [byte_for(-((128 * i + r) % 11)) for r in range(min(128, rows - 128 * i))]
            assert got[(i * tc + j) * 512:(i * tc + j + 1) * 512] == _expected_atom(lines), ("row", i, j)
    # COL tiles, transposed storage: the operand's rows are the matrix's columns, the contraction runs over the
    # matrix's rows: atom [column tile j][row chunk i], line = column inside the tile, amax = 2^-(col % 7)
    q = orc.quantize(x, fmt, orc.BLOCK_COL, pow2_scale=True)
    got = orc.sf_atoms(q, True).tobytes()
    for j in range(tc):
        for i in range(tr):
            lines = [byte_for(-((128 * j + c) % 7)) for c in range(min(128, cols - 128 * j))]
            assert got[(j * tr + i) * 512:(j * tr + i + 1) * 512] == _expected_atom(lines), ("col", j, i)
    # 128x128 blocks: every line of an atom carries the block's byte (amax of every block here is 1);
    # as stored [i][j], transposed [j][i]; ragged tiles have fewer lines only where the line index is the
    # ragged dimension: for blocks the library fills all 128 lines with the block's byte
    q = orc.quantize(x, fmt, orc.BLOCK_BLK, pow2_scale=True)
    assert (q.scales == np.float32(2.0 ** fmax_e)).all()
    for transposed in (False, True):
        got = orc.sf_atoms(q, transposed).tobytes()
        assert len(got) == tr * tc * 512
        assert got == _expected_atom([byte_for(0)] * 128) * (tr * tc)
    # a block grid with distinct bytes: the transposed order really swaps the tile indices
    y = orc.bf16_to_float(x).astype(np.float32).copy()
    y[:128, 128:256] *= np.float32(0.25)          # block (0, 1) gets amax 2^-2
    q = orc.quantize(wl.to_bf16_bits(y), fmt, orc.BLOCK_BLK, pow2_scale=True)
    plain, swapped = orc.sf_atoms(q, False).tobytes(), orc.sf_atoms(q, True).tobytes()
    special = _expected_atom([byte_for(-2)] * 128)
    assert plain[1 * 512:2 * 512] == special                       # [i=0][j=1] -> index 0*3+1
    assert swapped[(1 * tr + 0) * 512:(1 * tr + 1) * 512] == special   # [j=1][i=0] -> index 1*2+0
    assert plain.count(special) == 1 and swapped.count(special) == 1
