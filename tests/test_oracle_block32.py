"""Pins for the 32-long tile kinds of the oracle (1x32 / 32x1 tiles with power-of-two scales: an added
quantization option next to the paper's 1x128 / 128x128 tiles, Sec. 2.3 / 3.2).  Every expectation here is
worked out without the routine under test: exact rational arithmetic per tile, a brute-force nearest-code search,
reductions to tile kinds that are pinned elsewhere, and invariants that follow from the definitions."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

FP8, FP4 = orc.FMT_FP8_E4M3, orc.FMT_FP4_E2M1
ROW32, COL32 = orc.BLOCK_ROW32, orc.BLOCK_COL32


def bits(rng, rows, cols, spread=3.0):
    # magnitudes that differ from tile to tile, so that neighbouring tiles get different scales
    x = rng.standard_normal((rows, cols)) * np.exp(spread * rng.standard_normal((rows, (cols + 31) // 32))).repeat(32, axis=1)[:, :cols]
    return wl.to_bf16_bits(x.astype(np.float32))


def expected_scale(fmt, amax):
    """Largest 2^e with amax * 2^e <= FPX_MAX, e clamped to [-126, 127]; 1 for an empty tile (exact arithmetic)."""
    if amax == 0.0:
        return 1.0
    fmax, a = Fraction(orc.fpx_max(fmt)), Fraction(float(amax))
    e = 127
    while e > -126 and a * Fraction(2) ** e > fmax:
        e -= 1
    return float(Fraction(2) ** e)


def nearest_code(fmt, t):
    """Brute force: the code whose value is nearest to t, ties to the even code, magnitudes beyond FPX_MAX saturate."""
    n = 256 if fmt == FP8 else 16
    top = orc.fpx_max(fmt)
    best, bd = None, None
    for code in range(n):
        v = orc.decode_code(fmt, code)
        if not np.isfinite(v) or abs(v) > top:
            continue
        if (v < 0) != (np.signbit(t)) and v != 0:
            continue
        if v == 0 and (code != 0) != bool(np.signbit(t)):
            continue
        d = abs(Fraction(float(v)) - Fraction(float(np.clip(t, -top, top))))
        if bd is None or d < bd or (d == bd and code % 2 == 0):
            best, bd = code, d
    return best


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_row32_tile_by_tile_against_exact_arithmetic(fmt):
    rng = np.random.default_rng(11)
    rows, cols = 9, 160    # five tiles per row
    x = bits(rng, rows, cols)
    x[3, 64:96] = 0        # an empty tile
    q = orc.quantize(x, fmt, ROW32, True)
    xf = orc.bf16_to_float(x).astype(np.float64)
    assert q.scales.shape == (5, rows)
    err = 0.0
    for r in range(rows):
        for j in range(5):
            seg = xf[r, 32 * j:32 * j + 32]
            s = expected_scale(fmt, np.abs(seg).max())
            assert float(q.scales[j, r]) == s, (r, j)
            for k, v in enumerate(seg):
                t = np.float32(v) * np.float32(s)       # exact: a power of two
                code = nearest_code(fmt, float(t))
                assert int(q.codes[r, 32 * j + k]) == code, (r, j, k)
                xh = orc.decode_code(fmt, code) / s
                assert q.xhat[r, 32 * j + k] == xh
                err += (v - xh) ** 2
    assert abs(q.sumsq_err - err) <= 1e-12 * max(err, 1e-300)


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_col32_is_row32_of_the_transpose_and_row32_is_row_of_a_reshape(fmt):
    rng = np.random.default_rng(12)
    x = bits(rng, 96, 160)
    qc = orc.quantize(x, fmt, COL32, True)
    qr = orc.quantize(np.ascontiguousarray(x.T), fmt, ROW32, True)
    assert np.array_equal(qc.codes, qr.codes.T)
    assert np.array_equal(qc.xhat, qr.xhat.T)
    assert qc.scales.shape == (3, 160) and qr.scales.shape == (3, 160)
    assert np.array_equal(qc.scales, qr.scales)          # scales[tile along the rows of x][column of x] in both
    assert qc.sumsq_err == pytest.approx(qr.sumsq_err, rel=1e-12)
    # every 1x32 tile is a whole (ragged) 1x128 tile of the matrix reshaped to 32 columns
    qa = orc.quantize(x, fmt, ROW32, True)
    qb = orc.quantize(np.ascontiguousarray(x.reshape(-1, 32)), fmt, orc.BLOCK_ROW, True)
    assert np.array_equal(qa.codes.reshape(-1, 32), qb.codes)
    assert np.array_equal(qa.scales.T.reshape(-1), qb.scales.reshape(-1))   # qa: [tile][row] -> (row, tile) order of the reshape


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_finer_tiles_never_increase_an_element_error(fmt):
    # inside a 1x32 tile the scale is a power-of-two multiple of the 1x128 tile's, so every value the coarse grid offers
    # in the tile's range is also on the fine grid: |x - xhat| cannot grow for any element
    rng = np.random.default_rng(13)
    x = bits(rng, 64, 384)
    xf = orc.bf16_to_float(x).astype(np.float64)
    fine, coarse = orc.quantize(x, fmt, ROW32, True), orc.quantize(x, fmt, orc.BLOCK_ROW, True)
    assert (np.abs(xf - fine.xhat) <= np.abs(xf - coarse.xhat)).all()
    assert fine.sumsq_err < coarse.sumsq_err
    assert (fine.scales.reshape(3, 4, 64) >= coarse.scales[:, None, :]).all()
    finec, coarsec = orc.quantize(x, fmt, COL32, True), orc.quantize(x, fmt, orc.BLOCK_COL, True)
    assert (np.abs(xf - finec.xhat) <= np.abs(xf - coarsec.xhat)).all()


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_lossless_tiles_and_ragged_tail(fmt):
    grid = np.array([orc.decode_code(fmt, c) for c in range(8)], dtype=np.float64)   # small non-negative values of the format
    rows, cols = 5, 80    # two whole tiles and a 16-wide tail per row
    x = np.zeros((rows, cols))
    rng = np.random.default_rng(14)
    for r in range(rows):
        for j in range(3):
            w = min(32, cols - 32 * j)
            seg = rng.choice(grid, w) * rng.choice([-1.0, 1.0], w)
            seg[0] = orc.fpx_max(fmt)                    # the tile's maximum is FPX_MAX * 2^-(r+j): S = 2^(r+j) exactly
            x[r, 32 * j:32 * j + w] = seg * 2.0 ** -(r + j)
    xb = wl.to_bf16_bits(x.astype(np.float32))
    assert np.array_equal(orc.bf16_to_float(xb).astype(np.float64), x)   # representable in bf16
    q = orc.quantize(xb, fmt, ROW32, True)
    assert q.sumsq_err == 0.0 and np.array_equal(q.xhat, x)
    for r in range(rows):
        for j in range(3):
            assert float(q.scales[j, r]) == 2.0 ** (r + j)


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_scale_factor_atoms_of_32_long_tiles_byte_by_byte(fmt):
    # tile (line l, 32-block b) is given the maximum FPX_MAX * 2^-((l + 3 b) % 11): S = 2^n with n = (l + 3 b) % 11 and the
    # byte, which encodes 1/S in UE8M0, must be 127 - n
    fmax = orc.fpx_max(fmt)
    rows, cols = 192, 320    # 2 x 3 atoms as stored, the last ones ragged (64 lines; 64 of 128 contraction elements)
    x = np.zeros((rows, cols))
    for r in range(rows):
        for b in range(cols // 32):
            x[r, 32 * b] = fmax * 2.0 ** -((r + 3 * b) % 11)
    xb = wl.to_bf16_bits(x.astype(np.float32))
    q = orc.quantize(xb, fmt, ROW32, True)
    atoms = orc.sf_atoms(q, False).reshape(2, 3, 512)
    for i in range(2):
        for j in range(3):
            for line in range(128):
                for k in range(4):
                    got = int(atoms[i, j, (line % 32) * 16 + (line // 32) * 4 + k])
                    r, b = 128 * i + line, 4 * j + k
                    want = 127 - (r + 3 * b) % 11 if (r < rows and b < cols // 32) else 127
                    assert got == want, (i, j, line, k)
    # the transposed operand: lines are columns of x, chunks run along its rows
    qt = orc.quantize(np.ascontiguousarray(xb.T), fmt, COL32, True)     # [320, 192], 32x1 tiles along its rows
    at = orc.sf_atoms(qt, True).reshape(2, 3, 512)                       # [line tile (192 columns)][chunk (320 rows)]
    assert np.array_equal(at, atoms)


def test_gemms_with_32_long_tiles_match_an_explicit_sum():
    rng = np.random.default_rng(15)
    M, K, N = 96, 160, 64
    x, w, dy = bits(rng, M, K, 1.0), bits(rng, N, K, 1.0), bits(rng, M, N, 1.0)
    y, qx, qw = orc.linear_fwd(x, w, FP4, FP8, pow2_scale=2)
    assert qx.block == ROW32 and qw.block == ROW32
    want = np.zeros((M, N))
    vx = np.vectorize(lambda c: orc.decode_code(FP4, int(c)))(qx.codes)
    vw = np.vectorize(lambda c: orc.decode_code(FP8, int(c)))(qw.codes)
    for b in range(K // 32):      # per 32-long tile of the contraction: code products, then both scales removed
        part = vx[:, 32 * b:32 * b + 32] @ vw[:, 32 * b:32 * b + 32].T
        want += part / (qx.scales[b].astype(np.float64)[:, None] * qw.scales[b].astype(np.float64)[None, :])
    assert np.allclose(y, want, rtol=1e-12, atol=0)
    dx, qdy, qw2 = orc.linear_dgrad(dy, w, FP8, FP4, pow2_scale=2)
    assert qdy.block == ROW32 and qw2.block == COL32
    assert np.allclose(dx, qdy.xhat @ qw2.xhat, rtol=1e-12, atol=0)
    dw, qdy2, qx2 = orc.linear_wgrad(dy, x, FP4, FP4, pow2_scale=2)
    assert qdy2.block == COL32 and qx2.block == COL32
    assert np.allclose(dw, qdy2.xhat.T @ qx2.xhat, rtol=1e-12, atol=0)
