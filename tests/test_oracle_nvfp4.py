"""Pins for the two-level (NVFP4-style) option of the oracle: E2M1 codes in 16-long tiles, one E4M3 scale byte per tile, one
binary32 factor per tensor (an added quantization option, Sec. 3.2; the rule itself is this library's and is written out in
the oracle's header).  Expectations are rebuilt here from the rule with numpy binary32 steps and brute-force nearest searches
over the formats' value tables, or follow from invariants; nothing calls the routine under test to produce them."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

FP8, FP4 = orc.FMT_FP8_E4M3, orc.FMT_FP4_E2M1
f32 = np.float32


def nearest(fmt, t, ncodes, top):
    """Code of the non-negative value nearest to |t| (ties to the even code, saturating at top), sign bit from t."""
    a = min(abs(float(t)), top)
    best, bd = 0, None
    for code in range(ncodes):
        v = orc.decode_code(fmt, code)
        if not np.isfinite(v) or v < 0 or v > top:
            continue
        d = abs(Fraction(float(v)) - Fraction(a))
        if bd is None or d < bd or (d == bd and code % 2 == 0):
            best, bd = code, d
    return best | ((ncodes) if np.signbit(t) else 0)


def rebuild(xf, tensor_amax):
    """The rule, step by step, for a [lines, 16 * k] float array with tiles along the columns."""
    enc = f32(1.0) if tensor_amax == 0 else f32(2688.0) / f32(tensor_amax)
    rows, cols = xf.shape
    codes = np.zeros((rows, cols), dtype=np.uint8)
    sf = np.zeros((cols // 16, rows), dtype=np.uint8)
    xhat = np.zeros((rows, cols))
    for r in range(rows):
        for j in range(cols // 16):
            seg = xf[r, 16 * j:16 * j + 16].astype(f32)
            d = (np.abs(seg).max() / f32(6.0)) * enc              # two binary32 roundings
            s = nearest(FP8, d, 128, 448.0)
            sf[j, r] = s
            sv = orc.decode_code(FP8, s)
            for k, v in enumerate(seg):
                if sv == 0.0:
                    code = 8 if np.signbit(v) else 0
                else:
                    E = enc / f32(sv)
                    code = nearest(FP4, v * E, 8, 6.0)
                codes[r, 16 * j + k] = code
                xhat[r, 16 * j + k] = orc.decode_code(FP4, code) * sv / float(enc)
    return codes, sf, enc, xhat


def data(rng, rows, cols, scale):
    x = rng.standard_normal((rows, cols)) * np.exp(1.5 * rng.standard_normal((rows, cols // 16))).repeat(16, axis=1) * scale
    return wl.to_bf16_bits(x.astype(np.float32))


@pytest.mark.parametrize("scale", [1.0, 1e-3, 300.0])
def test_tile_by_tile_against_the_rule_written_out(scale):
    rng = np.random.default_rng(31)
    x = data(rng, 7, 96, scale)
    x[2, 32:48] = 0                      # an empty tile
    xf = orc.bf16_to_float(x).astype(np.float64)
    q = orc.quantize_nvfp4(x)
    codes, sf, enc, xhat = rebuild(xf, np.abs(xf).max())
    assert q.enc == enc
    assert np.array_equal(q.sf, sf)
    assert np.array_equal(q.codes, codes)
    assert np.array_equal(q.xhat, xhat)
    assert q.sumsq_err == pytest.approx(((xf - xhat) ** 2).sum(), rel=1e-12)
    assert q.sumsq_x == pytest.approx((xf ** 2).sum(), rel=1e-12)
    assert (q.sf[:, 2][2] == 0) and (q.codes[2, 32:48] & 7 == 0).all()


def test_column_tiles_are_row_tiles_of_the_transpose():
    rng = np.random.default_rng(32)
    x = data(rng, 48, 64, 0.02)
    qc = orc.quantize_nvfp4(x, col_tiles=True)
    qr = orc.quantize_nvfp4(np.ascontiguousarray(x.T), col_tiles=False)
    assert np.array_equal(qc.codes, qr.codes.T) and np.array_equal(qc.sf, qr.sf) and qc.enc == qr.enc
    assert np.array_equal(qc.xhat, qr.xhat.T)


def test_powers_of_two_pass_through_and_a_given_bound_is_used():
    rng = np.random.default_rng(33)
    x = data(rng, 16, 64, 1.0)
    xf = orc.bf16_to_float(x)
    q = orc.quantize_nvfp4(x)
    for k in (-9, 5):
        xs = wl.to_bf16_bits((xf * f32(2.0 ** k)).astype(np.float32))
        qs = orc.quantize_nvfp4(xs)
        assert np.array_equal(qs.codes, q.codes) and np.array_equal(qs.sf, q.sf)
        assert np.array_equal(qs.xhat, q.xhat * 2.0 ** k)
    # a caller-supplied bound twice the true maximum: every scale byte drops by one binade, codes unchanged
    amax = float(np.abs(xf).max())
    q2 = orc.quantize_nvfp4(x, tensor_amax=2 * amax)
    assert np.array_equal(q2.codes, q.codes)
    v = np.vectorize(lambda c: orc.decode_code(FP8, int(c)))
    normal = v(q.sf) >= 2.0 ** -5           # halving keeps the significand only for normal values
    assert np.array_equal(v(q2.sf)[normal], v(q.sf)[normal] / 2)


def test_lossless_tiles_and_bounds():
    # tensor maximum 2688 * 2^-3 -> enc = 8; a tile with maximum 6 * sv / 8 and values on the E2M1 grid times sv / 8
    grid = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6])
    rng = np.random.default_rng(34)
    rows, cols = 6, 64
    x = np.zeros((rows, cols))
    svs = [2.0 ** e for e in (-6, -2, 0, 3)]        # power-of-two scale values: enc / sv is exact
    for r in range(rows):
        for j in range(4):
            seg = rng.choice(grid, 16) * rng.choice([-1.0, 1.0], 16)
            seg[0] = 6.0
            x[r, 16 * j:16 * j + 16] = seg * svs[j] / 8.0
    x[0, 0] = 2688.0 / 8.0                            # the tensor's maximum (a tile maximum of 6 * 448 / 8)
    x[0, 1:16] = 0
    xb = wl.to_bf16_bits(x.astype(np.float32))
    assert np.array_equal(orc.bf16_to_float(xb).astype(np.float64), x)
    q = orc.quantize_nvfp4(xb)
    assert float(q.enc) == 8.0 and q.sumsq_err == 0.0 and np.array_equal(q.xhat, x)
    assert int(q.sf[0, 0]) == 0x7E                    # 448
    # general data: the error of an element is at most half the widest grid step plus what the rounding of the scale byte clips
    x2 = data(rng, 32, 128, 0.05)
    q2 = orc.quantize_nvfp4(x2)
    xf = orc.bf16_to_float(x2).astype(np.float64)
    v = np.vectorize(lambda c: orc.decode_code(FP8, int(c)))
    sv = v(q2.sf).T.repeat(16, axis=1)               # [rows, cols]
    unit = sv / float(q2.enc)
    assert (np.abs(xf - q2.xhat) <= unit * (1.0 + 6.0 / 16.0) + 1e-300).all()
    assert (np.abs(q2.xhat) <= 6.0 * unit * (1 + 1e-12)).all()
    assert q2.sumsq_err / q2.sumsq_x < 0.02           # finer tiles than the paper's 1x128 FP4 tiles: a smaller error
    assert q2.sumsq_err < orc.quantize(x2, FP4, orc.BLOCK_ROW).sumsq_err


def test_zero_tensor_and_argument_checks():
    z = np.zeros((4, 32), dtype=np.uint16)
    q = orc.quantize_nvfp4(z)
    assert float(q.enc) == 1.0 and not q.codes.any() and not q.sf.any() and q.sumsq_err == 0.0
    with pytest.raises(ValueError):
        orc.quantize_nvfp4(z, tensor_amax=-1.0)


def test_atoms_byte_by_byte():
    # every 16-long tile gets a different maximum, so every scale byte is different from its neighbours
    rows, cols = 192, 320          # 2 line tiles (the second ragged), 3 chunks (the last with 4 of its 8 tiles)
    x = np.zeros((rows, cols))
    for r in range(rows):
        for t in range(cols // 16):
            x[r, 16 * t] = 2.0 ** -((r + 5 * t) % 9) * (1.0 + 0.25 * ((r + t) % 4))
    xb = wl.to_bf16_bits(x.astype(np.float32))
    q = orc.quantize_nvfp4(xb)
    atoms = orc.nvfp4_atoms(q, False).reshape(2, 3, 2, 512)
    assert len(np.unique(q.sf)) > 20
    for i in range(2):
        for j in range(3):
            for half in range(2):
                for line in range(128):
                    for k in range(4):
                        r, t = 128 * i + line, 8 * j + 4 * half + k
                        want = int(q.sf[t, r]) if (r < rows and t < cols // 16) else 0
                        assert int(atoms[i, j, half, (line % 32) * 16 + (line // 32) * 4 + k]) == want
    qt = orc.quantize_nvfp4(np.ascontiguousarray(xb.T), col_tiles=True)
    assert np.array_equal(orc.nvfp4_atoms(qt, True), atoms.reshape(-1))


def test_gemms_match_explicit_sums_over_tiles():
    rng = np.random.default_rng(35)
    M, K, N = 48, 64, 32
    x, w, dy = data(rng, M, K, 1.0), data(rng, N, K, 0.02), data(rng, M, N, 1e-3)
    val4 = np.vectorize(lambda c: orc.decode_code(FP4, int(c)))
    val8 = np.vectorize(lambda c: orc.decode_code(FP8, int(c)))
    y, qx, qw = orc.linear_nvfp4("fwd", x, w)
    want = np.zeros((M, N))
    for t in range(K // 16):      # per tile of the contraction: code products times both scale bytes; both tensor factors at the end
        part = val4(qx.codes[:, 16 * t:16 * t + 16]) @ val4(qw.codes[:, 16 * t:16 * t + 16]).T
        want += part * val8(qx.sf[t])[:, None] * val8(qw.sf[t])[None, :]
    want /= float(qx.enc) * float(qw.enc)
    assert np.abs(y - want).max() <= 1e-12 * np.abs(want).max()
    dx, qdy, qwc = orc.linear_nvfp4("dgrad", dy, w)
    assert not qdy.col_tiles and qwc.col_tiles
    ref = qdy.xhat @ qwc.xhat
    assert np.abs(dx - ref).max() <= 1e-12 * np.abs(ref).max()      # sums of both signs: relative to the largest entry
    dw, qdyc, qxc = orc.linear_nvfp4("wgrad", dy, x)
    assert qdyc.col_tiles and qxc.col_tiles
    ref = qdyc.xhat.T @ qxc.xhat
    assert np.abs(dw - ref).max() <= 1e-12 * np.abs(ref).max()


def test_stochastic_codes_follow_the_rule_and_are_unbiased():
    # Sec. 6.1: the product t = x * E goes to one of its two neighbours on the E2M1 grid, up iff (t - lo)/(hi - lo) > (u + 1/2)/2^16
    rng = np.random.default_rng(36)
    x = data(rng, 6, 64, 0.05)
    xf = orc.bf16_to_float(x).astype(np.float64)
    q0 = orc.quantize_nvfp4(x)
    grid = [0, 0.5, 1, 1.5, 2, 3, 4, 6]
    seed = 1234
    q = orc.quantize_nvfp4(x, sr_seed=seed)
    assert np.array_equal(q.sf, q0.sf) and q.enc == q0.enc          # the scale bytes do not depend on the rounding
    for r in range(6):
        for c in range(64):
            sv = orc.decode_code(FP8, int(q.sf[c // 16, r]))
            t = f32(xf[r, c]) * (q.enc / f32(sv))
            a = min(abs(float(t)), 6.0)
            lo = max(g for g in grid if g <= a)
            hi = min([g for g in grid if g > a], default=lo)
            u = orc.sr_uniform16(seed, r * 64 + c)
            up = hi > lo and (Fraction(a) - Fraction(lo)) / (Fraction(hi) - Fraction(lo)) > Fraction(2 * u + 1, 131072)
            want = (hi if up else lo) * (-1.0 if np.signbit(t) else 1.0)
            assert orc.decode_code(FP4, int(q.codes[r, c])) == want, (r, c)
    # the mean over seeds approaches x wherever the value does not saturate
    acc = np.zeros_like(xf)
    n = 400
    for s in range(n):
        acc += orc.quantize_nvfp4(x, sr_seed=1000 + s).xhat
    v8 = np.vectorize(lambda c: orc.decode_code(FP8, int(c)))
    unit = v8(q0.sf).T.repeat(16, axis=1) / float(q0.enc)
    inside = np.abs(xf) <= 6.0 * unit
    assert (np.abs(acc / n - xf)[inside] <= 2.0 * unit[inside] * 4.0 / np.sqrt(n)).all()   # 4 sigma of a step of at most 2 units
