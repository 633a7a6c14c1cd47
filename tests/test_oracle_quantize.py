"""Pins for the oracle's quantizer (Sec. 2.3 scaling rule and granularity) and statistics
(Sec. 3.1).  Checked against closed forms, invariants and brute force -- never the CUDA path."""
import numpy as np
import pytest

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

FP8, FP4, BF16 = orc.FMT_FP8_E4M3, orc.FMT_FP4_E2M1, orc.FMT_BF16
ROW, COL, BLK = orc.BLOCK_ROW, orc.BLOCK_COL, orc.BLOCK_BLK
FMTS = [FP8, FP4]


def bits(a):
    return wl.to_bf16_bits(np.asarray(a, dtype=np.float32))


def rand_bits(shape, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    return bits(rng.standard_normal(shape) * scale)


def representable(fmt):
    n = 0x7F if fmt == FP8 else 8
    return np.array([orc.decode_code(fmt, c) for c in range(n)])


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("j", [-9, 0, 5])
def test_lossless_tile_is_idempotent(fmt, j):
    # a tile made of representable values times 2^j, with +-FPX_MAX*2^j present:
    # S = 2^-j exactly, codes enumerate the table, the error is exactly zero
    vals = representable(fmt)
    vals = np.concatenate([vals, -vals])
    tile = np.resize(vals, 128)
    tile[0] = orc.fpx_max(fmt)
    x = bits(tile[None, :] * 2.0 ** j)
    assert np.array_equal(orc.bf16_to_float(x)[0], tile * 2.0 ** j)  # exactly bf16
    q = orc.quantize(x, fmt, ROW)
    assert q.scales.shape == (1, 1) and q.scales[0, 0] == np.float32(2.0 ** -j)
    assert q.sumsq_err == 0.0
    assert np.array_equal(q.xhat, orc.bf16_to_float(x))
    for c, v in zip(q.codes[0], tile):
        assert orc.decode_code(fmt, int(c)) == v
    # quantizing the dequantized tile again returns the same codes
    q2 = orc.quantize(bits(q.xhat), fmt, ROW)
    assert np.array_equal(q2.codes, q.codes) and np.array_equal(q2.scales, q.scales)


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("block", [ROW, COL, BLK])
def test_scale_rule_and_saturation_invariants(fmt, block):
    x = rand_bits((300, 200), 11)     # ragged in both directions
    xf = orc.bf16_to_float(x)
    q = orc.quantize(x, fmt, block)
    d0, d1 = orc.scale_shape(300, 200, block)
    assert q.scales.shape == (d0, d1)
    top = 0x7E if fmt == FP8 else 7
    mask = 0x7F if fmt == FP8 else 7
    for a in range(d0):
        for b in range(d1):
            if block == ROW:
                sl = (slice(b, b + 1), slice(128 * a, 128 * a + 128))
            elif block == COL:
                sl = (slice(128 * a, 128 * a + 128), slice(b, b + 1))
            else:
                sl = (slice(128 * a, 128 * a + 128), slice(128 * b, 128 * b + 128))
            amax = np.abs(xf[sl]).max()
            want = np.float32(orc.fpx_max(fmt)) / np.float32(amax)   # binary32 division
            assert q.scales[a, b] == want
            # at least one element of every tile sits at +-FPX_MAX, and nothing above it
            assert ((q.codes[sl] & mask) == top).any()
    if fmt == FP8:
        assert ((q.codes & 0x7F) != 0x7F).all()   # never a NaN code
    else:
        assert (q.codes < 16).all()


@pytest.mark.parametrize("fmt", FMTS)
def test_codes_follow_the_two_rounding_steps(fmt):
    # code = RNE_fmt(fl32(x * S)), recomputed per element with numpy float32 and the scalar encoder
    x = rand_bits((4, 256), 5, scale=3.0)
    q = orc.quantize(x, fmt, ROW)
    xf32 = wl.bf16_bits_to_f32(x)
    for r in range(4):
        for c in range(256):
            s = q.scales[c // 128, r]
            t = np.float32(xf32[r, c] * s)
            assert q.codes[r, c] == orc.encode(fmt, float(t))
            assert q.xhat[r, c] == orc.decode_code(fmt, int(q.codes[r, c])) / float(s)


@pytest.mark.parametrize("fmt", FMTS)
def test_error_bound_per_element(fmt):
    x = rand_bits((64, 384), 21)
    q = orc.quantize(x, fmt, ROW)
    xf = orc.bf16_to_float(x)
    S = np.repeat(q.scales.T.astype(np.float64), 128, axis=1)   # [rows, cols]
    t = np.abs(xf * S)
    err = np.abs(xf - q.xhat) * S
    ulp = t * 2.0 ** -23
    if fmt == FP8:
        bound = np.maximum(t * 2.0 ** -4, 2.0 ** -10)
    else:
        bound = np.where(t < 2, 0.25, np.where(t < 4, 0.5, 1.0))
    assert (err <= bound + ulp).all()


def test_e2m1_rms_error_on_uniform_inputs():
    # closed form: spacing d on a length-L stretch contributes L*d^2/12 ->
    # (2*0.25 + 2*1 + 2*4)/12 / 6 = 7/48
    rng = np.random.default_rng(0)
    v = rng.uniform(-6, 6, (256, 128)).astype(np.float32)
    v[:, 0] = 6.0                       # pins S = 1 in every tile
    x = bits(v)
    q = orc.quantize(x, FP4, ROW)
    assert (q.scales == 1.0).all()
    rms = np.sqrt(q.sumsq_err / x.size)
    assert abs(rms - np.sqrt(7 / 48)) < 0.01 * np.sqrt(7 / 48)


@pytest.mark.parametrize("fmt", FMTS)
def test_power_of_two_scaling_and_locality(fmt):
    x = rand_bits((130, 260), 9)
    q = orc.quantize(x, fmt, BLK)
    x8 = bits(wl.bf16_bits_to_f32(x) * np.float32(2.0 ** -7))
    q8 = orc.quantize(x8, fmt, BLK)
    assert np.array_equal(q8.codes, q.codes)
    assert np.array_equal(q8.scales, q.scales * np.float32(2.0 ** 7))
    # changing one element only changes its own block
    y = x.copy()
    y[5, 5] = bits([1000.0])[0]
    qy = orc.quantize(y, fmt, BLK)
    assert np.array_equal(qy.codes[:, 128:], q.codes[:, 128:])
    assert np.array_equal(qy.codes[128:, :], q.codes[128:, :])
    assert not np.array_equal(qy.codes[:128, :128], q.codes[:128, :128])
    assert np.array_equal(qy.scales.ravel()[1:], q.scales.ravel()[1:])


@pytest.mark.parametrize("fmt", FMTS)
def test_orientation_identities_and_ragged_tiles(fmt):
    x = rand_bits((192, 320), 4)      # 192 = 1.5 tiles, 320 = 2.5 tiles
    xt = np.ascontiguousarray(x.T)
    qb, qbt = orc.quantize(x, fmt, BLK), orc.quantize(xt, fmt, BLK)
    assert np.array_equal(qbt.codes, qb.codes.T) and np.array_equal(qbt.scales, qb.scales.T)
    qc, qr = orc.quantize(x, fmt, COL), orc.quantize(xt, fmt, ROW)
    assert np.array_equal(qc.codes, qr.codes.T) and np.array_equal(qc.scales, qr.scales)
    assert qc.sumsq_err == pytest.approx(qr.sumsq_err, rel=1e-12)
    # a 64-wide last tile equals quantizing that slice on its own
    qrow = orc.quantize(x, fmt, ROW)
    tail = orc.quantize(np.ascontiguousarray(x[:, 256:]), fmt, ROW)
    assert np.array_equal(qrow.codes[:, 256:], tail.codes)
    assert np.array_equal(qrow.scales[2], tail.scales[0])


@pytest.mark.parametrize("fmt", FMTS)
def test_zero_and_tiny_tiles(fmt):
    sbit = 0x80 if fmt == FP8 else 8
    x = np.zeros((2, 256), dtype=np.uint16)
    x[0, 3] = 0x8000                                  # -0
    x[1, 128:] = 0x0001                               # smallest bf16 subnormal, 9.2e-41
    x[1, 130] = 0x8001
    q = orc.quantize(x, fmt, ROW)
    assert q.scales[0, 0] == 1.0 and q.scales[1, 0] == 1.0 and q.scales[0, 1] == 1.0
    assert q.codes[0, 3] == sbit and q.codes[0, 4] == 0
    assert q.scales[1, 1] == np.finfo(np.float32).max    # FPX_MAX/amax overflows -> clamped
    assert np.isfinite(q.xhat).all() and q.sumsq_err >= 0
    assert q.codes[1, 130] & sbit and not (q.codes[1, 129] & sbit)


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("block", [ROW, COL, BLK])
def test_stats_against_separate_recomputation(fmt, block):
    x = rand_bits((200, 264), 17)
    q = orc.quantize(x, fmt, block)
    xf = orc.bf16_to_float(x)
    # plain float64 sums written here, and xhat rebuilt by the separate dequantize routine
    xh = orc.dequantize(q.codes, q.scales, fmt, block)
    assert np.array_equal(xh, q.xhat)
    assert q.sumsq_x == pytest.approx(float((xf * xf).sum()), rel=1e-13)
    assert q.sumsq_err == pytest.approx(float(((xf - xh) ** 2).sum()), rel=1e-13)
    assert np.allclose(q.row_sumsq_x, (xf * xf).sum(axis=1), rtol=1e-13)
    assert np.allclose(q.row_sumsq_err, ((xf - xh) ** 2).sum(axis=1), rtol=1e-13)
    assert q.sumsq_x == pytest.approx(orc.sumsq_bf16(x), rel=1e-13)
    # and an independent per-element dequantization: value(code) / S with explicit indexing
    r, c = 137, 201
    idx = {ROW: (c // 128, r), COL: (r // 128, c), BLK: (r // 128, c // 128)}[block]
    s = q.scales[idx]
    assert xh[r, c] == orc.decode_code(fmt, int(q.codes[r, c])) / float(s)


def test_bf16_tag_is_identity():
    x = rand_bits((64, 128), 2)
    q = orc.quantize(x, BF16, ROW)
    assert q.codes is None and q.scales is None and q.sumsq_err == 0.0
    assert np.array_equal(q.xhat, orc.bf16_to_float(x))


def test_pack_layout():
    codes = (np.arange(4 * 6, dtype=np.uint8).reshape(4, 6) * 5) % 16
    p = orc.pack_codes(codes, FP4)
    assert p.shape == (4, 3)
    for r in range(4):
        for b in range(3):
            assert p[r, b] == codes[r, 2 * b] | (codes[r, 2 * b + 1] << 4)
    pt = orc.pack_codes(codes, FP4, transposed=True)
    assert pt.shape == (6, 2)
    for c in range(6):
        for b in range(2):
            assert pt[c, b] == codes[2 * b, c] | (codes[2 * b + 1, c] << 4)
    c8 = np.arange(12, dtype=np.uint8).reshape(3, 4) + 100
    assert np.array_equal(orc.pack_codes(c8, FP8), c8)
    assert np.array_equal(orc.pack_codes(c8, FP8, transposed=True), c8.T)


def test_expected_error_magnitudes_on_gaussian_inputs():
    # sanity window, not a tight pin: relative error of 1x128 quantization of N(0,1)
    x = rand_bits((256, 1024), 33)
    r8 = orc.quantize(x, FP8, ROW)
    r4 = orc.quantize(x, FP4, ROW)
    rel8 = np.sqrt(r8.sumsq_err / r8.sumsq_x)
    rel4 = np.sqrt(r4.sumsq_err / r4.sumsq_x)
    assert 0.015 < rel8 < 0.04
    assert 0.07 < rel4 < 0.16
