"""Pins for the oracle's three GEMMs (Fig. 5; shapes of Sec. 4.2 / 4.3): textbook matmul for
BF16 tags, exactness under lossless quantization, hand-expanded sums, linearity."""
import numpy as np
import pytest

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

FP8, FP4, BF16 = orc.FMT_FP8_E4M3, orc.FMT_FP4_E2M1, orc.FMT_BF16


def bits(a):
    return wl.to_bf16_bits(np.asarray(a, dtype=np.float32))


def rand_bits(shape, seed, scale=1.0):
    return bits(np.random.default_rng(seed).standard_normal(shape) * scale)


def lossless(shape, fmt, seed):
    """Matrix of representable values times per-128x128-block powers of two, with +-FPX_MAX in
    every row and column segment of every block, so that ROW, COL and BLK quantization are all
    exact (S is a power of two, error zero)."""
    rng = np.random.default_rng(seed)
    n = 0x7F if fmt == FP8 else 8
    table = np.array([orc.decode_code(fmt, c) for c in range(n)])
    R, C = shape
    v = rng.choice(table, size=shape) * rng.choice([-1.0, 1.0], size=shape)
    mx = orc.fpx_max(fmt)
    for r in range(R):                      # a full-scale element on a shifted diagonal
        for cb in range(0, C, 128):
            v[r, cb + (r % min(128, C - cb))] = mx
    for c in range(C):
        for rb in range(0, R, 128):
            v[rb + (c % min(128, R - rb)), c] = -mx if (c % 2) else mx
    exps = rng.integers(-3, 4, size=((R + 127) // 128, (C + 127) // 128))
    scale = np.repeat(np.repeat(2.0 ** exps, 128, axis=0), 128, axis=1)[:R, :C]
    return bits(v * scale)


def test_bf16_tags_equal_textbook_matmul():
    x, w, dy = rand_bits((48, 160), 1), rand_bits((40, 160), 2), rand_bits((48, 40), 3)
    xf, wf, dyf = orc.bf16_to_float(x), orc.bf16_to_float(w), orc.bf16_to_float(dy)
    y, _, _ = orc.linear_fwd(x, w, BF16, BF16)
    dx, _, _ = orc.linear_dgrad(dy, w, BF16, BF16)
    dw, _, _ = orc.linear_wgrad(dy, x, BF16, BF16)
    assert np.allclose(y, xf @ wf.T, rtol=1e-12, atol=1e-12)
    assert np.allclose(dx, dyf @ wf, rtol=1e-12, atol=1e-12)
    assert np.allclose(dw, dyf.T @ xf, rtol=1e-12, atol=1e-12)
    assert y.shape == (48, 40) and dx.shape == (48, 160) and dw.shape == (40, 160)


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_lossless_quantization_gives_the_plain_product(fmt):
    M, K, N = 256, 384, 192           # several tiles, ragged N
    x, w, dy = lossless((M, K), fmt, 5), lossless((N, K), fmt, 6), lossless((M, N), fmt, 7)
    xf, wf, dyf = orc.bf16_to_float(x), orc.bf16_to_float(w), orc.bf16_to_float(dy)
    y, qx, qw = orc.linear_fwd(x, w, fmt, fmt)
    assert qx.sumsq_err == 0 and qw.sumsq_err == 0
    assert np.array_equal(qx.xhat, xf) and np.array_equal(qw.xhat, wf)
    assert np.allclose(y, xf @ wf.T, rtol=1e-12, atol=0)
    dx, qdy, _ = orc.linear_dgrad(dy, w, fmt, fmt)
    assert qdy.sumsq_err == 0
    assert np.allclose(dx, dyf @ wf, rtol=1e-12, atol=0)
    dw, qdyc, qxc = orc.linear_wgrad(dy, x, fmt, fmt)
    assert qdyc.sumsq_err == 0 and qxc.sumsq_err == 0
    assert np.allclose(dw, dyf.T @ xf, rtol=1e-12, atol=0)


def test_tiny_case_expanded_by_hand():
    # X = [[6, 3], [-1.5, 0.5]] (one ROW tile per row), W = [[4, 2]] (one block), FP4.
    # row 0: amax 6 -> S=1, codes exact.  row 1: amax 1.5 -> S=4: 1.5*4=6, 0.5*4=2 -> exact.
    # W: amax 4 -> S=1.5: 4*1.5=6, 2*1.5=3 -> exact.  Y = X W^T = [[30], [-5]].
    x, w = bits([[6.0, 3.0], [-1.5, 0.5]]), bits([[4.0, 2.0]])
    y, qx, qw = orc.linear_fwd(x, w, FP4, FP4)
    assert qx.scales[0].tolist() == [1.0, 4.0] and qw.scales[0, 0] == 1.5
    assert qx.codes.tolist() == [[7, 5], [7 | 8, 4]] and qw.codes.tolist() == [[7, 5]]
    assert y.tolist() == [[30.0], [-5.0]]
    # a lossy element: X = [[6, 2.6]] -> 2.6 rounds to 3 (nearest of 2, 3); bf16(2.6)=2.59375
    y2, q2, _ = orc.linear_fwd(bits([[6.0, 2.6]]), w, FP4, FP4)
    assert q2.codes.tolist() == [[7, 5]] and y2.tolist() == [[30.0]]
    assert q2.sumsq_err == pytest.approx((3 - 2.59375) ** 2, rel=1e-12)
    # dgrad / wgrad with one token: dY = [[2]], FP8 (exact): dX = dY W = [[8, 4]]; dW = dY^T X
    dy = bits([[2.0]])
    dx, _, _ = orc.linear_dgrad(dy, w, FP8, FP8)
    assert dx.tolist() == [[8.0, 4.0]]
    # X = [[7, 3.5]]: COL tiles of one element -> S = 448/7 = 64 and 448/3.5 = 128, both exact
    dw, _, _ = orc.linear_wgrad(dy, bits([[7.0, 3.5]]), FP8, FP8)
    assert dw.tolist() == [[14.0, 7.0]]
    # when S is not a power of two the round trip is not exact: 448 / fl32(448/6) != 6
    q6 = orc.quantize(bits([[6.0]]), FP8, orc.BLOCK_ROW)
    s6 = np.float32(448.0) / np.float32(6.0)
    assert q6.codes[0, 0] == 0x7E and q6.xhat[0, 0] == 448.0 / float(s6) != 6.0


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_linearity_in_powers_of_two(fmt):
    x, w = rand_bits((32, 256), 8), rand_bits((24, 256), 9)
    y, _, _ = orc.linear_fwd(x, w, fmt, fmt)
    x4 = bits(wl.bf16_bits_to_f32(x) * np.float32(4.0))
    y4, _, _ = orc.linear_fwd(x4, w, fmt, fmt)
    assert np.array_equal(y4, 4.0 * y)


def test_quantized_gemm_matches_explicit_double_sum():
    # brute force over two K tiles with the scale bookkeeping written out:
    # Y[m,n] = sum_j (S_x[j,m] S_w[n/128,j])^-1 sum_{k in tile j} v_x[m,k] v_w[n,k]
    x, w = rand_bits((3, 256), 12), rand_bits((2, 256), 13, 0.02)
    y, qx, qw = orc.linear_fwd(x, w, FP8, FP4)
    for m in range(3):
        for n in range(2):
            acc = 0.0
            for j in range(2):
                part = 0.0
                for k in range(128 * j, 128 * j + 128):
                    part += orc.decode_code(FP8, int(qx.codes[m, k])) * orc.decode_code(FP4, int(qw.codes[n, k]))
                acc += part / (float(qx.scales[j, m]) * float(qw.scales[0, j]))
            assert y[m, n] == pytest.approx(acc, rel=1e-12)


def test_layer_stats_keys_and_values():
    x, w, dy = rand_bits((128, 256), 1), rand_bits((64, 256), 2, 0.02), rand_bits((128, 64), 3, 1e-3)
    st = orc.layer_stats(x, w, None, dy, None, None)
    assert set(st["sumsq"]) == {"X", "W", "dY"}
    assert len(st["sumsq_err"]) == 2 * (2 + 1 + 2)
    assert st["sumsq_err"][("W", FP4, orc.BLOCK_BLK)] == orc.quantize(w, FP4, orc.BLOCK_BLK).sumsq_err
    assert st["sumsq"]["X"] == pytest.approx(float((orc.bf16_to_float(x) ** 2).sum()), rel=1e-13)
