"""snip_layer_stats against the oracle's Step-1 statistics (Sec. 3.1 of the paper)."""
import numpy as np
import pytest
import torch

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

pytestmark = pytest.mark.gpu
from gpu_util import to_dev  # noqa: E402


def test_layer_stats_all_tensors_all_formats():
    from paper_2602_01410_b200 import api
    M, K, N = 256, 320, 192
    rng = np.random.default_rng(3)
    x, w, dy = wl.make_x(rng, M, K), wl.make_w(rng, N, K), wl.make_dy(rng, M, N)
    y = wl.to_bf16_bits(rng.standard_normal((M, N)).astype(np.float32))
    dx = wl.to_bf16_bits(rng.standard_normal((M, K)).astype(np.float32) * np.float32(1e-4))
    dw = wl.to_bf16_bits(rng.standard_normal((N, K)).astype(np.float32) * np.float32(1e-2))
    out = api.snip_layer_stats(to_dev(x), to_dev(w), to_dev(y), to_dev(dy), to_dev(dx), to_dev(dw), M=M, N=N, K=K)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    ref = orc.layer_stats(x, w, y, dy, dx, dw)
    for i, name in enumerate(("X", "W", "Y", "dY", "dX", "dW")):
        assert got[i] == pytest.approx(ref["sumsq"][name], rel=1e-4), name
    err = got[6:].reshape(3, 2, 3)
    seen = 0
    for (name, fmt, block), v in ref["sumsq_err"].items():
        t = {"X": 0, "W": 1, "dY": 2}[name]
        assert err[t, fmt - 1, block] == pytest.approx(v, rel=1e-4), (name, fmt, block)
        seen += 1
    assert seen == 10 and np.count_nonzero(err) == 10


def test_layer_stats_skips_missing_tensors_and_formats():
    from paper_2602_01410_b200 import api
    M, K, N = 128, 128, 128
    x = wl.make_x(np.random.default_rng(1), M, K)
    out = api.snip_layer_stats(X=to_dev(x), M=M, N=N, K=K, fmt_mask=0b010).cpu().numpy()
    ref = orc.quantize(x, orc.FMT_FP8_E4M3, orc.BLOCK_ROW)
    assert out[0] == pytest.approx(ref.sumsq_x, rel=1e-4) and out[1:6].sum() == 0
    err = out[6:].reshape(3, 2, 3)
    assert err[0, 0, 0] == pytest.approx(ref.sumsq_err, rel=1e-4) and err[0, 1].sum() == 0


@pytest.mark.parametrize("fmt_mask", [0b010, 0b100, 0b110])
def test_layer_stats_ragged_tiles_match_per_option_quantizer_runs(fmt_mask):
    """Dimensions that end in a 64-wide tile; every option of the one-read kernel against the oracle's
    quantizer run for that option alone."""
    from paper_2602_01410_b200 import api
    M, K, N = 448, 576, 320
    rng = np.random.default_rng(11)
    x, w, dy = wl.make_x(rng, M, K), wl.make_w(rng, N, K), wl.make_dy(rng, M, N)
    out = api.snip_layer_stats(X=to_dev(x), W=to_dev(w), dY=to_dev(dy), M=M, N=N, K=K, fmt_mask=fmt_mask).cpu().numpy()
    err = out[6:].reshape(3, 2, 3)
    for t, (bits, blocks) in enumerate(((x, (orc.BLOCK_ROW, orc.BLOCK_COL)), (w, (orc.BLOCK_BLK,)), (dy, (orc.BLOCK_ROW, orc.BLOCK_COL)))):
        for f, fmt in enumerate((orc.FMT_FP8_E4M3, orc.FMT_FP4_E2M1)):
            for b in range(3):
                if (fmt_mask >> (f + 1)) & 1 and b in blocks:
                    ref = orc.quantize(bits, fmt, b)
                    assert err[t, f, b] == pytest.approx(ref.sumsq_err, rel=1e-4), (t, f, b)
                    assert out[(0, 1, 3)[t]] == pytest.approx(ref.sumsq_x, rel=1e-4)
                else:
                    assert err[t, f, b] == 0.0


def test_layer_stats_lossless_tensor_has_zero_error():
    """A tensor made of representable values times one power of two per 128x128 block with the format's
    largest value present in every row and column tile quantizes without error under every option."""
    from paper_2602_01410_b200 import api
    M = K = N = 256
    rng = np.random.default_rng(5)
    vals = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0], dtype=np.float32)
    a = vals[rng.integers(0, 8, size=(M, K))] * rng.choice(np.array([-1.0, 1.0], dtype=np.float32), size=(M, K))
    for i in range(M):          # 6 in every 1x128 row tile and every 128x1 column tile
        a[i, (i % 128)] = 6.0
        a[i, 128 + (i % 128)] = -6.0
    for bi in range(2):
        for bj in range(2):
            a[bi * 128:(bi + 1) * 128, bj * 128:(bj + 1) * 128] *= np.float32(2.0 ** (bi - 2 * bj))
    bits = wl.to_bf16_bits(a)
    out = api.snip_layer_stats(X=to_dev(bits), W=to_dev(bits), dY=to_dev(bits), M=M, N=N, K=K, fmt_mask=0b100).cpu().numpy()
    assert out[0] == pytest.approx(float((a.astype(np.float64) ** 2).sum()), rel=1e-6)
    assert np.all(out[6:] == 0.0)
