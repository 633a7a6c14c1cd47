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
