"""snip_linear_fwd_bwd (every tensor read once, six quantized copies, three GEMMs) against the CPU
oracle: outputs within the GEMM tolerance, the six statistics within 1e-4, under the paper's scale
rule and under the power-of-two option."""
import numpy as np
import pytest
import torch

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

pytestmark = pytest.mark.gpu
from gpu_util import to_dev, rel_fro, bf16_out_to_f64  # noqa: E402

FP8, FP4 = 1, 2
ROW, COL, BLK = 0, 1, 2
TOL = 1e-3


def stats6(api, t):
    return [api.stats_to_host(t[24 * i:24 * i + 24]) for i in range(6)]


@pytest.mark.parametrize("triple", [(FP8, FP8, FP8), (FP4, FP4, FP4), (FP8, FP8, FP4), (FP4, FP8, FP4), (FP8, FP4, FP8)])
@pytest.mark.parametrize("pow2", [False, True])
@pytest.mark.parametrize("shape", [(256, 384, 192), (384, 320, 448)])
def test_fwd_bwd_outputs_and_statistics(triple, pow2, shape):
    from paper_2602_01410_b200 import api
    M, K, N = shape
    rng = np.random.default_rng(M + 3 * K + 7 * N)
    x, w, dy = wl.make_x(rng, M, K), wl.make_w(rng, N, K), wl.make_dy(rng, M, N)
    ff, fd, fw = triple
    y, dx, dw, st = api.snip_linear_fwd_bwd(to_dev(x), to_dev(w), to_dev(dy), ff, fd, fw, api.OUT_FP32, pow2_scale=pow2)
    torch.cuda.synchronize()
    want = (orc.linear_fwd(x, w, ff, ff, pow2_scale=pow2)[0], orc.linear_dgrad(dy, w, fd, fd, pow2_scale=pow2)[0],
            orc.linear_wgrad(dy, x, fw, fw, pow2_scale=pow2)[0])
    for name, g, ref in zip(("fwd", "dgrad", "wgrad"), (y, dx, dw), want):
        assert rel_fro(g.cpu().numpy(), ref) <= 1e-5, name
    got = stats6(api, st)
    cases = ((x, ff, ROW), (x, fw, COL), (w, ff, BLK), (w, fd, BLK), (dy, fd, ROW), (dy, fw, COL))
    for s, (bits, fmt, block) in zip(got, cases):
        q = orc.quantize(bits, fmt, block, pow2_scale=pow2)
        assert s["sumsq_x"] == pytest.approx(q.sumsq_x, rel=1e-4)
        assert s["sumsq_err"] == pytest.approx(q.sumsq_err, rel=1e-4)


def test_fwd_bwd_bf16_outputs_match_the_three_separate_calls_bit_for_bit():
    from paper_2602_01410_b200 import api
    cfg = wl.CONFIGS[0]
    x, w, dy = wl.linear_inputs(cfg, 0, 0)
    xd, wd, dyd = to_dev(x), to_dev(w), to_dev(dy)
    y, dx, dw, _ = api.snip_linear_fwd_bwd(xd, wd, dyd, FP8, FP8, FP4)
    y1 = api.snip_linear_fwd(xd, wd, FP8, FP8)[0]
    dx1 = api.snip_linear_dgrad(dyd, wd, FP8, FP8)[0]
    dw1 = api.snip_linear_wgrad(dyd, xd, FP4, FP4)[0]
    torch.cuda.synchronize()
    assert torch.equal(y, y1) and torch.equal(dx, dx1) and torch.equal(dw, dw1)
    ref16 = orc.bf16_to_float(orc.round_to_bf16(orc.linear_fwd(x, w, FP8, FP8)[0]))
    assert rel_fro(bf16_out_to_f64(y), ref16) <= TOL


def test_fwd_bwd_rejects_bf16_tags_and_small_workspace():
    from paper_2602_01410_b200 import api
    x, w, dy = (to_dev(wl.make_x(np.random.default_rng(i), 128, 128)) for i in range(3))
    with pytest.raises(api.SnipError):
        api.snip_linear_fwd_bwd(x, w, dy, 0, FP8, FP8)
    with pytest.raises(api.SnipError):
        api.snip_linear_fwd_bwd(x, w, dy, FP8, FP8, FP8, ws=torch.zeros(1024, dtype=torch.uint8, device="cuda"))
