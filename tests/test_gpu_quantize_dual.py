"""Two-output quantizer against the CPU oracle: each output must be bit-identical (codes, scales,
scale-factor atoms) to the oracle's single-output quantization with the same format, tile kind and
scale rule; statistics within 1e-4."""
import numpy as np
import pytest
import torch

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

pytestmark = pytest.mark.gpu
from gpu_util import to_dev  # noqa: E402

FP8, FP4 = 1, 2
ROW, COL, BLK = 0, 1, 2


def check_output(api, o, x_bits, fmt, block, transposed, pow2):
    q = orc.quantize(x_bits, fmt, block, pow2_scale=pow2)
    want = q.packed(transposed)
    got = o["codes"].cpu().numpy()[:want.size].reshape(want.shape)
    assert np.array_equal(got, want), (fmt, block, transposed, np.argwhere(got != want)[:4])
    got_s = o["scales"].cpu().numpy().reshape(q.scales.shape)
    assert np.array_equal(got_s.view(np.uint32), q.scales.view(np.uint32))
    if o["stats"] is not None:
        st = api.stats_to_host(o["stats"][:24])
        assert st["sumsq_x"] == pytest.approx(q.sumsq_x, rel=1e-4)
        assert st["sumsq_err"] == pytest.approx(q.sumsq_err, rel=1e-4, abs=1e-300)
        assert st["amax"] == float(np.abs(orc.bf16_to_float(x_bits)).max())
    if o["sf"] is not None:
        want_sf = orc.sf_atoms(q, transposed)
        assert np.array_equal(o["sf"].cpu().numpy(), want_sf.reshape(-1))


@pytest.mark.parametrize("fa,fb", [(FP8, FP8), (FP8, FP4), (FP4, FP8), (FP4, FP4)])
@pytest.mark.parametrize("kind", [0, 1])
@pytest.mark.parametrize("shape", [(128, 128), (256, 384), (192, 320), (64, 64), (448, 576)])
def test_dual_matches_two_single_quantizations(fa, fb, kind, shape):
    from paper_2602_01410_b200 import api
    rng = np.random.default_rng(hash((fa, fb, kind, shape)) % 2 ** 31)
    x = wl.make_x(rng, *shape)
    a, b = api.snip_quantize_dual(to_dev(x), kind, fa, fb)
    torch.cuda.synchronize()
    blocks = (ROW, COL) if kind == api.DUAL_ROW_COLT else (BLK, BLK)
    check_output(api, a, x, fa, blocks[0], False, False)
    check_output(api, b, x, fb, blocks[1], True, False)


@pytest.mark.parametrize("fa,fb", [(FP8, FP4), (FP4, FP4)])
@pytest.mark.parametrize("kind", [0, 1])
def test_dual_power_of_two_rule_with_scale_factor_atoms(fa, fb, kind):
    from paper_2602_01410_b200 import api
    rng = np.random.default_rng(77 + kind)
    x = wl.make_dy(rng, 320, 256)
    a, b = api.snip_quantize_dual(to_dev(x), kind, fa, fb, pow2_scale=True, want_sf=True)
    torch.cuda.synchronize()
    blocks = (ROW, COL) if kind == api.DUAL_ROW_COLT else (BLK, BLK)
    check_output(api, a, x, fa, blocks[0], False, True)
    check_output(api, b, x, fb, blocks[1], True, True)


def test_dual_without_statistics_and_argument_checks():
    from paper_2602_01410_b200 import api
    x = wl.make_x(np.random.default_rng(2), 128, 256)
    a, b = api.snip_quantize_dual(to_dev(x), api.DUAL_ROW_COLT, FP8, FP4, want_stats=False)
    torch.cuda.synchronize()
    check_output(api, a, x, FP8, ROW, False, False)
    check_output(api, b, x, FP4, COL, True, False)
    with pytest.raises(api.SnipError):   # BF16 is not a quantized output
        api.snip_quantize_dual(to_dev(x), api.DUAL_ROW_COLT, 0, FP4)
    with pytest.raises(api.SnipError):   # atoms need the power-of-two rule
        api.snip_quantize_dual(to_dev(x), api.DUAL_ROW_COLT, FP8, FP4, want_sf=True)
