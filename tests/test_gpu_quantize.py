"""GPU parity of the quantizers against the CPU oracle: codes and scales bit-exact, error-norm
statistics within 1e-4 relative.  Everything goes through the C-ABI binding."""
import numpy as np
import pytest
import torch

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

pytestmark = pytest.mark.gpu

FP8, FP4, BF16 = 1, 2, 0
ROW, COL, BLK = 0, 1, 2
STATS_RTOL = 1e-4


@pytest.fixture(scope="module")
def api():
    from paper_2602_01410_b200 import api as _api
    return _api


from gpu_util import to_dev  # noqa: E402


def check_quantize(api, x_bits, fmt, block, transposed, row_stats=False):
    rows, cols = x_bits.shape
    q = orc.quantize(x_bits, fmt, block)
    flags = api.Q_STATS | (api.Q_TRANSPOSED if transposed else 0)
    codes, scales, stats, rstats = api.snip_quantize(to_dev(x_bits), fmt, block, flags, want_row_stats=row_stats)
    torch.cuda.synchronize()
    want_codes = q.packed(transposed)
    got_codes = codes.cpu().numpy()[:want_codes.size].reshape(want_codes.shape)
    assert np.array_equal(got_codes, want_codes), f"codes differ at {np.argwhere(got_codes != want_codes)[:5]}"
    got_scales = scales.cpu().numpy().reshape(q.scales.shape)
    assert np.array_equal(got_scales.view(np.uint32), q.scales.view(np.uint32))
    st = api.stats_to_host(stats)
    assert st["sumsq_x"] == pytest.approx(q.sumsq_x, rel=STATS_RTOL)
    assert st["sumsq_err"] == pytest.approx(q.sumsq_err, rel=STATS_RTOL, abs=1e-300)
    assert st["amax"] == float(np.abs(orc.bf16_to_float(x_bits)).max())
    if row_stats:
        r = rstats.cpu().numpy()
        assert np.allclose(r[:, 0], q.row_sumsq_x, rtol=STATS_RTOL)
        assert np.allclose(r[:, 1], q.row_sumsq_err, rtol=STATS_RTOL, atol=1e-300)


@pytest.mark.parametrize("fmt", [FP8, FP4])
@pytest.mark.parametrize("block", [ROW, COL, BLK])
@pytest.mark.parametrize("transposed", [False, True])
@pytest.mark.parametrize("shape", [(128, 128), (256, 384), (192, 320), (64, 64)])
def test_codes_scales_stats_small(api, fmt, block, transposed, shape):
    rng = np.random.default_rng(hash((fmt, block, shape)) % 2 ** 31)
    x = wl.to_bf16_bits(rng.standard_normal(shape).astype(np.float32) * np.float32(3.0))
    check_quantize(api, x, fmt, block, transposed)


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_config0_tensors_all_tile_kinds(api, fmt):
    cfg = wl.CONFIGS[0]
    x, w, dy = wl.linear_inputs(cfg, 0, 0)
    check_quantize(api, x, fmt, ROW, False, row_stats=True)
    check_quantize(api, x, fmt, COL, True, row_stats=True)
    check_quantize(api, w, fmt, BLK, False)
    check_quantize(api, w, fmt, BLK, True)
    check_quantize(api, dy, fmt, ROW, False)
    check_quantize(api, dy, fmt, COL, True)


@pytest.mark.parametrize("fmt", [FP8, FP4])
@pytest.mark.parametrize("block", [ROW, COL, BLK])
def test_degenerate_tiles(api, fmt, block):
    # all-zero tiles, negative zeros, bf16 subnormals (scale clamps to FLT_MAX), huge values
    x = np.zeros((128, 256), dtype=np.uint16)
    x[3, 5] = 0x8000
    x[:, 128:] = 0x0001
    x[7, 130] = 0x8001
    x[64:, :64] = wl.to_bf16_bits(np.full((64, 64), 3.0e38, dtype=np.float32))
    x[65, 1] = wl.to_bf16_bits(np.array([-1e-30], dtype=np.float32))[0]
    rows, cols = x.shape
    q = orc.quantize(x, fmt, block)
    codes, scales, _, _ = api.snip_quantize(to_dev(x), fmt, block, 0)
    torch.cuda.synchronize()
    assert np.array_equal(codes.cpu().numpy()[:q.packed().size].reshape(q.packed().shape), q.packed())
    assert np.array_equal(scales.cpu().numpy().reshape(q.scales.shape).view(np.uint32), q.scales.view(np.uint32))


def test_stats_only_and_bf16_identity(api):
    x = wl.make_dy(np.random.default_rng(5), 256, 192)
    q = orc.quantize(x, FP4, COL)
    _, _, stats, _ = api.snip_quantize(to_dev(x), FP4, COL, api.Q_STATS | api.Q_NO_CODES)
    st = api.stats_to_host(stats)
    assert st["sumsq_err"] == pytest.approx(q.sumsq_err, rel=STATS_RTOL)
    _, _, stats, rs = api.snip_quantize(to_dev(x), BF16, BLK, api.Q_STATS, want_row_stats=True)
    st = api.stats_to_host(stats)
    assert st["sumsq_err"] == 0.0 and st["sumsq_x"] == pytest.approx(q.sumsq_x, rel=STATS_RTOL)
    assert np.allclose(rs.cpu().numpy()[:, 0], q.row_sumsq_x, rtol=STATS_RTOL)


def test_strided_input_and_repeatability(api):
    rng = np.random.default_rng(9)
    big = wl.to_bf16_bits(rng.standard_normal((128, 512)).astype(np.float32))
    xd = to_dev(big)[:, 128:384]          # row stride 512, 256 columns
    sub = np.ascontiguousarray(big[:, 128:384])
    q = orc.quantize(sub, FP8, ROW)
    c1, s1, st1, _ = api.snip_quantize(xd, FP8, ROW, api.Q_STATS)
    c2, s2, st2, _ = api.snip_quantize(xd, FP8, ROW, api.Q_STATS)
    torch.cuda.synchronize()
    assert np.array_equal(c1.cpu().numpy().reshape(sub.shape), q.packed())
    assert torch.equal(c1, c2) and torch.equal(s1, s2) and torch.equal(st1, st2)   # bit-identical reruns


@pytest.mark.parametrize("fmt,block,transposed", [(FP8, ROW, False), (FP4, COL, True), (FP4, BLK, True), (FP8, COL, True)])
def test_full_size_7b_activation(api, fmt, block, transposed):
    # one tensor of the roofline configuration, the whole of it compared bit by bit
    cfg = wl.CONFIGS[3]
    x = wl.make_x(wl.rng_for(3, 0, 1, "X"), cfg.M, 4096, cfg.outlier_frac, cfg.outlier_scale)
    check_quantize(api, x, fmt, block, transposed)


def test_ragged_3b_ffn_width(api):
    x = wl.make_x(wl.rng_for(2, 0, 4, "X"), 1024, 8640, 0.005, 50.0)   # 8640 = 67.5 tiles
    for fmt in (FP8, FP4):
        check_quantize(api, x, fmt, ROW, False)
        check_quantize(api, x, fmt, COL, True)
        check_quantize(api, x, fmt, BLK, True)


@pytest.mark.parametrize("fmt", [FP8, FP4])
@pytest.mark.parametrize("block,transposed", [(ROW, False), (COL, True), (BLK, False), (BLK, True)])
@pytest.mark.parametrize("shape", [(256, 384), (192, 320)])
def test_power_of_two_scale_option(api, fmt, block, transposed, shape):
    rng = np.random.default_rng(77)
    x = wl.to_bf16_bits(rng.standard_normal(shape).astype(np.float32) * np.exp(rng.standard_normal((shape[0], 1))).astype(np.float32))
    q = orc.quantize(x, fmt, block, pow2_scale=True)
    flags = api.Q_STATS | (api.Q_TRANSPOSED if transposed else 0)
    codes, scales, sf, stats = api.snip_quantize_mx(to_dev(x), fmt, block, flags)
    torch.cuda.synchronize()
    want = q.packed(transposed)
    assert np.array_equal(codes.cpu().numpy()[:want.size].reshape(want.shape), want)
    assert np.array_equal(scales.cpu().numpy().reshape(q.scales.shape).view(np.uint32), q.scales.view(np.uint32))
    assert np.array_equal(sf.cpu().numpy(), orc.sf_atoms(q, transposed))
    st = api.stats_to_host(stats)
    assert st["sumsq_err"] == pytest.approx(q.sumsq_err, rel=STATS_RTOL)
    assert st["sumsq_x"] == pytest.approx(q.sumsq_x, rel=STATS_RTOL)


def test_power_of_two_scales_on_degenerate_tiles(api):
    x = np.zeros((128, 256), dtype=np.uint16)
    x[:, 128:] = 0x0001                                   # bf16 subnormals: exponent clamp
    x[5, 7] = wl.to_bf16_bits(np.array([3.0e38], dtype=np.float32))[0]
    for fmt in (FP8, FP4):
        q = orc.quantize(x, fmt, ROW, pow2_scale=True)
        codes, scales, sf, _ = api.snip_quantize_mx(to_dev(x), fmt, ROW, 0)
        torch.cuda.synchronize()
        assert np.array_equal(codes.cpu().numpy()[:q.packed().size].reshape(q.packed().shape), q.packed())
        assert np.array_equal(scales.cpu().numpy().reshape(q.scales.shape).view(np.uint32), q.scales.view(np.uint32))
        assert np.array_equal(sf.cpu().numpy(), orc.sf_atoms(q, False))
