"""Stochastic rounding on the GPU against the CPU oracle (paper Sec. 6.1): the same counter-based
generator and the same exact decision rule on both sides, so codes are bit-identical."""
import numpy as np
import pytest
import torch

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

pytestmark = pytest.mark.gpu
from gpu_util import to_dev, rel_fro  # noqa: E402

FP8, FP4 = 1, 2
ROW, COL = 0, 1


def check(api, got_codes, got_scales, got_stats, q, transposed):
    want = q.packed(transposed)
    got = got_codes.cpu().numpy()[:want.size].reshape(want.shape)
    assert np.array_equal(got, want), np.argwhere(got != want)[:4]
    assert np.array_equal(got_scales.cpu().numpy().reshape(q.scales.shape).view(np.uint32), q.scales.view(np.uint32))
    if got_stats is not None:
        st = api.stats_to_host(got_stats[:24])
        assert st["sumsq_x"] == pytest.approx(q.sumsq_x, rel=1e-4)
        assert st["sumsq_err"] == pytest.approx(q.sumsq_err, rel=1e-4)


@pytest.mark.parametrize("block,transposed", [(ROW, False), (COL, True)])
@pytest.mark.parametrize("shape", [(128, 128), (256, 384), (192, 320), (448, 576)])
@pytest.mark.parametrize("pow2", [False, True])
def test_sr_codes_bit_exact(block, transposed, shape, pow2):
    from paper_2602_01410_b200 import api
    rng = np.random.default_rng(shape[0] + shape[1] + block)
    x = wl.make_dy(rng, *shape)
    seed = 0x5EED0000ABCD0000 + shape[0]
    flags = api.Q_STATS | (api.Q_TRANSPOSED if transposed else 0)
    codes, scales, sf, stats = api.snip_quantize_sr(to_dev(x), block, flags, seed, pow2_scale=pow2, want_sf=pow2)
    torch.cuda.synchronize()
    q = orc.quantize(x, FP4, block, pow2_scale=pow2, sr_seed=seed)
    check(api, codes, scales, stats, q, transposed)
    if pow2:
        assert np.array_equal(sf.cpu().numpy(), orc.sf_atoms(q, transposed).reshape(-1))
    # a different seed gives different codes, the same seed the same
    c2 = api.snip_quantize_sr(to_dev(x), block, flags, seed + 1)[0]
    c3 = api.snip_quantize_sr(to_dev(x), block, flags, seed, pow2_scale=pow2)[0]
    n = shape[0] * shape[1] // 2                       # the buffer may carry tail slack beyond the codes
    assert not torch.equal(c2[:n], codes[:n]) and torch.equal(c3[:n], codes[:n])


def test_sr_extreme_values_and_index_beyond_32_bits_of_columns():
    from paper_2602_01410_b200 import api
    x = np.zeros((128, 256), dtype=np.uint16)
    x[3, 5] = 0x8000                                   # -0
    x[:, 128:] = 0x0001                                # bf16 subnormals: the scale clamps
    x[64:, :64] = wl.to_bf16_bits(np.full((64, 64), 3.0e38, dtype=np.float32))
    x[65, 1] = wl.to_bf16_bits(np.array([-1e-30], dtype=np.float32))[0]
    seed = 99
    codes, scales, _, stats = api.snip_quantize_sr(to_dev(x), ROW, api.Q_STATS, seed)
    q = orc.quantize(x, FP4, ROW, sr_seed=seed)
    want = q.packed(False)
    assert np.array_equal(codes.cpu().numpy()[:want.size].reshape(want.shape), want)


@pytest.mark.parametrize("fa,fb,seeds", [(FP4, FP4, (5, 6)), (FP4, FP4, (7, 7)), (FP4, FP8, (8, None)), (FP8, FP4, (None, 9)), (FP4, FP4, (None, 3)),
                                         (FP4, FP4, (4, None))])
def test_dual_with_stochastic_outputs(fa, fb, seeds):
    from paper_2602_01410_b200 import api
    x = wl.make_dy(np.random.default_rng(21), 320, 256)
    a, b = api.snip_quantize_dual(to_dev(x), api.DUAL_ROW_COLT, fa, fb, sr_seeds=seeds)
    torch.cuda.synchronize()
    check(api, a["codes"], a["scales"], a["stats"], orc.quantize(x, fa, ROW, sr_seed=seeds[0]), False)
    check(api, b["codes"], b["scales"], b["stats"], orc.quantize(x, fb, COL, sr_seed=seeds[1]), True)


def test_sr_is_refused_where_the_paper_does_not_use_it():
    from paper_2602_01410_b200 import api
    x = to_dev(wl.make_dy(np.random.default_rng(1), 128, 128))
    with pytest.raises(api.SnipError):                 # FP8 output
        api.snip_quantize_dual(x, api.DUAL_ROW_COLT, FP8, FP4, sr_seeds=(1, None))
    with pytest.raises(api.SnipError):                 # weight blocks
        api.snip_quantize_dual(x, api.DUAL_BLK_BLKT, FP4, FP4, sr_seeds=(1, 1))
    with pytest.raises(api.SnipError):                 # 128x128 blocks
        api.snip_quantize_sr(x, 2, 0, 1)


def test_fwd_bwd_with_stochastic_output_gradients():
    from paper_2602_01410_b200 import api
    M, K, N = 256, 384, 192
    rng = np.random.default_rng(4)
    x, w, dy = wl.make_x(rng, M, K), wl.make_w(rng, N, K), wl.make_dy(rng, M, N)
    seed = 1234
    y, dx, dw, st = api.snip_linear_fwd_bwd(to_dev(x), to_dev(w), to_dev(dy), FP8, FP4, FP4, api.OUT_FP32, dy_sr_seed=seed)
    torch.cuda.synchronize()
    qd_row = orc.quantize(dy, FP4, ROW, sr_seed=seed)
    qd_col = orc.quantize(dy, FP4, COL, sr_seed=seed)
    qw = orc.quantize(w, FP4, orc.BLOCK_BLK)
    qx = orc.quantize(x, FP4, COL)
    assert rel_fro(dx.cpu().numpy(), orc.gemm_dgrad(qd_row.xhat, qw.xhat)) <= 1e-5
    assert rel_fro(dw.cpu().numpy(), orc.gemm_wgrad(qd_col.xhat, qx.xhat)) <= 1e-5
    assert rel_fro(y.cpu().numpy(), orc.linear_fwd(x, w, FP8, FP8)[0]) <= 1e-5
    got = [api.stats_to_host(st[24 * i:24 * i + 24]) for i in range(6)]
    assert got[4]["sumsq_err"] == pytest.approx(qd_row.sumsq_err, rel=1e-4)
    assert got[5]["sumsq_err"] == pytest.approx(qd_col.sumsq_err, rel=1e-4)
