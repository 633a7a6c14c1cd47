"""Parity at the full sizes of the benchmark configurations, on sampled output rows that the CPU
oracle can compute one by one (complete dot products over the whole contraction).

Row-wise (1x128) and column-wise (128x1) quantization act on each row / column independently, so the
oracle only quantizes the sampled rows / columns of that operand; the other operand is quantized in
full.  Same launch configuration as bench.py (snip_linear_* on the full tensors)."""
import numpy as np
import pytest
import torch

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

pytestmark = pytest.mark.gpu
from gpu_util import bf16_out_to_f64, rel_fro, to_dev  # noqa: E402

FP8, FP4, BF16 = 1, 2, 0
N_SAMPLE = 24


def sampled_three(cfg_index, linear, fa, fb, seed, one_read=False, pow2=False):
    """one_read: the launch configuration bench.py times (snip_linear_fwd_bwd: X, W, dY read once each by the
    two-output quantizer); otherwise the three separate calls.  pow2: the power-of-two scale option."""
    from paper_2602_01410_b200 import api
    cfg = wl.CONFIGS[cfg_index]
    lin = cfg.linears[linear]
    x, w, dy = wl.linear_inputs(cfg, 0, linear)
    M, K, N = cfg.M, lin.K, lin.N
    X, W, DY = to_dev(x), to_dev(w), to_dev(dy)
    if one_read:
        assert fa == fb
        y, dx, _, _ = api.snip_linear_fwd_bwd(X, W, DY, fa, fa, fa, api.OUT_BF16, pow2_scale=pow2)
        _, _, dw, _ = api.snip_linear_fwd_bwd(X, W, DY, fa, fa, fa, api.OUT_FP32, pow2_scale=pow2)
    else:
        y, _, _ = api.snip_linear_fwd(X, W, fa, fb, api.OUT_BF16)
        dx, _, _ = api.snip_linear_dgrad(DY, W, fa, fb, api.OUT_BF16)
        dw, _, _ = api.snip_linear_wgrad(DY, X, fa, fb, api.OUT_FP32)
    torch.cuda.synchronize()
    rng = np.random.default_rng(seed)
    rows = np.sort(rng.choice(M, N_SAMPLE, replace=False))
    rows[-1] = M - 1                                     # include the last row (tile tails)
    ncols = np.sort(rng.choice(N, N_SAMPLE, replace=False))
    ncols[-1] = N - 1

    qw = orc.quantize(w, fb, orc.BLOCK_BLK, pow2_scale=pow2)
    # fwd: Y[rows, :] = Xq[rows, :] . Wq^T   (bf16 output vs bf16-rounded oracle)
    qx = orc.quantize(np.ascontiguousarray(x[rows]), fa, orc.BLOCK_ROW, pow2_scale=pow2)
    ref = orc.gemm_fwd(qx.xhat, qw.xhat)
    ref16 = orc.bf16_to_float(orc.round_to_bf16(ref))
    assert rel_fro(bf16_out_to_f64(y[torch.from_numpy(rows).cuda()]), ref16) <= 1e-3
    # dgrad: dX[rows, :] = dYq[rows, :] . Wq
    qdy = orc.quantize(np.ascontiguousarray(dy[rows]), fa, orc.BLOCK_ROW, pow2_scale=pow2)
    ref = orc.gemm_dgrad(qdy.xhat, qw.xhat)
    ref16 = orc.bf16_to_float(orc.round_to_bf16(ref))
    assert rel_fro(bf16_out_to_f64(dx[torch.from_numpy(rows).cuda()]), ref16) <= 1e-3
    # wgrad: dW[ncols, :] = dYq[:, ncols]^T . Xq   (FP32 output vs raw oracle)
    qdyc = orc.quantize(np.ascontiguousarray(dy[:, ncols]), fa, orc.BLOCK_COL, pow2_scale=pow2)
    qxc = orc.quantize(x, fb, orc.BLOCK_COL, pow2_scale=pow2)
    ref = orc.gemm_wgrad(qdyc.xhat, qxc.xhat)
    got = dw[torch.from_numpy(ncols).cuda()].cpu().numpy()
    assert rel_fro(got, ref) <= 1e-3
    assert rel_fro(got, ref) <= 2e-5                     # FP32 accumulation over up to 128 chunks


@pytest.mark.parametrize("fmt", [FP4, FP8])
def test_7b_fused_qkv(fmt):
    # BASELINE configs[3]: tokens 16384, 4096 -> 12288, every GEMM in one format
    sampled_three(3, 0, fmt, fmt, 31)


@pytest.mark.parametrize("fmt", [FP4, FP8])
@pytest.mark.parametrize("pow2", [False, True])
def test_7b_fused_qkv_one_read_path_as_benchmarked(fmt, pow2):
    # the configuration bench.py times: two-output quantizers + the three GEMMs, paper rule and power-of-two option
    sampled_three(3, 0, fmt, fmt, 41, one_read=True, pow2=pow2)


def test_7b_two_output_quantizer_full_tensor_bit_exact():
    """16384 x 4096 activation through snip_quantize_dual (FP8 as stored + FP4 transposed): every code and scale
    against the oracle's two single-output runs."""
    from paper_2602_01410_b200 import api
    cfg = wl.CONFIGS[3]
    x, _, _ = wl.linear_inputs(cfg, 0, 1)
    a, b = api.snip_quantize_dual(to_dev(x), api.DUAL_ROW_COLT, FP8, FP4)
    torch.cuda.synchronize()
    qa, qb = orc.quantize(x, FP8, orc.BLOCK_ROW), orc.quantize(x, FP4, orc.BLOCK_COL)
    wa, wb = qa.packed(False), qb.packed(True)
    assert np.array_equal(a["codes"].cpu().numpy()[:wa.size].reshape(wa.shape), wa)
    assert np.array_equal(b["codes"].cpu().numpy()[:wb.size].reshape(wb.shape), wb)
    assert np.array_equal(a["scales"].cpu().numpy().reshape(qa.scales.shape).view(np.uint32), qa.scales.view(np.uint32))
    assert np.array_equal(b["scales"].cpu().numpy().reshape(qb.scales.shape).view(np.uint32), qb.scales.view(np.uint32))
    sa, sb = api.stats_to_host(a["stats"][:24]), api.stats_to_host(b["stats"][:24])
    assert sa["sumsq_err"] == pytest.approx(qa.sumsq_err, rel=1e-4) and sb["sumsq_err"] == pytest.approx(qb.sumsq_err, rel=1e-4)
    assert sa["sumsq_x"] == pytest.approx(qa.sumsq_x, rel=1e-4)


def test_7b_down_projection_long_contraction():
    sampled_three(3, 4, FP4, FP4, 32)        # 11008 -> 4096: K = 86 chunks, N-contraction 4096


@pytest.mark.parametrize("linear,fa,fb", [(2, FP8, FP4), (4, FP4, FP8), (4, FP4, FP4), (2, BF16, BF16)])
def test_3b_ragged_ffn(linear, fa, fb):
    # BASELINE configs[2]: FFN width 8640 = 67.5 tiles, as N (gate) and as K (down); mixed pairs included
    sampled_three(2, linear, fa, fb, 33 + linear)


def test_70b_slice_down_projection():
    # BASELINE configs[4]: 28672 -> 8192 (224 chunks in fwd)
    sampled_three(4, 4, FP4, FP4, 35)


def test_1b_block_with_seeded_precision_triples():
    # BASELINE configs[1]: each of the 7 linears draws (fwd, dgrad, wgrad) tags from {BF16, FP8, FP4}
    from paper_2602_01410_b200 import api
    cfg = wl.CONFIGS[1]
    tags = wl.precision_tags(cfg)[0]                     # [7 linears, 3 gemms]
    rng = np.random.default_rng(36)
    for li, lin in enumerate(cfg.linears):
        x, w, dy = wl.linear_inputs(cfg, 0, li)
        X, W, DY = to_dev(x), to_dev(w), to_dev(dy)
        f_fwd, f_dg, f_wg = (int(t) for t in tags[li])
        rows = np.sort(rng.choice(cfg.M, 8, replace=False))
        ncols = np.sort(rng.choice(lin.N, 8, replace=False))
        y, _, _ = api.snip_linear_fwd(X, W, f_fwd, f_fwd, api.OUT_FP32)
        dx, _, _ = api.snip_linear_dgrad(DY, W, f_dg, f_dg, api.OUT_FP32)
        dw, _, _ = api.snip_linear_wgrad(DY, X, f_wg, f_wg, api.OUT_FP32)
        torch.cuda.synchronize()
        r = torch.from_numpy(rows).cuda()
        ref = orc.gemm_fwd(orc.quantize(np.ascontiguousarray(x[rows]), f_fwd, orc.BLOCK_ROW).xhat, orc.quantize(w, f_fwd, orc.BLOCK_BLK).xhat)
        assert rel_fro(y[r].cpu().numpy(), ref) <= 2e-5, (lin.name, "fwd", f_fwd)
        ref = orc.gemm_dgrad(orc.quantize(np.ascontiguousarray(dy[rows]), f_dg, orc.BLOCK_ROW).xhat, orc.quantize(w, f_dg, orc.BLOCK_BLK).xhat)
        assert rel_fro(dx[r].cpu().numpy(), ref) <= 2e-5, (lin.name, "dgrad", f_dg)
        ref = orc.gemm_wgrad(orc.quantize(np.ascontiguousarray(dy[:, ncols]), f_wg, orc.BLOCK_COL).xhat, orc.quantize(x, f_wg, orc.BLOCK_COL).xhat)
        assert rel_fro(dw[torch.from_numpy(ncols).cuda()].cpu().numpy(), ref) <= 2e-5, (lin.name, "wgrad", f_wg)
