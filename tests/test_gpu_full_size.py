"""Parity at the full sizes of the benchmark configurations, on sampled output rows that the CPU
oracle can compute one by one (complete dot products over the whole contraction).  The sample holds
one row of EVERY 128-row tile of the output (so every tile of the persistent tile walk, every wave and
every accumulator-buffer phase is compared), the last row of the matrix, and random rows up to 256.

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
N_SAMPLE = 256


def tile_sample(n, rng, count=N_SAMPLE):
    """Sorted indices in [0, n): one at a random offset inside every 128-wide tile, the last index, and random
    others up to `count` (more if there are more tiles than that)."""
    idx = {min(n - 1, 128 * t + int(rng.integers(0, 128))) for t in range(-(-n // 128))}
    idx.add(n - 1)
    while len(idx) < min(count, n):
        idx.add(int(rng.integers(0, n)))
    return np.array(sorted(idx))


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
    rows = tile_sample(M, rng)                           # rows of Y and dX
    ncols = tile_sample(N, rng)                          # rows of dW

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
    # the 7B configuration: tokens 16384, 4096 -> 12288, every GEMM in one format
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
    # the 3B configuration: FFN width 8640 = 67.5 tiles, as N (gate) and as K (down); mixed pairs included
    sampled_three(2, linear, fa, fb, 33 + linear)


def test_70b_slice_down_projection():
    # the 70B slice: 28672 -> 8192 (224 chunks in fwd)
    sampled_three(4, 4, FP4, FP4, 35)


def test_1b_block_with_seeded_precision_triples():
    # the 1B configuration: each of the 7 linears draws (fwd, dgrad, wgrad) tags from {BF16, FP8, FP4}
    from paper_2602_01410_b200 import api
    cfg = wl.CONFIGS[1]
    tags = wl.precision_tags(cfg)[0]                     # [7 linears, 3 gemms]
    rng = np.random.default_rng(36)
    for li, lin in enumerate(cfg.linears):
        x, w, dy = wl.linear_inputs(cfg, 0, li)
        X, W, DY = to_dev(x), to_dev(w), to_dev(dy)
        f_fwd, f_dg, f_wg = (int(t) for t in tags[li])
        rows = tile_sample(cfg.M, rng, 64)
        ncols = tile_sample(lin.N, rng, 64)
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


def check_layer_with_seeded_tags(cfg, layer, count):
    """Every linear of one layer of `cfg` under the layer's row of the seeded precision table: the three GEMMs
    through snip_linear_fwd / dgrad / wgrad (one tag per GEMM, BF16 tags included), FP32 outputs against the
    oracle on one sampled row per 128-row tile."""
    from paper_2602_01410_b200 import api
    tags = wl.precision_tags(cfg)[layer]                 # [linears, 3 gemms]
    rng = np.random.default_rng(1000 * cfg.index + layer)
    seen = set()
    for li, lin in enumerate(cfg.linears):
        x, w, dy = wl.linear_inputs(cfg, layer, li)
        X, W, DY = to_dev(x), to_dev(w), to_dev(dy)
        f_fwd, f_dg, f_wg = (int(t) for t in tags[li])
        seen.update((f_fwd, f_dg, f_wg))
        rows = tile_sample(cfg.M, rng, count)
        ncols = tile_sample(lin.N, rng, count)
        r, c = torch.from_numpy(rows).cuda(), torch.from_numpy(ncols).cuda()
        y, _, _ = api.snip_linear_fwd(X, W, f_fwd, f_fwd, api.OUT_FP32)
        got = y[r].cpu().numpy(); del y
        ref = orc.gemm_fwd(orc.quantize(np.ascontiguousarray(x[rows]), f_fwd, orc.BLOCK_ROW).xhat, orc.quantize(w, f_fwd, orc.BLOCK_BLK).xhat)
        assert rel_fro(got, ref) <= 2e-5, (cfg.name, layer, lin.name, "fwd", f_fwd)
        dx, _, _ = api.snip_linear_dgrad(DY, W, f_dg, f_dg, api.OUT_FP32)
        got = dx[r].cpu().numpy(); del dx
        ref = orc.gemm_dgrad(orc.quantize(np.ascontiguousarray(dy[rows]), f_dg, orc.BLOCK_ROW).xhat, orc.quantize(w, f_dg, orc.BLOCK_BLK).xhat)
        assert rel_fro(got, ref) <= 2e-5, (cfg.name, layer, lin.name, "dgrad", f_dg)
        dw, _, _ = api.snip_linear_wgrad(DY, X, f_wg, f_wg, api.OUT_FP32)
        got = dw[c].cpu().numpy(); del dw
        ref = orc.gemm_wgrad(orc.quantize(np.ascontiguousarray(dy[:, ncols]), f_wg, orc.BLOCK_COL).xhat, orc.quantize(x, f_wg, orc.BLOCK_COL).xhat)
        assert rel_fro(got, ref) <= 2e-5, (cfg.name, layer, lin.name, "wgrad", f_wg)
        del X, W, DY
        torch.cuda.empty_cache()
    return seen


@pytest.mark.parametrize("layer", [0, 1])
def test_3b_layers_with_their_seeded_precision_table(layer):
    # the 3B configuration: each GEMM drawn FP4 / FP8 / BF16 with p = .5 / .3 / .2; 8640 ragged as N and as K
    seen = check_layer_with_seeded_tags(wl.CONFIGS[2], layer, 64)
    assert len(seen) >= 2


def test_70b_layer_with_its_seeded_precision_table():
    # the 70B slice: seeded assignment with at least 80 % of the linear-layer FLOPs in FP4, the rest FP8
    cfg = wl.CONFIGS[4]
    tags = wl.precision_tags(cfg)
    flops = np.array([2.0 * cfg.M * l.K * l.N for l in cfg.linears])[None, :, None] * np.ones(tags.shape)
    assert (flops * (tags == FP4)).sum() >= 0.8 * flops.sum()
    assert set(np.unique(tags)) <= {FP8, FP4}
    check_layer_with_seeded_tags(cfg, 0, 64)


def test_7b_layer_stats_full_size():
    """snip_layer_stats on a 16384 x 4096 X, a 12288 x 4096 W and the matching dY (thousands of per-CTA partials in
    the fixed-order reduction) against the oracle: every sum within 1e-4."""
    from paper_2602_01410_b200 import api
    cfg = wl.CONFIGS[3]
    x, w, dy = wl.linear_inputs(cfg, 0, 0)
    M, K, N = cfg.M, 4096, 12288
    out = api.snip_layer_stats(X=to_dev(x), W=to_dev(w), dY=to_dev(dy), M=M, N=N, K=K).cpu().numpy()
    ref = orc.layer_stats(x, w, None, dy, None, None)
    names = ["X", "W", "Y", "dY", "dX", "dW"]
    for i, nme in enumerate(names):
        if nme in ref["sumsq"]:
            assert out[i] == pytest.approx(ref["sumsq"][nme], rel=1e-4), nme
    err = out[6:].reshape(3, 2, 3)
    for (nme, fmt, block), want in ref["sumsq_err"].items():
        ti = {"X": 0, "W": 1, "dY": 2}[nme]
        assert err[ti, fmt - 1, block] == pytest.approx(want, rel=1e-4), (nme, fmt, block)
    # a second run is bit-identical (fixed-order reduction)
    out2 = api.snip_layer_stats(X=to_dev(x), W=to_dev(w), dY=to_dev(dy), M=M, N=N, K=K).cpu().numpy()
    assert np.array_equal(out, out2)
