"""Block-32 power-of-two scale option (1x32 tiles as stored, 32x1 tiles transposed) against the oracle run with the
same tiles and rule: codes, scales and scale-factor atoms bit for bit, statistics within 1e-4, the three
hardware-scaled GEMMs within 1e-5 (FP32 output) / 1e-3 (bf16 output)."""
import numpy as np
import pytest
import torch

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

pytestmark = pytest.mark.gpu
from gpu_util import bf16_out_to_f64, rel_fro, to_dev  # noqa: E402

FP8, FP4 = 1, 2


@pytest.fixture(scope="module")
def api():
    from paper_2602_01410_b200 import api as _api
    return _api


def spread_inputs(rng, rows, cols):
    # magnitudes that change from one 32-long piece to the next, so that the four scales of a 128-long tile differ
    x = rng.standard_normal((rows, cols)) * np.exp(2.0 * rng.standard_normal((rows, cols // 32))).repeat(32, axis=1)
    x *= np.exp(1.5 * rng.standard_normal((rows // 32, cols))).repeat(32, axis=0)
    return wl.to_bf16_bits(x.astype(np.float32))


def check_output(api, got_codes, got_scales, got_sf, got_stats, q, transposed):
    assert np.array_equal(got_codes.cpu().numpy()[:q.packed(transposed).size], q.packed(transposed).reshape(-1))
    assert np.array_equal(got_scales.cpu().numpy(), q.scales.reshape(-1))
    if got_sf is not None:
        assert np.array_equal(got_sf.cpu().numpy(), orc.sf_atoms(q, transposed))
    if got_stats is not None:
        st = api.stats_to_host(got_stats)
        assert st["sumsq_x"] == pytest.approx(q.sumsq_x, rel=1e-6)
        assert st["sumsq_err"] == pytest.approx(q.sumsq_err, rel=1e-4)


# whole tiles; every dimension ending in a 64-wide tile (two of a tile's four pieces lie outside); several tiles per CTA
SHAPES = [(128, 128), (256, 384), (320, 448), (1024, 1600)]


@pytest.mark.parametrize("fmt", [FP8, FP4])
@pytest.mark.parametrize("shape", SHAPES)
def test_single_output_kinds_bit_exact(api, fmt, shape):
    rows, cols = shape
    x = spread_inputs(np.random.default_rng(rows + cols + fmt), rows, cols)
    X = to_dev(x)
    c, s, sf, st = api.snip_quantize_mx(X, fmt, api.BLOCK_ROW32, api.Q_STATS)
    torch.cuda.synchronize()
    check_output(api, c, s, sf, st, orc.quantize(x, fmt, orc.BLOCK_ROW32, True), False)
    c, s, sf, st = api.snip_quantize_mx(X, fmt, api.BLOCK_COL32, api.Q_STATS | api.Q_TRANSPOSED)
    torch.cuda.synchronize()
    check_output(api, c, s, sf, st, orc.quantize(x, fmt, orc.BLOCK_COL32, True), True)
    # without statistics the codes do not change
    c2, s2, sf2, _ = api.snip_quantize_mx(X, fmt, api.BLOCK_COL32, api.Q_TRANSPOSED)
    torch.cuda.synchronize()
    n = rows * cols // (2 if fmt == FP4 else 1)      # FP4 buffers of ragged shapes end in slack bytes that nothing writes
    assert torch.equal(c[:n], c2[:n]) and torch.equal(s, s2) and torch.equal(sf, sf2)


@pytest.mark.parametrize("fa,fb", [(FP8, FP8), (FP4, FP4), (FP8, FP4), (FP4, FP8)])
@pytest.mark.parametrize("shape", SHAPES)
def test_two_output_form_bit_exact(api, fa, fb, shape):
    rows, cols = shape
    x = spread_inputs(np.random.default_rng(7 * rows + cols), rows, cols)
    a, b = api.snip_quantize_dual(to_dev(x), api.DUAL_ROW32_COL32T, fa, fb, pow2_scale=True, want_sf=True)
    torch.cuda.synchronize()
    check_output(api, a["codes"], a["scales"], a["sf"], a["stats"], orc.quantize(x, fa, orc.BLOCK_ROW32, True), False)
    check_output(api, b["codes"], b["scales"], b["sf"], b["stats"], orc.quantize(x, fb, orc.BLOCK_COL32, True), True)


def test_refused_combinations(api):
    X = to_dev(spread_inputs(np.random.default_rng(1), 128, 128))
    with pytest.raises(RuntimeError):     # 32-long tiles exist for the power-of-two rule only
        api.snip_quantize(X, FP8, api.BLOCK_ROW32)
    with pytest.raises(RuntimeError):     # 1x32 tiles are stored as they are, 32x1 tiles transposed
        api.snip_quantize_mx(X, FP8, api.BLOCK_ROW32, api.Q_TRANSPOSED)
    with pytest.raises(RuntimeError):
        api.snip_quantize_mx(X, FP8, api.BLOCK_COL32)
    with pytest.raises(RuntimeError):
        api.snip_quantize_dual(X, api.DUAL_ROW32_COL32T, FP8, FP8, pow2_scale=False)


def three_gemms(api, x, w, dy, fa, fb, out_dtype):
    M, K = x.shape
    N = w.shape[0]
    X, W, DY = to_dev(x), to_dev(w), to_dev(dy)
    kind = api.DUAL_ROW32_COL32T
    xa, xt = api.snip_quantize_dual(X, kind, fa, fb, pow2_scale=True, want_sf=True, want_stats=False)     # fwd: A = X;  wgrad: B = X^T
    wa, wt = api.snip_quantize_dual(W, kind, fb, fb, pow2_scale=True, want_sf=True, want_stats=False)     # fwd: B = W;  dgrad: B = W^T
    da, dt = api.snip_quantize_dual(DY, kind, fa, fa, pow2_scale=True, want_sf=True, want_stats=False)    # dgrad: A = dY; wgrad: A = dY^T
    q = api.make_qtensor
    outs = [
        api.snip_gemm_mx(api.OP_FWD, q(xa["codes"], xa["scales"], M, K, fa, api.BLOCK_ROW32), xa["sf"],
                         q(wa["codes"], wa["scales"], N, K, fb, api.BLOCK_ROW32), wa["sf"], (M, N), out_dtype),
        api.snip_gemm_mx(api.OP_DGRAD, q(da["codes"], da["scales"], M, N, fa, api.BLOCK_ROW32), da["sf"],
                         q(wt["codes"], wt["scales"], N, K, fb, api.BLOCK_COL32, True), wt["sf"], (M, K), out_dtype),
        api.snip_gemm_mx(api.OP_WGRAD, q(dt["codes"], dt["scales"], M, N, fa, api.BLOCK_COL32, True), dt["sf"],
                         q(xt["codes"], xt["scales"], M, K, fb, api.BLOCK_COL32, True), xt["sf"], (N, K), out_dtype),
    ]
    torch.cuda.synchronize()
    return outs


@pytest.mark.parametrize("fa,fb", [(FP8, FP8), (FP4, FP4), (FP8, FP4), (FP4, FP8)])
@pytest.mark.parametrize("shape", [(128, 128, 256), (512, 512, 512), (256, 320, 192), (384, 640, 448)])
def test_three_gemms_with_32_long_tiles(api, fa, fb, shape):
    M, K, N = shape
    rng = np.random.default_rng(M + K + N)
    x, w, dy = spread_inputs(rng, M, K), wl.make_w(rng, N, K), wl.make_dy(rng, M, N)
    # wgrad multiplies dY (format fa) with X (format fb); fwd X (fa) with W (fb); dgrad dY (fa) with W (fb)
    want = (orc.linear_fwd(x, w, fa, fb, 2)[0], orc.linear_dgrad(dy, w, fa, fb, 2)[0], orc.linear_wgrad(dy, x, fa, fb, 2)[0])
    got32 = three_gemms(api, x, w, dy, fa, fb, api.OUT_FP32)
    got16 = three_gemms(api, x, w, dy, fa, fb, api.OUT_BF16)
    for name, g32, g16, ref in zip(("fwd", "dgrad", "wgrad"), got32, got16, want):
        e32 = rel_fro(g32.cpu().numpy(), ref)
        assert e32 <= 1e-5, (name, e32)
        assert rel_fro(bf16_out_to_f64(g16), orc.bf16_to_float(orc.round_to_bf16(ref))) <= 1e-3, name


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_fwd_bwd_with_32_long_tiles(api, fmt):
    M, K, N = 384, 640, 448
    rng = np.random.default_rng(21)
    x, w, dy = spread_inputs(rng, M, K), wl.make_w(rng, N, K), wl.make_dy(rng, M, N)
    y, dx, dw, stats = api.snip_linear_fwd_bwd(to_dev(x), to_dev(w), to_dev(dy), fmt, fmt, fmt, api.OUT_FP32, pow2_scale=2)
    torch.cuda.synchronize()
    ref_y, qx, qw = orc.linear_fwd(x, w, fmt, fmt, 2)
    ref_dx, qdy, qwt = orc.linear_dgrad(dy, w, fmt, fmt, 2)
    ref_dw, qdyc, qxc = orc.linear_wgrad(dy, x, fmt, fmt, 2)
    assert rel_fro(y.cpu().numpy(), ref_y) <= 1e-5
    assert rel_fro(dx.cpu().numpy(), ref_dx) <= 1e-5
    assert rel_fro(dw.cpu().numpy(), ref_dw) <= 1e-5
    # statistics of the six copies: X (1x32, 32x1), W (1x32, 32x1), dY (1x32, 32x1)
    for i, q in enumerate((qx, qxc, qw, qwt, qdy, qdyc)):
        assert api.stats_to_host(stats[24 * i:24 * i + 24])["sumsq_err"] == pytest.approx(q.sumsq_err, rel=1e-4), i
    # finer tiles: never a larger quantization error than the 128-long tiles of the same rule
    _, _, _, stats128 = api.snip_linear_fwd_bwd(to_dev(x), to_dev(w), to_dev(dy), fmt, fmt, fmt, api.OUT_FP32, pow2_scale=1)
    torch.cuda.synchronize()
    for i in (0, 1, 4, 5):
        assert api.stats_to_host(stats[24 * i:24 * i + 24])["sumsq_err"] <= api.stats_to_host(stats128[24 * i:24 * i + 24])["sumsq_err"]


def test_7b_activation_tensor_bit_exact(api):
    cfg = wl.CONFIGS[3]
    x, _, _ = wl.linear_inputs(cfg, 0, 0)      # 16384 x 4096
    a, b = api.snip_quantize_dual(to_dev(x), api.DUAL_ROW32_COL32T, FP4, FP8, pow2_scale=True, want_sf=True)
    torch.cuda.synchronize()
    check_output(api, a["codes"], a["scales"], a["sf"], a["stats"], orc.quantize(x, FP4, orc.BLOCK_ROW32, True), False)
    check_output(api, b["codes"], b["scales"], b["sf"], b["stats"], orc.quantize(x, FP8, orc.BLOCK_COL32, True), True)


@pytest.mark.parametrize("shape", [(256, 384), (320, 448)])
def test_stochastic_rounding_of_fp4_outputs(api, shape):
    # Sec. 6.1: FP4 output gradients are rounded stochastically; the 32-long tile kinds take the same rule and generator
    rows, cols = shape
    x = spread_inputs(np.random.default_rng(rows + 3 * cols), rows, cols)
    seeds = (77, 0xFEEDFACE1)
    a, b = api.snip_quantize_dual(to_dev(x), api.DUAL_ROW32_COL32T, FP4, FP4, pow2_scale=True, want_sf=True, sr_seeds=seeds)
    torch.cuda.synchronize()
    check_output(api, a["codes"], a["scales"], a["sf"], a["stats"], orc.quantize(x, FP4, orc.BLOCK_ROW32, True, sr_seed=seeds[0]), False)
    check_output(api, b["codes"], b["scales"], b["sf"], b["stats"], orc.quantize(x, FP4, orc.BLOCK_COL32, True, sr_seed=seeds[1]), True)
    # one stochastic FP4 output next to a nearest-even FP8 output
    a, b = api.snip_quantize_dual(to_dev(x), api.DUAL_ROW32_COL32T, FP8, FP4, pow2_scale=True, want_sf=True, sr_seeds=(None, 5))
    torch.cuda.synchronize()
    check_output(api, a["codes"], a["scales"], a["sf"], a["stats"], orc.quantize(x, FP8, orc.BLOCK_ROW32, True), False)
    check_output(api, b["codes"], b["scales"], b["sf"], b["stats"], orc.quantize(x, FP4, orc.BLOCK_COL32, True, sr_seed=5), True)
