"""Two-level (NVFP4-style) option against the oracle: E2M1 codes and E4M3 scale bytes (as atoms) bit for bit, statistics
within 1e-4, the three block-scaled GEMMs within 1e-5 (FP32 output) / 1e-3 (bf16 output) — first on operands quantized by
the oracle (the GEMM alone), then on the library's own quantizer output."""
import numpy as np
import pytest
import torch

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

pytestmark = pytest.mark.gpu
from gpu_util import bf16_out_to_f64, rel_fro, to_dev  # noqa: E402

FP4 = 2


@pytest.fixture(scope="module")
def api():
    from paper_2602_01410_b200 import api as _api
    return _api


def spread(rng, rows, cols, scale):
    # magnitudes that change from one 16-long tile to the next, in both directions
    x = rng.standard_normal((rows, cols)) * np.exp(1.2 * rng.standard_normal((rows, cols // 16))).repeat(16, axis=1)
    x *= np.exp(0.8 * rng.standard_normal((rows // 16, cols))).repeat(16, axis=0) * scale
    return wl.to_bf16_bits(x.astype(np.float32))


def amax_of(bits):
    return float(np.abs(orc.bf16_to_float(bits)).max())


def dev_u8(a):
    return torch.from_numpy(np.ascontiguousarray(a).reshape(-1)).cuda()


def dev_f32(v):
    return torch.tensor([v], dtype=torch.float32, device="cuda")


def oracle_operand(api, q, transposed, block):
    """Device copies of an oracle-quantized operand: qtensor, atoms, bound."""
    codes = dev_u8(q.packed(transposed))
    pad = torch.zeros(64, dtype=torch.uint8, device="cuda")          # tail slack the 4-bit reads may touch
    codes = torch.cat([codes, pad])
    atoms = dev_u8(orc.nvfp4_atoms(q, transposed))
    return api.make_qtensor(codes, None, q.rows, q.cols, FP4, block, transposed), atoms, codes


SHAPES = [(128, 128, 256), (512, 512, 512), (256, 320, 192), (384, 640, 448), (1024, 1536, 768)]


@pytest.mark.parametrize("shape", SHAPES)
def test_gemms_on_oracle_operands(api, shape):
    M, K, N = shape
    rng = np.random.default_rng(M + K + N)
    x, w, dy = spread(rng, M, K, 1.0), spread(rng, N, K, 0.02), spread(rng, M, N, 1e-3)
    ax, aw, ady = dev_f32(amax_of(x)), dev_f32(amax_of(w)), dev_f32(amax_of(dy))
    cases = (("fwd", api.OP_FWD, x, w, ax, aw, (False, api.BLOCK_ROW16), (False, api.BLOCK_ROW16), (M, N)),
             ("dgrad", api.OP_DGRAD, dy, w, ady, aw, (False, api.BLOCK_ROW16), (True, api.BLOCK_COL16), (M, K)),
             ("wgrad", api.OP_WGRAD, dy, x, ady, ax, (True, api.BLOCK_COL16), (True, api.BLOCK_COL16), (N, K)))
    for name, op, a_bits, b_bits, am_a, am_b, (ta, ba), (tb, bb), oshape in cases:
        ref, qa, qb = orc.linear_nvfp4(name, a_bits, b_bits)
        a, sfa, keep_a = oracle_operand(api, qa, ta, ba)
        b, sfb, keep_b = oracle_operand(api, qb, tb, bb)
        out32 = api.snip_gemm_nvfp4(op, a, sfa, am_a, b, sfb, am_b, oshape, api.OUT_FP32)
        out16 = api.snip_gemm_nvfp4(op, a, sfa, am_a, b, sfb, am_b, oshape, api.OUT_BF16)
        torch.cuda.synchronize()
        e = rel_fro(out32.cpu().numpy(), ref)
        assert e <= 1e-5, (name, e)
        assert rel_fro(bf16_out_to_f64(out16), orc.bf16_to_float(orc.round_to_bf16(ref))) <= 1e-3, name
        again = api.snip_gemm_nvfp4(op, a, sfa, am_a, b, sfb, am_b, oshape, api.OUT_FP32)
        torch.cuda.synchronize()
        assert torch.equal(again, out32)


def check_copy(api, got, q, transposed):
    n = q.rows * q.cols // 2
    assert np.array_equal(got["codes"].cpu().numpy()[:n], q.packed(transposed).reshape(-1))
    assert np.array_equal(got["sf"].cpu().numpy(), orc.nvfp4_atoms(q, transposed))
    if got["stats"] is not None:
        st = api.stats_to_host(got["stats"])
        assert st["sumsq_x"] == pytest.approx(q.sumsq_x, rel=1e-6)
        assert st["sumsq_err"] == pytest.approx(q.sumsq_err, rel=1e-4)


@pytest.mark.parametrize("scale", [1.0, 1e-3, 40.0])
@pytest.mark.parametrize("shape", [(128, 128), (256, 384), (320, 448), (1024, 1600)])
def test_quantizer_bit_exact(api, shape, scale):
    rows, cols = shape
    x = spread(np.random.default_rng(rows * 3 + cols), rows, cols, scale)
    x[5, 16:32] = 0            # an empty 1x16 tile
    a, b = api.snip_quantize_nvfp4_dual(to_dev(x), dev_f32(amax_of(x)))
    torch.cuda.synchronize()
    check_copy(api, a, orc.quantize_nvfp4(x, False), False)
    check_copy(api, b, orc.quantize_nvfp4(x, True), True)
    # without statistics: the same codes and bytes
    a2, b2 = api.snip_quantize_nvfp4_dual(to_dev(x), dev_f32(amax_of(x)), want_stats=False)
    torch.cuda.synchronize()
    n = rows * cols // 2
    assert torch.equal(a["codes"][:n], a2["codes"][:n]) and torch.equal(a["sf"], a2["sf"])
    assert torch.equal(b["codes"][:n], b2["codes"][:n]) and torch.equal(b["sf"], b2["sf"])


def test_a_bound_that_is_an_estimate(api):
    # the bound may come from an earlier step: half the true maximum saturates the largest values, twice it loses a binade
    x = spread(np.random.default_rng(9), 256, 256, 0.3)
    for factor in (0.5, 2.0, 0.0):
        bound = factor * amax_of(x)
        a, b = api.snip_quantize_nvfp4_dual(to_dev(x), dev_f32(bound))
        torch.cuda.synchronize()
        check_copy(api, a, orc.quantize_nvfp4(x, False, tensor_amax=bound), False)
        check_copy(api, b, orc.quantize_nvfp4(x, True, tensor_amax=bound), True)


def test_quantize_then_multiply(api):
    M, K, N = 384, 640, 448
    rng = np.random.default_rng(77)
    x, w, dy = spread(rng, M, K, 1.0), spread(rng, N, K, 0.02), spread(rng, M, N, 1e-3)
    ax, aw, ady = dev_f32(amax_of(x)), dev_f32(amax_of(w)), dev_f32(amax_of(dy))
    xa, xt = api.snip_quantize_nvfp4_dual(to_dev(x), ax, want_stats=False)
    wa, wt = api.snip_quantize_nvfp4_dual(to_dev(w), aw, want_stats=False)
    da, dt = api.snip_quantize_nvfp4_dual(to_dev(dy), ady, want_stats=False)
    q = api.make_qtensor
    y = api.snip_gemm_nvfp4(api.OP_FWD, q(xa["codes"], None, M, K, FP4, api.BLOCK_ROW16), xa["sf"], ax,
                            q(wa["codes"], None, N, K, FP4, api.BLOCK_ROW16), wa["sf"], aw, (M, N), api.OUT_FP32)
    dx = api.snip_gemm_nvfp4(api.OP_DGRAD, q(da["codes"], None, M, N, FP4, api.BLOCK_ROW16), da["sf"], ady,
                             q(wt["codes"], None, N, K, FP4, api.BLOCK_COL16, True), wt["sf"], aw, (M, K), api.OUT_FP32)
    dw = api.snip_gemm_nvfp4(api.OP_WGRAD, q(dt["codes"], None, M, N, FP4, api.BLOCK_COL16, True), dt["sf"], ady,
                             q(xt["codes"], None, M, K, FP4, api.BLOCK_COL16, True), xt["sf"], ax, (N, K), api.OUT_FP32)
    torch.cuda.synchronize()
    assert rel_fro(y.cpu().numpy(), orc.linear_nvfp4("fwd", x, w)[0]) <= 1e-5
    assert rel_fro(dx.cpu().numpy(), orc.linear_nvfp4("dgrad", dy, w)[0]) <= 1e-5
    assert rel_fro(dw.cpu().numpy(), orc.linear_nvfp4("wgrad", dy, x)[0]) <= 1e-5


def test_7b_activation_tensor_bit_exact(api):
    cfg = wl.CONFIGS[3]
    x, _, _ = wl.linear_inputs(cfg, 0, 0)      # 16384 x 4096
    a, b = api.snip_quantize_nvfp4_dual(to_dev(x), dev_f32(amax_of(x)))
    torch.cuda.synchronize()
    check_copy(api, a, orc.quantize_nvfp4(x, False), False)
    check_copy(api, b, orc.quantize_nvfp4(x, True), True)


@pytest.mark.parametrize("shape", [(256, 384), (320, 448)])
def test_stochastic_rounding_bit_exact(api, shape):
    # Sec. 6.1: output gradients in FP4 are rounded stochastically; same rule and generator as snip_quantize_sr
    rows, cols = shape
    x = spread(np.random.default_rng(rows + 5 * cols), rows, cols, 1e-3)
    seed = 0x1234ABCD5
    a, b = api.snip_quantize_nvfp4_dual(to_dev(x), dev_f32(amax_of(x)), sr_seed=seed)
    torch.cuda.synchronize()
    check_copy(api, a, orc.quantize_nvfp4(x, False, sr_seed=seed), False)
    check_copy(api, b, orc.quantize_nvfp4(x, True, sr_seed=seed), True)
    a2, b2 = api.snip_quantize_nvfp4_dual(to_dev(x), dev_f32(amax_of(x)), sr_seed=seed + 1)
    torch.cuda.synchronize()
    n = rows * cols // 2
    assert not torch.equal(a["codes"][:n], a2["codes"][:n]) and torch.equal(a["sf"], a2["sf"])


def test_fwd_bwd_composition(api):
    M, K, N = 384, 640, 448
    rng = np.random.default_rng(78)
    x, w, dy = spread(rng, M, K, 1.0), spread(rng, N, K, 0.02), spread(rng, M, N, 1e-3)
    bounds = torch.tensor([amax_of(x), amax_of(w), amax_of(dy)], dtype=torch.float32, device="cuda")
    y, dx, dw, stats = api.snip_linear_fwd_bwd_nvfp4(to_dev(x), to_dev(w), to_dev(dy), bounds, api.OUT_FP32)
    torch.cuda.synchronize()
    ref_y, qx, qw = orc.linear_nvfp4("fwd", x, w)
    ref_dx, qdy, qwt = orc.linear_nvfp4("dgrad", dy, w)
    ref_dw, qdyc, qxc = orc.linear_nvfp4("wgrad", dy, x)
    assert rel_fro(y.cpu().numpy(), ref_y) <= 1e-5
    assert rel_fro(dx.cpu().numpy(), ref_dx) <= 1e-5
    assert rel_fro(dw.cpu().numpy(), ref_dw) <= 1e-5
    for i, q in enumerate((qx, qxc, qw, qwt, qdy, qdyc)):
        assert api.stats_to_host(stats[24 * i:24 * i + 24])["sumsq_err"] == pytest.approx(q.sumsq_err, rel=1e-4), i
    # stochastic rounding of dY changes dX and dW only
    y2, dx2, dw2, _ = api.snip_linear_fwd_bwd_nvfp4(to_dev(x), to_dev(w), to_dev(dy), bounds, api.OUT_FP32, dy_sr_seed=11)
    torch.cuda.synchronize()
    assert torch.equal(y2, y) and not torch.equal(dx2, dx)
    want_dx = orc.gemm_dgrad(orc.quantize_nvfp4(dy, False, sr_seed=11).xhat, qwt.xhat)
    assert rel_fro(dx2.cpu().numpy(), want_dx) <= 1e-5


def test_a_wait_that_runs_out_reports_timeout(api):
    # the host-made condition of test_gpu_gemm_kernels.py (a stage barrier that expects 16 bytes too many, a 20 ms wait limit)
    M, K, N = 512, 512, 256
    rng = np.random.default_rng(79)
    x, w = spread(rng, M, K, 1.0), spread(rng, N, K, 0.02)
    ax, aw = dev_f32(amax_of(x)), dev_f32(amax_of(w))
    xa, _ = api.snip_quantize_nvfp4_dual(to_dev(x), ax, want_stats=False)
    wa, _ = api.snip_quantize_nvfp4_dual(to_dev(w), aw, want_stats=False)
    a = api.make_qtensor(xa["codes"], None, M, K, FP4, api.BLOCK_ROW16)
    b = api.make_qtensor(wa["codes"], None, N, K, FP4, api.BLOCK_ROW16)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    try:
        api.snip_debug_set(api.DEBUG_WAIT_LIMIT_NS, 20_000_000)
        api.snip_debug_set(api.DEBUG_TX_SKEW_BYTES, 16)
        api.snip_gemm_nvfp4(api.OP_FWD, a, xa["sf"], ax, b, wa["sf"], aw, (M, N), api.OUT_FP32, ws=ws)
        torch.cuda.synchronize()
        assert api.snip_poll_status(ws) == api.ERR_TIMEOUT
    finally:
        api.snip_debug_set(api.DEBUG_TX_SKEW_BYTES, 0)
        api.snip_debug_set(api.DEBUG_WAIT_LIMIT_NS, 2_000_000_000)
    y = api.snip_gemm_nvfp4(api.OP_FWD, a, xa["sf"], ax, b, wa["sf"], aw, (M, N), api.OUT_FP32, ws=ws)
    torch.cuda.synchronize()
    assert api.snip_poll_status(ws) == api.OK
    assert rel_fro(y.cpu().numpy(), orc.linear_nvfp4("fwd", x, w)[0]) <= 1e-5
