"""GPU parity of the three GEMMs of a linear layer against the CPU oracle.

Bar (relative Frobenius error): FP32 output vs the raw float64 oracle <= 1e-3; BF16 output vs the
oracle rounded to bf16 <= 1e-3 (bf16 rounding alone is ~1.7e-3 of the signal, so both sides are
rounded before comparing).  Codes and scales used by the GEMMs are checked bit-exact in
test_gpu_quantize.py."""
import numpy as np
import pytest
import torch

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

pytestmark = pytest.mark.gpu

FP8, FP4, BF16 = 1, 2, 0
TOL = 1e-3
PAIRS = [(BF16, BF16), (FP8, FP8), (FP4, FP4), (FP8, FP4), (FP4, FP8)]

from gpu_util import bf16_out_to_f64, rel_fro, to_dev  # noqa: E402


@pytest.fixture(scope="module")
def api():
    from paper_2602_01410_b200 import api as _api
    return _api


def inputs(M, K, N, seed):
    rng = np.random.default_rng(seed)
    return (wl.make_x(rng, M, K, 0.01, 20.0), wl.make_w(rng, N, K), wl.make_dy(rng, M, N))


def run_three(api, x, w, dy, fa, fb, out_dtype):
    X, W, DY = to_dev(x), to_dev(w), to_dev(dy)
    y, _, _ = api.snip_linear_fwd(X, W, fa, fb, out_dtype)
    dx, _, _ = api.snip_linear_dgrad(DY, W, fa, fb, out_dtype)
    dw, _, _ = api.snip_linear_wgrad(DY, X, fa, fb, out_dtype)
    torch.cuda.synchronize()
    return y, dx, dw


def oracle_three(x, w, dy, fa, fb):
    return (orc.linear_fwd(x, w, fa, fb)[0], orc.linear_dgrad(dy, w, fa, fb)[0], orc.linear_wgrad(dy, x, fa, fb)[0])


@pytest.mark.parametrize("fa,fb", PAIRS)
@pytest.mark.parametrize("shape", [(128, 128, 256), (512, 512, 512), (256, 320, 192), (384, 640, 448)])
def test_three_gemms_fp32_and_bf16_outputs(api, fa, fb, shape):
    M, K, N = shape
    x, w, dy = inputs(M, K, N, 100 + M + K + N)
    want = oracle_three(x, w, dy, fa, fb)
    got32 = run_three(api, x, w, dy, fa, fb, api.OUT_FP32)
    got16 = run_three(api, x, w, dy, fa, fb, api.OUT_BF16)
    for name, g32, g16, ref in zip(("fwd", "dgrad", "wgrad"), got32, got16, want):
        e32 = rel_fro(g32.cpu().numpy(), ref)
        assert e32 <= TOL, (name, e32)
        assert e32 <= 1e-5, (name, e32)          # FP32 accumulation should be far inside the bar
        ref16 = orc.bf16_to_float(orc.round_to_bf16(ref))
        e16 = rel_fro(bf16_out_to_f64(g16), ref16)
        assert e16 <= TOL, (name, e16)


@pytest.mark.parametrize("fa,fb", PAIRS)
def test_config0_precision_assignment(api, fa, fb):
    cfg = wl.CONFIGS[0]
    x, w, dy = wl.linear_inputs(cfg, 0, 0)
    want = oracle_three(x, w, dy, fa, fb)
    got = run_three(api, x, w, dy, fa, fb, api.OUT_FP32)
    for g, ref in zip(got, want):
        assert rel_fro(g.cpu().numpy(), ref) <= 1e-5


def test_gemm_on_prequantized_operands_and_accumulate(api):
    M, K, N = 256, 384, 256
    x, w, dy = inputs(M, K, N, 7)
    X, W = to_dev(x), to_dev(w)
    cx, sx, _, _ = api.snip_quantize(X, FP8, api.BLOCK_ROW)
    cw, sw, _, _ = api.snip_quantize(W, FP8, api.BLOCK_BLK)
    a = api.make_qtensor(cx, sx, M, K, FP8, api.BLOCK_ROW)
    b = api.make_qtensor(cw, sw, N, K, FP8, api.BLOCK_BLK)
    y = api.snip_gemm_quantized(api.OP_FWD, a, b, (M, N), api.OUT_FP32)
    ref = orc.linear_fwd(x, w, FP8, FP8)[0]
    assert rel_fro(y.cpu().numpy(), ref) <= 1e-5
    # accumulate adds a second product into the same FP32 buffer
    y2 = api.snip_gemm_quantized(api.OP_FWD, a, b, (M, N), api.OUT_FP32, accumulate=True, out=y.clone())
    assert rel_fro(y2.cpu().numpy(), 2 * ref) <= 1e-5
    # bit-identical on rerun (catches races in the shared-memory / tensor-memory hand-offs)
    y3 = api.snip_gemm_quantized(api.OP_FWD, a, b, (M, N), api.OUT_FP32)
    assert torch.equal(y, y3)


def test_lossless_inputs_give_the_plain_product(api):
    # representable values with power-of-two tile scales: quantization is exact, so the GEMM must
    # reproduce the plain matmul (pins scale indexing and transposes on the GPU side too)
    from test_oracle_gemm import lossless
    M, K, N = 256, 384, 192
    for fmt in (FP8, FP4):
        x, w, dy = lossless((M, K), fmt, 5), lossless((N, K), fmt, 6), lossless((M, N), fmt, 7)
        xf, wf, dyf = orc.bf16_to_float(x), orc.bf16_to_float(w), orc.bf16_to_float(dy)
        y, dx, dw = run_three(api, x, w, dy, fmt, fmt, api.OUT_FP32)
        assert rel_fro(y.cpu().numpy(), xf @ wf.T) <= 1e-6
        assert rel_fro(dx.cpu().numpy(), dyf @ wf) <= 1e-6
        assert rel_fro(dw.cpu().numpy(), dyf.T @ xf) <= 1e-6


def test_unsupported_and_bad_arguments(api):
    X = torch.zeros(128, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(api.SnipError) as e:
        api.snip_linear_fwd(X, X, BF16, FP8)
    assert e.value.status == api.ERR_UNSUPPORTED
    with pytest.raises(api.SnipError) as e:
        api.snip_linear_wgrad(X, X, FP8, FP8, api.OUT_BF16, accumulate=True)
    assert e.value.status == api.ERR_UNSUPPORTED
    ws = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    assert api.snip_poll_status(ws) == api.OK


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_sampled_rows_of_a_1b_linear(api, fmt):
    # one linear of the 1B configuration at its full size; the oracle computes 48 sampled output
    # rows / columns of each GEMM in full
    cfg = wl.CONFIGS[1]
    x, w, dy = wl.linear_inputs(cfg, 0, 3)      # o-proj 2048 -> 2048, M = 8192
    y, dx, dw = run_three(api, x, w, dy, fmt, fmt, api.OUT_FP32)
    rng = np.random.default_rng(11)
    rows = np.sort(rng.choice(cfg.M, 48, replace=False))
    qx, qw = orc.quantize(x, fmt, orc.BLOCK_ROW), orc.quantize(w, fmt, orc.BLOCK_BLK)
    ref = orc.gemm_fwd(qx.xhat[rows], qw.xhat)
    assert rel_fro(y[rows].cpu().numpy(), ref) <= 1e-5
    qdy = orc.quantize(dy, fmt, orc.BLOCK_ROW)
    ref = orc.gemm_dgrad(qdy.xhat[rows], qw.xhat)
    assert rel_fro(dx[rows].cpu().numpy(), ref) <= 1e-5
    qdyc, qxc = orc.quantize(dy, fmt, orc.BLOCK_COL), orc.quantize(x, fmt, orc.BLOCK_COL)
    nrows = np.sort(rng.choice(2048, 48, replace=False))
    ref = orc.gemm_wgrad(np.ascontiguousarray(qdyc.xhat[:, nrows]), qxc.xhat)
    assert rel_fro(dw[nrows].cpu().numpy(), ref) <= 1e-5
