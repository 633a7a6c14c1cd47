"""Hardware-scaled GEMMs of the power-of-two scale option against the oracle run with the same rule."""
import numpy as np
import pytest
import torch

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

pytestmark = pytest.mark.gpu
from gpu_util import bf16_out_to_f64, rel_fro, to_dev  # noqa: E402

FP8, FP4 = 1, 2


def mx_three(api, x, w, dy, fa, fb, out_dtype):
    M, K = x.shape
    N = w.shape[0]
    X, W, DY = to_dev(x), to_dev(w), to_dev(dy)
    T = api.Q_TRANSPOSED
    outs = []
    # fwd: X rows, W blocks
    cx, sx, fx, _ = api.snip_quantize_mx(X, fa, api.BLOCK_ROW)
    cw, sw, fw, _ = api.snip_quantize_mx(W, fb, api.BLOCK_BLK)
    a = api.make_qtensor(cx, sx, M, K, fa, api.BLOCK_ROW); b = api.make_qtensor(cw, sw, N, K, fb, api.BLOCK_BLK)
    outs.append(api.snip_gemm_mx(api.OP_FWD, a, fx, b, fw, (M, N), out_dtype))
    # dgrad: dY rows, W blocks stored transposed
    cd, sd, fd, _ = api.snip_quantize_mx(DY, fa, api.BLOCK_ROW)
    cwt, swt, fwt, _ = api.snip_quantize_mx(W, fb, api.BLOCK_BLK, T)
    a = api.make_qtensor(cd, sd, M, N, fa, api.BLOCK_ROW); b = api.make_qtensor(cwt, swt, N, K, fb, api.BLOCK_BLK, True)
    outs.append(api.snip_gemm_mx(api.OP_DGRAD, a, fd, b, fwt, (M, K), out_dtype))
    # wgrad: dY and X columns, stored transposed
    cdc, sdc, fdc, _ = api.snip_quantize_mx(DY, fa, api.BLOCK_COL, T)
    cxc, sxc, fxc, _ = api.snip_quantize_mx(X, fb, api.BLOCK_COL, T)
    a = api.make_qtensor(cdc, sdc, M, N, fa, api.BLOCK_COL, True); b = api.make_qtensor(cxc, sxc, M, K, fb, api.BLOCK_COL, True)
    outs.append(api.snip_gemm_mx(api.OP_WGRAD, a, fdc, b, fxc, (N, K), out_dtype))
    torch.cuda.synchronize()
    return outs


@pytest.mark.parametrize("fa,fb", [(FP8, FP8), (FP4, FP4), (FP8, FP4), (FP4, FP8)])
@pytest.mark.parametrize("shape", [(128, 128, 256), (512, 512, 512), (256, 320, 192), (384, 640, 448)])
def test_three_gemms_hardware_scaled(fa, fb, shape):
    from paper_2602_01410_b200 import api
    M, K, N = shape
    rng = np.random.default_rng(M + K + N)
    x, w, dy = wl.make_x(rng, M, K, 0.01, 20.0), wl.make_w(rng, N, K), wl.make_dy(rng, M, N)
    want = (orc.linear_fwd(x, w, fa, fb, True)[0], orc.linear_dgrad(dy, w, fa, fb, True)[0], orc.linear_wgrad(dy, x, fa, fb, True)[0])
    got32 = mx_three(api, x, w, dy, fa, fb, api.OUT_FP32)
    got16 = mx_three(api, x, w, dy, fa, fb, api.OUT_BF16)
    for name, g32, g16, ref in zip(("fwd", "dgrad", "wgrad"), got32, got16, want):
        e32 = rel_fro(g32.cpu().numpy(), ref)
        assert e32 <= 1e-5, (name, e32)
        ref16 = orc.bf16_to_float(orc.round_to_bf16(ref))
        assert rel_fro(bf16_out_to_f64(g16), ref16) <= 1e-3, name


def test_same_operands_through_the_promotion_gemm():
    # the FP32 scales written by snip_quantize_mx feed the paper-rule GEMM kernel unchanged
    from paper_2602_01410_b200 import api
    M, K, N = 256, 384, 256
    rng = np.random.default_rng(3)
    x, w = wl.make_x(rng, M, K), wl.make_w(rng, N, K)
    cx, sx, fx, _ = api.snip_quantize_mx(to_dev(x), FP8, api.BLOCK_ROW)
    cw, sw, fw, _ = api.snip_quantize_mx(to_dev(w), FP8, api.BLOCK_BLK)
    a = api.make_qtensor(cx, sx, M, K, FP8, api.BLOCK_ROW); b = api.make_qtensor(cw, sw, N, K, FP8, api.BLOCK_BLK)
    y1 = api.snip_gemm_quantized(api.OP_FWD, a, b, (M, N), api.OUT_FP32)
    y2 = api.snip_gemm_mx(api.OP_FWD, a, fx, b, fw, (M, N), api.OUT_FP32)
    ref = orc.linear_fwd(x, w, FP8, FP8, True)[0]
    assert rel_fro(y1.cpu().numpy(), ref) <= 1e-5 and rel_fro(y2.cpu().numpy(), ref) <= 1e-5


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_linear_mx_entry_point_with_stats(fmt):
    from paper_2602_01410_b200 import api
    M, K, N = 384, 640, 448
    rng = np.random.default_rng(11)
    x, w, dy = wl.make_x(rng, M, K), wl.make_w(rng, N, K), wl.make_dy(rng, M, N)
    X, W, DY = to_dev(x), to_dev(w), to_dev(dy)
    y, sx, sw = api.snip_linear_mx(api.OP_FWD, X, W, fmt, fmt, api.OUT_FP32, want_stats=True)
    dx, _, _ = api.snip_linear_mx(api.OP_DGRAD, DY, W, fmt, fmt, api.OUT_FP32)
    dw, _, _ = api.snip_linear_mx(api.OP_WGRAD, DY, X, fmt, fmt, api.OUT_FP32)
    torch.cuda.synchronize()
    ref, qx, qw = orc.linear_fwd(x, w, fmt, fmt, True)
    assert rel_fro(y.cpu().numpy(), ref) <= 1e-5
    assert rel_fro(dx.cpu().numpy(), orc.linear_dgrad(dy, w, fmt, fmt, True)[0]) <= 1e-5
    assert rel_fro(dw.cpu().numpy(), orc.linear_wgrad(dy, x, fmt, fmt, True)[0]) <= 1e-5
    assert api.stats_to_host(sx)["sumsq_err"] == pytest.approx(qx.sumsq_err, rel=1e-4)
    assert api.stats_to_host(sw)["sumsq_err"] == pytest.approx(qw.sumsq_err, rel=1e-4)


def test_7b_qkv_sampled_rows_hardware_scaled():
    from paper_2602_01410_b200 import api
    cfg = wl.CONFIGS[3]
    x, w, dy = wl.linear_inputs(cfg, 0, 0)
    X, W = to_dev(x), to_dev(w)
    y, _, _ = api.snip_linear_mx(api.OP_FWD, X, W, FP4, FP4, api.OUT_BF16)
    torch.cuda.synchronize()
    rows = np.array([0, 17, 4095, 8191, 16383])
    qx = orc.quantize(np.ascontiguousarray(x[rows]), FP4, orc.BLOCK_ROW, True)
    qw = orc.quantize(w, FP4, orc.BLOCK_BLK, True)
    ref16 = orc.bf16_to_float(orc.round_to_bf16(orc.gemm_fwd(qx.xhat, qw.xhat)))
    assert rel_fro(bf16_out_to_f64(y[torch.from_numpy(rows).cuda()]), ref16) <= 1e-3


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_a_wait_that_runs_out_in_the_hardware_scaled_gemm(fmt):
    # Host-made condition (see test_gpu_gemm_kernels.py): the first stage's barrier expects 16 bytes more than the copies
    # deliver, every copy lands, the phase never completes.  With a 20 ms wait limit the kernel gives up by itself, releases
    # its tensor memory and raises the status word; nothing traps, faults or spins without a bound.
    from paper_2602_01410_b200 import api
    M, K, N = 512, 512, 256
    rng = np.random.default_rng(19)
    x, w = wl.make_x(rng, M, K), wl.make_w(rng, N, K)
    cx, sx, fx, _ = api.snip_quantize_mx(to_dev(x), fmt, api.BLOCK_ROW)
    cw, sw, fw, _ = api.snip_quantize_mx(to_dev(w), fmt, api.BLOCK_BLK)
    a = api.make_qtensor(cx, sx, M, K, fmt, api.BLOCK_ROW); b = api.make_qtensor(cw, sw, N, K, fmt, api.BLOCK_BLK)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    try:
        api.snip_debug_set(api.DEBUG_WAIT_LIMIT_NS, 20_000_000)
        api.snip_debug_set(api.DEBUG_TX_SKEW_BYTES, 16)
        api.snip_gemm_mx(api.OP_FWD, a, fx, b, fw, (M, N), api.OUT_FP32, ws=ws)
        torch.cuda.synchronize()
        assert api.snip_poll_status(ws) == api.ERR_TIMEOUT
    finally:
        api.snip_debug_set(api.DEBUG_TX_SKEW_BYTES, 0)
        api.snip_debug_set(api.DEBUG_WAIT_LIMIT_NS, 2_000_000_000)
    y = api.snip_gemm_mx(api.OP_FWD, a, fx, b, fw, (M, N), api.OUT_FP32, ws=ws)
    torch.cuda.synchronize()
    assert api.snip_poll_status(ws) == api.OK
    assert rel_fro(y.cpu().numpy(), orc.linear_fwd(x, w, fmt, fmt, True)[0]) <= 1e-5
