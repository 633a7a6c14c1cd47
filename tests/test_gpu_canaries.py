"""Canary bytes behind every output buffer on shapes that end in 64-wide tiles: a kernel that writes past the
size the library reports (snip_quantize_sizes, the GEMM's output shape) would be seen here.  Stands in for a
memory checker; the transposed writers clip by hand and the GEMM's output boxes are clipped by the TMA unit."""
import numpy as np
import pytest
import torch

from paper_2602_01410_b200 import workloads as wl

pytestmark = pytest.mark.gpu
from gpu_util import to_dev  # noqa: E402

FP8, FP4 = 1, 2
CANARY, PAD = 0xC5, 4096


def guarded(nbytes, dtype=torch.uint8):
    """A buffer of `nbytes` bytes with PAD canary bytes before and after it; returns (whole, view)."""
    whole = torch.full((PAD + nbytes + PAD,), CANARY, dtype=torch.uint8, device="cuda")
    view = whole[PAD:PAD + nbytes]
    return whole, (view if dtype == torch.uint8 else view.view(dtype))


def intact(whole, nbytes):
    w = whole.cpu().numpy()
    return bool((w[:PAD] == CANARY).all() and (w[PAD + nbytes:] == CANARY).all())


@pytest.mark.parametrize("fmt", [FP8, FP4])
@pytest.mark.parametrize("block,transposed", [(0, False), (1, True), (2, False), (2, True)])
@pytest.mark.parametrize("shape", [(320, 448), (192, 64), (64, 704)])
def test_quantizer_outputs_stay_inside_their_buffers(fmt, block, transposed, shape):
    from paper_2602_01410_b200 import api
    rows, cols = shape
    x = to_dev(wl.make_x(np.random.default_rng(rows + cols), rows, cols, 0.01, 20.0))
    flags = api.Q_STATS | (api.Q_TRANSPOSED if transposed else 0)
    cb, sb, wb = api.snip_quantize_sizes(rows, cols, fmt, block, flags)
    wc, codes = guarded(cb)
    ws_, scales = guarded(sb, torch.float32)
    wst, stats = guarded(32)
    ww, ws = guarded(wb)
    api.snip_quantize(x, fmt, block, flags, codes=codes, scales=scales, stats=stats[:24], ws=ws)
    torch.cuda.synchronize()
    assert intact(wc, cb) and intact(ws_, sb) and intact(wst, 32) and intact(ww, wb)
    # and the call did write its outputs
    assert not (scales.view(torch.uint8).cpu().numpy() == CANARY).all()


@pytest.mark.parametrize("fmt", [FP8, FP4])
@pytest.mark.parametrize("shape", [(320, 448), (192, 320)])
def test_two_output_quantizer_stays_inside_its_buffers(fmt, shape):
    from paper_2602_01410_b200 import api
    rows, cols = shape
    x = to_dev(wl.make_x(np.random.default_rng(5), rows, cols, 0.01, 20.0))
    for kind, blocks in ((api.DUAL_ROW_COLT, (api.BLOCK_ROW, api.BLOCK_COL)), (api.DUAL_BLK_BLKT, (api.BLOCK_BLK, api.BLOCK_BLK))):
        bufs, wholes = [], []
        for i in range(2):
            cb, sb, _ = api.snip_quantize_sizes(rows, cols, fmt, blocks[i], api.Q_TRANSPOSED if i else 0)
            wc, codes = guarded(cb); wsc, scales = guarded(sb, torch.float32); wst, stats = guarded(32)
            bufs.append({"codes": codes, "scales": scales, "sf": None, "stats": stats})
            wholes += [(wc, cb), (wsc, sb), (wst, 32)]
        wb = api.snip_quantize_dual_workspace(rows, cols)
        ww, ws = guarded(wb)
        api.snip_quantize_dual(x, kind, fmt, fmt, bufs=tuple(bufs), ws=ws)
        torch.cuda.synchronize()
        assert all(intact(w, n) for w, n in wholes) and intact(ww, wb)


@pytest.mark.parametrize("choice", [1, 2])
@pytest.mark.parametrize("fa,fb", [(FP8, FP8), (FP4, FP4), (FP8, FP4), (FP4, FP8)])
@pytest.mark.parametrize("out_dtype", [0, 1])
def test_gemm_outputs_stay_inside_their_buffers(choice, fa, fb, out_dtype):
    # M, K, N all ending in a 64-wide tile: ragged output rows and columns, ragged contraction
    from paper_2602_01410_b200 import api
    M, K, N = 320, 448, 192
    rng = np.random.default_rng(9)
    x, w, dy = wl.make_x(rng, M, K, 0.01, 20.0), wl.make_w(rng, N, K), wl.make_dy(rng, M, N)
    X, W, DY = to_dev(x), to_dev(w), to_dev(dy)
    esz = 4 if out_dtype == api.OUT_FP32 else 2
    dt = torch.float32 if out_dtype == api.OUT_FP32 else torch.bfloat16
    api.snip_debug_set(api.DEBUG_GEMM_KERNEL, choice)
    try:
        wy, y = guarded(M * N * esz, dt); wdx, dx = guarded(M * K * esz, dt); wdw, dw = guarded(N * K * esz, dt)
        api.snip_linear_fwd(X, W, fa, fb, out_dtype, out=y.view(M, N))
        api.snip_linear_dgrad(DY, W, fa, fb, out_dtype, out=dx.view(M, K))
        api.snip_linear_wgrad(DY, X, fa, fb, out_dtype, out=dw.view(N, K))
        torch.cuda.synchronize()
    finally:
        api.snip_debug_set(api.DEBUG_GEMM_KERNEL, api.GEMM_KERNEL_AUTO)
    assert intact(wy, M * N * esz) and intact(wdx, M * K * esz) and intact(wdw, N * K * esz)
    assert torch.isfinite(y.float()).all() and torch.isfinite(dw.float()).all()
