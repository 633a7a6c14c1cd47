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


@pytest.mark.parametrize("shape", [(320, 448), (192, 320), (64, 704)])
def test_added_quantizer_forms_stay_inside_their_buffers(shape):
    # 32-long tiles with power-of-two scales (codes, scales, atoms) and the two-level form (codes, atoms), two outputs each
    from paper_2602_01410_b200 import api
    rows, cols = shape
    x = to_dev(wl.make_x(np.random.default_rng(6), rows, cols, 0.01, 20.0))
    n = api.ctypes.c_size_t()
    api._check("snip_quantize_mx_sizes", api._lib.snip_quantize_mx_sizes(rows, cols, api.ctypes.byref(n)))
    for fmt in (FP8, FP4):
        bufs, wholes = [], []
        for i, blk in enumerate((api.BLOCK_ROW32, api.BLOCK_COL32)):
            cb, sb, _ = api.snip_quantize_sizes(rows, cols, fmt, blk, api.Q_TRANSPOSED if i else 0)
            wc, codes = guarded(cb); wsc, scales = guarded(sb, torch.float32); wsf, sf = guarded(n.value); wst, stats = guarded(32)
            bufs.append({"codes": codes, "scales": scales, "sf": sf, "stats": stats[:24]})
            wholes += [(wc, cb), (wsc, sb), (wsf, n.value), (wst, 32)]
        wb = api.snip_quantize_dual_workspace(rows, cols)
        ww, ws = guarded(wb)
        api.snip_quantize_dual(x, api.DUAL_ROW32_COL32T, fmt, fmt, pow2_scale=True, bufs=tuple(bufs), ws=ws)
        torch.cuda.synchronize()
        assert all(intact(w, nb) for w, nb in wholes) and intact(ww, wb)
        assert not (bufs[0]["sf"].cpu().numpy() == CANARY).all()
    cb, fb = api.snip_quantize_nvfp4_sizes(rows, cols)
    bufs, wholes = [], []
    for i in range(2):
        wc, codes = guarded(cb); wsf, sf = guarded(fb); wst, stats = guarded(32)
        bufs.append({"codes": codes, "sf": sf, "stats": stats[:24]})
        wholes += [(wc, cb), (wsf, fb), (wst, 32)]
    wb = api.snip_quantize_dual_workspace(rows, cols)
    ww, ws = guarded(wb)
    bound = x.float().abs().max().reshape(1).contiguous()
    api.snip_quantize_nvfp4_dual(x, bound, bufs=tuple(bufs), ws=ws)
    torch.cuda.synchronize()
    assert all(intact(w, nb) for w, nb in wholes) and intact(ww, wb)
    assert not (bufs[1]["sf"].cpu().numpy() == CANARY).all()


@pytest.mark.parametrize("shape", [(320, 448, 192), (64, 192, 320)])
def test_hardware_scaled_gemm_outputs_stay_inside_their_buffers(shape):
    from paper_2602_01410_b200 import api
    M, K, N = shape
    rng = np.random.default_rng(8)
    x, w = to_dev(wl.make_x(rng, M, K, 0.01, 20.0)), to_dev(wl.make_w(rng, N, K))
    bx, bw = x.float().abs().max().reshape(1).contiguous(), w.float().abs().max().reshape(1).contiguous()
    xa, _ = api.snip_quantize_nvfp4_dual(x, bx, want_stats=False)
    wa, _ = api.snip_quantize_nvfp4_dual(w, bw, want_stats=False)
    a = api.make_qtensor(xa["codes"], None, M, K, FP4, api.BLOCK_ROW16)
    b = api.make_qtensor(wa["codes"], None, N, K, FP4, api.BLOCK_ROW16)
    for dt, esz in ((api.OUT_BF16, 2), (api.OUT_FP32, 4)):
        wo, out = guarded(M * N * esz, torch.bfloat16 if esz == 2 else torch.float32)
        api.snip_gemm_nvfp4(api.OP_FWD, a, xa["sf"], bx, b, wa["sf"], bw, (M, N), dt, out=out.view(M, N))
        torch.cuda.synchronize()
        assert intact(wo, M * N * esz)
