"""Stream ordering of back-to-back calls.  The quantizer kernels are launched with programmatic stream
serialization (their CTAs may be scheduled while the statistics reduction of the previous call drains), so
this pins what the caller relies on: calls issued one after the other on one stream, without any
synchronisation in between and sharing output buffers and workspace, behave as if run one at a time."""
import numpy as np
import pytest
import torch

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

pytestmark = pytest.mark.gpu
from gpu_util import to_dev  # noqa: E402

FP8, FP4 = 1, 2
ROW, COL, BLK = 0, 1, 2


def _check(api, x_bits, fmt, block, transposed, codes, scales, stats):
    q = orc.quantize(x_bits, fmt, block)
    want = q.packed(transposed)
    got = codes.cpu().numpy()[:want.size].reshape(want.shape)
    assert np.array_equal(got, want)
    assert np.array_equal(scales.cpu().numpy().reshape(q.scales.shape).view(np.uint32), q.scales.view(np.uint32))
    st = api.stats_to_host(stats[:24])
    assert st["sumsq_x"] == pytest.approx(q.sumsq_x, rel=1e-4)
    assert st["sumsq_err"] == pytest.approx(q.sumsq_err, rel=1e-4, abs=1e-300)


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_single_output_calls_back_to_back_share_workspace(fmt):
    from paper_2602_01410_b200 import api
    rng = np.random.default_rng(4100 + fmt)
    shape = (1024, 768)
    xs = [wl.make_x(rng, *shape), wl.make_dy(rng, *shape), wl.make_x(rng, *shape)]
    dev = [to_dev(x) for x in xs]
    flags = api.Q_STATS
    cb, sb, wb = api.snip_quantize_sizes(*shape, fmt, ROW, flags)
    ws = torch.empty(wb, dtype=torch.uint8, device="cuda")
    outs = []
    torch.cuda.synchronize()
    # twelve calls without a synchronisation: three inputs in turn, one workspace, outputs of their own
    for i in range(12):
        codes = torch.empty(cb, dtype=torch.uint8, device="cuda")
        scales = torch.empty(sb // 4, dtype=torch.float32, device="cuda")
        stats = torch.empty(32, dtype=torch.uint8, device="cuda")
        api.snip_quantize(dev[i % 3], fmt, ROW, flags, codes=codes, scales=scales, stats=stats, ws=ws)
        outs.append((i % 3, codes, scales, stats))
    torch.cuda.synchronize()
    for j, codes, scales, stats in outs:
        _check(api, xs[j], fmt, ROW, False, codes, scales, stats)


def test_later_call_overwrites_the_buffers_of_an_earlier_one():
    from paper_2602_01410_b200 import api
    rng = np.random.default_rng(4200)
    shape = (896, 640)
    x1, x2 = wl.make_x(rng, *shape), wl.make_dy(rng, *shape)
    d1, d2 = to_dev(x1), to_dev(x2)
    a, b = api.snip_quantize_dual(d1, api.DUAL_ROW_COLT, FP8, FP4, want_stats=True)
    ws = torch.empty(api.snip_quantize_dual_workspace(*shape), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    for i in range(6):   # the same output buffers, alternating inputs, no synchronisation
        api.snip_quantize_dual(d1 if i % 2 == 0 else d2, api.DUAL_ROW_COLT, FP8, FP4, want_stats=True, bufs=(a, b), ws=ws)
    torch.cuda.synchronize()
    _check(api, x2, FP8, ROW, False, a["codes"], a["scales"], a["stats"])
    _check(api, x2, FP4, COL, True, b["codes"], b["scales"], b["stats"])


def test_quantizer_behind_a_gemm_that_reads_the_same_buffers():
    """quantize(x1) -> GEMM reading those codes -> quantize(x2) into the same buffers: the GEMM must see x1."""
    from paper_2602_01410_b200 import api
    rng = np.random.default_rng(4300)
    M, N, K = 512, 384, 512
    x1, x2, w = wl.make_x(rng, M, K), wl.make_x(rng, M, K), wl.make_w(rng, N, K)
    d1, d2, dw = to_dev(x1), to_dev(x2), to_dev(w)
    qw = api.snip_quantize(dw, FP8, BLK)
    cb, sb, wb = api.snip_quantize_sizes(M, K, FP8, ROW, api.Q_STATS)
    codes = torch.empty(cb, dtype=torch.uint8, device="cuda")
    scales = torch.empty(sb // 4, dtype=torch.float32, device="cuda")
    stats = torch.empty(32, dtype=torch.uint8, device="cuda")
    ws = torch.empty(wb, dtype=torch.uint8, device="cuda")
    y = torch.empty(M, N, dtype=torch.float32, device="cuda")
    gws = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    b = api.make_qtensor(qw[0], qw[1], N, K, FP8, BLK)
    torch.cuda.synchronize()
    api.snip_quantize(d1, FP8, ROW, api.Q_STATS, codes=codes, scales=scales, stats=stats, ws=ws)
    a = api.make_qtensor(codes, scales, M, K, FP8, ROW)
    api.snip_gemm_quantized(api.OP_FWD, a, b, (M, N), api.OUT_FP32, out=y, ws=gws)
    api.snip_quantize(d2, FP8, ROW, api.Q_STATS, codes=codes, scales=scales, stats=stats, ws=ws)
    torch.cuda.synchronize()
    assert api.snip_poll_status(gws) == 0
    want = orc.gemm_fwd(orc.quantize(x1, FP8, ROW).xhat, orc.quantize(w, FP8, BLK).xhat)
    got = y.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - want) / np.linalg.norm(want) <= 1e-3
    _check(api, x2, FP8, ROW, False, codes, scales, stats)
