"""The no-allocation variant of the quantizer (statistics scratch built into the library, for hosts
that cannot pass any) must give exactly what snip_quantize gives.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from paper_2602_01410_b200 import workloads as wl

pytestmark = pytest.mark.gpu
from gpu_util import to_dev  # noqa: E402


def _both(api, x, fmt, block, flags):
    want_codes, want_scales, want_stats, _ = api.snip_quantize(x, fmt, block, flags)
    codes = torch.full_like(want_codes, 0xAA)
    scales = torch.full_like(want_scales, -1.0)
    stats = torch.zeros(32, dtype=torch.uint8, device=x.device)
    api.snip_quantize_noalloc(x, fmt, block, flags, codes, scales, stats)
    torch.cuda.synchronize()
    assert torch.equal(codes, want_codes)
    assert torch.equal(scales, want_scales)
    got, want = api.stats_to_host(stats), api.stats_to_host(want_stats)
    # same kernels, fixed-order reduction: identical, far inside the 1e-4 bar of the statistics
    for k in ("sumsq_x", "sumsq_err", "amax"):
        assert got[k] == pytest.approx(want[k], rel=1e-4, abs=0.0) and got[k] == want[k]


def test_two_calls_in_a_row_match_the_allocating_entry_point():
    from paper_2602_01410_b200 import api
    rng = np.random.default_rng(42)
    x1 = to_dev(wl.make_x(rng, 512, 640, 0.01, 20.0))
    x2 = to_dev(wl.make_dy(rng, 256, 384))          # smaller: leaves stale partials of call 1 behind it
    _both(api, x1, api.FMT_FP8_E4M3, api.BLOCK_ROW, api.Q_STATS)
    _both(api, x2, api.FMT_FP4_E2M1, api.BLOCK_COL, api.Q_STATS | api.Q_TRANSPOSED)
    _both(api, x1, api.FMT_FP4_E2M1, api.BLOCK_BLK, api.Q_STATS)


def test_inputs_beyond_the_built_in_scratch_are_rejected():
    from paper_2602_01410_b200 import api
    rows, cols = 128 * 200, 128 * 128          # 25600 tiles > 16384
    x = torch.empty((1, 1), dtype=torch.bfloat16, device="cuda")
    codes = torch.empty(16, dtype=torch.uint8, device="cuda")
    scales = torch.empty(16, dtype=torch.float32, device="cuda")
    stats = torch.zeros(32, dtype=torch.uint8, device="cuda")
    with pytest.raises(api.SnipError) as e:
        api._check("snip_quantize_noalloc", api._lib.snip_quantize_noalloc(api._p(x), rows, cols, cols, api.FMT_FP8_E4M3, api.BLOCK_ROW,
                                                                           api.Q_STATS, api._p(codes), api._p(scales), api._p(stats), None))
    assert e.value.status == api.ERR_WORKSPACE
    assert b"built-in array" in api._lib.snip_last_cuda_error()


def test_without_statistics_the_size_limit_does_not_apply():
    # No SNIP_Q_STATS: the built-in array is not used, so a tensor of more than 16384 tiles goes through
    # and gives what snip_quantize gives.
    from paper_2602_01410_b200 import api
    rows, cols = 129 * 128, 128 * 128          # 16512 tiles
    g = torch.Generator(device="cuda"); g.manual_seed(7)
    x = torch.randn(rows, cols, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    want_codes, want_scales, _, _ = api.snip_quantize(x, api.FMT_FP8_E4M3, api.BLOCK_ROW, 0)
    codes = torch.full_like(want_codes, 0xAA)
    scales = torch.full_like(want_scales, -1.0)
    api.snip_quantize_noalloc(x, api.FMT_FP8_E4M3, api.BLOCK_ROW, 0, codes, scales, None)
    torch.cuda.synchronize()
    assert torch.equal(codes, want_codes) and torch.equal(scales, want_scales)
