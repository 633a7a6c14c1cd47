"""Both families of paper-rule GEMM kernels (single CTA, CTA pair) against the CPU oracle on the same
inputs, forced through the library's testing hook; shapes with ragged row, column and contraction
tiles and outputs shorter than one pair tile.  Also: the status word of a workspace the caller never
initialised, and a device-side wait that is made to run out.

Bar: FP32 output within 1e-5 (relative Frobenius) of the float64 oracle, as in test_gpu_gemm.py."""
import numpy as np
import pytest
import torch

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

pytestmark = pytest.mark.gpu

FP8, FP4 = 1, 2
PAIRS = [(FP8, FP8), (FP4, FP4), (FP8, FP4), (FP4, FP8)]

from gpu_util import bf16_out_to_f64, rel_fro, to_dev  # noqa: E402


@pytest.fixture(scope="module")
def api():
    from paper_2602_01410_b200 import api as _api
    return _api


@pytest.fixture
def kernel_choice(api):
    def choose(v):
        api.snip_debug_set(api.DEBUG_GEMM_KERNEL, v)
    yield choose
    api.snip_debug_set(api.DEBUG_GEMM_KERNEL, api.GEMM_KERNEL_AUTO)


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


# (M, K, N): one pair tile; several tiles; every dimension ending in a 64-wide tile; fewer rows than a pair tile;
# more tiles than resident CTA pairs with a long contraction (the shared-memory and tensor-memory rings wrap many times)
SHAPES = [(256, 128, 128), (512, 384, 256), (320, 448, 192), (64, 192, 320), (2560, 1600, 1152)]


@pytest.mark.parametrize("fa,fb", PAIRS)
@pytest.mark.parametrize("shape", SHAPES)
def test_pair_and_single_kernels_match_the_oracle(api, kernel_choice, fa, fb, shape):
    M, K, N = shape
    x, w, dy = inputs(M, K, N, 900 + M + K + N)
    want = (orc.linear_fwd(x, w, fa, fb)[0], orc.linear_dgrad(dy, w, fa, fb)[0], orc.linear_wgrad(dy, x, fa, fb)[0])
    got = {}
    for choice in (api.GEMM_KERNEL_PAIR, api.GEMM_KERNEL_SINGLE):
        kernel_choice(choice)
        got[choice] = run_three(api, x, w, dy, fa, fb, api.OUT_FP32)
        for name, g, ref in zip(("fwd", "dgrad", "wgrad"), got[choice], want):
            e = rel_fro(g.cpu().numpy(), ref)
            assert e <= 1e-5, (choice, name, e)
        # a second run is bit-identical (races in the ring hand-offs would show here)
        again = run_three(api, x, w, dy, fa, fb, api.OUT_FP32)
        for g, h in zip(got[choice], again):
            assert torch.equal(g, h)
    kernel_choice(api.GEMM_KERNEL_PAIR)
    got16 = run_three(api, x, w, dy, fa, fb, api.OUT_BF16)
    for name, g, ref in zip(("fwd", "dgrad", "wgrad"), got16, want):
        ref16 = orc.bf16_to_float(orc.round_to_bf16(ref))
        assert rel_fro(bf16_out_to_f64(g), ref16) <= 1e-3, name


@pytest.mark.parametrize("choice", [1, 2])
def test_accumulate_into_fp32(api, kernel_choice, choice):
    kernel_choice(choice)
    M, K, N = 512, 256, 320
    x, w, dy = inputs(M, K, N, 5)
    X, DY = to_dev(x), to_dev(dy)
    ref = orc.linear_wgrad(dy, x, FP8, FP8)[0]
    dw, _, _ = api.snip_linear_wgrad(DY, X, FP8, FP8, api.OUT_FP32)
    dw2, _, _ = api.snip_linear_wgrad(DY, X, FP8, FP8, api.OUT_FP32, accumulate=True, out=dw.clone())
    torch.cuda.synchronize()
    assert rel_fro(dw.cpu().numpy(), ref) <= 1e-5
    assert rel_fro(dw2.cpu().numpy(), 2 * ref) <= 1e-5


@pytest.mark.parametrize("choice", [1, 2])
def test_status_word_needs_no_initialisation(api, kernel_choice, choice):
    # the caller's workspace holds garbage; the call clears the status word itself
    kernel_choice(choice)
    M, K, N = 256, 256, 256
    x, w, _ = inputs(M, K, N, 3)
    X, W = to_dev(x), to_dev(w)
    cx, sx, _, _ = api.snip_quantize(X, FP8, api.BLOCK_ROW)
    cw, sw, _, _ = api.snip_quantize(W, FP8, api.BLOCK_BLK)
    a = api.make_qtensor(cx, sx, M, K, FP8, api.BLOCK_ROW)
    b = api.make_qtensor(cw, sw, N, K, FP8, api.BLOCK_BLK)
    ws = torch.full((256,), 0xFF, dtype=torch.uint8, device="cuda")
    y = api.snip_gemm_quantized(api.OP_FWD, a, b, (M, N), api.OUT_FP32, ws=ws)
    torch.cuda.synchronize()
    assert api.snip_poll_status(ws) == api.OK
    assert rel_fro(y.cpu().numpy(), orc.linear_fwd(x, w, FP8, FP8)[0]) <= 1e-5


@pytest.mark.parametrize("choice", [1, 2])
@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_a_wait_that_runs_out_reports_timeout_and_the_next_call_is_fine(api, kernel_choice, choice, fmt):
    # Host-made condition: the first stage's barrier expects 16 bytes more than the copies deliver, so every
    # copy lands but the phase never completes.  With the wait limit at 20 ms the kernel gives up by itself,
    # releases its tensor memory and raises the status word; nothing traps, faults or spins without a bound.
    kernel_choice(choice)
    M, K, N = 512, 512, 256
    x, w, _ = inputs(M, K, N, 17)
    X, W = to_dev(x), to_dev(w)
    cx, sx, _, _ = api.snip_quantize(X, fmt, api.BLOCK_ROW)
    cw, sw, _, _ = api.snip_quantize(W, fmt, api.BLOCK_BLK)
    a = api.make_qtensor(cx, sx, M, K, fmt, api.BLOCK_ROW)
    b = api.make_qtensor(cw, sw, N, K, fmt, api.BLOCK_BLK)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    try:
        api.snip_debug_set(api.DEBUG_WAIT_LIMIT_NS, 20_000_000)
        api.snip_debug_set(api.DEBUG_TX_SKEW_BYTES, 16)
        api.snip_gemm_quantized(api.OP_FWD, a, b, (M, N), api.OUT_FP32, ws=ws)
        torch.cuda.synchronize()
        assert api.snip_poll_status(ws) == api.ERR_TIMEOUT
    finally:
        api.snip_debug_set(api.DEBUG_TX_SKEW_BYTES, 0)
        api.snip_debug_set(api.DEBUG_WAIT_LIMIT_NS, 2_000_000_000)
    # the context is intact and the same workspace serves a normal call
    y = api.snip_gemm_quantized(api.OP_FWD, a, b, (M, N), api.OUT_FP32, ws=ws)
    torch.cuda.synchronize()
    assert api.snip_poll_status(ws) == api.OK
    assert rel_fro(y.cpu().numpy(), orc.linear_fwd(x, w, fmt, fmt)[0]) <= 1e-5
