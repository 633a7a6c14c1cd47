"""Weight-gradient product with the tiles of its last wave cut into slices of the contraction: the sliced and the
unsliced run against the CPU oracle and against each other, on shapes whose token count (the contraction) is long
enough for two, three and four slices, with ragged row / column / contraction tiles, in every format pair.

Bar: FP32 output within 1e-5 (relative Frobenius) of the float64 oracle, as in test_gpu_gemm.py; sliced runs
repeat bit for bit (the slices are added in slice order, not in order of arrival)."""
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
def slicing(api):
    def choose(v):
        api.snip_debug_set(api.DEBUG_GEMM_SLICING, v)
    yield choose
    api.snip_debug_set(api.DEBUG_GEMM_SLICING, 1)


def operands(api, M, K, N, fa, fb, seed):
    rng = np.random.default_rng(seed)
    x, dy = wl.make_x(rng, M, K, 0.01, 20.0), wl.make_dy(rng, M, N)
    X, DY = to_dev(x), to_dev(dy)
    cd, sd, _, _ = api.snip_quantize(DY, fa, api.BLOCK_COL, api.Q_TRANSPOSED)
    cx, sx, _, _ = api.snip_quantize(X, fb, api.BLOCK_COL, api.Q_TRANSPOSED)
    a = api.make_qtensor(cd, sd, M, N, fa, api.BLOCK_COL, True)
    b = api.make_qtensor(cx, sx, M, K, fb, api.BLOCK_COL, True)
    return x, dy, a, b, (cd, sd, cx, sx)


# (tokens M, in-features K, out-features N): 4 tiles x 4 slices; 6 ragged tiles x 2 slices (17 stages); 12 tiles with a
# contraction ending in a 64-wide tile; 48 tiles x 3 slices
SHAPES = [(4096, 512, 256), (2176, 448, 320), (3136, 768, 512), (3072, 1536, 1024)]


@pytest.mark.parametrize("fa,fb", PAIRS)
@pytest.mark.parametrize("shape", SHAPES)
def test_sliced_and_unsliced_match_the_oracle(api, slicing, fa, fb, shape):
    M, K, N = shape
    x, dy, a, b, keep = operands(api, M, K, N, fa, fb, 4000 + M + K + N)
    ref = orc.linear_wgrad(dy, x, fa, fb)[0]
    outs = {}
    for mode in (1, 0):
        slicing(mode)
        outs[mode] = api.snip_gemm_quantized(api.OP_WGRAD, a, b, (N, K), api.OUT_FP32)
        torch.cuda.synchronize()
        e = rel_fro(outs[mode].cpu().numpy(), ref)
        assert e <= 1e-5, (mode, e)
    # the two differ only in the order of FP32 additions
    assert rel_fro(outs[1].cpu().numpy(), outs[0].cpu().numpy().astype(np.float64)) <= 1e-6
    slicing(1)
    for _ in range(3):
        again = api.snip_gemm_quantized(api.OP_WGRAD, a, b, (N, K), api.OUT_FP32)
        torch.cuda.synchronize()
        assert torch.equal(again, outs[1])
    out16 = api.snip_gemm_quantized(api.OP_WGRAD, a, b, (N, K), api.OUT_BF16)
    torch.cuda.synchronize()
    assert rel_fro(bf16_out_to_f64(out16), orc.bf16_to_float(orc.round_to_bf16(ref))) <= 1e-3


def test_sliced_accumulate_garbage_workspace_and_minimum_workspace(api, slicing):
    slicing(1)
    M, K, N = 4096, 512, 256
    x, dy, a, b, keep = operands(api, M, K, N, FP8, FP8, 77)
    ref = orc.linear_wgrad(dy, x, FP8, FP8)[0]
    gbytes, _ = api.snip_workspace_size(api.OP_WGRAD, M, N, K, FP8, FP8)
    assert gbytes > (1 << 20)
    # the caller's workspace holds garbage: status word and arrival counters are cleared by the call itself
    ws = torch.full((gbytes,), 0xFF, dtype=torch.uint8, device="cuda")
    out = api.snip_gemm_quantized(api.OP_WGRAD, a, b, (N, K), api.OUT_FP32, ws=ws)
    torch.cuda.synchronize()
    assert api.snip_poll_status(ws) == api.OK
    assert rel_fro(out.cpu().numpy(), ref) <= 1e-5
    # accumulate: the slice sums are added to what the output holds
    out2 = api.snip_gemm_quantized(api.OP_WGRAD, a, b, (N, K), api.OUT_FP32, accumulate=True, out=out.clone(), ws=ws)
    torch.cuda.synchronize()
    assert rel_fro(out2.cpu().numpy(), 2 * ref) <= 1e-5
    # a 256-byte workspace is still enough (the product then runs unsliced)
    small = torch.full((256,), 0xFF, dtype=torch.uint8, device="cuda")
    out3 = api.snip_gemm_quantized(api.OP_WGRAD, a, b, (N, K), api.OUT_FP32, ws=small)
    torch.cuda.synchronize()
    assert api.snip_poll_status(small) == api.OK
    assert rel_fro(out3.cpu().numpy(), ref) <= 1e-5
