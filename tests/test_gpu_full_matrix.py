"""Full-matrix comparison at the 7B size through a bridge: a deliberately naive FP64 matrix product on the GPU
(tests/cuda_ref/naive_gemm.cu: one thread per output, one loop, no tensor cores, nothing in common with the
library) fed with the CPU oracle's dequantized operands.  The bridge is first compared with the oracle's own FP64
GEMMs IN FULL on the small configuration, on a ragged shape and on one linear of the 1B configuration; only then
are the library's outputs compared with it, every element of Y, dX and dW of the 7B fused-QKV linear."""
import numpy as np
import pytest
import torch

from oracle import snip_oracle as orc
from paper_2602_01410_b200 import workloads as wl

pytestmark = pytest.mark.gpu
from gpu_util import to_dev  # noqa: E402

FP8, FP4 = 1, 2


@pytest.fixture(scope="module")
def naive():
    import cuda_ref
    lib = cuda_ref.load()

    def run(op, a64, b64, M, N, K):
        """a64, b64: numpy float64 operands in the oracle's orientation; returns a CUDA float64 tensor."""
        A = torch.from_numpy(np.ascontiguousarray(a64)).cuda()
        B = torch.from_numpy(np.ascontiguousarray(b64)).cuda()
        shape = {0: (M, N), 1: (M, K), 2: (N, K)}[op]
        C = torch.empty(shape, dtype=torch.float64, device="cuda")
        rc = lib.naive_gemm_f64(op, A.data_ptr(), B.data_ptr(), C.data_ptr(), M, N, K)
        assert rc == 0, rc
        return C
    return run


def rel(got: torch.Tensor, want: torch.Tensor) -> float:
    g, w = got.double(), want.double()
    return float((g - w).norm() / w.norm())


def oracle_operands(x, w, dy, fmt):
    """Dequantized operands of the three GEMMs, as the oracle defines them."""
    qx, qw, qdy = orc.quantize(x, fmt, orc.BLOCK_ROW), orc.quantize(w, fmt, orc.BLOCK_BLK), orc.quantize(dy, fmt, orc.BLOCK_ROW)
    qdyc, qxc = orc.quantize(dy, fmt, orc.BLOCK_COL), orc.quantize(x, fmt, orc.BLOCK_COL)
    return qx.xhat, qw.xhat, qdy.xhat, qdyc.xhat, qxc.xhat


@pytest.mark.parametrize("case", ["config0", "ragged", "1b-k-projection"])
@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_bridge_equals_the_oracle_in_full(naive, case, fmt):
    if case == "config0":
        x, w, dy = wl.linear_inputs(wl.CONFIGS[0], 0, 0)
    elif case == "ragged":
        rng = np.random.default_rng(3)
        x, w, dy = wl.make_x(rng, 320, 448, 0.01, 20.0), wl.make_w(rng, 192, 448), wl.make_dy(rng, 320, 192)
    else:
        x, w, dy = wl.linear_inputs(wl.CONFIGS[1], 0, 1)       # 8192 tokens, 2048 -> 256
    M, K = x.shape
    N = w.shape[0]
    xh, wh, dyh, dych, xch = oracle_operands(x, w, dy, fmt)
    for op, a, b, ref in ((0, xh, wh, orc.gemm_fwd(xh, wh)), (1, dyh, wh, orc.gemm_dgrad(dyh, wh)), (2, dych, xch, orc.gemm_wgrad(dych, xch))):
        got = naive(op, a, b, M, N, K).cpu().numpy()
        # both are FP64 sums of the same exact products; only the order of additions differs
        assert np.linalg.norm(got - ref) <= 1e-13 * np.linalg.norm(ref), (case, op)


def check_all_elements(name, got, ref):
    assert rel(got, ref) <= 1e-5, (name, rel(got, ref))
    # no single block of 128 rows x 128 columns may be off either (a wrong tile of the persistent walk would hide in
    # the total); a ragged edge (64 rows or columns left over) is checked in 64-row strips / as one strip
    r, c = ref.shape
    d2, t2 = (got.double() - ref).pow(2), ref.pow(2)
    rr, cc = r // 128 * 128, c // 128 * 128
    tiles = lambda m: m[:rr, :cc].reshape(rr // 128, 128, cc // 128, 128).sum(dim=(1, 3))
    worst = float((tiles(d2) / tiles(t2)).max().sqrt())
    if cc < c:
        strips = lambda m: m[:, cc:].reshape(r // 64, 64, -1).sum(dim=(1, 2))
        worst = max(worst, float((strips(d2) / strips(t2)).max().sqrt()))
    if rr < r:
        worst = max(worst, float((d2[rr:, :].sum() / t2[rr:, :].sum()).sqrt()))
    assert worst <= 1e-4, (name, worst)


def three_gemms_against_the_bridge(naive, cfg, linear, fmt, kernel_choice=0):
    from paper_2602_01410_b200 import api
    x, w, dy = wl.linear_inputs(cfg, 0, linear)
    M, K = x.shape
    N = w.shape[0]
    X, W, DY = to_dev(x), to_dev(w), to_dev(dy)
    xh, wh, dyh, dych, xch = oracle_operands(x, w, dy, fmt)
    api.snip_debug_set(api.DEBUG_GEMM_KERNEL, kernel_choice)
    try:
        y, _, _ = api.snip_linear_fwd(X, W, fmt, fmt, api.OUT_FP32)
        check_all_elements("fwd", y, naive(0, xh, wh, M, N, K)); del y
        dx, _, _ = api.snip_linear_dgrad(DY, W, fmt, fmt, api.OUT_FP32)
        check_all_elements("dgrad", dx, naive(1, dyh, wh, M, N, K)); del dx
        dw, _, _ = api.snip_linear_wgrad(DY, X, fmt, fmt, api.OUT_FP32)
        check_all_elements("wgrad", dw, naive(2, dych, xch, M, N, K))
    finally:
        api.snip_debug_set(api.DEBUG_GEMM_KERNEL, 0)


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_7b_fused_qkv_every_output_element(naive, fmt):
    three_gemms_against_the_bridge(naive, wl.CONFIGS[3], 0, fmt)


def test_7b_o_projection_every_output_element_pair_kernels(naive):
    # the CTA-pair form of the GEMM, forced through the testing hook
    three_gemms_against_the_bridge(naive, wl.CONFIGS[3], 1, FP8, kernel_choice=2)


@pytest.mark.parametrize("fmt", [FP8, FP4])
def test_3b_down_projection_ragged_every_output_element(naive, fmt):
    # 8640 -> 3200: the contraction of fwd / the output width of dgrad and wgrad end in a 64-wide tile
    three_gemms_against_the_bridge(naive, wl.CONFIGS[2], 4, fmt)


def test_7b_one_read_path_bf16_outputs_every_element(naive):
    """The launch configuration bench.py times (snip_linear_fwd_bwd, BF16 outputs): every element of Y, dX, dW against
    the bridge rounded to bf16 (both sides rounded: bf16 rounding alone is 1.7e-3 of the signal)."""
    from paper_2602_01410_b200 import api
    cfg = wl.CONFIGS[3]
    x, w, dy = wl.linear_inputs(cfg, 0, 1)       # O projection 4096 -> 4096
    M, K = x.shape
    N = w.shape[0]
    fmt = FP4
    y, dx, dw, _ = api.snip_linear_fwd_bwd(to_dev(x), to_dev(w), to_dev(dy), fmt, fmt, fmt, api.OUT_BF16)
    xh, wh, dyh, dych, xch = oracle_operands(x, w, dy, fmt)
    for name, got, ref in (("fwd", y, naive(0, xh, wh, M, N, K)), ("dgrad", dx, naive(1, dyh, wh, M, N, K)), ("wgrad", dw, naive(2, dych, xch, M, N, K))):
        ref16 = ref.float().to(torch.bfloat16)      # FP64 -> FP32 -> BF16 double rounding differs from direct RNE on a negligible fraction
        assert rel(got.double(), ref16.double()) <= 1e-3, name
        assert float((got.double() - ref16.double()).abs().max() / ref.abs().max()) <= 2.0 ** -7, name
