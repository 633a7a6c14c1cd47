"""The calls enqueue work on the caller's stream only (no allocation, no synchronisation), so a whole
layer step can be captured into a CUDA graph and replayed; the replay must reproduce the eager results
bit for bit."""
import numpy as np
import pytest
import torch

from paper_2602_01410_b200 import workloads as wl

pytestmark = pytest.mark.gpu
from gpu_util import to_dev  # noqa: E402

FP8, FP4 = 1, 2


@pytest.mark.parametrize("pow2", [False, True])
def test_fwd_bwd_step_replays_from_a_cuda_graph(pow2):
    from paper_2602_01410_b200 import api
    M, K, N = 512, 384, 640
    rng = np.random.default_rng(9)
    x, w, dy = (to_dev(a) for a in (wl.make_x(rng, M, K), wl.make_w(rng, N, K), wl.make_dy(rng, M, N)))
    ws = torch.zeros(api.snip_linear_fwd_bwd_workspace(M, N, K, FP8, FP4, FP4, pow2), dtype=torch.uint8, device="cuda")
    stats = torch.zeros(6 * 24, dtype=torch.uint8, device="cuda")
    outs = [torch.empty(s, dtype=torch.bfloat16, device="cuda") for s in ((M, N), (M, K), (N, K))]

    def step():
        api.snip_linear_fwd_bwd(x, w, dy, FP8, FP4, FP4, pow2_scale=pow2, dy_sr_seed=None if pow2 else 5, y=outs[0], dx=outs[1], dw=outs[2],
                                stats=stats, ws=ws)

    step()                                            # eager reference (and first-use initialisation outside the capture)
    torch.cuda.synchronize()
    want = [o.clone() for o in outs] + [stats.clone()]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step()
    for _ in range(2):
        for o in outs:
            o.zero_()
        stats.zero_()
        graph.replay()
        torch.cuda.synchronize()
        for got, ref in zip(outs + [stats], want):
            assert torch.equal(got, ref)
    assert api.snip_poll_status(ws) == 0
