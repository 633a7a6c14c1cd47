"""AdamW sensitivity-term norm on the GPU against the CPU oracle (paper Sec. 4.3)."""
import numpy as np
import pytest
import torch

from oracle import snip_oracle as orc

pytestmark = pytest.mark.gpu


def moments(rng, n, steps=5, b1=0.9, b2=0.95):
    """AdamW moments after a few steps of random gradients with per-element scales spanning decades."""
    scale = np.exp(rng.normal(size=n) * 2.0).astype(np.float32) * np.float32(1e-3)
    m = np.zeros(n, dtype=np.float32)
    v = np.zeros(n, dtype=np.float32)
    g = None
    for _ in range(steps):
        g = (rng.normal(size=n).astype(np.float32) * scale).astype(np.float32)
        m = (np.float32(b1) * m + np.float32(1 - b1) * g).astype(np.float32)
        v = (np.float32(b2) * v + np.float32(1 - b2) * g * g).astype(np.float32)
    return m, v, g


@pytest.mark.parametrize("n", [4, 1024, 128 * 320, 1_000_000])
@pytest.mark.parametrize("g_bf16", [False, True])
def test_matches_the_oracle(n, g_bf16):
    from paper_2602_01410_b200 import api
    rng = np.random.default_rng(n)
    b1, b2, eps = float(np.float32(0.9)), float(np.float32(0.95)), float(np.float32(1e-8))
    m, v, g = moments(rng, n)
    gt = torch.from_numpy(g).cuda()
    if g_bf16:
        gt = gt.to(torch.bfloat16)
        g = gt.float().cpu().numpy()
    out = api.snip_adamw_sensitivity(torch.from_numpy(m).cuda(), torch.from_numpy(v).cuda(), gt, b1, b2, eps)
    want = orc.adamw_sensitivity_sumsq(m, v, g, b1, b2, eps)
    assert float(out.cpu()[0]) == pytest.approx(want, rel=1e-4)


def test_zero_second_moment_and_argument_checks():
    from paper_2602_01410_b200 import api
    m = torch.zeros(8, device="cuda"); v = torch.zeros(8, device="cuda"); g = torch.zeros(8, device="cuda")
    v[4:] = 4.0; m[4:] = 3.0; g[4:] = 2.0
    out = api.snip_adamw_sensitivity(m, v, g, 0.5, 0.75, 1.0)
    # four elements with v = 0: (1/2)/1 each; four with the hand-worked value 1/12
    assert float(out.cpu()[0]) == pytest.approx(4 * 0.25 + 4 / 144, rel=1e-6)
    with pytest.raises(api.SnipError):
        api.snip_adamw_sensitivity(m[:6], v[:6], g[:6], 0.9, 0.95, 1e-8)     # not a multiple of 4
