"""Host side of scheme generation (paper Sec. 4.2, 4.3, 5.2, 5.3): the oracle's formulas against
hand-worked values, the library's exact selection against exhaustive search and against the
properties the paper states (E_t = 0 keeps every layer at its best-quality option, E_t = 1 forces FP4
everywhere, pipeline stages are balanced).  No GPU needed: these entry points are host-only."""
import itertools
import math

import numpy as np
import pytest

from oracle import scheme_oracle as so


@pytest.fixture(scope="module")
def api():
    from paper_2602_01410_b200 import api as _api
    return _api


def test_oracle_loss_divergence_hand_worked():
    # |dL/dX| = 3, |err X| = 4, M K = 16 -> 3; |dL/dW| = 8, |err W| = 2, N K = 16 -> 4; sqrt(9 + 16) = 5; |L| = 2.5 -> 2
    assert so.loss_divergence(3, 4, 4, 4, 8, 2, 4, -2.5) == pytest.approx(2.0, rel=1e-15)
    # only one tensor perturbed: the other term vanishes
    assert so.loss_divergence(3, 4, 4, 4, 8, 0, 4, 1.0) == pytest.approx(3.0, rel=1e-15)


def test_oracle_weight_divergence_hand_worked():
    # step 1: sqrt(1 - b2) / (1 - b1); b1 = 0.5, b2 = 0.75 -> 0.5 / 0.5 = 1; lr 0.1, |T| 6, |g_err| 2, N K = 16 -> 0.1 * 12 / 4 = 0.3;
    # |W| = 3, 2 layers -> 0.05
    assert so.weight_divergence(6, 2, 4, 4, 0.1, 0.5, 0.75, 1, 3.0, 2) == pytest.approx(0.05, rel=1e-15)
    # large step: the bias correction tends to 1
    assert so.weight_divergence(6, 2, 4, 4, 0.1, 0.9, 0.95, 10 ** 6, 3.0, 1) == pytest.approx(0.1, rel=1e-12)


def test_library_formulas_match_the_oracle(api):
    rng = np.random.default_rng(0)
    for _ in range(20):
        a = [float(v) for v in rng.uniform(0.1, 10, 4)]
        M, K, N = (int(v) for v in rng.integers(64, 4096, 3))
        loss = float(rng.uniform(-5, 5))
        assert api.snip_loss_divergence(a[0], a[1], M, K, a[2], a[3], N, loss) == pytest.approx(so.loss_divergence(a[0], a[1], M, K, a[2], a[3], N, loss), rel=1e-14)
        step = int(rng.integers(1, 1000))
        assert api.snip_weight_divergence(a[0], a[1], N, K, 1e-3, 0.9, 0.95, step, a[2], 7) == pytest.approx(
            so.weight_divergence(a[0], a[1], N, K, 1e-3, 0.9, 0.95, step, a[2], 7), rel=1e-14)


def random_problem(rng, m, n, distinct_work=3):
    """Layers of a few distinct sizes; option j runs k_j of the layer's three GEMMs in FP4; more FP4 costs quality."""
    sizes = rng.integers(1, 50, distinct_work)
    ks = sorted(rng.integers(0, 4, n))
    ks[0], ks[-1] = 0, 3
    q = [[float(rng.uniform(0, 1)) * (1 + k) for k in ks] for _ in range(m)]
    w = [[int(sizes[i % distinct_work]) * int(k) for k in ks] for i in range(m)]
    return q, w


@pytest.mark.parametrize("m,n,groups", [(1, 2, 1), (3, 4, 1), (5, 3, 1), (6, 4, 1), (6, 3, 2), (6, 2, 3), (4, 8, 2)])
def test_selection_equals_exhaustive_search(api, m, n, groups):
    rng = np.random.default_rng(100 * m + n + groups)
    for trial in range(12):
        q, w = random_problem(rng, m, n)
        total = sum(max(row) for row in w)
        for frac in (0.0, 0.2, 0.5, 0.8, 1.0):
            target = math.ceil(frac * total)
            ref = so.select_scheme_bruteforce(q, w, target, groups)
            if ref is None:
                with pytest.raises(api.SnipError):
                    api.snip_select_scheme(q, w, target, groups)
                continue
            choice, loss, work = api.snip_select_scheme(q, w, target, groups)
            assert loss == pytest.approx(ref[0], rel=1e-12, abs=1e-15)
            # the returned assignment is valid and attains the reported totals (it need not be the same optimum)
            assert sum(q[i][c] for i, c in enumerate(choice)) == pytest.approx(loss, rel=1e-12, abs=1e-15)
            assert work == sum(w[i][c] for i, c in enumerate(choice))
            per = m // groups
            for k in range(groups):
                assert sum(w[i][choice[i]] for i in range(k * per, (k + 1) * per)) >= -(-target // groups)


def test_paper_endpoints_all_fp8_and_all_fp4(api):
    """Options 0..7 = which of (fwd, dgrad, wgrad) run in FP4; FP4 always costs quality.  E_t = 0 -> option 0
    everywhere, E_t = 1 -> option 7 everywhere (Sec. 5.2)."""
    rng = np.random.default_rng(7)
    m = 28
    flops = [int(v) for v in rng.choice([16, 43, 48], m)]
    opts = list(itertools.product((0, 1), repeat=3))
    q = [[sum(o) * float(rng.uniform(0.5, 1.5)) + 1e-3 * sum(o) for o in opts] for _ in range(m)]
    w = [[f * sum(o) for o in opts] for f in flops]
    total = 3 * sum(flops)
    choice, loss, work = api.snip_select_scheme(q, w, 0)
    assert choice == [0] * m and loss == 0.0 and work == 0
    choice, loss, work = api.snip_select_scheme(q, w, total)
    assert choice == [7] * m and work == total
    # the loss never decreases as the target grows
    prev = -1.0
    for frac in np.linspace(0, 1, 11):
        _, loss, work = api.snip_select_scheme(q, w, math.ceil(frac * total))
        assert loss >= prev - 1e-12 and work >= math.ceil(frac * total)
        prev = loss


def test_llama_sized_problem_runs_and_beats_uniform_assignment(api):
    """32 blocks x 7 linears x 8 options with the 7B shapes' FLOPs: the optimum at E_t = 0.5 is at least as good as
    any uniform per-layer rule that reaches the same efficiency."""
    rng = np.random.default_rng(11)
    shapes = [(4096, 4096)] * 4 + [(4096, 11008)] * 2 + [(11008, 4096)]
    opts = list(itertools.product((0, 1), repeat=3))
    q, w = [], []
    for layer in range(32):
        for (K, N) in shapes:
            sens = float(np.exp(rng.normal()))
            q.append([sens * (0.2 * o[0] + 0.5 * o[1] + 1.0 * o[2]) for o in opts])
            w.append([2 * 16384 * K * N // (1 << 24) * sum(o) for o in opts])
    total = sum(max(r) for r in w)
    target = math.ceil(0.5 * total)
    choice, loss, work = api.snip_select_scheme(q, w, target)
    assert work >= target
    # uniform rule: fwd + dgrad... pick the cheapest single option that reaches >= 0.5 when applied everywhere
    for j, o in enumerate(opts):
        if sum(w[i][j] for i in range(len(w))) >= target:
            assert loss <= sum(q[i][j] for i in range(len(q))) + 1e-9
    # pipeline form: 4 stages of 56 layers, each reaching a quarter of the target
    choice_pp, loss_pp, _ = api.snip_select_scheme(q, w, target, 4)
    assert loss_pp >= loss - 1e-12
    for k in range(4):
        assert sum(w[i][choice_pp[i]] for i in range(56 * k, 56 * (k + 1))) >= -(-target // 4)


def test_malformed_input_is_refused(api):
    with pytest.raises(api.SnipError):
        api.snip_select_scheme([[0.0, 1.0]] * 3, [[0, 1]] * 3, 1, 2)          # 3 layers, 2 groups
    with pytest.raises(api.SnipError):
        api.snip_select_scheme([[0.0, float("nan")]], [[0, 1]], 1)
    with pytest.raises(api.SnipError):
        api.snip_select_scheme([[0.0, 1.0]], [[0, 1]], 5)                       # unreachable target
