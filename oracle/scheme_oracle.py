"""Plain, slow reference for the host side of scheme generation (test infrastructure only; nothing in the
product path imports this module).

Follows the paper's Sec. 4.2 (loss divergence), Sec. 4.3 (weight divergence) and Sec. 5.2 / 5.3 (one
option per layer minimising the summed quality loss subject to an efficiency target, optionally per
pipeline stage) by writing the definitions out: the selection is an exhaustive search over all n^m
assignments, so it is only usable for tiny problems."""
from __future__ import annotations

import itertools
import math


def loss_divergence(grad_x_norm, err_x_norm, M, K, grad_w_norm, err_w_norm, N, loss):
    """Sec. 4.2: the two first-order terms |dL/dX||dX_err|/sqrt(MK) and |dL/dW||dW_err|/sqrt(NK) add in
    quadrature (the cross term is dropped), normalised by |L| (Definition of Delta L)."""
    tx = grad_x_norm * err_x_norm / math.sqrt(M * K)
    tw = grad_w_norm * err_w_norm / math.sqrt(N * K)
    return math.sqrt(tx * tx + tw * tw) / abs(loss)


def weight_divergence(sens_norm, grad_err_norm, N, K, lr, beta1, beta2, step, weight_norm, num_layers):
    """Sec. 4.3: |W' - W| ~ alpha sqrt(1-beta2^t)/(1-beta1^t) |T|_F |g_err|_F / sqrt(NK); Definition of
    Delta W divides by |W| and averages over the layers."""
    bias = math.sqrt(1.0 - beta2 ** step) / (1.0 - beta1 ** step)
    return lr * bias * sens_norm * grad_err_norm / math.sqrt(N * K) / weight_norm / num_layers


def select_scheme_bruteforce(q, w, target, num_groups=1):
    """Sec. 5.2 / 5.3 by enumeration.  q[i][j]: quality loss, w[i][j]: integer work (FLOPs run in FP4) of
    option j for layer i.  Every group of m / num_groups consecutive layers must reach
    ceil(target / num_groups).  Returns (min total loss, one optimal assignment) or None if infeasible."""
    m, n = len(q), len(q[0])
    per = m // num_groups
    group_target = -(-target // num_groups)
    best = None
    for assign in itertools.product(range(n), repeat=m):
        ok = True
        for k in range(num_groups):
            if sum(w[i][assign[i]] for i in range(k * per, (k + 1) * per)) < group_target:
                ok = False
                break
        if not ok:
            continue
        loss = sum(q[i][assign[i]] for i in range(m))
        if best is None or loss < best[0]:
            best = (loss, assign)
    return best
