"""Host-side bookkeeping for running N independent replicas of the single-GPU path.

The hot path does not shard (one GPU, no collectives): with N GPUs, N processes each run the whole
path on their own inputs.  The only thing they exchange is the timing: the job's time is the slowest
replica's, the job's work is the sum."""
from __future__ import annotations


def combine_replicas(ms_local: float, units_local: float, dist=None, device=None):
    """Returns (max ms over ranks, total units over ranks).  `dist` is torch.distributed (initialised)
    or None for a single process."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(ms_local), float(units_local)
    import torch
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())
