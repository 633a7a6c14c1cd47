"""The multi-GPU mode is 'replicas only': ranks share nothing but their timing.  Two gloo ranks on
CPU check that bookkeeping (max time, summed work)."""
import os

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2602_01410_b200.replicas import combine_replicas
    ms, units = combine_replicas(10.0 + 5.0 * rank, 100.0 * (rank + 1), dist)
    out[rank] = (ms, units)
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_max_time_and_total_work():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29517, out), nprocs=2, join=True)
    assert out[0] == out[1] == (15.0, 300.0)


def test_single_process_passthrough():
    from paper_2602_01410_b200.replicas import combine_replicas
    assert combine_replicas(3.5, 7.0) == (3.5, 7.0)
