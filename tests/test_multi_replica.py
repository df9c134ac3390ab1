"""Replica bookkeeping of multi-GPU runs (no data-path collective): two gloo ranks on CPU check that timings
are reduced with MAX, work with SUM, and that whole-job throughput divides by the slowest rank."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world_size, port, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world_size)
    from paper_2607_24434_b200 import multi
    assert multi.world() == world_size and multi.rank() == rank
    multi.barrier()
    # rank r "ran" 100 steps of 4 tokens in (10 + 5 r) ms and launched 500 kernels
    agg = multi.aggregate({"step": 10.0 + 5.0 * rank, "e2e": 20.0 - 3.0 * rank}, units=400, launches=500)
    ret[rank] = (agg["step"], agg["e2e"], agg["units"], agg["launches"], multi.throughput(agg["units"], agg["step"]))
    multi.barrier()
    dist.destroy_process_group()


def test_two_replicas_aggregate_max_time_and_summed_work():
    world_size = 2
    port = _free_port()
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(world_size, port, ret), nprocs=world_size, join=True)
    for r in range(world_size):
        step, e2e, units, launches, thr = ret[r]
        assert step == 15.0 and e2e == 20.0            # max over ranks
        assert units == 800.0 and launches == 1000.0   # summed over ranks
        assert abs(thr - 800.0 / 0.015) < 1e-6


def test_single_process_is_identity():
    from paper_2607_24434_b200 import multi
    agg = multi.aggregate({"step": 7.0}, units=12, launches=3)
    assert agg == {"step": 7.0, "units": 12.0, "launches": 3.0}
    assert multi.world() == 1 and multi.rank() == 0
