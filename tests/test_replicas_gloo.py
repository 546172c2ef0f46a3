"""The N > 1 accounting (independent replicas, max over ranks) with two gloo ranks on the CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2510_08431_b200 import replicas
    # rank 1 is the slow one: 30 ms for 3 steps against 12 ms
    ms = 12.0 if rank == 0 else 30.0
    dist.barrier()
    thr, ms_per_step, w = replicas.aggregate_throughput(work_per_rank=5.0e12, ms_this_rank=ms, steps=3, dist=dist)
    mx = replicas.max_over_ranks(float(rank + 1), dist)
    dist.barrier()
    out.put((rank, thr, ms_per_step, w, mx))
    dist.destroy_process_group()


def test_two_rank_aggregation_takes_the_slowest_rank():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, thr, ms_per_step, w, mx in res:
        assert w == 2 and mx == 2.0
        assert ms_per_step == 10.0                      # 30 ms / 3 steps: the slowest rank decides
        assert abs(thr - 2 * 5.0e12 / 10.0e-3) < 1.0   # all ranks' work over that time


def test_single_process_is_identity():
    from paper_2510_08431_b200 import replicas
    thr, ms, w = replicas.aggregate_throughput(2.0e12, 8.0, 4)
    assert w == 1 and ms == 2.0 and thr == 2.0e12 / 2.0e-3
    assert replicas.max_over_ranks(3.5) == 3.5
