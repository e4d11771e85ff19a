"""The N > 1 path of the benchmark is "independent replicas": each rank draws its own batch and the
slowest rank's time counts.  Its host logic, exercised with two gloo ranks on the CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    import workloads as W
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = bench.rank_config(W.get_config("cfg1"), rank)
    topk = W.routing_topk(cfg)
    # every rank reports a different time; the job's step time is the slowest one
    slowest = bench.max_over_ranks(10.0 * (rank + 1), world, "cpu")
    rate = bench.whole_job_rate(cfg.L, 4, world, slowest)
    digest = int(topk.to(torch.int64).sum())
    gathered = [None] * world
    dist.all_gather_object(gathered, (cfg.seed, digest))
    if rank == 0:
        ret["slowest"] = slowest
        ret["rate"] = rate
        ret["seeds"] = [g[0] for g in gathered]
        ret["digests"] = [g[1] for g in gathered]
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_are_independent_replicas_timed_by_the_slowest():
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        ret = mgr.dict()
        mp.spawn(_worker, args=(world, port, ret), nprocs=world, join=True)
        assert ret["slowest"] == 20.0
        assert ret["rate"] == world * 1 * 4 / 20e-3            # whole-job plans/s
        assert len(set(ret["seeds"])) == world and len(set(ret["digests"])) == world
