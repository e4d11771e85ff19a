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


def test_bench_starts_its_own_ranks_when_asked_for_more_than_one_gpu():
    """`python bench.py --gpus 2` with no launcher around it must itself start two processes (here on the CPU:
    gloo, the launch path only) and report a two-rank job."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--rendezvous-only",
                        "--workload", "cfg1"], capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads([ln for ln in r.stdout.splitlines() if ln.startswith("{")][-1])
    assert line["n_gpus"] == 2 and line["gpus_requested"] == 2
    assert line["slowest_ms"] == 20.0                      # the slower of the two ranks' times
    assert len(set(line["seeds"])) == 2                    # every rank plans its own batch


def test_both_arms_describe_the_workload_with_the_same_config_object():
    import argparse
    import bench
    import workloads as W
    args = argparse.Namespace(workload="cfg4", gpus=1)
    cfg = W.get_config("cfg4")
    a = bench.config_dict(args, cfg)
    b = bench.config_dict(args, bench.rank_config(cfg, 0))
    assert a == b and a["workload"] == "cfg4" and a["routing_table_bytes"] == 48 * 1048576 * 8 * 4
    assert a["l2"] == "inputs larger than L2"
    sys_argv = sys.argv
    try:
        sys.argv = ["bench.py"]
        assert bench.parse_args().workload == "cfg4"       # the default is the largest single-GPU configuration
    finally:
        sys.argv = sys_argv
