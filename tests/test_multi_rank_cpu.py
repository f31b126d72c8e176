"""N > 1 path on CPU (gloo, world size 2): the path shards over independent replicas with no data-path
collective; what the ranks exchange is the timing (MAX over ranks) behind the whole-job rate."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # rank 1 is the slow replica
    value, ms = bench.aggregate_over_ranks(2.0 + rank, work_per_replica=6e12, unit_scale=1e12, dist=dist)
    # every rank's replica is generated from the same seeds: identical inputs, independent work
    from paper_2607_02980_b200 import workloads as wl
    cfg = wl.CONFIGS[1].scaled(L=256, K=2)
    q = wl.make_prefill_inputs(cfg, "cpu")["q"]
    digest = torch.tensor([float(q.float().sum())], dtype=torch.float64)
    both = [torch.zeros_like(digest) for _ in range(world)]
    dist.all_gather(both, digest)
    out[rank] = (value, ms, [float(x) for x in both])
    dist.barrier()
    dist.destroy_process_group()


def test_replica_timing_is_max_over_ranks_and_rate_is_whole_job():
    world, port = 2, _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    for rank in range(world):
        value, ms, digests = out[rank]
        assert ms == 3.0                                  # the slowest rank sets the job's step time
        assert abs(value - 2 * 6e12 / 3e-3 / 1e12) < 1e-9     # units of all ranks / that time
        assert digests[0] == digests[1]                   # replicas see the same seeded inputs


def test_single_process_aggregate_is_plain_rate():
    sys.path.insert(0, ROOT)
    import bench
    value, ms = bench.aggregate_over_ranks(4.0, work_per_replica=8e9, unit_scale=1e9)
    assert ms == 4.0 and abs(value - 8e9 / 4e-3 / 1e9) < 1e-9


def test_bench_gpus_2_spawns_its_own_ranks():
    """`python bench.py --gpus 2` started by hand (no RANK in the environment) starts two ranks itself: here the
    host-only self-test of that plumbing (gloo), whose rank 0 prints the line with n_gpus = 2 and the MAX-over-ranks
    step time."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--selftest-ranks"],
                         capture_output=True, text=True, env=env, cwd=ROOT, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["n_gpus"] == 2 and line["ms_per_step"] == 2.0          # ranks report 1.0 and 2.0 ms
    assert abs(line["value"] - 2 * 2.0e12 / 2e-3 / 1e12) < 1e-9


def test_reference_arm_through_the_spawner_prints_one_line():
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference",
                          "--workload", "cfg0", "--steps", "1", "--warmup", "0"],
                         capture_output=True, text=True, env=env, cwd=ROOT, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [x for x in res.stdout.strip().splitlines() if x.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2
