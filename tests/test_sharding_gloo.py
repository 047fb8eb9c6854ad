"""The N > 1 host logic (rank-owned workloads, barrier, max-over-ranks timing, aggregate throughput) on two
CPU processes over gloo."""

import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_05326_b200 import sharding, workloads


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = sharding.rank_workload(workloads.config(0), rank)
    k, _ = workloads.gen_prompt_kv(wl, 0)
    sharding.barrier()
    ms, e2e = sharding.max_over_ranks([10.0 + 5.0 * rank, 3.0 - rank])
    out[rank] = (wl.seed, float(k.float().sum()), ms, e2e, sharding.aggregate_steps_per_second(world, 64, ms))
    dist.destroy_process_group()


def test_two_ranks_own_disjoint_sequences_and_agree_on_the_slowest_time():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    (s0, k0, ms0, e0, v0), (s1, k1, ms1, e1, v1) = out[0], out[1]
    assert s1 == s0 + 1 and k0 != k1           # same shape, different seeded sequences
    assert ms0 == ms1 == 15.0 and e0 == e1 == 3.0  # max over ranks, identical everywhere
    assert v0 == v1 == 2 * 64 / 15e-3


def test_single_process_is_the_identity():
    assert sharding.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert sharding.aggregate_steps_per_second(1, 100, 50.0) == 2000.0


def _bench(*argv):
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    return subprocess.run([sys.executable, os.path.join(root, "bench.py")] + list(argv), capture_output=True, text=True,
                          env=env, timeout=600)


def test_bench_gpus_n_starts_n_ranks_and_prints_one_line():
    """`python bench.py --gpus 2` outside a launcher starts two ranks itself; the CPU arm shows it without a GPU:
    rank 0 alone prints the line, which names two ranks."""
    import json
    r = _bench("--gpus", "2", "--impl", "reference", "--steps", "1", "--warmup", "0")
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["impl"] == "reference" and line["value"] > 0


def test_bench_refuses_to_run_fewer_ranks_than_asked():
    if torch.cuda.is_available() and torch.cuda.device_count() >= 8:
        return
    r = _bench("--gpus", "8", "--steps", "1", "--warmup", "0")
    assert r.returncode != 0 and "--gpus 8" in r.stderr
    assert not [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
