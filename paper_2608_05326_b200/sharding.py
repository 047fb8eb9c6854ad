"""Host-side helpers for running the path on several GPUs.

The path shards by unit (one (layer, sequence) pair) with no exchange between units, so N GPUs simply run N
disjoint sets of sequences of the same shape (weak scaling).  The only communication is for measurement: a
barrier and a max over ranks of the device-timed durations."""

from dataclasses import replace

import torch
import torch.distributed as dist


def rank_workload(wl, rank):
    """The workload a rank owns: same shape, its own seeded sequences."""
    return replace(wl, seed=wl.seed + rank)


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum over all ranks of a list of floats (identity without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    if dist.get_backend() == "gloo":
        device = "cpu"
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def barrier():
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def aggregate_steps_per_second(world, steps, slowest_rank_ms):
    """Whole-job throughput: every rank ran `steps` steps of its own sequences in the slowest rank's time."""
    return world * steps / (slowest_rank_ms * 1e-3)
