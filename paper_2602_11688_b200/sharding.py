"""Multi-GPU plumbing: candidates are independent replays, so a population is split across
ranks (one process per GPU) with no collective on the data path; the only exchanges are the
max-over-ranks of a device time and an all-gather of the per-candidate results.  Works with any
``torch.distributed`` backend (NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

from typing import List, Tuple

import numpy as np


def shard_bounds(n_candidates: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous, balanced split: the first ``n % world`` ranks get one candidate more."""
    base, extra = divmod(int(n_candidates), int(world))
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def shard_population(params: np.ndarray, rank: int, world: int) -> np.ndarray:
    lo, hi = shard_bounds(params.shape[0], rank, world)
    return np.ascontiguousarray(params[lo:hi])


def weak_scaling_population(base_params: np.ndarray, rank: int) -> np.ndarray:
    """Population of one rank when every rank evaluates as many candidates as a single GPU
    would: rank 0 keeps the base draw, the others redraw the three weights (seeded by rank) and
    keep any per-replica normalisers."""
    if rank == 0:
        return np.ascontiguousarray(base_params)
    rng = np.random.default_rng(1000 + rank)
    w = rng.normal(1.0, 0.3, size=(base_params.shape[0], 3))
    return np.ascontiguousarray(np.concatenate([w, base_params[:, 3:]], axis=1))


def max_over_ranks(value: float, device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def gather_results(local: np.ndarray, n_candidates: int, device=None) -> np.ndarray:
    """All-gather per-candidate results (first axis = candidates of this rank's shard, split by
    ``shard_bounds``) into the full population order on every rank."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return np.asarray(local)
    world, rank = dist.get_world_size(), dist.get_rank()
    sizes = [shard_bounds(n_candidates, r, world) for r in range(world)]
    longest = max(hi - lo for lo, hi in sizes)
    pad = np.zeros((longest,) + tuple(local.shape[1:]), dtype=local.dtype)
    pad[: local.shape[0]] = local
    mine = torch.from_numpy(pad).to(device) if device is not None else torch.from_numpy(pad)
    parts: List = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine)
    out = [parts[r][: hi - lo].cpu().numpy() for r, (lo, hi) in enumerate(sizes)]
    return np.concatenate(out, axis=0)


def run_ranks(rank: int, world: int, base_params: np.ndarray, evaluate, steps: int, warmup: int,
              timer, barrier, device=None):
    """The rank logic of the benchmark, independent of what evaluates a population: every rank
    takes a population of the single-GPU size (weak scaling), runs `warmup` untimed and `steps`
    timed evaluations between two barriers, and the job's time is the slowest rank's.
    `evaluate(params)` returns this rank's per-candidate results [P, 2]; `timer()` returns a
    callable that gives the milliseconds since it was created (CUDA events on the launching stream
    in the benchmark, a wall clock in the CPU test).  Returns (ms_per_step of the job, this rank's
    results of the last step, candidates evaluated per step by the whole job)."""
    params = weak_scaling_population(base_params, rank)
    last = None
    for _ in range(warmup):
        last = evaluate(params)
    barrier()
    elapsed = timer()
    for _ in range(steps):
        last = evaluate(params)
    ms = elapsed()
    barrier()
    ms_job = max_over_ranks(ms, device)
    return ms_job / max(1, steps), np.asarray(last), int(params.shape[0]) * int(world)
