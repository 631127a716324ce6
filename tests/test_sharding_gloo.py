"""The multi-GPU path without GPUs: two gloo ranks split a population, "evaluate" their shards
(a stand-in function of the parameters) and exchange only the timing maximum and the results."""
import os
import socket

import numpy as np
import torch.multiprocessing as mp

from paper_2602_11688_b200 import sharding as sh


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, n_cand, out_dir):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rng = np.random.default_rng(7)
    params = rng.normal(1.0, 0.3, size=(n_cand, 3))
    mine = sh.shard_population(params, rank, world)
    local = np.stack([mine.sum(axis=1), mine[:, 0] * 2.0], axis=1)      # stand-in "p95" pair
    full = sh.gather_results(local, n_cand)
    slowest = sh.max_over_ranks(10.0 + rank)
    weak = sh.weak_scaling_population(params, rank)
    np.savez(os.path.join(out_dir, f"r{rank}.npz"), full=full, slowest=slowest, weak=weak,
             lo_hi=np.array(sh.shard_bounds(n_cand, rank, world)))
    dist.destroy_process_group()


def _bench_worker(rank, world, port, out_dir):
    """The benchmark's own rank logic (sharding.run_ranks) with the evaluator stubbed: rank r
    "evaluates" in (r + 1) x 20 ms."""
    import time
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    base = np.random.default_rng(3).normal(1.0, 0.3, size=(6, 5))
    calls = []

    def evaluate(params):
        calls.append(params.copy())
        time.sleep(0.02 * (rank + 1))
        return np.stack([params[:, 0], params[:, 1] + rank], axis=1)

    def timer():
        t0 = time.perf_counter()
        return lambda: (time.perf_counter() - t0) * 1e3

    ms_per_step, last, per_step = sh.run_ranks(rank, world, base, evaluate, steps=3, warmup=2,
                                               timer=timer, barrier=dist.barrier)
    np.savez(os.path.join(out_dir, f"b{rank}.npz"), ms=ms_per_step, last=last, per_step=per_step,
             n_calls=len(calls), first=calls[0], same=all(np.array_equal(c, calls[0]) for c in calls))
    dist.destroy_process_group()


def test_two_gloo_ranks_run_the_benchmark_rank_logic(tmp_path):
    world = 2
    mp.spawn(_bench_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    base = np.random.default_rng(3).normal(1.0, 0.3, size=(6, 5))
    b0, b1 = np.load(tmp_path / "b0.npz"), np.load(tmp_path / "b1.npz")
    # weak scaling: every rank evaluates a population of the single-GPU size, warm-up + steps times
    assert int(b0["n_calls"]) == 5 and int(b1["n_calls"]) == 5 and bool(b0["same"]) and bool(b1["same"])
    assert int(b0["per_step"]) == 12 and int(b1["per_step"]) == 12
    assert np.array_equal(b0["first"], base)                   # rank 0 keeps the base draw
    assert b1["first"].shape == base.shape and not np.array_equal(b1["first"][:, :3], base[:, :3])
    assert np.array_equal(b1["first"][:, 3:], base[:, 3:])     # normalisers are kept
    # the job's time is the slowest rank's (40 ms per step), on both ranks
    assert float(b0["ms"]) == float(b1["ms"]) and 38.0 <= float(b0["ms"]) < 80.0
    assert np.array_equal(b1["last"][:, 1], b1["first"][:, 1] + 1)


def test_shard_bounds_cover_every_candidate_once():
    for n in (1, 7, 8, 256, 1000):
        for world in (1, 2, 3, 8):
            b = [sh.shard_bounds(n, r, world) for r in range(world)]
            assert b[0][0] == 0 and b[-1][1] == n
            assert all(b[i][1] == b[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in b]
            assert max(sizes) - min(sizes) <= 1


def test_two_gloo_ranks_split_and_gather(tmp_path):
    world, n_cand = 2, 11
    port = _free_port()
    mp.spawn(_worker, args=(world, port, n_cand, str(tmp_path)), nprocs=world, join=True)
    rng = np.random.default_rng(7)
    params = rng.normal(1.0, 0.3, size=(n_cand, 3))
    want = np.stack([params.sum(axis=1), params[:, 0] * 2.0], axis=1)
    r0 = np.load(tmp_path / "r0.npz")
    r1 = np.load(tmp_path / "r1.npz")
    assert np.array_equal(r0["full"], want) and np.array_equal(r1["full"], want)
    assert float(r0["slowest"]) == 11.0 and float(r1["slowest"]) == 11.0
    assert r0["lo_hi"].tolist() == [0, 6] and r1["lo_hi"].tolist() == [6, 11]
    assert np.array_equal(r0["weak"], params)                 # rank 0 keeps the base draw
    assert r1["weak"].shape == params.shape and not np.array_equal(r1["weak"], params)
