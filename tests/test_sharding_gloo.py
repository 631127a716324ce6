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
