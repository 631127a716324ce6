"""GPU parity at the full sizes of the three large configurations, in the launch configuration
the benchmark times (whole population, waves when the state does not fit).  The oracle replays a
handful of candidates in full (one thread each); for those, every route, every prefix-hit length,
the cache digests, the counters and both p95 values are compared.  For all other candidates the
properties that hold at any size are checked."""
import numpy as np
import pytest

from paper_2602_11688_b200 import workloads as W
from tests.util import assert_candidate_matches, gpu_eval, oracle_eval

pytestmark = pytest.mark.gpu


def check_full(name, scale, n_oracle, seed_pick=0):
    import torch
    w = W.make_workload(name)
    P, N, R = w.params.shape[0], w.n_requests, w.spec.n_replicas
    free_b, _ = torch.cuda.mem_get_info()
    gpu = gpu_eval(w, scale=scale, route=True, hit=True, digest=True, stats=True,
                   max_bytes=int(free_b * 0.8) - P * N * 3)
    # properties for every candidate
    assert gpu["route"].max() < R
    nblk = np.diff(w.hash_off.astype(np.int64))
    assert (gpu["hit"] <= nblk[None, :]).all()
    assert (gpu["digest"][:, :, 0] <= w.spec.cache_blocks).all()
    assert (gpu["stats"][:, 2] == nblk.sum()).all()
    assert (gpu["stats"][:, 1] == gpu["hit"].astype(np.int64).sum(axis=1)).all()
    assert np.isfinite(gpu["p95_ttft"]).all() and (gpu["p95_e2e"] >= gpu["p95_ttft"]).all()
    # occupancy bookkeeping: blocks inserted minus blocks evicted is what the caches hold
    # (inserted = all blocks - blocks found present; at least the prefix hits were present)
    assert (gpu["digest"][:, :, 0].sum(axis=1).astype(np.int64)
            <= gpu["stats"][:, 2].astype(np.int64) - gpu["stats"][:, 1].astype(np.int64)
            - gpu["stats"][:, 3].astype(np.int64)).all()
    # full comparison on a few candidates: the first, the last, extreme weights
    rng = np.random.default_rng(seed_pick)
    pick = {0, P - 1, int(np.argmin(w.params[:, 2])), int(np.argmax(w.params[:, 1]))}
    while len(pick) < n_oracle:
        pick.add(int(rng.integers(P)))
    pick = sorted(pick)[:n_oracle] if len(pick) > n_oracle else sorted(pick)
    refs = oracle_eval(w, w.params[pick], scale, threads=8)
    for idx, ref in zip(pick, refs):
        assert_candidate_matches(gpu, idx, ref)


def test_longctx_full_size():
    check_full("longctx", 0.5, n_oracle=6)


def test_sweep_full_size_most_and_least_saturated_scale():
    check_full("sweep", 0.25, n_oracle=4)
    check_full("sweep", 1.0, n_oracle=2, seed_pick=1)


def test_largest_full_size_in_waves():
    check_full("largest", 0.5, n_oracle=4)


def test_longctx_full_size_cache_digests_every_65536_requests():
    """One candidate of the full-size long-context workload routed in batches of 2^16 requests on a
    persistent state; after every batch the digests of all replica caches equal the oracle's at
    the same request, so a divergence would be pinned down to one batch."""
    import torch
    from oracle import gorgo_oracle as O
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload("longctx")
    N, R = w.n_requests, w.spec.n_replicas
    weights = w.params[3]
    sim = gb.GorgoSim(w)
    rc, nbytes = gb.gorgo_state_bytes(sim.h)
    assert rc == gb.GORGO_OK
    state = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    assert gb.gorgo_sim_reset(sim.h, state, sim.stream) == gb.GORGO_OK
    oracle = O.Oracle.from_workload(w)
    step = 1 << 16
    route = torch.empty(step, dtype=torch.uint8, device="cuda")
    digest = torch.empty((R, 2), dtype=torch.uint64, device="cuda")
    checkpoints = 0
    for first in range(0, N, step):
        count = min(step, N - first)
        rc = gb.gorgo_route_batch(sim.h, weights, 0.5, first, count, state, sim.stream, route)
        assert rc == gb.GORGO_OK
        assert gb.gorgo_state_digest(sim.h, state, sim.stream, digest) == gb.GORGO_OK
        torch.cuda.synchronize()
        ref = oracle.run(weights, 0.5, count=count)
        assert (route[:count].cpu().numpy() == ref.route).all(), f"routes differ in [{first}, {first + count})"
        assert digest.cpu().numpy().tolist() == oracle.digest().tolist(), \
            f"cache digests differ after request {first + count}"
        checkpoints += 1
    rc, seen = gb.gorgo_state_status(sim.h, state, sim.stream)
    assert rc == gb.GORGO_OK and seen == N and checkpoints == -(-N // step)
    oracle.close()
    sim.close()
