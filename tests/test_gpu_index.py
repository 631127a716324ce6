"""GPU parity of the drifting proxy index (gorgo_sim_set_proxy_index: the score takes its prefix
hits from the blocks ever dispatched to a replica, prefill and cache follow the real LRU) against
the oracle."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import gorgo_oracle as O
from paper_2602_11688_b200 import workloads as W
from tests.util import small_trace


def _population(sim, w, scale):
    import torch
    out = sim.eval_population(w.params, scale, want_route=True, want_hit=True, want_digest=True)
    torch.cuda.synchronize()
    assert int(out["status"].abs().sum()) == 0
    return {k: (None if v is None else v.cpu().numpy()) for k, v in out.items()}


def _check(got, w, scale, **model):
    for p in range(w.params.shape[0]):
        res, pt, pe, dg, _ = O.replay(w, w.params[p], scale, **model)
        assert got["route"][p].tolist() == res.route.tolist(), p
        assert got["hit"][p].tolist() == res.hit.tolist()
        assert got["digest"][p].tolist() == dg.tolist()
        assert abs(got["p95_ttft"][p] - pt) <= 1e-9 * abs(pt) and abs(got["p95_e2e"][p] - pe) <= 1e-9 * abs(pe)


@pytest.mark.parametrize("R,structured", [(3, True), (17, False), (64, True)])
def test_population_scored_with_the_index(R, structured):
    from paper_2602_11688_b200 import binding as gb
    rng = np.random.default_rng(R)
    reqs = small_trace(R + 2, n_req=400, structured=structured)
    K = 3 + R if R > 32 else 3
    params = np.concatenate([rng.normal(1.0, 0.3, size=(5, 3)), rng.lognormal(0, 0.3, size=(5, K - 3))], axis=1)
    params[0, :3] = (0.0, 1.0, 0.0)                         # follow the believed prefix alone
    w = W.handmade(rng.uniform(5, 60, size=R), reqs, slots=2, cache_blocks=9, params=params)
    sim = gb.GorgoSim(w)
    try:
        assert gb.gorgo_sim_set_proxy_index(sim.h, True) == gb.GORGO_OK
        index = _population(sim, w, 1.0)
        index_half = _population(sim, w, 0.5)
        assert gb.gorgo_sim_set_proxy_index(sim.h, False) == gb.GORGO_OK
        cache = _population(sim, w, 1.0)
    finally:
        sim.close()
    _check(index, w, 1.0, proxy_index=True)
    _check(index_half, w, 0.5, proxy_index=True)
    _check(cache, w, 1.0)
    assert not np.array_equal(index["route"], cache["route"])     # 9-block caches evict all the time


def test_hand_case_promised_hit_is_not_there_on_gpu():
    # (the oracle's hand case) two replicas with 2-block caches: the index of replica 0 still lists
    # A,B after C,D pushed them out, so [A,B] goes there again and pays the full prefill
    import torch
    from paper_2602_11688_b200 import binding as gb
    reqs = [(0.0, 1024, 1, [1, 2]), (100.0, 1024, 1, [3, 4]), (200.0, 1024, 1, [1, 2]),
            (300.0, 1024, 1, [3, 4])]
    w = W.handmade([10.0, 10.0], reqs, slots=4, cache_blocks=2, prefill_ms_per_token=0.01,
                   params=[(0.0, 1.0, 0.0)])
    sim = gb.GorgoSim(w)
    assert gb.gorgo_sim_set_proxy_index(sim.h, True) == gb.GORGO_OK
    rc, nbytes = gb.gorgo_state_bytes(sim.h)
    state = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    assert gb.gorgo_sim_reset(sim.h, state, sim.stream) == gb.GORGO_OK
    N = len(reqs)
    route = torch.empty(N, dtype=torch.uint8, device="cuda")
    ttft = torch.empty(N, dtype=torch.float64, device="cuda")
    # in two batches: the index spans the batches of a persistent state
    assert gb.gorgo_route_batch(sim.h, w.params[0], 1.0, 0, 2, state, sim.stream, route, None, ttft) == gb.GORGO_OK
    assert gb.gorgo_route_batch(sim.h, w.params[0], 1.0, 2, 2, state, sim.stream, route[2:], None, ttft[2:]) == gb.GORGO_OK
    torch.cuda.synchronize()
    assert route.cpu().numpy().tolist() == [0, 0, 0, 0]
    np.testing.assert_allclose(ttft.cpu().numpy(), [10.0 + 10.24] * 4, rtol=1e-12)
    sim.close()


def test_roomy_caches_index_equals_cache_on_gpu():
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload("regions", n_requests=4000, cache_blocks=200_000, population=4)
    sim = gb.GorgoSim(w)
    try:
        cache = _population(sim, w, 1.0)
        assert gb.gorgo_sim_set_proxy_index(sim.h, True) == gb.GORGO_OK
        index = _population(sim, w, 1.0)
    finally:
        sim.close()
    for k in ("route", "hit", "digest", "p95_ttft", "p95_e2e"):
        assert np.array_equal(cache[k], index[k]), k


def test_regions_reduced_with_index_and_everything_else_switched_on():
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload("regions", n_requests=6000, cache_blocks=1500, population=5)
    G, R = w.spec.n_regions, w.spec.n_replicas
    rng = np.random.default_rng(5)
    span = float(w.ts_ms[-1])
    E = 30
    series = w.rtt_ms[None] * np.exp(np.cumsum(rng.normal(0, 0.15, size=(E, G, R)), axis=0))
    sim = gb.GorgoSim(w)
    try:
        assert gb.gorgo_sim_set_proxy_index(sim.h, True) == gb.GORGO_OK
        only_index = _population(sim, w, 1.0)
        assert gb.gorgo_sim_set_rtt_series(sim.h, series, span / E, 0.3) == gb.GORGO_OK
        assert gb.gorgo_sim_set_service_model(sim.h, 0.05, 0) == gb.GORGO_OK
        got = _population(sim, w, 1.0)
    finally:
        sim.close()
    _check(only_index, w, 1.0, proxy_index=True)
    _check(got, w, 1.0, proxy_index=True, rtt_series=series, epoch_ms=span / E, alpha=0.3, decode_slowdown=0.05)
