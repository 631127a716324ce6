"""GPU parity of the extended service model (gorgo_sim_set_service_model: decode slow-down with
the busy slots, admission under a KV-token budget) against the oracle: population evaluation on
small and reduced workloads, per-request times through batched routing, the hand cases, and
switching it off again."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import gorgo_oracle as O
from paper_2602_11688_b200 import workloads as W
from tests.util import small_trace


def _population(sim, gb, w, scale):
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


@pytest.mark.parametrize("R,slots", [(3, 2), (16, 5), (64, 3), (5, 40)])
@pytest.mark.parametrize("slowdown,budget", [(0.4, 0), (0.0, 3000), (0.15, 2500)])
def test_population_with_the_extended_service_model(R, slots, slowdown, budget):
    from paper_2602_11688_b200 import binding as gb
    rng = np.random.default_rng(R * 7 + slots)
    reqs = small_trace(R + slots, n_req=400, rate_ms=12.0)
    K = 3 + R if R > 32 else 3
    params = np.concatenate([rng.normal(1.0, 0.3, size=(4, 3)), rng.lognormal(0, 0.3, size=(4, K - 3))], axis=1)
    w = W.handmade(rng.uniform(5, 60, size=R), reqs, slots=slots, cache_blocks=9, params=params)
    sim = gb.GorgoSim(w)
    try:
        assert gb.gorgo_sim_set_service_model(sim.h, slowdown, budget) == gb.GORGO_OK
        on = _population(sim, gb, w, 0.8)
        assert gb.gorgo_sim_set_service_model(sim.h, 0.0, 0) == gb.GORGO_OK
        off = _population(sim, gb, w, 0.8)
        assert gb.gorgo_sim_set_service_model(sim.h, -1.0, 0) == gb.GORGO_ERR_INVALID_ARG
        assert gb.gorgo_sim_set_service_model(sim.h, float("nan"), 0) == gb.GORGO_ERR_INVALID_ARG
    finally:
        sim.close()
    _check(on, w, 0.8, decode_slowdown=slowdown, kv_budget_tokens=budget)
    _check(off, w, 0.8)
    assert not np.array_equal(on["p95_e2e"], off["p95_e2e"])


def test_regions_reduced_with_slowdown_and_budget_and_replica_speeds():
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload("regions", n_requests=6000, cache_blocks=1500, population=6)
    R = w.spec.n_replicas
    rng = np.random.default_rng(2)
    tpot = rng.uniform(8.0, 30.0, size=R)
    sim = gb.GorgoSim(w)
    try:
        assert gb.gorgo_sim_set_service_model(sim.h, 0.05, 40_000) == gb.GORGO_OK
        assert gb.gorgo_sim_set_replica_speeds(sim.h, None, tpot) == gb.GORGO_OK
        got = _population(sim, gb, w, 1.0)
    finally:
        sim.close()
    _check(got, w, 1.0, decode_slowdown=0.05, kv_budget_tokens=40_000, rep_tpot_ms=tpot)


def _route_all(gb, sim, w, chunks):
    import torch
    rc, nbytes = gb.gorgo_state_bytes(sim.h)
    state = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    assert gb.gorgo_sim_reset(sim.h, state, sim.stream) == gb.GORGO_OK
    N = w.n_requests
    ttft = torch.empty(N, dtype=torch.float64, device="cuda")
    e2e = torch.empty(N, dtype=torch.float64, device="cuda")
    route = torch.empty(N, dtype=torch.uint8, device="cuda")
    first = 0
    for c in chunks:
        rc = gb.gorgo_route_batch(sim.h, w.params[0], 1.0, first, c, state, sim.stream,
                                  route[first:], None, ttft[first:], e2e[first:])
        assert rc == gb.GORGO_OK
        first += c
    rc, seen = gb.gorgo_state_status(sim.h, state, sim.stream)
    assert rc == gb.GORGO_OK and seen == N
    return ttft.cpu().numpy(), e2e.cpu().numpy(), route.cpu().numpy()


def test_hand_cases_and_batches_on_a_persistent_state():
    from paper_2602_11688_b200 import binding as gb
    # the two hand cases of the oracle's pins, request by request
    reqs = [(0.0, 1000, 11, [1, 2]), (10.0, 1000, 3, [3, 4]), (20.0, 1000, 2, [5, 6]),
            (200.0, 1000, 2, [7, 8])]
    w = W.handmade([5.0], reqs, slots=2, cache_blocks=100, prefill_ms_per_token=0.01,
                   tpot_ms=10.0, params=[(1.0, 1.0, 1.0)])
    sim = gb.GorgoSim(w)
    assert gb.gorgo_sim_set_service_model(sim.h, 0.5, 0) == gb.GORGO_OK
    ttft, e2e, _ = _route_all(gb, sim, w, [4])
    sim.close()
    np.testing.assert_allclose(ttft, [15.0, 15.0, 45.0, 15.0], rtol=1e-14)
    np.testing.assert_allclose(e2e, [115.0, 45.0, 60.0, 25.0], rtol=1e-14)
    reqs = [(0.0, 1000, 11, [1, 2]), (1.0, 1500, 6, [3, 4, 5]), (2.0, 1000, 3, [6, 7]),
            (3.0, 4000, 1, list(range(10, 18)))]
    w = W.handmade([5.0], reqs, slots=3, cache_blocks=100, prefill_ms_per_token=0.01,
                   tpot_ms=10.0, params=[(1.0, 1.0, 1.0)])
    sim = gb.GorgoSim(w)
    assert gb.gorgo_sim_set_service_model(sim.h, 0.0, 3000) == gb.GORGO_OK
    ttft, e2e, _ = _route_all(gb, sim, w, [1, 2, 1])          # the KV state carries over batches
    sim.close()
    np.testing.assert_allclose(ttft, [15.0, 20.0, 79.0, 152.0], rtol=1e-14)
    np.testing.assert_allclose(e2e, [115.0, 70.0, 99.0, 152.0], rtol=1e-14)
    # a random trace in uneven batches equals the oracle's one-shot run, time for time
    rng = np.random.default_rng(9)
    reqs = small_trace(21, n_req=500, rate_ms=10.0)
    w = W.handmade(rng.uniform(5, 40, size=4), reqs, slots=3, cache_blocks=12, params=[(0.9, 1.0, 0.4)])
    sim = gb.GorgoSim(w)
    assert gb.gorgo_sim_set_service_model(sim.h, 0.2, 2600) == gb.GORGO_OK
    ttft, e2e, route = _route_all(gb, sim, w, [1, 99, 250, 150])
    sim.close()
    ref = O.replay(w, w.params[0], 1.0, decode_slowdown=0.2, kv_budget_tokens=2600)[0]
    assert route.tolist() == ref.route.tolist()
    assert ttft.tolist() == ref.ttft.tolist() and e2e.tolist() == ref.e2e.tolist()
