"""GPU parity of the time-varying network (gorgo_sim_set_rtt_series: per-epoch RTT probes, the
proxy scoring with their moving average, requests delayed by the probe of their epoch) against
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


@pytest.mark.parametrize("R,G", [(3, 1), (17, 2), (64, 1)])
def test_population_under_a_changing_network(R, G):
    from paper_2602_11688_b200 import binding as gb
    rng = np.random.default_rng(R)
    reqs = small_trace(R + 1, n_req=400, rate_ms=15.0)
    K = 3 + R if R > 32 else 3
    params = np.concatenate([rng.normal(1.0, 0.3, size=(4, 3)), rng.lognormal(0, 0.3, size=(4, K - 3))], axis=1)
    params[0, :3] = (1.0, 0.0, 0.0)                        # follow the network signal alone
    org = rng.integers(0, G, size=len(reqs))
    base = rng.uniform(5, 60, size=(G, R))
    w = W.handmade(base, reqs, slots=2, cache_blocks=9, params=params, n_regions=G, origin=org)
    E = 9                                                   # the trace spans about 6 s: epochs of 700 ms
    series = base[None] * rng.uniform(0.3, 3.0, size=(E, G, R))
    sim = gb.GorgoSim(w)
    try:
        assert gb.gorgo_sim_set_rtt_series(sim.h, series, 700.0, 0.4) == gb.GORGO_OK
        moving = _population(sim, w, 1.0)
        half = _population(sim, w, 0.5)                     # the time scale moves requests across epochs
        flat = np.tile(base[None], (4, 1, 1))
        assert gb.gorgo_sim_set_rtt_series(sim.h, flat, 700.0, 0.4) == gb.GORGO_OK
        constant = _population(sim, w, 1.0)
        assert gb.gorgo_sim_set_rtt_series(sim.h, None) == gb.GORGO_OK
        static = _population(sim, w, 1.0)
        bad = gb.GORGO_ERR_INVALID_ARG
        assert gb.gorgo_sim_set_rtt_series(sim.h, series, 0.0, 0.4) == bad
        assert gb.gorgo_sim_set_rtt_series(sim.h, series, 700.0, 1.5) == bad
        assert gb.gorgo_sim_set_rtt_series(sim.h, -series, 700.0, 0.4) == bad
    finally:
        sim.close()
    _check(moving, w, 1.0, rtt_series=series, epoch_ms=700.0, alpha=0.4)
    _check(half, w, 0.5, rtt_series=series, epoch_ms=700.0, alpha=0.4)
    _check(static, w, 1.0)
    for k in ("route", "hit", "digest", "p95_ttft", "p95_e2e"):     # a constant series is the static matrix
        assert np.array_equal(constant[k], static[k]), k
    assert not np.array_equal(moving["route"], static["route"])


def test_belief_lags_the_network_hand_case_on_gpu():
    import torch
    from paper_2602_11688_b200 import binding as gb
    series = np.array([[[10.0, 40.0]], [[10.0, 40.0]], [[90.0, 40.0]], [[90.0, 40.0]]])
    ts = [50.0, 199.9, 200.0, 250.0, 350.0, 900.0]
    reqs = [(t, 512, 1, [100 + k]) for k, t in enumerate(ts)]
    w = W.handmade([10.0, 40.0], reqs, slots=8, cache_blocks=64, prefill_ms_per_token=0.0,
                   params=[(1.0, 0.0, 0.0)])
    sim = gb.GorgoSim(w)
    assert gb.gorgo_sim_set_rtt_series(sim.h, series, 100.0, 0.5) == gb.GORGO_OK
    rc, nbytes = gb.gorgo_state_bytes(sim.h)
    state = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    N = len(ts)
    for scale, routes, ttfts in ((1.0, [0, 0, 1, 1, 1, 1], [10.0, 10.0, 40.0, 40.0, 40.0, 40.0]),
                                 (0.5, [0, 0, 0, 0, 0, 1], [10.0, 10.0, 10.0, 10.0, 10.0, 40.0])):
        assert gb.gorgo_sim_reset(sim.h, state, sim.stream) == gb.GORGO_OK
        route = torch.empty(N, dtype=torch.uint8, device="cuda")
        ttft = torch.empty(N, dtype=torch.float64, device="cuda")
        rc = gb.gorgo_route_batch(sim.h, w.params[0], scale, 0, N, state, sim.stream, route, None, ttft)
        assert rc == gb.GORGO_OK
        torch.cuda.synchronize()
        assert route.cpu().numpy().tolist() == routes
        assert ttft.cpu().numpy().tolist() == ttfts
    sim.close()


def test_regions_reduced_with_a_drifting_network_and_the_extended_service_model():
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload("regions", n_requests=6000, cache_blocks=1500, population=5)
    G, R = w.spec.n_regions, w.spec.n_replicas
    rng = np.random.default_rng(4)
    span = float(w.ts_ms[-1])
    E = 40
    series = w.rtt_ms[None] * np.exp(np.cumsum(rng.normal(0, 0.15, size=(E, G, R)), axis=0))
    sim = gb.GorgoSim(w)
    try:
        assert gb.gorgo_sim_set_rtt_series(sim.h, series, span / E, 0.3) == gb.GORGO_OK
        assert gb.gorgo_sim_set_service_model(sim.h, 0.05, 0) == gb.GORGO_OK
        got = _population(sim, w, 1.0)
    finally:
        sim.close()
    _check(got, w, 1.0, rtt_series=series, epoch_ms=span / E, alpha=0.3, decode_slowdown=0.05)
