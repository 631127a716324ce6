"""GPU parity of per-replica service speeds (gorgo_sim_set_replica_speeds) against the oracle:
population evaluation, a baseline policy, batched routing, and switching the speeds off again."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import gorgo_oracle as O
from oracle import gorgo_policies as OP
from paper_2602_11688_b200 import workloads as W
from tests.util import small_trace


def _case(R, seed, n_req=400):
    rng = np.random.default_rng(seed)
    reqs = small_trace(seed, n_req=n_req, rate_ms=15.0)
    K = 3 + R if R > 32 else 3
    params = np.concatenate([rng.normal(1.0, 0.3, size=(4, 3)),
                             rng.lognormal(0, 0.3, size=(4, K - 3))], axis=1)
    w = W.handmade(rng.uniform(5, 60, size=R), reqs, slots=2, cache_blocks=9, params=params)
    pre = rng.uniform(0.01, 0.12, size=R)
    tpot = rng.uniform(4.0, 40.0, size=R)
    return w, pre, tpot


@pytest.mark.parametrize("R", [3, 16, 64])
def test_population_with_replica_speeds(R):
    import torch
    from paper_2602_11688_b200 import binding as gb
    w, pre, tpot = _case(R, seed=40 + R)
    sim = gb.GorgoSim(w)
    try:
        assert gb.gorgo_sim_set_replica_speeds(sim.h, pre, tpot) == gb.GORGO_OK
        het = sim.eval_population(w.params, 0.8, want_route=True, want_hit=True, want_digest=True)
        assert gb.gorgo_sim_set_replica_speeds(sim.h, None, tpot) == gb.GORGO_OK
        half = sim.eval_population(w.params, 0.8, want_route=True)
        assert gb.gorgo_sim_set_replica_speeds(sim.h, None, None) == gb.GORGO_OK
        uni = sim.eval_population(w.params, 0.8, want_route=True)
        torch.cuda.synchronize()
        het = {k: (None if v is None else v.cpu().numpy()) for k, v in het.items()}
        half = {k: (None if v is None else v.cpu().numpy()) for k, v in half.items()}
        uni = {k: (None if v is None else v.cpu().numpy()) for k, v in uni.items()}
        bad = gb.GORGO_ERR_INVALID_ARG
        assert gb.gorgo_sim_set_replica_speeds(sim.h, np.full(R, -1.0), None) == bad
        assert gb.gorgo_sim_set_replica_speeds(sim.h, None, np.full(R, np.inf)) == bad
    finally:
        sim.close()
    for p in range(w.params.shape[0]):
        res, pt, pe, dg, _ = O.replay(w, w.params[p], 0.8, rep_prefill_ms=pre, rep_tpot_ms=tpot)
        assert het["route"][p].tolist() == res.route.tolist() and het["hit"][p].tolist() == res.hit.tolist()
        assert het["digest"][p].tolist() == dg.tolist()
        assert abs(het["p95_ttft"][p] - pt) <= 1e-9 * abs(pt) and abs(het["p95_e2e"][p] - pe) <= 1e-9 * abs(pe)
        res2, pt2, pe2, _, _ = O.replay(w, w.params[p], 0.8, rep_tpot_ms=tpot)
        assert half["route"][p].tolist() == res2.route.tolist()
        assert abs(half["p95_ttft"][p] - pt2) <= 1e-9 * abs(pt2) and abs(half["p95_e2e"][p] - pe2) <= 1e-9 * abs(pe2)
        res3, pt3, pe3, _, _ = O.replay(w, w.params[p], 0.8)
        assert uni["route"][p].tolist() == res3.route.tolist()
        assert abs(uni["p95_ttft"][p] - pt3) <= 1e-9 * abs(pt3)
    assert not np.array_equal(het["p95_e2e"], uni["p95_e2e"])


def test_policy_and_batched_routing_with_replica_speeds():
    import torch
    from paper_2602_11688_b200 import binding as gb
    w, pre, tpot = _case(5, seed=77, n_req=300)
    N = w.n_requests
    sim = gb.GorgoSim(w)
    try:
        assert gb.gorgo_sim_set_replica_speeds(sim.h, pre, tpot) == gb.GORGO_OK
        sim.ensure_workspace(1)
        dev = sim.device
        pt = torch.zeros(1, dtype=torch.float64, device=dev)
        pe = torch.zeros(1, dtype=torch.float64, device=dev)
        route = torch.zeros(N, dtype=torch.uint8, device=dev)
        assert gb.gorgo_eval_policy(sim.h, "least-request", None, 1.0, sim.workspace, sim.stream, pt, pe,
                                    route) == gb.GORGO_OK
        torch.cuda.synchronize()
        pol = (route.cpu().numpy().copy(), float(pt.item()), float(pe.item()))
        # the same trace in three batches on a persistent state
        rc, sbytes = gb.gorgo_state_bytes(sim.h)
        state = torch.empty(sbytes, dtype=torch.uint8, device=dev)
        assert gb.gorgo_sim_reset(sim.h, state, sim.stream) == gb.GORGO_OK
        r_all = torch.zeros(N, dtype=torch.uint8, device=dev)
        t_all = torch.zeros(N, dtype=torch.float64, device=dev)
        e_all = torch.zeros(N, dtype=torch.float64, device=dev)
        for first, count in ((0, 100), (100, 7), (107, N - 107)):
            assert gb.gorgo_route_batch(sim.h, w.params[0], 1.0, first, count, state, sim.stream,
                                        r_all[first:first + count], None, t_all[first:first + count],
                                        e_all[first:first + count]) == gb.GORGO_OK
        torch.cuda.synchronize()
        batched = (r_all.cpu().numpy(), t_all.cpu().numpy(), e_all.cpu().numpy())
    finally:
        sim.close()
    o = O.Oracle.from_workload(w)
    o.set_policy(queue_in_requests=True)
    o.set_replica_speeds(pre, tpot)
    wts = np.zeros(w.n_params); wts[2] = 1.0
    res = o.run(wts, 1.0)
    o.close()
    assert pol[0].tolist() == res.route.tolist()
    assert abs(pol[1] - O.p95(res.ttft)) <= 1e-9 * O.p95(res.ttft)
    assert abs(pol[2] - O.p95(res.e2e)) <= 1e-9 * O.p95(res.e2e)
    ref = O.replay(w, w.params[0], 1.0, rep_prefill_ms=pre, rep_tpot_ms=tpot)[0]
    assert batched[0].tolist() == ref.route.tolist()
    assert batched[1].tolist() == ref.ttft.tolist() and batched[2].tolist() == ref.e2e.tolist()
