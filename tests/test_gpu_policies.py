"""GPU parity of the baseline routing policies (paper Section 4) through gorgo_eval_policy against
oracle/gorgo_policies.py: routes, prefix hits and cache digests bit-exact, p95 within 1e-9."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import gorgo_policies as OP
from paper_2602_11688_b200 import workloads as W
from tests.util import small_trace

POLICIES = ["least-load", "least-request", "prefix-cache", "session-affinity", "random"]


def _gpu_policy(sim, policy, scale, draws):
    import torch
    from paper_2602_11688_b200 import binding as gb
    sim.ensure_workspace(1)
    dev = sim.device
    pt = torch.zeros(1, dtype=torch.float64, device=dev)
    pe = torch.zeros(1, dtype=torch.float64, device=dev)
    route = torch.full((sim.N,), 255, dtype=torch.uint8, device=dev)
    hit = torch.zeros(sim.N, dtype=torch.uint16, device=dev)
    dg = torch.zeros((sim.R, 2), dtype=torch.uint64, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    rc = gb.gorgo_eval_policy(sim.h, policy, draws if policy == "random" else None, scale,
                              sim.workspace, sim.stream, pt, pe, route, hit, dg, st)
    torch.cuda.synchronize()
    assert rc == gb.GORGO_OK, rc
    assert int(st.item()) == 0
    return dict(p95_ttft=float(pt.item()), p95_e2e=float(pe.item()), route=route.cpu().numpy(),
                hit=hit.cpu().numpy(), digest=dg.cpu().numpy())


def _check(w, scale, seed):
    from paper_2602_11688_b200 import binding as gb
    rng = np.random.default_rng(seed)
    draws = rng.integers(0, 2 ** 32, size=w.n_requests, dtype=np.uint64).astype(np.uint32)
    sim = gb.GorgoSim(w)
    try:
        got = {p: _gpu_policy(sim, p, scale, draws) for p in POLICIES}
        # a cost-model evaluation afterwards is not affected by the policy runs
        plain = sim.eval_population(w.params[:1], scale, want_route=True)
        import torch
        torch.cuda.synchronize()
        plain_route = plain["route"].cpu().numpy()[0]
    finally:
        sim.close()
    for p in POLICIES:
        res, p_ttft, p_e2e, dg, _ = OP.replay_policy(w, p, scale, draws=draws)
        g = got[p]
        bad = np.nonzero(g["route"] != res.route)[0]
        assert bad.size == 0, (p, "route", bad[:5])
        bad = np.nonzero(g["hit"] != res.hit)[0]
        assert bad.size == 0, (p, "hit", bad[:5])
        assert g["digest"].tolist() == dg.tolist(), (p, "digest")
        assert abs(g["p95_ttft"] - p_ttft) <= 1e-9 * abs(p_ttft), p
        assert abs(g["p95_e2e"] - p_e2e) <= 1e-9 * abs(p_e2e), p
    from oracle import gorgo_oracle as O
    assert plain_route.tolist() == O.replay(w, w.params[0], scale)[0].route.tolist()
    # the policies really differ on this input
    assert len({tuple(got[p]["route"].tolist()) for p in POLICIES}) >= 4


@pytest.mark.parametrize("R,structured", [(3, True), (5, False), (17, True), (64, True)])
def test_policies_on_small_traces(R, structured):
    rng = np.random.default_rng(R)
    reqs = small_trace(R + 100, n_req=400, structured=structured, rate_ms=15.0)
    K = 3 + R if R == 64 else 3
    params = np.concatenate([rng.normal(1.0, 0.3, size=(1, 3)),
                             rng.lognormal(0, 0.3, size=(1, K - 3))], axis=1)
    w = W.handmade(rng.uniform(5, 60, size=R), reqs, slots=2, cache_blocks=9, params=params)
    _check(w, 0.8, seed=R)


def test_policies_on_the_tiny_workload_and_regions():
    _check(W.make_workload("tiny", n_requests=1500, population=1), 1.0, seed=1)
    _check(W.make_workload("regions", n_requests=3000, population=1, cache_blocks=1500), 1.0, seed=2)


def test_policy_arguments():
    import torch
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload("tiny", n_requests=200, population=1)
    sim = gb.GorgoSim(w)
    try:
        sim.ensure_workspace(1)
        pt = torch.zeros(1, dtype=torch.float64, device=sim.device)
        pe = torch.zeros(1, dtype=torch.float64, device=sim.device)
        assert gb.gorgo_eval_policy(sim.h, 5, None, 1.0, sim.workspace, sim.stream, pt, pe) == gb.GORGO_ERR_INVALID_ARG
        assert gb.gorgo_eval_policy(sim.h, "random", None, 1.0, sim.workspace, sim.stream, pt, pe) == gb.GORGO_ERR_INVALID_ARG
        small = sim.workspace[:256]
        assert gb.gorgo_eval_policy(sim.h, "least-load", None, 1.0, small, sim.stream, pt, pe) == gb.GORGO_ERR_WORKSPACE_TOO_SMALL
        assert gb.gorgo_eval_policy(sim.h, "least-load", None, 1.0, sim.workspace, sim.stream, pt, pe) == gb.GORGO_OK
    finally:
        sim.close()


def test_policies_under_eviction_pressure_at_a_larger_size():
    # long prompts, full caches, scout rings in use: the policy build of the replay kernel at a
    # size that spans many rounds of eviction (60,000 requests, 12,000 blocks per replica)
    _check(W.make_workload("longctx", n_requests=60000, population=1, cache_blocks=12000), 0.5,
           seed=3)
