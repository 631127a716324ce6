"""GPU parity on the paths of the replay kernel that ordinary traces rarely or never take:
prompts longer than a shared-memory stage, replays without the helper warps (the probe warps
that stage prefix hits ahead, the scout warps that pre-validate eviction victims), a wait that
runs out, and the hand-worked timing cases.  Everything goes through the C ABI; results are
compared bit for bit with the CPU oracle."""
import numpy as np
import pytest

from oracle import gorgo_oracle as O
from paper_2602_11688_b200 import workloads as W
from tests.util import check_population, gpu_eval, oracle_eval, small_trace

pytestmark = pytest.mark.gpu


def long_prompt_trace(seed, n_req, max_blocks, n_sessions=9, B=512):
    """Sessions whose prompts grow to `max_blocks` blocks (several stages' worth), with restarts,
    plus unrelated short requests in between."""
    rng = np.random.default_rng(seed)
    reqs, t, nxt, conv = [], 0.0, 10_000, {}
    for _ in range(n_req):
        t += float(rng.exponential(30.0))
        s = int(rng.integers(n_sessions))
        ids = conv.get(s)
        if ids is None or len(ids) >= max_blocks or rng.random() < 0.15:
            k = min(max_blocks, int(rng.choice([1, 40, 70, 130, max_blocks - 1, max_blocks])))
            ids = list(range(nxt, nxt + k)); nxt += k
        else:
            k = int(rng.integers(1, 90))
            ids = (ids + list(range(nxt, nxt + k)))[:max_blocks]; nxt += k
        conv[s] = ids
        n = len(ids)
        reqs.append((t, (n - 1) * B + int(rng.integers(1, B + 1)), int(rng.integers(0, 40)), ids))
    return reqs


@pytest.mark.parametrize("R,max_blocks,C", [(3, 257, 700), (17, 300, 650), (64, 600, 600),
                                            (8, 65, 200), (33, 129, 400)])
def test_prompts_longer_than_a_stage(R, max_blocks, C):
    rng = np.random.default_rng(R)
    reqs = long_prompt_trace(R, 260, max_blocks)
    assert max(len(q[3]) for q in reqs) == max_blocks
    params = rng.normal(1.0, 0.3, size=(5, 3))
    params[0] = (0.0, 1.0, 0.0)                       # follow the cache: long prefix hits
    params[1] = (0.0, 0.0, 1.0)                       # spread out: many evictions everywhere
    w = W.handmade(rng.uniform(5, 80, size=R), reqs, slots=3, cache_blocks=C, params=params)
    gpu, refs = check_population(w, scale=1.0)
    assert sum(int(r[4][3]) for r in refs) > 0        # evictions happened
    assert max(int(r[0].hit.max()) for r in refs) > min(128, max_blocks // 2)   # long prefix hits


def _switches(gb, probe_off, scout_off, ring_polls):
    d = {gb.GORGO_DEBUG_PROBE_OFF: int(probe_off), gb.GORGO_DEBUG_SCOUT_OFF: int(scout_off)}
    if ring_polls is not None:
        d[gb.GORGO_DEBUG_RING_POLLS] = ring_polls
    return d


@pytest.mark.parametrize("probe_off,scout_off,ring_polls", [(1, 0, None), (0, 1, 0), (1, 1, 0),
                                                            (0, 0, 0)])
@pytest.mark.parametrize("R,structured", [(3, True), (9, False), (17, True), (33, False), (64, True)])
def test_small_traces_without_the_helper_warps(R, structured, probe_off, scout_off, ring_polls):
    """The probe and scout warps only prepare work ahead of time: without them (every request
    probed by the gate warp, every victim found by the commit warps themselves) the bits are the
    same."""
    from paper_2602_11688_b200 import binding as gb
    rng = np.random.default_rng(R)
    reqs = small_trace(R + 3, n_req=400, structured=structured)
    params = rng.normal(1.0, 0.3, size=(4, 3))
    w = W.handmade(rng.uniform(5, 60, size=R), reqs, slots=2, cache_blocks=9, params=params)
    check_population(w, scale=1.0, debug=_switches(gb, probe_off, scout_off, ring_polls))


@pytest.mark.parametrize("probe_off,scout_off,ring_polls", [(1, 0, None), (0, 1, 0), (1, 1, 0)])
def test_longctx_reduced_without_the_helper_warps(probe_off, scout_off, ring_polls):
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload("longctx", n_requests=12_000, cache_blocks=3_000, population=6)
    gpu, refs = check_population(w, debug=_switches(gb, probe_off, scout_off, ring_polls))
    assert sum(int(r[4][3]) for r in refs) > 0


def test_a_wait_that_runs_out_is_reported_and_nothing_hangs():
    """With the bound of the warps' waits for one another set to zero, the first wait that is
    not satisfied at once gives up: the candidate's status says so, the host-output entry point
    returns GORGO_ERR_DEVICE_LIMIT, and the next evaluation with the normal bound is exact."""
    import torch
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload("tiny", n_requests=400, cache_blocks=150, population=5)
    sim = gb.GorgoSim(w)
    assert gb.gorgo_debug_set(sim.h, gb.GORGO_DEBUG_POLL_LIMIT, 0) == gb.GORGO_OK
    out = sim.eval_population(w.params, 1.0)
    torch.cuda.synchronize()
    assert (out["status"].cpu().numpy() == gb.GORGO_ERR_DEVICE_LIMIT).all()
    P = w.params.shape[0]
    h_t, h_e = np.zeros(P), np.zeros(P)
    rc = gb.gorgo_eval_population_host(sim.h, P, np.ascontiguousarray(w.params), 1.0, sim.workspace,
                                       sim.stream, h_t, h_e)
    assert rc == gb.GORGO_ERR_DEVICE_LIMIT
    assert gb.gorgo_debug_set(sim.h, gb.GORGO_DEBUG_POLL_LIMIT, 1 << 24) == gb.GORGO_OK
    assert gb.gorgo_debug_set(sim.h, 99, 1) == gb.GORGO_ERR_INVALID_ARG
    res = gpu_eval(w, scale=1.0, sim=sim)
    refs = oracle_eval(w, w.params, 1.0)
    for p, ref in enumerate(refs):
        assert (res["route"][p] == ref[0].route).all() and (res["hit"][p] == ref[0].hit).all()
    sim.close()


def test_w3_two_slots_third_request_takes_the_earlier_finish_on_gpu():
    reqs = [(0.0, 1000, 11, [1, 2]), (10.0, 1000, 3, [3, 4]), (20.0, 1000, 1, [5, 6])]
    w = W.handmade([5.0], reqs, slots=2, cache_blocks=100, prefill_ms_per_token=0.01,
                   tpot_ms=10.0, params=[(1.0, 1.0, 1.0)])
    from paper_2602_11688_b200 import binding as gb
    import torch
    sim = gb.GorgoSim(w)
    st = _route_all(gb, sim, w)
    np.testing.assert_allclose(st["ttft"], [15.0, 15.0, 35.0], rtol=1e-14)
    np.testing.assert_allclose(st["e2e"], [115.0, 35.0, 35.0], rtol=1e-14)
    ref = O.Oracle.from_workload(w).run(w.params[0])
    assert st["ttft"].tolist() == ref.ttft.tolist() and st["e2e"].tolist() == ref.e2e.tolist()
    sim.close()


def _route_all(gb, sim, w, scale=1.0):
    """All requests through gorgo_route_batch on a fresh persistent state (per-request times)."""
    import torch
    rc, nbytes = gb.gorgo_state_bytes(sim.h)
    assert rc == gb.GORGO_OK
    state = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    assert gb.gorgo_sim_reset(sim.h, state, sim.stream) == gb.GORGO_OK
    N = w.n_requests
    route = torch.empty(N, dtype=torch.uint8, device="cuda")
    hit = torch.empty(N, dtype=torch.uint16, device="cuda")
    ttft = torch.empty(N, dtype=torch.float64, device="cuda")
    e2e = torch.empty(N, dtype=torch.float64, device="cuda")
    rc = gb.gorgo_route_batch(sim.h, w.params[0], scale, 0, N, state, sim.stream, route, hit, ttft, e2e)
    assert rc == gb.GORGO_OK
    rc, seen = gb.gorgo_state_status(sim.h, state, sim.stream)
    assert rc == gb.GORGO_OK and seen == N
    return {"route": route.cpu().numpy(), "hit": hit.cpu().numpy(), "ttft": ttft.cpu().numpy(),
            "e2e": e2e.cpu().numpy()}


@pytest.mark.parametrize("t1,routes", [(42.0, [0, 0]), (41.5, [0, 1])])
def test_w4_completion_exactly_at_arrival_is_not_in_flight_on_gpu(t1, routes):
    # pure queue-load routing; prefill 0.0625 ms/token * 512 = 32 ms exactly -> finish = 42.0:
    # a request arriving at exactly 42.0 no longer sees it in flight, one at 41.5 does
    from paper_2602_11688_b200 import binding as gb
    reqs = [(0.0, 512, 1, [1]), (t1, 512, 1, [2])]
    w = W.handmade([10.0, 10.0], reqs, slots=1, cache_blocks=8,
                   prefill_ms_per_token=0.0625, params=[(0.0, 0.0, 1.0)])
    sim = gb.GorgoSim(w)
    st = _route_all(gb, sim, w)
    assert st["route"].tolist() == routes
    assert st["e2e"][0] == 42.0
    ref, *_ = O.replay(w, w.params[0])
    assert st["route"].tolist() == ref.route.tolist() and st["e2e"].tolist() == ref.e2e.tolist()
    sim.close()
    res = gpu_eval(w, scale=1.0)
    assert res["route"][0].tolist() == routes


def test_w5_queue_normalisers_multiply_the_load_on_gpu():
    # two replicas at equal distance, nothing cached: replica 0 holds 1000 tokens in flight, its
    # normaliser 0.25 makes them count as 250 against replica 1's 600 * 1.0
    reqs = [(0.0, 1000, 50, [1, 2]), (1.0, 600, 50, [3, 4]), (2.0, 512, 1, [5])]
    for norm, third in (((1.0, 1.0), 1), ((0.25, 1.0), 0)):
        w = W.handmade([10.0, 10.0], reqs, slots=4, cache_blocks=64,
                       params=[(0.0, 0.0, 1.0) + norm])
        ref, *_ = O.replay(w, w.params[0])
        assert ref.route.tolist() == [0, 1, third]
        res = gpu_eval(w, scale=1.0)
        assert res["route"][0].tolist() == [0, 1, third]
