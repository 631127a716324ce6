"""GPU parity of the growing trace (gorgo_trace_begin / gorgo_trace_append): routing appended
requests batch by batch on a persistent state gives bit for bit what the oracle gives for the
whole trace, and what the library gives when the whole trace is uploaded at once."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import gorgo_oracle as O
from paper_2602_11688_b200 import workloads as W
from tests.util import small_trace


def _create(w):
    from paper_2602_11688_b200 import binding as gb
    rc, h = gb.gorgo_sim_create(rtt_ms=w.rtt_ms, device=0, **w.config_dict())
    assert rc == gb.GORGO_OK
    return h


def _append(h, w, a, b, stream=0):
    from paper_2602_11688_b200 import binding as gb
    off = w.hash_off[a:b + 1].astype(np.uint64)
    ids = w.hash_ids[int(off[0]):int(off[-1])]
    org = None if w.origin is None else w.origin[a:b]
    return gb.gorgo_trace_append(h, w.ts_ms[a:b], w.input_tokens[a:b], w.output_tokens[a:b], org,
                                 off - off[0], ids, stream)


def _route_all(h, w, p, scale, plan, known=0):
    """plan: list of (append up to, route up to) steps; returns route, hit, ttft, e2e, digest."""
    import torch
    from paper_2602_11688_b200 import binding as gb
    N, R = w.n_requests, w.spec.n_replicas
    route = torch.empty(N, dtype=torch.uint8, device="cuda")
    hit = torch.empty(N, dtype=torch.uint16, device="cuda")
    ttft = torch.empty(N, dtype=torch.float64, device="cuda")
    e2e = torch.empty(N, dtype=torch.float64, device="cuda")
    state = None
    done = 0
    for upto, route_to in plan:
        if upto > known:
            assert _append(h, w, known, upto) == gb.GORGO_OK
            known = upto
        if state is None:
            rc, nbytes = gb.gorgo_state_bytes(h)
            assert rc == gb.GORGO_OK
            state = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
            assert gb.gorgo_sim_reset(h, state, 0) == gb.GORGO_OK
        if route_to > done:
            rc = gb.gorgo_route_batch(h, w.params[p], scale, done, route_to - done, state, 0,
                                      route[done:], hit[done:], ttft[done:], e2e[done:])
            assert rc == gb.GORGO_OK
            done = route_to
    assert done == N
    rc, seen = gb.gorgo_state_status(h, state, 0)
    assert rc == gb.GORGO_OK and seen == N
    digest = torch.empty((R, 2), dtype=torch.uint64, device="cuda")
    assert gb.gorgo_state_digest(h, state, 0, digest) == gb.GORGO_OK
    torch.cuda.synchronize()
    return [x.cpu().numpy() for x in (route, hit, ttft, e2e, digest)]


def _plans(N, rng):
    one_by_one = [(k + 1, k + 1) for k in range(N)]            # every request routed before the next is known
    cuts = sorted(set(rng.integers(1, N, size=9).tolist())) + [N]
    chunks = [(c, c) for c in cuts]
    lag, known = [], 0                                          # routing lags the appends
    for c in cuts:
        lag.append((c, max(known - 5, 0)))
        known = c
    lag.append((N, N))
    return {"one by one": one_by_one, "chunks": chunks, "lagging": lag}


@pytest.mark.parametrize("R,structured", [(3, True), (17, False), (64, True)])
def test_appended_batches_equal_the_whole_trace(R, structured):
    import torch
    from paper_2602_11688_b200 import binding as gb
    rng = np.random.default_rng(R)
    reqs = small_trace(R + 5, n_req=260, structured=structured, rate_ms=12.0)
    K = 3 + R if R > 32 else 3
    params = np.concatenate([rng.normal(1.0, 0.3, size=(2, 3)), rng.lognormal(0, 0.3, size=(2, K - 3))], axis=1)
    w = W.handmade(rng.uniform(5, 60, size=R), reqs, slots=2, cache_blocks=9, params=params)
    N, T = w.n_requests, int(w.hash_off[-1])
    want = {}
    for p in range(2):
        res, _, _, dg, _ = O.replay(w, w.params[p], 0.8)
        want[p] = (res.route, res.hit, res.ttft, res.e2e, dg)
    rc, nbytes = gb.gorgo_trace_bytes(N + 10, T + 100)
    for name, plan in _plans(N, rng).items():
        for p in range(2):
            h = _create(w)
            buf = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
            assert gb.gorgo_trace_append(h, w.ts_ms[:1], w.input_tokens[:1], w.output_tokens[:1], None,
                                         w.hash_off[:2], w.hash_ids, 0) == gb.GORGO_ERR_NO_TRACE
            assert gb.gorgo_trace_begin(h, N + 10, T + 100, buf) == gb.GORGO_OK
            got = _route_all(h, w, p, 0.8, plan)
            torch.cuda.synchronize()
            gb.gorgo_sim_destroy(h)
            r, hb, tt, ee, dg = want[p]
            assert got[0].tolist() == r.tolist(), (name, p)
            assert got[1].tolist() == hb.tolist(), (name, p)
            assert np.array_equal(got[2], tt) and np.array_equal(got[3], ee), (name, p)
            assert got[4].tolist() == dg.tolist(), (name, p)


def test_population_on_a_grown_trace_equals_the_uploaded_one():
    import torch
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload("regions", n_requests=3000, cache_blocks=700, population=6)
    N, T = w.n_requests, int(w.hash_off[-1])
    sim = gb.GorgoSim(w)
    ref = sim.eval_population(w.params, 1.0, want_route=True, want_hit=True, want_digest=True)
    torch.cuda.synchronize()
    ref = {k: (None if v is None else v.cpu().numpy()) for k, v in ref.items()}
    # the same handle, now with a growing trace of a larger capacity, filled in uneven batches
    rc, nbytes = gb.gorgo_trace_bytes(2 * N, 2 * T)
    buf = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    assert gb.gorgo_trace_begin(sim.h, 2 * N, 2 * T, buf) == gb.GORGO_OK
    cuts = [0, 1, 2, 700, 701, 1999, N]
    for a, b in zip(cuts[:-1], cuts[1:]):
        assert _append(sim.h, w, a, b, sim.stream) == gb.GORGO_OK
    assert gb.gorgo_trace_info(sim.h)[1:3] == (N, T)
    got = sim.eval_population(w.params, 1.0, want_route=True, want_hit=True, want_digest=True)
    torch.cuda.synchronize()
    got = {k: (None if v is None else v.cpu().numpy()) for k, v in got.items()}
    sim.close()
    assert int(np.abs(got["status"]).sum()) == 0
    for k in ("route", "hit", "digest", "p95_ttft", "p95_e2e"):
        assert np.array_equal(got[k], ref[k]), k


def test_refused_batches_leave_the_trace_as_it_was():
    import torch
    from paper_2602_11688_b200 import binding as gb
    reqs = small_trace(3, n_req=60)
    w = W.handmade([10.0, 20.0, 30.0], reqs, slots=2, cache_blocks=9, params=[(1.0, 1.0, 1.0)])
    N, T = w.n_requests, int(w.hash_off[-1])
    res, _, _, dg, _ = O.replay(w, w.params[0], 1.0)
    h = _create(w)
    rc, nbytes = gb.gorgo_trace_bytes(N, T)
    buf = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    assert gb.gorgo_trace_begin(h, N, T, buf) == gb.GORGO_OK
    assert _append(h, w, 0, 30) == gb.GORGO_OK
    t = float(w.ts_ms[29])
    B = w.spec.block_tokens
    one = np.array([0, 2], dtype=np.uint64)
    bad = gb.GORGO_ERR_BAD_TRACE
    # a block twice in one request (one of them known already), time running backwards, wrong block
    # count, more than the capacity: all refused
    assert gb.gorgo_trace_append(h, [t], [2 * B], [5], None, one, np.array([w.hash_ids[0], w.hash_ids[0]], dtype=np.uint64)) == bad
    assert gb.gorgo_trace_append(h, [t], [2 * B], [5], None, one, np.array([777777, 777777], dtype=np.uint64)) == bad
    assert gb.gorgo_trace_append(h, [t - 1.0], [2 * B], [5], None, one, np.array([5, 6], dtype=np.uint64)) == bad
    assert gb.gorgo_trace_append(h, [t], [3 * B], [5], None, one, np.array([5, 6], dtype=np.uint64)) == bad
    m = N - 30 + 1
    assert gb.gorgo_trace_append(h, np.full(m, t), np.full(m, B), np.full(m, 1), None,
                                 np.arange(m + 1, dtype=np.uint64),
                                 np.arange(10 ** 6, 10 ** 6 + m, dtype=np.uint64)) == gb.GORGO_ERR_WORKSPACE_TOO_SMALL
    assert gb.gorgo_trace_info(h)[1:3] == (30, int(w.hash_off[30]))
    got = _route_all(h, w, 0, 1.0, [(30, 30), (N, N)], known=30)
    gb.gorgo_sim_destroy(h)
    assert got[0].tolist() == res.route.tolist() and got[1].tolist() == res.hit.tolist()
    assert np.array_equal(got[2], res.ttft) and got[4].tolist() == dg.tolist()
