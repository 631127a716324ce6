"""Pins of the CPU oracle against things other than itself (no GPU needed).

Hand-worked traces, brute force, an independently formulated recency-list cache, textbook
queueing recursions, closed forms, invariants and special cases of the score of Eq. 3.
"""
import json
import os

import numpy as np
import pytest

from oracle import gorgo_oracle as O
from paper_2602_11688_b200 import workloads as W
from tests.util import small_trace

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def recency_list_replay(requests, routes, R, C):
    """Independent cache model: one plain recency list per replica (front = next victim).
    A routed request pulls its own blocks out of the list, trims the front until the request
    fits, then appends its blocks deepest first (so the shallowest block is the most recent).
    Returns per-request (prefix hit on every replica before the commit, number of the
    request's blocks resident on the chosen replica, evictions) and the final lists."""
    lists = [[] for _ in range(R)]
    out = []
    for (t, in_tok, o, ids), i in zip(requests, routes):
        hits = []
        for lst in lists:
            h = 0
            while h < len(ids) and ids[h] in lst:
                h += 1
            hits.append(h)
        lst = lists[i]
        resident = sum(1 for b in ids if b in lst)
        lst[:] = [b for b in lst if b not in ids]
        ev = 0
        while len(lst) + len(ids) > C:
            lst.pop(0); ev += 1
        lst.extend(reversed(ids))
        out.append((hits, resident, ev))
    return out, lists


# ----------------------------------------------------------------------------- hand cases
def test_w1_handworked_trace():
    g = json.load(open(os.path.join(GOLDEN, "w1_handworked.json")))
    names = {}
    reqs = []
    for q in g["requests"]:
        ids = [names.setdefault(b, 100 + len(names)) for b in q["blocks"]]
        reqs.append((q["t_ms"], q["input_tokens"], q["output_tokens"], ids))
    c = g["config"]
    w = W.handmade(c["rtt_ms"], reqs, slots=c["slots"], cache_blocks=c["cache_blocks"],
                   block_tokens=c["block_tokens"], prefill_ms_per_token=c["prefill_ms_per_token"],
                   tpot_ms=c["tpot_ms"], params=[c["params"]])
    o = O.Oracle.from_workload(w)
    res = o.run(w.params[0], c["time_scale"], detail=True)
    e = g["expected"]
    assert res.route.tolist() == e["route"]
    assert res.hit.tolist() == e["hit_blocks"]
    assert res.load_all.tolist() == e["load_tokens"]
    assert res.evicted.tolist() == e["evicted"]
    np.testing.assert_allclose(res.cost_all, e["cost"], rtol=1e-12)
    np.testing.assert_allclose(res.ttft, e["ttft_ms"], rtol=1e-12)
    np.testing.assert_allclose(res.e2e, e["e2e_ms"], rtol=1e-12)
    assert O.p95(res.ttft) == pytest.approx(e["p95_ttft_ms"], rel=1e-12)
    assert O.p95(res.e2e) == pytest.approx(e["p95_e2e_ms"], rel=1e-12)
    inv = {v: k for k, v in names.items()}
    for i, want in enumerate(e["final_cache"]):
        ids, seq, pos = o.dump(i)
        assert sorted(inv[int(b)] for b in ids) == want
    # replica 0 in eviction order: F (request 3, pos 2) goes first, then C, B, A of request 4
    ids, seq, pos = o.dump(0)
    assert [inv[int(b)] for b in ids] == ["F", "C", "B", "A"]
    assert seq.tolist() == [3, 4, 4, 4] and pos.tolist() == [2, 2, 1, 0]
    # the four counters the byte model of the benchmark is built from, counted by hand
    assert o.stats().tolist() == e["counters"]


def test_w2_equal_costs_go_to_lowest_index():
    reqs = small_trace(1, n_req=50)
    w = W.handmade([30.0, 20.0, 10.0], reqs, slots=2, cache_blocks=16, params=[(0.0, 0.0, 0.0)])
    res, *_ = O.replay(w, w.params[0])
    assert (res.route == 0).all()
    # -0.0 and +0.0 compare equal: still the lowest index
    w2 = W.handmade([30.0, 20.0, 10.0], reqs, slots=2, cache_blocks=16, params=[(-0.0, 0.0, 0.0)])
    res2, *_ = O.replay(w2, w2.params[0])
    assert (res2.route == 0).all()


def test_w3_two_slots_third_request_takes_the_earlier_finish():
    reqs = [(0.0, 1000, 11, [1, 2]), (10.0, 1000, 3, [3, 4]), (20.0, 1000, 1, [5, 6])]
    w = W.handmade([5.0], reqs, slots=2, cache_blocks=100, prefill_ms_per_token=0.01,
                   tpot_ms=10.0, params=[(1.0, 1.0, 1.0)])
    o = O.Oracle.from_workload(w)
    res = o.run(w.params[0])
    # r0: arrive 5, first 15, finish 115 (slot 0).  r1: arrive 15, slot 1, first 25, finish 45.
    # r2: arrive 25, both busy (115, 45) -> waits for 45, first 55 = finish.
    np.testing.assert_allclose(res.ttft, [15.0, 15.0, 35.0], rtol=1e-14)
    np.testing.assert_allclose(res.e2e, [115.0, 35.0, 35.0], rtol=1e-14)
    _, _, free_at = o.queues()
    assert free_at.tolist() == [[115.0, 55.0]]


def test_w4_completion_exactly_at_arrival_is_not_in_flight():
    # pure queue-load routing; prefill 0.0625 ms/token * 512 = 32 ms exactly -> finish = 42.0
    def run(t1):
        reqs = [(0.0, 512, 1, [1]), (t1, 512, 1, [2])]
        w = W.handmade([10.0, 10.0], reqs, slots=1, cache_blocks=8,
                       prefill_ms_per_token=0.0625, params=[(0.0, 0.0, 1.0)])
        res, *_ = O.replay(w, w.params[0], detail=True)
        return res
    res = run(42.0)
    assert res.e2e[0] == 42.0
    assert res.load_all[1].tolist() == [0, 0] and res.route.tolist() == [0, 0]
    res = run(41.5)
    assert res.load_all[1].tolist() == [512, 0] and res.route.tolist() == [0, 1]


# ------------------------------------------------------------- brute force / other models
@pytest.mark.parametrize("structured", [True, False])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_prefix_hits_and_lru_against_recency_list_model(seed, structured):
    R, C = 3, 11
    reqs = small_trace(seed, structured=structured)
    rng = np.random.default_rng(100 + seed)
    w = W.handmade(rng.uniform(5, 60, size=R), reqs, slots=2, cache_blocks=C,
                   params=[rng.normal(1.0, 0.3, size=3)])
    o = O.Oracle.from_workload(w)
    res = o.run(w.params[0], detail=True)
    model, lists = recency_list_replay(reqs, res.route.tolist(), R, C)
    for r, (hits, resident, ev) in enumerate(model):
        assert res.hit_all[r].tolist() == hits, r
        assert res.evicted[r] == ev, r
        assert res.hit[r] == hits[res.route[r]]
        if structured:   # ids imply their prefix -> resident blocks of a request are a prefix
            assert resident == hits[res.route[r]]
    for i in range(R):
        ids, seq, pos = o.dump(i)
        assert [int(b) for b in ids] == lists[i]
        assert len(ids) <= C
    assert (res.occ_after <= C).all()


@pytest.mark.parametrize("seed,structured", [(5, True), (6, False), (7, True)])
def test_counters_recomputed_from_per_request_outputs_and_the_recency_list_model(seed, structured):
    """Oracle.stats() = [sum_r sum_i min(h_{r,i}+1, n_r), sum_r h_{r,i*}, sum_r n_r, sum_r E_r].
    Recomputed twice without the oracle's own accumulators: from its per-request outputs, and
    from the independent recency-list cache model driven by the routes alone."""
    reqs = small_trace(seed, n_req=400, n_sessions=10, max_blocks=7, structured=structured)
    R, C = 3, 11
    w = W.handmade(np.array([20.0, 35.0, 50.0]), reqs, slots=2, cache_blocks=C,
                   params=[[1.0, 0.05, 0.001]])
    o = O.Oracle.from_workload(w)
    res = o.run(w.params[0], 1.0, detail=True)
    st = o.stats().tolist()
    n = np.array([len(q[3]) for q in reqs], dtype=np.int64)
    probes = np.minimum(res.hit_all.astype(np.int64) + 1, n[:, None]).sum()
    chosen = res.hit_all[np.arange(len(reqs)), res.route].astype(np.int64)
    assert (chosen == res.hit).all()
    assert st == [int(probes), int(chosen.sum()), int(n.sum()), int(res.evicted.sum())]
    model, _ = recency_list_replay(reqs, res.route.tolist(), R, C)
    m_probes = sum(min(h + 1, len(q[3])) for (hits, _, _), q in zip(model, reqs) for h in hits)
    m_hit = sum(hits[i] for (hits, _, _), i in zip(model, res.route.tolist()))
    m_ev = sum(ev for (_, _, ev) in model)
    assert st == [m_probes, m_hit, int(n.sum()), m_ev]
    assert m_ev > 0 and m_hit > 0
    # a second run continues the sums; a reset clears them
    o.reset()
    assert o.stats().tolist() == [0, 0, 0, 0]
    o.run(w.params[0], 1.0, count=150)
    o.run(w.params[0], 1.0)
    assert o.stats().tolist() == st


def test_prefix_hit_brute_force_without_eviction():
    # capacity above the number of distinct blocks: a replica holds exactly the union of the
    # blocks of the requests routed to it, so every hit follows from the route vector alone
    w = W.make_workload("tiny", n_requests=400, cache_blocks=10**6)
    res, *_ = O.replay(w, w.params[3], detail=True)
    R = w.spec.n_replicas
    seen = [set() for _ in range(R)]
    off = w.hash_off.astype(np.int64)
    for r in range(w.n_requests):
        ids = w.hash_ids[off[r]:off[r + 1]].tolist()
        for i in range(R):
            h = 0
            while h < len(ids) and ids[h] in seen[i]:
                h += 1
            assert res.hit_all[r, i] == h
            assert h <= len(ids)
        seen[res.route[r]].update(ids)
    assert res.evicted.sum() == 0


def test_lru_inclusion_property_single_replica():
    # stack property of LRU (Mattson et al. 1970): with one replica the content under capacity
    # C is a subset of the content under C+1 at every step, so hits never drop as C grows
    reqs = small_trace(5, n_req=250, structured=False)
    prev_hits, prev_sets = None, None
    for C in (7, 8, 9, 12, 20):
        w = W.handmade([10.0], reqs, slots=4, cache_blocks=C, params=[(1.0, 1.0, 1.0)])
        o = O.Oracle.from_workload(w)
        hits, sets = [], []
        for r in range(len(reqs)):
            rr = o.run(w.params[0], count=1)
            hits.append(int(rr.hit[0]))
            sets.append(set(int(b) for b in o.dump(0)[0]))
        if prev_hits is not None:
            assert all(a <= b for a, b in zip(prev_hits, hits))
            assert all(a <= b for a, b in zip(prev_sets, sets))
        prev_hits, prev_sets = hits, sets


# ---------------------------------------------------------------------------- queue model
def test_enough_slots_gives_closed_form_ttft():
    w = W.make_workload("tiny", n_requests=300)
    w.spec.slots = 300                                     # never wait
    res, *_ = O.replay(w, w.params[0], detail=True)
    R = w.spec.n_replicas
    rtt = w.rtt_ms[0][res.route]
    unc = w.input_tokens.astype(np.int64) - np.minimum(
        res.hit.astype(np.int64) * 512, w.input_tokens.astype(np.int64))
    np.testing.assert_allclose(res.ttft, rtt + 0.05 * unc, rtol=1e-9)
    dec = 20.0 * np.maximum(w.output_tokens.astype(np.int64) - 1, 0)
    np.testing.assert_allclose(res.e2e, rtt + 0.05 * unc + dec, rtol=1e-9)


def test_single_server_matches_lindley_recursion():
    # R = 1, S = 1, cache too small to hit across sessions is irrelevant: use measured service
    w = W.make_workload("tiny", n_requests=400, cache_blocks=50)
    w.rtt_ms = w.rtt_ms[:, :1].copy()
    w.spec.n_replicas, w.spec.slots = 1, 1
    scale = 3.0
    res, *_ = O.replay(w, w.params[0], scale, detail=True)
    unc = w.input_tokens.astype(np.int64) - np.minimum(
        res.hit.astype(np.int64) * 512, w.input_tokens.astype(np.int64))
    service = 0.05 * unc + 20.0 * np.maximum(w.output_tokens.astype(np.int64) - 1, 0)
    t = scale * w.ts_ms
    wait = np.zeros(len(t))
    for r in range(len(t) - 1):                            # Lindley (1952)
        wait[r + 1] = max(0.0, wait[r] + service[r] - (t[r + 1] - t[r]))
    np.testing.assert_allclose(res.ttft, w.rtt_ms[0, 0] + wait + 0.05 * unc, rtol=1e-9, atol=1e-6)
    assert wait.max() > 0


def test_load_signal_is_sum_of_in_flight_input_tokens():
    w = W.make_workload("tiny", n_requests=600)
    res, *_ = O.replay(w, w.params[1], detail=True)
    t = w.ts_ms
    fin = t + res.e2e
    R = w.spec.n_replicas
    for r in range(0, w.n_requests, 7):
        for i in range(R):
            live = (res.route[:r] == i) & (fin[:r] > t[r] + 1e-6)
            maybe = (res.route[:r] == i) & (np.abs(fin[:r] - t[r]) <= 1e-6)
            assert not maybe.any()
            assert res.load_all[r, i] == int(w.input_tokens[:r][live].sum())
    # far in the future everything has completed
    o = O.Oracle(rtt_ms=w.rtt_ms, ts_ms=np.append(w.ts_ms, 1e15),
                 input_tokens=np.append(w.input_tokens, 1), output_tokens=np.append(w.output_tokens, 1),
                 origin=np.append(w.origin, 0), hash_off=np.append(w.hash_off, w.hash_off[-1] + 1),
                 hash_ids=np.append(w.hash_ids, 7), **w.config_dict())
    rr = o.run(w.params[1], detail=True)
    assert rr.load_all[-1].tolist() == [0] * R


# ------------------------------------------------------------------- score special cases
def test_only_network_weight_routes_to_min_rtt():
    w = W.make_workload("regions", n_requests=800)
    res, *_ = O.replay(w, np.array([0.7, 0.0, 0.0]))
    want = np.argmin(w.rtt_ms[w.origin], axis=1)           # first minimum = lowest index
    assert (res.route == want).all()


def test_only_prefill_weight_is_the_prefix_cache_policy():
    # Section 4, "prefix-cache": route to the replica with the highest prefix overlap
    w = W.make_workload("regions", n_requests=1500, cache_blocks=3000)
    res, *_ = O.replay(w, np.array([0.0, 1.3, 0.0]), detail=True)
    assert (res.route == np.argmax(res.hit_all, axis=1)).all()
    assert res.hit.sum() > 0


def test_only_queue_weight_is_least_in_flight_tokens():
    w = W.make_workload("tiny", n_requests=800)
    res, *_ = O.replay(w, np.array([0.0, 0.0, 0.4]), detail=True)
    assert (res.route == np.argmin(res.load_all, axis=1)).all()
    assert len(set(res.route.tolist())) == w.spec.n_replicas


def test_only_the_ratio_of_weights_matters_power_of_two_scaling_is_exact():
    # Section 2.3: routing depends on relative replica cost only
    w = W.make_workload("regions", n_requests=2000, cache_blocks=2500)
    base = w.params[5]
    a, pa, pb, da, _ = O.replay(w, base, detail=True)
    for f in (2.0, 0.25, 1024.0):
        b, qa, qb, db, _ = O.replay(w, base * f, detail=True)
        assert (a.route == b.route).all() and (a.hit_all == b.hit_all).all()
        assert (a.ttft == b.ttft).all() and (a.e2e == b.e2e).all()
        assert (da == db).all() and pa == qa and pb == qb
        assert (b.cost_all == a.cost_all * f).all()


def test_per_replica_normalisers_of_one_change_nothing_and_relabelling_permutes_routes():
    w = W.make_workload("tiny", n_requests=700)
    R = w.spec.n_replicas
    a, *_ = O.replay(w, w.params[2])
    cfg = w.config_dict(); cfg["n_params"] = 3 + R
    kw = dict(rtt_ms=w.rtt_ms, ts_ms=w.ts_ms, input_tokens=w.input_tokens,
              output_tokens=w.output_tokens, origin=w.origin, hash_off=w.hash_off,
              hash_ids=w.hash_ids)
    o = O.Oracle(**kw, **cfg)
    b = o.run(np.concatenate([w.params[2], np.ones(R)]))
    assert (a.route == b.route).all() and (a.ttft == b.ttft).all()
    # permute the replicas (RTT columns and normalisers): routes are permuted the same way
    norm = np.array([0.6, 1.7, 1.0, 0.9])
    perm = np.array([2, 0, 3, 1])
    o1 = O.Oracle(**kw, **cfg)
    c = o1.run(np.concatenate([w.params[2], norm]), detail=True)
    kw2 = dict(kw); kw2["rtt_ms"] = w.rtt_ms[:, perm]
    o2 = O.Oracle(**kw2, **cfg)
    d = o2.run(np.concatenate([w.params[2], norm[perm]]), detail=True)
    srt = np.sort(c.cost_all, axis=1)
    assert (srt[:, 0] < srt[:, 1]).all()                   # no ties in this instance
    assert (perm[d.route] == c.route).all()
    assert (c.ttft == d.ttft).all()
    assert (c.route != a.route).any()                      # the normalisers do matter


def test_w5_queue_normalisers_multiply_the_load():
    # K = 3 + R: q_i = load_i * s_i.  Pure queue routing, s = (4, 0.25), by hand:
    # r1 sees loads (1000, 0) -> costs (4000, 0) -> replica 1;
    # r2 sees loads (1000, 3000) -> costs (4000, 750) -> replica 1 (a divide would give 250 vs 12000)
    reqs = [(0.0, 1000, 50, [1, 2]), (1.0, 3000, 50, [3, 4, 5, 6, 7, 8]), (2.0, 10, 50, [9])]
    w = W.handmade([10.0, 10.0], reqs, slots=4, cache_blocks=64,
                   params=[(0.0, 0.0, 1.0, 4.0, 0.25)])
    res, *_ = O.replay(w, w.params[0], detail=True)
    assert res.route.tolist() == [0, 1, 1]
    assert res.cost_all.tolist() == [[0.0, 0.0], [4000.0, 0.0], [4000.0, 750.0]]


def test_time_scale_multiplies_timestamps():
    w = W.make_workload("tiny", n_requests=500)
    a, *_ = O.replay(w, w.params[0], 0.5)
    w2 = W.make_workload("tiny", n_requests=500)
    w2.ts_ms = w2.ts_ms * 0.5
    b, *_ = O.replay(w2, w2.params[0], 1.0)
    assert (a.route == b.route).all() and (a.ttft == b.ttft).all() and (a.e2e == b.e2e).all()
    c, p_fast, *_ = O.replay(w, w.params[0], 0.25)
    d, p_slow, *_ = O.replay(w, w.params[0], 8.0)
    assert p_slow < p_fast                                 # lighter load, lower p95 TTFT


def test_zero_queue_weight_concentrates_on_the_nearest_replica():
    # Section 5 / Appendix D: with w_queue = 0 almost all traffic goes to one replica
    w = W.make_workload("tiny", n_requests=1000)
    w.rtt_ms = np.array([[12.0, 150.0, 220.0, 300.0]])
    res, *_ = O.replay(w, np.array([1.0, 0.001, 0.0]))
    assert np.mean(res.route == 0) > 0.95


# -------------------------------------------------------------------------------- p95
def test_p95_nearest_rank():
    assert O.p95(np.array([3.5])) == 3.5
    v = np.arange(1, 21, dtype=np.float64)[::-1].copy()
    assert O.p95(v) == 19.0
    v = np.arange(1, 101, dtype=np.float64)
    np.random.default_rng(0).shuffle(v)
    assert O.p95(v) == 95.0
    assert O.p95(np.arange(1, 102, dtype=np.float64)) == 96.0   # ceil(95.95) = 96
    assert O.p95(np.full(37, 2.25)) == 2.25
    rng = np.random.default_rng(1)
    for n in (7, 33, 999, 4567):
        v = rng.lognormal(size=n)
        assert O.p95(v) == np.percentile(v, 95, method="inverted_cdf")


# ------------------------------------------------------------------------------ digest
def test_digest_known_answer_and_recomputation():
    # splitmix64's first output for seed 0 is the finaliser applied to the golden-ratio
    # increment: mix64(0x9E3779B97F4A7C15) = 0xE220A8397B1DCDAF; mix64(0) = 0, so one block
    # cached by request 0 at position 0 has exactly that digest sum.
    w = W.handmade([10.0, 20.0], [(0.0, 100, 1, [0x9E3779B97F4A7C15])], cache_blocks=4)
    _, _, _, dg, _ = O.replay(w, w.params[0])
    assert dg.tolist() == [[1, 0xE220A8397B1DCDAF], [0, 0]]

    M = (1 << 64) - 1

    def mix(z):
        z ^= z >> 30; z = (z * 0xbf58476d1ce4e5b9) & M
        z ^= z >> 27; z = (z * 0x94d049bb133111eb) & M
        return z ^ (z >> 31)

    w = W.make_workload("tiny", n_requests=500, cache_blocks=300)
    o = O.Oracle.from_workload(w)
    o.run(w.params[4])
    dg = o.digest()
    for i in range(w.spec.n_replicas):
        ids, seq, pos = o.dump(i)
        s = 0
        for b, q, k in zip(ids.tolist(), seq.tolist(), pos.tolist()):
            s = (s + mix(b ^ mix(q * 65536 + k))) & M
        assert dg[i].tolist() == [len(ids), s]
        assert len(ids) <= 300


def test_generator_shapes():
    w = W.make_workload("longctx", n_requests=20000)
    nb = np.diff(w.hash_off.astype(np.int64))
    assert (nb == -(-w.input_tokens.astype(np.int64) // 512)).all()
    assert nb.max() <= 250 and (np.diff(w.ts_ms) >= 0).all()
    assert w.info["multi_turn_fraction"] > 0.6
    # every later turn re-sends at least 80 % of its blocks as a prior-turn prefix
    off = w.hash_off.astype(np.int64)
    last = {}
    for r in range(w.n_requests):
        ids = w.hash_ids[off[r]:off[r + 1]]
        s = int(w.session[r])
        if w.turn[r] > 0:
            prev = last[s]
            m = min(len(prev), len(ids))
            same = int(np.argmin(np.append(prev[:m] == ids[:m], False)))
            assert same * 5 >= len(ids) * 4
        last[s] = ids
