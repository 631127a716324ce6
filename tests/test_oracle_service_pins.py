"""CPU pins of the oracle's extended service model: decode slow-down with the number of busy
slots and admission under a KV-token budget (paper Section 2.2: continuous batching "bounded by
max concurrency and KV budget"; Section 5 / Appendix D: concentrating traffic on one replica
lowers TTFT but inflates E2E latency).  Hand cases, closed forms, a brute-force re-simulation of
one replica, and what must not change."""
import numpy as np
import pytest

from oracle import gorgo_oracle as O
from paper_2602_11688_b200 import workloads as W
from tests.util import small_trace

B = 512


def test_switched_off_it_changes_nothing():
    rng = np.random.default_rng(1)
    reqs = small_trace(4, n_req=300)
    w = W.handmade(rng.uniform(5, 80, size=4), reqs, slots=3, cache_blocks=10, params=[(0.8, 1.0, 0.7)])
    a = O.replay(w, w.params[0], 0.9)
    b = O.replay(w, w.params[0], 0.9, decode_slowdown=0.0, kv_budget_tokens=0)
    c = O.replay(w, w.params[0], 0.9, decode_slowdown=0.0, kv_budget_tokens=10 ** 12)   # never binds
    for x in (b, c):
        assert a[0].route.tolist() == x[0].route.tolist() and a[0].ttft.tolist() == x[0].ttft.tolist()
        assert a[0].e2e.tolist() == x[0].e2e.tolist()


def test_hand_case_decode_slows_down_with_the_busy_slots():
    # one replica, two slots, nothing cached, prefill 0.01 ms/token, tpot 10 ms, slow-down 0.5 per
    # extra busy slot.  r0 (t=0, 1000 tokens, 11 out): arrive 5, first 15; alone -> 10 ms/token,
    # finish 115.  r1 (t=10, 1000 tokens, 3 out): arrive 15 on slot 1, first 25; slot 0 is busy
    # until 115 > 25 -> b = 2 -> 15 ms/token, finish 25 + 2*15 = 55.  r2 (t=20, 1000, 2 out):
    # arrive 25, slots free at (115, 55) -> waits for 55, first 65; slot 0 still busy -> b = 2,
    # finish 65 + 15 = 80.  r3 (t=200): both free -> b = 1, first 215, finish 215 + 10 = 225.
    reqs = [(0.0, 1000, 11, [1, 2]), (10.0, 1000, 3, [3, 4]), (20.0, 1000, 2, [5, 6]),
            (200.0, 1000, 2, [7, 8])]
    w = W.handmade([5.0], reqs, slots=2, cache_blocks=100, prefill_ms_per_token=0.01,
                   tpot_ms=10.0, params=[(1.0, 1.0, 1.0)])
    res = O.replay(w, w.params[0], decode_slowdown=0.5)[0]
    np.testing.assert_allclose(res.ttft, [15.0, 15.0, 45.0, 15.0], rtol=1e-14)
    np.testing.assert_allclose(res.e2e, [115.0, 45.0, 60.0, 25.0], rtol=1e-14)
    plain = O.replay(w, w.params[0])[0]
    np.testing.assert_allclose(plain.e2e, [115.0, 35.0, 45.0, 25.0], rtol=1e-14)


def test_hand_case_kv_budget_delays_admission():
    # one replica, three slots, budget 3000 tokens; every request holds in + out tokens.
    # r0 (t=0): 1000+11 = 1011 tokens, first 15, finish 115.  r1 (t=1): 1500+6 = 1506, arrive 6,
    # first 21, finish 71; usage 1011 + 1506 fits.  r2 (t=2): 1000+3 = 1003 tokens, free slot 2,
    # arrive 7, but 1011 + 1506 + 1003 = 3520 > 3000: it waits for the first of the others to
    # finish (r1 at 71): then 1011 + 1003 fits -> start 71, first 81, finish 101.
    # r3 (t=3): 4000+1 tokens alone exceed the budget: it takes the slot that frees first (r1's,
    # at 71), waits until no other slot is busy (115) and runs alone: first 155, finish 155.
    reqs = [(0.0, 1000, 11, [1, 2]), (1.0, 1500, 6, [3, 4, 5]), (2.0, 1000, 3, [6, 7]),
            (3.0, 4000, 1, list(range(10, 18)))]
    w = W.handmade([5.0], reqs, slots=3, cache_blocks=100, prefill_ms_per_token=0.01,
                   tpot_ms=10.0, params=[(1.0, 1.0, 1.0)])
    o = O.Oracle.from_workload(w)
    o.set_service_model(0.0, 3000)
    res = o.run(w.params[0], 1.0)
    np.testing.assert_allclose(res.ttft, [15.0, 20.0, 79.0, 152.0], rtol=1e-14)
    np.testing.assert_allclose(res.e2e, [115.0, 70.0, 99.0, 152.0], rtol=1e-14)
    _, _, free_at = o.queues()
    assert free_at.tolist() == [[115.0, 155.0, 101.0]]
    plain = O.replay(w, w.params[0])[0]
    # (without the budget r2 runs at once, 17..37, and r3 follows it on that slot: first 37 + 40)
    np.testing.assert_allclose(plain.ttft, [15.0, 20.0, 15.0, 74.0], rtol=1e-14)


def _resimulate_one_replica(reqs, rtt, S, prefill, tpot, slowdown, budget):
    """Independent model of ONE replica without cache (all ids distinct): keeps, per slot, the
    whole list of (start, finish, tokens) it has run, finds admission times by scanning event
    times, and counts busy slots from those lists."""
    slots = [[] for _ in range(S)]
    out = []
    for (t, in_tok, o, ids) in reqs:
        free = [sl[-1][1] if sl else 0.0 for sl in slots]
        s = min(range(S), key=lambda i: (free[i], i))
        arrive = t + rtt
        need = in_tok + o
        T = max(arrive, free[s])
        if budget:
            events = sorted({f for i, f in enumerate(free) if i != s and f > T})
            for cand in [T] + events:
                usage = sum(slots[i][-1][2] for i in range(S) if i != s and slots[i] and free[i] > cand)
                busy = any(i != s and free[i] > cand for i in range(S))
                if not busy or usage + need <= budget:
                    T = cand
                    break
        first = T + prefill * in_tok
        b = 1 + sum(1 for i in range(S) if i != s and free[i] > first)
        finish = first + (tpot * (1.0 + slowdown * (b - 1))) * max(o - 1, 0)
        slots[s].append((T, finish, need))
        out.append((first - t, finish - t))
    return out


@pytest.mark.parametrize("slowdown,budget", [(0.0, 0), (0.3, 0), (0.0, 6000), (0.25, 5000)])
def test_one_replica_matches_an_independent_resimulation(slowdown, budget):
    rng = np.random.default_rng(7)
    reqs, t = [], 0.0
    for k in range(400):
        t += float(rng.exponential(25.0))
        n = int(rng.integers(1, 6))
        reqs.append((t, (n - 1) * B + int(rng.integers(1, B + 1)), int(rng.integers(0, 40)),
                     list(range(1000 * k, 1000 * k + n))))
    S, rtt, prefill, tpot = 4, 12.0, 0.02, 9.0
    w = W.handmade([rtt], reqs, slots=S, cache_blocks=10 ** 6, prefill_ms_per_token=prefill,
                   tpot_ms=tpot, params=[(1.0, 1.0, 1.0)])
    res = O.replay(w, w.params[0], decode_slowdown=slowdown, kv_budget_tokens=budget)[0]
    want = _resimulate_one_replica(reqs, rtt, S, prefill, tpot, slowdown, budget)
    np.testing.assert_allclose(res.ttft, [a for a, _ in want], rtol=1e-12)
    np.testing.assert_allclose(res.e2e, [b for _, b in want], rtol=1e-12)
    if budget:
        plain = O.replay(w, w.params[0], decode_slowdown=slowdown)[0]
        assert (res.ttft >= plain.ttft - 1e-9).all() and (res.ttft > plain.ttft + 1e-9).any()


def test_single_slot_is_never_slowed_down():
    rng = np.random.default_rng(5)
    reqs = small_trace(9, n_req=200)
    w = W.handmade(rng.uniform(5, 50, size=3), reqs, slots=1, cache_blocks=12, params=[(1.0, 1.0, 0.5)])
    a = O.replay(w, w.params[0])[0]
    b = O.replay(w, w.params[0], decode_slowdown=2.0, kv_budget_tokens=10)[0]
    # one slot per replica: never another busy slot, so neither rule can bind
    assert a.e2e.tolist() == b.e2e.tolist() and a.route.tolist() == b.route.tolist()


def test_the_service_model_does_not_enter_the_score():
    rng = np.random.default_rng(3)
    reqs = small_trace(3, n_req=1)
    w = W.handmade(rng.uniform(5, 80, size=3), reqs, slots=2, cache_blocks=10, params=[(0.8, 1.0, 0.7)])
    o = O.Oracle.from_workload(w)
    a = o.run(w.params[0], 1.0, detail=True).cost_all.copy()
    o.reset(); o.set_service_model(0.7, 1234)
    b = o.run(w.params[0], 1.0, detail=True).cost_all
    assert a.tolist() == b.tolist()
    with pytest.raises(ValueError):
        o.set_service_model(-0.1, 0)
    o.close()


def test_concentrating_traffic_inflates_e2e_not_ttft_once_decode_slows_down():
    # Section 5 / Appendix D: with a zero queue weight nearly all traffic goes to one replica; the
    # paper sees the lowest TTFT and the worst E2E latency there.  Under the plain service model a
    # lightly loaded replica shows nothing of it; with a decode slow-down its full batch decodes
    # slower, so p95 E2E grows while p95 TTFT barely moves, and it grows more than for a policy
    # that spreads the load.
    w = W.make_workload("tiny", n_requests=1500)
    w.spec.slots = 16
    near = np.array([1.0, 1.0, 0.0])          # network and prefill only
    fair = np.array([1.0, 1.0, 0.02])
    scale = 12.0                              # light load: hardly any waiting for a slot
    near0, near1 = O.replay(w, near, scale), O.replay(w, near, scale, decode_slowdown=0.1)
    fair0, fair1 = O.replay(w, fair, scale), O.replay(w, fair, scale, decode_slowdown=0.1)
    assert np.bincount(near1[0].route, minlength=4).max() / w.n_requests > 0.8
    assert near1[2] / near0[2] > 1.3 and near1[1] / near0[1] < 1.1      # E2E up, TTFT about the same
    assert near1[2] / near0[2] > fair1[2] / fair0[2]                    # spreading the load suffers less
    assert near1[2] > fair1[2]
