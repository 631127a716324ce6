"""CPU pins of the oracle's per-replica service speeds (heterogeneous replicas, which the paper's
Section 7 names as a limitation of its uniform fleet): closed forms without waiting or eviction,
equality with the uniform constants, a single-slot queue recursion, and what must NOT change."""
import numpy as np
import pytest

from oracle import gorgo_oracle as O
from paper_2602_11688_b200 import workloads as W
from tests.util import small_trace

B = 512


def test_uniform_arrays_change_nothing():
    rng = np.random.default_rng(1)
    reqs = small_trace(1, n_req=300)
    w = W.handmade(rng.uniform(5, 80, size=4), reqs, slots=2, cache_blocks=10, params=[(0.8, 1.0, 0.7)])
    a = O.replay(w, w.params[0], 0.9)
    b = O.replay(w, w.params[0], 0.9, rep_prefill_ms=np.full(4, 0.05), rep_tpot_ms=np.full(4, 20.0))
    assert a[0].route.tolist() == b[0].route.tolist() and a[0].ttft.tolist() == b[0].ttft.tolist()
    assert a[0].e2e.tolist() == b[0].e2e.tolist() and a[3].tolist() == b[3].tolist()


def test_closed_form_without_waiting_or_eviction():
    rng = np.random.default_rng(2)
    reqs = small_trace(2, n_req=250, structured=True)
    R = 4
    rtt = rng.uniform(5, 80, size=R)
    pre = np.array([0.05, 0.1, 0.02, 0.07])
    tpot = np.array([20.0, 5.0, 40.0, 12.0])
    w = W.handmade(rtt, reqs, slots=len(reqs), cache_blocks=10 ** 6, params=[(0.0, 0.0, 1.0)])
    res = O.replay(w, w.params[0], 1.0, rep_prefill_ms=pre, rep_tpot_ms=tpot)[0]
    for r, (t, in_tok, out, ids) in enumerate(reqs):
        i = int(res.route[r])
        unc = in_tok - min(int(res.hit[r]) * B, in_tok)
        assert res.ttft[r] == pytest.approx(rtt[i] + pre[i] * unc, rel=1e-12, abs=1e-12)
        assert res.e2e[r] - res.ttft[r] == pytest.approx(tpot[i] * max(out - 1, 0), rel=1e-9, abs=1e-9)
    assert len(set(res.route.tolist())) > 1            # several replicas really served


def test_speeds_do_not_enter_the_score():
    # same state, same request: the score of Eq. 3 has no term for the replica's speed
    rng = np.random.default_rng(3)
    reqs = small_trace(3, n_req=1)
    w = W.handmade(rng.uniform(5, 80, size=3), reqs, slots=1, cache_blocks=10, params=[(0.8, 1.0, 0.7)])
    o = O.Oracle.from_workload(w)
    a = o.run(w.params[0], 1.0, detail=True).cost_all.copy()
    o.reset(); o.set_replica_speeds(np.array([1.0, 2.0, 3.0]), np.array([7.0, 8.0, 9.0]))
    b = o.run(w.params[0], 1.0, detail=True).cost_all
    o.close()
    assert a.tolist() == b.tolist()


def test_single_slot_queue_recursion_with_a_slow_replica():
    # one replica, one slot: start_{r+1} = max(arrival + rtt, finish_r), with the replica's rates
    rng = np.random.default_rng(4)
    reqs = [(float(t), int(rng.integers(1, 4)) * B, int(rng.integers(1, 20)), [100 + k])
            for k, t in enumerate(np.cumsum(rng.exponential(30.0, size=120)))]
    w = W.handmade([12.0], reqs, slots=1, cache_blocks=10 ** 6, params=[(1.0, 1.0, 1.0)])
    pre, tp = 0.03, 11.0
    res = O.replay(w, w.params[0], 1.0, rep_prefill_ms=[pre], rep_tpot_ms=[tp])[0]
    free = 0.0
    for r, (t, in_tok, out, ids) in enumerate(reqs):
        start = max(t + 12.0, free)
        first = start + pre * in_tok                   # distinct ids: nothing is ever cached
        free = first + tp * max(out - 1, 0)
        assert res.ttft[r] == pytest.approx(first - t, rel=1e-12)
        assert res.e2e[r] == pytest.approx(free - t, rel=1e-12)


def test_bad_speeds_are_rejected():
    w = W.handmade([10.0, 20.0], small_trace(5, n_req=5), slots=1, cache_blocks=10)
    o = O.Oracle.from_workload(w)
    with pytest.raises(ValueError):
        o.set_replica_speeds(np.array([0.05, -1.0]), None)
    with pytest.raises(ValueError):
        o.set_replica_speeds(None, np.array([np.nan, 1.0]))
    o.close()
