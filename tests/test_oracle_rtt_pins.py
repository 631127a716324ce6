"""CPU pins of the oracle's time-varying network (paper Section 2.2: the proxy's RTT signal is an
exponentially weighted moving average of a probe sent every 30 s): a constant series is the
static matrix bit for bit, the EWMA's closed form after a step, epoch boundaries, and a hand case
in which the proxy's lagging belief decides the route while the real delay decides the TTFT."""
import numpy as np
import pytest

from oracle import gorgo_oracle as O
from paper_2602_11688_b200 import workloads as W
from tests.util import small_trace


def test_constant_series_is_the_static_matrix():
    rng = np.random.default_rng(1)
    reqs = small_trace(5, n_req=300)
    rtt = rng.uniform(5, 80, size=4)
    w = W.handmade(rtt, reqs, slots=2, cache_blocks=10, params=[(0.8, 1.0, 0.7)])
    a = O.replay(w, w.params[0], 0.9)
    series = np.tile(rtt.reshape(1, 1, 4), (7, 1, 1))
    b = O.replay(w, w.params[0], 0.9, rtt_series=series, epoch_ms=1500.0, alpha=0.37)
    assert a[0].route.tolist() == b[0].route.tolist() and a[0].ttft.tolist() == b[0].ttft.tolist()
    assert a[0].e2e.tolist() == b[0].e2e.tolist() and a[3].tolist() == b[3].tolist()


def test_belief_lags_the_network_route_follows_belief_ttft_follows_the_network():
    # two replicas, nothing cached, only the network weight counts.  Epochs of 100 ms, alpha 0.5.
    # replica 0: probes 10, 10, 90, 90 -> belief 10, 10, 50, 70; replica 1: constant 40.
    # t = 50  (epoch 0): belief (10, 40) -> replica 0, delay 10.
    # t = 250 (epoch 2): belief (50, 40) -> replica 1, delay 40.
    # t = 200 exactly is already epoch 2.  t = 199.9 (epoch 1): belief (10, 40) -> replica 0, delay 10.
    # t = 350 (epoch 3): belief (70, 40) -> replica 1.   t = 900 (past the last epoch): epoch 3 again.
    series = np.array([[[10.0, 40.0]], [[10.0, 40.0]], [[90.0, 40.0]], [[90.0, 40.0]]])
    ts = [50.0, 199.9, 200.0, 250.0, 350.0, 900.0]
    reqs = [(t, 512, 1, [100 + k]) for k, t in enumerate(ts)]
    w = W.handmade([10.0, 40.0], reqs, slots=8, cache_blocks=64, prefill_ms_per_token=0.0,
                   params=[(1.0, 0.0, 0.0)])
    o = O.Oracle.from_workload(w)
    o.set_rtt_series(series, epoch_ms=100.0, alpha=0.5)
    res = o.run(w.params[0], 1.0, detail=True)
    assert res.route.tolist() == [0, 0, 1, 1, 1, 1]
    assert res.cost_all.tolist() == [[10.0, 40.0], [10.0, 40.0], [50.0, 40.0], [50.0, 40.0],
                                     [70.0, 40.0], [70.0, 40.0]]
    assert res.ttft.tolist() == [10.0, 10.0, 40.0, 40.0, 40.0, 40.0]
    # a weight of zero on the network ignores the belief; the delay is still the epoch's probe:
    # everything goes to replica 0, whose real RTT is 90 from epoch 2 on
    o.reset()
    res = o.run(np.array([0.0, 0.0, 0.0]), 1.0)
    assert res.route.tolist() == [0] * 6 and res.ttft.tolist() == [10.0, 10.0, 90.0, 90.0, 90.0, 90.0]
    # the time scale moves the requests, not the epochs: at scale 0.5 the request of t = 350 arrives
    # at 175, in epoch 1
    o.reset()
    res = o.run(w.params[0], 0.5)
    assert res.route.tolist() == [0, 0, 0, 0, 0, 1]
    o.close()


def test_ewma_closed_form_after_a_step():
    # probe jumps from a to b at epoch 5: belief = b - (b - a) * (1 - alpha)^(e - 4)
    a_, b_, alpha, E = 20.0, 120.0, 0.3, 30
    series = np.full((E, 1, 2), a_)
    series[5:, 0, 0] = b_
    reqs = [(1000.0 * e + 1.0, 512, 1, [e + 1]) for e in range(E)]
    w = W.handmade([a_, a_], reqs, slots=64, cache_blocks=1000, prefill_ms_per_token=0.0,
                   params=[(1.0, 0.0, 0.0)])
    res = O.replay(w, w.params[0], 1.0, detail=True, rtt_series=series, epoch_ms=1000.0, alpha=alpha)[0]
    for e in range(E):
        want = a_ if e < 5 else b_ - (b_ - a_) * (1 - alpha) ** (e - 4)
        assert res.cost_all[e, 0] == pytest.approx(want, rel=1e-12)
        assert res.cost_all[e, 1] == a_
    # alpha = 1: the belief is the last probe
    res = O.replay(w, w.params[0], 1.0, detail=True, rtt_series=series, epoch_ms=1000.0, alpha=1.0)[0]
    assert res.cost_all[:, 0].tolist() == series[:, 0, 0].tolist()


def test_bad_series_are_rejected_and_none_restores_the_matrix():
    reqs = small_trace(2, n_req=20)
    w = W.handmade([10.0, 20.0], reqs, slots=2, cache_blocks=10, params=[(1.0, 1.0, 1.0)])
    o = O.Oracle.from_workload(w)
    base = o.run(w.params[0], 1.0).ttft.tolist()
    good = np.full((3, 1, 2), 15.0)
    for bad in (dict(epoch_ms=0.0), dict(alpha=0.0), dict(alpha=1.5)):
        with pytest.raises(ValueError):
            o.set_rtt_series(good, **{**dict(epoch_ms=10.0, alpha=0.5), **bad})
    with pytest.raises(ValueError):
        o.set_rtt_series(-good, 10.0, 0.5)
    o.set_rtt_series(good, 10.0, 0.5)
    o.reset()
    assert o.run(w.params[0], 1.0).ttft.tolist() != base
    o.set_rtt_series(None)
    o.reset()
    assert o.run(w.params[0], 1.0).ttft.tolist() == base
    o.close()
