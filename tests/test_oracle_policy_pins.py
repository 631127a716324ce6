"""CPU pins of the baseline-policy switches of the oracle (Section 4, "Baseline policies"):
hand case, brute-force request counts, closed forms, and consistency with the plain replay."""
import numpy as np
import pytest

from oracle import gorgo_oracle as O
from oracle import gorgo_policies as P
from paper_2602_11688_b200 import workloads as W
from tests.util import small_trace

B = 512


def test_mix64_known_answer():
    # splitmix64 finaliser, published test value
    assert P.mix64(0x9E3779B97F4A7C15) == 0xE220A8397B1DCDAF


def test_least_request_differs_from_least_load_hand_case():
    # two replicas, same RTT, nothing completes (long decodes, 1 ms apart)
    reqs = [(0.0, 4 * B, 500, [1, 2, 3, 4]),      # -> replica 0 (all equal, lowest index)
            (1.0, 1 * B, 500, [10]),              # -> replica 1 (0 in flight there)
            (2.0, 1 * B, 500, [11]),              # requests: (1, 1) tie -> 0; tokens: (2048, 512) -> 1
            (3.0, 1 * B, 500, [12])]              # requests: (2, 1) -> 1;   tokens: (2048, 1024) -> 1
    w = W.handmade([10.0, 10.0], reqs, slots=8, cache_blocks=100)
    by_req = P.replay_policy(w, "least-request")[0]
    by_tok = P.replay_policy(w, "least-load")[0]
    assert by_req.route.tolist() == [0, 1, 0, 1]
    assert by_tok.route.tolist() == [0, 1, 1, 1]


@pytest.mark.parametrize("seed", [1, 2])
def test_request_signal_is_the_number_of_unfinished_requests(seed):
    rng = np.random.default_rng(seed)
    reqs = small_trace(seed, n_req=250, rate_ms=30.0)
    w = W.handmade(rng.uniform(5, 80, size=4), reqs, slots=2, cache_blocks=12)
    wts = np.array([0.0, 0.0, 1.0])
    o = O.Oracle.from_workload(w)
    o.set_policy(queue_in_requests=True)
    res = o.run(wts, 0.7, detail=True)
    o.close()
    t = 0.7 * w.ts_ms
    finish = t + res.e2e
    for r in range(w.n_requests):
        for i in range(4):
            count = sum(1 for j in range(r) if res.route[j] == i and finish[j] > t[r])
            assert res.cost_all[r, i] == float(count)
        assert res.route[r] == int(np.argmin(res.cost_all[r]))        # lowest index on ties


def test_equal_prompts_make_request_and_token_signals_agree():
    rng = np.random.default_rng(5)
    reqs = [(float(t), 3 * B, int(rng.integers(0, 40)), [1000 + 3 * k, 1001 + 3 * k, 1002 + 3 * k])
            for k, t in enumerate(np.cumsum(rng.exponential(20.0, size=200)))]
    w = W.handmade(rng.uniform(5, 50, size=3), reqs, slots=2, cache_blocks=50)
    a = P.replay_policy(w, "least-request")[0]
    b = P.replay_policy(w, "least-load")[0]
    assert a.route.tolist() == b.route.tolist() and a.ttft.tolist() == b.ttft.tolist()


def test_forced_routes_are_taken_and_change_nothing_else():
    rng = np.random.default_rng(9)
    reqs = small_trace(9, n_req=300)
    w = W.handmade(rng.uniform(5, 80, size=3), reqs, slots=2, cache_blocks=10,
                   params=[(0.7, 1.1, 0.9)])
    plain = O.replay(w, w.params[0], 1.0)
    again = O.replay(w, w.params[0], 1.0, forced_route=plain[0].route)
    assert again[0].route.tolist() == plain[0].route.tolist()
    assert again[0].hit.tolist() == plain[0].hit.tolist()
    assert again[0].ttft.tolist() == plain[0].ttft.tolist()
    assert again[3].tolist() == plain[3].tolist() and again[1] == plain[1] and again[2] == plain[2]
    with pytest.raises(ValueError):
        O.replay(w, w.params[0], 1.0, forced_route=np.full(w.n_requests, 3, np.uint8))


def test_session_affinity_and_random_closed_forms():
    rng = np.random.default_rng(4)
    reqs = small_trace(4, n_req=300, structured=True)
    R = 5
    rtt = rng.uniform(5, 80, size=R)
    # no eviction (huge cache) and no waiting (a slot per request): everything has a closed form
    w = W.handmade(rtt, reqs, slots=len(reqs), cache_blocks=10 ** 6)
    draws = rng.integers(0, 2 ** 32, size=len(reqs), dtype=np.uint64)
    for policy, want in (("session-affinity", P.affinity_routes(w)),
                         ("random", P.random_routes(w, draws))):
        res = P.replay_policy(w, policy, draws=draws)[0]
        assert res.route.tolist() == want.tolist()
        held = [set() for _ in range(R)]
        for r, (t, in_tok, out, ids) in enumerate(reqs):
            i = int(want[r])
            h = 0
            while h < len(ids) and ids[h] in held[i]:
                h += 1
            assert res.hit[r] == h
            unc = in_tok - min(h * B, in_tok)
            assert res.ttft[r] == pytest.approx(rtt[i] + 0.05 * unc, rel=1e-12)
            held[i].update(ids)
    aff = P.affinity_routes(w)
    first = {}
    for r, q in enumerate(reqs):                         # same first block -> same replica
        assert first.setdefault(q[3][0], aff[r]) == aff[r]
        assert aff[r] == P.mix64(q[3][0]) % R
    assert P.random_routes(w, [7, 5, 2 ** 32 - 1]).tolist() == [2, 0, (2 ** 32 - 1) % 5]


def test_prefix_cache_policy_takes_the_longest_cached_prefix():
    rng = np.random.default_rng(6)
    reqs = small_trace(6, n_req=300)
    w = W.handmade(rng.uniform(5, 80, size=4), reqs, slots=2, cache_blocks=15)
    o = O.Oracle.from_workload(w)
    res = o.run(np.array([0.0, 1.0, 0.0]), 1.0, detail=True)
    o.close()
    ref = P.replay_policy(w, "prefix-cache")[0]
    assert ref.route.tolist() == res.route.tolist()
    for r in range(w.n_requests):
        assert res.route[r] == int(np.argmax(res.hit_all[r]))          # first maximum
