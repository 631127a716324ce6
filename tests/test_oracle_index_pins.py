"""CPU pins of the oracle's drifting proxy index (paper Section 7: the proxy's prefix index is
built from the requests it dispatched and does not see the replica's evictions): without
evictions it is the cache, a hand case where the index promises a hit the replica no longer has,
a brute-force recount of the index from the routes alone, and what stays untouched."""
import numpy as np
import pytest

from oracle import gorgo_oracle as O
from paper_2602_11688_b200 import workloads as W
from tests.util import small_trace

B = 512


def test_without_evictions_the_index_is_the_cache():
    rng = np.random.default_rng(1)
    reqs = small_trace(8, n_req=300)
    w = W.handmade(rng.uniform(5, 80, size=4), reqs, slots=2, cache_blocks=10 ** 6, params=[(0.8, 1.0, 0.7)])
    a = O.replay(w, w.params[0], 0.9)
    b = O.replay(w, w.params[0], 0.9, proxy_index=True)
    assert a[0].route.tolist() == b[0].route.tolist() and a[0].ttft.tolist() == b[0].ttft.tolist()
    assert a[0].hit.tolist() == b[0].hit.tolist() and a[3].tolist() == b[3].tolist()


def test_hand_case_the_index_promises_a_hit_the_replica_has_evicted():
    # two replicas, cache of 2 blocks each, only the prefill weight counts (ties go to replica 0).
    # r0 [A,B] -> replica 0 (tie).  r1 [C,D]: nothing known anywhere -> replica 0 again; its cache
    # now holds C,D: A,B are evicted, but the proxy's index of replica 0 still lists A,B,C,D.
    # r2 [A,B]: the index promises 2 hits on replica 0 (score 0 against 1024) -> replica 0, where
    # the real cache has neither: reported hit 0 and the full prefill of 1024 tokens is paid.
    # r3 [C,D]: the same the other way round (r2 has pushed C,D out again).
    reqs = [(0.0, 1024, 1, [1, 2]), (100.0, 1024, 1, [3, 4]), (200.0, 1024, 1, [1, 2]),
            (300.0, 1024, 1, [3, 4])]
    w = W.handmade([10.0, 10.0], reqs, slots=4, cache_blocks=2, prefill_ms_per_token=0.01,
                   params=[(0.0, 1.0, 0.0)])
    o = O.Oracle.from_workload(w)
    o.set_proxy_index(True)
    res = o.run(w.params[0], 1.0, detail=True)
    assert res.route.tolist() == [0, 0, 0, 0]
    assert res.cost_all.tolist() == [[1024.0, 1024.0], [1024.0, 1024.0], [0.0, 1024.0], [0.0, 1024.0]]
    assert res.hit.tolist() == [0, 0, 0, 0]                      # the replica never has the prefix
    np.testing.assert_allclose(res.ttft, [10.0 + 10.24] * 4, rtol=1e-12)   # full prefill every time
    assert res.hit_all.tolist() == [[0, 0]] * 4                  # real caches: C,D / A,B alternate
    o.close()
    plain = O.replay(w, w.params[0], 1.0, detail=True)[0]
    assert plain.cost_all.tolist() == [[1024.0, 1024.0]] * 4     # the real cache never promises anything


@pytest.mark.parametrize("structured", [True, False])
def test_index_hits_recomputed_from_the_routes_alone(structured):
    # weights (0, 1, 0): the score of replica i is exactly the tokens the proxy believes uncached,
    # so the index's prefix hit can be read off the score and recomputed by brute force as the
    # prefix over the union of the blocks of all earlier requests routed to i
    reqs = small_trace(13, n_req=300, structured=structured)
    R, C = 3, 9
    w = W.handmade([20.0, 35.0, 50.0], reqs, slots=2, cache_blocks=C, params=[(0.0, 1.0, 0.0)])
    res = O.replay(w, w.params[0], 1.0, detail=True, proxy_index=True)[0]
    seen = [set() for _ in range(R)]
    beyond = 0
    for r, (t, in_tok, out, ids) in enumerate(reqs):
        for i in range(R):
            hb = 0
            while hb < len(ids) and ids[hb] in seen[i]:
                hb += 1
            assert res.cost_all[r, i] == float(in_tok - min(hb * B, in_tok)), (r, i)
            assert res.hit_all[r, i] <= hb                       # the index never knows less than the cache
            beyond += int(res.hit_all[r, i] < hb)
        seen[int(res.route[r])].update(ids)
    assert beyond > 0                                            # the two did drift apart
    assert int(res.evicted.sum()) > 0


def test_the_cache_and_the_service_model_follow_the_replica_not_the_index():
    # forcing the routes of an index-scored run through the plain model gives the same caches,
    # hits and times: the index only enters the score
    reqs = small_trace(5, n_req=250)
    w = W.handmade([20.0, 35.0, 50.0], reqs, slots=2, cache_blocks=9, params=[(0.3, 1.0, 0.2)])
    a = O.replay(w, w.params[0], 1.0, proxy_index=True)
    b = O.replay(w, w.params[0], 1.0, forced_route=a[0].route)
    assert a[0].hit.tolist() == b[0].hit.tolist() and a[0].ttft.tolist() == b[0].ttft.tolist()
    assert a[0].e2e.tolist() == b[0].e2e.tolist() and a[3].tolist() == b[3].tolist()
    plain = O.replay(w, w.params[0], 1.0)
    assert plain[0].route.tolist() != a[0].route.tolist()        # and it does change decisions
