"""CPU pins of the tuning-loop oracle (oracle/gorgo_tuning.py): the paper's own arithmetic,
closed forms, a library percentile per window, invariants of the 1/5 rule and of Eq. 4."""
import math

import numpy as np
import pytest

from oracle import gorgo_tuning as T


def test_paper_arithmetic_672_samples_is_the_18th_step():
    # Section 5 / convergence figure: the strategy converges after 672 samples, the 18th step,
    # with a 128-request window and hop 32: 128 + 17 * 32 = 672.
    assert T.window_count(672) == 18
    assert T.window_count(671) == 17
    assert T.window_count(127) == 0 and T.window_count(128) == 1 and T.window_count(159) == 1
    assert T.window_count(160) == 2


def test_window_p95_closed_forms():
    v = [float(i) for i in range(1000)]                     # sorted: rank 122 of window j
    w = T.window_p95(v)
    assert w == [float(j * 32 + 121) for j in range(len(w))]
    assert T.window_p95([3.5] * 300) == [3.5] * T.window_count(300)
    d = [float(-i) for i in range(400)]                     # descending: 122nd smallest
    assert T.window_p95(d) == [float(-(j * 32 + 127 - 121)) for j in range(T.window_count(400))]
    # other shapes: k = ceil(0.95 W)
    assert T.window_p95([float(i) for i in range(40)], window=20, hop=10) == [18.0, 28.0, 38.0]
    assert T.window_p95([5.0, 1.0, 3.0], window=1, hop=1) == [5.0, 1.0, 3.0]


def test_window_p95_equals_library_percentile_per_window():
    rng = np.random.default_rng(3)
    v = rng.lognormal(5.0, 1.0, size=777)
    v[rng.integers(0, 777, size=100)] = v[0]                # ties
    got = T.window_p95(list(v), 128, 32)
    for j, g in enumerate(got):
        assert g == np.percentile(v[j * 32: j * 32 + 128], 95, method="inverted_cdf")
    got = T.window_p95(list(v), 100, 7)
    for j, g in enumerate(got):
        assert g == np.percentile(v[j * 7: j * 7 + 100], 95, method="inverted_cdf")
    best, idx = T.best_window(list(v))
    assert best == min(T.window_p95(list(v))) and T.window_p95(list(v))[idx] == best
    assert idx == int(np.argmin(T.window_p95(list(v))))


def test_mutation_eq4():
    lo, hi = [0.05, 0.05], [2.0, 0.5]
    x = [0.5, 0.1]                                          # Section 4: initial weights
    same = T.mutate(x, 0.5, [0.0, 0.0], lo, hi)
    assert same == pytest.approx(x, rel=4e-16)              # exp(ln x) within rounding
    up = T.mutate(x, 0.5, [1.0, -2.0], lo, hi)
    assert up[0] == pytest.approx(0.5 * math.exp(0.5), rel=1e-15)    # multiplicative in log space
    assert 0.1 * math.exp(-1.0) < 0.05 and up[1] == 0.05            # below the range: clamped
    assert T.mutate(x, 0.5, [10.0, 10.0], lo, hi) == hi     # clamped above
    assert T.mutate(x, 0.5, [-10.0, -10.0], lo, hi) == lo   # clamped below
    # symmetric in log space: +z then -z returns to the start
    there = T.mutate(x, 0.3, [0.7, -0.4], [1e-9] * 2, [1e9] * 2)
    back = T.mutate(there, 0.3, [-0.7, 0.4], [1e-9] * 2, [1e9] * 2)
    assert back == pytest.approx(x, rel=1e-15)


def test_one_fifth_rule_is_stationary_at_one_success_in_five():
    def obj(x):
        return abs(math.log(x[0]) - math.log(1.0))

    # step 1 moves towards the target (accepted), the next four move away (rejected)
    z = [[[0.5]], [[-3.0]], [[-3.0]], [[-3.0]], [[-3.0]]]
    x, f, sigma, hist = T.es_run(obj, [0.5], [0], [1e-3], [1e3], 0.5, 1.5, z)
    assert [h[1] for h in hist] == [True, False, False, False, False]
    assert sigma == pytest.approx(0.5, rel=1e-14)           # 1.5 * (1.5 ** -0.25) ** 4 == 1
    assert hist[0][2] == pytest.approx(0.75) and hist[1][2] == pytest.approx(0.75 * 1.5 ** -0.25)
    assert x[0] == pytest.approx(0.5 * math.exp(0.25))


def test_es_keeps_the_best_and_never_gets_worse():
    rng = np.random.default_rng(11)
    target = np.array([0.276, 0.5])                         # the weights the paper reports learning

    def obj(x):
        return float(np.sum((np.log([x[0], x[2]]) - np.log(target)) ** 2))

    z = rng.standard_normal((60, 4, 2)).tolist()
    x, f, sigma, hist = T.es_run(obj, [0.5, 1.0, 0.1], [0, 2], [0.05, 0.05], [2.0, 0.5], 0.5, 1.5, z)
    parents = [h[3] for h in hist]
    assert all(b <= a for a, b in zip(parents, parents[1:]))          # elitist
    assert f == parents[-1] and f < obj([0.5, 1.0, 0.1]) * 0.05       # converges on a convex bowl
    assert x[1] == 1.0                                                # untuned weight untouched
    assert 0.05 <= x[0] <= 2.0 and 0.05 <= x[2] <= 0.5
    for h in hist:
        if h[1]:
            assert h[0] == h[3]                                       # accepted: parent takes it
        else:
            assert h[0] >= h[3]                                       # rejected: did not beat it


def test_es_ties_go_to_the_lowest_index_and_equal_does_not_beat():
    def obj(x):
        return 1.0                                                   # flat: nothing beats the parent

    z = [[[0.3], [0.1], [-0.2]]] * 3
    x, f, sigma, hist = T.es_run(obj, [0.5], [0], [0.05], [2.0], 0.5, 2.0, z)
    assert x == [0.5] and all(not h[1] for h in hist)
    assert sigma == pytest.approx(0.5 * 2.0 ** -0.75)

    # two offspring with the same best objective: the first is taken
    def obj2(x):
        return round(abs(x[0] - 0.5), 12) if x[0] != 0.5 else 9.0

    z2 = [[[0.2], [-0.2], [0.2]]]
    x2, f2, _, h2 = T.es_run(obj2, [0.5], [0], [0.05], [2.0], 0.5, 1.5, z2)
    cand = [0.5 * math.exp(0.1), 0.5 * math.exp(-0.1), 0.5 * math.exp(0.1)]
    fs = [obj2([c]) for c in cand]
    assert x2[0] == pytest.approx(cand[fs.index(min(fs))])


# ------------------------------------------------------------------ online tuning (one replay)
def _stub_chunks(values):
    """run_chunk stand-in: hands out prescribed TTFTs and records (weights, count) per chunk."""
    it, calls = iter(values), []

    def run_chunk(weights, count):
        calls.append((list(weights), count))
        return [next(it) for _ in range(count)]
    return run_chunk, calls


def test_online_steps_follow_the_papers_sample_count():
    # step k happens after 128 + (k-1)*32 requests: the 18th after 672 samples (convergence figure)
    n = 700
    run_chunk, calls = _stub_chunks([1.0] * n)
    z = [[0.1, -0.1]] * 40
    ttft, schedule, history = T.online_tune(run_chunk, n, [0.5, 1.0, 0.1], [0, 2], [0.05, 0.05],
                                            [2.0, 0.5], 0.5, 1.5, z)
    assert [c for _, c in calls] == [128] + [32] * 17 + [700 - 672]
    assert len(history) == T.window_count(n) == 18 and len(ttft) == n
    assert sum(c for _, c in calls[:18]) == 672
    # weights change only between chunks, and the chunk after step k runs under step k's offspring
    for k, h in enumerate(history):
        assert [calls[k + 1][0][i] for i in (0, 2)] == h[5]
        assert calls[k + 1][0][1] == 1.0                      # the untuned weight stays
    assert schedule == [c[0] for c in calls]
    # fewer draws than windows: the last offspring stays in force
    run_chunk, calls = _stub_chunks([1.0] * n)
    _, _, history = T.online_tune(run_chunk, n, [0.5, 1.0, 0.1], [0, 2], [0.05, 0.05], [2.0, 0.5],
                                  0.5, 1.5, z[:3])
    assert len(history) == 3 and all(c[0] == calls[3][0] for c in calls[3:])


def test_online_accept_reject_and_sigma():
    # window values (constant chunks make the p95 of a window the maximum of its four hops ...
    # here every chunk is flat, and levels are chosen so that the window value is known):
    # chunk levels: first window 10; then hops 10, 4, 4, 4, 4, 9 -> window values
    # 10 (step 1: start weights), 10 (not < 10: rejected), 10, 10, 10 (still holds a 10-hop), ...
    levels = [10.0] * 128 + [10.0] * 32 + [4.0] * 128 + [9.0] * 32 + [1.0] * 32
    run_chunk, calls = _stub_chunks(levels)
    z = [[0.3]] * 20
    ttft, schedule, hist = T.online_tune(run_chunk, len(levels), [0.5], [0], [0.05], [2.0], 0.5, 1.5, z)
    values = [h[0] for h in hist]
    assert values == T.window_p95(levels)                      # each step sees the last 128 TTFTs
    assert values[:2] == [10.0, 10.0] and values[5] == 4.0
    accepted = [h[1] for h in hist]
    assert accepted[0] is False and accepted[1] is False       # step 1 only scores the start weights
    first_acc = accepted.index(True)
    assert values[first_acc] < 10.0 and all(v >= 10.0 for v in values[1:first_acc])
    # sigma: x a after an accepted step, x a^(-1/4) after a rejected one (step 1 changes nothing)
    sigma = 0.5
    parent_f = values[0]
    for k, h in enumerate(hist[1:], start=1):
        if h[0] < parent_f:
            sigma *= 1.5; parent_f = h[0]
        else:
            sigma *= 1.5 ** -0.25
        assert h[2] == sigma and h[3] == parent_f and h[1] == (h[0] == parent_f and hist[k - 1][3] != parent_f)
    # an accepted step makes the offspring in force the new parent; the next offspring mutates it
    k = first_acc
    assert hist[k][4] == hist[k - 1][5]
    assert hist[k][5] == T.mutate(hist[k][4], hist[k][2], z[k], [0.05], [2.0])


def test_online_with_clamped_weights_is_the_plain_replay():
    # lo = hi pins every tuned weight: the schedule never changes and the chunked replay must be
    # the one-shot replay, request for request
    from oracle import gorgo_oracle as O
    from paper_2602_11688_b200 import workloads as W
    w = W.make_workload("tiny", n_requests=500, cache_blocks=300)
    x0 = [0.7, 1.0, 0.3]
    o = O.Oracle.from_workload(w)
    chunks = []

    def run_chunk(weights, count):
        r = o.run(np.array(weights), 1.0, count=count)
        chunks.append(r)
        return list(r.ttft)
    rng = np.random.default_rng(0)
    z = rng.normal(size=(20, 2)).tolist()
    ttft, schedule, hist = T.online_tune(run_chunk, w.n_requests, x0, [0, 2], [0.7, 0.3], [0.7, 0.3],
                                         0.5, 1.5, z)
    assert all(s == x0 for s in schedule) and len(hist) == T.window_count(500)
    plain, *_ = O.replay(w, np.array(x0), 1.0)
    assert ttft == list(plain.ttft)
    assert np.concatenate([c.route for c in chunks]).tolist() == plain.route.tolist()
