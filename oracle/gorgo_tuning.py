"""TEST INFRASTRUCTURE ONLY -- plain CPU statement of the tuning loop around the routing simulator.

Nothing in the product path may import this file; it shares no code with the CUDA library.
Pure-Python loops over small inputs, fp64, steps in the paper's order and notation:

* ``window_p95``: the tuner's objective (paper Section 4): p95 TTFT of a rolling window of 128
  requests with hop 32; window j covers requests [j*hop, j*hop + window); nearest-rank p95, the
  k-th smallest with k = ceil(0.95 * window) in integers (the reading taken for every p95 here).
* ``mutate``: Eq. 4 (Section 2.3): x'_k = clip(exp(ln x_k + sigma z_k), [lo_k, hi_k]).
* ``es_run``: the (1+1)-ES of Section 2.3, generalised to lambda offspring per step: the best
  offspring (lowest index among equals) replaces the parent iff its objective is strictly
  smaller.  Rechenberg's 1/5 rule with the reading  sigma *= a  after an accepted step and
  sigma *= a**(-1/4)  after a rejected one (the paper names the rule, not its constants).

* ``online_tune``: the same strategy run ONLINE, inside one replay, as the paper's proxy does
  (Section 4): the weights in force change every `hop` requests.  Step k (k = 1, 2, ...) takes
  place when 128 + (k-1)*32 requests have been routed (so the 18th step comes after 672 samples,
  as the paper counts); its value is the p95 TTFT of the last `window` requests.  Step 1 scores
  the start weights; every later step scores the offspring that was in force during the last hop
  (the window still holds requests routed under earlier weights: that is what a rolling window
  does), keeps it iff it is strictly better than the parent's value, adapts sigma and puts a
  new offspring of the parent in force for the next hop.

Pinned by tests/test_oracle_tuning_pins.py (the paper's own arithmetic 128 + 17*32 = 672 samples
at the 18th step, sorted and constant inputs, numpy's inverted-CDF percentile per window, the
stationarity of sigma at one success in five, clamp bounds, a convex toy objective).
"""
from __future__ import annotations

import math
from typing import Callable, List, Sequence, Tuple


def window_count(n: int, window: int = 128, hop: int = 32) -> int:
    return (n - window) // hop + 1 if n >= window else 0


def window_p95(values: Sequence[float], window: int = 128, hop: int = 32) -> List[float]:
    k = (95 * window + 99) // 100
    out = []
    for j in range(window_count(len(values), window, hop)):
        w = sorted(values[j * hop: j * hop + window])
        out.append(w[k - 1])
    return out


def best_window(values: Sequence[float], window: int = 128, hop: int = 32) -> Tuple[float, int]:
    """Smallest window value and the first window that attains it."""
    w = window_p95(values, window, hop)
    best = min(w)
    return best, w.index(best)


def mutate(x: Sequence[float], sigma: float, z: Sequence[float], lo: Sequence[float],
           hi: Sequence[float]) -> List[float]:
    out = []
    for xk, zk, lk, hk in zip(x, z, lo, hi):
        step = sigma * zk
        v = math.exp(math.log(xk) + step)
        out.append(min(max(v, lk), hk))
    return out


def es_run(objective: Callable[[List[float]], float], x0: Sequence[float], tuned: Sequence[int],
           lo: Sequence[float], hi: Sequence[float], sigma0: float, sigma_up: float,
           z: Sequence[Sequence[Sequence[float]]]):
    """z[t][l][k]: normal draw of step t, offspring l, tuned parameter k.  ``objective`` maps a
    full parameter vector to the value to minimise.  Returns (x, f, sigma, history) with
    history[t] = (best offspring objective, accepted, sigma after, parent objective after,
    parent tuned values after)."""
    parent = list(x0)
    f_parent = objective(parent)
    sigma = sigma0
    down = sigma_up ** -0.25
    history = []
    for zt in z:
        offspring = []
        for zl in zt:
            child = list(parent)
            for idx, v in zip(tuned, mutate([parent[i] for i in tuned], sigma, zl, lo, hi)):
                child[idx] = v
            offspring.append(child)
        f = [objective(c) for c in offspring]
        best = min(range(len(f)), key=lambda l: (f[l], l))
        accept = f[best] < f_parent
        if accept:
            parent, f_parent = offspring[best], f[best]
            sigma = sigma * sigma_up
        else:
            sigma = sigma * down
        history.append((f[best], accept, sigma, f_parent, [parent[i] for i in tuned]))
    return parent, f_parent, sigma, history


def online_tune(run_chunk: Callable[[List[float], int], Sequence[float]], n_requests: int,
                x0: Sequence[float], tuned: Sequence[int], lo: Sequence[float], hi: Sequence[float],
                sigma0: float, sigma_up: float, z: Sequence[Sequence[float]], window: int = 128,
                hop: int = 32):
    """Online (1+1)-ES over one replay.  ``run_chunk(weights, count)`` routes the next ``count``
    requests of the trace with the full parameter vector ``weights`` on one persistent simulator
    state and returns their TTFTs.  ``z[k-1]`` holds the normal draws of step k (one per tuned
    parameter); the replay ends with the trace, steps that have no draws left keep the weights
    in force.  Returns (ttft of every request, schedule, history): schedule[h] = the full
    weights in force for chunk h (chunk 0 = the first `window` requests, then one per hop),
    history[k-1] = (window value, accepted, sigma after, parent value after, parent tuned values
    after, tuned values put in force for the next hop)."""
    parent = list(x0)
    live = list(x0)
    f_parent = None
    sigma = sigma0
    down = sigma_up ** -0.25
    kth = (95 * window + 99) // 100
    ttft: List[float] = []
    schedule, history = [], []
    step = 0
    while len(ttft) < n_requests:
        count = min(window if not ttft else hop, n_requests - len(ttft))
        schedule.append(list(live))
        ttft.extend(run_chunk(list(live), count))
        if len(ttft) < window or (len(ttft) - window) % hop != 0:
            continue                                   # no full window ends here (short last chunk)
        if step >= len(z):
            continue                                   # out of draws: keep the weights in force
        value = sorted(ttft[len(ttft) - window:])[kth - 1]
        if step == 0:
            f_parent, accept = value, False            # the start weights themselves
        else:
            accept = value < f_parent
            if accept:
                parent, f_parent = list(live), value
                sigma = sigma * sigma_up
            else:
                sigma = sigma * down
        live = list(parent)
        for idx, v in zip(tuned, mutate([parent[i] for i in tuned], sigma, z[step], lo, hi)):
            live[idx] = v
        history.append((value, accept, sigma, f_parent, [parent[i] for i in tuned],
                        [live[i] for i in tuned]))
        step += 1
    return ttft, schedule, history
