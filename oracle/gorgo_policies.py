"""TEST INFRASTRUCTURE ONLY -- the baseline routing policies of the paper (Section 4, "Baseline
policies"; `random` appears in its appendix tables) stated on top of the CPU replay oracle.
Nothing in the product path may import this file.

Readings (the paper runs these against live engines; here they run inside the same simulator):
  least-load        minimise the in-flight input tokens the proxy has recorded
                    (the engine-side metrics of the paper's sum do not exist in the simulator):
                    the cost model with weights (0, 0, 1);
  least-request     minimise the in-flight REQUESTS: weights (0, 0, 1) on a request count;
  prefix-cache      maximise the cached prefix: weights (0, 1, 0) (fewest uncached tokens);
  session-affinity  the paper hashes the first 256 tokens; a request's first block id stands for
                    them: replica = splitmix64_finaliser(first id) mod R, replica 0 without blocks;
  random            replica = draw mod R with one caller-supplied 32-bit draw per request.
Ties go to the lowest replica index, as everywhere.
"""
from __future__ import annotations

import numpy as np

from oracle import gorgo_oracle as O

M64 = (1 << 64) - 1


def mix64(z: int) -> int:
    z &= M64
    z ^= z >> 30
    z = (z * 0xbf58476d1ce4e5b9) & M64
    z ^= z >> 27
    z = (z * 0x94d049bb133111eb) & M64
    z ^= z >> 31
    return z


def affinity_routes(workload) -> np.ndarray:
    R = workload.spec.n_replicas
    out = np.zeros(workload.n_requests, dtype=np.uint8)
    for r in range(workload.n_requests):
        a, b = int(workload.hash_off[r]), int(workload.hash_off[r + 1])
        out[r] = mix64(int(workload.hash_ids[a])) % R if b > a else 0
    return out


def random_routes(workload, draws) -> np.ndarray:
    R = workload.spec.n_replicas
    return np.array([int(d) % R for d in draws], dtype=np.uint8)


def replay_policy(workload, policy: str, scale: float = 1.0, draws=None):
    """(RunResult, p95_ttft, p95_e2e, digest, stats) of one replay under a baseline policy."""
    K = workload.n_params
    w = np.zeros(K)
    w[3:] = 1.0
    if policy == "least-load":
        w[2] = 1.0
        return O.replay(workload, w, scale)
    if policy == "least-request":
        w[2] = 1.0
        return O.replay(workload, w, scale, queue_in_requests=True)
    if policy == "prefix-cache":
        w[1] = 1.0
        return O.replay(workload, w, scale)
    if policy == "session-affinity":
        return O.replay(workload, w, scale, forced_route=affinity_routes(workload))
    if policy == "random":
        return O.replay(workload, w, scale, forced_route=random_routes(workload, draws))
    raise ValueError(policy)
