"""Seeded synthetic request traces and cost-model populations.

This module only *produces inputs*: Mooncake-style traces (per-request timestamp,
input/output token counts and the 512-token-block ``hash_ids`` of the prompt), a
replica RTT matrix and a population of cost-model parameter vectors.  It holds none
of the routing/caching/queueing arithmetic; both the CUDA library and the CPU
reference consume what it emits.

The traces stand in for the paper's ART-Chat-2.5M trace (Section 3, Table 1 and
Appendix A): long prompts, multi-turn sessions in which every later turn re-sends
the previous prompt as a prefix, and reuse that is almost entirely intra-session.
No item of any public dataset is reproduced; everything is drawn from
``numpy.random.default_rng(seed)``.

Shape of one session: arrivals form a Poisson process, every arrival picks a session
uniformly at random, the session continues its current conversation with probability
``1 - 1/mean_turns`` (geometric number of turns) and otherwise opens a new one.  The
prompt of turn t>1 is the previous prompt plus the previous answer plus new user
tokens, so its block list is the *full* blocks of the previous prompt followed by
fresh block ids (a previously partial last block gets a fresh id, as a real prefix
hash would).  Block ids are a bijective 64-bit mix of a global counter, so an id
never repeats outside its own conversation prefix.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, Optional, Sequence

import numpy as np

BLOCK_TOKENS = 512

_U64 = np.uint64


def _mix64(x: np.ndarray) -> np.ndarray:
    """Bijective 64-bit scrambler used only to make block ids look like hashes."""
    x = x.astype(np.uint64, copy=True)
    with np.errstate(over="ignore"):
        x ^= x >> _U64(33)
        x *= _U64(0xFF51AFD7ED558CCD)
        x ^= x >> _U64(33)
        x *= _U64(0xC4CEB9FE1A85EC53)
        x ^= x >> _U64(33)
    return x


@dataclass
class WorkloadSpec:
    """Recipe of one configuration (all quantities are inputs of the simulator)."""

    name: str
    seed: int
    n_replicas: int
    n_regions: int
    n_requests: int
    n_sessions: int
    cache_blocks: int
    slots: int
    population: int
    per_replica_normaliser: bool = False     # K = 3 + R instead of 3
    rtt: str = "uniform"                      # "uniform" | "regions" | "loguniform"
    first_prompt_median: float = 1000.0       # tokens, lognormal
    first_prompt_sigma: float = 1.0
    new_tokens_median: float = 1000.0         # per later turn, lognormal
    new_tokens_sigma: float = 1.0
    output_median: float = 300.0
    output_sigma: float = 0.7
    max_prompt_tokens: int = 128_000          # 250 blocks
    mean_turns: float = 5.0
    min_reuse_num: int = 0                    # later turns keep >= num/den of their blocks
    min_reuse_den: int = 1                    #   as a prior-turn prefix (0 => no constraint)
    shared_prefix_fraction: float = 0.0       # sessions whose conversations start with
    shared_prefix_blocks: int = 0             #   one common system-prompt prefix
    arrival_rate_per_s: Optional[float] = None  # fixed Poisson rate, else from utilisation
    utilisation: float = 0.7                  # nominal rho used when no fixed rate is given
    time_scales: Sequence[float] = (1.0,)
    prefill_ms_per_token: float = 0.05
    tpot_ms: float = 20.0
    block_tokens: int = BLOCK_TOKENS


SPECS: Dict[str, WorkloadSpec] = {
    # 4 replicas, 2,000 requests from 200 sessions, 5 req/s, population 8
    "tiny": WorkloadSpec(
        name="tiny", seed=0, n_replicas=4, n_regions=1, n_requests=2_000, n_sessions=200,
        cache_blocks=2_000, slots=4, population=8, rtt="uniform", arrival_rate_per_s=5.0),
    # 8 replicas in 4 regions, shared 4-block system prompt in 20 % of the sessions
    "regions": WorkloadSpec(
        name="regions", seed=1, n_replicas=8, n_regions=4, n_requests=50_000,
        n_sessions=5_000, cache_blocks=20_000, slots=16, population=64, rtt="regions",
        shared_prefix_fraction=0.2, shared_prefix_blocks=4, utilisation=0.7),
    # long-context, high reuse: 16 replicas, 500,000 requests, timestamps x0.5
    "longctx": WorkloadSpec(
        name="longctx", seed=2, n_replicas=16, n_regions=1, n_requests=500_000,
        n_sessions=50_000, cache_blocks=100_000, slots=16, population=256,
        rtt="loguniform", first_prompt_median=20_000.0, first_prompt_sigma=0.8,
        min_reuse_num=4, min_reuse_den=5, utilisation=0.6, time_scales=(0.5,)),
    # saturation sweep: 32 replicas, 1,000,000 requests, five timestamp scale factors
    "sweep": WorkloadSpec(
        name="sweep", seed=3, n_replicas=32, n_regions=1, n_requests=1_000_000,
        n_sessions=100_000, cache_blocks=100_000, slots=32, population=512,
        rtt="loguniform", first_prompt_median=20_000.0, first_prompt_sigma=0.8,
        min_reuse_num=4, min_reuse_den=5, utilisation=0.6,
        time_scales=(1.0, 0.75, 0.5, 0.35, 0.25)),
    # largest: 64 replicas, 2,500,000 requests, per-replica queue-load normalisers
    "largest": WorkloadSpec(
        name="largest", seed=4, n_replicas=64, n_regions=1, n_requests=2_500_000,
        n_sessions=250_000, cache_blocks=200_000, slots=64, population=1_024,
        per_replica_normaliser=True, rtt="loguniform", first_prompt_median=20_000.0,
        first_prompt_sigma=0.8, min_reuse_num=4, min_reuse_den=5, utilisation=0.6,
        time_scales=(0.5,)),
}


@dataclass
class Workload:
    """One generated instance: simulator configuration, trace, RTT matrix, population."""

    spec: WorkloadSpec
    rtt_ms: np.ndarray          # f64 [G, R]
    ts_ms: np.ndarray           # f64 [N], non-decreasing
    input_tokens: np.ndarray    # u32 [N]
    output_tokens: np.ndarray   # u32 [N]
    origin: np.ndarray          # u16 [N], region of the proxy that saw the request
    hash_off: np.ndarray        # u64 [N+1], CSR offsets into hash_ids
    hash_ids: np.ndarray        # u64 [sum n_blocks]
    params: np.ndarray          # f64 [P, K]
    session: np.ndarray         # u32 [N]  (generator-side bookkeeping only)
    turn: np.ndarray            # u32 [N]  turn index inside its conversation (0 = first)
    info: Dict[str, float] = field(default_factory=dict)

    @property
    def n_requests(self) -> int:
        return int(self.ts_ms.shape[0])

    @property
    def n_params(self) -> int:
        return int(self.params.shape[1])

    def config_dict(self) -> Dict[str, object]:
        s = self.spec
        return dict(n_replicas=s.n_replicas, n_regions=s.n_regions,
                    slots_per_replica=s.slots, block_tokens=s.block_tokens,
                    cache_blocks=s.cache_blocks, n_params=self.n_params,
                    prefill_ms_per_token=s.prefill_ms_per_token, tpot_ms=s.tpot_ms)


def _lognormal(rng: np.random.Generator, median: float, sigma: float, n: int) -> np.ndarray:
    return rng.lognormal(mean=math.log(median), sigma=sigma, size=n)


def make_rtt(spec: WorkloadSpec, rng: np.random.Generator) -> np.ndarray:
    R, G = spec.n_replicas, spec.n_regions
    if spec.rtt == "uniform":            # 10-300 ms
        return rng.uniform(10.0, 300.0, size=(G, R))
    if spec.rtt == "loguniform":         # 10 ms - 1 s
        return np.exp(rng.uniform(math.log(10.0), math.log(1000.0), size=(G, R)))
    if spec.rtt == "regions":            # 10 ms inside a region, 80-400 ms across
        pair = rng.uniform(80.0, 400.0, size=(G, G))
        pair = np.triu(pair, 1)
        pair = pair + pair.T
        region_of = (np.arange(R) * G) // R
        out = np.empty((G, R), dtype=np.float64)
        for g in range(G):
            for i in range(R):
                out[g, i] = 10.0 if region_of[i] == g else pair[g, region_of[i]]
        return out
    raise ValueError(f"unknown rtt recipe {spec.rtt!r}")


def make_params(spec: WorkloadSpec, rng: np.random.Generator) -> np.ndarray:
    P, R = spec.population, spec.n_replicas
    w = rng.normal(1.0, 0.3, size=(P, 3))
    if spec.per_replica_normaliser:
        s = rng.lognormal(mean=0.0, sigma=0.3, size=(P, R))
        w = np.concatenate([w, s], axis=1)
    return np.ascontiguousarray(w, dtype=np.float64)


def make_workload(name: str, *, n_requests: Optional[int] = None,
                  n_sessions: Optional[int] = None, cache_blocks: Optional[int] = None,
                  population: Optional[int] = None, seed: Optional[int] = None,
                  max_prompt_tokens: Optional[int] = None) -> Workload:
    """Generate configuration ``name``; the keyword overrides give reduced-size variants
    of the same recipe (fewer requests/sessions, smaller caches) for quick parity cases."""
    base = SPECS[name]
    spec = WorkloadSpec(**{**base.__dict__})
    if n_requests is not None:
        spec.n_requests = int(n_requests)
        spec.n_sessions = max(1, int(n_requests) // 10) if n_sessions is None else int(n_sessions)
    elif n_sessions is not None:
        spec.n_sessions = int(n_sessions)
    if cache_blocks is not None:
        spec.cache_blocks = int(cache_blocks)
    if population is not None:
        spec.population = int(population)
    if seed is not None:
        spec.seed = int(seed)
    if max_prompt_tokens is not None:
        spec.max_prompt_tokens = int(max_prompt_tokens)

    rng = np.random.default_rng(spec.seed)
    N, B, cap = spec.n_requests, spec.block_tokens, spec.max_prompt_tokens
    rtt = make_rtt(spec, rng)
    params = make_params(spec, rng)

    sess = rng.integers(0, spec.n_sessions, size=N)
    u_cont = rng.random(N)
    first_len = np.clip(np.rint(_lognormal(rng, spec.first_prompt_median,
                                           spec.first_prompt_sigma, N)), 1, cap).astype(np.int64)
    new_tok = np.clip(np.rint(_lognormal(rng, spec.new_tokens_median,
                                         spec.new_tokens_sigma, N)), 1, cap).astype(np.int64)
    out_tok = np.clip(np.rint(_lognormal(rng, spec.output_median, spec.output_sigma, N)),
                      1, 4096).astype(np.int64)
    sess_region = rng.integers(0, spec.n_regions, size=spec.n_sessions)
    sess_shared = rng.random(spec.n_sessions) < spec.shared_prefix_fraction
    gaps = rng.exponential(1.0, size=N)

    p_new = 1.0 / spec.mean_turns
    nshared = spec.shared_prefix_blocks
    shared_ids = np.arange(nshared, dtype=np.int64)
    ctr = nshared                      # next fresh block counter
    cur_len = [0] * spec.n_sessions
    cur_out = [0] * spec.n_sessions
    cur_turn = [0] * spec.n_sessions
    cur_ids = [None] * spec.n_sessions

    in_tok = np.empty(N, dtype=np.int64)
    turn = np.empty(N, dtype=np.uint32)
    nblk = np.empty(N, dtype=np.int64)
    chunks = []
    sess_l = sess.tolist()
    u_l = u_cont.tolist()
    first_l = first_len.tolist()
    new_l = new_tok.tolist()
    out_l = out_tok.tolist()
    shared_l = sess_shared.tolist()
    rnum, rden = spec.min_reuse_num, spec.min_reuse_den

    for r in range(N):
        s = sess_l[r]
        lp = cur_len[s]
        cont = lp > 0 and lp < cap and u_l[r] >= p_new
        if cont:
            L = lp + cur_out[s] + new_l[r]
            f = lp // B
            if rnum > 0:
                lmax = ((f * rden) // rnum) * B
                if lmax <= lp:
                    cont = False          # reuse floor cannot hold -> open a new conversation
                elif L > lmax:
                    L = lmax
        if cont:
            if L > cap:
                L = cap
            n = -(-L // B)
            k = n - f
            ids = np.concatenate([cur_ids[s][:f], np.arange(ctr, ctr + k, dtype=np.int64)])
            ctr += k
            cur_turn[s] += 1
        else:
            L = first_l[r]
            if shared_l[s]:
                L = min(cap, L + nshared * B)
                n = -(-L // B)
                ids = np.concatenate([shared_ids, np.arange(ctr, ctr + n - nshared, dtype=np.int64)])
                ctr += n - nshared
            else:
                n = -(-L // B)
                ids = np.arange(ctr, ctr + n, dtype=np.int64)
                ctr += n
            cur_turn[s] = 0
        cur_len[s] = L
        cur_out[s] = out_l[r]
        cur_ids[s] = ids
        in_tok[r] = L
        nblk[r] = n
        turn[r] = cur_turn[s]
        chunks.append(ids)

    hash_off = np.zeros(N + 1, dtype=np.uint64)
    np.cumsum(nblk, out=hash_off[1:].view(np.int64))
    flat = np.concatenate(chunks) if chunks else np.zeros(0, dtype=np.int64)
    salt = _U64((0x9E3779B97F4A7C15 * (spec.seed + 1)) & 0xFFFFFFFFFFFFFFFF)
    hash_ids = _mix64(flat.astype(np.uint64) ^ salt)

    # arrival rate: fixed, or from the nominal utilisation rho = lambda * E[service] / (R*S)
    if spec.arrival_rate_per_s is not None:
        lam_per_ms = spec.arrival_rate_per_s / 1000.0
    else:
        mean_service = float(np.mean(spec.prefill_ms_per_token * 0.2 * in_tok
                                     + spec.tpot_ms * (out_tok - 1)))
        lam_per_ms = spec.utilisation * spec.n_replicas * spec.slots / mean_service
    ts = np.cumsum(gaps / lam_per_ms)

    total_blocks = int(hash_off[-1])
    distinct = int(ctr)
    info = dict(total_blocks=total_blocks, distinct_blocks=distinct,
                block_reuse=1.0 - distinct / max(1, total_blocks),
                mean_blocks=total_blocks / max(1, N),
                mean_input_tokens=float(np.mean(in_tok)) if N else 0.0,
                multi_turn_fraction=float(np.mean(turn > 0)) if N else 0.0,
                arrival_rate_per_s=lam_per_ms * 1000.0)

    return Workload(
        spec=spec, rtt_ms=np.ascontiguousarray(rtt, dtype=np.float64),
        ts_ms=np.ascontiguousarray(ts, dtype=np.float64),
        input_tokens=in_tok.astype(np.uint32), output_tokens=out_tok.astype(np.uint32),
        origin=sess_region[sess].astype(np.uint16), hash_off=hash_off, hash_ids=hash_ids,
        params=params, session=sess.astype(np.uint32), turn=turn, info=info)


def handmade(rtt_ms, requests, *, slots=1, cache_blocks=4, block_tokens=BLOCK_TOKENS,
             prefill_ms_per_token=0.05, tpot_ms=20.0, params=((1.0, 1.0, 1.0),),
             n_regions=1, origin=None, name="handmade") -> Workload:
    """Wrap a hand-written trace: ``requests`` is a list of (t_ms, input_tokens,
    output_tokens, [block ids])."""
    rtt = np.asarray(rtt_ms, dtype=np.float64).reshape(n_regions, -1)
    N = len(requests)
    ts = np.array([q[0] for q in requests], dtype=np.float64)
    it = np.array([q[1] for q in requests], dtype=np.uint32)
    ot = np.array([q[2] for q in requests], dtype=np.uint32)
    off = np.zeros(N + 1, dtype=np.uint64)
    for i, q in enumerate(requests):
        off[i + 1] = off[i] + np.uint64(len(q[3]))
    ids = np.array([b for q in requests for b in q[3]], dtype=np.uint64)
    par = np.ascontiguousarray(np.asarray(params, dtype=np.float64).reshape(len(params), -1))
    spec = WorkloadSpec(name=name, seed=0, n_replicas=rtt.shape[1], n_regions=n_regions,
                        n_requests=N, n_sessions=1, cache_blocks=cache_blocks, slots=slots,
                        population=par.shape[0], block_tokens=block_tokens,
                        per_replica_normaliser=par.shape[1] != 3,
                        prefill_ms_per_token=prefill_ms_per_token, tpot_ms=tpot_ms)
    org = np.zeros(N, dtype=np.uint16) if origin is None else np.asarray(origin, dtype=np.uint16)
    return Workload(spec=spec, rtt_ms=rtt, ts_ms=ts, input_tokens=it, output_tokens=ot,
                    origin=org, hash_off=off, hash_ids=ids, params=par,
                    session=np.zeros(N, dtype=np.uint32), turn=np.zeros(N, dtype=np.uint32))
