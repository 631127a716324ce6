"""ctypes loader and thin convenience wrapper for ``gorgo_oracle.cpp``.

TEST INFRASTRUCTURE ONLY (see the header of ``gorgo_oracle.cpp``).  The wrapper only
marshals arrays; every step of the simulation runs in the C++ file.  ctypes releases the
GIL during the call, so independent ``Oracle`` objects may run on Python threads.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gorgo_oracle.cpp")
_LIB = os.path.join(_HERE, "libgorgo_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (g++, strict IEEE: no FMA contraction) if it is out of date."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-shared",
                               "-fPIC", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


class _Config(C.Structure):
    _fields_ = [("n_replicas", C.c_uint32), ("n_regions", C.c_uint32),
                ("slots_per_replica", C.c_uint32), ("block_tokens", C.c_uint32),
                ("cache_blocks", C.c_uint64), ("n_params", C.c_uint32), ("_pad", C.c_uint32),
                ("prefill_ms_per_token", C.c_double), ("tpot_ms", C.c_double)]


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        vp, u64, dbl = C.c_void_p, C.c_uint64, C.c_double
        lib.gorgo_oracle_create.restype = vp
        lib.gorgo_oracle_create.argtypes = [C.POINTER(_Config), vp, u64, vp, vp, vp, vp, vp, vp]
        lib.gorgo_oracle_destroy.argtypes = [vp]
        lib.gorgo_oracle_reset.argtypes = [vp]
        lib.gorgo_oracle_run.restype = u64
        lib.gorgo_oracle_run.argtypes = [vp, vp, dbl, u64] + [vp] * 9
        lib.gorgo_oracle_p95.restype = dbl
        lib.gorgo_oracle_p95.argtypes = [vp, u64]
        lib.gorgo_oracle_digest.argtypes = [vp, vp]
        lib.gorgo_oracle_dump.restype = u64
        lib.gorgo_oracle_dump.argtypes = [vp, C.c_uint32, u64, vp, vp, vp]
        lib.gorgo_oracle_queues.argtypes = [vp, vp, vp, vp]
        lib.gorgo_oracle_stats.argtypes = [vp, vp]
        lib.gorgo_oracle_set_policy.restype = C.c_int
        lib.gorgo_oracle_set_policy.argtypes = [vp, C.c_uint32, vp]
        lib.gorgo_oracle_set_replica_speeds.restype = C.c_int
        lib.gorgo_oracle_set_replica_speeds.argtypes = [vp, vp, vp]
        lib.gorgo_oracle_set_proxy_index.restype = None
        lib.gorgo_oracle_set_proxy_index.argtypes = [vp, C.c_uint32]
        lib.gorgo_oracle_set_rtt_series.restype = C.c_int
        lib.gorgo_oracle_set_rtt_series.argtypes = [vp, C.c_uint32, C.c_double, C.c_double, vp]
        lib.gorgo_oracle_set_service_model.restype = C.c_int
        lib.gorgo_oracle_set_service_model.argtypes = [vp, C.c_double, C.c_uint64]
        lib.gorgo_oracle_position.restype = u64
        lib.gorgo_oracle_position.argtypes = [vp]
        _lib = lib
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def p95(values: np.ndarray) -> float:
    v = np.ascontiguousarray(values, dtype=np.float64)
    return float(_load().gorgo_oracle_p95(_ptr(v), v.shape[0]))


@dataclass
class RunResult:
    route: np.ndarray
    hit: np.ndarray
    ttft: np.ndarray
    e2e: np.ndarray
    hit_all: Optional[np.ndarray] = None
    load_all: Optional[np.ndarray] = None
    cost_all: Optional[np.ndarray] = None
    evicted: Optional[np.ndarray] = None
    occ_after: Optional[np.ndarray] = None


class Oracle:
    """One simulator instance (one candidate's state) over one trace."""

    def __init__(self, *, n_replicas, n_regions, slots_per_replica, block_tokens, cache_blocks,
                 n_params, prefill_ms_per_token, tpot_ms, rtt_ms, ts_ms, input_tokens,
                 output_tokens, origin, hash_off, hash_ids):
        lib = _load()
        self._lib = lib
        self.R, self.S, self.K = int(n_replicas), int(slots_per_replica), int(n_params)
        cfg = _Config(n_replicas, n_regions, slots_per_replica, block_tokens, cache_blocks,
                      n_params, 0, prefill_ms_per_token, tpot_ms)
        rtt = np.ascontiguousarray(rtt_ms, dtype=np.float64)
        ts = np.ascontiguousarray(ts_ms, dtype=np.float64)
        it = np.ascontiguousarray(input_tokens, dtype=np.uint32)
        ot = np.ascontiguousarray(output_tokens, dtype=np.uint32)
        org = None if origin is None else np.ascontiguousarray(origin, dtype=np.uint16)
        off = np.ascontiguousarray(hash_off, dtype=np.uint64)
        ids = np.ascontiguousarray(hash_ids, dtype=np.uint64)
        self.N = int(ts.shape[0])
        self._h = lib.gorgo_oracle_create(C.byref(cfg), _ptr(rtt), self.N, _ptr(ts), _ptr(it),
                                          _ptr(ot), _ptr(org), _ptr(off), _ptr(ids))
        if not self._h:
            raise ValueError("oracle rejected the configuration")

    @classmethod
    def from_workload(cls, w) -> "Oracle":
        return cls(rtt_ms=w.rtt_ms, ts_ms=w.ts_ms, input_tokens=w.input_tokens,
                   output_tokens=w.output_tokens, origin=w.origin, hash_off=w.hash_off,
                   hash_ids=w.hash_ids, **w.config_dict())

    def close(self):
        if getattr(self, "_h", None):
            self._lib.gorgo_oracle_destroy(self._h)
            self._h = None

    __del__ = close

    def reset(self):
        self._lib.gorgo_oracle_reset(self._h)

    def set_policy(self, queue_in_requests: bool = False, forced_route=None):
        """Baseline policies of Section 4: queue signal in requests instead of tokens, and/or one
        fixed replica per request (None: route by the score)."""
        fr = None if forced_route is None else np.ascontiguousarray(forced_route, dtype=np.uint8)
        assert fr is None or fr.shape == (self.N,)
        rc = self._lib.gorgo_oracle_set_policy(self._h, int(bool(queue_in_requests)), _ptr(fr))
        if rc != 0:
            raise ValueError("forced route out of range")

    def set_replica_speeds(self, prefill_ms_per_token=None, tpot_ms=None):
        """Heterogeneous replicas: per-replica prefill time per token and time per output token
        (None: the uniform constant)."""
        a = None if prefill_ms_per_token is None else np.ascontiguousarray(prefill_ms_per_token, np.float64)
        b = None if tpot_ms is None else np.ascontiguousarray(tpot_ms, np.float64)
        assert (a is None or a.shape == (self.R,)) and (b is None or b.shape == (self.R,))
        if self._lib.gorgo_oracle_set_replica_speeds(self._h, _ptr(a), _ptr(b)) != 0:
            raise ValueError("replica speeds must be finite and >= 0")

    def set_proxy_index(self, on: bool = True):
        """Score with the proxy's own index (every block ever dispatched to a replica) instead of
        the replica's real cache; set it on the empty state."""
        self._lib.gorgo_oracle_set_proxy_index(self._h, int(bool(on)))

    def set_rtt_series(self, samples=None, epoch_ms: float = 30_000.0, alpha: float = 0.3):
        """Time-varying network: samples[e, g, i] = RTT probe of epoch e (also the delay of requests
        dispatched in it); the score uses their EWMA.  None restores the static matrix."""
        if samples is None:
            self._lib.gorgo_oracle_set_rtt_series(self._h, 0, 0.0, 0.0, None)
            return
        s = np.ascontiguousarray(samples, dtype=np.float64)
        assert s.ndim == 3 and s.shape[2] == self.R
        if self._lib.gorgo_oracle_set_rtt_series(self._h, s.shape[0], float(epoch_ms), float(alpha),
                                                 _ptr(s)) != 0:
            raise ValueError("bad RTT series")

    def set_service_model(self, decode_slowdown: float = 0.0, kv_budget_tokens: int = 0):
        """Decode slow-down per additional busy slot and KV budget per replica in tokens
        (0 = unlimited); both off by default."""
        if self._lib.gorgo_oracle_set_service_model(self._h, float(decode_slowdown),
                                                    int(kv_budget_tokens)) != 0:
            raise ValueError("decode slow-down must be finite and >= 0")

    @property
    def position(self) -> int:
        return int(self._lib.gorgo_oracle_position(self._h))

    def run(self, w, scale: float = 1.0, count: Optional[int] = None,
            detail: bool = False) -> RunResult:
        w = np.ascontiguousarray(w, dtype=np.float64)
        assert w.shape == (self.K,)
        n = self.N - self.position if count is None else min(int(count), self.N - self.position)
        res = RunResult(route=np.zeros(n, np.uint8), hit=np.zeros(n, np.uint16),
                        ttft=np.zeros(n, np.float64), e2e=np.zeros(n, np.float64))
        if detail:
            res.hit_all = np.zeros((n, self.R), np.uint16)
            res.load_all = np.zeros((n, self.R), np.int64)
            res.cost_all = np.zeros((n, self.R), np.float64)
            res.evicted = np.zeros(n, np.uint32)
            res.occ_after = np.zeros(n, np.uint64)
        done = self._lib.gorgo_oracle_run(
            self._h, _ptr(w), float(scale), n, _ptr(res.route), _ptr(res.hit), _ptr(res.ttft),
            _ptr(res.e2e), _ptr(res.hit_all), _ptr(res.load_all), _ptr(res.cost_all),
            _ptr(res.evicted), _ptr(res.occ_after))
        assert done == n
        return res

    def digest(self) -> np.ndarray:
        out = np.zeros((self.R, 2), np.uint64)
        self._lib.gorgo_oracle_digest(self._h, _ptr(out))
        return out

    def dump(self, replica: int):
        n = int(self._lib.gorgo_oracle_dump(self._h, replica, 0, None, None, None))
        ids, seq, pos = np.zeros(n, np.uint64), np.zeros(n, np.uint64), np.zeros(n, np.uint32)
        self._lib.gorgo_oracle_dump(self._h, replica, n, _ptr(ids), _ptr(seq), _ptr(pos))
        return ids, seq, pos

    def queues(self):
        loads = np.zeros(self.R, np.int64)
        infl = np.zeros(self.R, np.uint64)
        free_at = np.zeros((self.R, self.S), np.float64)
        self._lib.gorgo_oracle_queues(self._h, _ptr(loads), _ptr(infl), _ptr(free_at))
        return loads, infl, free_at

    def stats(self) -> np.ndarray:
        out = np.zeros(4, np.uint64)
        self._lib.gorgo_oracle_stats(self._h, _ptr(out))
        return out


def replay(workload, w, scale: float = 1.0, detail: bool = False, queue_in_requests: bool = False,
           forced_route=None, rep_prefill_ms=None, rep_tpot_ms=None, decode_slowdown: float = 0.0,
           kv_budget_tokens: int = 0, rtt_series=None, epoch_ms: float = 30_000.0, alpha: float = 0.3,
           proxy_index: bool = False):
    """Full replay of one candidate from the empty state: (RunResult, p95_ttft, p95_e2e,
    digest[R,2], stats[4])."""
    o = Oracle.from_workload(workload)
    try:
        if queue_in_requests or forced_route is not None:
            o.set_policy(queue_in_requests, forced_route)
        if rep_prefill_ms is not None or rep_tpot_ms is not None:
            o.set_replica_speeds(rep_prefill_ms, rep_tpot_ms)
        if decode_slowdown or kv_budget_tokens:
            o.set_service_model(decode_slowdown, kv_budget_tokens)
        if rtt_series is not None:
            o.set_rtt_series(rtt_series, epoch_ms, alpha)
        if proxy_index:
            o.set_proxy_index(True)
        res = o.run(w, scale, detail=detail)
        return res, p95(res.ttft), p95(res.e2e), o.digest(), o.stats()
    finally:
        o.close()
