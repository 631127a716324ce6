"""ctypes binding of ``libgorgo_b200.so``: the functions of ``include/gorgo.h`` under the same
names (argument marshalling only), plus ``GorgoSim``, a small holder of the torch tensors that
serve as device buffers.  Every step of the simulation runs in the CUDA library; if the library
is missing this module raises instead of computing anything on the CPU.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgorgo_b200.so")

GORGO_OK = 0
GORGO_ERR_INVALID_ARG = -1
GORGO_ERR_BAD_TRACE = -2
GORGO_ERR_NONFINITE_PARAM = -3
GORGO_ERR_WORKSPACE_TOO_SMALL = -4
GORGO_ERR_CUDA = -5
GORGO_ERR_DEVICE_LIMIT = -6
GORGO_ERR_NO_TRACE = -7
GORGO_ERR_OUT_OF_ORDER = -8
GORGO_ERR_STATIC_LIMIT = -9
GORGO_STATIC_SCRATCH_BYTES = 64 << 20

EXPORTS = [
    "gorgo_sim_create", "gorgo_sim_destroy", "gorgo_trace_bytes", "gorgo_trace_upload",
    "gorgo_trace_info", "gorgo_workspace_bytes", "gorgo_eval_population",
    "gorgo_eval_population_host", "gorgo_state_bytes", "gorgo_sim_reset", "gorgo_route_batch",
    "gorgo_state_digest", "gorgo_state_status", "gorgo_set_profiling", "gorgo_last_replay_ms",
    "gorgo_eval_population_static", "gorgo_replay_occupancy", "gorgo_strerror",
    "gorgo_window_count", "gorgo_eval_population_windows", "gorgo_es_run",
    "gorgo_last_window_ms", "gorgo_eval_policy", "gorgo_eval_population_scales",
    "gorgo_sim_set_replica_speeds", "gorgo_debug_set", "gorgo_measure_gather", "gorgo_tune_online",
    "gorgo_sim_set_service_model", "gorgo_sim_set_rtt_series", "gorgo_sim_set_proxy_index",
    "gorgo_trace_begin", "gorgo_trace_append",
]
GORGO_DEBUG_POLL_LIMIT, GORGO_DEBUG_RING_POLLS, GORGO_DEBUG_PROBE_OFF, GORGO_DEBUG_SCOUT_OFF = 0, 1, 2, 3


class gorgo_config_t(C.Structure):
    _fields_ = [("n_replicas", C.c_uint32), ("n_regions", C.c_uint32),
                ("slots_per_replica", C.c_uint32), ("block_tokens", C.c_uint32),
                ("cache_blocks", C.c_uint64), ("n_params", C.c_uint32), ("reserved", C.c_uint32),
                ("prefill_ms_per_token", C.c_double), ("tpot_ms", C.c_double),
                ("rtt_ms", C.c_void_p), ("device", C.c_int32)]


class gorgo_es_config_t(C.Structure):
    _fields_ = [("n_steps", C.c_uint32), ("lambda_", C.c_uint32), ("n_tuned", C.c_uint32),
                ("objective", C.c_uint32), ("tuned", C.c_void_p), ("lo", C.c_void_p),
                ("hi", C.c_void_p), ("sigma0", C.c_double), ("sigma_up", C.c_double),
                ("time_scale", C.c_double)]


class gorgo_online_config_t(C.Structure):
    _fields_ = [("n_tuned", C.c_uint32), ("n_draw_steps", C.c_uint32), ("window", C.c_uint32),
                ("hop", C.c_uint32), ("tuned", C.c_void_p), ("lo", C.c_void_p), ("hi", C.c_void_p),
                ("sigma0", C.c_double), ("sigma_up", C.c_double), ("time_scale", C.c_double)]


class GorgoError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {gorgo_strerror(code)} ({code})")


_lib = None


def load():
    """Load the shared library (built by ``paper_2602_11688_b200.build``); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2602_11688_b200.build` "
                          "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, u32, u64, dbl, i32 = C.c_void_p, C.c_uint32, C.c_uint64, C.c_double, C.c_int
    pu64 = C.POINTER(C.c_uint64)
    sig = {
        "gorgo_sim_create": [C.POINTER(gorgo_config_t), C.POINTER(vp)],
        "gorgo_sim_destroy": [vp],
        "gorgo_trace_bytes": [u64, u64, pu64],
        "gorgo_trace_upload": [vp, u64, vp, vp, vp, vp, vp, vp, vp, u64, vp],
        "gorgo_trace_info": [vp, pu64, pu64, pu64],
        "gorgo_workspace_bytes": [vp, u32, pu64],
        "gorgo_eval_population": [vp, u32, vp, dbl, vp, u64, vp, vp, vp, vp, vp, vp, vp, vp],
        "gorgo_eval_population_host": [vp, u32, vp, dbl, vp, u64, vp, vp, vp],
        "gorgo_state_bytes": [vp, pu64],
        "gorgo_sim_reset": [vp, vp, u64, vp],
        "gorgo_route_batch": [vp, vp, dbl, u64, u64, vp, u64, vp, vp, vp, vp, vp],
        "gorgo_state_digest": [vp, vp, u64, vp, vp],
        "gorgo_state_status": [vp, vp, u64, vp, pu64],
        "gorgo_eval_population_static": [vp, u32, vp, dbl, vp, vp, vp, vp, vp, vp],
        "gorgo_debug_set": [vp, u32, u32],
        "gorgo_sim_set_service_model": [vp, dbl, u64],
        "gorgo_sim_set_rtt_series": [vp, u32, dbl, dbl, vp],
        "gorgo_sim_set_proxy_index": [vp, i32],
        "gorgo_trace_begin": [vp, u64, u64, vp, u64],
        "gorgo_trace_append": [vp, u64, vp, vp, vp, vp, vp, vp, vp],
        "gorgo_tune_online": [vp, C.POINTER(gorgo_online_config_t), u32, vp, vp, vp, u64, vp, vp, vp,
                              C.POINTER(C.c_uint32), vp, vp, vp, vp],
        "gorgo_measure_gather": [i32, vp, u64, u64, vp, C.POINTER(C.c_double)],
        "gorgo_replay_occupancy": [vp, C.POINTER(C.c_int32), pu64],
        "gorgo_window_count": [u64, u32, u32, pu64],
        "gorgo_sim_set_replica_speeds": [vp, vp, vp],
        "gorgo_eval_population_scales": [vp, u32, vp, vp, vp, u64, vp, vp, vp, vp, vp, vp, vp],
        "gorgo_eval_policy": [vp, u32, vp, dbl, vp, u64, vp, vp, vp, vp, vp, vp, vp],
        "gorgo_eval_population_windows": [vp, u32, vp, dbl, vp, u64, vp, u32, u32, vp, vp, vp, vp,
                                          vp, vp],
        "gorgo_es_run": [vp, C.POINTER(gorgo_es_config_t), vp, vp, vp, u64, vp, vp,
                         C.POINTER(C.c_double), C.POINTER(C.c_double), vp],
        "gorgo_set_profiling": [vp, i32],
        "gorgo_last_replay_ms": [vp, C.POINTER(C.c_double), C.POINTER(C.c_uint32)],
        "gorgo_last_window_ms": [vp, C.POINTER(C.c_double), C.POINTER(C.c_uint32)],
    }
    for name, argtypes in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = argtypes
        fn.restype = i32
    lib.gorgo_strerror.argtypes = [i32]
    lib.gorgo_strerror.restype = C.c_char_p
    _lib = lib
    return lib


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dev_ptr(t) -> Optional[int]:
    """Raw device address of a torch tensor (None passes NULL)."""
    return None if t is None else int(t.data_ptr())


# ------------------------------------------------------------------ same-name entry points
def gorgo_strerror(code: int) -> str:
    return load().gorgo_strerror(int(code)).decode()


def gorgo_sim_create(*, n_replicas, n_regions, slots_per_replica, block_tokens, cache_blocks,
                     n_params, prefill_ms_per_token, tpot_ms, rtt_ms, device=0):
    """Returns (status, handle)."""
    rtt = np.ascontiguousarray(rtt_ms, dtype=np.float64)
    cfg = gorgo_config_t(int(n_replicas), int(n_regions), int(slots_per_replica),
                         int(block_tokens), int(cache_blocks), int(n_params), 0,
                         float(prefill_ms_per_token), float(tpot_ms),
                         rtt.ctypes.data, int(device))
    h = C.c_void_p()
    rc = load().gorgo_sim_create(C.byref(cfg), C.byref(h))
    return rc, h


def gorgo_sim_destroy(sim) -> int:
    return load().gorgo_sim_destroy(sim)


def gorgo_trace_bytes(n_requests: int, n_block_ids: int):
    out = C.c_uint64()
    rc = load().gorgo_trace_bytes(int(n_requests), int(n_block_ids), C.byref(out))
    return rc, out.value


def gorgo_trace_upload(sim, ts_ms, input_tokens, output_tokens, origin, hash_off, hash_ids,
                       dev_trace_buf, stream: int = 0) -> int:
    ts = np.ascontiguousarray(ts_ms, dtype=np.float64)
    it = np.ascontiguousarray(input_tokens, dtype=np.uint32)
    ot = np.ascontiguousarray(output_tokens, dtype=np.uint32)
    org = None if origin is None else np.ascontiguousarray(origin, dtype=np.uint16)
    off = np.ascontiguousarray(hash_off, dtype=np.uint64)
    ids = np.ascontiguousarray(hash_ids, dtype=np.uint64)
    return load().gorgo_trace_upload(sim, ts.shape[0], _np_ptr(ts), _np_ptr(it), _np_ptr(ot),
                                     _np_ptr(org), _np_ptr(off), _np_ptr(ids),
                                     _dev_ptr(dev_trace_buf), dev_trace_buf.numel(), stream)


def gorgo_trace_begin(sim, max_requests: int, max_block_ids: int, dev_trace_buf) -> int:
    return load().gorgo_trace_begin(sim, int(max_requests), int(max_block_ids),
                                    _dev_ptr(dev_trace_buf), dev_trace_buf.numel())


def gorgo_trace_append(sim, ts_ms, input_tokens, output_tokens, origin, hash_off, hash_ids,
                       stream: int = 0) -> int:
    """Appends requests (``hash_off`` starts at 0 for the first new one)."""
    ts = np.ascontiguousarray(ts_ms, dtype=np.float64)
    it = np.ascontiguousarray(input_tokens, dtype=np.uint32)
    ot = np.ascontiguousarray(output_tokens, dtype=np.uint32)
    org = None if origin is None else np.ascontiguousarray(origin, dtype=np.uint16)
    off = np.ascontiguousarray(hash_off, dtype=np.uint64)
    ids = np.ascontiguousarray(hash_ids, dtype=np.uint64)
    return load().gorgo_trace_append(sim, ts.shape[0], _np_ptr(ts), _np_ptr(it), _np_ptr(ot),
                                     _np_ptr(org), _np_ptr(off), _np_ptr(ids), stream)


def gorgo_trace_info(sim):
    a, b, c = C.c_uint64(), C.c_uint64(), C.c_uint64()
    rc = load().gorgo_trace_info(sim, C.byref(a), C.byref(b), C.byref(c))
    return rc, a.value, b.value, c.value


def gorgo_workspace_bytes(sim, resident_candidates: int):
    out = C.c_uint64()
    rc = load().gorgo_workspace_bytes(sim, int(resident_candidates), C.byref(out))
    return rc, out.value


def gorgo_eval_population(sim, n_candidates, params, time_scale, workspace, stream,
                          p95_ttft_ms, p95_e2e_ms, route=None, hit_blocks=None,
                          state_digest=None, stats=None, cand_status=None) -> int:
    """``params`` is a contiguous float64 numpy array (host) or torch CUDA tensor (device);
    every other array argument is a torch CUDA tensor or None."""
    pp = _np_ptr(params) if isinstance(params, np.ndarray) else _dev_ptr(params)
    return load().gorgo_eval_population(
        sim, int(n_candidates), pp, float(time_scale), _dev_ptr(workspace), workspace.numel(),
        stream, _dev_ptr(p95_ttft_ms), _dev_ptr(p95_e2e_ms), _dev_ptr(route),
        _dev_ptr(hit_blocks), _dev_ptr(state_digest), _dev_ptr(stats), _dev_ptr(cand_status))


def gorgo_eval_population_host(sim, n_candidates, params, time_scale, workspace, stream,
                               p95_ttft_ms, p95_e2e_ms) -> int:
    """``params`` / ``p95_*`` are host buffers: numpy arrays or (pinned) CPU torch tensors."""
    def host_ptr(x):
        return _np_ptr(x) if isinstance(x, np.ndarray) else int(x.data_ptr())
    return load().gorgo_eval_population_host(
        sim, int(n_candidates), host_ptr(params), float(time_scale), _dev_ptr(workspace),
        workspace.numel(), stream, host_ptr(p95_ttft_ms), host_ptr(p95_e2e_ms))


def gorgo_measure_gather(device: int, buffer, footprint_bytes: int, stream: int = 0):
    """Random 32-byte-sector read rate over the first ``footprint_bytes`` of ``buffer`` (a torch CUDA
    uint8 tensor at least 256 bytes longer).  Returns (status, GB/s of sectors)."""
    out = C.c_double()
    rc = load().gorgo_measure_gather(int(device), _dev_ptr(buffer), buffer.numel(),
                                     int(footprint_bytes), stream, C.byref(out))
    return rc, out.value


def gorgo_debug_set(sim, what: int, value: int) -> int:
    """Test switches of the replay kernel (GORGO_DEBUG_* constants)."""
    return load().gorgo_debug_set(sim, int(what), int(value))


def gorgo_eval_population_static(sim, n_candidates, params, time_scale, stream, p95_ttft_ms,
                                 p95_e2e_ms, route=None, hit_blocks=None, cand_status=None) -> int:
    """Evaluation that uses the scratch array built into the library instead of a workspace, for
    callers that may not allocate device memory.  ``params``: float64 numpy array (host) or torch
    CUDA tensor; outputs: torch CUDA tensors.  Returns GORGO_ERR_STATIC_LIMIT when one
    candidate's scratch exceeds GORGO_STATIC_SCRATCH_BYTES.  Calls must not overlap on the GPU."""
    pp = _np_ptr(params) if isinstance(params, np.ndarray) else _dev_ptr(params)
    return load().gorgo_eval_population_static(
        sim, int(n_candidates), pp, float(time_scale), stream, _dev_ptr(p95_ttft_ms),
        _dev_ptr(p95_e2e_ms), _dev_ptr(route), _dev_ptr(hit_blocks), _dev_ptr(cand_status))


def gorgo_sim_set_replica_speeds(sim, prefill_ms_per_token=None, tpot_ms=None) -> int:
    """Per-replica prefill time per token and time per output token (host float64 arrays of R
    values, or None for the uniform constant) for every later replay of ``sim``."""
    a = None if prefill_ms_per_token is None else np.ascontiguousarray(prefill_ms_per_token, np.float64)
    b = None if tpot_ms is None else np.ascontiguousarray(tpot_ms, np.float64)
    return load().gorgo_sim_set_replica_speeds(sim, _np_ptr(a), _np_ptr(b))


def gorgo_sim_set_proxy_index(sim, enable: bool = True) -> int:
    """Score with the proxy's own index (blocks ever dispatched to a replica) instead of the
    replica's cache."""
    return load().gorgo_sim_set_proxy_index(sim, int(bool(enable)))


def gorgo_sim_set_rtt_series(sim, samples=None, epoch_ms: float = 30_000.0, alpha: float = 0.3) -> int:
    """Time-varying network: ``samples`` [n_epochs, G, R] RTT probes per epoch (None: back to the
    static matrix)."""
    if samples is None:
        return load().gorgo_sim_set_rtt_series(sim, 0, 0.0, 0.0, None)
    s = np.ascontiguousarray(samples, dtype=np.float64)
    return load().gorgo_sim_set_rtt_series(sim, int(s.shape[0]), float(epoch_ms), float(alpha), _np_ptr(s))


def gorgo_sim_set_service_model(sim, decode_slowdown: float = 0.0, kv_budget_tokens: int = 0) -> int:
    """Decode slow-down per additional busy slot and KV budget per replica in tokens (0 = off)."""
    return load().gorgo_sim_set_service_model(sim, float(decode_slowdown), int(kv_budget_tokens))


def gorgo_eval_population_scales(sim, n_candidates, params, time_scales, workspace, stream,
                                 p95_ttft_ms, p95_e2e_ms, route=None, hit_blocks=None,
                                 state_digest=None, cand_status=None) -> int:
    """Population evaluation with one time scale per candidate.  ``params``: float64 numpy array
    (host) or torch CUDA tensor; ``time_scales``: host float64 numpy array [P]; every other
    array: torch CUDA tensor or None."""
    pp = _np_ptr(params) if isinstance(params, np.ndarray) else _dev_ptr(params)
    ts = np.ascontiguousarray(time_scales, dtype=np.float64)
    assert ts.shape == (int(n_candidates),)
    return load().gorgo_eval_population_scales(
        sim, int(n_candidates), pp, _np_ptr(ts), _dev_ptr(workspace), workspace.numel(), stream,
        _dev_ptr(p95_ttft_ms), _dev_ptr(p95_e2e_ms), _dev_ptr(route), _dev_ptr(hit_blocks),
        _dev_ptr(state_digest), _dev_ptr(cand_status))


POLICIES = {"least-load": 0, "least-request": 1, "prefix-cache": 2, "session-affinity": 3,
            "random": 4}


def gorgo_eval_policy(sim, policy, draws, time_scale, workspace, stream, p95_ttft_ms, p95_e2e_ms,
                      route=None, hit_blocks=None, state_digest=None, cand_status=None) -> int:
    """One replay under a baseline policy (name from POLICIES or its number).  ``draws``: host
    uint32 numpy array with one entry per request (``random`` only, else None); every other
    array: torch CUDA tensor or None."""
    pid = POLICIES[policy] if isinstance(policy, str) else int(policy)
    d = None if draws is None else np.ascontiguousarray(draws, dtype=np.uint32)
    return load().gorgo_eval_policy(
        sim, pid, _np_ptr(d), float(time_scale), _dev_ptr(workspace), workspace.numel(), stream,
        _dev_ptr(p95_ttft_ms), _dev_ptr(p95_e2e_ms), _dev_ptr(route), _dev_ptr(hit_blocks),
        _dev_ptr(state_digest), _dev_ptr(cand_status))


def gorgo_window_count(n_requests: int, window: int, hop: int):
    out = C.c_uint64()
    rc = load().gorgo_window_count(int(n_requests), int(window), int(hop), C.byref(out))
    return rc, out.value


def gorgo_eval_population_windows(sim, n_candidates, params, time_scale, workspace, stream, window,
                                  hop, win_p95_ttft_ms, best_win_p95_ttft_ms, best_window=None,
                                  p95_ttft_ms=None, p95_e2e_ms=None, cand_status=None) -> int:
    """Population evaluation reduced to the rolling-window objective.  ``params``: float64 numpy
    array (host) or torch CUDA tensor; every other array: torch CUDA tensor or None."""
    pp = _np_ptr(params) if isinstance(params, np.ndarray) else _dev_ptr(params)
    return load().gorgo_eval_population_windows(
        sim, int(n_candidates), pp, float(time_scale), _dev_ptr(workspace), workspace.numel(),
        stream, int(window), int(hop), _dev_ptr(win_p95_ttft_ms), _dev_ptr(best_win_p95_ttft_ms),
        _dev_ptr(best_window), _dev_ptr(p95_ttft_ms), _dev_ptr(p95_e2e_ms), _dev_ptr(cand_status))


def gorgo_es_run(sim, *, x0, z, tuned, lo, hi, sigma0, sigma_up, n_steps, lam, workspace, stream,
                 time_scale=1.0, objective=0):
    """Runs the evolution strategy; returns (status, x_best[K], objective_best, sigma_final,
    history[n_steps, 4 + n_tuned]).  All array arguments are host numpy arrays except
    ``workspace`` (torch CUDA tensor)."""
    x0 = np.ascontiguousarray(x0, dtype=np.float64)
    z = np.ascontiguousarray(z, dtype=np.float64)
    tuned = np.ascontiguousarray(tuned, dtype=np.uint32)
    lo = np.ascontiguousarray(lo, dtype=np.float64)
    hi = np.ascontiguousarray(hi, dtype=np.float64)
    T = tuned.shape[0]
    assert z.size == n_steps * lam * T and lo.shape == (T,) and hi.shape == (T,)
    cfg = gorgo_es_config_t(int(n_steps), int(lam), int(T), int(objective), tuned.ctypes.data,
                            lo.ctypes.data, hi.ctypes.data, float(sigma0), float(sigma_up),
                            float(time_scale))
    x_best = np.zeros_like(x0)
    hist = np.zeros((int(n_steps), 4 + T), dtype=np.float64)
    fb, sg = C.c_double(), C.c_double()
    rc = load().gorgo_es_run(sim, C.byref(cfg), _np_ptr(x0), _np_ptr(z), _dev_ptr(workspace),
                             workspace.numel(), stream, _np_ptr(x_best), C.byref(fb), C.byref(sg),
                             _np_ptr(hist))
    return rc, x_best, fb.value, sg.value, hist


def gorgo_tune_online(sim, *, x0, z, tuned, lo, hi, sigma0, sigma_up, workspace, stream,
                      time_scale=1.0, window=128, hop=32, route=None):
    """Online (1+1)-ES inside one replay for ``P = x0.shape[0]`` independent tuners.  ``x0``
    [P, K], ``z`` [P, n_draw_steps, n_tuned] host arrays; ``route`` a torch CUDA uint8 tensor
    [P, N] or None.  Returns (status, x_final [P, K], sigma_final [P], steps_done,
    history [P, n_draw_steps, 4 + 2*n_tuned], p95_ttft [P], p95_e2e [P])."""
    x0 = np.ascontiguousarray(x0, dtype=np.float64)
    z = np.ascontiguousarray(z, dtype=np.float64)
    tuned = np.ascontiguousarray(tuned, dtype=np.uint32)
    lo = np.ascontiguousarray(lo, dtype=np.float64)
    hi = np.ascontiguousarray(hi, dtype=np.float64)
    P, T = x0.shape[0], tuned.shape[0]
    n_steps = z.shape[1] if z.ndim == 3 else 0
    assert z.shape == (P, n_steps, T) and lo.shape == (T,) and hi.shape == (T,)
    cfg = gorgo_online_config_t(int(T), int(n_steps), int(window), int(hop), tuned.ctypes.data,
                                lo.ctypes.data, hi.ctypes.data, float(sigma0), float(sigma_up),
                                float(time_scale))
    x_final = np.zeros_like(x0)
    sig = np.zeros(P, np.float64)
    hist = np.zeros((P, n_steps, 4 + 2 * T), np.float64)
    pt, pe = np.zeros(P, np.float64), np.zeros(P, np.float64)
    done = C.c_uint32()
    rc = load().gorgo_tune_online(sim, C.byref(cfg), int(P), _np_ptr(x0), _np_ptr(z),
                                  _dev_ptr(workspace), workspace.numel(), stream, _np_ptr(x_final),
                                  _np_ptr(sig), C.byref(done), _np_ptr(hist), _np_ptr(pt), _np_ptr(pe),
                                  _dev_ptr(route))
    return rc, x_final, sig, done.value, hist, pt, pe


def gorgo_state_bytes(sim):
    out = C.c_uint64()
    rc = load().gorgo_state_bytes(sim, C.byref(out))
    return rc, out.value


def gorgo_sim_reset(sim, state_workspace, stream: int = 0) -> int:
    return load().gorgo_sim_reset(sim, _dev_ptr(state_workspace), state_workspace.numel(), stream)


def gorgo_route_batch(sim, params, time_scale, first, count, state_workspace, stream, route,
                      hit_blocks=None, ttft_ms=None, e2e_ms=None) -> int:
    w = np.ascontiguousarray(params, dtype=np.float64)
    return load().gorgo_route_batch(sim, _np_ptr(w), float(time_scale), int(first), int(count),
                                    _dev_ptr(state_workspace), state_workspace.numel(), stream,
                                    _dev_ptr(route), _dev_ptr(hit_blocks), _dev_ptr(ttft_ms),
                                    _dev_ptr(e2e_ms))


def gorgo_state_digest(sim, state_workspace, stream, digest) -> int:
    return load().gorgo_state_digest(sim, _dev_ptr(state_workspace), state_workspace.numel(),
                                     stream, _dev_ptr(digest))


def gorgo_state_status(sim, state_workspace, stream: int = 0):
    seen = C.c_uint64()
    rc = load().gorgo_state_status(sim, _dev_ptr(state_workspace), state_workspace.numel(),
                                   stream, C.byref(seen))
    return rc, seen.value


def gorgo_replay_occupancy(sim):
    """Returns (status, replay CTAs per SM, dynamic shared-memory bytes per CTA)."""
    n, b = C.c_int32(), C.c_uint64()
    rc = load().gorgo_replay_occupancy(sim, C.byref(n), C.byref(b))
    return rc, n.value, b.value


def gorgo_set_profiling(sim, enable: bool) -> int:
    return load().gorgo_set_profiling(sim, int(bool(enable)))


def gorgo_last_replay_ms(sim):
    """Returns (status, summed replay-kernel milliseconds, timed launches) of the last evaluation."""
    ms, n = C.c_double(), C.c_uint32()
    rc = load().gorgo_last_replay_ms(sim, C.byref(ms), C.byref(n))
    return rc, ms.value, n.value


def gorgo_last_window_ms(sim):
    """Returns (status, summed window-kernel milliseconds, timed launches) of the last
    gorgo_eval_population_windows."""
    ms, n = C.c_double(), C.c_uint32()
    rc = load().gorgo_last_window_ms(sim, C.byref(ms), C.byref(n))
    return rc, ms.value, n.value


# ------------------------------------------------------------------------ buffer holder
class GorgoSim:
    """Owns the handle and the torch tensors used as device buffers (plumbing only)."""

    def __init__(self, workload, device: int = 0):
        import torch
        self.torch = torch
        self.device = torch.device("cuda", device)
        self.w = workload
        rc, self.h = gorgo_sim_create(rtt_ms=workload.rtt_ms, device=device,
                                      **workload.config_dict())
        if rc != GORGO_OK:
            raise GorgoError(rc, "gorgo_sim_create")
        self.R = workload.spec.n_replicas
        self.K = workload.n_params
        self.N = workload.n_requests
        rc, nbytes = gorgo_trace_bytes(self.N, int(workload.hash_off[-1]))
        self.trace_buf = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        rc = gorgo_trace_upload(self.h, workload.ts_ms, workload.input_tokens,
                                workload.output_tokens, workload.origin, workload.hash_off,
                                workload.hash_ids, self.trace_buf, self.stream)
        if rc != GORGO_OK:
            raise GorgoError(rc, "gorgo_trace_upload")
        self.workspace = None

    @property
    def stream(self) -> int:
        return int(self.torch.cuda.current_stream(self.device).cuda_stream)

    def close(self):
        if getattr(self, "h", None):
            self.torch.cuda.synchronize(self.device)
            gorgo_sim_destroy(self.h)
            self.h = None
        self.trace_buf = None
        self.workspace = None

    def ensure_workspace(self, resident: int, max_bytes: Optional[int] = None) -> int:
        """Allocate a workspace for up to ``resident`` candidates in flight (fewer if
        ``max_bytes`` does not allow it).  Returns the resident count actually provided."""
        torch = self.torch
        while True:
            rc, nbytes = gorgo_workspace_bytes(self.h, resident)
            if rc != GORGO_OK:
                raise GorgoError(rc, "gorgo_workspace_bytes")
            if max_bytes is None or nbytes <= max_bytes or resident == 1:
                break
            resident = max(1, min(resident - 1, int(resident * max_bytes / nbytes)))
        if self.workspace is None or self.workspace.numel() < nbytes:
            self.workspace = None
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        return resident

    def eval_population(self, params, time_scale=1.0, *, want_route=False, want_hit=False,
                        want_digest=False, want_stats=False, resident=None, max_bytes=None):
        """Device-output evaluation; returns a dict of torch CUDA tensors."""
        torch = self.torch
        params = np.ascontiguousarray(params, dtype=np.float64)
        P = params.shape[0]
        self.ensure_workspace(P if resident is None else resident, max_bytes)
        dev = self.device
        out = dict(p95_ttft=torch.empty(P, dtype=torch.float64, device=dev),
                   p95_e2e=torch.empty(P, dtype=torch.float64, device=dev),
                   status=torch.zeros(P, dtype=torch.int32, device=dev))
        out["route"] = torch.empty((P, self.N), dtype=torch.uint8, device=dev) if want_route else None
        out["hit"] = torch.empty((P, self.N), dtype=torch.uint16, device=dev) if want_hit else None
        out["digest"] = torch.empty((P, self.R, 2), dtype=torch.uint64, device=dev) if want_digest else None
        out["stats"] = torch.empty((P, 4), dtype=torch.uint64, device=dev) if want_stats else None
        rc = gorgo_eval_population(self.h, P, params, time_scale, self.workspace, self.stream,
                                   out["p95_ttft"], out["p95_e2e"], out["route"], out["hit"],
                                   out["digest"], out["stats"], out["status"])
        if rc != GORGO_OK:
            raise GorgoError(rc, "gorgo_eval_population")
        return out
