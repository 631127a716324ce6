"""Helpers shared by the GPU parity tests: run the CUDA library through its C ABI and the CPU
oracle on the same seeded workload and compare them."""
from concurrent.futures import ThreadPoolExecutor

import numpy as np

from oracle import gorgo_oracle as O


def small_trace(seed, n_req=300, n_sessions=12, max_blocks=7, structured=True, B=512,
                rate_ms=40.0):
    """Tiny random trace.  structured: sessions extend their own prefix (ids imply their
    prefix); otherwise every request is a random subset of a small id pool in random order."""
    rng = np.random.default_rng(seed)
    reqs, t = [], 0.0
    conv = {}
    nxt = 1000
    for _ in range(n_req):
        t += float(rng.exponential(rate_ms))
        if structured:
            s = int(rng.integers(n_sessions))
            ids = conv.get(s)
            if ids is None or len(ids) >= max_blocks or rng.random() < 0.25:
                k = int(rng.integers(1, 4))
                ids = list(range(nxt, nxt + k)); nxt += k
            else:
                k = int(rng.integers(1, 3))
                ids = ids + list(range(nxt, nxt + k)); nxt += k
                ids = ids[:max_blocks]
            conv[s] = ids
        else:
            k = int(rng.integers(1, max_blocks + 1))
            ids = [int(x) for x in rng.choice(np.arange(1, 40), size=k, replace=False)]
        n = len(ids)
        in_tok = (n - 1) * B + int(rng.integers(1, B + 1))
        out = int(rng.integers(0, 30))
        reqs.append((t, in_tok, out, ids))
    return reqs


def gpu_eval(workload, params=None, scale=None, *, resident=None, max_bytes=None, route=True,
             hit=True, digest=True, stats=True, sim=None, debug=None):
    """Evaluate a population through gorgo_eval_population; returns numpy arrays.  `debug` maps
    GORGO_DEBUG_* switches to values (set on a simulator created here)."""
    import torch
    from paper_2602_11688_b200 import binding as gb
    own = sim is None
    if own:
        sim = gb.GorgoSim(workload)
        for what, value in (debug or {}).items():
            assert gb.gorgo_debug_set(sim.h, what, value) == gb.GORGO_OK
    try:
        params = workload.params if params is None else np.ascontiguousarray(params, np.float64)
        scale = workload.spec.time_scales[0] if scale is None else scale
        out = sim.eval_population(params, scale, want_route=route, want_hit=hit,
                                  want_digest=digest, want_stats=stats, resident=resident,
                                  max_bytes=max_bytes)
        torch.cuda.synchronize()
        res = {k: (None if v is None else v.cpu().numpy()) for k, v in out.items()}
    finally:
        if own:
            sim.close()
    assert (res["status"] == 0).all(), res["status"]
    return res


def oracle_eval(workload, params, scale, threads=8):
    """Replay the given parameter rows on the oracle (one thread per candidate; ctypes drops
    the GIL).  Returns a list of (RunResult, p95_ttft, p95_e2e, digest, stats)."""
    params = np.ascontiguousarray(params, np.float64)
    with ThreadPoolExecutor(max_workers=threads) as ex:
        return list(ex.map(lambda w: O.replay(workload, w, scale), params))


def assert_candidate_matches(gpu, idx, ref, *, rel=1e-9):
    """Bit-exact routes, hit lengths, cache digests and counters; p95 within `rel` relative
    (the stated tolerance; in practice the values are identical)."""
    res, p_ttft, p_e2e, dg, st = ref
    if gpu.get("route") is not None:
        bad = np.nonzero(gpu["route"][idx] != res.route)[0]
        assert bad.size == 0, f"candidate {idx}: first route mismatch at request {bad[:5]}"
    if gpu.get("hit") is not None:
        bad = np.nonzero(gpu["hit"][idx] != res.hit)[0]
        assert bad.size == 0, f"candidate {idx}: first hit mismatch at request {bad[:5]}"
    if gpu.get("digest") is not None:
        assert gpu["digest"][idx].tolist() == dg.tolist(), f"candidate {idx}: cache digest"
    if gpu.get("stats") is not None:
        assert gpu["stats"][idx].tolist() == st.tolist(), f"candidate {idx}: counters"
    for name, want in (("p95_ttft", p_ttft), ("p95_e2e", p_e2e)):
        got = float(gpu[name][idx])
        assert abs(got - want) <= rel * abs(want), (idx, name, got, want)


def check_population(workload, params=None, scale=None, candidates=None, **kw):
    params = workload.params if params is None else np.ascontiguousarray(params, np.float64)
    scale = workload.spec.time_scales[0] if scale is None else scale
    gpu = gpu_eval(workload, params, scale, **kw)
    cand = list(range(params.shape[0])) if candidates is None else list(candidates)
    refs = oracle_eval(workload, params[cand], scale)
    for idx, ref in zip(cand, refs):
        assert_candidate_matches(gpu, idx, ref)
    return gpu, refs
