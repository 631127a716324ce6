"""Cycle accounting of the replay kernel's warps.

Builds a second copy of the library with ``-DGORGO_PROF`` (SM-clock laps compiled into the
replay kernel), replays a workload once through it and prints, per role, the mean clock ticks
per request spent in each phase of its loop.  The product library is never built with the
accounting and this module never touches it.

    python -m paper_2602_11688_b200.phase_profile --workload longctx --requests 30000 \
        --cache-blocks 6000
"""
from __future__ import annotations

import argparse
import ctypes as C
import json

import numpy as np

ROLES = {
    "route": (0, ["load update of the previous route, wait for the completion sums",
                  "completion sums, queue term of the score", "wait for the prefix hits (barrier)",
                  "staged part of the score, order key", "argmin over replicas",
                  "hit of the chosen replica, route stores, barrier arrive"]),
    "service": (16, ["retire: list entry, window vote, grid value", "fence and publish",
                     "next pipeline stage: list exchange, window loads", "slot argmin",
                     "times, outputs, grid load", "idle round"]),
    "gate": (32, ["own turn: probe here if needed, hand over", "wait for the route (barrier)",
                  "job post, early hand-over of the next request",
                  "own turn: staged? recent route to a holder?", "own turn: wait for commits",
                  None, None, None, None, None, None,
                  "#probes done by this warp", "#next request not staged yet at hand-over time",
                  "#next request not handed over early (shared block or recent route to a holder)",
                  "#hits handed over early"]),
    "commit (all three warps)": (48, ["wait for the next routed request", "need and eviction",
                                      "mask bits of the inserted blocks", "recency list, progress",
                                      "requests of other warps' replicas", None, None, None,
                                      "#evictions: clean case (victims taken from the ring as listed)",
                                      "#evictions: an entry was void or touched again",
                                      "#evictions: ring held too few entries",
                                      "#evictions: more than 96 victims or ring not in use",
                                      "#requests that evict", "#evictions finished by own walk",
                                      "#polls for ring entries", "#blocks evicted"]),
}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="longctx")
    ap.add_argument("--requests", type=int, default=None)
    ap.add_argument("--population", type=int, default=None)
    ap.add_argument("--cache-blocks", type=int, default=None)
    ap.add_argument("--repeat", type=int, default=3)
    args = ap.parse_args()

    import torch
    from paper_2602_11688_b200 import binding as gb
    from paper_2602_11688_b200 import build as gbuild
    from paper_2602_11688_b200 import workloads as W

    gb.LIB_PATH = gbuild.build_phase_profile()
    lib = gb.load()
    lib.gorgo_debug_phase_cycles.argtypes = [C.c_void_p, C.POINTER(C.c_uint64)]
    lib.gorgo_debug_phase_cycles.restype = C.c_int

    kw = {}
    if args.requests:
        kw["n_requests"] = args.requests
    if args.population:
        kw["population"] = args.population
    if args.cache_blocks:
        kw["cache_blocks"] = args.cache_blocks
    w = W.make_workload(args.workload, **kw)
    scale = float(w.spec.time_scales[0])
    P, N = w.params.shape[0], w.n_requests
    sim = gb.GorgoSim(w)
    buf = (C.c_uint64 * 64)()
    gb.gorgo_set_profiling(sim.h, True)
    ms = 0.0
    for it in range(args.repeat):
        lib.gorgo_debug_phase_cycles(sim.h, buf)            # clears the accumulators
        sim.eval_population(w.params, scale)
        torch.cuda.synchronize()
        rc, ms, _ = gb.gorgo_last_replay_ms(sim.h)
    lib.gorgo_debug_phase_cycles(sim.h, buf)
    cyc = np.array(list(buf), dtype=np.float64) / (float(P) * N)
    rc, ctas, smem = gb.gorgo_replay_occupancy(sim.h)
    out = {"workload": w.spec.name, "requests": N, "population": P,
           "replay_ms": ms, "us_per_request": ms * 1e3 / N, "ctas_per_sm": ctas,
           "smem_bytes_per_cta": smem, "per_request": {}}
    for role, (base, names) in ROLES.items():
        d = {}
        for k, name in enumerate(names):
            if name:
                d[name] = round(float(cyc[base + k]), 3 if name.startswith("#") else 1)
        d["sum of laps"] = round(float(sum(cyc[base + k] for k, nm in enumerate(names)
                                         if nm and not nm.startswith("#"))), 1)
        out["per_request"][role] = d
    print(json.dumps(out, indent=1))
    sim.close()


if __name__ == "__main__":
    main()
