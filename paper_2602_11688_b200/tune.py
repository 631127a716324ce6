"""Command-line tuner: runs the paper's evolution strategy (Section 2.3) on a seeded synthetic
workload through the CUDA library and sets the tuned cost model beside the baseline routing
policies of Section 4, all replayed through the same simulator.

    python -m paper_2602_11688_b200.tune --workload regions --steps 30 --lam 32

Prints one JSON line per ES step and a final JSON object with the policy table.  Everything is
computed by the library (there is no CPU path); numpy only draws the normal perturbations, which
are an input of the strategy.
"""
from __future__ import annotations

import argparse
import json
import time

import numpy as np


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawTextHelpFormatter)
    ap.add_argument("--workload", default="regions")
    ap.add_argument("--requests", type=int, default=None)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--lam", type=int, default=32, help="offspring per step (1 = the paper's (1+1)-ES)")
    ap.add_argument("--sigma0", type=float, default=0.5)
    ap.add_argument("--sigma-up", type=float, default=1.5)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--objective", choices=["ttft", "e2e"], default="ttft")
    ap.add_argument("--scale", type=float, default=None, help="time scale (default: the workload's)")
    args = ap.parse_args(argv)

    import torch
    from . import binding as gb
    from . import workloads as W

    kw = {"population": 1}
    if args.requests:
        kw["n_requests"] = args.requests
    w = W.make_workload(args.workload, **kw)
    scale = float(w.spec.time_scales[0]) if args.scale is None else args.scale
    K, R, N = w.n_params, w.spec.n_replicas, w.n_requests
    sim = gb.GorgoSim(w)
    dev = sim.device
    sim.ensure_workspace(max(args.lam, 1), max_bytes=int(torch.cuda.mem_get_info(dev)[0] * 0.8))

    # Section 4: W_rtt and W_queue start at 0.5 and 0.1 in [0.05, 2.0] and [0.05, 0.5]; the
    # prefill weight stays 1; per-replica normalisers (if the workload has them) stay 1.
    x0 = np.ones(K)
    x0[0], x0[2] = 0.5, 0.1
    tuned = np.array([0, 2], dtype=np.uint32)
    lo, hi = np.array([0.05, 0.05]), np.array([2.0, 0.5])
    z = np.random.default_rng(args.seed).standard_normal((args.steps, args.lam, 2))
    t0 = time.perf_counter()
    rc, x, f, sigma, hist = gb.gorgo_es_run(
        sim.h, x0=x0, z=z, tuned=tuned, lo=lo, hi=hi, sigma0=args.sigma0, sigma_up=args.sigma_up,
        n_steps=args.steps, lam=args.lam, workspace=sim.workspace, stream=sim.stream,
        time_scale=scale, objective=0 if args.objective == "ttft" else 1)
    if rc != gb.GORGO_OK:
        raise gb.GorgoError(rc, "gorgo_es_run")
    es_s = time.perf_counter() - t0
    for t, h in enumerate(hist):
        print(json.dumps({"step": t + 1, "best_offspring_ms": h[0], "accepted": bool(h[1]),
                          "sigma": h[2], "parent_ms": h[3], "w_rtt": h[4], "w_queue": h[5]}))

    def one(params):
        out = sim.eval_population(np.asarray(params, dtype=np.float64).reshape(1, K), scale)
        torch.cuda.synchronize(dev)
        return float(out["p95_ttft"][0]), float(out["p95_e2e"][0])

    table = {"gorgo-initial": one(x0), "gorgo-tuned": one(x)}
    pt = torch.zeros(1, dtype=torch.float64, device=dev)
    pe = torch.zeros(1, dtype=torch.float64, device=dev)
    draws = np.random.default_rng(args.seed + 1).integers(0, 2 ** 32, size=N, dtype=np.uint64)
    for name in gb.POLICIES:
        rc = gb.gorgo_eval_policy(sim.h, name, draws.astype(np.uint32) if name == "random" else None,
                                  scale, sim.workspace, sim.stream, pt, pe)
        if rc != gb.GORGO_OK:
            raise gb.GorgoError(rc, "gorgo_eval_policy")
        torch.cuda.synchronize(dev)
        table[name] = (float(pt.item()), float(pe.item()))
    print(json.dumps({
        "workload": w.spec.name, "requests": N, "replicas": R, "time_scale": scale,
        "es": {"steps": args.steps, "lambda": args.lam, "replays": 1 + args.steps * args.lam,
               "seconds": es_s, "w_rtt": float(x[0]), "w_queue": float(x[2]), "sigma": sigma,
               "objective_ms": f},
        "p95_ttft_ms_and_p95_e2e_ms": table}))
    sim.close()


if __name__ == "__main__":
    main()
