#!/usr/bin/env python
"""Benchmark of the population-replay hot path.

One step = one full pass of the hot path: `gorgo_eval_population` over the whole trace for the
whole population (reset, replay of every candidate, p95 selection).  Prints one JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload longctx] [--impl reference]

`--impl reference` times the CPU oracle (as it stands) on a bounded sample of the same workload.
With N > 1 every rank evaluates its own population of the single-GPU size on its own GPU
(candidates are independent: no collective on the data path, weak scaling).  Started without
torchrun, `--gpus N` starts the N ranks itself.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "candidate-request-replica routing evals/sec"
UNIT = "evals/s"


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(path))["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-i", str(self.gpu), "-lms", "200"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                      "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one replay-kernel launch per
# candidate x request, from the single-pass ncu capture of the full-size workload summarised under
# profiles/ (the per-request figure grows with the footprint, so a reduced case is not scaled up).
# Reported only while the kernel source is the one that was captured (first 16 hex digits of its
# sha256) and only for the unreduced workload.
NCU_TRAFFIC = {"longctx": {"bytes_per_candidate_request": (120_785_143_040 + 44_431_718_144) / (256 * 500_000),
                           "kernel_sha256_16": "31f37f777b3f47f3"}}


def kernel_sha16():
    import hashlib
    src = os.path.join(ROOT, "paper_2602_11688_b200", "csrc", "gorgo_kernels.cu")
    try:
        return hashlib.sha256(open(src, "rb").read()).hexdigest()[:16]
    except OSError:
        return None


def captured_traffic(workload: str, candidate_requests_per_launch: float):
    rec = NCU_TRAFFIC.get(workload)
    if rec is None or rec["bytes_per_candidate_request"] is None:
        return None
    if kernel_sha16() != rec["kernel_sha256_16"]:
        return None
    return rec["bytes_per_candidate_request"] * candidate_requests_per_launch


def algorithmic_bytes(stats: np.ndarray, n_requests: int) -> float:
    """Bytes the method itself must move for one evaluation, from the per-candidate counters
    (sum_i min(h_i+1, n), sum h*, sum n, sum evicted), 32-byte sectors:
      probe 32*sum_i min(h_i+1,n); commit 32*h* + 64*(n-h*) + 64*E; stream 8*n + 22;
      emit 17 (TTFT, E2E, route; the optional hit length is not asked for in the timed step)."""
    s = stats.astype(np.float64)
    probe = 32.0 * s[:, 0]
    commit = 32.0 * s[:, 1] + 64.0 * (s[:, 2] - s[:, 1]) + 64.0 * s[:, 3]
    stream = 8.0 * s[:, 2] + 22.0 * n_requests
    emit = 17.0 * n_requests
    return float(np.sum(probe + commit + stream + emit))


def oracle_sample_rate(w, scale, n_candidates, n_requests, threads=None):
    """Oracle throughput on `n_candidates` candidates x the first `n_requests` requests, one
    candidate per task on a pool of `threads` Python threads (the C++ call releases the GIL)."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import gorgo_oracle as O
    O.build()
    threads = threads or max(1, min(os.cpu_count() or 1, 8))
    oracles = [O.Oracle.from_workload(w) for _ in range(n_candidates)]
    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=min(threads, n_candidates)) as ex:
        list(ex.map(lambda io: io[1].run(w.params[io[0] % w.params.shape[0]], scale, n_requests),
                    enumerate(oracles)))
    dt = time.perf_counter() - t0
    for o in oracles:
        o.close()
    evals = float(n_candidates) * n_requests * w.spec.n_replicas
    return evals / dt, dt


def oracle_candidates(w, cores):
    """Candidates of one oracle sample: the whole population for the two small workloads, one
    per host thread otherwise (the rate per candidate x request does not depend on how many
    candidates run, they are independent)."""
    P = int(w.params.shape[0])
    return P if w.spec.name in ("tiny", "regions") else cores


def bench_reference(args, w, scale):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = max(1, min(os.cpu_count() or 1, 8))
    n_cand = oracle_candidates(w, cores)
    n_req = min(w.n_requests, args.ref_requests)
    for _ in range(args.warmup):
        oracle_sample_rate(w, scale, min(n_cand, cores), min(n_req, 2000))
    rates, times = [], []
    for _ in range(args.steps):
        r, dt = oracle_sample_rate(w, scale, n_cand, n_req)
        rates.append(r); times.append(dt)
    value = float(np.mean(rates))
    sample = (f"{n_cand} candidates x first {n_req} requests of '{w.spec.name}' per step, one thread "
              f"per candidate, at most {cores} at a time")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": float(np.mean(times) * 1e3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(w, scale),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": min(cores, n_cand), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(w, scale):
    s = w.spec
    return {"workload": s.name, "n_replicas": s.n_replicas, "n_requests": w.n_requests,
            "population": int(w.params.shape[0]), "cache_blocks": s.cache_blocks,
            "slots": s.slots, "n_params": w.n_params, "time_scale": scale,
            "block_ids_total": int(w.hash_off[-1]), "seed": s.seed}


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(args) -> int:
    """`--gpus N` without torchrun: start the N ranks (one process per GPU) and pass their output on."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
           f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
           "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "WARN")
    return subprocess.call(cmd, env=env)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="longctx")
    ap.add_argument("--requests", type=int, default=None, help="reduced trace length (debug)")
    ap.add_argument("--population", type=int, default=None)
    ap.add_argument("--cache-blocks", type=int, default=None)
    ap.add_argument("--ref-requests", type=int, default=None,
                    help="requests per candidate in one reference / cpu-baseline sample")
    ap.add_argument("--all-scales", action="store_true",
                    help="evaluate the population at every time scale of the workload as ONE "
                         "population (candidates x scales) instead of the first scale only")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-yardsticks", action="store_true",
                    help="skip the random-sector and L2 gather measurements")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "ours" and args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))

    from paper_2602_11688_b200 import workloads as W
    kw = {}
    if args.requests:
        kw["n_requests"] = args.requests
    if args.population:
        kw["population"] = args.population
    if args.cache_blocks:
        kw["cache_blocks"] = args.cache_blocks
    w = W.make_workload(args.workload, **kw)
    scale = float(w.spec.time_scales[0])

    if args.impl == "reference":
        # a step is a bounded sample: about 5 s of oracle time, so that 20 + 5 steps end in minutes
        if args.ref_requests is None:
            args.ref_requests = 150_000
        bench_reference(args, w, scale)
        return
    if args.ref_requests is None:
        args.ref_requests = 500_000

    import torch
    import torch.distributed as dist
    from paper_2602_11688_b200 import binding as gb
    from paper_2602_11688_b200 import sharding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        print(f"bench.py: --gpus {args.gpus} but {world} rank(s) were started", file=sys.stderr)
        sys.exit(2)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)

    base_params = w.params
    w.params = sharding.weak_scaling_population(base_params, rank)
    cand_scales = None
    if args.all_scales:
        all_scales = np.asarray(w.spec.time_scales, dtype=np.float64)
        P0 = w.params.shape[0]
        cand_scales = np.repeat(all_scales, P0)
        w.params = np.tile(w.params, (len(all_scales), 1))
    P, N, R, K = w.params.shape[0], w.n_requests, w.spec.n_replicas, w.n_params

    sim = gb.GorgoSim(w, device=local)
    free_b, _ = torch.cuda.mem_get_info(dev)
    resident = sim.ensure_workspace(P, max_bytes=int(free_b * 0.9))
    waves = -(-P // resident)
    stream = sim.stream
    d_params = torch.from_numpy(w.params).to(dev)
    p95_t = torch.empty(P, dtype=torch.float64, device=dev)
    p95_e = torch.empty(P, dtype=torch.float64, device=dev)
    stats = torch.zeros((P, 4), dtype=torch.uint64, device=dev)
    status = torch.zeros(P, dtype=torch.int32, device=dev)
    h_params = torch.from_numpy(w.params.copy()).pin_memory()
    h_p95_t = torch.empty(P, dtype=torch.float64).pin_memory()
    h_p95_e = torch.empty(P, dtype=torch.float64).pin_memory()

    def step_device(with_stats=False):
        if cand_scales is not None and not with_stats:
            rc = gb.gorgo_eval_population_scales(sim.h, P, d_params, cand_scales, sim.workspace,
                                                 stream, p95_t, p95_e, None, None, None, status)
        elif cand_scales is not None:
            # counters of the byte model: one evaluation per scale (the call with per-candidate
            # scales has no counter output)
            P0 = P // len(all_scales)
            rc = gb.GORGO_OK
            for k, sc in enumerate(all_scales):
                sl = slice(k * P0, (k + 1) * P0)
                rc = rc or gb.gorgo_eval_population(sim.h, P0, d_params[sl], float(sc), sim.workspace,
                                                    stream, p95_t[sl], p95_e[sl], None, None, None,
                                                    stats[sl], status[sl])
        else:
            rc = gb.gorgo_eval_population(sim.h, P, d_params, scale, sim.workspace, stream, p95_t,
                                          p95_e, None, None, None, stats if with_stats else None,
                                          status)
        if rc != gb.GORGO_OK:
            raise gb.GorgoError(rc, "gorgo_eval_population")

    def step_host():
        if cand_scales is not None:       # (no host-buffer call with per-candidate scales: copies here)
            d_params.copy_(h_params, non_blocking=True)
            step_device()
            h_p95_t.copy_(p95_t, non_blocking=True)
            h_p95_e.copy_(p95_e, non_blocking=True)
            torch.cuda.current_stream(dev).synchronize()
            return
        rc = gb.gorgo_eval_population_host(sim.h, P, h_params, scale, sim.workspace, stream,
                                           h_p95_t, h_p95_e)
        if rc != gb.GORGO_OK:
            raise gb.GorgoError(rc, "gorgo_eval_population_host")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def event_timer():
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(torch.cuda.current_stream(dev))

        def elapsed():
            e1.record(torch.cuda.current_stream(dev))
            e1.synchronize()
            return e0.elapsed_time(e1)
        return elapsed

    # the first evaluation collects the counters of the byte model
    step_device(with_stats=True)
    torch.cuda.synchronize(dev)
    assert int(status.abs().sum().item()) == 0, "a candidate reported a device-side limit"
    alg_bytes = algorithmic_bytes(stats.cpu().numpy(), N)

    # ---- device-resident timing: K steps, CUDA events on the launching stream
    gb.gorgo_set_profiling(sim.h, True)
    sampler = ClockSampler(local)
    replay = {"ms": 0.0, "launches": 0, "timed": False}

    def evaluate(_params):
        step_device()
        if replay["timed"]:
            # reading the event pair waits for this step; the stream has nothing else queued
            rc, ms, nl = gb.gorgo_last_replay_ms(sim.h)
            replay["ms"] += ms
            replay["launches"] += nl
        return None

    def timed_barrier():
        barrier()
        if not replay["timed"]:
            replay["timed"] = True
            sampler.start()

    ms_per_step, _, _ = sharding.run_ranks(rank, world, base_params, evaluate, args.steps,
                                           args.warmup, event_timer, timed_barrier, dev)
    clocks = sampler.stop()
    gb.gorgo_set_profiling(sim.h, False)
    evals_per_step = float(P) * N * R * world
    value = evals_per_step / (ms_per_step * 1e-3)

    # ---- end to end: host buffers in, host results out, copies inside the timed region
    step_host()
    barrier()
    t0 = time.perf_counter()
    elapsed = event_timer()
    for _ in range(args.steps):
        step_host()
    ev_ms = elapsed()
    barrier()
    wall_ms = (time.perf_counter() - t0) * 1e3
    e2e_ms = sharding.max_over_ranks(max(ev_ms, wall_ms), dev) / args.steps
    e2e_value = evals_per_step / (e2e_ms * 1e-3)
    p95_check = np.array_equal(h_p95_t.numpy(), p95_t.cpu().numpy())

    # ---- tuning objective (rolling window of 128 requests, hop 32) on top of the same replay:
    #      its kernels timed by the library's own events on the launching stream
    win_ms, win_launches = None, 0
    rc, n_win = gb.gorgo_window_count(N, 128, 32)
    if n_win > 0 and cand_scales is None:
        best_w = torch.empty(P, dtype=torch.float64, device=dev)
        gb.gorgo_set_profiling(sim.h, True)
        rc = gb.gorgo_eval_population_windows(sim.h, P, d_params, scale, sim.workspace, stream, 128,
                                              32, None, best_w, None, None, None, status)
        if rc != gb.GORGO_OK:
            raise gb.GorgoError(rc, "gorgo_eval_population_windows")
        rc, win_ms, win_launches = gb.gorgo_last_window_ms(sim.h)
        gb.gorgo_set_profiling(sim.h, False)
        barrier()

    # ---- yardsticks for a gather-bound kernel: random 32-byte sectors over the workspace
    #      (DRAM when it is far larger than L2) and over a footprint inside L2
    l2_bytes = int(torch.cuda.get_device_properties(dev).L2_cache_size)
    ws_bytes = int(sim.workspace.numel())
    yard = {}
    if rank == 0 and not args.no_yardsticks:
        big = min(ws_bytes - 4096, 9_000_000_000) // 4096 * 4096
        if big > 4 * l2_bytes:
            rc, gbs = gb.gorgo_measure_gather(local, sim.workspace, big, stream)
            if rc == gb.GORGO_OK:
                yard["random_sector_peak"] = {"value": gbs, "unit": "GB/s", "footprint_bytes": big}
        small = min(l2_bytes // 4, ws_bytes - 4096) // 4096 * 4096
        if small >= 4096:
            rc, gbs = gb.gorgo_measure_gather(local, sim.workspace, small, stream)
            if rc == gb.GORGO_OK:
                yard["l2_peak"] = {"value": gbs, "unit": "GB/s", "footprint_bytes": small}

    if rank == 0:
        rc, ctas_per_sm, smem_cta = gb.gorgo_replay_occupancy(sim.h)
        peak, peak_kind = measured_peak_gbs()
        launch_ms = replay["ms"] / max(1, replay["launches"])
        bytes_per_launch = alg_bytes / waves
        achieved = bytes_per_launch / (launch_ms * 1e-3) / 1e9
        l2_resident = ws_bytes <= l2_bytes
        l2_note = ("state touched per step (%.3f GB) fits the %.0f MB L2: L2-resident, timed warm "
                   "(bound: L2, see roofline.l2_peak)" % (ws_bytes / 1e9, l2_bytes / 1e6)) if l2_resident else \
                  ("state touched per step (%.1f GB) far exceeds the %.0f MB L2; no flush needed"
                   % (ws_bytes / 1e9, l2_bytes / 1e6))
        traffic = None
        if not (args.requests or args.population or args.cache_blocks):
            traffic = captured_traffic(args.workload, float(min(P, resident)) * N)
        roof = {
            "bound": "hbm", "kernel": "replay_kernel", "achieved": achieved, "peak": peak,
            "unit": "GB/s", "frac": achieved / peak, "peak_kind": peak_kind + " HBM copy",
            "traffic": traffic,
            "algorithmic_bytes_per_launch": bytes_per_launch,
            "bytes_per_eval": alg_bytes / (float(P) * N * R),
            "replay_ms_per_launch": launch_ms,
            "replay_share_of_step": (replay["ms"] / args.steps) / ms_per_step,
            "limited_by": "latency of each candidate's serial chain and instruction issue, "
                          "not bandwidth (see profiles/)",
        }
        if traffic is not None:
            roof["moved_frac"] = traffic / (launch_ms * 1e-3) / 1e9 / peak
        for k, v in yard.items():
            roof[k] = v
            roof["frac_of_" + k] = achieved / v["value"]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {**workload_config(w, "all of %s" % list(map(float, all_scales)) if args.all_scales else scale),
                       "resident_candidates": resident, "waves": waves,
                       "replay_ctas_per_sm": int(ctas_per_sm), "replay_smem_bytes_per_cta": int(smem_cta),
                       "l2": l2_note},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(P * K * 8),
                    "d2h_bytes_per_step": int(P * 20), "ms_per_step": e2e_ms,
                    "matches_device_run": bool(p95_check)},
            "gpu_launches": int(args.steps * waves * 3),
            "clocks": clocks,
            "roofline": roof,
        }
        if win_ms is not None:
            win_bytes = float(P) * 8.0 * (N + n_win)      # read every TTFT once, write every window
            line["window_objective"] = {
                "window": 128, "hop": 32, "windows_per_candidate": int(n_win),
                "ms_per_evaluation": win_ms, "launches": int(win_launches),
                "achieved": win_bytes / (win_ms * 1e-3) / 1e9, "unit": "GB/s",
                "frac_of_hbm_peak": win_bytes / (win_ms * 1e-3) / 1e9 / peak,
                "share_of_step": win_ms / ms_per_step}
        if not args.no_cpu_baseline and world == 1 and cand_scales is None:
            cores = max(1, min(os.cpu_count() or 1, 8))
            n_cand = oracle_candidates(w, cores)
            n_req = min(N, args.ref_requests)
            rate, dt = oracle_sample_rate(w, scale, n_cand, n_req)
            one_req = min(n_req, 100_000)
            rate1, dt1 = oracle_sample_rate(w, scale, 1, one_req)
            line["cpu_baseline"] = {
                "value": rate, "unit": UNIT, "cores": min(cores, n_cand), "kind": "oracle",
                "sample": f"{n_cand} candidates x first {n_req} requests of '{w.spec.name}', "
                          f"{dt:.1f} s, one thread per candidate",
                "single_thread": {"value": rate1, "unit": UNIT,
                                  "sample": f"1 candidate x first {one_req} requests, {dt1:.1f} s"}}
        print(json.dumps(line), flush=True)
    sim.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
