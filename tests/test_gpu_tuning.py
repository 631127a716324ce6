"""GPU parity of the tuning loop: rolling-window objective and evolution strategy, through the
C ABI, against oracle/gorgo_tuning.py driven by the CPU replay oracle."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import gorgo_oracle as O
from oracle import gorgo_tuning as T
from paper_2602_11688_b200 import workloads as W
from tests.util import small_trace


def _windows(sim, params, scale, window, hop, with_array=True, with_p95=True):
    import torch
    from paper_2602_11688_b200 import binding as gb
    P = params.shape[0]
    sim.ensure_workspace(P)
    rc, n_win = gb.gorgo_window_count(sim.N, window, hop)
    if rc != gb.GORGO_OK:
        n_win = 0                      # the evaluation call below reports the bad shape itself
    dev = sim.device
    win = torch.full((P, max(n_win, 1)), -1.0, dtype=torch.float64, device=dev) if with_array else None
    best = torch.full((P,), -1.0, dtype=torch.float64, device=dev)
    bidx = torch.full((P,), 12345, dtype=torch.int32, device=dev)
    pt = torch.zeros(P, dtype=torch.float64, device=dev) if with_p95 else None
    pe = torch.zeros(P, dtype=torch.float64, device=dev) if with_p95 else None
    st = torch.zeros(P, dtype=torch.int32, device=dev)
    rc = gb.gorgo_eval_population_windows(sim.h, P, params, scale, sim.workspace, sim.stream, window,
                                          hop, win, best, bidx, pt, pe, st)
    torch.cuda.synchronize()
    if rc != gb.GORGO_OK:
        return rc, None
    assert int(st.abs().sum()) == 0
    return rc, dict(n_win=n_win, win=None if win is None else win.cpu().numpy(),
                    best=best.cpu().numpy(), bidx=bidx.cpu().numpy(),
                    p95_ttft=None if pt is None else pt.cpu().numpy(),
                    p95_e2e=None if pe is None else pe.cpu().numpy())


@pytest.mark.parametrize("window,hop", [(128, 32), (100, 7), (1, 1), (2048, 500), (33, 64)])
def test_window_objective_matches_oracle(window, hop):
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload("tiny", n_requests=2300, population=5)
    scale = 1.0
    sim = gb.GorgoSim(w)
    try:
        rc, got = _windows(sim, w.params, scale, window, hop)
        assert rc == gb.GORGO_OK
        rc2, got2 = _windows(sim, w.params, scale, window, hop, with_array=False, with_p95=False)
        assert rc2 == gb.GORGO_OK
    finally:
        sim.close()
    assert got["n_win"] == T.window_count(w.n_requests, window, hop)
    for p in range(w.params.shape[0]):
        res, p_ttft, p_e2e, _, _ = O.replay(w, w.params[p], scale)
        want = T.window_p95(res.ttft.tolist(), window, hop)
        assert got["win"][p, :len(want)].tolist() == want          # bit-exact: exact selection
        best, idx = T.best_window(res.ttft.tolist(), window, hop)
        assert got["best"][p] == best and got["bidx"][p] == idx
        assert got2["best"][p] == best and got2["bidx"][p] == idx  # window values kept in scratch
        assert abs(got["p95_ttft"][p] - p_ttft) <= 1e-9 * abs(p_ttft)
        assert abs(got["p95_e2e"][p] - p_e2e) <= 1e-9 * abs(p_e2e)


def test_window_objective_rejects_bad_shapes():
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload("tiny", n_requests=300, population=2)
    sim = gb.GorgoSim(w)
    try:
        assert _windows(sim, w.params, 1.0, 2049, 32)[0] == gb.GORGO_ERR_INVALID_ARG   # too wide
        assert _windows(sim, w.params, 1.0, 301, 32)[0] == gb.GORGO_ERR_INVALID_ARG    # N < window
        assert _windows(sim, w.params, 1.0, 0, 32)[0] == gb.GORGO_ERR_INVALID_ARG
        assert _windows(sim, w.params, 1.0, 128, 0)[0] == gb.GORGO_ERR_INVALID_ARG
        rc, got = _windows(sim, w.params, 1.0, 300, 32)                               # one window
        assert rc == gb.GORGO_OK and got["n_win"] == 1
        assert got["best"].tolist() == got["win"][:, 0].tolist() and (got["bidx"] == 0).all()
    finally:
        sim.close()


def _es_case(lam, steps, seed):
    rng = np.random.default_rng(seed)
    reqs = small_trace(seed, n_req=500, n_sessions=20, rate_ms=25.0)
    w = W.handmade(rng.uniform(5, 120, size=3), reqs, slots=2, cache_blocks=14,
                   params=np.array([[0.5, 1.0, 0.1]]))
    tuned = np.array([0, 2], dtype=np.uint32)                 # W_rtt and W_queue (Section 4)
    lo, hi = np.array([0.05, 0.05]), np.array([2.0, 0.5])
    z = rng.standard_normal((steps, lam, 2))
    return w, tuned, lo, hi, z


@pytest.mark.parametrize("lam,steps,objective", [(1, 12, 0), (4, 8, 0), (3, 6, 1)])
def test_es_run_matches_oracle(lam, steps, objective):
    from paper_2602_11688_b200 import binding as gb
    w, tuned, lo, hi, z = _es_case(lam, steps, seed=7 + lam)
    x0 = np.array([0.5, 1.0, 0.1])
    scale = 0.6
    sim = gb.GorgoSim(w)
    try:
        sim.ensure_workspace(lam)
        rc, x, f, sigma, hist = gb.gorgo_es_run(sim.h, x0=x0, z=z, tuned=tuned, lo=lo, hi=hi,
                                                sigma0=0.5, sigma_up=1.5, n_steps=steps, lam=lam,
                                                workspace=sim.workspace, stream=sim.stream,
                                                time_scale=scale, objective=objective)
        assert rc == gb.GORGO_OK
    finally:
        sim.close()

    def obj(xv):
        _, p_ttft, p_e2e, _, _ = O.replay(w, np.array(xv), scale)
        return p_ttft if objective == 0 else p_e2e

    rx, rf, rsigma, rhist = T.es_run(obj, x0.tolist(), tuned.tolist(), lo.tolist(), hi.tolist(),
                                     0.5, 1.5, z.tolist())
    assert hist.shape == (steps, 6)
    for t, h in enumerate(rhist):
        assert hist[t, 0] == h[0], (t, "best offspring objective")
        assert bool(hist[t, 1]) == h[1], (t, "accepted")
        assert hist[t, 2] == h[2], (t, "sigma")
        assert hist[t, 3] == h[3], (t, "parent objective")
        assert hist[t, 4:].tolist() == h[4], (t, "parent weights")
    assert x.tolist() == rx and f == rf and sigma == rsigma


def test_es_run_rejects_bad_arguments():
    from paper_2602_11688_b200 import binding as gb
    w, tuned, lo, hi, z = _es_case(2, 2, seed=3)
    sim = gb.GorgoSim(w)
    try:
        sim.ensure_workspace(2)
        kw = dict(z=z, tuned=tuned, lo=lo, hi=hi, sigma0=0.5, sigma_up=1.5, n_steps=2, lam=2,
                  workspace=sim.workspace, stream=sim.stream)
        good = np.array([0.5, 1.0, 0.1])
        bad = gb.GORGO_ERR_INVALID_ARG
        assert gb.gorgo_es_run(sim.h, x0=np.array([0.5, 1.0, 0.0]), **kw)[0] == bad     # ln(0)
        assert gb.gorgo_es_run(sim.h, x0=good, **{**kw, "lo": np.array([0.0, 0.05])})[0] == bad
        assert gb.gorgo_es_run(sim.h, x0=good, **{**kw, "tuned": np.array([0, 3], np.uint32)})[0] == bad
        assert gb.gorgo_es_run(sim.h, x0=good, **{**kw, "sigma_up": 1.0})[0] == gb.GORGO_ERR_NONFINITE_PARAM
        zz = z.copy(); zz[0, 0, 0] = np.nan
        assert gb.gorgo_es_run(sim.h, x0=good, **{**kw, "z": zz})[0] == gb.GORGO_ERR_NONFINITE_PARAM
        assert gb.gorgo_es_run(sim.h, x0=good, **kw)[0] == gb.GORGO_OK
    finally:
        sim.close()


@pytest.mark.parametrize("workload,kw,scale,steps,start,accepts", [
    ("tiny", dict(n_requests=900, cache_blocks=300), 1.0, 40, [0.5, 1.0, 0.1], False),
    ("regions", dict(n_requests=1500, cache_blocks=500, population=4), 1.0, 40, [2.0, 1.0, 0.05], True),
])
def test_online_tuning_inside_one_replay_matches_oracle(workload, kw, scale, steps, start, accepts):
    """The paper's online tuner: weights change every 32 requests inside one replay.  Three tuners
    with their own draws run side by side in the library; each is compared with the oracle's
    chunked replay: every route, the whole strategy trajectory, final weights and p95s."""
    import torch
    from oracle import gorgo_oracle as O
    from oracle import gorgo_tuning as T
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload(workload, **kw)
    N, K = w.n_requests, w.n_params
    P = 3
    rng = np.random.default_rng(11)
    x0 = np.tile(np.array(start + [1.0] * (K - 3)), (P, 1))
    tuned, lo, hi = [0, 2], [0.05, 0.05], [2.0, 0.5]
    z = rng.normal(size=(P, steps, 2))
    sim = gb.GorgoSim(w)
    sim.ensure_workspace(P)
    route = torch.empty((P, N), dtype=torch.uint8, device="cuda")
    rc, x_fin, sig, done, hist, pt, pe = gb.gorgo_tune_online(
        sim.h, x0=x0, z=z, tuned=tuned, lo=lo, hi=hi, sigma0=0.5, sigma_up=1.5,
        workspace=sim.workspace, stream=sim.stream, time_scale=scale, route=route)
    assert rc == gb.GORGO_OK, gb.gorgo_strerror(rc)
    torch.cuda.synchronize()
    route = route.cpu().numpy()
    for p in range(P):
        o = O.Oracle.from_workload(w)
        routes, e2e = [], []

        def run_chunk(weights, count):
            r = o.run(np.array(weights), scale, count=count)
            routes.append(r.route); e2e.extend(r.e2e)
            return list(r.ttft)
        ttft, schedule, h = T.online_tune(run_chunk, N, list(x0[p]), tuned, lo, hi, 0.5, 1.5,
                                          z[p].tolist())
        assert done == len(h) == min(steps, T.window_count(N))
        assert (route[p] == np.concatenate(routes)).all()
        for k, (value, acc, sigma, f_par, par, live) in enumerate(h):
            assert hist[p, k].tolist() == [value, 1.0 if acc else 0.0, sigma, f_par] + par + live, (p, k)
        assert [x_fin[p, i] for i in tuned] == h[-1][4] and sig[p] == h[-1][2]
        assert pt[p] == O.p95(np.array(ttft)) and pe[p] == O.p95(np.array(e2e))
        o.close()
    if accepts:                                         # on this case some offspring do get accepted
        assert any(hist[p, 1:done, 1].sum() > 0 for p in range(P))
    sim.close()


def test_online_tuning_rejects_bad_arguments():
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload("tiny", n_requests=300, cache_blocks=100)
    sim = gb.GorgoSim(w)
    sim.ensure_workspace(1)
    x0 = np.array([[0.5, 1.0, 0.1]])
    z = np.zeros((1, 4, 2))
    ok = dict(x0=x0, z=z, tuned=[0, 2], lo=[0.05, 0.05], hi=[2.0, 0.5], sigma0=0.5, sigma_up=1.5,
              workspace=sim.workspace, stream=sim.stream)
    assert gb.gorgo_tune_online(sim.h, **ok)[0] == gb.GORGO_OK
    assert gb.gorgo_tune_online(sim.h, **{**ok, "sigma_up": 1.0})[0] == gb.GORGO_ERR_NONFINITE_PARAM
    assert gb.gorgo_tune_online(sim.h, **{**ok, "lo": [0.0, 0.05]})[0] == gb.GORGO_ERR_INVALID_ARG
    assert gb.gorgo_tune_online(sim.h, **{**ok, "tuned": [0, 7]})[0] == gb.GORGO_ERR_INVALID_ARG
    assert gb.gorgo_tune_online(sim.h, **{**ok, "window": 4096})[0] == gb.GORGO_ERR_INVALID_ARG
    assert gb.gorgo_tune_online(sim.h, **{**ok, "x0": np.array([[0.5, 1.0, -0.1]])})[0] == gb.GORGO_ERR_INVALID_ARG
    import torch
    small = torch.empty(4096, dtype=torch.uint8, device="cuda")
    assert gb.gorgo_tune_online(sim.h, **{**ok, "workspace": small})[0] == gb.GORGO_ERR_WORKSPACE_TOO_SMALL
    sim.close()
