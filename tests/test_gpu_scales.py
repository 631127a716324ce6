"""GPU parity of gorgo_eval_population_scales (one time scale per candidate; paper Section 3: the
time between requests is scaled linearly) against the CPU oracle run once per (weights, scale)."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

from oracle import gorgo_oracle as O
from paper_2602_11688_b200 import workloads as W
from tests.util import small_trace


def _run(sim, params, scales, resident=None):
    import torch
    from paper_2602_11688_b200 import binding as gb
    P = params.shape[0]
    sim.ensure_workspace(P if resident is None else resident)
    dev = sim.device
    pt = torch.zeros(P, dtype=torch.float64, device=dev)
    pe = torch.zeros(P, dtype=torch.float64, device=dev)
    route = torch.full((P, sim.N), 255, dtype=torch.uint8, device=dev)
    hit = torch.zeros((P, sim.N), dtype=torch.uint16, device=dev)
    dg = torch.zeros((P, sim.R, 2), dtype=torch.uint64, device=dev)
    st = torch.zeros(P, dtype=torch.int32, device=dev)
    rc = gb.gorgo_eval_population_scales(sim.h, P, params, scales, sim.workspace, sim.stream, pt, pe,
                                         route, hit, dg, st)
    torch.cuda.synchronize()
    return rc, pt.cpu().numpy(), pe.cpu().numpy(), route.cpu().numpy(), hit.cpu().numpy(), \
        dg.cpu().numpy(), st.cpu().numpy()


@pytest.mark.parametrize("resident", [None, 3])           # all at once, and in waves of three
def test_scale_sweep_as_one_population(resident):
    from paper_2602_11688_b200 import binding as gb
    rng = np.random.default_rng(21)
    reqs = small_trace(21, n_req=500, rate_ms=20.0)
    base = rng.normal(1.0, 0.3, size=(2, 3))
    w = W.handmade(rng.uniform(5, 80, size=5), reqs, slots=2, cache_blocks=11, params=base)
    sweep = [1.0, 0.75, 0.5, 0.35, 0.25]                  # the saturation sweep's scale factors
    params = np.repeat(base, len(sweep), axis=0)          # candidate = (weights, scale)
    scales = np.tile(np.array(sweep), base.shape[0])
    sim = gb.GorgoSim(w)
    try:
        rc, pt, pe, route, hit, dg, st = _run(sim, params, scales, resident)
        assert rc == gb.GORGO_OK and (st == 0).all()
        # the same through the single-scale entry point, one call per scale
        for s in (1.0, 0.25):
            one = sim.eval_population(base, s, want_route=True)
            import torch
            torch.cuda.synchronize()
            idx = [p for p in range(params.shape[0]) if scales[p] == s]
            assert one["route"].cpu().numpy().tolist() == route[idx].tolist()
            assert one["p95_ttft"].cpu().numpy().tolist() == pt[idx].tolist()
    finally:
        sim.close()
    for p in range(params.shape[0]):
        res, p_ttft, p_e2e, ref_dg, _ = O.replay(w, params[p], float(scales[p]))
        assert route[p].tolist() == res.route.tolist(), p
        assert hit[p].tolist() == res.hit.tolist(), p
        assert dg[p].tolist() == ref_dg.tolist(), p
        assert abs(pt[p] - p_ttft) <= 1e-9 * abs(p_ttft) and abs(pe[p] - p_e2e) <= 1e-9 * abs(p_e2e)
    # a lighter load (larger scale) never queues more: p95 TTFT at scale 1 <= at scale 0.25
    assert pt[0] <= pt[4] and pt[5] <= pt[9]


def test_scales_are_checked():
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload("tiny", n_requests=200, population=2)
    sim = gb.GorgoSim(w)
    try:
        assert _run(sim, w.params, np.array([1.0, np.nan]))[0] == gb.GORGO_ERR_NONFINITE_PARAM
        assert _run(sim, w.params, np.array([1.0, -0.5]))[0] == gb.GORGO_ERR_NONFINITE_PARAM
        assert _run(sim, w.params, np.array([1.0, 0.0]))[0] == gb.GORGO_OK
    finally:
        sim.close()
