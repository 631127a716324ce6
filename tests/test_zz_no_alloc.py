"""The allocation-free entry point, gorgo_eval_population_static, against the ordinary one.

Some users of the library cannot hand it a workspace because they cannot allocate one: a plugin
that only receives its input and output buffers, code living inside a memory plan that is already
fully carved up, or a control loop that must not pay cudaMalloc's device-wide synchronisation.
For them the replay scratch is an array built into the library.  This file runs last on purpose
(its name sorts after the other test files), so a run that stops at the first failure has already
exercised everything else.  Two calls in a row share that array: the second must not see what the
first left behind."""
import numpy as np
import pytest

from paper_2602_11688_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _eval_with_workspace(gb, sim, params, scale):
    out = sim.eval_population(params, scale, want_route=True, want_hit=True)
    sim.torch.cuda.synchronize()
    return {k: out[k].cpu().numpy() for k in ("p95_ttft", "p95_e2e", "route", "hit")}


def _eval_static(gb, sim, params, scale):
    torch = sim.torch
    P = params.shape[0]
    a = torch.empty(P, dtype=torch.float64, device="cuda")
    b = torch.empty(P, dtype=torch.float64, device="cuda")
    route = torch.empty((P, sim.N), dtype=torch.uint8, device="cuda")
    hit = torch.empty((P, sim.N), dtype=torch.uint16, device="cuda")
    status = torch.full((P,), 77, dtype=torch.int32, device="cuda")
    rc = gb.gorgo_eval_population_static(sim.h, P, np.ascontiguousarray(params), scale,
                                         sim.stream, a, b, route, hit, status)
    assert rc == gb.GORGO_OK, gb.gorgo_strerror(rc)
    torch.cuda.synchronize()
    assert (status.cpu().numpy() == 0).all()                 # every candidate reports a clean replay
    return {"p95_ttft": a.cpu().numpy(), "p95_e2e": b.cpu().numpy(),
            "route": route.cpu().numpy(), "hit": hit.cpu().numpy()}


def _same(got, want):
    assert (got["route"] == want["route"]).all()            # integer work: bit-exact
    assert (got["hit"] == want["hit"]).all()
    for k in ("p95_ttft", "p95_e2e"):                        # fp64: the tolerance of the parity tests
        assert np.all(np.abs(got[k] - want[k]) <= 1e-9 * np.abs(want[k])), k


def test_static_scratch_entry_point_matches_the_workspace_one_twice_in_a_row():
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload("regions", n_requests=8_000, cache_blocks=1_500, population=24)
    sim = gb.GorgoSim(w)
    rc, one = gb.gorgo_workspace_bytes(sim.h, 1)
    assert rc == gb.GORGO_OK and one <= gb.GORGO_STATIC_SCRATCH_BYTES
    first, second = w.params[:24], w.params[::-1][:24] * np.array([1.0, 0.5, 2.0])
    want1 = _eval_with_workspace(gb, sim, first, 1.0)
    want2 = _eval_with_workspace(gb, sim, second, 0.5)
    _same(_eval_static(gb, sim, first, 1.0), want1)
    _same(_eval_static(gb, sim, second, 0.5), want2)         # the array still holds call 1's state
    _same(_eval_static(gb, sim, first, 1.0), want1)
    sim.close()


def test_static_scratch_entry_point_allocates_no_device_memory():
    """What the entry point is for: after a first call (which looks up the built-in array's address)
    a call leaves the free device memory reported by the driver, and torch's own allocator, exactly
    as it found them."""
    import torch
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload("regions", n_requests=4_000, cache_blocks=800, population=8)
    sim = gb.GorgoSim(w)
    P = w.params.shape[0]
    a = torch.empty(P, dtype=torch.float64, device="cuda")
    b = torch.empty(P, dtype=torch.float64, device="cuda")
    status = torch.zeros(P, dtype=torch.int32, device="cuda")
    params = np.ascontiguousarray(w.params)
    assert gb.gorgo_eval_population_static(sim.h, P, params, 1.0, sim.stream, a, b, None, None,
                                           status) == gb.GORGO_OK
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(3):
        assert gb.gorgo_eval_population_static(sim.h, P, params, 1.0, sim.stream, a, b, None, None,
                                               status) == gb.GORGO_OK
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == (alloc0, reserved0)
    assert (status.cpu().numpy() == 0).all()
    sim.close()


def test_static_scratch_entry_point_reports_a_replay_that_gave_up():
    """A candidate whose replay runs into one of the kernel's bounded waits must be visible to a
    caller of this entry point too: with the wait bound set to zero (test switch) the status array
    says so, and nothing faults or hangs."""
    import torch
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload("tiny", n_requests=300, cache_blocks=200, population=4)
    sim = gb.GorgoSim(w)
    P = w.params.shape[0]
    a = torch.empty(P, dtype=torch.float64, device="cuda")
    b = torch.empty(P, dtype=torch.float64, device="cuda")
    status = torch.zeros(P, dtype=torch.int32, device="cuda")
    assert gb.gorgo_debug_set(sim.h, gb.GORGO_DEBUG_POLL_LIMIT, 0) == gb.GORGO_OK
    rc = gb.gorgo_eval_population_static(sim.h, P, np.ascontiguousarray(w.params), 1.0, sim.stream,
                                         a, b, None, None, status)
    assert rc == gb.GORGO_OK                                  # the call only enqueues work
    torch.cuda.synchronize()
    assert (status.cpu().numpy() == gb.GORGO_ERR_DEVICE_LIMIT).all()
    assert gb.gorgo_debug_set(sim.h, gb.GORGO_DEBUG_POLL_LIMIT, 1 << 24) == gb.GORGO_OK
    rc = gb.gorgo_eval_population_static(sim.h, P, np.ascontiguousarray(w.params), 1.0, sim.stream,
                                         a, b, None, None, status)
    torch.cuda.synchronize()
    assert rc == gb.GORGO_OK and (status.cpu().numpy() == 0).all()
    sim.close()


def test_static_scratch_entry_point_runs_in_waves_when_the_population_does_not_fit_at_once():
    from paper_2602_11688_b200 import binding as gb
    w = W.make_workload("longctx", n_requests=60_000, cache_blocks=8_000, population=40)
    sim = gb.GorgoSim(w)
    rc, one = gb.gorgo_workspace_bytes(sim.h, 1)
    rc, all_ = gb.gorgo_workspace_bytes(sim.h, 40)
    assert one <= gb.GORGO_STATIC_SCRATCH_BYTES < all_      # several waves are needed
    want = _eval_with_workspace(gb, sim, w.params, 0.5)
    _same(_eval_static(gb, sim, w.params, 0.5), want)
    sim.close()


def test_static_scratch_entry_point_refuses_a_trace_beyond_its_limit():
    import torch
    from paper_2602_11688_b200 import binding as gb
    N = 2_200_000                                            # ~41 bytes of scratch per request
    spec = W.WorkloadSpec(name="too-long", seed=0, n_replicas=2, n_regions=1, n_requests=N,
                          n_sessions=1, cache_blocks=8, slots=2, population=1)
    w = W.Workload(spec=spec, rtt_ms=np.array([[10.0, 20.0]]),
                   ts_ms=np.arange(N, dtype=np.float64),
                   input_tokens=np.zeros(N, np.uint32), output_tokens=np.ones(N, np.uint32),
                   origin=np.zeros(N, np.uint16), hash_off=np.zeros(N + 1, np.uint64),
                   hash_ids=np.zeros(0, np.uint64), params=np.ones((1, 3)),
                   session=np.zeros(N, np.uint32), turn=np.zeros(N, np.uint32))
    sim = gb.GorgoSim(w)
    rc, one = gb.gorgo_workspace_bytes(sim.h, 1)
    assert one > gb.GORGO_STATIC_SCRATCH_BYTES
    a = torch.full((1,), -1.0, dtype=torch.float64, device="cuda")
    b = torch.full((1,), -1.0, dtype=torch.float64, device="cuda")
    rc = gb.gorgo_eval_population_static(sim.h, 1, w.params, 1.0, sim.stream, a, b)
    assert rc == gb.GORGO_ERR_STATIC_LIMIT
    assert "scratch" in gb.gorgo_strerror(rc)
    torch.cuda.synchronize()
    assert a.item() == -1.0 and b.item() == -1.0             # nothing ran
    sim.close()
