"""Host-only checks of the C-ABI library: it loads, exports every function the header declares,
and rejects bad arguments before touching a device."""
import ctypes as C
import os
import re

import numpy as np

from paper_2602_11688_b200 import binding as gb
from paper_2602_11688_b200 import build as gbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "gorgo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gorgo_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    gbuild.build()
    lib = gb.load()
    names = declared_functions()
    assert "gorgo_eval_population" in names and "gorgo_route_batch" in names
    assert "gorgo_sim_create" in names and "gorgo_trace_upload" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(gb.EXPORTS) == names


def test_strerror_and_size_queries_need_no_device():
    assert gb.gorgo_strerror(0) == "ok"
    assert "trace" in gb.gorgo_strerror(gb.GORGO_ERR_BAD_TRACE)
    assert gb.gorgo_strerror(-99).startswith("unknown")
    rc, n = gb.gorgo_trace_bytes(1000, 50_000)
    assert rc == gb.GORGO_OK
    assert n >= 1000 * 32 + 50_000 * (4 + 8 + 8) and n % 256 == 0


def test_null_and_out_of_range_arguments_are_rejected_on_the_host():
    lib = gb.load()
    h = C.c_void_p()
    assert lib.gorgo_sim_create(None, C.byref(h)) == gb.GORGO_ERR_INVALID_ARG
    rtt = np.array([[10.0, 20.0]])
    base = dict(n_replicas=2, n_regions=1, slots_per_replica=4, block_tokens=512,
                cache_blocks=100, n_params=3, prefill_ms_per_token=0.05, tpot_ms=20.0)
    for bad in (dict(n_replicas=0), dict(n_replicas=65), dict(slots_per_replica=0),
                dict(block_tokens=0), dict(cache_blocks=0), dict(n_params=4),
                dict(prefill_ms_per_token=float("nan")), dict(tpot_ms=-1.0)):
        rc, h = gb.gorgo_sim_create(rtt_ms=rtt, **{**base, **bad})
        assert rc == gb.GORGO_ERR_INVALID_ARG, bad
    rc, h = gb.gorgo_sim_create(rtt_ms=np.array([[10.0, float("inf")]]), **base)
    assert rc == gb.GORGO_ERR_INVALID_ARG
    assert lib.gorgo_sim_destroy(None) == gb.GORGO_ERR_INVALID_ARG
    assert lib.gorgo_trace_bytes(1, 1, None) == gb.GORGO_ERR_INVALID_ARG
    out = C.c_uint64()
    assert lib.gorgo_workspace_bytes(None, 1, C.byref(out)) == gb.GORGO_ERR_INVALID_ARG
    assert lib.gorgo_state_bytes(None, C.byref(out)) == gb.GORGO_ERR_INVALID_ARG
    assert lib.gorgo_eval_population(None, 1, None, 1.0, None, 0, None, None, None, None, None,
                                     None, None, None) == gb.GORGO_ERR_INVALID_ARG
    assert lib.gorgo_route_batch(None, None, 1.0, 0, 0, None, 0, None, None, None, None,
                                 None) == gb.GORGO_ERR_INVALID_ARG
