"""The C-ABI library: loads, exports what the header declares, and its host-side logic
(validation, index decoding, sizes) behaves as documented.  No GPU work here."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2412_04788_b200 import build, guide, inputs as I

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    build.build()


def small_space(**over):
    w = I.workload(1)["space"]
    sp = dict(w)
    sp.update(over)
    return sp


def test_header_symbols_are_exported():
    text = open(os.path.join(ROOT, "include", "guide.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(guide_[a-z_]+)\s*\(", text))
    assert {"guide_space_create", "guide_trace_load", "guide_simulate", "guide_select_topk", "guide_pareto"} <= declared
    L = C.CDLL(guide.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(L, name), name
    assert set(guide.EXPORTS) == declared


def test_space_size_and_decode_follow_the_mixed_radix_order():
    sp = guide.Space(I.workload(1)["space"])
    assert sp.size == 504
    for idx in (0, 1, 6, 17, 18, 250, 503):
        got = sp.decode(idx)
        m, h, f, b, t, l = I.decode_index(I.workload(1)["space"], idx)
        assert (got["model"], got["hw"], got["fw"], got["batch_pos"], got["tp_pos"], got["pair_pos"]) == (m, h, f, b, t, l)
    w = I.workload(1)["space"]
    got = sp.decode(503)
    assert got["batch"] == 64 and got["tp"] == 4 and (got["lin"], got["lout"]) == tuple(w["pairs"][5])
    with pytest.raises(guide.GuideError) as e:
        sp.decode(504)
    assert e.value.code == guide.GUIDE_ERR_INVALID
    for k in range(2, 6):
        w = I.workload(k)
        assert guide.Space(w["space"]).size == I.space_size(w["space"])
    # the data-parallel degree rides on the TP axis: 1 everywhere when none is given
    assert {sp.decode(i)["dp"] for i in range(504)} == {1}
    w = I.hybrid_workload(8)["space"]
    hy = guide.Space(w)
    assert hy.size == I.space_size(w) == 8 * 8 * 3 * 12 * 15 * 64
    for idx in (0, 63, 64, 15 * 64 - 1, 1234567):
        got = hy.decode(idx)
        assert (got["dp"], got["tp"]) == (int(w["dp"][got["tp_pos"]]), int(w["tp"][got["tp_pos"]]))
        assert got["dp"] * got["tp"] <= 8
    with pytest.raises(ValueError):
        guide.Space(dict(w, dp=w["dp"][:3]))


def test_space_validation():
    bad = [
        (dict(tp=np.array([1, 3], np.uint32)), guide.GUIDE_ERR_UNSUPPORTED),          # not a power of two
        (dict(batch=np.array([0, 1], np.uint32)), guide.GUIDE_ERR_INVALID),
        (dict(pairs=np.array([[0, 4]], np.uint32)), guide.GUIDE_ERR_INVALID),
        (dict(batch=np.zeros(0, np.uint32)), guide.GUIDE_ERR_INVALID),                 # empty axis
        (dict(dp=np.array([1, 0, 1], np.uint32)), guide.GUIDE_ERR_INVALID),            # no replicas
        (dict(dp=np.array([1, 1, 65537], np.uint32)), guide.GUIDE_ERR_INVALID),
    ]
    for over, code in bad:
        with pytest.raises(guide.GuideError) as e:
            guide.Space(small_space(**over))
        assert e.value.code == code, over
        assert guide.guide_last_error()
    m = I.workload(1)["space"]["models"].copy()
    m[0, 1] = 4097                                                                      # hidden % heads != 0
    with pytest.raises(guide.GuideError):
        guide.Space(small_space(models=m))
    fw_i = I.workload(1)["space"]["fw_i"].copy()
    fw_i[0, 1] = 0                                                                      # kv_block 0
    with pytest.raises(guide.GuideError):
        guide.Space(small_space(fw_i=fw_i))
    hw = I.workload(1)["space"]["hw"].copy()
    hw[0, 0] = 0.0
    with pytest.raises(guide.GuideError):
        guide.Space(small_space(hw=hw))


def test_overflow_is_refused_at_create():
    big = np.array([[200, 2**20, 32, 32, 2**22, 2**20, 1, 2, 2, 2]], np.uint32)
    with pytest.raises(guide.GuideError) as e:
        guide.Space(small_space(models=big, batch=np.array([2**10], np.uint32), pairs=np.array([[2**20, 2]], np.uint32)))
    assert e.value.code == guide.GUIDE_ERR_OVERFLOW
    # the full-size workloads are far from the limit
    guide.Space(I.workload(5)["space"])


def test_trace_validation():
    ok = {"arrival": np.array([0.0, 0.5, 0.5]), "in_len": np.array([4, 0, 7], np.uint32), "out_len": np.array([2, 0, 1], np.uint32)}
    t = guide.Trace(ok)
    assert int(guide.lib().guide_trace_size(t.handle)) == 3
    for bad in (
        {"arrival": np.array([1.0, 0.5]), "in_len": np.array([4, 4], np.uint32), "out_len": np.array([2, 2], np.uint32)},
        {"arrival": np.array([-1.0]), "in_len": np.array([4], np.uint32), "out_len": np.array([2], np.uint32)},
        {"arrival": np.array([0.0]), "in_len": np.array([4], np.uint32), "out_len": np.array([0], np.uint32)},
        {"arrival": np.zeros(0), "in_len": np.zeros(0, np.uint32), "out_len": np.zeros(0, np.uint32)},
    ):
        with pytest.raises(guide.GuideError) as e:
            guide.Trace(bad)
        assert e.value.code == guide.GUIDE_ERR_INVALID


def test_workspace_sizes():
    sp = guide.Space(I.workload(1)["space"])
    tr = guide.Trace(I.workload(1)["trace"])
    assert guide.guide_workspace_bytes(sp, None) == 0
    w256 = guide.guide_workspace_bytes(sp, tr)
    assert w256 > 0 and w256 % 256 == 0
    big = guide.Trace(I.workload(3)["trace"])
    assert guide.guide_workspace_bytes(sp, big) > w256
    assert guide.guide_select_workspace_bytes(sp, 64) > 0
    assert guide.guide_select_workspace_bytes(sp, 0) == 0
    assert guide.guide_select_workspace_bytes(sp, 1025) == 0
    assert guide.guide_pareto_workspace_bytes(sp) > 0


def test_null_arguments_are_errors_not_crashes():
    L = guide.lib()
    assert L.guide_space_create(None, None) == guide.GUIDE_ERR_INVALID
    assert L.guide_simulate(None, None, None, None, None, 0, None) == guide.GUIDE_ERR_INVALID
    assert L.guide_select_topk(None, None, None, None, None, 0, 1, None, None, None, None, 0, None) == guide.GUIDE_ERR_INVALID
    assert L.guide_pareto(None, None, None, None, None, 0, 5, None, 0, None, None, 0, None) == guide.GUIDE_ERR_INVALID
    assert L.guide_space_size(None) == 0
    L.guide_space_destroy(None)
    L.guide_trace_destroy(None)
    sp = guide.Space(I.workload(1)["space"])
    out = guide.Outputs()
    # a range that runs off the end of the space is refused before any GPU work
    opts = guide.SimOpts(500, 10, 0, 0, 0)
    assert L.guide_simulate(sp.handle, None, C.byref(opts), C.byref(out), None, 0, None) == guide.GUIDE_ERR_INVALID
    # batch sizes above the trace kernel's residency limit
    w2 = I.workload(2)["space"]
    sp2 = guide.Space(w2)
    tr = guide.Trace(I.workload(1)["trace"])
    assert L.guide_simulate(sp2.handle, tr.handle, None, C.byref(out), None, 0, None) == guide.GUIDE_ERR_UNSUPPORTED
    # missing workspace for a trace run
    assert L.guide_simulate(sp.handle, tr.handle, None, C.byref(out), None, 0, None) == guide.GUIDE_ERR_WORKSPACE
    cons = guide._cons({})
    assert L.guide_select_topk(sp.handle, None, None, None, C.byref(cons), 0, 0, None, None, None, None, 0, None) == guide.GUIDE_ERR_INVALID
    assert L.guide_select_topk(sp.handle, tr.handle, None, None, C.byref(cons), 0, 4, None, None, None, None, 0, None) == guide.GUIDE_ERR_UNSUPPORTED


def test_simulate_select_refuses_bad_arguments_before_any_gpu_work():
    L = guide.lib()
    assert L.guide_simulate_select(None, None, None, None, None, 0, None, 0, None) == guide.GUIDE_ERR_INVALID
    sp = guide.Space(I.workload(1)["space"])
    out = guide.Outputs()
    cons = guide._cons({})
    sel = guide.Selection(C.pointer(cons), guide.METRICS["latency"], 4, None, None, None, C.pointer(cons),
                          guide.METRICS["latency"], guide.METRICS["cost_per_hr"], None, 0, None, None, None)
    # no status array among the outputs: the selections could not fall back on the arrays
    assert L.guide_simulate_select(sp.handle, None, C.byref(out), C.byref(sel), None, 0, None, 0, None) == guide.GUIDE_ERR_INVALID
    sel.key = 99
    assert L.guide_simulate_select(sp.handle, None, C.byref(out), C.byref(sel), None, 0, None, 0, None) == guide.GUIDE_ERR_INVALID
    opts = guide.SimOpts(0, 0, 0, 0, 0, 1, 0)                          # clamp_seq: the separate calls only
    assert L.guide_simulate_select(sp.handle, C.byref(opts), C.byref(out), C.byref(sel), None, 0, None, 0, None) == guide.GUIDE_ERR_UNSUPPORTED
    assert guide.guide_last_error()
