"""CPU-side checks of the C ABI: the library loads and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "bifrost.h")


def declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bf_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2606_17421_b200 import bifrost, build
    build.build()
    lib = ctypes.CDLL(bifrost.LIB_PATH)
    names = declared_symbols()
    assert len(names) >= 15
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(bifrost.exported_symbols()) == names      # the binding covers the whole header


def test_strerror_needs_no_device():
    from paper_2606_17421_b200 import bifrost
    assert bifrost.bf_strerror(0) == "ok"
    assert "key" in bifrost.bf_strerror(bifrost.BF_ERR_MISSING_KEY)


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2606_17421_b200 import bifrost
    monkeypatch.setattr(bifrost, "_lib", None)
    monkeypatch.setattr(bifrost, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libbifrost.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        bifrost.load()


def test_workload_splits_name_calls_and_factor_the_diagonals():
    # the per-call baby/giant splits of the workloads: every name is a call the runner issues (projections that
    # share an input joined with "+"), b and g are powers of two with b * g = D / tau, within what one launch holds,
    # and only the plan variant they were measured under takes them
    from paper_2606_17421_b200 import workloads as wl
    for name, w in wl.WORKLOADS.items():
        calls = {nm for nm, _, _ in wl.fuse_shared_inputs(w.layers, w.plan.D)}
        for call, (b, g) in w.splits.items():
            assert call in calls, (name, call)
            assert b * g == w.plan.D // w.plan.tau, (name, call)
            assert b & (b - 1) == 0 and g & (g - 1) == 0 and 1 <= b - 1 <= 64 and g - 1 <= 64, (name, call)
        headline = wl.PlanSpec(w.plan.D, w.plan.tau, w.plan.b, w.plan.g, "complex", "per_output", "double")
        for call in calls:
            assert w.split_of(call, w.plan) == (w.plan.b, w.plan.g)
            assert w.split_of(call, headline) == w.splits.get(call, (w.plan.b, w.plan.g))
