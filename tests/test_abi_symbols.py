"""The shared library loads on a machine without a GPU and exports every function that
include/pie_b200.h declares (no compute call is made here)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "pie_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pie_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    import paper_2510_24051_b200 as pie
    names = declared_functions()
    assert len(names) >= 18
    lib = ctypes.CDLL(pie.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in pie_b200.h but not exported"
    for n in names:                               # the Python binding mirrors the C names
        assert hasattr(pie, n), f"binding lacks {n}"


def test_strerror_and_host_only_context():
    import paper_2510_24051_b200 as pie
    assert pie.pie_strerror(0) == "ok"
    assert "conflict" in pie.pie_strerror(pie.PIE_ERR_CONFLICT)
    ctx = pie.pie_create(16, 16, 4, 2, 64, "bf16", 4, 64, device=-1)
    try:
        ids = pie.pie_alloc_kvpages(ctx, 2)
        plan = pie.pie_plan_forward(ctx, [0, 1], [0, 2], ids, [3])
        # device work on a host-only context fails loudly instead of falling back to anything
        assert pie.lib.pie_forward(ctx, plan, 1, 1, 1, 1, 1, None) == pie.PIE_ERR_NO_DEVICE
        assert pie.lib.pie_copy_kvpage(ctx, 0, None, None, None, None, None, None) == pie.PIE_ERR_NO_DEVICE
        pie.pie_plan_destroy(plan)
    finally:
        pie.pie_destroy(ctx)
