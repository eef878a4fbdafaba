"""What ptxas reported for the kernels of the hot path in the build under test: a spill in one of them is a
performance bug that no parity test sees (a merge routine inlined at the end of the decode kernel's item loop, and
the same routine as a call of its own, each made that loop spill and cost it up to half its speed)."""
from paper_2510_24051_b200 import build


def test_hot_kernels_do_not_spill():
    build.build()
    res = build.kernel_resources()
    assert res, "no ptxas record: the library was not built by paper_2510_24051_b200.build"
    split = {k: v for k, v in res.items() if "attn_split_kernel" in k}
    tc = {k: v for k, v in res.items() if "attn_tc_kernel" in k}
    nd = {k: v for k, v in res.items() if "next_dist" in k}
    assert len(split) == 8 and len(tc) == 6 and len(nd) >= 5          # every instantiation the launchers name
    for name, v in split.items():
        assert v["spill_stores"] == 0 and v["stack"] == 0, (name, v)
        assert v["registers"] <= 232, (name, v)                      # one block of 8 warps per SM, with room for the loop's temporaries
    for name, v in tc.items():
        assert v["spill_stores"] <= 16 and v["registers"] <= 168, (name, v)   # 11 warps per block: 168 is the most the SM's register file allows
    for name, v in nd.items():
        assert v["spill_stores"] == 0 and v["registers"] <= 64, (name, v)
