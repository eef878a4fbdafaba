"""Host checks of the synthetic workload generators that the benchmark and the GPU tests rely on (no attention
arithmetic lives there: shapes, page lists and masks only)."""
import numpy as np
import pytest

import paper_2510_24051_b200 as pie
from workloads import configs, synth


@pytest.mark.parametrize("name", ["batched_decode", "long_context_policy"])
def test_decode_loop_batches_are_valid_consecutive_steps(name):
    """Step s of a decode loop: every request one token longer than in step s - 1, a new page exactly when a page
    boundary is crossed (taken from the spare pages, never from another request), policy masks of the new length,
    the copy of the last page following it - and every step a batch the planner accepts."""
    wl = configs.small(name)
    total = wl.meta.get("pages_in_lists", len(wl.page_indices))
    perm = synth.permutation(wl.seed, 10, wl.num_pages)
    spare = perm[total + (wl.R if wl.copies is not None else 0):]
    steps = configs.decode_loop(wl, 40, spare)
    ctx = pie.pie_create(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype, wl.R, wl.T, device=-1)
    try:
        pie.pie_alloc_kvpages(ctx, wl.num_pages)
        kv0 = wl.kv_lens()
        seen = set(int(p) for p in wl.page_indices)
        for s, b in enumerate(steps):
            npages = np.diff(b["page_indptr"])
            kv = (npages - 1) * wl.P + b["last_page_len"]
            assert np.array_equal(kv, kv0 + s)
            assert len(set(b["page_indices"].tolist())) == len(b["page_indices"])          # no page in two lists
            new = set(b["page_indices"].tolist()) - seen
            assert new <= set(int(p) for p in spare)
            seen |= new
            if s == 0:
                assert np.array_equal(b["page_indices"], wl.page_indices) and np.array_equal(b["last_page_len"], wl.last_page_len)
            if wl.masks is not None:
                assert np.array_equal(np.diff(b["mask_indptr"]), kv)
                r = 1
                row = b["mask"][b["mask_indptr"][r]:b["mask_indptr"][r + 1]].astype(bool)
                assert row[:4].all() and row[-min(len(row), wl.meta["window"]):].all()        # sink and window are kept
            if b["copies"] is not None:
                last = b["page_indices"][b["page_indptr"][1:] - 1]
                assert np.array_equal(b["copies"]["src"], last) and np.array_equal(b["copies"]["ntok"], b["last_page_len"])
            plan = pie.pie_plan_forward(ctx, b["qo_indptr"], b["page_indptr"], b["page_indices"], b["last_page_len"],
                                        b["mask_indptr"], b["mask"])
            info = pie.pie_plan_get_info(plan)
            assert info["num_requests"] == wl.R and info["num_simple_rows"] == 0
            pie.pie_plan_destroy(plan)
    finally:
        pie.pie_destroy(ctx)


def test_batches_with_their_own_lengths_share_one_pool_without_overlap():
    """Several decode batches with different seeds (the independent loops of the end-to-end benchmark) placed one after
    the other in the same page permutation."""
    a = configs.batched_decode(R=12, lo=40, hi=700, num_pages=4096)
    b = configs.batched_decode(seed=a.seed + 100, R=12, lo=40, hi=700, num_pages=4096, perm_seed=a.seed,
                               page_offset=len(a.page_indices) + 50)
    assert not np.array_equal(a.kv_lens(), b.kv_lens())
    assert np.intersect1d(a.page_indices, b.page_indices).size == 0
    assert (b.page_owner[b.page_indices] >= 0).all()


def test_lazy_pool_prefetch_equals_page_by_page_generation():
    wl = configs.small("mixed_prefill_decode")
    one, many = wl.oracle_pool(), wl.oracle_pool()
    ids = wl.used_pages()[:9]
    many.prefetch(ids, chunk=4)
    for p in ids:
        K1, V1 = one[int(p)]
        K2, V2 = many[int(p)]
        assert np.array_equal(K1, K2) and np.array_equal(V1, V2)
