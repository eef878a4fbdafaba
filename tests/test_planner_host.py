"""Host logic of the library on a host-only context: allocator, batch validation (the
vertical-batching conflict rule, size limits), mask packing, page dropping, append positions."""
import numpy as np
import pytest

import paper_2510_24051_b200 as pie
from workloads import configs


@pytest.fixture
def ctx():
    c = pie.pie_create(256, 16, 8, 2, 64, "bf16", 8, 256, device=-1)
    yield c
    pie.pie_destroy(c)


def status_of(fn, *a, **k):
    try:
        fn(*a, **k)
    except pie.PieError as e:
        return e.status
    return pie.PIE_OK


def test_allocator_fcfs_and_errors(ctx):
    a = pie.pie_alloc_kvpages(ctx, 200)
    assert len(set(a.tolist())) == 200 and pie.pie_num_free_kvpages(ctx) == 56
    assert status_of(pie.pie_alloc_kvpages, ctx, 57) == pie.PIE_ERR_NO_PAGES      # nothing allocated
    assert pie.pie_num_free_kvpages(ctx) == 56
    pie.pie_dealloc_kvpages(ctx, a[:10])
    assert pie.pie_num_free_kvpages(ctx) == 66
    assert status_of(pie.pie_dealloc_kvpages, ctx, a[:1]) == pie.PIE_ERR_BAD_PAGE  # double free
    assert status_of(pie.pie_dealloc_kvpages, ctx, [a[20], a[20]]) == pie.PIE_ERR_BAD_PAGE
    assert status_of(pie.pie_dealloc_kvpages, ctx, [999]) == pie.PIE_ERR_BAD_PAGE
    assert pie.pie_num_free_kvpages(ctx) == 66
    assert len(pie.pie_alloc_kvpages(ctx, 0)) == 0


def test_validation_errors(ctx):
    ids = pie.pie_alloc_kvpages(ctx, 32)
    ok = lambda **k: status_of(pie.pie_plan_forward, ctx, **k)
    base = dict(qo_indptr=[0, 1, 3], page_indptr=[0, 2, 4], page_indices=ids[:4], last_page_len=[5, 16])
    assert ok(**base) == pie.PIE_OK
    assert ok(**dict(base, last_page_len=[0, 16])) == pie.PIE_ERR_INVALID
    assert ok(**dict(base, last_page_len=[5, 17])) == pie.PIE_ERR_INVALID
    assert ok(**dict(base, qo_indptr=[0, 0, 3])) == pie.PIE_ERR_INVALID            # q_len < 1
    assert ok(qo_indptr=[0, 20], page_indptr=[0, 1], page_indices=ids[:1], last_page_len=[16]) == pie.PIE_ERR_INVALID  # kv_len < q_len
    assert ok(**dict(base, page_indices=[ids[0], 250, ids[2], ids[3]])) == pie.PIE_ERR_BAD_PAGE  # not allocated
    assert ok(**dict(base, page_indices=[ids[0], -1, ids[2], ids[3]])) == pie.PIE_ERR_BAD_PAGE
    # batch size limits (the scheduler truncates; the library refuses)
    R = 9
    assert ok(qo_indptr=np.arange(R + 1), page_indptr=np.arange(R + 1), page_indices=ids[:R],
              last_page_len=np.ones(R)) == pie.PIE_ERR_BATCH_TOO_LARGE
    assert ok(qo_indptr=[0, 257], page_indptr=[0, 17], page_indices=ids[:17], last_page_len=[16]) == pie.PIE_ERR_BATCH_TOO_LARGE
    # mask of the wrong size / with a byte that is not 0 or 1
    assert ok(**dict(base, mask_indptr=[0, 0, 10], mask=np.ones(10, np.uint8))) == pie.PIE_ERR_MASK
    m = np.ones(2 * 32, np.uint8)
    assert ok(**dict(base, mask_indptr=[0, 0, 64], mask=m)) == pie.PIE_OK
    m[5] = 2
    assert ok(**dict(base, mask_indptr=[0, 0, 64], mask=m)) == pie.PIE_ERR_MASK
    # an empty batch plans to nothing
    assert ok(qo_indptr=[0], page_indptr=[0], page_indices=[], last_page_len=[]) == pie.PIE_OK


def test_conflict_rule(ctx):
    ids = pie.pie_alloc_kvpages(ctx, 8)
    plan = lambda **k: status_of(pie.pie_plan_forward, ctx, **k)
    # two requests append into the same slot of a shared last page
    assert plan(qo_indptr=[0, 1, 2], page_indptr=[0, 2, 4], page_indices=[ids[0], ids[1], ids[2], ids[1]],
                last_page_len=[4, 4]) == pie.PIE_ERR_CONFLICT
    # request 1 reads (as context) a slot the EARLIER request 0 appends: legal, the whole batch is
    # appended before anyone attends (the split forward of Section 4.2 as one batch) ...
    assert plan(qo_indptr=[0, 1, 2], page_indptr=[0, 1, 3], page_indices=[ids[0], ids[0], ids[2]],
                last_page_len=[4, 4]) == pie.PIE_OK
    # ... but reading a slot that a LATER request of the batch appends is a conflict
    assert plan(qo_indptr=[0, 1, 2], page_indptr=[0, 2, 3], page_indices=[ids[0], ids[2], ids[0]],
                last_page_len=[4, 4]) == pie.PIE_ERR_CONFLICT
    # sharing read-only pages is legal; so is reading slots below the other request's write
    assert plan(qo_indptr=[0, 1, 2], page_indptr=[0, 2, 4], page_indices=[ids[0], ids[1], ids[0], ids[2]],
                last_page_len=[4, 4]) == pie.PIE_OK
    assert plan(qo_indptr=[0, 1, 2], page_indptr=[0, 1, 3], page_indices=[ids[0], ids[3], ids[0]],
                last_page_len=[9, 3]) == pie.PIE_ERR_CONFLICT   # req 1 appends slot 2, the earlier req 0 reads slots 0..8
    # a request that lists the same page twice and would write it through both positions
    assert plan(qo_indptr=[0, 20], page_indptr=[0, 2], page_indices=[ids[4], ids[4]],
                last_page_len=[16]) == pie.PIE_ERR_CONFLICT
    # copy_kvpage conflicts are found on the host too
    assert status_of(pie.pie_copy_kvpage, ctx, [ids[0], ids[1]], [ids[2], ids[2]], [0, 0], [0, 4], [8, 8]) == pie.PIE_ERR_CONFLICT
    assert status_of(pie.pie_copy_kvpage, ctx, [ids[0]], [ids[0]], [0], [4], [8]) == pie.PIE_ERR_CONFLICT
    assert status_of(pie.pie_copy_kvpage, ctx, [ids[0]], [ids[1]], [10], [0], [8]) == pie.PIE_ERR_INVALID
    assert status_of(pie.pie_copy_kvpage, ctx, [ids[0]], [200], [0], [0], [8]) == pie.PIE_ERR_BAD_PAGE


@pytest.mark.parametrize("name", ["tiny_fp32", "shared_prefix_tree", "long_context_policy", "mixed_prefill_decode",
                                  "long_context_policy_full", "long_context_policy_p8", "long_context_policy_p32"])
def test_plan_arrays_match_numpy(name):
    # (the full-size batches list enough pages and mask bytes for the planner's worker threads, and walk the
    #  one-bit-per-page words of all three page sizes)
    big = {"long_context_policy_full": dict(), "long_context_policy_p8": dict(R=64, P=8), "long_context_policy_p32": dict(P=32)}
    wl = configs.long_context_policy(**big[name]) if name in big else configs.small(name)
    ctx = pie.pie_create(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype, wl.R, wl.T, device=-1)
    try:
        pie.pie_alloc_kvpages(ctx, wl.num_pages)
        mi, mb = wl.mask_bytes()
        plan = pie.pie_plan_forward(ctx, wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len, mi, mb)
        info = pie.pie_plan_get_info(plan)
        words = pie.pie_plan_debug_read(plan, 0)
        kept = pie.pie_plan_debug_read(plan, 1).reshape(-1, 2)
        app = pie.pie_plan_debug_read(plan, 2)
        pie.pie_plan_destroy(plan)
    finally:
        pie.pie_destroy(ctx)
    kv, ql, P = wl.kv_lens(), wl.q_lens(), wl.P
    # append destinations = the oracle's positions
    exp = []
    for r in range(wl.R):
        for i in range(ql[r]):
            pos = kv[r] - ql[r] + i
            exp.append(int(wl.pages_of(r)[pos // P]) * P + pos % P)
    assert app.tolist() == exp
    # packed masks: LSB first, rows padded to 128 bits; kept pages: exactly those some row attends to
    woff, koff = 0, 0
    for r in range(wl.R):
        m = None if wl.masks is None else wl.masks[r]
        npg = len(wl.pages_of(r))
        if m is None:
            keep = np.ones(npg, bool)
            lim0 = kv[r] - ql[r]
            needs = np.array([lp * P + P - 1 > lim0 for lp in range(npg)])
        else:
            rw = ((kv[r] + 127) // 128) * 4
            padded = np.zeros((ql[r], rw * 32), np.uint8)
            padded[:, :kv[r]] = m
            expw = np.packbits(padded, axis=1, bitorder="little").view(np.uint32).reshape(ql[r], rw)
            assert np.array_equal(words[woff:woff + ql[r] * rw].reshape(ql[r], rw), expw)
            woff += ql[r] * rw
            pg = padded[:, :npg * P].reshape(ql[r], npg, P)
            keep = pg.any(axis=(0, 2))
            needs = ~pg.all(axis=(0, 2))
        n = int(keep.sum())
        got = kept[koff:koff + n]
        assert np.array_equal(got[:, 0], wl.pages_of(r)[keep])
        assert np.array_equal(got[:, 1] & 0x7FFFFFFF, np.nonzero(keep)[0])
        assert np.array_equal((got[:, 1] < 0), needs[keep])
        koff += n
    assert koff == info["kept_pages"] and woff == info["mask_words"]


def test_mask_kvpage_is_anded_into_packed_rows_and_drops_hidden_pages():
    wl = configs.small("mixed_prefill_decode")
    ctx = pie.pie_create(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype, wl.R, wl.T, device=-1)
    try:
        pie.pie_alloc_kvpages(ctx, wl.num_pages)
        rng = np.random.RandomState(5)
        r = 4                                             # a decode request with several pages
        pages = wl.pages_of(r)
        pm = {int(pages[0]): 0x0000, int(pages[1]): 0x0F0F, int(pages[2]): 0xFFFF}
        pie.pie_mask_kvpage(ctx, list(pm), list(pm.values()))
        assert status_of(pie.pie_mask_kvpage, ctx, [wl.num_pages + 5], [1]) == pie.PIE_ERR_BAD_PAGE
        plan = pie.pie_plan_forward(ctx, wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len)
        words = pie.pie_plan_debug_read(plan, 0)
        kept = pie.pie_plan_debug_read(plan, 1).reshape(-1, 2)
        pie.pie_plan_destroy(plan)
        kv, ql, P = int(wl.kv_lens()[r]), int(wl.q_lens()[r]), wl.P
        assert ql == 1
        rw = ((kv + 127) // 128) * 4
        assert len(words) == rw                           # only the page-masked request got packed rows
        exp = np.zeros(rw * 32, np.uint8)
        exp[:kv] = 1                                      # inferred causal row of a decode: everything
        exp[0:P] = 0
        exp[P:2 * P] = [(0x0F0F >> s) & 1 for s in range(P)]
        assert np.array_equal(words, np.packbits(exp, bitorder="little").view(np.uint32))
        k0 = int(np.sum(np.diff(wl.page_indptr)[:r]))     # earlier requests keep all their pages
        mine = kept[k0:k0 + len(pages) - 1]
        assert np.array_equal(mine[:, 0], pages[1:])      # the fully hidden first page is dropped
        assert mine[0, 1] < 0 and mine[1, 1] >= 0         # partially hidden page needs mask bits, visible one not
        # re-allocating a page resets its mask
        pie.pie_dealloc_kvpages(ctx, [pages[1]])
        again = pie.pie_alloc_kvpages(ctx, 1)
        assert again[0] == pages[1]
        plan = pie.pie_plan_forward(ctx, wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len)
        w2 = pie.pie_plan_debug_read(plan, 0)
        pie.pie_plan_destroy(plan)
        exp[P:2 * P] = 1
        assert np.array_equal(w2, np.packbits(exp, bitorder="little").view(np.uint32))
    finally:
        pie.pie_destroy(ctx)


def test_shared_prefix_cascade_planning():
    """Decode requests that share a prompt's pages: the planner gathers their rows into row-tile
    work on the shared pages (once per group and kv head) and leaves each request only its
    private pages on the split-KV path; every (request, kv head) becomes a merge group."""
    def plan_info(wl, flags):
        c = pie.pie_create(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype, wl.R, wl.T, device=-1)
        try:
            pie.pie_alloc_kvpages(c, wl.num_pages)
            mi, mb = wl.mask_bytes()
            plan = pie.pie_plan_forward(c, wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len, mi, mb, flags)
            info = pie.pie_plan_get_info(plan)
            pie.pie_plan_destroy(plan)
            return info
        finally:
            pie.pie_destroy(c)

    small = configs.small("shared_prefix_decode")
    forced = plan_info(small, pie.PIE_PLAN_CASCADE_ALWAYS)
    assert forced["num_tile_items"] >= small.meta["groups"] * small.H_kv      # one row tile per (group, kv head), maybe cut
    assert forced["num_merge_groups"] == small.R * small.H_kv
    assert forced["launches"] == 4                                             # append, row tiles, split-KV, merge
    for flags in (0, pie.PIE_PLAN_NO_CASCADE):                                 # too small a saving / switched off
        info = plan_info(small, flags)
        assert info["num_tile_items"] == 0
    full = configs.shared_prefix_decode()
    auto = plan_info(full, 0)
    off = plan_info(full, pie.PIE_PLAN_NO_CASCADE)
    assert auto["num_tile_items"] > 0 and off["num_tile_items"] == 0
    assert auto["num_merge_groups"] == full.R * full.H_kv
    # token trees of 64 nodes fill a row tile per request (256 rows): they stay whole, shared pages served from L2
    tree64 = configs.shared_prefix_tree(groups=2, branches=3, prefix=256, suffix=32, tree=64, num_pages=256)
    assert plan_info(tree64, pie.PIE_PLAN_CASCADE_ALWAYS) == plan_info(tree64, pie.PIE_PLAN_NO_CASCADE)
    # trees of 32 nodes fill half a tile (128 rows): their rows are gathered over the shared prefix as well, and the
    # private pages run as row-tile items of their own - when the group fills a tile and shares >= 1,024 tokens
    tree32 = configs.small("shared_prefix_tree")
    forced = plan_info(tree32, pie.PIE_PLAN_CASCADE_ALWAYS)
    assert forced["num_merge_groups"] == tree32.R * tree32.H_kv and forced["num_split_items"] == 0
    assert forced["launches"] == 3                                             # append, row tiles, merge
    assert plan_info(tree32, 0) == plan_info(tree32, pie.PIE_PLAN_NO_CASCADE)  # 256 shared tokens: too few
    mid = configs.shared_prefix_tree(groups=2, branches=4, prefix=1024, suffix=48, tree=32, num_pages=512)
    auto = plan_info(mid, 0)
    assert auto["num_merge_groups"] == mid.R * mid.H_kv and plan_info(mid, pie.PIE_PLAN_NO_CASCADE)["num_merge_groups"] == 0


@pytest.mark.parametrize("name", ["long_context_policy", "shared_prefix_tree", "mixed_prefill_decode", "batched_decode"])
def test_recycled_plans_equal_fresh_ones(name):
    """pie_plan_destroy parks the plan object and pie_plan_forward reuses it: whatever batch the object held
    before, the image a reused object produces must be byte for byte the one a new context produces."""
    wl = configs.small(name)
    mi, mb = wl.mask_bytes()

    def batch(k):   # the first k requests of the workload
        npg = int(wl.page_indptr[k])
        args = [wl.qo_indptr[:k + 1], wl.page_indptr[:k + 1], wl.page_indices[:npg], wl.last_page_len[:k]]
        if mi is not None:
            args += [mi[:k + 1], mb[:int(mi[k])]]
        return args

    def new_ctx():
        ctx = pie.pie_create(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype, wl.R, wl.T, device=-1)
        pie.pie_alloc_kvpages(ctx, wl.num_pages)
        return ctx

    def image(ctx, k):
        plan = pie.pie_plan_forward(ctx, *batch(k))
        img, info = pie.pie_plan_debug_read(plan, 3), pie.pie_plan_get_info(plan)
        pie.pie_plan_destroy(plan)
        return img, info

    sizes = [wl.R, max(1, wl.R // 2), 1, wl.R, max(1, wl.R - 1)]
    fresh = []
    for k in sizes:
        ctx = new_ctx()
        try:
            fresh.append(image(ctx, k))
        finally:
            pie.pie_destroy(ctx)
    ctx = new_ctx()
    try:
        # a failed plan in between must leave the parked object usable
        bad = batch(wl.R)
        bad[3] = np.asarray(bad[3]).copy()
        bad[3][0] = wl.P + 1
        for k, (img0, info0) in zip(sizes, fresh):
            img, info = image(ctx, k)
            assert info == info0
            assert img.shape == img0.shape and np.array_equal(img, img0), f"first {k} requests"
            with pytest.raises(pie.PieError):
                pie.pie_plan_forward(ctx, *bad)
        # several live plans at once, destroyed in another order than they were made
        plans = [pie.pie_plan_forward(ctx, *batch(k)) for k in sizes]
        for p, (img0, _) in zip(plans, fresh):
            assert np.array_equal(pie.pie_plan_debug_read(p, 3), img0)
        for p in plans[::2] + plans[1::2]:
            pie.pie_plan_destroy(p)
        img, _ = image(ctx, sizes[1])
        assert np.array_equal(img, fresh[1][0])
    finally:
        pie.pie_destroy(ctx)


def _check_clean_prefix(P, H_q, H_kv, D, qo_indptr, page_indptr, page_indices, last_page_len, masks, num_pages):
    R, T = len(last_page_len), int(qo_indptr[-1])
    ctx = pie.pie_create(num_pages, P, H_q, H_kv, D, "bf16", R, T, device=-1)
    try:
        pie.pie_alloc_kvpages(ctx, num_pages)
        mi = mb = None
        if masks is not None and any(m is not None for m in masks):
            mi = np.zeros(R + 1, np.int64)
            for r, m in enumerate(masks):
                mi[r + 1] = mi[r] + (0 if m is None else np.asarray(m).size)
            mb = np.concatenate([np.asarray(m).reshape(-1).astype(np.uint8) for m in masks if m is not None])
        plan = pie.pie_plan_forward(ctx, qo_indptr, page_indptr, page_indices, last_page_len, mi, mb)
        items = pie.pie_plan_debug_read(plan, 5).reshape(-1, 16)
        kept = pie.pie_plan_debug_read(plan, 1).reshape(-1, 2)
        info = pie.pie_plan_get_info(plan)
        pie.pie_plan_destroy(plan)
    finally:
        pie.pie_destroy(ctx)
    assert len(items) == info["num_tile_items"] > 0
    G = H_q // H_kv
    ql = np.diff(qo_indptr)
    kv = (np.diff(page_indptr) - 1) * P + np.asarray(last_page_len)
    n_clean_items = 0
    for it in items:
        r, row0, nrows, pb, pe = int(it[0]), int(it[2]), int(it[3]), int(it[4]), int(it[5])
        clean = int(np.uint32(it[13])) >> 8
        assert 0 <= clean <= pe - pb
        if r >= R:
            continue                                    # (virtual request of a shared-prefix cascade: all visible)
        toks = np.arange(row0 // G, (row0 + nrows - 1) // G + 1)
        m = None if masks is None or masks[r] is None else np.asarray(masks[r]).astype(bool)

        def full(page_logical, rows):                   # every slot of the page allowed for every given row
            j = page_logical * P + np.arange(P)
            if (j >= kv[r]).any():
                return False
            if m is None:
                return bool((j[None, :] <= (kv[r] - ql[r] + rows)[:, None]).all())
            return bool(m[rows][:, j].all())

        logical = kept[pb:pe, 1] & 0x7FFFFFFF
        n_tile = 0
        while n_tile < pe - pb and full(int(logical[n_tile]), toks):
            n_tile += 1
        assert clean <= n_tile, (r, row0, clean, n_tile)  # never a page with a hidden slot
        if m is None:
            assert clean == n_tile                      # causal: exactly the pages below the first row's limit
        else:
            n_req = 0
            while n_req < pe - pb and full(int(logical[n_req]), np.arange(ql[r])):
                n_req += 1
            # the planner counts from the start of the request's kept list, so an item that begins behind the
            # first partly hidden page reports none
            assert clean in (n_req, 0)
        n_clean_items += clean > 0
    return n_clean_items


@pytest.mark.parametrize("name", ["mixed_prefill_decode", "shared_prefix_tree"])
def test_clean_page_prefix_of_row_tile_items(name):
    """Row-tile items carry the number of leading pages that every row of the tile sees in full; the
    kernel evaluates no mask there, so the count must never include a page with a hidden slot.  Checked
    against the mask definition: exact for inferred causal masks, and equal to the request-wide count
    (clipped to the item) for explicit ones."""
    wl = configs.small(name)
    assert _check_clean_prefix(wl.P, wl.H_q, wl.H_kv, wl.D, wl.qo_indptr, wl.page_indptr, wl.page_indices,
                               wl.last_page_len, wl.masks, wl.num_pages) > 0


def test_clean_page_prefix_with_dropped_and_partly_hidden_pages():
    """Explicit masks of an application KV policy on prefill chunks: whole pages dropped (they leave the kept
    list, so kept and logical indices differ), then a page one row sees only in part, then more visible pages."""
    rng = np.random.RandomState(11)
    P, H_q, H_kv, D = 16, 8, 2, 64
    shapes = [(24, 24 + 37 * P), (40, 40 + 20 * P + 5), (17, 17 + 9 * P)]
    masks, qo, pi, idx, last = [], [0], [0], [], []
    for n, (q_len, kv_len) in enumerate(shapes):
        pos = kv_len - q_len + np.arange(q_len)
        m = np.arange(kv_len)[None, :] <= pos[:, None]
        npg = (kv_len + P - 1) // P
        for pg in rng.choice(npg - 4, size=3, replace=False):      # dropped for every row
            m[:, pg * P:(pg + 1) * P] = False
        if n < 2:
            m[rng.randint(q_len), (5 + n) * P + 3] = False          # one slot hidden from one row
        masks.append(m)
        qo.append(qo[-1] + q_len)
        pi.append(pi[-1] + npg)
        idx.extend(range(pi[-2], pi[-1]))
        last.append(kv_len - (npg - 1) * P)
    masks[2] = None                                                  # and one inferred causal request
    assert _check_clean_prefix(P, H_q, H_kv, D, np.array(qo), np.array(pi), np.array(idx), np.array(last), masks,
                               pi[-1] + 2) > 0


def test_out_len_validation_and_work_lists():
    """Per-request output length (Section 4.2: output Embeds and / or output KvPages): bounds are checked,
    requests without output create no attention work, append destinations do not depend on it."""
    wl = configs.small("mixed_prefill_decode")
    ql = wl.q_lens()
    ctx = pie.pie_create(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype, wl.R, wl.T, device=-1)
    try:
        pie.pie_alloc_kvpages(ctx, wl.num_pages)
        base = (wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len)

        def plan(out_len):
            p = pie.pie_plan_forward(ctx, *base, out_len=out_len)
            r = (pie.pie_plan_get_info(p), pie.pie_plan_debug_read(p, 2), pie.pie_plan_debug_read(p, 4).reshape(-1, 16),
                 pie.pie_plan_debug_read(p, 5).reshape(-1, 16))
            pie.pie_plan_destroy(p)
            return r

        for bad in (ql + (np.arange(wl.R) == 3), -(np.arange(wl.R) == 0).astype(np.int32)):
            with pytest.raises(pie.PieError) as e:
                plan(bad)
            assert e.value.status == pie.PIE_ERR_INVALID
        info_all, app_all, split_all, tile_all = plan(None)
        info_same, app_same, split_same, tile_same = plan(ql)
        assert info_same == info_all and np.array_equal(split_same, split_all) and np.array_equal(tile_same, tile_all)
        out_len = np.minimum(ql, 1)
        out_len[::3] = 0
        info, app, split, tile = plan(out_len)
        assert np.array_equal(app, app_all)
        G = wl.H_q // wl.H_kv
        for items in (split, tile):
            for it in items:
                r, row0, nrows = int(it[0]), int(it[2]), int(it[3])
                assert out_len[r] > 0 and row0 + nrows <= out_len[r] * G
                assert int(it[7]) == wl.qo_indptr[r] + ql[r] - out_len[r] and int(it[8]) == out_len[r]   # query start and length of the view
        seen = {int(it[0]) for items in (split, tile) for it in items}
        assert seen == {r for r in range(wl.R) if out_len[r] > 0}
        nothing = plan(np.zeros(wl.R, np.int32))[0]
        assert nothing["num_split_items"] == nothing["num_tile_items"] == nothing["num_simple_rows"] == 0
    finally:
        pie.pie_destroy(ctx)


@pytest.mark.parametrize("name", ["shared_prefix_tree", "long_context_policy", "tiny_fp32"])
def test_masks_given_as_packed_bits_plan_like_bool_bytes(name):
    """PIE_PLAN_MASK_BITS: the caller hands over rows of ceil(kv_len / 32) words instead of q_len x kv_len bool
    bytes.  The plan must be byte for byte the one the bool matrix gives (bits past kv_len are ignored)."""
    wl = configs.small(name)
    mi, mb = wl.mask_bytes()
    assert mi is not None
    words, ptr = [], [0]
    kv, ql = wl.kv_lens(), wl.q_lens()
    rng = np.random.RandomState(2)
    for r, m in enumerate(wl.masks):
        if m is None:
            ptr.append(ptr[-1])
            continue
        rw = (kv[r] + 31) // 32
        bitsm = np.zeros((ql[r], rw * 32), dtype=np.uint8)
        bitsm[:, :kv[r]] = np.asarray(m, dtype=np.uint8)
        bitsm[:, kv[r]:] = rng.randint(0, 2, size=(ql[r], rw * 32 - kv[r]))      # garbage past the end
        packed = np.packbits(bitsm.reshape(ql[r], rw, 32), axis=2, bitorder="little").view(np.uint32).reshape(-1)
        words.append(packed)
        ptr.append(ptr[-1] + packed.size)
    ctx = pie.pie_create(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype, wl.R, wl.T, device=-1)
    try:
        pie.pie_alloc_kvpages(ctx, wl.num_pages)
        base = (wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len)
        a = pie.pie_plan_forward(ctx, *base, mi, mb)
        b = pie.pie_plan_forward(ctx, *base, np.array(ptr, np.int64), np.concatenate(words), pie.PIE_PLAN_MASK_BITS)
        assert np.array_equal(pie.pie_plan_debug_read(a, 3), pie.pie_plan_debug_read(b, 3))
        assert pie.pie_plan_get_info(a) == pie.pie_plan_get_info(b)
        pie.pie_plan_destroy(a)
        pie.pie_plan_destroy(b)
        with pytest.raises(pie.PieError) as e:                                   # wrong number of words
            pie.pie_plan_forward(ctx, *base, np.array(ptr, np.int64) + np.arange(len(ptr)), np.concatenate(words + [np.zeros(len(ptr), np.uint32)]),
                                 pie.PIE_PLAN_MASK_BITS)
        assert e.value.status == pie.PIE_ERR_MASK
    finally:
        pie.pie_destroy(ctx)


def test_requests_without_output_kvpages_borrow_and_return_pages(ctx):
    """no_store requests (Section 4.2: no output KvPages): the plan borrows pages from the free list for the new
    rows (and for the rows of a partly filled last input page), lists them behind the full input pages, and gives
    them back when it is destroyed, rebuilt or fails."""
    P = 16
    ids = pie.pie_alloc_kvpages(ctx, 6)
    free0 = pie.pie_num_free_kvpages(ctx)
    #   r0: 37 existing rows (3 pages, last holds 5) + 1 new, not stored: keeps 2 pages, borrows 1, copies 5 rows
    #   r1: 32 existing rows (2 full pages) + 20 new, not stored: keeps 2, borrows 2, no copy
    #   r2: no context, 3 new, not stored: borrows 1
    #   r3: stores as usual (1 page, 4 rows after the append)
    args = dict(qo_indptr=[0, 1, 21, 24, 25], page_indptr=[0, 3, 5, 5, 6],
                page_indices=[ids[0], ids[1], ids[2], ids[3], ids[4], ids[5]], last_page_len=[5, 16, 1, 4])
    plan = pie.pie_plan_forward(ctx, **args, no_store=[1, 1, 1, 0])
    assert pie.pie_num_free_kvpages(ctx) == free0 - 4
    info = pie.pie_plan_get_info(plan)
    kept = pie.pie_plan_debug_read(plan, 1).reshape(-1, 2)
    app = pie.pie_plan_debug_read(plan, 2)
    borrowed = [int(p) for p in kept[:, 0] if int(p) not in ids]
    assert len(set(borrowed)) == 4 and info["kept_pages"] == 2 + 1 + 2 + 2 + 1 + 1
    assert list(kept[:2, 0]) == [ids[0], ids[1]] and int(kept[2, 0]) == borrowed[0]          # r0: full pages, then the borrowed one
    assert int(app[0]) == borrowed[0] * P + 5                                                # its new row lands behind the 5 copied rows
    assert int(app[-1]) == ids[5] * P + 3                                                    # the storing request writes its own page
    assert all(int(a) // P in borrowed for a in app[:-1])
    pie.pie_plan_destroy(plan)
    assert pie.pie_num_free_kvpages(ctx) == free0
    # a failing batch (bad last_page_len of a later request) leaves nothing borrowed; so does running out of pages
    assert status_of(pie.pie_plan_forward, ctx, **dict(args, last_page_len=[5, 16, 1, 40]), no_store=[1, 1, 1, 0]) == pie.PIE_ERR_INVALID
    assert pie.pie_num_free_kvpages(ctx) == free0
    hog = pie.pie_alloc_kvpages(ctx, free0 - 3)
    assert status_of(pie.pie_plan_forward, ctx, **args, no_store=[1, 1, 1, 0]) == pie.PIE_ERR_NO_PAGES
    assert pie.pie_num_free_kvpages(ctx) == 3
    pie.pie_dealloc_kvpages(ctx, hog)
    # a recycled plan object starts clean
    for _ in range(3):
        p2 = pie.pie_plan_forward(ctx, **args, no_store=[1, 1, 1, 0])
        pie.pie_plan_destroy(p2)
        p3 = pie.pie_plan_forward(ctx, qo_indptr=[0, 1, 3], page_indptr=[0, 3, 5], page_indices=list(ids[:5]), last_page_len=[6, 2])
        assert pie.pie_num_free_kvpages(ctx) == free0
        pie.pie_plan_destroy(p3)
    pie.pie_dealloc_kvpages(ctx, ids)


def test_decode_work_list_reused_between_steps_equals_a_fresh_plan():
    """Consecutive decode steps bring the same requests with the same page counts; the context then reuses the
    block-local work list of the previous batch.  Every such plan must be byte for byte what a new context
    produces: same batch again, every context one token longer (same pages), one request a page longer (other
    units), and back."""
    _reused_work_list_case(configs.small("batched_decode"), 6, "block")   # few thread blocks: whole units per block, merged in the block
    _reused_work_list_case(configs.batched_decode(R=8), 0, "two_level")    # few long units on all blocks: merged in the kernel, blocks first
    _reused_work_list_case(configs.batched_decode(R=32), 0, "two_level")
    _reused_work_list_case(configs.batched_decode(R=32), 0, "launch")      # the same with in-kernel merges switched off: merge launch


def _reused_work_list_case(wl, sms, mode):
    P = wl.P

    def variants():
        base = (np.asarray(wl.qo_indptr), np.asarray(wl.page_indptr), np.asarray(wl.page_indices), np.asarray(wl.last_page_len))
        yield base
        yield base
        grown = base[3].copy()
        room = grown < P
        grown[room] += 1                                    # one more token in the same last page
        yield base[:3] + (grown,)
        yield base[:3] + (grown,)
        # request 0 gets one more page: other page counts, other work list
        pi = base[1].copy()
        pi[1:] += 1
        idx = np.concatenate([base[2][:base[1][1]], [wl.num_pages - 1], base[2][base[1][1]:]])
        last = base[3].copy()
        last[0] = 1
        yield (base[0], pi, idx, last)
        yield base

    def image(ctx, args):
        plan = pie.pie_plan_forward(ctx, *args)
        img, info = pie.pie_plan_debug_read(plan, 3), pie.pie_plan_get_info(plan)
        flags = pie.pie_plan_debug_read(plan, 4).view(np.int32).reshape(-1, 16)[:, 13]
        pie.pie_plan_destroy(plan)
        return img, info, flags

    def new_ctx(sms):
        c = pie.pie_create(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype, wl.R, wl.T, device=-1)
        pie.pie_set_option(c, pie.PIE_OPT_SPLIT_SMS, sms)
        pie.pie_set_option(c, pie.PIE_OPT_NO_FUSION, 2 if mode == "launch" else 0)
        pie.pie_alloc_kvpages(c, wl.num_pages)
        return c

    ctx = new_ctx(sms)
    try:
        for n, args in enumerate(variants()):
            fresh_ctx = new_ctx(sms)
            try:
                want = image(fresh_ctx, args)
            finally:
                pie.pie_destroy(fresh_ctx)
            got = image(ctx, args)
            assert got[1] == want[1], n
            assert np.array_equal(got[0], want[0]), n
            # pieces merged by a warp of their block carry flag 2; block partials of a unit cut across blocks, merged
            # by the block that writes its partial last, flag 8; without flags the merge launch combines the pieces
            if mode == "launch":
                assert got[1]["num_merge_groups"] > 0 and got[1]["launches"] == 2 and not (got[2] & 10).any()
            else:
                assert got[1]["num_merge_groups"] == 0 and got[1]["launches"] == 1
                assert (got[2] & 2).any() and bool((got[2] & 8).any()) == (mode == "two_level")
    finally:
        pie.pie_destroy(ctx)


def test_a_request_listing_its_append_page_twice_keeps_the_append_launch(ctx):
    """A decode batch normally lets the attention kernel write the new K/V row itself (one launch).  A request
    that lists the page it appends to a second time, below the appended row, would have that copy read by
    another warp than the one writing the row: the plan then keeps the separate append launch."""
    ids = pie.pie_alloc_kvpages(ctx, 4)
    plain = pie.pie_plan_forward(ctx, qo_indptr=[0, 1], page_indptr=[0, 3], page_indices=[ids[0], ids[1], ids[2]], last_page_len=[5])
    fused = pie.pie_plan_get_info(plain)["launches"]
    pie.pie_plan_destroy(plain)
    twice = pie.pie_plan_forward(ctx, qo_indptr=[0, 1], page_indptr=[0, 3], page_indices=[ids[2], ids[1], ids[2]], last_page_len=[5])
    assert pie.pie_plan_get_info(twice)["launches"] == fused + 1
    pie.pie_plan_destroy(twice)
    pie.pie_dealloc_kvpages(ctx, ids)


def _split_items(plan):
    return pie.pie_plan_debug_read(plan, 4).view(np.int32).reshape(-1, 16)


def test_decode_units_cover_two_adjacent_kv_heads_when_their_rows_fit_one_warp():
    """With 64-wide heads and pages of 8 or 16 tokens a decode unit is a pair of adjacent kv heads (their blocks of
    a page are neighbours in the pool: one copy of twice the size).  The pair needs both heads' rows inside the 16
    rows of a warp for every decode-shaped request of the batch; other shapes, an odd number of kv heads, or the
    option bit keep one kv head per unit."""
    def units_of(P, H_q, H_kv, D, q_lens, opt=0):
        c = pie.pie_create(64, P, H_q, H_kv, D, "bf16", 8, 64, device=-1)
        try:
            pie.pie_set_option(c, pie.PIE_OPT_NO_FUSION, opt)
            ids = pie.pie_alloc_kvpages(c, 3 * len(q_lens))
            qo = np.concatenate([[0], np.cumsum(q_lens)])
            plan = pie.pie_plan_forward(c, qo_indptr=qo, page_indptr=3 * np.arange(len(q_lens) + 1), page_indices=ids,
                                        last_page_len=[min(P, max(q_lens))] * len(q_lens))
            info, items = pie.pie_plan_get_info(plan), _split_items(plan)
            pie.pie_plan_destroy(plan)
            return info, items
        finally:
            pie.pie_destroy(c)

    G = 4
    for P in (8, 16):
        info, items = units_of(P, 32, 8, 64, [1, 1, 2])
        assert info["split_unit_kv_heads"] == 2
        assert set(items[:, 1].tolist()) == {0, 1, 2, 3}                     # kv head pairs
        for it in items:
            assert it[2] == 0 and it[3] == 2 * G * it[8]                     # rows of both heads of every query token (field 8: q_len)
        # every (request, pair) is covered exactly once over the request's kept pages
        for r in range(3):
            for pair in range(4):
                spans = sorted((it[4], it[5]) for it in items if it[0] == r and it[1] == pair)
                assert spans[0][0] == 3 * r and spans[-1][1] == 3 * r + 3
                assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
        info, items = units_of(P, 32, 8, 64, [1, 1, 2], opt=4)               # switched off
        assert info["split_unit_kv_heads"] == 1 and set(items[:, 1].tolist()) == set(range(8))
        info, items = units_of(P, 32, 8, 64, [1, 3, 2])                      # 12 rows per head: a pair would need 24
        assert info["split_unit_kv_heads"] == 1 and items[:, 3].max() == 12
    assert units_of(32, 32, 8, 64, [1, 1])[0]["split_unit_kv_heads"] == 1      # blocks of 8 KB already
    assert units_of(16, 32, 8, 128, [1, 1])[0]["split_unit_kv_heads"] == 1
    assert units_of(16, 12, 3, 64, [1, 1])[0]["split_unit_kv_heads"] == 1      # no partner for the last kv head
    assert units_of(16, 32, 2, 64, [1, 1])[0]["split_unit_kv_heads"] == 1      # 16 query heads per kv head fill the warp
    assert units_of(16, 16, 2, 64, [1, 1])[0]["split_unit_kv_heads"] == 2


def test_two_level_merge_fields_describe_the_block_partials():
    """A very short decode launch cuts every unit across many warps of several thread blocks.  The pieces a block
    holds are merged by the warp with the block's first piece (flags 2 / 4: counter and piece count of the group),
    which writes ONE partial per block into that piece's slot; the unit-level fields on it (flag 8: blocks spanned,
    index of this block, pieces in the first block) must let any block find the slots of all block partials:
    slot0, then slot0 + n0 + 8 (k - 1)."""
    wl = configs.batched_decode(R=4)
    c = pie.pie_create(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype, wl.R, wl.T, device=-1)
    try:
        pie.pie_alloc_kvpages(c, wl.num_pages)
        plan = pie.pie_plan_forward(c, wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len)
        info, items = pie.pie_plan_get_info(plan), _split_items(plan)
        pie.pie_plan_destroy(plan)
    finally:
        pie.pie_destroy(c)
    assert info["launches"] == 1 and info["num_merge_groups"] == 0
    NW = 8
    units = {}
    for it in items:
        units.setdefault((it[0], it[1]), []).append(it)
    n_cut = 0
    for pieces in units.values():
        assert all(a[5] == b[4] for a, b in zip(pieces, pieces[1:]))                 # contiguous page ranges, in order
        if len(pieces) == 1:
            assert pieces[0][6] == -1 and pieces[0][13] & 14 == 0
            continue
        n_cut += 1
        slot0 = pieces[0][6]
        assert [p[6] for p in pieces] == list(range(slot0, slot0 + len(pieces)))     # consecutive slots
        # block partials: pieces with flag 8, or a lone block-local group
        heads = [p for p in pieces if p[13] & 8]
        if not heads:
            f = int(pieces[0][13])
            assert f & 2 and f & 4 and ((f >> 7) & 15) == len(pieces)
            continue
        nb = (int(heads[0][13]) >> 11) & 255
        n0 = (int(heads[0][13]) >> 27) & 15
        assert len(heads) == nb and nb > 1
        covered = 0
        for k, h in enumerate(heads):
            f = int(h[13])
            assert ((f >> 11) & 255, (f >> 19) & 255, (f >> 27) & 15) == (nb, k, n0)
            assert h[6] == (slot0 if k == 0 else slot0 + n0 + NW * (k - 1))
            in_block = ((f >> 7) & 15) if f & 2 else 1                               # pieces this block holds
            assert bool(f & 4) == (in_block > 1) and in_block == (n0 if k == 0 else (NW if k + 1 < nb else in_block))
            followers = pieces[h[6] - slot0 + 1: h[6] - slot0 + in_block]
            assert all((int(q[13]) & 14) == 2 and ((int(q[13]) >> 4) & 7) == ((f >> 4) & 7) for q in followers)
            covered += in_block
        assert covered == len(pieces)
    assert n_cut == len(units) == wl.R * wl.H_kv // 2


def test_worker_threads_come_and_go_with_their_context():
    """A batch with many listed pages starts the context's planner threads; pie_destroy joins them.  Many contexts
    in a row (and two alive at once) plan the same batch to the same bytes, with and without having planned a small
    batch - which runs on the calling thread alone - in between."""
    wl = configs.long_context_policy(R=96)
    small = configs.small("batched_decode")
    mi, mb = wl.mask_bytes()

    def image(c, w, masks=(None, None)):
        plan = pie.pie_plan_forward(c, w.qo_indptr, w.page_indptr, w.page_indices, w.last_page_len, *masks)
        img = pie.pie_plan_debug_read(plan, 3).copy()
        pie.pie_plan_destroy(plan)
        return img

    want = None
    keep = None
    for k in range(12):
        c = pie.pie_create(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype, wl.R, wl.T, device=-1)
        pie.pie_alloc_kvpages(c, wl.num_pages)
        if k % 3 == 1:
            image(c, small)
        got = image(c, wl, (mi, mb))
        if want is None:
            want = got
        assert np.array_equal(got, want), k
        assert np.array_equal(image(c, wl, (mi, mb)), want), k      # recycled plan, parked workers woken again
        if k == 4:
            keep = c                                                 # stays alive next to the following contexts
        else:
            pie.pie_destroy(c)
    assert np.array_equal(image(keep, wl, (mi, mb)), want)
    pie.pie_destroy(keep)
