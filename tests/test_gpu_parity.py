"""GPU parity: the CUDA path against the fp64 oracle, element by element, on the same seeded
inputs, through the C ABI.  Tolerances: |O - O*| <= 2e-2 (bf16) / 1e-4 (fp32), |LSE - LSE*| <=
1e-3, plus a per-request relative RMS gate; append and copy are bit exact."""
import numpy as np
import pytest
import torch

from tests._util import bits, run_oracle, same_bits
from workloads import configs

pytestmark = pytest.mark.gpu

SMALL = ["tiny_fp32", "batched_decode", "mixed_prefill_decode", "shared_prefix_tree", "long_context_policy"]


def test_generator_is_bit_identical_on_cpu_and_gpu():
    wl = configs.small("mixed_prefill_decode")
    for f in (wl.q, wl.k_new, wl.v_new):
        assert torch.equal(f("cpu"), f("cuda").cpu())
    ids = wl.used_pages()[:7]
    Kc, Vc = wl.context_pages(ids, "cpu", poison=True)
    Kg, Vg = wl.context_pages(ids, "cuda", poison=True)
    assert same_bits(bits(Kc), bits(Kg)) and same_bits(bits(Vc), bits(Vg))


@pytest.mark.parametrize("name", SMALL)
@pytest.mark.parametrize("flags", [0, 1, 2])
def test_small_configs_match_oracle(name, flags):
    from tests._gpu import check_close, run_workload
    wl = configs.small(name)
    O_ref, L_ref, pool = run_oracle(wl, poison=True)
    O, L, info, gp = run_workload(wl, poison=True, flags=flags, keep=True)
    try:
        check_close(O, L, O_ref, L_ref, wl.dtype, wl.qo_indptr)
        # append is bit exact: every used page equals the oracle's pool after the call
        used = wl.used_pages()
        K, V = gp.read_pages(used)
        for n, p in enumerate(used):
            Ko, Vo = pool[int(p)]
            assert same_bits(K[n], Ko) and same_bits(V[n], Vo), f"page {p}"
    finally:
        gp.close()


def test_tiny_config_with_column_wise_drops_matches_oracle():
    """The tiny fp32 configuration with the same dropped tokens for all eight rows of request 3 (the other
    reading of "30 % of its earlier tokens masked off")."""
    from tests._gpu import check_close, run_workload
    wl = configs.tiny_fp32(column_wise=True)
    O_ref, L_ref, _ = run_oracle(wl, poison=True)
    O, L, _ = run_workload(wl, poison=True)
    check_close(O, L, O_ref, L_ref, wl.dtype, wl.qo_indptr)


@pytest.mark.parametrize("name", SMALL[1:])
@pytest.mark.parametrize("flags", [0, 2])
def test_small_configs_with_8_token_pages(name, flags):
    """KvPages of 8 tokens (the small end of the 8 - 32 tokens of Section 4.1) on the tensor-core kernels: the
    decode kernel takes them in pairs, the row-tile kernel as 16 page blocks per KV tile.  Outputs against the
    oracle, append bit exact, NaN-poisoned tails harmless."""
    import paper_2510_24051_b200 as pie
    from tests._gpu import check_close, run_workload
    wl = configs.small(name, P=8)
    O_ref, L_ref, pool = run_oracle(wl, poison=True)
    O, L, info, gp = run_workload(wl, poison=True, flags=flags, keep=True)
    try:
        assert info["num_simple_rows"] == 0 and info["num_split_items"] + info["num_tile_items"] > 0
        check_close(O, L, O_ref, L_ref, wl.dtype, wl.qo_indptr)
        used = wl.used_pages()
        K, V = gp.read_pages(used)
        for n, p in enumerate(used):
            Ko, Vo = pool[int(p)]
            assert same_bits(K[n], Ko) and same_bits(V[n], Vo), f"page {p}"
    finally:
        gp.close()


@pytest.mark.parametrize("name", SMALL[1:])
def test_peaked_scores_match_oracle(name):
    """Q scaled x4: the softmax concentrates and |O| = O(1), so a wrong kernel cannot hide
    behind small outputs."""
    from oracle import pie_oracle as orc
    from tests._gpu import check_close, run_workload
    wl = configs.small(name)
    q4 = (wl.q().float() * 4).to(torch.bfloat16)
    pool = wl.oracle_pool()
    O_ref, L_ref = orc.forward(pool, wl.P, wl.H_q, wl.qo_indptr, wl.page_indptr, wl.page_indices,
                               wl.last_page_len, bits(q4), bits(wl.k_new()), bits(wl.v_new()), wl.masks)
    O, L, _ = run_workload(wl, q_scale=4.0)
    check_close(O, L, O_ref, L_ref, wl.dtype, wl.qo_indptr)


def test_copy_kvpage_bit_exact_and_errors():
    import paper_2510_24051_b200 as pie
    from oracle import pie_oracle as orc
    from tests._gpu import GpuPool
    wl = configs.small("long_context_policy")
    pool = wl.oracle_pool()
    with GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype) as gp:
        c = wl.copies
        touched = np.unique(np.concatenate([c["src"], c["dst"]]))
        gp.install(wl, pages=touched)
        # whole-range copies of the workload plus token-level ones with shifted offsets
        src = np.concatenate([c["src"], c["src"][:3]])
        dst = np.concatenate([c["dst"], c["dst"][3:6]])
        so = np.concatenate([c["src_off"], [1, 2, 5]])
        do = np.concatenate([c["dst_off"], [9, 13, 10]])
        nt = np.concatenate([np.minimum(c["ntok"], 9), [7, 3, 6]])
        nt[3:6] = np.minimum(nt[3:6], 9)
        orc.copy_kvpage(pool, src, dst, so, do, nt)
        pie.pie_copy_kvpage(gp.ctx, src, dst, so, do, nt)
        K, V = gp.read_pages(touched)
        for n, p in enumerate(touched):
            assert same_bits(K[n], pool[int(p)][0]) and same_bits(V[n], pool[int(p)][1])
        with pytest.raises(pie.PieError) as e:      # two ops write the same slot
            pie.pie_copy_kvpage(gp.ctx, [1, 2], [3, 3], [0, 0], [0, 4], [8, 8])
        assert e.value.status == pie.PIE_ERR_CONFLICT
        with pytest.raises(pie.PieError) as e:      # overlapping in-place shift
            pie.pie_copy_kvpage(gp.ctx, [1], [1], [0], [4], [8])
        assert e.value.status == pie.PIE_ERR_CONFLICT
        with pytest.raises(pie.PieError) as e:
            pie.pie_copy_kvpage(gp.ctx, [1], [2], [10], [0], [8])
        assert e.value.status == pie.PIE_ERR_INVALID
        pie.pie_copy_kvpage(gp.ctx, [], [], [], [], [])          # empty call is fine


def test_forward_host_matches_device_call():
    import paper_2510_24051_b200 as pie
    from tests._gpu import GpuPool, check_close
    wl = configs.small("mixed_prefill_decode")
    O_ref, L_ref, _ = run_oracle(wl)
    with GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype) as gp:
        gp.install(wl)
        q, k, v = (t.pin_memory() for t in (wl.q(), wl.k_new(), wl.v_new()))
        out = torch.empty_like(q).pin_memory()
        lse = torch.empty((wl.T, wl.H_q), dtype=torch.float32).pin_memory()
        pie.pie_forward_host(gp.ctx, wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len,
                             q, k, v, out, lse)
        check_close(out.double().numpy(), lse.double().numpy(), O_ref, L_ref, wl.dtype, wl.qo_indptr)


def test_repeat_calls_are_bitwise_deterministic():
    from tests._gpu import GpuPool
    import paper_2510_24051_b200 as pie
    wl = configs.small("batched_decode")
    with GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype) as gp:
        gp.install(wl)
        plan = gp.plan(wl)
        q, k, v = wl.q("cuda"), wl.k_new("cuda"), wl.v_new("cuda")
        a = gp.forward(plan, q, k, v)
        b = gp.forward(plan, q, k, v)
        assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
        pie.pie_plan_destroy(plan)


def test_mixed_batch_side_by_side_option_matches_oracle():
    """PIE_OPT_OVERLAP: decode and prefill kernels on disjoint SM sets, forked / joined streams."""
    import paper_2510_24051_b200 as pie
    from tests._gpu import GpuPool, check_close
    wl = configs.small("mixed_prefill_decode")
    O_ref, L_ref, _ = run_oracle(wl)
    with GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype) as gp:
        gp.install(wl)
        pie.pie_set_option(gp.ctx, pie.PIE_OPT_OVERLAP, 1)
        plan = gp.plan(wl)
        q, k, v = wl.q("cuda"), wl.k_new("cuda"), wl.v_new("cuda")
        for _ in range(3):
            out, lse = gp.forward(plan, q, k, v)
            check_close(out.double().cpu().numpy(), lse.double().cpu().numpy(), O_ref, L_ref, wl.dtype, wl.qo_indptr)
        pie.pie_plan_destroy(plan)


@pytest.mark.parametrize("name", ["batched_decode", "mixed_prefill_decode", "shared_prefix_tree", "long_context_policy", "tiny_fp32"])
@pytest.mark.parametrize("flags", [0, 2])
def test_mask_kvpage_matches_oracle(name, flags):
    """Persistent page masks: random token masks on a third of the pages, some pages hidden entirely."""
    import paper_2510_24051_b200 as pie
    from oracle import pie_oracle as orc
    from tests._gpu import GpuPool, check_close
    wl = configs.small(name)
    rng = np.random.RandomState(99)
    used = wl.used_pages()
    chosen = used[rng.rand(len(used)) < 0.35]
    bits_ = rng.randint(0, 1 << wl.P, size=len(chosen), dtype=np.int64)
    bits_[rng.rand(len(chosen)) < 0.3] = 0                      # hidden pages
    page_masks = {int(p): np.array([(int(b) >> s) & 1 for s in range(wl.P)], bool) for p, b in zip(chosen, bits_)}
    pool = wl.oracle_pool()
    O_ref, L_ref = orc.forward(pool, wl.P, wl.H_q, wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len,
                               bits(wl.q()), bits(wl.k_new()), bits(wl.v_new()), wl.masks, page_masks=page_masks)
    with GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype) as gp:
        gp.install(wl)
        pie.pie_mask_kvpage(gp.ctx, chosen, bits_.astype(np.uint32))
        plan = gp.plan(wl, flags)
        out, lse = gp.forward(plan, wl.q("cuda"), wl.k_new("cuda"), wl.v_new("cuda"))
        pie.pie_plan_destroy(plan)
        check_close(out.double().cpu().numpy(), lse.double().cpu().numpy(), O_ref, L_ref, wl.dtype)


def test_split_forward_batched_together_equals_one_prefill():
    """Section 4.2: `forward([], iemb[:-1], kv)` and `forward(kv, iemb[-1:], oemb)` may be batched
    together (vertical batching).  As ONE batch - request 0 fills the pages, request 1 lists the same
    pages and reads the rows request 0 appends - the outputs equal a single 9-token prefill."""
    import paper_2510_24051_b200 as pie
    from oracle import pie_oracle as orc
    from tests._gpu import TOL_LSE, TOL_O
    n, P, H_q, H_kv, D = 41, 16, 8, 2, 128
    g = torch.Generator().manual_seed(5)
    q = torch.randn(n, H_q, D, generator=g).to(torch.bfloat16)
    k = torch.randn(n, H_kv, D, generator=g).to(torch.bfloat16)
    v = torch.randn(n, H_kv, D, generator=g).to(torch.bfloat16)
    ctx = pie.pie_create(16, P, H_q, H_kv, D, "bf16", 4, 64, 0)
    try:
        ids = pie.pie_alloc_kvpages(ctx, 8)
        pages = ids[[5, 2, 7]]
        # oracle: one prefill of n tokens into empty pages
        pool = {int(p): (np.zeros((P, H_kv, D), np.uint16), np.zeros((P, H_kv, D), np.uint16)) for p in pages}
        O_ref, L_ref = orc.forward(pool, P, H_q, np.array([0, n]), np.array([0, 3]), pages, np.array([n - 2 * P]),
                                   bits(q), bits(k), bits(v))
        # GPU: request 0 = first n-1 tokens (writes them), request 1 = last token, same page list
        plan = pie.pie_plan_forward(ctx, [0, n - 1, n], [0, 3, 6], np.concatenate([pages, pages]),
                                    [n - 1 - 2 * P, n - 2 * P])
        out = torch.empty((n, H_q, D), dtype=torch.bfloat16, device="cuda")
        lse = torch.empty((n, H_q), dtype=torch.float32, device="cuda")
        pie.pie_forward(ctx, plan, q.cuda(), k.cuda(), v.cuda(), out, lse)
        torch.cuda.synchronize()
        pie.pie_plan_destroy(plan)
        assert (out.double().cpu().numpy() - O_ref).__abs__().max() <= TOL_O["bf16"]
        assert np.abs(lse.double().cpu().numpy() - L_ref).max() <= TOL_LSE
    finally:
        pie.pie_destroy(ctx)


@pytest.mark.parametrize("name", ["tiny_fp32", "batched_decode", "mixed_prefill_decode", "shared_prefix_tree"])
@pytest.mark.parametrize("explicit_pos", [False, True])
def test_rope_inside_the_path_matches_oracle(name, explicit_pos):
    """Contexts created with rope_theta: K rows are rotated before they are stored, Q for the attention;
    positions default to the last q_len context positions or are given per token."""
    import paper_2510_24051_b200 as pie
    from oracle import pie_oracle as orc
    from tests._gpu import TDTYPE, check_close
    wl = configs.small(name)
    theta = 500000.0
    pos = None
    if explicit_pos:                                        # e.g. positions continuing after dropped context
        pos = orc.default_positions(wl.qo_indptr, wl.page_indptr, wl.last_page_len, wl.P) + 12345
    pool = wl.oracle_pool()
    O_ref, L_ref = orc.forward(pool, wl.P, wl.H_q, wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len,
                               bits(wl.q()), bits(wl.k_new()), bits(wl.v_new()), wl.masks, rope_theta=theta, positions=pos)
    ctx = pie.pie_create(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype, wl.R, wl.T, 0, rope_theta=theta)
    try:
        pie.pie_alloc_kvpages(ctx, wl.num_pages)
        used = wl.used_pages()
        K, V = wl.context_pages(used, "cuda")
        pie.pie_kvpage_write(ctx, used, K.contiguous(), V.contiguous())
        mi, mb = wl.mask_bytes()
        plan = pie.pie_plan_forward(ctx, wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len, mi, mb,
                                    positions=pos)
        q = wl.q("cuda")
        out = torch.empty_like(q)
        lse = torch.empty((wl.T, wl.H_q), dtype=torch.float32, device="cuda")
        pie.pie_forward(ctx, plan, q, wl.k_new("cuda"), wl.v_new("cuda"), out, lse)
        torch.cuda.synchronize()
        assert pie.pie_get_last_device_status(ctx) == 0
        pie.pie_plan_destroy(plan)
        check_close(out.double().cpu().numpy(), lse.double().cpu().numpy(), O_ref, L_ref, wl.dtype, wl.qo_indptr)
        # stored pages: V bit exact; K (rotated in fp32 on the GPU, fp64 in the oracle) within one unit in the
        # last place of the storage type, and mostly identical
        Kg = torch.empty((len(used), wl.P, wl.H_kv, wl.D), dtype=TDTYPE[wl.dtype], device="cuda")
        Vg = torch.empty_like(Kg)
        pie.pie_kvpage_read(ctx, used, Kg, Vg)
        torch.cuda.synchronize()
        Kg, Vg = bits(Kg), bits(Vg)
        Ko = np.stack([pool[int(p)][0] for p in used])
        Vo = np.stack([pool[int(p)][1] for p in used])
        assert same_bits(Vg, Vo)
        a, b = orc.widen(Kg), orc.widen(Ko)
        if wl.dtype == "bf16":     # a rounding flip at most: one unit in the last place of the stored value
            # (or the fp32 rotation error itself where the two products cancel to almost nothing)
            bad = np.abs(a - b) > np.maximum(np.abs(b) * 2.0 ** -7, 2e-6)
            assert not bad.any(), (int(bad.sum()), a[bad][:4], b[bad][:4])
            assert (a != b).mean() < 0.02
        else:                      # fp32 sine / cosine and products: a few 1e-7 of the row's magnitude
            assert np.abs(a - b).max() <= 2e-6
    finally:
        pie.pie_destroy(ctx)


@pytest.mark.parametrize("side_by_side", [0, 1])
def test_forward_can_be_captured_in_a_cuda_graph_and_replayed(side_by_side):
    """pie_forward only enqueues kernels (no allocation, no synchronisation), so a step can be captured
    once and replayed; the replay must reproduce the eager result bit for bit.  With the decode and
    prefill kernels side by side the capture includes the fork to and the join from the internal stream."""
    import paper_2510_24051_b200 as pie
    from tests._gpu import GpuPool
    wl = configs.small("mixed_prefill_decode")
    with GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype) as gp:
        gp.install(wl)
        if side_by_side:
            pie.pie_set_option(gp.ctx, pie.PIE_OPT_OVERLAP, 1)
        plan = gp.plan(wl)
        assert (pie.pie_plan_get_info(plan)["side_by_side_sms"] > 0) == bool(side_by_side)
        q, k, v = wl.q("cuda"), wl.k_new("cuda"), wl.v_new("cuda")
        ref_out, ref_lse = gp.forward(plan, q, k, v)
        out = torch.zeros_like(ref_out)
        lse = torch.zeros_like(ref_lse)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            pie.pie_forward(gp.ctx, plan, q, k, v, out, lse)          # warm-up on the capture stream
            side.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                pie.pie_forward(gp.ctx, plan, q, k, v, out, lse)
        torch.cuda.current_stream().wait_stream(side)
        for _ in range(3):
            out.zero_()
            lse.zero_()
            g.replay()
            torch.cuda.synchronize()
            assert torch.equal(out, ref_out) and torch.equal(lse, ref_lse)
        assert pie.pie_get_last_device_status(gp.ctx) == 0
        pie.pie_plan_destroy(plan)


@pytest.mark.parametrize("heads", [(6, 2), (12, 2), (5, 1)])
def test_head_groups_that_do_not_divide_the_row_tile(heads):
    """Group sizes 3, 6 and 5: a 128-row Q tile is not a whole number of tokens, so the tensor-core
    kernel takes its Q rows with plain copies instead of the tensor map (Section 4.2 forward)."""
    from tests._gpu import check_close, run_workload
    H_q, H_kv = heads
    for name in ("mixed_prefill_decode", "shared_prefix_tree"):
        wl = configs.small(name, H_q=H_q, H_kv=H_kv)
        O_ref, L_ref, _ = run_oracle(wl, poison=True)
        O, L, info = run_workload(wl, poison=True)
        assert info["num_tile_items"] > 0
        check_close(O, L, O_ref, L_ref, wl.dtype, wl.qo_indptr)


@pytest.mark.parametrize("heads", [(32, 1), (64, 2), (24, 1)])
def test_head_groups_above_16_run_on_the_row_tile_kernel(heads):
    """Multi-query style grouping (32 or 24 query heads per kv head): more rows per token than a decode warp
    holds, so every request, single-token decodes included, takes the tensor-core row-tile kernel."""
    from tests._gpu import check_close, run_workload
    H_q, H_kv = heads
    for name in ("batched_decode", "mixed_prefill_decode"):
        wl = configs.small(name, H_q=H_q, H_kv=H_kv)
        O_ref, L_ref, _ = run_oracle(wl, poison=True)
        for flags in (0, 2):
            O, L, info = run_workload(wl, poison=True, flags=flags)
            assert info["num_tile_items"] > 0 and info["num_simple_rows"] == 0 and info["num_split_items"] == 0
            check_close(O, L, O_ref, L_ref, wl.dtype, wl.qo_indptr)


def test_output_pointer_that_is_only_16_byte_aligned():
    """The kernels use 32-byte stores when the output pointer allows it; a view that starts 16 bytes
    into an allocation must give the same bits."""
    import paper_2510_24051_b200 as pie
    from tests._gpu import GpuPool
    wl = configs.small("shared_prefix_tree")
    with GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype) as gp:
        gp.install(wl)
        plan = gp.plan(wl)
        q, k, v = wl.q("cuda"), wl.k_new("cuda"), wl.v_new("cuda")
        T = q.shape[0]
        n = T * wl.H_q * wl.D
        outs = []
        for shift in (0, 8):                                   # elements: 8 bf16 = 16 bytes
            buf = torch.full((n + 64,), float("nan"), dtype=q.dtype, device="cuda")
            out = buf[shift:shift + n].view(T, wl.H_q, wl.D)
            assert out.data_ptr() % 32 == (16 if shift else 0)
            lse = torch.empty((T, wl.H_q), dtype=torch.float32, device="cuda")
            # the call appends into the pool: start both runs from the same pool contents
            gp.install(wl)
            pie.pie_forward(gp.ctx, plan, q, k, v, out, lse)
            torch.cuda.synchronize()
            assert pie.pie_get_last_device_status(gp.ctx) == 0
            outs.append((out.clone(), lse.clone()))
        assert torch.equal(outs[0][0].view(torch.int16), outs[1][0].view(torch.int16))
        assert torch.equal(outs[0][1], outs[1][1])
        pie.pie_plan_destroy(plan)


@pytest.mark.parametrize("P", [16, 8])
@pytest.mark.parametrize("name", ["batched_decode", "long_context_policy"])
def test_decode_fusions_equal_the_separate_launches(name, P):
    """Decode batches let the split-KV kernel write the new K/V rows itself and (short launches)
    merge the pieces of a (request, kv head) inside one thread block; PIE_OPT_NO_FUSION switches
    either off.  The append fusion must not change a bit of O, LSE or the pool; the merge fusion
    only changes the fp32 summation order, so it is held to the oracle tolerance."""
    import paper_2510_24051_b200 as pie
    from tests._gpu import GpuPool, check_close
    wl = configs.small(name, P=P)
    O_ref, L_ref, pool = run_oracle(wl, poison=True)
    res = {}
    for no_fusion in (0, 1, 2, 3):
        with GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype) as gp:
            pie.pie_set_option(gp.ctx, pie.PIE_OPT_NO_FUSION, no_fusion)
            gp.install(wl, poison=True)
            plan = gp.plan(wl)
            info = pie.pie_plan_get_info(plan)
            out, lse = gp.forward(plan, wl.q("cuda"), wl.k_new("cuda"), wl.v_new("cuda"))
            out2, lse2 = gp.forward(plan, wl.q("cuda"), wl.k_new("cuda"), wl.v_new("cuda"))   # plan reuse
            assert torch.equal(out.view(torch.int16), out2.view(torch.int16)) and torch.equal(lse, lse2)
            K, V = gp.read_pages(wl.used_pages())
            pie.pie_plan_destroy(plan)
        check_close(out.double().cpu().numpy(), lse.double().cpu().numpy(), O_ref, L_ref, wl.dtype, wl.qo_indptr)
        for n, pg in enumerate(wl.used_pages()):
            Ko, Vo = pool[int(pg)]
            assert same_bits(K[n], Ko) and same_bits(V[n], Vo), f"page {pg}"
        res[no_fusion] = (info["launches"], out.view(torch.int16).cpu(), lse.cpu())
    for a, b2 in ((0, 1), (2, 3)):                         # the append fusion alone: identical bits, one launch fewer
        assert res[b2][0] == res[a][0] + 1
        assert torch.equal(res[a][1], res[b2][1]) and torch.equal(res[a][2], res[b2][2])
    assert res[3][0] == 3 and res[0][0] <= 2              # append + split-KV + merge against split-KV (+ merge if dynamic)


@pytest.mark.parametrize("flags,P", [(8, 16), (4, 16), (0, 16), (8 | 2, 16), (8, 8), (8, 32)])
def test_shared_prefix_cascade_matches_oracle(flags, P):
    """Branches that decode from a shared prompt: with the cascade the prompt's pages are attended
    once per group (row-tile kernel over the gathered rows) and each request's private pages by the
    split-KV kernel, merged on LSE (Section 4.2: forked contexts share KvPages).  Flags: 8 = cascade
    however small the saving, 4 = never, 0 = the planner's own choice (this small batch: none)."""
    import paper_2510_24051_b200 as pie
    from tests._gpu import check_close, run_workload
    wl = configs.small("shared_prefix_decode", P=P)
    O_ref, L_ref, pool = run_oracle(wl, poison=True)
    O, L, info, gp = run_workload(wl, poison=True, flags=flags, keep=True)
    try:
        assert (info["num_tile_items"] > 0) == bool(flags & 8)
        check_close(O, L, O_ref, L_ref, wl.dtype, wl.qo_indptr)
        used = wl.used_pages()
        K, V = gp.read_pages(used)
        for n, p in enumerate(used):
            Ko, Vo = pool[int(p)]
            assert same_bits(K[n], Ko) and same_bits(V[n], Vo), f"page {p}"
    finally:
        gp.close()


@pytest.mark.parametrize("case", ["small_forced", "mid_auto", "mid_auto_8_token_pages", "causal_chunks"])
def test_shared_prefix_cascade_of_requests_with_row_tiles_of_their_own(case):
    """Branches that verify a token tree of 32 nodes over a shared prompt bring 128 rows each - half a row tile.
    The cascade gathers the group's rows over the shared pages (full tiles, no masks) and runs every request's
    private suffix + tree pages as a row-tile item of its own; both write partials that the merge combines.  Also
    with inferred causal masks (short prefill chunks of forked requests)."""
    import paper_2510_24051_b200 as pie
    from tests._gpu import check_close, run_workload
    flags = 0
    if case == "small_forced":
        wl, flags = configs.small("shared_prefix_tree"), pie.PIE_PLAN_CASCADE_ALWAYS
    elif case == "mid_auto":
        wl = configs.shared_prefix_tree(groups=2, branches=4, prefix=1024, suffix=48, tree=32, num_pages=512)
    elif case == "mid_auto_8_token_pages":
        wl = configs.shared_prefix_tree(groups=2, branches=5, prefix=1024, suffix=40, tree=32, num_pages=1024, P=8)
    else:
        wl = configs.shared_prefix_tree(groups=2, branches=4, prefix=1040, suffix=16, tree=16, num_pages=512)
        wl.masks = None                                   # 16 new tokens per branch under the inferred causal mask: 64 rows
    O_ref, L_ref, pool = run_oracle(wl, poison=True)
    O, L, info, gp = run_workload(wl, poison=True, flags=flags, keep=True)
    try:
        assert info["num_merge_groups"] == wl.R * wl.H_kv and info["num_split_items"] == 0
        check_close(O, L, O_ref, L_ref, wl.dtype, wl.qo_indptr)
        used = wl.used_pages()
        K, V = gp.read_pages(used)
        for n, p in enumerate(used):
            Ko, Vo = pool[int(p)]
            assert same_bits(K[n], Ko) and same_bits(V[n], Vo), f"page {p}"
    finally:
        gp.close()


@pytest.mark.parametrize("sms,P", [(6, 16), (16, 16), (6, 8)])
def test_block_local_merge_matches_oracle(sms, P):
    """Short decode launches deal whole (request, kv head) units to thread blocks and cut them only
    between warps of one block, which then merges the pieces itself: no merge launch.  Few SMs
    make the small batch balance well enough for that path to be chosen."""
    import paper_2510_24051_b200 as pie
    from tests._gpu import GpuPool, check_close
    wl = configs.small("batched_decode", P=P)
    O_ref, L_ref, pool = run_oracle(wl, poison=True)
    with GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype) as gp:
        pie.pie_set_option(gp.ctx, pie.PIE_OPT_SPLIT_SMS, sms)
        gp.install(wl, poison=True)
        plan = gp.plan(wl)
        info = pie.pie_plan_get_info(plan)
        assert info["num_merge_groups"] == 0 and info["launches"] == 1        # fused append, in-kernel merge
        assert info["num_split_items"] > wl.R * wl.H_kv // info["split_unit_kv_heads"]   # units were cut
        out, lse = gp.forward(plan, wl.q("cuda"), wl.k_new("cuda"), wl.v_new("cuda"))
        out2, lse2 = gp.forward(plan, wl.q("cuda"), wl.k_new("cuda"), wl.v_new("cuda"))
        assert torch.equal(out.view(torch.int16), out2.view(torch.int16)) and torch.equal(lse, lse2)
        pie.pie_plan_destroy(plan)
        check_close(out.double().cpu().numpy(), lse.double().cpu().numpy(), O_ref, L_ref, wl.dtype, wl.qo_indptr)
        K, V = gp.read_pages(wl.used_pages())
        for n, pg in enumerate(wl.used_pages()):
            Ko, Vo = pool[int(pg)]
            assert same_bits(K[n], Ko) and same_bits(V[n], Vo), f"page {pg}"


@pytest.mark.parametrize("name", ["mixed_prefill_decode", "long_context_policy"])
def test_plan_per_step_loop_with_recycled_plans_matches_oracle(name):
    """A serving loop plans every step and destroys the plan right after enqueueing its forward:
    the context hands the same plan objects (pinned image, device arrays) out again.  Forwards run
    on a non-blocking side stream while the uploads use another one, so only the library's own
    ordering keeps a reused device image from being overwritten under a running kernel."""
    import paper_2510_24051_b200 as pie
    from tests._gpu import GpuPool, check_close
    wl = configs.small(name)
    O_ref, L_ref, _ = run_oracle(wl)
    mi, mb = wl.mask_bytes()

    def batch(k):   # the first k requests
        npg = int(wl.page_indptr[k])
        args = [wl.qo_indptr[:k + 1], wl.page_indptr[:k + 1], wl.page_indices[:npg], wl.last_page_len[:k]]
        if mi is not None:
            args += [mi[:k + 1], mb[:int(mi[k])]]
        return args

    with GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype) as gp:
        gp.install(wl)
        q, k_new, v_new = wl.q("cuda"), wl.k_new("cuda"), wl.v_new("cuda")
        run, up = torch.cuda.Stream(), torch.cuda.Stream()
        torch.cuda.synchronize()
        sizes = [wl.R, max(1, wl.R // 2), wl.R, 1, max(1, wl.R - 1), wl.R, wl.R, max(1, wl.R // 3)] * 2
        results = []
        for k in sizes:
            T = int(wl.qo_indptr[k])
            plan = pie.pie_plan_forward(gp.ctx, *batch(k), stream=up.cuda_stream)
            out = torch.full((T, wl.H_q, wl.D), float("nan"), dtype=q.dtype, device="cuda")
            lse = torch.full((T, wl.H_q), float("nan"), dtype=torch.float32, device="cuda")
            run.wait_stream(torch.cuda.current_stream())      # (the fills above)
            pie.pie_forward(gp.ctx, plan, q[:T], k_new[:T], v_new[:T], out, lse, stream=run.cuda_stream)
            pie.pie_plan_destroy(plan)                        # no synchronisation in between
            results.append((T, out, lse))
        torch.cuda.synchronize()
        assert pie.pie_get_last_device_status(gp.ctx) == 0
        for T, out, lse in results:
            check_close(out.double().cpu().numpy(), lse.double().cpu().numpy(), O_ref[:T], L_ref[:T], wl.dtype,
                        wl.qo_indptr[:np.searchsorted(wl.qo_indptr, T) + 1])


@pytest.mark.parametrize("D", [128, 64])
def test_scores_that_keep_outgrowing_the_running_reference(D):
    """Row tiles whose scores climb a staircase along the context: every step is a jump of ~20
    binades, far beyond what the lagging softmax reference tolerates, in the middle of pages that
    need no mask (where the kernel takes no maximum as long as the sums stay small).  Rows with a
    negative gain see falling scores instead and share warps with the climbing ones."""
    from oracle import pie_oracle as orc
    from tests._gpu import TOL_LSE, TOL_O
    from tests._util import SmallBatch
    from tests.test_gpu_matrix import _bf16_round, run_gpu
    rng = np.random.RandomState(7 + D)
    H_q, H_kv, P = 8, 2, 16
    seqs = []
    for q_len, kv_len in [(64, 1400), (40, 900), (1, 300), (33, 33)]:
        pos = np.arange(kv_len)
        stairs = (pos // 96) * (14.0 * np.sqrt(D) / D)          # +14 nats of score per step for a gain of 1
        u = np.ones(D, np.float32)
        K = stairs[:, None, None] * u[None, None, :] + 0.5 * rng.randn(kv_len, H_kv, D)
        gain = rng.choice([1.0, 0.7, -0.8, 0.0], size=(q_len, H_q, 1))
        Q = gain * u[None, None, :] + 0.5 * rng.randn(q_len, H_q, D)
        seqs.append(dict(Q=_bf16_round(Q.astype(np.float32)), K=_bf16_round(K.astype(np.float32)),
                         V=_bf16_round(rng.randn(kv_len, H_kv, D).astype(np.float32))))
    args = SmallBatch(seqs, H_q).paged(P, "random", seed=3)
    total = len(args["pool"])
    O_ref, L_ref = orc.forward(**{k: (v if k != "pool" else {p: (a.copy(), b.copy()) for p, (a, b) in v.items()})
                                  for k, v in args.items()})
    args["masks"] = [None] * len(seqs)
    import paper_2510_24051_b200 as pie
    # (two thread blocks for the row tiles: the items stay long, ten and more steps of the staircase each)
    for flags, options in ((0, {pie.PIE_OPT_TILE_SMS: 2}), (0, None), (2, None)):
        O, L, info = run_gpu(args, total, H_kv, D, "bf16", flags, options)
        if flags == 0:
            assert info["num_tile_items"] > 0
        if options:
            assert info["num_tile_items"] <= 8
        assert np.isfinite(O).all()
        assert np.abs(O - O_ref).max() <= TOL_O["bf16"]
        assert np.abs(L - L_ref).max() <= TOL_LSE


def test_prefill_under_a_kv_policy_with_a_long_clean_prefix():
    """Prefill chunks under application masks that drop whole pages (kept and logical page indices differ),
    with the first partly hidden page far into the context: the kernel runs the pages before it without
    looking at any mask, and must pick the masks up exactly where the planner says."""
    from oracle import pie_oracle as orc
    from tests._gpu import TOL_LSE, TOL_O
    from tests._util import SmallBatch, random_seqs
    from tests.test_gpu_matrix import _bf16_round, run_gpu
    import paper_2510_24051_b200 as pie
    rng = np.random.RandomState(23)
    P, H_q, H_kv, D = 16, 8, 2, 128
    shapes = [(48, 48 + 61 * P + 3), (33, 33 + 40 * P), (64, 64 + 52 * P + 9)]
    masks = []
    for n, (q_len, kv_len) in enumerate(shapes):
        pos = kv_len - q_len + np.arange(q_len)
        m = np.arange(kv_len)[None, :] <= pos[:, None]
        for pg in rng.choice(24, size=4, replace=False):              # dropped for every row
            m[:, pg * P:(pg + 1) * P] = False
        m[rng.randint(q_len), (30 + 3 * n) * P + 5] = False           # first slot that only some rows see
        m[:, (34 + n) * P:(35 + n) * P] &= rng.rand(q_len, P) < 0.7   # and a page hidden at random
        masks.append(m)
    seqs = random_seqs(rng, shapes, H_q, H_kv, D, masks=masks)
    for s in seqs:
        for k in ("Q", "K", "V"):
            s[k] = _bf16_round(s[k])
    args = SmallBatch(seqs, H_q).paged(P, "random", seed=5)
    total = len(args["pool"])
    O_ref, L_ref = orc.forward(**{k: (v if k != "pool" else {p: (a.copy(), b.copy()) for p, (a, b) in v.items()})
                                  for k, v in args.items()})
    for options in ({pie.PIE_OPT_TILE_SMS: 3}, None):
        O, L, info = run_gpu(args, total, H_kv, D, "bf16", 0, options)
        assert info["num_tile_items"] > 0 and info["kept_pages"] < sum((kv + P - 1) // P for _, kv in shapes)
        assert np.isfinite(O).all()
        assert np.abs(O - O_ref).max() <= TOL_O["bf16"]
        assert np.abs(L - L_ref).max() <= TOL_LSE


@pytest.mark.parametrize("name", ["mixed_prefill_decode", "shared_prefix_tree", "tiny_fp32"])
@pytest.mark.parametrize("flags", [0, 1, 2])
def test_outputs_for_the_last_tokens_only(name, flags):
    """Section 4.2: a forward call fills output Embeds and / or output KvPages.  Requests ask for outputs of
    their last out_len tokens only (0 = store the rows, attend nothing): those rows match the oracle, all
    other rows of out / lse keep what the caller put there, and every row is appended bit for bit."""
    import paper_2510_24051_b200 as pie
    from tests._gpu import GpuPool, check_close
    wl = configs.small(name)
    rng = np.random.RandomState(3)
    ql = wl.q_lens()
    out_len = np.array([[0, 1, q, max(1, q // 3), q][rng.randint(5)] for q in ql], dtype=np.int32)
    out_len[0], out_len[-1] = 0, min(1, ql[-1])
    pool_ref = wl.oracle_pool(True)
    O_ref, L_ref = orc_forward_with_out_lens(wl, pool_ref, out_len)
    with GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype) as gp:
        gp.install(wl, poison=True)
        mi, mb = wl.mask_bytes()
        plan = pie.pie_plan_forward(gp.ctx, wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len, mi, mb,
                                    flags, out_len=out_len)
        out, lse = gp.forward(plan, wl.q("cuda"), wl.k_new("cuda"), wl.v_new("cuda"))   # (prefilled with NaN)
        pie.pie_plan_destroy(plan)
        O, L = out.double().cpu().numpy(), lse.double().cpu().numpy()
        produced = ~np.isnan(L_ref[:, 0])
        assert produced.any() and (~produced).any()
        assert np.isnan(O[~produced]).all() and np.isnan(L[~produced]).all()          # untouched
        check_close(O[produced], L[produced], O_ref[produced], L_ref[produced], wl.dtype)
        used = wl.used_pages()
        Kg, Vg = gp.read_pages(used)
        for n, pg in enumerate(used):
            assert same_bits(Kg[n], pool_ref[int(pg)][0]) and same_bits(Vg[n], pool_ref[int(pg)][1])


def orc_forward_with_out_lens(wl, pool, out_len):
    from oracle import pie_oracle as orc
    return orc.forward(pool, wl.P, wl.H_q, wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len,
                       bits(wl.q()), bits(wl.k_new()), bits(wl.v_new()), wl.masks, out_lens=out_len)


def no_store_case():
    """A batch that mixes requests with and without output KvPages (Section 4.2), its pool contents and the
    oracle's results: shared by the tests of both forward entry points."""
    from oracle import pie_oracle as orc
    from tests.test_gpu_matrix import _bf16_round
    rng = np.random.RandomState(77)
    P, H_q, H_kv, D = 16, 8, 2, 128
    #          kv_in q_len no_store
    shapes = [(37, 1, 1), (64, 1, 1), (0, 40, 1), (300, 70, 1), (45, 1, 0), (90, 33, 0), (21, 3, 1), (512, 1, 1)]
    R = len(shapes)
    num_pages = 160
    perm = rng.permutation(100)
    pool = {p: (np.full((P, H_kv, D), np.nan, np.float32), np.full((P, H_kv, D), np.nan, np.float32)) for p in range(num_pages)}
    qo, pi, idx, last, masks, out_len, no_store = [0], [0], [], [], [], [], []
    q_rows, k_rows, v_rows, cur = [], [], [], 0
    for r, (kv_in, q_len, ns) in enumerate(shapes):
        total = kv_in + q_len
        K = _bf16_round(rng.randn(total, H_kv, D).astype(np.float32))
        V = _bf16_round(rng.randn(total, H_kv, D).astype(np.float32))
        n_list = (kv_in + P - 1) // P if ns else (total + P - 1) // P
        pages = perm[cur:cur + n_list]
        cur += n_list
        for j in range(kv_in):
            pool[int(pages[j // P])][0][j % P] = K[j]
            pool[int(pages[j // P])][1][j % P] = V[j]
        qo.append(qo[-1] + q_len)
        pi.append(pi[-1] + n_list)
        idx.extend(int(p) for p in pages)
        last.append((kv_in if ns else total) - (n_list - 1) * P if n_list else 1)
        m = None
        if r == 3:                                                      # explicit mask over existing + new positions
            pos = kv_in + np.arange(q_len)
            m = (np.arange(total)[None, :] <= pos[:, None]) & (rng.rand(q_len, total) < 0.85)
            m[np.arange(q_len), pos] = True
        masks.append(m)
        out_len.append(1 if r == 2 else q_len)
        no_store.append(ns)
        q_rows.append(_bf16_round(rng.randn(q_len, H_q, D).astype(np.float32)))
        k_rows.append(K[kv_in:])
        v_rows.append(V[kv_in:])
    q, k_new, v_new = (np.concatenate(x) for x in (q_rows, k_rows, v_rows))
    qo, pi, idx, last = np.array(qo), np.array(pi), np.array(idx), np.array(last)
    hidden_page = int(idx[pi[6] + 1])                                   # request 6: second (partly filled) page, slots 1 and 3 hidden
    pm_bits = 0xFFFFFFFF & ~0b1010
    page_masks = {hidden_page: np.array([(pm_bits >> s) & 1 for s in range(P)], dtype=bool)}
    pool_ref = {p: (a.copy(), b.copy()) for p, (a, b) in pool.items()}
    O_ref, L_ref = orc.forward(pool_ref, P, H_q, qo, pi, idx, last, q, k_new, v_new, masks=masks, out_lens=out_len,
                               no_store=no_store, page_masks=page_masks)
    return dict(P=P, H_q=H_q, H_kv=H_kv, D=D, R=R, num_pages=num_pages, pool=pool, pool_ref=pool_ref, qo=qo, pi=pi, idx=idx,
                last=last, masks=masks, out_len=out_len, no_store=no_store, q=q, k_new=k_new, v_new=v_new,
                hidden_page=hidden_page, pm_bits=pm_bits, O_ref=O_ref, L_ref=L_ref)


@pytest.mark.parametrize("flags", [0, 1, 2])
def test_forward_without_output_kvpages(flags):
    """Section 4.2: a forward call may have no output KvPages - the new rows are attended as the last positions
    of the context but stored nowhere.  Requests with and without output pages share a batch: contexts that end
    in the middle of a page or on a page boundary, no context at all, prefill chunks and single tokens, an
    explicit mask, a page mask on the partly filled last page, outputs for the last token only.  Outputs match
    the oracle, the caller's pages are bit for bit what the oracle's pool holds (only storing requests appended),
    and the plan gives its borrowed pages back."""
    import paper_2510_24051_b200 as pie
    from tests._gpu import TOL_LSE, TOL_O
    c = no_store_case()
    P, H_q, H_kv, D, R, num_pages = c["P"], c["H_q"], c["H_kv"], c["D"], c["R"], c["num_pages"]
    pool, pool_ref, qo, pi, idx, last, masks = c["pool"], c["pool_ref"], c["qo"], c["pi"], c["idx"], c["last"], c["masks"]
    out_len, no_store, q, k_new, v_new = c["out_len"], c["no_store"], c["q"], c["k_new"], c["v_new"]
    hidden_page, pm_bits, O_ref, L_ref = c["hidden_page"], c["pm_bits"], c["O_ref"], c["L_ref"]
    produced = ~np.isnan(L_ref[:, 0])
    T = len(q)
    ctx = pie.pie_create(num_pages, P, H_q, H_kv, D, "bf16", R, T, 0)
    try:
        ids = pie.pie_alloc_kvpages(ctx, 100)                            # 60 pages stay free for the plan to borrow
        assert sorted(ids) == list(range(100))
        tdt = torch.bfloat16
        Kd = torch.from_numpy(np.stack([pool[int(p)][0] for p in ids])).to(tdt).cuda()
        Vd = torch.from_numpy(np.stack([pool[int(p)][1] for p in ids])).to(tdt).cuda()
        pie.pie_kvpage_write(ctx, ids, Kd, Vd)
        pie.pie_mask_kvpage(ctx, [hidden_page], [pm_bits])
        ptr = np.zeros(R + 1, np.int64)
        for r, m in enumerate(masks):
            ptr[r + 1] = ptr[r] + (0 if m is None else m.size)
        buf = np.concatenate([m.reshape(-1).astype(np.uint8) for m in masks if m is not None])
        free0 = pie.pie_num_free_kvpages(ctx)
        plan = pie.pie_plan_forward(ctx, qo, pi, idx, last, ptr, buf, flags, out_len=out_len, no_store=no_store)
        assert pie.pie_num_free_kvpages(ctx) < free0
        out = torch.full((T, H_q, D), float("nan"), dtype=tdt, device="cuda")
        lse = torch.full((T, H_q), float("nan"), dtype=torch.float32, device="cuda")
        pie.pie_forward(ctx, plan, *(torch.from_numpy(x).to(tdt).cuda() for x in (q, k_new, v_new)), out, lse)
        torch.cuda.synchronize()
        assert pie.pie_get_last_device_status(ctx) == 0
        pie.pie_plan_destroy(plan)
        assert pie.pie_num_free_kvpages(ctx) == free0
        O, L = out.double().cpu().numpy(), lse.double().cpu().numpy()
        assert np.isnan(O[~produced]).all()
        assert np.abs(O[produced] - O_ref[produced]).max() <= TOL_O["bf16"]
        assert np.abs(L[produced] - L_ref[produced]).max() <= TOL_LSE
        Kg = torch.empty((100, P, H_kv, D), dtype=tdt, device="cuda")
        Vg = torch.empty_like(Kg)
        pie.pie_kvpage_read(ctx, np.arange(100, dtype=np.int32), Kg, Vg)
        torch.cuda.synchronize()
        Kb, Vb = Kg.cpu().float().numpy(), Vg.cpu().float().numpy()
        for pg in range(100):
            assert same_bits(np.nan_to_num(Kb[pg], nan=7.0), np.nan_to_num(pool_ref[pg][0], nan=7.0)), pg
            assert same_bits(np.nan_to_num(Vb[pg], nan=7.0), np.nan_to_num(pool_ref[pg][1], nan=7.0)), pg
        # too few free pages for the borrowed ones
        extra = pie.pie_alloc_kvpages(ctx, pie.pie_num_free_kvpages(ctx) - 1)
        with pytest.raises(pie.PieError) as e:
            pie.pie_plan_forward(ctx, qo, pi, idx, last, ptr, buf, flags, out_len=out_len, no_store=no_store)
        assert e.value.status == pie.PIE_ERR_NO_PAGES and pie.pie_num_free_kvpages(ctx) == 1
        pie.pie_dealloc_kvpages(ctx, extra)
    finally:
        pie.pie_destroy(ctx)


def test_a_wait_that_cannot_complete_gives_up_and_the_context_stays_usable():
    """Failure path without a fault: a kernel whose only wait has no producer.  The bounded wait runs out
    after about a second, the status word reports it once, and a forward on the same context still matches
    the oracle afterwards."""
    import time
    import paper_2510_24051_b200 as pie
    from tests._gpu import GpuPool, check_close
    wl = configs.small("mixed_prefill_decode")
    O_ref, L_ref, _ = run_oracle(wl)
    with GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype) as gp:
        gp.install(wl)
        t0 = time.perf_counter()
        pie.pie_debug_bounded_wait(gp.ctx)
        assert pie.pie_get_last_device_status(gp.ctx) == pie.PIE_ERR_DEVICE_TIMEOUT      # (synchronises the stream)
        assert 0.5 < time.perf_counter() - t0 < 10.0
        assert pie.pie_get_last_device_status(gp.ctx) == 0                                # read and cleared
        plan = gp.plan(wl)
        out, lse = gp.forward(plan, wl.q("cuda"), wl.k_new("cuda"), wl.v_new("cuda"))
        pie.pie_plan_destroy(plan)
        check_close(out.double().cpu().numpy(), lse.double().cpu().numpy(), O_ref, L_ref, wl.dtype, wl.qo_indptr)


@pytest.mark.parametrize("kv_heads_per_unit", [2, 1])
@pytest.mark.parametrize("P", [16, 8])
@pytest.mark.parametrize("shape", ["decode", "two_tokens_masked"])
def test_decode_units_of_one_or_two_kv_heads_match_oracle(shape, P, kv_heads_per_unit):
    """64-wide heads with pages of 8 or 16 tokens: by default a decode unit covers two adjacent kv heads (one copy of
    twice the size per page; rows of the first head take K and V of the first head only, rows of the second of the
    second), with the option bit one kv head as everywhere else.  Both against the oracle: single-token decodes
    (the kernel also writes the new rows of both heads) and requests of two query tokens - 16 rows per pair - where
    some carry an explicit mask with dropped earlier tokens and ragged last pages."""
    import paper_2510_24051_b200 as pie
    from tests._gpu import GpuPool, check_close
    from workloads import synth
    seed = 0x5EED0 + P
    if shape == "decode":
        q_lens = [1] * 9
        kv_lens = [1, 15, 16, 17, 33, 250, 511, 640, 97]
        masks = None
    else:
        q_lens = [2, 1, 2, 2, 1, 2]
        kv_lens = [2, 40, 130, 257, 16, 600]
        masks = [None] * len(q_lens)
        for r in (2, 3, 5):
            ql, kl = q_lens[r], kv_lens[r]
            pos = kl - ql + np.arange(ql)
            causal = np.arange(kl)[None, :] <= pos[:, None]
            drop = synth.uniform_unit(seed, 30 + r, (ql, kl)) < (0.6 if r == 5 else 0.3)
            if r == 5:
                drop[:, 64:192] = True                    # whole pages that no row attends to are dropped from the lists
            masks[r] = causal & ~(drop & (np.arange(kl)[None, :] < pos[:, None]))
    wl = configs._assemble("decode_units", seed, 32, 8, 64, P, "bf16", 512, q_lens, kv_lens, masks)
    O_ref, L_ref, pool = run_oracle(wl, poison=True)
    with GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype) as gp:
        pie.pie_set_option(gp.ctx, pie.PIE_OPT_NO_FUSION, 0 if kv_heads_per_unit == 2 else 4)
        gp.install(wl, poison=True)
        plan = gp.plan(wl)
        info = pie.pie_plan_get_info(plan)
        assert info["split_unit_kv_heads"] == kv_heads_per_unit and info["num_tile_items"] == 0 and info["num_simple_rows"] == 0
        assert info["launches"] == (1 if shape == "decode" else 2) + (info["num_merge_groups"] > 0)
        out, lse = gp.forward(plan, wl.q("cuda"), wl.k_new("cuda"), wl.v_new("cuda"))
        pie.pie_plan_destroy(plan)
        check_close(out.double().cpu().numpy(), lse.double().cpu().numpy(), O_ref, L_ref, wl.dtype, wl.qo_indptr)
        K, V = gp.read_pages(wl.used_pages())
        for n, pg in enumerate(wl.used_pages()):
            Ko, Vo = pool[int(pg)]
            assert same_bits(K[n], Ko) and same_bits(V[n], Vo), f"page {pg}"


@pytest.mark.parametrize("R,D,P,lo", [(4, 64, 16, 512), (8, 64, 8, 512), (3, 128, 16, 512), (2, 128, 32, 3900)])
def test_very_short_decode_launches_merge_across_blocks_inside_the_kernel(R, D, P, lo):
    """A handful of single-token requests over contexts of 512 - 4,096 tokens: every (request, kv head) unit is cut
    across the warps of several thread blocks.  One launch: the pieces a block holds are merged by one of its warps,
    the block partials by whichever block writes its partial last.  Against the oracle, bitwise equal from run to
    run (the combine order is fixed), counters re-armed (the second call with the same plan), pool bit-exact."""
    import paper_2510_24051_b200 as pie
    from tests._gpu import GpuPool, check_close
    wl = configs.batched_decode(R=R, D=D, P=P, lo=lo, num_pages=4096 * 16 // P)
    O_ref, L_ref, pool = run_oracle(wl, poison=True)
    with GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype) as gp:
        gp.install(wl, poison=True)
        plan = gp.plan(wl)
        info = pie.pie_plan_get_info(plan)
        assert info["launches"] == 1 and info["num_merge_groups"] == 0 and info["num_split_items"] > 4 * R * wl.H_kv
        flags = pie.pie_plan_debug_read(plan, 4).view(np.int32).reshape(-1, 16)[:, 13]
        assert (flags & 8).any() and (flags & 4).any()
        q, k, v = wl.q("cuda"), wl.k_new("cuda"), wl.v_new("cuda")
        out, lse = gp.forward(plan, q, k, v)
        for _ in range(3):
            out2, lse2 = gp.forward(plan, q, k, v)
            assert torch.equal(out.view(torch.int16), out2.view(torch.int16)) and torch.equal(lse, lse2)
        pie.pie_plan_destroy(plan)
        check_close(out.double().cpu().numpy(), lse.double().cpu().numpy(), O_ref, L_ref, wl.dtype, wl.qo_indptr)
        K, V = gp.read_pages(wl.used_pages())
        for n, pg in enumerate(wl.used_pages()):
            Ko, Vo = pool[int(pg)]
            assert same_bits(K[n], Ko) and same_bits(V[n], Vo), f"page {pg}"


@pytest.mark.gpu
@pytest.mark.parametrize("tile_sms,D", [(4, 64), (8, 128), (40, 128)])
def test_row_tile_units_cut_across_blocks_are_merged_like_the_oracle(tile_sms, D):
    """One prefill chunk over a long context is two row-tile units (two kv heads) for far more thread blocks: the
    units are cut into pieces whose fp32 partials the tile merge combines - from two sources per row (eight rows per
    warp and step), from four (four rows), and from sixteen (row by row)."""
    import paper_2510_24051_b200 as pie
    from tests._gpu import GpuPool, check_close
    wl = configs._assemble("one_long_prefill", configs.SEED0 + 31, 8, 2, D, 16, "bf16", 1024,
                           np.array([64]), np.array([8192]), None)
    O_ref, L_ref, _ = run_oracle(wl, poison=True)
    with GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype) as gp:
        pie.pie_set_option(gp.ctx, pie.PIE_OPT_TILE_SMS, tile_sms)
        gp.install(wl, poison=True)
        plan = gp.plan(wl)
        info = pie.pie_plan_get_info(plan)
        pieces = min(tile_sms, 2 * 512 // 32)
        assert info["num_merge_groups"] == 2 and info["num_split_items"] == 0
        assert pieces <= info["num_tile_items"] <= pieces + 2          # two units over `pieces` equal shares
        out, lse = gp.forward(plan, wl.q("cuda"), wl.k_new("cuda"), wl.v_new("cuda"))
        out2, lse2 = gp.forward(plan, wl.q("cuda"), wl.k_new("cuda"), wl.v_new("cuda"))
        assert torch.equal(out.view(torch.int16), out2.view(torch.int16)) and torch.equal(lse, lse2)
        pie.pie_plan_destroy(plan)
        check_close(out.double().cpu().numpy(), lse.double().cpu().numpy(), O_ref, L_ref, wl.dtype, wl.qo_indptr)
