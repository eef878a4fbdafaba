"""pie_forward_static_scratch: the forward call for hosts that cannot allocate device memory when a
batch runs (a frozen or externally owned device heap, or a serving loop that must avoid the
implicit synchronisation of cudaMalloc / cudaFree).  Its plan arrays and split partials live in a
fixed device array inside the library instead of a per-plan allocation, and it enqueues the same
kernels on the same plan image as pie_plan_forward + pie_forward, so its results must be theirs
bit for bit - and the oracle's within the parity tolerances.  Checked through the C ABI on two
calls in a row (the second call reuses the array with the first call's contents still in it), on a
decode batch whose split partials go through the merge, on a mixed batch with explicit masks and on
a batch with requests that have no output KvPages (borrowed pool pages must all come back)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["batched_decode", "long_context_policy", "mixed_prefill_decode", "four_long_decodes"])
def test_static_scratch_forward_matches_planned_forward(name):
    import paper_2510_24051_b200 as pie
    from tests._gpu import GpuPool, check_close
    from tests._util import run_oracle
    from workloads import configs
    # (four_long_decodes: units cut across thread blocks and merged inside the kernel - the counters of that merge
    #  live in the scratch too, re-armed by the kernel and overwritten by the next call's upload)
    wl = configs.batched_decode(R=4, num_pages=4096) if name == "four_long_decodes" else configs.small(name)
    O_ref, L_ref, _ = run_oracle(wl)
    with GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype) as gp:
        gp.install(wl)
        pie.pie_set_option(gp.ctx, pie.PIE_OPT_OVERLAP, 2)      # the static-scratch call never runs kernels side by side
        q, k, v = wl.q("cuda"), wl.k_new("cuda"), wl.v_new("cuda")
        plan = gp.plan(wl)
        assert pie.pie_plan_get_info(plan)["workspace_bytes"] > 0       # the scratch partials are in use (merged in the kernel or by the merge launch)
        ref_out, ref_lse = gp.forward(plan, q, k, v)
        pie.pie_plan_destroy(plan)
        mi, mb = wl.mask_bytes()
        for call in range(2):
            out = torch.full_like(ref_out, float("nan"))
            lse = torch.full_like(ref_lse, float("nan"))
            pie.pie_forward_static_scratch(gp.ctx, wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len,
                                           q, k, v, out, lse, mi, mb)
            torch.cuda.synchronize()
            assert pie.pie_get_last_device_status(gp.ctx) == 0
            assert torch.equal(out, ref_out), f"call {call}"
            assert torch.equal(lse, ref_lse), f"call {call}"
        check_close(out.double().cpu().numpy(), lse.double().cpu().numpy(), O_ref, L_ref, wl.dtype, wl.qo_indptr)


def test_static_scratch_forward_without_output_kvpages():
    """Requests without output KvPages: the rows of a partly filled last input page are carried into a borrowed
    page before the append, outputs equal the planned path's bit for bit and the oracle's within tolerance, and
    after ten calls every borrowed page is back in the free list."""
    import paper_2510_24051_b200 as pie
    from tests._gpu import TOL_LSE, TOL_O
    from tests.test_gpu_parity import no_store_case
    c = no_store_case()
    P, H_q, H_kv, D, R = c["P"], c["H_q"], c["H_kv"], c["D"], c["R"]
    masks, qo, pi, idx, last = c["masks"], c["qo"], c["pi"], c["idx"], c["last"]
    T = len(c["q"])
    tdt = torch.bfloat16
    ctx = pie.pie_create(c["num_pages"], P, H_q, H_kv, D, "bf16", R, T, 0)
    try:
        ids = pie.pie_alloc_kvpages(ctx, 100)
        Kd = torch.from_numpy(np.stack([c["pool"][int(p)][0] for p in ids])).to(tdt).cuda()
        Vd = torch.from_numpy(np.stack([c["pool"][int(p)][1] for p in ids])).to(tdt).cuda()
        pie.pie_kvpage_write(ctx, ids, Kd, Vd)
        pie.pie_mask_kvpage(ctx, [c["hidden_page"]], [c["pm_bits"]])
        ptr = np.zeros(R + 1, np.int64)
        for r, m in enumerate(masks):
            ptr[r + 1] = ptr[r] + (0 if m is None else m.size)
        buf = np.concatenate([m.reshape(-1).astype(np.uint8) for m in masks if m is not None])
        q, k_new, v_new = (torch.from_numpy(x).to(tdt).cuda() for x in (c["q"], c["k_new"], c["v_new"]))
        free0 = pie.pie_num_free_kvpages(ctx)
        plan = pie.pie_plan_forward(ctx, qo, pi, idx, last, ptr, buf, 0, out_len=c["out_len"], no_store=c["no_store"])
        ref_out = torch.full((T, H_q, D), float("nan"), dtype=tdt, device="cuda")
        ref_lse = torch.full((T, H_q), float("nan"), dtype=torch.float32, device="cuda")
        pie.pie_forward(ctx, plan, q, k_new, v_new, ref_out, ref_lse)
        torch.cuda.synchronize()
        pie.pie_plan_destroy(plan)
        assert pie.pie_num_free_kvpages(ctx) == free0
        produced = ~np.isnan(c["L_ref"][:, 0])
        for call in range(10):
            out = torch.full_like(ref_out, float("nan"))
            lse = torch.full_like(ref_lse, float("nan"))
            pie.pie_forward_static_scratch(ctx, qo, pi, idx, last, q, k_new, v_new, out, lse, ptr, buf, 0,
                                           out_len=c["out_len"], no_store=c["no_store"])
            if call < 2:
                torch.cuda.synchronize()
                assert pie.pie_get_last_device_status(ctx) == 0
                assert torch.equal(out.view(torch.int16), ref_out.view(torch.int16)), f"call {call}"     # (bit patterns: untouched rows stay NaN)
                assert torch.equal(lse.view(torch.int32), ref_lse.view(torch.int32)), f"call {call}"
        assert pie.pie_num_free_kvpages(ctx) == free0          # waits for the calls in flight, then every borrowed page is back
        O, L = out.double().cpu().numpy(), lse.double().cpu().numpy()
        assert np.isnan(O[~produced]).all()
        assert np.abs(O[produced] - c["O_ref"][produced]).max() <= TOL_O["bf16"]
        assert np.abs(L[produced] - c["L_ref"][produced]).max() <= TOL_LSE
    finally:
        pie.pie_destroy(ctx)


def test_static_scratch_rejects_batches_beyond_its_size():
    import paper_2510_24051_b200 as pie
    from tests._gpu import GpuPool
    # 72 requests x 64 query tokens x 32,768 context positions of explicit mask pack to 18.9 MB of
    # mask words: more than the 16 MiB array on their own, whatever else the plan holds
    R, q_len, kv_len, P, H_q, H_kv, D = 72, 64, 32768, 16, 4, 2, 64
    npg = kv_len // P
    assert R * q_len * kv_len // 8 > pie.PIE_STATIC_SCRATCH_BYTES
    with GpuPool(R * npg, P, H_q, H_kv, D, "bf16") as gp:
        qo = np.arange(R + 1) * q_len
        pi = np.arange(R + 1) * npg
        mask = np.ones(R * q_len * kv_len, dtype=np.uint8)
        mi = np.arange(R + 1, dtype=np.int64) * q_len * kv_len
        q = torch.zeros((R * q_len, H_q, D), dtype=torch.bfloat16, device="cuda")
        k = torch.zeros((R * q_len, H_kv, D), dtype=torch.bfloat16, device="cuda")
        out = torch.empty_like(q)
        lse = torch.empty((R * q_len, H_q), dtype=torch.float32, device="cuda")
        with pytest.raises(pie.PieError) as e:
            pie.pie_forward_static_scratch(gp.ctx, qo, pi, np.arange(R * npg), np.full(R, P), q, k, k, out, lse, mi, mask)
        assert e.value.status == pie.PIE_ERR_BATCH_TOO_LARGE
