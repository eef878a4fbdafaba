"""pie_forward_static_scratch: the forward call for hosts that cannot allocate device memory when a
batch runs (a frozen or externally owned device heap, or a serving loop that must avoid the
implicit synchronisation of cudaMalloc / cudaFree).  Its plan arrays and split partials live in a
fixed device array inside the library instead of a per-plan allocation, so its results must be
the ones pie_plan_forward + pie_forward give.  Checked through the C ABI on two calls in a row
(the second call reuses the array with the first call's contents still in it), on a decode batch
whose split partials go through the merge and on a mixed batch with explicit masks."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["batched_decode", "long_context_policy", "mixed_prefill_decode"])
def test_static_scratch_forward_matches_planned_forward(name):
    import paper_2510_24051_b200 as pie
    from tests._gpu import GpuPool, TOL_LSE, TOL_O
    from workloads import configs
    wl = configs.small(name)
    with GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype) as gp:
        gp.install(wl)
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
            assert (out.float() - ref_out.float()).abs().max().item() <= TOL_O[wl.dtype], f"call {call}"
            fin = torch.isfinite(ref_lse)
            assert torch.equal(torch.isfinite(lse), fin)
            assert (lse[fin] - ref_lse[fin]).abs().max().item() <= TOL_LSE, f"call {call}"


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
