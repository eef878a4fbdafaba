"""GPU-side helpers for the parity tests: everything goes through the C ABI binding."""
from __future__ import annotations

import numpy as np
import torch

import paper_2510_24051_b200 as pie
from workloads import synth

TOL_O = {"bf16": 2e-2, "f32": 1e-4}
TOL_LSE = 1e-3
TOL_RMS = {"bf16": 1e-2, "f32": 1e-5}
TDTYPE = {"bf16": torch.bfloat16, "f32": torch.float32}


class GpuPool:
    """A context whose whole pool is allocated, so page ids equal the workload's ids."""

    def __init__(self, num_pages, P, H_q, H_kv, D, dtype, max_requests=4096, max_query_tokens=1 << 17):
        self.args = (num_pages, P, H_q, H_kv, D, dtype)
        self.ctx = pie.pie_create(num_pages, P, H_q, H_kv, D, dtype, max_requests, max_query_tokens, 0)
        ids = pie.pie_alloc_kvpages(self.ctx, num_pages)
        assert np.array_equal(ids, np.arange(num_pages))
        self.P, self.H_q, self.H_kv, self.D, self.dtype = P, H_q, H_kv, D, dtype

    def close(self):
        if self.ctx is not None:
            torch.cuda.synchronize()
            pie.pie_destroy(self.ctx)
            self.ctx = None

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    def install(self, wl, poison=False, chunk=2048, pages=None):
        used = wl.used_pages() if pages is None else np.asarray(pages)
        for i in range(0, len(used), chunk):
            ids = used[i:i + chunk]
            K, V = wl.context_pages(ids, "cuda", poison=poison)
            pie.pie_kvpage_write(self.ctx, ids, K.contiguous(), V.contiguous())
        torch.cuda.synchronize()

    def read_pages(self, ids):
        ids = np.asarray(ids, dtype=np.int32)
        shape = (len(ids), self.P, self.H_kv, self.D)
        K = torch.empty(shape, dtype=TDTYPE[self.dtype], device="cuda")
        V = torch.empty_like(K)
        pie.pie_kvpage_read(self.ctx, ids, K, V)
        torch.cuda.synchronize()
        return synth.to_numpy_bits(K), synth.to_numpy_bits(V)

    def plan(self, wl, flags=0):
        mi, mb = wl.mask_bytes()
        return pie.pie_plan_forward(self.ctx, wl.qo_indptr, wl.page_indptr, wl.page_indices,
                                    wl.last_page_len, mi, mb, flags)

    def forward(self, plan, q, k_new, v_new):
        T = q.shape[0]
        out = torch.full((T, self.H_q, self.D), float("nan"), dtype=q.dtype, device="cuda")
        lse = torch.full((T, self.H_q), float("nan"), dtype=torch.float32, device="cuda")
        pie.pie_forward(self.ctx, plan, q, k_new, v_new, out, lse)
        torch.cuda.synchronize()
        assert pie.pie_get_last_device_status(self.ctx) == 0
        return out, lse


def run_workload(wl, poison=False, flags=0, q_scale=1.0, keep=False):
    """Install context, plan, forward.  Returns O (fp64 numpy), LSE (fp64 numpy) [, pool]."""
    gp = GpuPool(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype)
    try:
        gp.install(wl, poison=poison)
        plan = gp.plan(wl, flags)
        q = wl.q("cuda")
        if q_scale != 1.0:
            q = (q.float() * q_scale).to(q.dtype)
        out, lse = gp.forward(plan, q, wl.k_new("cuda"), wl.v_new("cuda"))
        info = pie.pie_plan_get_info(plan)
        pie.pie_plan_destroy(plan)
        res = (out.double().cpu().numpy(), lse.double().cpu().numpy(), info)
        if keep:
            return res + (gp,)
        return res
    finally:
        if not keep:
            gp.close()


def check_close(O, LSE, O_ref, LSE_ref, dtype, qo_indptr=None, rows=None):
    """The acceptance gate: max-abs error on O, abs error on LSE, and per-request relative RMS."""
    if rows is not None:
        O, LSE, O_ref, LSE_ref = O[rows], LSE[rows], O_ref[rows], LSE_ref[rows]
    assert np.isfinite(O).all(), "non-finite output"
    err = np.abs(O - O_ref).max() if O.size else 0.0
    assert err <= TOL_O[dtype], f"max |O - O*| = {err}"
    neg = np.isneginf(LSE_ref)
    assert np.array_equal(np.isneginf(LSE), neg)
    if (~neg).any():
        lerr = np.abs(LSE[~neg] - LSE_ref[~neg]).max()
        assert lerr <= TOL_LSE, f"max |LSE - LSE*| = {lerr}"
    if qo_indptr is not None and rows is None:
        for r in range(len(qo_indptr) - 1):
            a, b = qo_indptr[r], qo_indptr[r + 1]
            den = np.sqrt((O_ref[a:b] ** 2).sum())
            if den > 0:
                rel = np.sqrt(((O[a:b] - O_ref[a:b]) ** 2).sum()) / den
                assert rel <= TOL_RMS[dtype], f"request {r}: relative RMS error {rel}"
    return err
