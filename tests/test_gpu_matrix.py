"""Tiny-case matrix on the GPU: page size x head grouping x head dim x element type, each as one
batch that mixes context lengths {1, P-1, P, P+1, 3P+5}, query lengths {1, 2, all}, every mask
form (inferred causal, explicit causal, one-hot rows, random, dropped pages, an empty row) and
every placement (contiguous, reversed, random, pages shared between two requests).  Unused
slots hold NaN bit patterns.  Compared element by element with the fp64 oracle."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

MASKS = ["inferred", "explicit_causal", "one_hot", "random", "page_dropped", "empty_row"]


def _bf16_round(x):
    return torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()


def build_case(P, H_q, H_kv, D, dtype, order, seed):
    rng = np.random.RandomState(seed)
    rnd = (lambda *s: _bf16_round(rng.randn(*s).astype(np.float32))) if dtype == "bf16" else \
        (lambda *s: rng.randn(*s).astype(np.float32))
    reqs, k = [], 0
    for kv_len in sorted({1, P - 1, P, P + 1, 3 * P + 5}):
        for q_len in sorted({1, 2, kv_len}):
            if q_len > kv_len:
                continue
            for rep in range(2):
                kind = MASKS[k % len(MASKS)]
                k += 1
                pos = kv_len - q_len + np.arange(q_len)
                causal = np.arange(kv_len)[None, :] <= pos[:, None]
                if kind == "inferred":
                    mask = None
                elif kind == "explicit_causal":
                    mask = causal.copy()
                elif kind == "one_hot":
                    mask = np.zeros((q_len, kv_len), bool)
                    mask[np.arange(q_len), rng.randint(0, kv_len, q_len)] = True
                elif kind == "random":
                    mask = rng.rand(q_len, kv_len) < 0.5
                elif kind == "page_dropped":
                    mask = causal.copy()
                    for pg in range(0, (kv_len + P - 1) // P, 2):
                        mask[:, pg * P:(pg + 1) * P] = False
                else:
                    mask = causal.copy()
                    mask[0, :] = False
                reqs.append(dict(Q=rnd(q_len, H_q, D), K=rnd(kv_len, H_kv, D), V=rnd(kv_len, H_kv, D), mask=mask,
                                 kind=kind))
    # a pair that shares its first two (full, read-only) pages
    base = dict(Q=rnd(1, H_q, D), K=rnd(2 * P + 3, H_kv, D), V=rnd(2 * P + 3, H_kv, D), mask=None, kind="inferred")
    twin = dict(Q=rnd(2, H_q, D), K=np.concatenate([base["K"][:2 * P], rnd(P + 2, H_kv, D)]),
                V=np.concatenate([base["V"][:2 * P], rnd(P + 2, H_kv, D)]), mask=None, kind="inferred", share=True)
    reqs += [base, twin]

    nps = [(len(r["K"]) + P - 1) // P for r in reqs]
    total = sum(nps) + 5
    ids = np.arange(total)
    if order == "reversed":
        ids = ids[::-1].copy()
    elif order == "random":
        ids = rng.permutation(total)
    pool = {int(p): (np.full((P, H_kv, D), np.nan, np.float32), np.full((P, H_kv, D), np.nan, np.float32))
            for p in range(total)}
    qo, pi, idx, last, cur = [0], [0], [], [], 0
    base_pages = None
    for r, n in zip(reqs, nps):
        pages = ids[cur:cur + n].copy()
        cur += n
        if r is base:
            base_pages = pages
        if r.get("share"):
            pages[:2] = base_pages[:2]
        kv_len, q_len = len(r["K"]), len(r["Q"])
        for j in range(kv_len - q_len):
            Kp, Vp = pool[int(pages[j // P])]
            Kp[j % P], Vp[j % P] = r["K"][j], r["V"][j]
        qo.append(qo[-1] + q_len)
        pi.append(pi[-1] + n)
        idx.extend(pages.tolist())
        last.append(kv_len - (n - 1) * P)
    args = dict(pool=pool, P=P, H_q=H_q, qo_indptr=np.array(qo), page_indptr=np.array(pi), page_indices=np.array(idx),
                last_page_len=np.array(last), q=np.concatenate([r["Q"] for r in reqs]),
                k_new=np.concatenate([r["K"][len(r["K"]) - len(r["Q"]):] for r in reqs]),
                v_new=np.concatenate([r["V"][len(r["V"]) - len(r["Q"]):] for r in reqs]),
                masks=[r["mask"] for r in reqs])
    return args, reqs, total


def run_gpu(args, total, H_kv, D, dtype, flags=0, options=None):
    import paper_2510_24051_b200 as pie
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    P, H_q = args["P"], args["H_q"]
    T = len(args["q"])
    ctx = pie.pie_create(total, P, H_q, H_kv, D, dtype, len(args["last_page_len"]), T, 0)
    try:
        for opt, value in (options or {}).items():
            pie.pie_set_option(ctx, opt, value)
        ids = pie.pie_alloc_kvpages(ctx, total)
        K = torch.from_numpy(np.stack([args["pool"][int(p)][0] for p in ids])).to(tdt).cuda()
        V = torch.from_numpy(np.stack([args["pool"][int(p)][1] for p in ids])).to(tdt).cuda()
        pie.pie_kvpage_write(ctx, ids, K, V)
        ptr = np.zeros(len(args["masks"]) + 1, np.int64)
        for r, m in enumerate(args["masks"]):
            ptr[r + 1] = ptr[r] + (0 if m is None else m.size)
        given = [m.reshape(-1).astype(np.uint8) for m in args["masks"] if m is not None]
        buf = np.concatenate(given) if given else np.zeros(0, np.uint8)
        plan = pie.pie_plan_forward(ctx, args["qo_indptr"], args["page_indptr"], args["page_indices"],
                                    args["last_page_len"], ptr, buf, flags)
        q, k, v = (torch.from_numpy(args[n]).to(tdt).cuda() for n in ("q", "k_new", "v_new"))
        out = torch.full((T, H_q, D), float("nan"), dtype=tdt, device="cuda")
        lse = torch.full((T, H_q), float("nan"), dtype=torch.float32, device="cuda")
        pie.pie_forward(ctx, plan, q, k, v, out, lse)
        torch.cuda.synchronize()
        assert pie.pie_get_last_device_status(ctx) == 0
        info = pie.pie_plan_get_info(plan)
        pie.pie_plan_destroy(plan)
        return out.double().cpu().numpy(), lse.double().cpu().numpy(), info
    finally:
        pie.pie_destroy(ctx)


@pytest.mark.parametrize("order", ["contiguous", "reversed", "random"])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("heads", [(1, 1), (4, 2), (8, 1)])
@pytest.mark.parametrize("P", [8, 16, 32])
def test_tiny_case_matrix(P, heads, D, dtype, order):
    from oracle import pie_oracle as orc
    from tests._gpu import TOL_LSE, TOL_O
    H_q, H_kv = heads
    if order != "random" and dtype == "f32":
        pytest.skip("placement variants are run on the tensor-core paths only")
    args, reqs, total = build_case(P, H_q, H_kv, D, dtype, order, seed=P * 1000 + H_q * 10 + D)
    O_ref, L_ref = orc.forward(**{k: (v if k != "pool" else {p: (a.copy(), b.copy()) for p, (a, b) in v.items()})
                                  for k, v in args.items()})
    for flags in ([0, 2] if dtype == "bf16" else [0]):
        O, L, info = run_gpu(args, total, H_kv, D, dtype, flags)
        if dtype == "bf16":    # every page size runs on the tensor-core kernels (8-token pages in pairs / 16 page boxes per tile)
            assert info["num_split_items"] + info["num_tile_items"] > 0
        assert np.isfinite(O).all()
        assert np.abs(O - O_ref).max() <= TOL_O[dtype], (flags, np.abs(O - O_ref).max())
        neg = np.isneginf(L_ref)
        assert np.array_equal(np.isneginf(L), neg)
        assert np.abs(L[~neg] - L_ref[~neg]).max() <= TOL_LSE
        assert not O[neg].any()                               # empty rows: exact zeros
        # one-hot rows return the selected V row exactly, also in bf16
        t = 0
        for r in reqs:
            q_len = len(r["Q"])
            if r["kind"] == "one_hot":
                assert np.array_equal(O[t:t + q_len], O_ref[t:t + q_len]), f"one-hot rows not exact (flags {flags})"
            t += q_len


def test_empty_batch_and_degenerate_calls():
    import paper_2510_24051_b200 as pie
    ctx = pie.pie_create(8, 16, 4, 2, 64, "bf16", 4, 16, 0)
    try:
        plan = pie.pie_plan_forward(ctx, [0], [0], [], [])
        pie.pie_forward(ctx, plan, None, None, None, None, None)      # nothing to do, nothing enqueued
        assert pie.pie_plan_get_info(plan)["launches"] == 0
        pie.pie_plan_destroy(plan)
        pie.pie_kvpage_write(ctx, [], None, None)
        pie.pie_copy_kvpage(ctx, [], [], [], [], [])
        torch.cuda.synchronize()
        assert pie.pie_get_last_device_status(ctx) == 0
    finally:
        pie.pie_destroy(ctx)
