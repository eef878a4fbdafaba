"""Seeded random batches through the whole path against the fp64 oracle: random head grouping, head
dimension and page size, request shapes from one-token decodes to prefill chunks over long contexts,
every mask form (inferred, explicit causal, dropped pages, random token drops, rows with a hidden slot far
into the context), outputs for the last tokens only, all kernel selections.  Outputs, LSE and the pool
after the call (append bit-exact) are compared."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _random_batch(seed):
    from tests.test_gpu_matrix import _bf16_round
    rng = np.random.RandomState(1000 + seed)
    P = int(rng.choice([8, 16, 32]))
    H_q, H_kv = [(8, 2), (32, 8), (4, 4), (6, 2), (16, 1)][rng.randint(5)]
    D = int(rng.choice([64, 128]))
    R = rng.randint(3, 11)
    seqs, out_len = [], []
    for r in range(R):
        kind = rng.choice(["decode", "few", "chunk", "long"], p=[0.35, 0.2, 0.3, 0.15])
        q_len = {"decode": 1, "few": rng.randint(2, 7), "chunk": rng.randint(17, 90), "long": rng.randint(40, 140)}[kind]
        ctx = rng.randint(0, 2200 if kind == "long" else 700)
        kv_len = ctx + q_len
        pos = kv_len - q_len + np.arange(q_len)
        causal = np.arange(kv_len)[None, :] <= pos[:, None]
        form = rng.choice(["inferred", "causal", "pages", "tokens", "late_hole"])
        if form == "inferred":
            mask = None
        else:
            mask = causal.copy()
            npg = (kv_len + P - 1) // P
            if form == "pages" and npg > 2:
                for pg in rng.choice(npg - 1, size=max(1, npg // 4), replace=False):
                    mask[:, pg * P:(pg + 1) * P] = False
            elif form == "tokens":
                mask &= rng.rand(q_len, kv_len) < 0.8
            elif form == "late_hole" and ctx > 4 * P:
                mask[rng.randint(q_len), rng.randint(ctx // 2, ctx)] = False
            mask[np.arange(q_len), pos] = True                       # every row keeps its own token
        s = dict(Q=_bf16_round(rng.randn(q_len, H_q, D).astype(np.float32)),
                 K=_bf16_round(rng.randn(kv_len, H_kv, D).astype(np.float32)),
                 V=_bf16_round(rng.randn(kv_len, H_kv, D).astype(np.float32)))
        if mask is not None:
            s["mask"] = mask
        seqs.append(s)
        out_len.append(q_len if rng.rand() < 0.7 else int(rng.randint(0, q_len + 1)))
    return P, H_q, H_kv, D, seqs, np.array(out_len, dtype=np.int32)


def _random_decode_batch(seed):
    """Decode-shaped batches only (one or two new tokens per request, contexts up to 6,000 tokens, 1 - 24 requests):
    what the split-KV kernel's planner variants see - units of one or two kv heads, whole units per thread block with
    merges inside the block, units cut across blocks with the two-level merge, the kernel writing the new rows."""
    from tests.test_gpu_matrix import _bf16_round
    rng = np.random.RandomState(5000 + seed)
    P = int(rng.choice([8, 16, 32]))
    H_q, H_kv = [(8, 2), (32, 8), (4, 4), (16, 2), (16, 1), (12, 4)][rng.randint(6)]
    D = int(rng.choice([64, 128]))
    R = int(rng.choice([1, 2, 3, 5, 8, 13, 24]))
    two = rng.rand() < 0.3                       # some batches bring two tokens per request (no fused append then)
    long_ctx = 6000 if R <= 5 else 1500
    seqs = []
    for r in range(R):
        q_len = 2 if two and rng.rand() < 0.5 else 1
        ctx = int(rng.randint(0, long_ctx))
        kv_len = ctx + q_len
        pos = kv_len - q_len + np.arange(q_len)
        form = rng.choice(["inferred", "pages", "tokens"], p=[0.6, 0.25, 0.15])
        mask = None
        if form != "inferred":
            mask = np.arange(kv_len)[None, :] <= pos[:, None]
            npg = (kv_len + P - 1) // P
            if form == "pages" and npg > 2:
                for pg in rng.choice(npg - 1, size=max(1, npg // 3), replace=False):
                    mask[:, pg * P:(pg + 1) * P] = False
            elif form == "tokens":
                mask &= rng.rand(q_len, kv_len) < 0.7
            mask[np.arange(q_len), pos] = True
        s = dict(Q=_bf16_round(rng.randn(q_len, H_q, D).astype(np.float32)),
                 K=_bf16_round(rng.randn(kv_len, H_kv, D).astype(np.float32)),
                 V=_bf16_round(rng.randn(kv_len, H_kv, D).astype(np.float32)))
        if mask is not None:
            s["mask"] = mask
        seqs.append(s)
    return P, H_q, H_kv, D, seqs, np.array([len(s["Q"]) for s in seqs], dtype=np.int32)


@pytest.mark.parametrize("seed", range(14))
def test_random_decode_batches_match_oracle(seed):
    _run_random_batch(seed, _random_decode_batch(seed), decode_only=True)


@pytest.mark.parametrize("seed", range(16))
def test_random_batches_match_oracle(seed):
    _run_random_batch(seed, _random_batch(seed))


def _run_random_batch(seed, batch, decode_only=False):
    import paper_2510_24051_b200 as pie
    from oracle import pie_oracle as orc
    from tests._gpu import TOL_LSE, TOL_O
    from tests._util import SmallBatch, same_bits
    P, H_q, H_kv, D, seqs, out_len = batch
    args = SmallBatch(seqs, H_q).paged(P, "random", seed=seed)
    total = len(args["pool"])
    pool_ref = {p: (a.copy(), b.copy()) for p, (a, b) in args["pool"].items()}
    O_ref, L_ref = orc.forward(**dict(args, pool=pool_ref), out_lens=out_len)
    produced = ~np.isnan(L_ref[:, 0])
    T = len(args["q"])
    ptr = np.zeros(len(seqs) + 1, np.int64)
    for r, m in enumerate(args["masks"]):
        ptr[r + 1] = ptr[r] + (0 if m is None else m.size)
    given = [m.reshape(-1).astype(np.uint8) for m in args["masks"] if m is not None]
    buf = np.concatenate(given) if given else np.zeros(0, np.uint8)
    runs = [("bf16", 0, 0), ("bf16", pie.PIE_PLAN_NO_TENSOR_TILES, 0), ("bf16", pie.PIE_PLAN_FORCE_SIMPLE, 0)]
    if decode_only:   # default fusions, then each switched off: append launch, merge launch, one kv head per unit, partials in global memory
        runs = [("bf16", 0, 0), ("bf16", 0, 1 | 2), ("bf16", 0, 4 | 8)]
    if seed % 4 == 3:
        runs.append(("f32", 0, 0))       # the same values in an fp32 pool (the plain kernel), at the fp32 tolerance
    for dtype, flags, no_fusion in runs:
        tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
        ctx = pie.pie_create(total, P, H_q, H_kv, D, dtype, len(seqs), T, 0)
        try:
            pie.pie_set_option(ctx, pie.PIE_OPT_NO_FUSION, no_fusion)
            ids = pie.pie_alloc_kvpages(ctx, total)
            K = torch.from_numpy(np.stack([args["pool"][int(p)][0] for p in ids])).to(tdt).cuda()
            V = torch.from_numpy(np.stack([args["pool"][int(p)][1] for p in ids])).to(tdt).cuda()
            pie.pie_kvpage_write(ctx, ids, K, V)
            plan = pie.pie_plan_forward(ctx, args["qo_indptr"], args["page_indptr"], args["page_indices"],
                                        args["last_page_len"], ptr, buf, flags, out_len=out_len)
            q, k, v = (torch.from_numpy(args[n]).to(tdt).cuda() for n in ("q", "k_new", "v_new"))
            out = torch.full((T, H_q, D), float("nan"), dtype=tdt, device="cuda")
            lse = torch.full((T, H_q), float("nan"), dtype=torch.float32, device="cuda")
            pie.pie_forward(ctx, plan, q, k, v, out, lse)
            torch.cuda.synchronize()
            assert pie.pie_get_last_device_status(ctx) == 0
            pie.pie_plan_destroy(plan)
            O, L = out.double().cpu().numpy(), lse.double().cpu().numpy()
            assert np.isnan(O[~produced]).all() and np.isnan(L[~produced]).all()
            if produced.any():
                assert np.isfinite(O[produced]).all()
                assert np.abs(O[produced] - O_ref[produced]).max() <= TOL_O[dtype], (seed, dtype, flags)
                assert np.abs(L[produced] - L_ref[produced]).max() <= TOL_LSE, (seed, flags)
            Kg = torch.empty((total, P, H_kv, D), dtype=tdt, device="cuda")
            Vg = torch.empty_like(Kg)
            pie.pie_kvpage_read(ctx, np.arange(total, dtype=np.int32), Kg, Vg)
            torch.cuda.synchronize()
            Kb, Vb = Kg.cpu().float().numpy(), Vg.cpu().float().numpy()
            for pg in range(total):
                assert same_bits(np.nan_to_num(Kb[pg], nan=7.0), np.nan_to_num(pool_ref[pg][0], nan=7.0))
                assert same_bits(np.nan_to_num(Vb[pg], nan=7.0), np.nan_to_num(pool_ref[pg][1], nan=7.0))
        finally:
            pie.pie_destroy(ctx)


@pytest.mark.parametrize("seed", range(8))
def test_random_batches_with_requests_that_do_not_store(seed):
    """The same, with a random subset of requests that have no output KvPages (their page lists hold the
    existing context only, possibly nothing) next to requests that store as usual."""
    import paper_2510_24051_b200 as pie
    from oracle import pie_oracle as orc
    from tests._gpu import TOL_LSE, TOL_O
    from tests._util import same_bits
    from tests.test_gpu_matrix import _bf16_round
    rng = np.random.RandomState(5000 + seed)
    P = int(rng.choice([8, 16, 32]))
    H_q, H_kv = [(8, 2), (32, 8), (4, 4), (6, 2)][rng.randint(4)]
    D = int(rng.choice([64, 128]))
    R = rng.randint(3, 9)
    shapes = []
    for r in range(R):
        q_len = int(rng.choice([1, 1, 1, rng.randint(2, 6), rng.randint(17, 80)]))
        kv_in = int(rng.choice([0, rng.randint(1, 2 * P), rng.randint(1, 40) * P, rng.randint(100, 900)]))
        shapes.append((kv_in, q_len, int(rng.rand() < 0.5)))
    n_user = sum(((kv_in if ns else kv_in + q_len) + P - 1) // P for kv_in, q_len, ns in shapes)
    n_borrow = sum((P + q_len + P - 1) // P for kv_in, q_len, ns in shapes if ns)
    num_pages = n_user + n_borrow + 2
    perm = rng.permutation(n_user)
    pool = {p: (np.full((P, H_kv, D), np.nan, np.float32), np.full((P, H_kv, D), np.nan, np.float32)) for p in range(n_user)}
    qo, pi, idx, last, masks, out_len, no_store = [0], [0], [], [], [], [], []
    q_rows, k_rows, v_rows, cur = [], [], [], 0
    for kv_in, q_len, ns in shapes:
        total = kv_in + q_len
        K = _bf16_round(rng.randn(total, H_kv, D).astype(np.float32))
        V = _bf16_round(rng.randn(total, H_kv, D).astype(np.float32))
        n_list = ((kv_in if ns else total) + P - 1) // P
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
        if rng.rand() < 0.4:
            pos = kv_in + np.arange(q_len)
            m = (np.arange(total)[None, :] <= pos[:, None]) & (rng.rand(q_len, total) < 0.8)
            m[np.arange(q_len), pos] = True
        masks.append(m)
        out_len.append(q_len if rng.rand() < 0.7 else int(rng.randint(0, q_len + 1)))
        no_store.append(ns)
        q_rows.append(_bf16_round(rng.randn(q_len, H_q, D).astype(np.float32)))
        k_rows.append(K[kv_in:])
        v_rows.append(V[kv_in:])
    q, k_new, v_new = (np.concatenate(x) for x in (q_rows, k_rows, v_rows))
    qo, pi, idx, last = np.array(qo), np.array(pi), np.array(idx, dtype=np.int64), np.array(last)
    pool_ref = {p: (a.copy(), b.copy()) for p, (a, b) in pool.items()}
    O_ref, L_ref = orc.forward(pool_ref, P, H_q, qo, pi, idx, last, q, k_new, v_new, masks=masks, out_lens=out_len, no_store=no_store)
    produced = ~np.isnan(L_ref[:, 0])
    T = len(q)
    ptr = np.zeros(R + 1, np.int64)
    for r, m in enumerate(masks):
        ptr[r + 1] = ptr[r] + (0 if m is None else m.size)
    given = [m.reshape(-1).astype(np.uint8) for m in masks if m is not None]
    buf = np.concatenate(given) if given else np.zeros(0, np.uint8)
    tdt = torch.bfloat16
    for flags in (0, pie.PIE_PLAN_NO_TENSOR_TILES):
        ctx = pie.pie_create(num_pages, P, H_q, H_kv, D, "bf16", R, T, 0)
        try:
            ids = pie.pie_alloc_kvpages(ctx, n_user)
            assert sorted(ids) == list(range(n_user))
            Kd = torch.from_numpy(np.stack([pool[int(p)][0] for p in ids])).to(tdt).cuda()
            Vd = torch.from_numpy(np.stack([pool[int(p)][1] for p in ids])).to(tdt).cuda()
            pie.pie_kvpage_write(ctx, ids, Kd, Vd)
            free0 = pie.pie_num_free_kvpages(ctx)
            plan = pie.pie_plan_forward(ctx, qo, pi, idx, last, ptr, buf, flags, out_len=out_len, no_store=no_store)
            out = torch.full((T, H_q, D), float("nan"), dtype=tdt, device="cuda")
            lse = torch.full((T, H_q), float("nan"), dtype=torch.float32, device="cuda")
            pie.pie_forward(ctx, plan, *(torch.from_numpy(x).to(tdt).cuda() for x in (q, k_new, v_new)), out, lse)
            torch.cuda.synchronize()
            assert pie.pie_get_last_device_status(ctx) == 0
            pie.pie_plan_destroy(plan)
            assert pie.pie_num_free_kvpages(ctx) == free0
            O, L = out.double().cpu().numpy(), lse.double().cpu().numpy()
            assert np.isnan(O[~produced]).all()
            if produced.any():
                assert np.abs(O[produced] - O_ref[produced]).max() <= TOL_O["bf16"], (seed, flags)
                assert np.abs(L[produced] - L_ref[produced]).max() <= TOL_LSE, (seed, flags)
            Kg = torch.empty((n_user, P, H_kv, D), dtype=tdt, device="cuda")
            Vg = torch.empty_like(Kg)
            pie.pie_kvpage_read(ctx, np.arange(n_user, dtype=np.int32), Kg, Vg)
            torch.cuda.synchronize()
            Kb, Vb = Kg.cpu().float().numpy(), Vg.cpu().float().numpy()
            for pg in range(n_user):
                assert same_bits(np.nan_to_num(Kb[pg], nan=7.0), np.nan_to_num(pool_ref[pg][0], nan=7.0)), pg
                assert same_bits(np.nan_to_num(Vb[pg], nan=7.0), np.nan_to_num(pool_ref[pg][1], nan=7.0)), pg
        finally:
            pie.pie_destroy(ctx)
