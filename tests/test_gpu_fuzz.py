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
    P = int(rng.choice([16, 32]))
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


@pytest.mark.parametrize("seed", range(16))
def test_random_batches_match_oracle(seed):
    import paper_2510_24051_b200 as pie
    from oracle import pie_oracle as orc
    from tests._gpu import TOL_LSE, TOL_O
    from tests._util import SmallBatch, same_bits
    P, H_q, H_kv, D, seqs, out_len = _random_batch(seed)
    args = SmallBatch(seqs, H_q).paged(P, "random", seed=seed)
    total = len(args["pool"])
    pool_ref = {p: (a.copy(), b.copy()) for p, (a, b) in args["pool"].items()}
    O_ref, L_ref = orc.forward(**dict(args, pool=pool_ref), out_lens=out_len)
    produced = ~np.isnan(L_ref[:, 0])
    T = len(args["q"])
    tdt = torch.bfloat16
    ptr = np.zeros(len(seqs) + 1, np.int64)
    for r, m in enumerate(args["masks"]):
        ptr[r + 1] = ptr[r] + (0 if m is None else m.size)
    given = [m.reshape(-1).astype(np.uint8) for m in args["masks"] if m is not None]
    buf = np.concatenate(given) if given else np.zeros(0, np.uint8)
    for flags in (0, pie.PIE_PLAN_NO_TENSOR_TILES, pie.PIE_PLAN_FORCE_SIMPLE):
        ctx = pie.pie_create(total, P, H_q, H_kv, D, "bf16", len(seqs), T, 0)
        try:
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
                assert np.abs(O[produced] - O_ref[produced]).max() <= TOL_O["bf16"], (seed, flags)
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
