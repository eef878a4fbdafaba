"""Pins for the fp64 oracle: each test fixes it to something other than itself - scalar
textbook loops, brute force, closed forms, invariants, and the equivalences the paper
states in Section 4.2 (split forward, prefill == decode loop, page omission == masking)."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import pie_oracle as orc
from tests._util import SmallBatch, oracle_on, random_seqs, run_oracle
from workloads import configs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_example.txt")


# ---------------------------------------------------------------- scalar textbook reference
def textbook_attention(Q, K, V, allowed):
    """Scalar-loop softmax attention over dense arrays: the definition, nothing else."""
    q_len, H_q, D = Q.shape
    G = H_q // K.shape[1]
    O = np.zeros((q_len, H_q, D))
    L = np.full((q_len, H_q), -math.inf)
    for i in range(q_len):
        for h in range(H_q):
            js = [j for j in range(K.shape[0]) if allowed[i][j]]
            if not js:
                continue
            s = [sum(float(Q[i, h, d]) * float(K[j, h // G, d]) for d in range(D)) / math.sqrt(D)
                 for j in js]
            Z = math.fsum(math.exp(x) for x in s)
            for d in range(D):
                O[i, h, d] = math.fsum(math.exp(x) * float(V[j, h // G, d]) for x, j in zip(s, js)) / Z
            L[i, h] = math.log(Z)
    return O, L


def causal(q_len, kv_len):
    return [[j <= kv_len - q_len + i for j in range(kv_len)] for i in range(q_len)]


# p1 ------------------------------------------------------------------------------------
@pytest.mark.parametrize("P", [8, 16])
def test_p1_contiguous_causal_equals_textbook(P):
    rng = np.random.RandomState(1)
    shapes = [(1, 19), (5, 5), (7, 33)]
    seqs = random_seqs(rng, shapes, H_q=4, H_kv=2, D=8)
    O, L = oracle_on(SmallBatch(seqs, 4).paged(P, "contiguous"))
    t = 0
    for s, (q_len, kv_len) in zip(seqs, shapes):
        Or, Lr = textbook_attention(s["Q"], s["K"], s["V"], causal(q_len, kv_len))
        np.testing.assert_allclose(O[t:t + q_len], Or, rtol=0, atol=1e-12)
        np.testing.assert_allclose(L[t:t + q_len], Lr, rtol=0, atol=1e-12)
        t += q_len


# p2 ------------------------------------------------------------------------------------
def test_p2_physical_page_permutation_is_bit_invariant():
    rng = np.random.RandomState(2)
    m = rng.rand(4, 50) < 0.6
    m[:, 0] = True
    seqs = random_seqs(rng, [(1, 37), (4, 50), (3, 16)], 4, 2, 16, masks=[None, m, None])
    ref = oracle_on(SmallBatch(seqs, 4).paged(16, "contiguous"))
    for order, seed in [("reversed", 0), ("random", 3), ("random", 4)]:
        got = oracle_on(SmallBatch(seqs, 4).paged(16, order, seed=seed))
        assert np.array_equal(ref[0], got[0]) and np.array_equal(ref[1], got[1])


# p3 ------------------------------------------------------------------------------------
def test_p3_page_size_is_bit_invariant():
    rng = np.random.RandomState(3)
    seqs = random_seqs(rng, [(1, 31), (6, 70), (2, 8)], 8, 1, 16)
    ref = oracle_on(SmallBatch(seqs, 8).paged(8, "random", seed=1))
    for P in (16, 32):
        got = oracle_on(SmallBatch(seqs, 8).paged(P, "random", seed=P))
        assert np.array_equal(ref[0], got[0]) and np.array_equal(ref[1], got[1])


# p4 ------------------------------------------------------------------------------------
def test_p4_one_hot_rows_return_that_v_row_exactly():
    rng = np.random.RandomState(4)
    kv_len, q_len = 45, 6
    pick = rng.randint(0, kv_len, size=q_len)
    m = np.zeros((q_len, kv_len), dtype=bool)
    m[np.arange(q_len), pick] = True
    seqs = random_seqs(rng, [(q_len, kv_len)], 4, 2, 16, masks=[m])
    O, L = oracle_on(SmallBatch(seqs, 4).paged(16, "random"))
    s = seqs[0]
    for i in range(q_len):
        for h in range(4):
            assert np.array_equal(O[i, h], s["V"][pick[i], h // 2].astype(np.float64))
            sc = float(np.dot(s["Q"][i, h].astype(np.float64), s["K"][pick[i], h // 2].astype(np.float64))) / 4.0
            assert abs(L[i, h] - sc) < 1e-13


# p5 ------------------------------------------------------------------------------------
def test_p5_brute_force_all_masks_tiny():
    rng = np.random.RandomState(5)
    D = 4
    for kv_len in (1, 2, 3, 4):
        for q_len in (1, 2):
            if q_len > kv_len:
                continue
            rows = list(itertools.product([False, True], repeat=kv_len))
            for combo in itertools.islice(itertools.product(rows, repeat=q_len), 0, None, 3 if q_len == 2 else 1):
                m = np.array(combo, dtype=bool)
                seqs = random_seqs(rng, [(q_len, kv_len)], 2, 1, D, masks=[m])
                O, L = oracle_on(SmallBatch(seqs, 2).paged(8))
                Or, Lr = textbook_attention(seqs[0]["Q"], seqs[0]["K"], seqs[0]["V"], m)
                np.testing.assert_allclose(O, Or, rtol=0, atol=1e-13)
                assert np.array_equal(np.isneginf(L), np.isneginf(Lr))
                fin = np.isfinite(Lr)
                np.testing.assert_allclose(L[fin], Lr[fin], rtol=0, atol=1e-13)
                for i in range(q_len):      # empty row: zero output, LSE = -inf
                    if not m[i].any():
                        assert not O[i].any() and np.isneginf(L[i]).all()


# p6 ------------------------------------------------------------------------------------
def test_p6_closed_forms():
    rng = np.random.RandomState(6)
    kv_len, q_len = 40, 3
    m = rng.rand(q_len, kv_len) < 0.5
    m[:, 5] = True
    seqs = random_seqs(rng, [(q_len, kv_len)], 4, 2, 16, masks=[m])
    base = seqs[0]
    # Q = 0: uniform weights over the allowed set
    z = dict(base, Q=np.zeros_like(base["Q"]))
    O, L = oracle_on(SmallBatch([z], 4).paged(16))
    for i in range(q_len):
        for h in range(4):
            np.testing.assert_allclose(O[i, h], base["V"][m[i], h // 2].astype(np.float64).mean(0), atol=1e-14)
            assert abs(L[i, h] - math.log(m[i].sum())) < 1e-14
    # all K rows equal: uniform weights again, LSE = score + ln|S|
    kk = dict(base, K=np.broadcast_to(base["K"][:1], base["K"].shape).copy())
    O2, L2 = oracle_on(SmallBatch([kk], 4).paged(16))
    np.testing.assert_allclose(O2, O, atol=1e-13)
    # V constant: output is that constant for any mask
    c = rng.randn(2, 16).astype(np.float32)
    vc = dict(base, V=np.broadcast_to(c, base["V"].shape).copy())
    O3, _ = oracle_on(SmallBatch([vc], 4).paged(16))
    for h in range(4):
        np.testing.assert_allclose(O3[:, h], np.broadcast_to(c[h // 2].astype(np.float64), (q_len, 16)), atol=1e-14)
    # V + u shifts O by u and leaves LSE alone (V on a 2^-10 grid so the shift is exact in fp32)
    Vq = (np.round(base["V"].astype(np.float64) * 1024) / 1024).astype(np.float32)
    O4, L4 = oracle_on(SmallBatch([dict(base, V=Vq)], 4).paged(16))
    O5, L5 = oracle_on(SmallBatch([dict(base, V=(Vq.astype(np.float64) + 0.5).astype(np.float32))], 4).paged(16))
    np.testing.assert_allclose(O5, O4 + 0.5, atol=1e-13)
    np.testing.assert_array_equal(L5, L4)


# p7 ------------------------------------------------------------------------------------
def test_p7_lse_merge_identity():
    rng = np.random.RandomState(7)
    kv_len, q_len = 64, 4
    full = rng.rand(q_len, kv_len) < 0.7
    full[:, 0] = True
    part = rng.randint(0, 3, size=kv_len)                 # three disjoint column classes
    part[10:20] = 2
    seqs = random_seqs(rng, [(q_len, kv_len)], 4, 2, 16, masks=[full])
    O, L = oracle_on(SmallBatch(seqs, 4).paged(16))
    Os, Ls = [], []
    for c in range(3):
        mc = full & (part[None, :] == c)
        if c == 1:
            mc[2, :] = False                              # an empty part for one row
            full_row2 = full[2] & (part != 1)
        s = dict(seqs[0], mask=mc)
        o, l = oracle_on(SmallBatch([s], 4).paged(16))
        Os.append(o), Ls.append(l)
    # row 2 lost its class-1 columns: recompute the reference for that row's reduced set
    f2 = full.copy()
    f2[2] = full_row2
    O, L = oracle_on(SmallBatch([dict(seqs[0], mask=f2)], 4).paged(16))
    Om, Lm = orc.merge_partials(Os, Ls)
    np.testing.assert_allclose(Om, O, atol=1e-13)
    np.testing.assert_allclose(Lm, L, atol=1e-13)


# p8 ------------------------------------------------------------------------------------
def test_p8_split_forward_and_decode_loop_equal_one_prefill():
    """Section 4.2: a 9-token prefill equals an 8-token forward that fills KvPages followed
    by a 1-token forward that reads them; and prefill equals the token-by-token loop."""
    rng = np.random.RandomState(8)
    n, P, H_q, H_kv, D = 21, 8, 4, 2, 16
    Q = rng.randn(n, H_q, D).astype(np.float32)
    K = rng.randn(n, H_kv, D).astype(np.float32)
    V = rng.randn(n, H_kv, D).astype(np.float32)
    O_full, L_full = oracle_on(SmallBatch([dict(Q=Q, K=K, V=V)], H_q).paged(P, "random", seed=1))

    npg = (n + P - 1) // P
    pages = np.random.RandomState(9).permutation(npg + 2)[:npg]
    pool = {int(p): (np.full((P, H_kv, D), np.nan, np.float32), np.full((P, H_kv, D), np.nan, np.float32))
            for p in range(npg + 2)}

    def step(lo, hi):
        np_r = (hi + P - 1) // P
        return orc.forward(pool, P, H_q, np.array([0, hi - lo]), np.array([0, np_r]), pages[:np_r],
                           np.array([hi - (np_r - 1) * P]), Q[lo:hi], K[lo:hi], V[lo:hi])

    O1, L1 = step(0, n - 1)          # fills the pages with n-1 tokens
    O2, L2 = step(n - 1, n)          # one token reading them
    np.testing.assert_allclose(np.concatenate([O1, O2]), O_full, atol=1e-14)
    np.testing.assert_allclose(np.concatenate([L1, L2]), L_full, atol=1e-14)

    for p in pool:                    # token-by-token from an empty cache
        pool[p][0][:] = np.nan
        pool[p][1][:] = np.nan
    outs = [step(i, i + 1) for i in range(n)]
    np.testing.assert_allclose(np.concatenate([o for o, _ in outs]), O_full, atol=1e-14)
    np.testing.assert_allclose(np.concatenate([l for _, l in outs]), L_full, atol=1e-14)


# p9 ------------------------------------------------------------------------------------
def test_p9_page_omission_equals_masking():
    rng = np.random.RandomState(10)
    P, kv_len, H_q, H_kv, D = 8, 48, 4, 2, 16
    seq = random_seqs(rng, [(1, kv_len)], H_q, H_kv, D)[0]
    drop_pages = [1, 3]
    keep = np.ones(kv_len, dtype=bool)
    for p in drop_pages:
        keep[p * P:(p + 1) * P] = False
    O_mask, L_mask = oracle_on(SmallBatch([dict(seq, mask=keep[None, :])], H_q).paged(P, "random"))
    short = dict(Q=seq["Q"], K=seq["K"][keep], V=seq["V"][keep])     # pages simply left out
    O_omit, L_omit = oracle_on(SmallBatch([short], H_q).paged(P, "random", seed=5))
    np.testing.assert_allclose(O_omit, O_mask, atol=1e-14)
    np.testing.assert_allclose(L_omit, L_mask, atol=1e-14)


# p10 -----------------------------------------------------------------------------------
def test_p10_shared_pages_equal_private_copies():
    wl = configs.small("shared_prefix_tree")
    O, L, _ = run_oracle(wl)
    # give every branch a private copy of its group's prefix pages via copy_kvpage
    pool = wl.oracle_pool()
    n_pre = wl.meta["prefix"] // wl.P
    free = [p for p in range(wl.num_pages) if wl.page_owner[p] < 0]
    idx = wl.page_indices.copy()
    src, dst = [], []
    for r in range(wl.R):
        if r % wl.meta["branches"] == 0:
            continue                                       # first branch keeps the original
        base = wl.page_indptr[r]
        for k in range(n_pre):
            new = free.pop()
            src.append(idx[base + k]), dst.append(new)
            idx[base + k] = new
    for p in dst:
        pool[p] = (np.zeros((wl.P, wl.H_kv, wl.D), np.uint16), np.zeros((wl.P, wl.H_kv, wl.D), np.uint16))
    n = len(src)
    orc.copy_kvpage(pool, src, dst, [0] * n, [0] * n, [wl.P] * n)
    from tests._util import bits
    O2, L2 = orc.forward(pool, wl.P, wl.H_q, wl.qo_indptr, wl.page_indptr, idx, wl.last_page_len,
                         bits(wl.q()), bits(wl.k_new()), bits(wl.v_new()), wl.masks)
    assert np.array_equal(O, O2) and np.array_equal(L, L2)


def test_copy_kvpage_token_ranges():
    P, H, D = 8, 2, 4
    rng = np.random.RandomState(11)
    pool = {p: (rng.randn(P, H, D).astype(np.float32), rng.randn(P, H, D).astype(np.float32)) for p in range(4)}
    before = {p: (k.copy(), v.copy()) for p, (k, v) in pool.items()}
    orc.copy_kvpage(pool, [0, 1], [2, 0], [1, 0], [3, 5], [4, 2])
    for kv in (0, 1):
        exp2 = before[2][kv].copy()
        exp2[3:7] = before[0][kv][1:5]
        exp0 = before[0][kv].copy()
        exp0[5:7] = before[1][kv][0:2]
        assert np.array_equal(pool[2][kv], exp2) and np.array_equal(pool[0][kv], exp0)
        assert np.array_equal(pool[1][kv], before[1][kv]) and np.array_equal(pool[3][kv], before[3][kv])


# p11 -----------------------------------------------------------------------------------
def test_p11_tree_mask_equals_causal_path():
    wl = configs.small("shared_prefix_tree")
    O, L, pool = run_oracle(wl)
    from tests._util import bits
    q, k_new, v_new = bits(wl.q()), bits(wl.k_new()), bits(wl.v_new())
    ctx = wl.meta["prefix"] + wl.meta["suffix"]
    for r in (0, wl.R - 1):
        par = wl.meta["parents"][r]
        t0 = wl.qo_indptr[r]
        pages = wl.pages_of(r)
        Kc, Vc = orc.gather_kv(pool, wl.P, pages, ctx)      # context rows (post-append pool)
        for n in (0, 5, len(par) - 1):
            path = []
            a = n
            while a >= 0:
                path.append(a)
                a = par[a]
            path = path[::-1]                                # root .. n
            K = np.concatenate([Kc, orc.widen(k_new[t0 + np.array(path)])])
            V = np.concatenate([Vc, orc.widen(v_new[t0 + np.array(path)])])
            Or, Lr = textbook_free(orc.widen(q[t0 + n])[None], K, V)
            np.testing.assert_allclose(O[t0 + n], Or[0], atol=1e-12)
            np.testing.assert_allclose(L[t0 + n], Lr[0], atol=1e-12)


def textbook_free(Q, K, V):
    """Dense unmasked attention of the LAST query position over all rows, vectorised
    differently from the oracle (einsum + logsumexp by hand)."""
    q_len, H_q, D = Q.shape
    G = H_q // K.shape[1]
    Kh = np.repeat(K, G, axis=1)
    Vh = np.repeat(V, G, axis=1)
    s = np.einsum("ihd,jhd->ihj", Q, Kh) / math.sqrt(D)
    Z = np.exp(s).sum(-1)
    return np.einsum("ihj,jhd->ihd", np.exp(s), Vh) / Z[..., None], np.log(Z)


# p12 -----------------------------------------------------------------------------------
def test_p12_gqa_equals_repeated_mha():
    rng = np.random.RandomState(12)
    seqs = random_seqs(rng, [(3, 29), (1, 12)], 8, 2, 16)
    O, L = oracle_on(SmallBatch(seqs, 8).paged(8, "random"))
    rep = [dict(Q=s["Q"], K=np.repeat(s["K"], 4, axis=1), V=np.repeat(s["V"], 4, axis=1)) for s in seqs]
    O2, L2 = oracle_on(SmallBatch(rep, 8).paged(8, "random"))
    np.testing.assert_allclose(O2, O, atol=1e-14)
    np.testing.assert_allclose(L2, L, atol=1e-14)


# p13 -----------------------------------------------------------------------------------
def test_p13_append_touches_exactly_the_new_rows_and_poison_is_harmless():
    wl = configs.small("mixed_prefill_decode")
    from tests._util import bits
    pool = wl.oracle_pool(poison=True)
    used = wl.used_pages()
    before = {int(p): (pool[int(p)][0].copy(), pool[int(p)][1].copy()) for p in used}
    O, L, _ = run_oracle(wl, pool=pool)
    k_new, v_new = bits(wl.k_new()), bits(wl.v_new())
    changed = 0
    kv, ql = wl.kv_lens(), wl.q_lens()
    expect = {}
    for r in range(wl.R):
        for i in range(ql[r]):
            pos = kv[r] - ql[r] + i
            expect[(int(wl.pages_of(r)[pos // wl.P]), int(pos % wl.P))] = wl.qo_indptr[r] + i
    for p in used:
        for slot in range(wl.P):
            key = (int(p), slot)
            for kvsel, new in ((0, k_new), (1, v_new)):
                now, old = pool[int(p)][kvsel][slot], before[int(p)][kvsel][slot]
                if key in expect:
                    assert np.array_equal(now, new[expect[key]])
                    changed += now.size
                else:
                    assert np.array_equal(now, old)
    assert changed == wl.T * wl.H_kv * wl.D * 2
    O2, L2, _ = run_oracle(wl, poison=False)                # NaN in unused slots changes nothing
    assert np.isfinite(O).all()
    assert np.array_equal(O, O2) and np.array_equal(L, L2)


# golden --------------------------------------------------------------------------------
def test_golden_worked_example():
    vec, cases = {}, []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] == "mask":
            cases.append(([bool(int(tok[1])), bool(int(tok[2]))], [float(x) for x in tok[5:9]], float(tok[10])))
        else:
            vec[tok[0]] = np.array([float(x) for x in tok[1:]], dtype=np.float64)
    assert len(cases) == 3
    for mask, O_exp, L_exp in cases:
        seq = dict(Q=vec["q"][None, None, :], K=np.stack([vec["k0"], vec["k1"]])[:, None, :],
                   V=np.stack([vec["v0"], vec["v1"]])[:, None, :], mask=np.array([mask]))
        args = SmallBatch([{k: (v.astype(np.float64) if k != "mask" else v) for k, v in seq.items()}], 1).paged(8)
        for p in args["pool"]:      # keep fp64 storage so ln 3 is not rounded to fp32
            args["pool"][p] = (args["pool"][p][0].astype(np.float64), args["pool"][p][1].astype(np.float64))
        O, L = oracle_on(args)
        np.testing.assert_allclose(O[0, 0], O_exp, atol=1e-14)
        assert abs(L[0, 0] - L_exp) < 1e-14


# mask_kvpage ---------------------------------------------------------------------------
def test_page_masks_equal_textbook_with_columns_removed_and_page_omission():
    """Persistent page masks (Table 1 `mask_kvpage`): attention with per-page token masks equals the
    scalar textbook computation over (batch mask AND page-mask) columns; a page with every slot hidden
    equals leaving the page out of the list (Section 4.2)."""
    rng = np.random.RandomState(21)
    P, H_q, H_kv, D = 8, 4, 2, 8
    shapes = [(1, 37), (5, 30)]
    m1 = rng.rand(5, 30) < 0.7
    m1[:, 3] = True
    seqs = random_seqs(rng, shapes, H_q, H_kv, D, masks=[None, m1])
    args = SmallBatch(seqs, H_q).paged(P, "random", seed=2)
    pages0 = args["page_indices"][args["page_indptr"][0]:args["page_indptr"][1]]
    pages1 = args["page_indices"][args["page_indptr"][1]:args["page_indptr"][2]]
    page_masks = {int(pages0[1]): rng.rand(P) < 0.5, int(pages0[3]): np.zeros(P, bool),
                  int(pages1[0]): rng.rand(P) < 0.5, int(pages1[2]): np.zeros(P, bool)}
    O, L = orc.forward(**args, page_masks=page_masks)
    t = 0
    for s, (q_len, kv_len), pages in zip(seqs, shapes, (pages0, pages1)):
        allowed = np.array(causal(q_len, kv_len)) if s.get("mask") is None else s["mask"].copy()
        col = np.ones(kv_len, bool)
        for lp, pg in enumerate(pages):
            if int(pg) in page_masks:
                col[lp * P:(lp + 1) * P] = page_masks[int(pg)][: max(0, min(P, kv_len - lp * P))]
        allowed = allowed & col[None, :]
        Or, Lr = textbook_attention(s["Q"], s["K"], s["V"], allowed)
        np.testing.assert_allclose(O[t:t + q_len], Or, atol=1e-12)
        fin = np.isfinite(Lr)
        assert np.array_equal(np.isfinite(L[t:t + q_len]), fin)
        np.testing.assert_allclose(L[t:t + q_len][fin], Lr[fin], atol=1e-12)
        t += q_len
    # hidden page == omitted page, for a decode whose hidden page is a full, earlier one
    seq = random_seqs(rng, [(1, 5 * P)], H_q, H_kv, D)[0]
    a = SmallBatch([seq], H_q).paged(P, "random", seed=3)
    hidden = int(a["page_indices"][2])
    O_h, L_h = orc.forward(**a, page_masks={hidden: np.zeros(P, bool)})
    keep = np.ones(5 * P, bool)
    keep[2 * P:3 * P] = False
    short = dict(Q=seq["Q"], K=seq["K"][keep], V=seq["V"][keep])
    O_o, L_o = oracle_on(SmallBatch([short], H_q).paged(P, "random", seed=4))
    np.testing.assert_allclose(O_h, O_o, atol=1e-14)
    np.testing.assert_allclose(L_h, L_o, atol=1e-14)


# RoPE ----------------------------------------------------------------------------------
def test_rope_pins():
    """Rotary positions inside the path: hand-derived quarter turn, identity at position 0, norm
    preservation, and the defining property - scores depend only on position differences, so
    shifting every position of a request by a constant leaves its attention output unchanged."""
    # D = 2, theta arbitrary: one pair, angle = pos.  (1, 0) at pos = pi/2 (as a float) -> (cos, sin)
    x = np.array([[[1.0, 0.0]]])
    y = orc.rope(x, np.array([1]), 10000.0)
    np.testing.assert_allclose(y[0, 0], [math.cos(1.0), math.sin(1.0)], atol=1e-15)
    # D = 4: second pair turns at theta^(-1/2)
    x = np.array([[[1.0, 2.0, 0.0, 0.0]]])
    y = orc.rope(x, np.array([3]), 100.0)
    np.testing.assert_allclose(y[0, 0], [math.cos(3.0), 2 * math.cos(0.3), math.sin(3.0), 2 * math.sin(0.3)], atol=1e-14)
    rng = np.random.RandomState(31)
    x = rng.randn(5, 3, 16)
    assert np.array_equal(orc.rope(x, np.zeros(5, int), 500000.0), x)                       # position 0: identity
    y = orc.rope(x, rng.randint(0, 100000, 5), 500000.0)
    np.testing.assert_allclose((y[..., :8] ** 2 + y[..., 8:] ** 2), (x[..., :8] ** 2 + x[..., 8:] ** 2), rtol=1e-12)
    # relative-position property through the whole forward (fp64 storage so nothing is rounded)
    P, H_q, H_kv, D, n = 8, 4, 2, 16, 19
    Q, K, V = rng.randn(n, H_q, D), rng.randn(n, H_kv, D), rng.randn(n, H_kv, D)
    outs = []
    for shift in (0, 1000):
        pool = {p: (np.zeros((P, H_kv, D)), np.zeros((P, H_kv, D))) for p in range(3)}
        outs.append(orc.forward(pool, P, H_q, np.array([0, n]), np.array([0, 3]), np.array([2, 0, 1]), np.array([n - 2 * P]),
                                Q, K, V, rope_theta=10000.0, positions=np.arange(n) + shift))
    np.testing.assert_allclose(outs[0][0], outs[1][0], atol=1e-10)
    np.testing.assert_allclose(outs[0][1], outs[1][1], atol=1e-10)
    # and against the textbook computation on explicitly rotated dense arrays
    Qr, Kr = orc.rope(Q, np.arange(n), 10000.0), orc.rope(K, np.arange(n), 10000.0)
    Or, Lr = textbook_attention(Qr, Kr, V, causal(n, n))
    np.testing.assert_allclose(outs[0][0], Or, atol=1e-12)
    np.testing.assert_allclose(outs[0][1], Lr, atol=1e-12)
    # to_storage: bf16 bit patterns round to nearest even
    v = np.array([1.0, 1.00390625, 1.01171875, -2.5])          # 1 + 2^-8 is a tie -> even (1.0); 1 + 3*2^-8 -> 1.015625
    b = orc.to_storage(v, np.zeros(1, np.uint16))
    np.testing.assert_array_equal(orc.widen(b), [1.0, 1.0, 1.015625, -2.5])


def test_default_positions_are_the_last_q_len_context_positions():
    # request 0: 2 pages of 8, last page holds 3 -> kv_len 11, 1 new token -> position 10
    # request 1: 3 pages, last holds 8 -> kv_len 24, 4 new tokens -> positions 20..23
    pos = orc.default_positions(np.array([0, 1, 5]), np.array([0, 2, 5]), np.array([3, 8]), 8)
    assert pos.tolist() == [10, 20, 21, 22, 23]


def test_out_lens_follow_the_papers_listing_and_the_textbook():
    """Section 4.2 listing: `forward([], iemb, [], oemb)` gives ONE output from nine inputs, and the
    same result comes from `forward([], iemb[:-1], kv)` (rows stored, no output) followed by
    `forward(kv, iemb[-1:], oemb)`.  Rows with an output equal scalar-loop textbook attention of that
    row; rows without come back as NaN; the stored rows do not depend on how many outputs were asked for."""
    rng = np.random.RandomState(31)
    P, H_q, H_kv, D = 8, 4, 2, 8
    shapes = [(9, 9), (5, 21), (3, 17), (1, 12)]
    out_lens = [1, 0, 2, 1]
    m = rng.rand(3, 17) < 0.6
    m[:, 0] = True
    seqs = random_seqs(rng, shapes, H_q, H_kv, D, masks=[None, None, m, None])
    args = SmallBatch(seqs, H_q).paged(P, "random", seed=2)
    pool_a = {p: (a.copy(), b.copy()) for p, (a, b) in args["pool"].items()}
    pool_b = {p: (a.copy(), b.copy()) for p, (a, b) in args["pool"].items()}
    O_all, L_all = orc.forward(**dict(args, pool=pool_a))
    O, L = orc.forward(**dict(args, pool=pool_b), out_lens=out_lens)
    for p in pool_a:                                   # every row is stored either way
        assert np.array_equal(pool_a[p][0], pool_b[p][0], equal_nan=True)
        assert np.array_equal(pool_a[p][1], pool_b[p][1], equal_nan=True)
    t = 0
    for s, (q_len, kv_len), ol in zip(seqs, shapes, out_lens):
        first = q_len - ol
        assert np.isnan(O[t:t + first]).all() and np.isnan(L[t:t + first]).all()
        allowed = s["mask"] if "mask" in s else np.array(causal(q_len, kv_len))
        Or, Lr = textbook_attention(s["Q"][first:], s["K"], s["V"], np.asarray(allowed)[first:])
        np.testing.assert_allclose(O[t + first:t + q_len], Or, rtol=0, atol=1e-12)
        np.testing.assert_allclose(L[t + first:t + q_len], Lr, rtol=0, atol=1e-12)
        np.testing.assert_allclose(O[t + first:t + q_len], O_all[t + first:t + q_len], rtol=0, atol=1e-13)
        t += q_len

    # the listing itself: 8 tokens stored with no output, then one token that reads them
    s0 = seqs[0]
    npg = 2
    pool = {p: (np.full((P, H_kv, D), np.nan, np.float32), np.full((P, H_kv, D), np.nan, np.float32)) for p in range(3)}
    pages = np.array([2, 0])
    Oa, La = orc.forward(pool, P, H_q, np.array([0, 8]), np.array([0, 1]), pages[:1], np.array([8]),
                         s0["Q"][:8], s0["K"][:8], s0["V"][:8], out_lens=[0])
    assert np.isnan(Oa).all() and np.isnan(La).all()
    Ob, Lb = orc.forward(pool, P, H_q, np.array([0, 1]), np.array([0, npg]), pages, np.array([1]),
                         s0["Q"][8:], s0["K"][8:], s0["V"][8:])
    np.testing.assert_allclose(Ob[0], O[8], atol=1e-14)
    np.testing.assert_allclose(Lb[0], L[8], atol=1e-14)


def test_next_dist_pins():
    """Top-K truncated next-token distribution (Section 4.2 "Sample API"): closed forms (logits = log of a
    known distribution), K = V returns the whole distribution summing to 1, shift invariance, equal logits
    in ascending token order, permutation equivariance, and a scalar-loop definition on small rows."""
    rng = np.random.RandomState(41)
    # closed form: logits = ln(p) + c  =>  probs = p, ids = argsort of p
    p = rng.dirichlet(np.ones(50))
    for c in (0.0, 7.5, -300.0):
        ids, pr = orc.next_dist((np.log(p) + c)[None, :].astype(np.float64).astype(np.float32), 50)
        assert np.array_equal(ids[0], np.argsort(-p, kind="stable"))
        np.testing.assert_allclose(pr[0], np.sort(p)[::-1], rtol=2e-6 + abs(c) * 2e-7)   # (float32 storage of the logits)
        assert abs(pr.sum() - 1.0) < 1e-12
    # scalar-loop definition, with ties, on small rows
    x = rng.randint(-3, 4, size=(6, 23)).astype(np.float32)
    ids, pr = orc.next_dist(x, 5)
    for r in range(6):
        Z = math.fsum(math.exp(float(v)) for v in x[r])
        want = sorted(range(23), key=lambda t: (-float(x[r, t]), t))[:5]
        assert list(ids[r]) == want
        for k, t in enumerate(want):
            assert abs(pr[r, k] - math.exp(float(x[r, t])) / Z) < 1e-14
        assert all(pr[r, k] >= pr[r, k + 1] for k in range(4))
        for k in range(4):                                                   # equal probabilities: ascending ids
            if x[r, ids[r, k]] == x[r, ids[r, k + 1]]:
                assert ids[r, k] < ids[r, k + 1]
    # permutation equivariance (no ties): permuting the vocabulary permutes the ids
    y = rng.randn(3, 40).astype(np.float32)
    perm = rng.permutation(40)
    ids_a, pr_a = orc.next_dist(y, 7)
    ids_b, pr_b = orc.next_dist(y[:, perm], 7)
    assert np.array_equal(perm[ids_b], ids_a)
    np.testing.assert_allclose(pr_a, pr_b, rtol=1e-13)
    # bf16 storage: the bit patterns are widened exactly
    import torch
    z = torch.from_numpy(y).to(torch.bfloat16)
    ids_c, pr_c = orc.next_dist(z.view(torch.int16).numpy().view(np.uint16), 7)
    ids_d, pr_d = orc.next_dist(z.float().numpy(), 7)
    assert np.array_equal(ids_c, ids_d) and np.array_equal(pr_c, pr_d)


def test_no_store_follows_the_papers_listing_and_the_textbook():
    """Section 4.2 listing: `forward([], iemb, [], oemb)` - nine tokens in, no KvPages at all, one output -
    and `forward(kv, iemb[-1:], oemb)` - eight stored tokens plus one that is attended but not stored - give the
    output of a plain nine-token prefill.  Checked against scalar-loop textbook attention; the pool is untouched."""
    rng = np.random.RandomState(51)
    P, H_q, H_kv, D, n = 4, 4, 2, 8, 9
    Q = rng.randn(n, H_q, D).astype(np.float32)
    K = rng.randn(n, H_kv, D).astype(np.float32)
    V = rng.randn(n, H_kv, D).astype(np.float32)
    Or, Lr = textbook_attention(Q, K, V, causal(n, n))

    def fresh_pool():
        return {p: (np.full((P, H_kv, D), np.nan, np.float32), np.full((P, H_kv, D), np.nan, np.float32)) for p in range(4)}

    # line 3 of the listing: no pages in, none out, one output
    pool = fresh_pool()
    O, L = orc.forward(pool, P, H_q, np.array([0, n]), np.array([0, 0]), np.array([], np.int64), np.array([1]),
                       Q, K, V, out_lens=[1], no_store=[1])
    np.testing.assert_allclose(O[-1], Or[-1], atol=1e-12)
    np.testing.assert_allclose(L[-1], Lr[-1], atol=1e-12)
    assert np.isnan(O[:-1]).all() and all(np.isnan(a).all() and np.isnan(b).all() for a, b in pool.values())
    # all nine outputs without storing anything
    O, L = orc.forward(pool, P, H_q, np.array([0, n]), np.array([0, 0]), np.array([], np.int64), np.array([1]),
                       Q, K, V, no_store=[1])
    np.testing.assert_allclose(O, Or, atol=1e-12)
    np.testing.assert_allclose(L, Lr, atol=1e-12)
    # lines 6-7: eight tokens stored (pages 3 and 1), then one token attended over them without being stored
    pages = np.array([3, 1])
    orc.forward(pool, P, H_q, np.array([0, 8]), np.array([0, 2]), pages, np.array([4]), Q[:8], K[:8], V[:8], out_lens=[0])
    before = {p: (a.copy(), b.copy()) for p, (a, b) in pool.items()}
    O, L = orc.forward(pool, P, H_q, np.array([0, 1]), np.array([0, 2]), pages, np.array([4]), Q[8:], K[8:], V[8:],
                       no_store=[1])
    np.testing.assert_allclose(O[0], Or[-1], atol=1e-12)
    np.testing.assert_allclose(L[0], Lr[-1], atol=1e-12)
    for p in pool:
        assert np.array_equal(pool[p][0], before[p][0], equal_nan=True) and np.array_equal(pool[p][1], before[p][1], equal_nan=True)
    # a partly filled last page, an explicit mask over existing + new positions, mixed with a storing request
    m = rng.rand(3, 6 + 3) < 0.6
    m[:, 0] = True
    pool = fresh_pool()
    orc.forward(pool, P, H_q, np.array([0, 6]), np.array([0, 2]), np.array([2, 0]), np.array([2]), Q[:6], K[:6], V[:6], out_lens=[0])
    O, L = orc.forward(pool, P, H_q, np.array([0, 3, 4]), np.array([0, 2, 3]), np.array([2, 0, 1]), np.array([2, 1]),
                       Q[5:9], K[5:9], V[5:9], masks=[m, None], no_store=[1, 0])
    Kc = np.concatenate([K[:6], K[5:8]])
    Vc = np.concatenate([V[:6], V[5:8]])
    Om, Lm = textbook_attention(Q[5:8], Kc, Vc, m)
    np.testing.assert_allclose(O[:3], Om, atol=1e-12)
    np.testing.assert_allclose(L[:3], Lm, atol=1e-12)
    Os, Ls = textbook_attention(Q[8:9], K[8:9], V[8:9], [[True]])
    np.testing.assert_allclose(O[3], Os[0], atol=1e-12)
    assert np.array_equal(pool[1][0][0], K[8]) and np.isnan(pool[1][0][1:]).all() and np.isnan(pool[3][0]).all()
