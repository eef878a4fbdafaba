"""The five synthetic workloads (and scaled-down versions of them for fast tests).

Each builder returns a `Workload`: the CSR arrays of one coalesced `forward` batch
(qo_indptr, page_indptr, page_indices, last_page_len), optional per-request boolean masks,
and the keys from which every Q/K/V value is regenerated on demand (workloads.synth).
No attention arithmetic lives here.

Shapes follow the serving scenarios of the paper's evaluation: batched text-completion
decode, horizontally batched prefill chunks plus decodes, forked generations that share a
prefix through exported KvPages and verify a speculative token tree, and application KV
policies (attention sink + window + dropped pages) followed by `copy_kvpage`.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

from . import synth

SEED0 = 0x50494500


class LazyPool(dict):
    """page id -> (K, V) numpy arrays [P, H_kv, D] in storage bits, generated on first use."""

    def __init__(self, wl, poison=False):
        super().__init__()
        self._wl, self._poison = wl, poison

    def __missing__(self, page):
        K, V = self._wl.context_pages(np.array([page]), "cpu", poison=self._poison)
        val = (synth.to_numpy_bits(K[0]).copy(), synth.to_numpy_bits(V[0]).copy())
        self[page] = val
        return val

    def prefetch(self, pages, chunk=1024):
        """Generate many pages at once (the same bits as page-by-page generation)."""
        todo = np.array(sorted({int(p) for p in pages} - set(self.keys())), dtype=np.int64)
        for i in range(0, len(todo), chunk):
            ids = todo[i:i + chunk]
            K, V = self._wl.context_pages(ids, "cpu", poison=self._poison)
            Kb, Vb = synth.to_numpy_bits(K), synth.to_numpy_bits(V)
            for n, p in enumerate(ids):
                self[int(p)] = (Kb[n].copy(), Vb[n].copy())


@dataclass
class Workload:
    name: str
    seed: int
    H_q: int
    H_kv: int
    D: int
    P: int
    dtype: str                      # "bf16" | "f32"
    num_pages: int                  # size of the KvPage pool
    qo_indptr: np.ndarray
    page_indptr: np.ndarray
    page_indices: np.ndarray
    last_page_len: np.ndarray
    masks: list | None              # per request: None (inferred causal) or bool [q_len, kv_len]
    page_owner: np.ndarray          # [num_pages] content key (-1: unused page)
    page_logical: np.ndarray        # [num_pages] logical page number within the owner
    page_fill: np.ndarray           # [num_pages] slots holding context before this call
    copies: dict | None = None      # src, dst, src_off, dst_off, ntok (after the forward)
    meta: dict = field(default_factory=dict)

    # ---- sizes
    @property
    def R(self):
        return len(self.qo_indptr) - 1

    @property
    def T(self):
        return int(self.qo_indptr[-1])

    @property
    def esize(self):
        return 2 if self.dtype == "bf16" else 4

    def q_lens(self):
        return np.diff(self.qo_indptr).astype(np.int64)

    def kv_lens(self):
        return (np.diff(self.page_indptr).astype(np.int64) - 1) * self.P + self.last_page_len

    def pages_of(self, r):
        return self.page_indices[self.page_indptr[r]:self.page_indptr[r + 1]]

    def used_pages(self):
        return np.unique(self.page_indices)

    # ---- values
    def q(self, device="cpu"):
        return synth.normal_tensor(self.seed, 1, (self.T, self.H_q, self.D), self.dtype, device)

    def k_new(self, device="cpu"):
        return synth.normal_tensor(self.seed, 2, (self.T, self.H_kv, self.D), self.dtype, device)

    def v_new(self, device="cpu"):
        return synth.normal_tensor(self.seed, 3, (self.T, self.H_kv, self.D), self.dtype, device)

    def context_pages(self, ids, device="cpu", poison=False):
        """Pre-call contents of physical pages `ids`: K, V [n, P, H_kv, D] (canonical)."""
        ids_t = torch.as_tensor(np.asarray(ids), dtype=torch.int64, device=device)
        owner = torch.as_tensor(self.page_owner, device=device)[ids_t]
        logical = torch.as_tensor(self.page_logical, device=device)[ids_t]
        slot = torch.arange(self.P, dtype=torch.int64, device=device)
        pos = (logical[:, None] * self.P + slot[None, :]).reshape(-1)
        own = owner[:, None].expand(-1, self.P).reshape(-1)
        out = []
        for which in (0, 1):
            x = synth.kv_rows(self.seed, which, own, pos, self.H_kv, self.D, self.dtype)
            x = x.reshape(len(ids_t), self.P, self.H_kv, self.D)
            if poison:  # slots that hold no context yet get NaN bit patterns
                fill = torch.as_tensor(self.page_fill, device=device)[ids_t]
                bad = slot[None, :] >= fill[:, None]
                x = torch.where(bad[:, :, None, None], torch.full_like(x, float("nan")), x)
            out.append(x)
        return out[0], out[1]

    def oracle_pool(self, poison=False):
        return LazyPool(self, poison)

    def mask_bytes(self):
        """(mask_indptr int64 [R+1], mask uint8 [sum q_len*kv_len]) for the C ABI, or (None, None)."""
        if self.masks is None or all(m is None for m in self.masks):
            return None, None
        ptr = np.zeros(self.R + 1, dtype=np.int64)
        for r, m in enumerate(self.masks):
            ptr[r + 1] = ptr[r] + (0 if m is None else m.size)
        buf = np.empty(int(ptr[-1]), dtype=np.uint8)
        for r, m in enumerate(self.masks):
            if m is not None:
                buf[ptr[r]:ptr[r + 1]] = np.ascontiguousarray(m, dtype=np.uint8).reshape(-1)
        return ptr, buf

    # ---- algorithmic work (one K row + one V row per distinct (request, kept token))
    def kept_tokens(self):
        """Per request: number of context positions at least one query row attends to."""
        kv = self.kv_lens()
        out = np.empty(self.R, dtype=np.int64)
        for r in range(self.R):
            m = None if self.masks is None else self.masks[r]
            out[r] = kv[r] if m is None else int(m.any(axis=0).sum())
        return out

    def algorithmic_bytes(self):
        b_tok = 2 * self.H_kv * self.D * self.esize
        kv = int(self.kept_tokens().sum()) * b_tok
        qo = self.T * self.H_q * self.D * self.esize * 2 + self.T * self.H_q * 4
        new = self.T * b_tok * 2                      # new rows read once and written once
        mask = 0
        if self.masks is not None:
            mask = sum(0 if m is None else (m.size + 7) // 8 for m in self.masks)
        return {"kv": kv, "qo": qo, "append": new, "mask": mask, "total": kv + qo + new + mask}

    def useful_flops(self):
        """4*D flops per (query row, q head, allowed position)."""
        kv, ql = self.kv_lens(), self.q_lens()
        n = 0
        for r in range(self.R):
            m = None if self.masks is None else self.masks[r]
            if m is None:  # causal trapezoid
                n += int(ql[r]) * int(kv[r]) - int(ql[r]) * (int(ql[r]) - 1) // 2
            else:
                n += int(m.sum())
        return 4 * self.D * self.H_q * n


def _csr(lengths):
    p = np.zeros(len(lengths) + 1, dtype=np.int32)
    p[1:] = np.cumsum(lengths)
    return p


def _assemble(name, seed, H_q, H_kv, D, P, dtype, num_pages, q_lens, kv_lens, masks,
              placement=0, perm_stream=10, meta=None, perm_seed=None, page_offset=None):
    """Private pages for every request, taken in order from a seeded shuffle of the pool:
    the `placement`-th run of the batch's page count, or the run that starts at `page_offset`
    of the shuffle seeded by `perm_seed` (several batches with different seeds in one pool)."""
    q_lens = np.asarray(q_lens, dtype=np.int64)
    kv_lens = np.asarray(kv_lens, dtype=np.int64)
    npages = (kv_lens + P - 1) // P
    total = int(npages.sum())
    first = placement * total if page_offset is None else int(page_offset)
    assert first + total <= num_pages, "pool too small for this placement"
    perm = synth.permutation(seed if perm_seed is None else perm_seed, perm_stream, num_pages)
    ids = perm[first:first + total]
    page_indptr = _csr(npages)
    owner = np.full(num_pages, -1, dtype=np.int64)
    logical = np.zeros(num_pages, dtype=np.int64)
    fill = np.zeros(num_pages, dtype=np.int64)
    for r in range(len(q_lens)):
        pr = ids[page_indptr[r]:page_indptr[r + 1]]
        owner[pr] = r
        logical[pr] = np.arange(len(pr))
        pre = kv_lens[r] - q_lens[r]
        fill[pr] = np.clip(pre - np.arange(len(pr)) * P, 0, P)
    return Workload(
        name=name, seed=seed, H_q=H_q, H_kv=H_kv, D=D, P=P, dtype=dtype, num_pages=num_pages,
        qo_indptr=_csr(q_lens), page_indptr=page_indptr, page_indices=ids.astype(np.int32),
        last_page_len=(kv_lens - (npages - 1) * P).astype(np.int32), masks=masks,
        page_owner=owner, page_logical=logical, page_fill=fill, meta=meta or {})


# ------------------------------------------------------------------------------- config 1
def tiny_fp32(seed=SEED0 + 1, column_wise=False, P=16, dtype="f32", H_q=4, H_kv=2, D=64):
    """4 requests, GQA 4/2, D 64: two decodes and two 8-token prefill chunks; request 3 has a
    seeded random 30% of its earlier tokens masked off (diagonal always kept)."""
    q_lens = [1, 1, 8, 8]
    kv_lens = [17, 40, 64, 100]
    masks = [None, None, None, None]
    ql, kl = q_lens[3], kv_lens[3]
    pos = kl - ql + np.arange(ql)
    causal = np.arange(kl)[None, :] <= pos[:, None]
    if column_wise:
        drop = np.broadcast_to(synth.uniform_unit(seed, 20, (1, kl)) < 0.3, (ql, kl))
    else:
        drop = synth.uniform_unit(seed, 20, (ql, kl)) < 0.3
    earlier = np.arange(kl)[None, :] < pos[:, None]
    masks[3] = causal & ~(drop & earlier)
    return _assemble("tiny_fp32", seed, H_q, H_kv, D, P, dtype, 32, q_lens, kv_lens, masks)


# ------------------------------------------------------------------------------- config 2
def batched_decode(seed=SEED0 + 2, R=64, lo=512, hi=4096, num_pages=65536, placement=0,
                   H_q=32, H_kv=8, D=64, P=16, dtype="bf16", perm_seed=None, page_offset=None):
    """Single-token decodes over scattered pages, causal, one appended row per request."""
    kv = synth.uniform_ints(seed, 11, R, lo, hi)
    return _assemble("batched_decode", seed, H_q, H_kv, D, P, dtype, num_pages,
                     np.ones(R, dtype=np.int64), kv, None, placement=placement,
                     perm_seed=perm_seed, page_offset=page_offset)


# ------------------------------------------------------------------------------- config 3
def mixed_prefill_decode(seed=SEED0 + 3, n_prefill=8, chunk=512, prefix_hi=2048, n_decode=120,
                         dec_lo=1024, dec_hi=8192, num_pages=65536, placement=0,
                         H_q=32, H_kv=8, D=128, P=16, dtype="bf16", only=None):
    """Prefill chunks over existing prefixes plus decodes in one batch (prefills first).
    `only` = "prefill" | "decode" keeps one class (for the per-class roofline runs)."""
    prefix = synth.uniform_ints(seed, 11, n_prefill, 0, prefix_hi)
    dec = synth.uniform_ints(seed, 12, n_decode, dec_lo, dec_hi)
    q_lens = np.concatenate([np.full(n_prefill, chunk), np.ones(n_decode, dtype=np.int64)])
    kv_lens = np.concatenate([prefix + chunk, dec])
    if only == "prefill":
        q_lens, kv_lens = q_lens[:n_prefill], kv_lens[:n_prefill]
    elif only == "decode":
        q_lens, kv_lens = q_lens[n_prefill:], kv_lens[n_prefill:]
    return _assemble("mixed_prefill_decode" + ("" if only is None else "_" + only), seed, H_q,
                     H_kv, D, P, dtype, num_pages, q_lens, kv_lens, None, placement=placement)


# ------------------------------------------------------------------------------- config 4
def tree_parents(seed, stream, n_nodes, lead=()):
    """Node 0 is the root (parent -1); node n>=1 draws its parent uniformly from 0..n-1."""
    par = np.full(n_nodes, -1, dtype=np.int64)
    idx = torch.arange(n_nodes, dtype=torch.int64)
    h = synth.hash_coords(seed, stream, *lead, idx).numpy()
    for n in range(1, n_nodes):
        par[n] = int(h[n] % n)
    return par


def ancestor_matrix(par):
    """anc[n, a] = True iff a == n or a is an ancestor of n."""
    n_nodes = len(par)
    anc = np.zeros((n_nodes, n_nodes), dtype=bool)
    for n in range(n_nodes):
        a = n
        while a >= 0:
            anc[n, a] = True
            a = par[a]
    return anc


def shared_prefix_tree(seed=SEED0 + 4, groups=16, branches=16, prefix=4096, suffix=256,
                       tree=64, num_pages=16384, H_q=32, H_kv=8, D=128, P=16, dtype="bf16"):
    """Forked branches share each group's prefix pages; every branch verifies a token tree
    whose nodes see prefix + suffix + their own ancestors (bit mask given explicitly)."""
    assert prefix % P == 0 and suffix % P == 0 and tree % P == 0
    R = groups * branches
    n_pre, n_suf, n_tree = prefix // P, suffix // P, tree // P
    perm = synth.permutation(seed, 10, num_pages)
    owner = np.full(num_pages, -1, dtype=np.int64)
    logical = np.zeros(num_pages, dtype=np.int64)
    fill = np.zeros(num_pages, dtype=np.int64)
    cur = 0
    pre_ids = []
    for g in range(groups):
        ids = perm[cur:cur + n_pre]
        cur += n_pre
        owner[ids], logical[ids], fill[ids] = g, np.arange(n_pre), P
        pre_ids.append(ids)
    lists, masks, parents = [], [], []
    kv_len = prefix + suffix + tree
    for g in range(groups):
        for b in range(branches):
            rid = g * branches + b
            ids = perm[cur:cur + n_suf + n_tree]
            cur += n_suf + n_tree
            owner[ids] = 1000 + rid
            logical[ids] = n_pre + np.arange(n_suf + n_tree)
            fill[ids[:n_suf]] = P
            lists.append(np.concatenate([pre_ids[g], ids]))
            par = tree_parents(seed, 21, tree, lead=(rid,))
            m = np.ones((tree, kv_len), dtype=bool)
            m[:, prefix + suffix:] = ancestor_matrix(par)
            masks.append(m)
            parents.append(par)
    assert cur <= num_pages
    npages = np.full(R, n_pre + n_suf + n_tree, dtype=np.int64)
    return Workload(
        name="shared_prefix_tree", seed=seed, H_q=H_q, H_kv=H_kv, D=D, P=P, dtype=dtype,
        num_pages=num_pages, qo_indptr=_csr(np.full(R, tree)), page_indptr=_csr(npages),
        page_indices=np.concatenate(lists).astype(np.int32),
        last_page_len=np.full(R, P, dtype=np.int32), masks=masks, page_owner=owner,
        page_logical=logical, page_fill=fill,
        meta={"parents": parents, "groups": groups, "branches": branches, "prefix": prefix,
              "suffix": suffix, "tree": tree})


# ------------------------------------------------------------------------------- config 5
def policy_mask(seed, stream, rid, L, P, sink=4, window=2048, keep_frac=0.2):
    """Application KV policy over a context of L tokens: keep the first `sink` tokens, the
    last `window` tokens and a seeded `keep_frac` of the middle pages; the rest is masked."""
    keep = np.zeros(L, dtype=bool)
    keep[:sink] = True
    w0 = max(L - window, 0)
    keep[w0:] = True
    first_mid, end_mid = 1, w0 // P          # middle pages: 1 .. floor((L - window)/P) - 1
    M = max(end_mid - first_mid, 0)
    if M > 0:
        n_keep = int(round(keep_frac * M))
        idx = torch.arange(M, dtype=torch.int64)
        h = synth.hash_coords(seed, stream, rid, idx)
        order = torch.argsort(h * M + idx).numpy()
        for p in order[:n_keep] + first_mid:
            keep[p * P:(p + 1) * P] = True
    return keep


def long_context_policy(seed=SEED0 + 5, R=256, lo=16384, hi=32768, sink=4, window=2048,
                        keep_frac=0.2, num_pages=None, H_q=32, H_kv=8, D=128, P=16,
                        dtype="bf16"):
    """Long-context decodes under sink + window + 20%-of-middle-pages policies, one appended
    token each, then a `copy_kvpage` of every request's last page to a fresh page."""
    kv = synth.uniform_ints(seed, 11, R, lo, hi)
    total = int(((kv + P - 1) // P).sum())
    if num_pages is None:
        num_pages = total + R + 1024
    masks = [policy_mask(seed, 22, r, int(kv[r]), P, sink, window, keep_frac)[None, :]
             for r in range(R)]
    wl = _assemble("long_context_policy", seed, H_q, H_kv, D, P, dtype, num_pages,
                   np.ones(R, dtype=np.int64), kv, masks)
    perm = synth.permutation(seed, 10, num_pages)
    dst = perm[total:total + R]
    src = np.array([wl.pages_of(r)[-1] for r in range(R)], dtype=np.int64)
    wl.copies = {"src": src.astype(np.int32), "dst": dst.astype(np.int32),
                 "src_off": np.zeros(R, dtype=np.int32), "dst_off": np.zeros(R, dtype=np.int32),
                 "ntok": wl.last_page_len.astype(np.int32).copy()}
    wl.page_owner[dst] = 100000 + np.arange(R)
    wl.name = "long_context_policy"
    wl.meta = {"sink": sink, "window": window, "keep_frac": keep_frac, "pages_in_lists": total}
    return wl


def decode_loop(wl, n_steps, spare_pages):
    """The batches of a decode loop that starts from the decode workload `wl` (every request one
    query token): step s has every request s tokens longer than in `wl`, a request that crosses a
    page boundary takes its next page from `spare_pages`, and application KV policies (the
    long-context workload) are re-evaluated at the new length.  Returns one dict per step with
    the CSR arrays (int32), the mask arrays of Workload.mask_bytes() and, for workloads with
    page copies, the copy arrays of that step."""
    assert (wl.q_lens() == 1).all(), "a decode loop needs single-token requests"
    P, R = wl.P, wl.R
    spare = [int(p) for p in spare_pages]
    lists = [[int(p) for p in wl.pages_of(r)] for r in range(R)]
    kv0 = wl.kv_lens()
    policy = wl.masks is not None
    if policy:
        assert "window" in wl.meta, "only the sink / window / kept-pages policy can be re-evaluated"
    steps = []
    for s in range(n_steps):
        kv = kv0 + s
        for r in range(R):
            need = (int(kv[r]) + P - 1) // P
            while len(lists[r]) < need:
                lists[r].append(spare.pop())
        npages = np.array([len(x) for x in lists], dtype=np.int64)
        b = {"qo_indptr": wl.qo_indptr.astype(np.int32), "page_indptr": _csr(npages),
             "page_indices": np.fromiter((p for x in lists for p in x), dtype=np.int32, count=int(npages.sum())),
             "last_page_len": (kv - (npages - 1) * P).astype(np.int32), "mask_indptr": None, "mask": None,
             "copies": None}
        if policy:
            rows = [policy_mask(wl.seed, 22, r, int(kv[r]), P, wl.meta["sink"], wl.meta["window"],
                                wl.meta["keep_frac"]) for r in range(R)]
            ptr = np.zeros(R + 1, dtype=np.int64)
            ptr[1:] = np.cumsum([len(x) for x in rows])
            b["mask_indptr"], b["mask"] = ptr, np.concatenate(rows).astype(np.uint8)
        if wl.copies is not None:
            b["copies"] = dict(wl.copies, src=np.array([x[-1] for x in lists], dtype=np.int32),
                               ntok=b["last_page_len"].copy())
        steps.append(b)
    return steps


# ------------------------------------------------------------------------------- shared-prefix decode
def shared_prefix_decode(seed=SEED0 + 6, groups=16, branches=32, prefix=4096, priv_lo=16, priv_hi=256,
                         num_pages=16384, H_q=32, H_kv=8, D=128, P=16, dtype="bf16"):
    """Parallel generation from shared prompts (fork / join, beams, samples of one prompt): every
    group's branches share the prompt's pages and each decodes one token after a private
    continuation of its own, seeded log-uniform length in [priv_lo, priv_hi].  Not one of the five
    baseline configurations: the workload of the shared-prefix cascade."""
    assert prefix % P == 0
    R = groups * branches
    n_pre = prefix // P
    u = synth.uniform_unit(seed, 11, (R,))
    priv = np.floor(np.exp(np.log(priv_lo) + u * (np.log(priv_hi + 1) - np.log(priv_lo)))).astype(np.int64)
    priv = np.clip(priv, priv_lo, priv_hi)
    perm = synth.permutation(seed, 10, num_pages)
    owner = np.full(num_pages, -1, dtype=np.int64)
    logical = np.zeros(num_pages, dtype=np.int64)
    fill = np.zeros(num_pages, dtype=np.int64)
    cur = 0
    pre_ids = []
    for g in range(groups):
        ids = perm[cur:cur + n_pre]
        cur += n_pre
        owner[ids], logical[ids], fill[ids] = g, np.arange(n_pre), P
        pre_ids.append(ids)
    lists, npages, last = [], [], []
    for g in range(groups):
        for b in range(branches):
            rid = g * branches + b
            n_priv = int((priv[rid] + 1 + P - 1) // P)     # private context + the new token
            assert cur + n_priv <= num_pages, "pool too small"
            ids = perm[cur:cur + n_priv]
            cur += n_priv
            owner[ids] = 1000 + rid
            logical[ids] = n_pre + np.arange(n_priv)
            fill[ids] = np.clip(priv[rid] - np.arange(n_priv) * P, 0, P)
            lists.append(np.concatenate([pre_ids[g], ids]))
            npages.append(n_pre + n_priv)
            last.append(priv[rid] + 1 - (n_priv - 1) * P)
    assert cur <= num_pages, "pool too small"
    return Workload(
        name="shared_prefix_decode", seed=seed, H_q=H_q, H_kv=H_kv, D=D, P=P, dtype=dtype,
        num_pages=num_pages, qo_indptr=_csr(np.ones(R, dtype=np.int64)), page_indptr=_csr(np.array(npages)),
        page_indices=np.concatenate(lists).astype(np.int32), last_page_len=np.array(last, dtype=np.int32),
        masks=None, page_owner=owner, page_logical=logical, page_fill=fill,
        meta={"groups": groups, "branches": branches, "prefix": prefix})


FULL = {
    "tiny_fp32": tiny_fp32,
    "batched_decode": batched_decode,
    "mixed_prefill_decode": mixed_prefill_decode,
    "shared_prefix_tree": shared_prefix_tree,
    "long_context_policy": long_context_policy,
}
# further workloads (not baseline configurations)
EXTRA = {"shared_prefix_decode": shared_prefix_decode}


def small(name, **kw):
    """Scaled-down version of a workload that the oracle finishes in seconds but that still
    spans several tiles, split-KV chunks and ragged tails."""
    if name == "tiny_fp32":
        return tiny_fp32(**kw)
    if name == "batched_decode":
        return batched_decode(R=12, lo=40, hi=700, num_pages=1024, **kw)
    if name == "mixed_prefill_decode":
        return mixed_prefill_decode(n_prefill=3, chunk=80, prefix_hi=300, n_decode=9, dec_lo=60,
                                    dec_hi=900, num_pages=1024, **kw)
    if name == "shared_prefix_tree":
        return shared_prefix_tree(groups=2, branches=3, prefix=256, suffix=32, tree=32,
                                  num_pages=256, **kw)
    if name == "long_context_policy":
        return long_context_policy(R=6, lo=1500, hi=4000, window=256, **kw)
    if name == "shared_prefix_decode":
        return shared_prefix_decode(groups=3, branches=5, prefix=320, priv_lo=3, priv_hi=70, num_pages=256, **kw)
    raise KeyError(name)
