"""fp64 CPU oracle for the attention part of the batched `forward` handler.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the path must
compute; it shares no code with the CUDA library and is never on the product path.  Only
the tests, the smoke check and the benchmark's CPU-baseline leg may import it.

What it states (paper: Table 1 `forward`, `copy_kvpage`; Section 4.1 "Resources" for
KvPages; Section 4.2 "Forward API" for masks, positions and the append-then-read listings):

  1. append   - every new token's K and V rows are stored, bit for bit, in the request's
                output KvPages, at the last q_len logical positions of its page list;
  2. gather   - the request's context is read back page by page through its page list
                (arbitrary, possibly shared physical page ids);
  3. attend   - O = softmax(Q K^T / sqrt(D) + mask) V row by row, LSE = ln sum exp(score),
                with an explicit boolean mask (true = attend) or, when none is given, the
                causal mask inferred from positions; grouped-query heads (kv = q // G);
  4. copy     - token-range copy of K and V rows between pages, bit for bit.
  5. page masks (`mask_kvpage`) - persistent per-page token masks ANDed into the allowed set.
  6. next_dist - the sample stage's `get_next_dist` from the logits on: the next-token
                distribution truncated to its K most probable tokens (Section 4.2 "Sample API").

All floating point is fp64 on exactly widened inputs.  There is no tiling, no online
softmax and no reordering: a reader can check each function against the definition by eye.

Pins (tests/test_oracle_pins.py): dense contiguous causal attention written as scalar
loops; brute-force enumeration of every mask on tiny inputs; closed forms (zero query,
constant V, one-hot rows); invariance to physical page permutation and to page size;
the paper's split-forward and prefill==decode-loop equivalences; page omission == masking;
shared pages == private copies; tree mask == causal path; GQA == repeated MHA; the
LSE-merge identity; a hand-derived worked example under tests/golden/.

Storage convention: a pool is a mapping  page id -> (K, V)  with K, V numpy arrays of
shape [P, H_kv, D] in the storage type: float32, or uint16 holding bf16 bit patterns.
"""
from __future__ import annotations

import math

import numpy as np


# --------------------------------------------------------------------------- element types
def widen(x: np.ndarray) -> np.ndarray:
    """Exact conversion of stored elements (fp32, fp64, or uint16 bf16 bits) to fp64."""
    x = np.asarray(x)
    if x.dtype == np.uint16:  # bf16 bit pattern: the upper half of an fp32
        return (x.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    if x.dtype in (np.float32, np.float64):
        return x.astype(np.float64)
    raise TypeError(f"unsupported element type {x.dtype}")


def kv_len_of(num_pages_r: int, last_page_len_r: int, P: int) -> int:
    """Context length after the append: full pages plus the filled part of the last one."""
    return (num_pages_r - 1) * P + last_page_len_r


# --------------------------------------------------------------------------- positions (RoPE)
def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary position embedding in the rotate-half form used by the Llama family: for i < D/2,
    with angle a = pos * theta**(-2i/D),
        y[i]       = x[i] cos a - x[i + D/2] sin a
        y[i + D/2] = x[i + D/2] cos a + x[i] sin a.
    x [T, H, D] fp64, pos [T] integers.  (`forward` "operates based on explicit sequence positions",
    Section 4.2; the paper gives no formula, this is the reading built here.)"""
    T, H, D = x.shape
    half = D // 2
    inv_freq = theta ** (-2.0 * np.arange(half, dtype=np.float64) / D)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * inv_freq[None, :]          # [T, D/2]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    y = np.empty_like(x)
    y[..., :half] = x[..., :half] * c - x[..., half:] * s
    y[..., half:] = x[..., half:] * c + x[..., :half] * s
    return y


def to_storage(x64: np.ndarray, like: np.ndarray) -> np.ndarray:
    """Round fp64 values to the storage type of `like` (fp32, or bf16 bit patterns, both round to
    nearest even; bf16 goes through fp32)."""
    if like.dtype == np.float64:   # fp64 storage (pins only): nothing to round
        return x64
    f32 = x64.astype(np.float32)
    if like.dtype == np.uint16:
        u = f32.view(np.uint32)
        return ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)
    return f32.astype(like.dtype)


def default_positions(qo_indptr, page_indptr, last_page_len, P) -> np.ndarray:
    """Position of every new token when none is given: the last q_len positions of its context."""
    R = len(qo_indptr) - 1
    pos = np.zeros(int(qo_indptr[R]), dtype=np.int64)
    for r in range(R):
        q_len = int(qo_indptr[r + 1] - qo_indptr[r])
        kv_len = kv_len_of(int(page_indptr[r + 1] - page_indptr[r]), int(last_page_len[r]), P)
        pos[qo_indptr[r]:qo_indptr[r + 1]] = kv_len - q_len + np.arange(q_len)
    return pos


# --------------------------------------------------------------------------- step 1: append
def append_kv(pool, P, qo_indptr, page_indptr, page_indices, last_page_len, k_new, v_new, skip=None):
    """Store the new K/V rows of every request in its pages (Table 1 `forward`, output
    KvPages; Section 4.2 listings: the new tokens occupy the last q_len positions).

    k_new, v_new: [T, H_kv, D] in the storage type.  The pool is updated in place; element
    bits are copied unchanged.  Requests with skip[r] set have no output KvPages: nothing is stored.
    """
    R = len(qo_indptr) - 1
    for r in range(R):
        if skip is not None and skip[r]:
            continue
        q_len = int(qo_indptr[r + 1] - qo_indptr[r])
        pages = page_indices[page_indptr[r]:page_indptr[r + 1]]
        kv_len = kv_len_of(len(pages), int(last_page_len[r]), P)
        for i in range(q_len):
            pos = kv_len - q_len + i
            page = int(pages[pos // P])
            slot = pos % P
            K, V = pool[page]
            K[slot] = k_new[qo_indptr[r] + i]
            V[slot] = v_new[qo_indptr[r] + i]
            pool[page] = (K, V)


# --------------------------------------------------------------------------- step 2: gather
def gather_kv(pool, P, pages, kv_len, needed=None):
    """Read a request's context page by page: K_r[j] = pool[pages[j // P]][j % P].

    `needed` (bool [kv_len]) marks positions some query row may attend to; pages holding no
    such position are not read (their rows stay zero and are never used, because the sums
    of step 3 run over allowed positions only).
    """
    K = V = None
    for p, page in enumerate(pages):
        lo, hi = p * P, min((p + 1) * P, kv_len)
        if lo >= kv_len:
            break
        if needed is not None and not needed[lo:hi].any():
            continue
        Kp, Vp = pool[int(page)]
        if K is None:
            K = np.zeros((kv_len,) + Kp.shape[1:], dtype=np.float64)
            V = np.zeros_like(K)
        K[lo:hi] = widen(Kp[: hi - lo])
        V[lo:hi] = widen(Vp[: hi - lo])
    return K, V


# --------------------------------------------------------------------------- step 3: attend
def allowed_matrix(q_len: int, kv_len: int, mask) -> np.ndarray:
    """The set of positions each query row may attend to, as bool [q_len, kv_len].

    Explicit mask: used as given (true = attend); it is the complete specification and is
    not combined with causality.  No mask: inferred from positions - query token i sits at
    position kv_len - q_len + i and sees every position up to and including its own
    (Section 4.2 "Forward API").
    """
    if mask is not None:
        m = np.asarray(mask).astype(bool)
        if m.shape != (q_len, kv_len):
            raise ValueError(f"mask shape {m.shape} != {(q_len, kv_len)}")
        return m
    j = np.arange(kv_len)[None, :]
    i = np.arange(q_len)[:, None]
    return j <= (kv_len - q_len + i)


def attend(q_r: np.ndarray, K: np.ndarray, V: np.ndarray, allowed: np.ndarray):
    """softmax(Q K^T / sqrt(D) + mask) V for one request, all heads.

    q_r [q_len, H_q, D], K/V [kv_len, H_kv, D] in fp64; allowed bool [q_len, kv_len].
    Returns O [q_len, H_q, D] and LSE [q_len, H_q] (natural log of the sum of exponentials
    of the scaled scores over the allowed set).  A row with an empty allowed set gives
    O = 0 and LSE = -inf.
    """
    q_len, H_q, D = q_r.shape
    O = np.zeros((q_len, H_q, D), dtype=np.float64)
    LSE = np.full((q_len, H_q), -np.inf, dtype=np.float64)
    if K is None:
        return O, LSE
    G = H_q // K.shape[1]
    for h in range(H_q):
        g = h // G
        s = (q_r[:, h, :] @ K[:, g, :].T) / math.sqrt(D)          # [q_len, kv_len]
        s = np.where(allowed, s, -np.inf)
        m = s.max(axis=1)                                          # -inf for an empty row
        live = np.isfinite(m)
        e = np.exp(s - np.where(live, m, 0.0)[:, None])            # masked entries -> 0
        Z = e.sum(axis=1)
        num = e @ V[:, g, :]
        O[live, h, :] = num[live] / Z[live, None]
        LSE[live, h] = m[live] + np.log(Z[live])
    return O, LSE


def apply_page_masks(allowed: np.ndarray, pages, P: int, page_masks) -> np.ndarray:
    """Persistent per-page token masks (Table 1 `mask_kvpage`): position j of a request stays
    attendable only if slot j % P of its page pages[j // P] is visible.  page_masks maps a page id
    to a bool [P] array (true = visible); pages without an entry are fully visible."""
    if not page_masks:
        return allowed
    out = allowed.copy()
    kv_len = allowed.shape[1]
    for lp, page in enumerate(pages):
        pm = page_masks.get(int(page))
        if pm is None:
            continue
        lo, hi = lp * P, min((lp + 1) * P, kv_len)
        if lo >= kv_len:
            break
        out[:, lo:hi] &= np.asarray(pm, dtype=bool)[None, : hi - lo]
    return out


def forward(pool, P, H_q, qo_indptr, page_indptr, page_indices, last_page_len,
            q, k_new, v_new, masks=None, append=True, requests=None, page_masks=None,
            rope_theta=None, positions=None, out_lens=None, no_store=None):
    """One batched `forward`: append, then gather and attend for every request.

    q [T, H_q, D], k_new/v_new [T, H_kv, D] in the storage type; masks is None or a list
    with, per request, None (inferred causal) or a bool [q_len, kv_len] matrix.
    `requests` restricts step 3 to some request ids (rows of the others stay 0 / -inf); the
    append is always done for the whole batch.  Returns O [T, H_q, D] fp64, LSE [T, H_q].

    out_lens (Section 4.2 "Forward API": a call populates output Embeds and/or output KvPages;
    its listing stores 8 tokens with no output and produces 1 output from 9 inputs): request r
    produces outputs for its LAST out_lens[r] query tokens only - 0 = the rows are stored and
    nothing else.  Rows that produce no output come back as NaN (O and LSE); every row is
    appended and keeps its own position and mask row.

    no_store (same passage: a call WITHOUT output KvPages, `forward(kv, iemb[-1:], oemb)` and
    `forward([], iemb, [], oemb)` in the listing): request r's new rows take part in the attention
    - they are the last q_len positions of its context - but are stored nowhere.  For such a request
    the page list and last_page_len describe the EXISTING context only (an empty page list = none),
    and an explicit mask is [q_len, existing + q_len].
    """
    R = len(qo_indptr) - 1
    T = int(qo_indptr[R])
    D = q.shape[-1]
    q64 = widen(q)
    if rope_theta:
        # positions inside the path: Q is rotated for the attention, K is rotated before it is stored
        # (the pages hold position-encoded keys)
        pos = default_positions(qo_indptr, page_indptr, last_page_len, P) if positions is None else np.asarray(positions)
        # (both rotated operands are values of the element type: the attention consumes bf16 / fp32 Q and K)
        q64 = widen(to_storage(rope(q64, pos, rope_theta), np.asarray(q)))
        k_new = to_storage(rope(widen(k_new), pos, rope_theta), k_new)
    if append:
        append_kv(pool, P, qo_indptr, page_indptr, page_indices, last_page_len, k_new, v_new, skip=no_store)
    O = np.zeros((T, H_q, D), dtype=np.float64)
    LSE = np.full((T, H_q), -np.inf, dtype=np.float64)
    for r in (range(R) if requests is None else requests):
        t0, t1 = int(qo_indptr[r]), int(qo_indptr[r + 1])
        pages = page_indices[page_indptr[r]:page_indptr[r + 1]]
        unstored = no_store is not None and bool(no_store[r])
        if unstored:   # the pages hold the existing context; the new rows follow it without being stored
            kv_in = kv_len_of(len(pages), int(last_page_len[r]), P) if len(pages) else 0
            kv_len = kv_in + (t1 - t0)
        else:
            kv_in = kv_len = kv_len_of(len(pages), int(last_page_len[r]), P)
        allowed = allowed_matrix(t1 - t0, kv_len, None if masks is None else masks[r])
        if page_masks:   # (page masks belong to stored rows: the existing context)
            allowed = allowed.copy()
            allowed[:, :kv_in] = apply_page_masks(allowed[:, :kv_in], pages, P, page_masks)
        first = 0 if out_lens is None else (t1 - t0) - int(out_lens[r])   # first query token that produces an output
        O[t0:t0 + first], LSE[t0:t0 + first] = np.nan, np.nan
        if first == t1 - t0:
            continue
        allowed = allowed[first:]
        K, V = gather_kv(pool, P, pages, kv_in, needed=allowed[:, :kv_in].any(axis=0))
        if unstored:
            shape = (kv_len,) + tuple(np.asarray(k_new).shape[1:])
            Kc, Vc = np.zeros(shape), np.zeros(shape)
            if K is not None:
                Kc[:kv_in], Vc[:kv_in] = K, V
            Kc[kv_in:], Vc[kv_in:] = widen(k_new[t0:t1]), widen(v_new[t0:t1])
            K, V = Kc, Vc
        O[t0 + first:t1], LSE[t0 + first:t1] = attend(q64[t0 + first:t1], K, V, allowed)
    return O, LSE


# --------------------------------------------------------------------------- step 4: copy
def copy_kvpage(pool, src, dst, src_off, dst_off, ntok):
    """Token-level page copy (Table 1 `copy_kvpage`): for every op, rows
    [src_off, src_off + ntok) of page src are copied, K and V, to rows starting at dst_off
    of page dst.  All sources are read before any destination is written."""
    staged = []
    for s, d, so, do, n in zip(src, dst, src_off, dst_off, ntok):
        Ks, Vs = pool[int(s)]
        staged.append((int(d), int(do), int(n), Ks[so:so + n].copy(), Vs[so:so + n].copy()))
    for d, do, n, Kc, Vc in staged:
        Kd, Vd = pool[d]
        Kd[do:do + n] = Kc
        Vd[do:do + n] = Vc
        pool[d] = (Kd, Vd)


# --------------------------------------------------------------------------- merge identity
def merge_partials(o_parts, lse_parts):
    """Combine attention results computed over disjoint parts of the allowed set:
    lse = ln sum_c exp(lse_c),  o = sum_c exp(lse_c - lse) o_c.
    o_parts [C, ..., D], lse_parts [C, ...]; parts with lse = -inf contribute nothing."""
    o_parts = np.asarray(o_parts, dtype=np.float64)
    lse_parts = np.asarray(lse_parts, dtype=np.float64)
    m = lse_parts.max(axis=0)
    live = np.isfinite(m)
    w = np.exp(lse_parts - np.where(live, m, 0.0))
    Z = w.sum(axis=0)
    lse = np.where(live, m + np.log(np.where(live, Z, 1.0)), -np.inf)
    o = (w[..., None] * o_parts).sum(axis=0) / np.where(live, Z, 1.0)[..., None]
    o = np.where(live[..., None], o, 0.0)
    return o, lse


# --------------------------------------------------------------------------- sample stage
def next_dist(logits: np.ndarray, K: int):
    """`get_next_dist` from the logits on (Section 4.2 "Sample API": the next-token probability
    distribution, truncated to the top-K tokens, K = 256 by default).

    logits [n, V] in the storage type (float32, or uint16 holding bf16 bit patterns).  Row by row:
    p = softmax over the WHOLE vocabulary in fp64; the K most probable tokens are returned in order
    of descending probability, equal logits in order of ascending token id, with their
    probabilities as they stand in the full distribution (not renormalised over the K kept).
    Returns ids [n, K] int64, probs [n, K] fp64.
    """
    x = widen(np.asarray(logits))
    n, V = x.shape
    assert 1 <= K <= V
    ids = np.zeros((n, K), dtype=np.int64)
    probs = np.zeros((n, K), dtype=np.float64)
    for r in range(n):
        m = x[r].max()
        e = np.exp(x[r] - m)
        p = e / e.sum()
        order = sorted(range(V), key=lambda t: (-x[r, t], t))[:K]   # (by logit: exp is monotone, ties stay ties)
        ids[r] = order
        probs[r] = p[order]
    return ids, probs
