"""Helpers shared by the tests: small random batches and oracle runs on a Workload."""
from __future__ import annotations

import numpy as np

from oracle import pie_oracle as orc
from workloads import synth


def bits(t):
    return synth.to_numpy_bits(t)


def same_bits(a, b):
    """Bitwise equality (NaN patterns included) of two arrays of the same storage type."""
    a, b = np.ascontiguousarray(a), np.ascontiguousarray(b)
    if a.dtype == np.float32:
        a, b = a.view(np.uint32), b.view(np.uint32)
    return a.shape == b.shape and np.array_equal(a, b)


def run_oracle(wl, poison=False, requests=None, pool=None):
    """Oracle forward on a Workload; returns (O fp64, LSE fp64, pool after the append)."""
    pool = wl.oracle_pool(poison) if pool is None else pool
    O, LSE = orc.forward(pool, wl.P, wl.H_q, wl.qo_indptr, wl.page_indptr, wl.page_indices,
                         wl.last_page_len, bits(wl.q()), bits(wl.k_new()), bits(wl.v_new()),
                         wl.masks, requests=requests)
    return O, LSE, pool


class SmallBatch:
    """A batch built from dense per-request sequences, paged with an arbitrary placement.

    seqs: list of dicts with K, V [kv_len, H_kv, D] float32 (all rows, incl. the new ones),
    Q [q_len, H_q, D] float32, and optional mask.  `paged(P, order)` lays the rows that
    precede the query tokens into pages and returns the oracle's arguments.
    """

    def __init__(self, seqs, H_q):
        self.seqs, self.H_q = seqs, H_q

    def paged(self, P, order="contiguous", seed=0, num_extra=3):
        rng = np.random.RandomState(seed)
        nps = [(len(s["K"]) + P - 1) // P for s in self.seqs]
        total = sum(nps) + num_extra
        ids = np.arange(total)
        if order == "reversed":
            ids = ids[::-1].copy()
        elif order == "random":
            ids = rng.permutation(total)
        H_kv, D = self.seqs[0]["K"].shape[1:]
        pool = {int(p): (np.full((P, H_kv, D), np.nan, np.float32),
                         np.full((P, H_kv, D), np.nan, np.float32)) for p in range(total)}
        qo, pi, idx, last = [0], [0], [], []
        cur = 0
        for s, n in zip(self.seqs, nps):
            pages = ids[cur:cur + n]
            cur += n
            kv_len, q_len = len(s["K"]), len(s["Q"])
            for j in range(kv_len - q_len):            # context that already exists
                K, V = pool[int(pages[j // P])]
                K[j % P], V[j % P] = s["K"][j], s["V"][j]
            qo.append(qo[-1] + q_len)
            pi.append(pi[-1] + n)
            idx.extend(pages.tolist())
            last.append(kv_len - (n - 1) * P)
        q = np.concatenate([s["Q"] for s in self.seqs])
        k_new = np.concatenate([s["K"][len(s["K"]) - len(s["Q"]):] for s in self.seqs])
        v_new = np.concatenate([s["V"][len(s["V"]) - len(s["Q"]):] for s in self.seqs])
        masks = [s.get("mask") for s in self.seqs]
        return dict(pool=pool, P=P, H_q=self.H_q, qo_indptr=np.array(qo), page_indptr=np.array(pi),
                    page_indices=np.array(idx), last_page_len=np.array(last), q=q, k_new=k_new,
                    v_new=v_new, masks=masks)


def random_seqs(rng, shapes, H_q, H_kv, D, masks=None):
    seqs = []
    for n, (q_len, kv_len) in enumerate(shapes):
        s = dict(Q=rng.randn(q_len, H_q, D).astype(np.float32),
                 K=rng.randn(kv_len, H_kv, D).astype(np.float32),
                 V=rng.randn(kv_len, H_kv, D).astype(np.float32))
        if masks is not None and masks[n] is not None:
            s["mask"] = masks[n]
        seqs.append(s)
    return seqs


def oracle_on(args):
    return orc.forward(**args)
