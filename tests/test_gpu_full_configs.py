"""Full-size workloads, in the launch configuration bench.py times, checked against the oracle
on sampled requests (the oracle computes any request on its own), plus size-independent
properties: finite outputs everywhere, bit-exact append on sampled pages."""
import numpy as np
import pytest

from tests._util import bits, same_bits
from workloads import configs

pytestmark = pytest.mark.gpu


def _sampled_check(wl, sample, peaked=False):
    from oracle import pie_oracle as orc
    from tests._gpu import check_close, run_workload
    q = wl.q()
    if peaked:
        q = (q.float() * 4).to(q.dtype)
    O, L, info, gp = run_workload(wl, q_scale=4.0 if peaked else 1.0, keep=True)
    try:
        assert np.isfinite(O).all()
        pool = wl.oracle_pool()
        O_ref, L_ref = orc.forward(pool, wl.P, wl.H_q, wl.qo_indptr, wl.page_indptr, wl.page_indices,
                                   wl.last_page_len, bits(q), bits(wl.k_new()), bits(wl.v_new()),
                                   wl.masks, requests=sample)
        for r in sample:
            rows = slice(int(wl.qo_indptr[r]), int(wl.qo_indptr[r + 1]))
            check_close(O, L, O_ref, L_ref, wl.dtype, rows=rows)
            den = np.sqrt((O_ref[rows] ** 2).sum())
            rel = np.sqrt(((O[rows] - O_ref[rows]) ** 2).sum()) / den
            assert rel <= 1e-2, f"request {r}: relative RMS {rel}"
        # appended rows landed bit-exactly (pages that received new tokens, sampled requests)
        pages = np.unique(np.concatenate([
            wl.pages_of(r)[(int(wl.kv_lens()[r]) - int(wl.q_lens()[r])) // wl.P:] for r in sample]))
        K, V = gp.read_pages(pages)
        for n, p in enumerate(pages):
            assert same_bits(K[n], pool[int(p)][0]) and same_bits(V[n], pool[int(p)][1])
        return info, gp
    except Exception:
        gp.close()
        raise


def test_full_batched_decode():
    wl = configs.batched_decode()
    info, gp = _sampled_check(wl, sample=list(range(0, wl.R, 4)))
    gp.close()
    assert info["num_split_items"] > 0 and info["num_tile_items"] == 0


def test_full_mixed_prefill_decode():
    wl = configs.mixed_prefill_decode()
    kv = wl.kv_lens()
    pre = list(np.argsort(kv[:8])[[0, 7]])            # shortest and longest prefill chunk
    dec = [8, 8 + int(np.argmax(kv[8:])), 8 + int(np.argmin(kv[8:])), 127]
    info, gp = _sampled_check(wl, sample=pre + dec)
    gp.close()
    assert info["num_split_items"] > 0 and info["num_tile_items"] > 0


def test_full_shared_prefix_decode_cascade():
    wl = configs.shared_prefix_decode()
    B = wl.meta["branches"]
    sample = [0, 1, B - 1, B, 5 * B + 7, wl.R - 1] + list(range(3, wl.R, 61))
    info, gp = _sampled_check(wl, sample=sample)
    gp.close()
    assert info["num_tile_items"] > 0 and info["num_merge_groups"] == wl.R * wl.H_kv   # the planner chose the cascade


def test_full_shared_prefix_tree():
    wl = configs.shared_prefix_tree()
    info, gp = _sampled_check(wl, sample=[0, 17, 255])
    gp.close()


def test_full_shared_prefix_tree_peaked():
    wl = configs.shared_prefix_tree()
    info, gp = _sampled_check(wl, sample=[100], peaked=True)
    gp.close()


def test_full_long_context_policy_with_copy():
    import paper_2510_24051_b200 as pie
    wl = configs.long_context_policy()
    kv = wl.kv_lens()
    sample = [0, int(np.argmax(kv)), int(np.argmin(kv)), 255]
    info, gp = _sampled_check(wl, sample=sample)
    try:
        # dropped pages are never fetched: the kept list is ~27% of the page lists
        assert info["kept_pages"] < 0.4 * len(wl.page_indices)
        c = wl.copies
        pie.pie_copy_kvpage(gp.ctx, c["src"], c["dst"], c["src_off"], c["dst_off"], c["ntok"])
        for r in sample:                              # copied rows equal the source rows, bit for bit
            Ks, Vs = gp.read_pages([c["src"][r]])
            Kd, Vd = gp.read_pages([c["dst"][r]])
            n = int(c["ntok"][r])
            assert same_bits(Ks[0][:n], Kd[0][:n]) and same_bits(Vs[0][:n], Vd[0][:n])
    finally:
        gp.close()


def test_long_context_policy_with_8_token_pages():
    """A launch long enough for the dynamic chunk list (1.7 GB of kept K/V) on 8-token pages: chunks of odd page
    counts, pairs of pages per ring stage, partials through the merge kernel."""
    wl = configs.long_context_policy(R=64, P=8)
    kv = wl.kv_lens()
    info, gp = _sampled_check(wl, sample=[0, int(np.argmax(kv)), 63])
    gp.close()
    assert info["num_merge_groups"] == wl.R * wl.H_kv and info["num_split_items"] > 4 * wl.R * wl.H_kv


@pytest.mark.parametrize("P", [16, 8])
def test_large_single_requests(P):
    """Index arithmetic at the large end: a 131,071-token decode (8,192 pages of 16 tokens, many split chunks and a
    ragged last page) and a 300-token prefill chunk over a 20,000-token prefix in one batch."""
    from workloads.configs import _assemble
    wl = _assemble("large", 0x50494500 + 77, 32, 8, 128, P, "bf16", 9600 * 16 // P, [1, 300], [131071, 20300], None)
    info, gp = _sampled_check(wl, sample=[0, 1])
    gp.close()
    assert info["num_split_items"] > 100 and info["num_tile_items"] > 0
