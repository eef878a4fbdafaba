"""GPU parity of pie_get_next_dist (Section 4.2 "Sample API": the next-token distribution truncated to the
top-K tokens) against the fp64 oracle: token ids bit-exact - the order is fixed by descending logit, then
ascending token id -, probabilities to 2e-5 relative (fp32 exponentials and a 128 K-term fp32 sum)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _ctx():
    import paper_2510_24051_b200 as pie
    return pie.pie_create(4, 16, 4, 2, 64, "bf16", 4, 64, 0)


def _check(logits_dev, K):
    import paper_2510_24051_b200 as pie
    from oracle import pie_oracle as orc
    n = logits_dev.shape[0]
    ids = torch.full((n, K), -1, dtype=torch.int32, device="cuda")
    probs = torch.full((n, K), float("nan"), dtype=torch.float32, device="cuda")
    ctx = _ctx()
    try:
        pie.pie_get_next_dist(ctx, logits_dev, K, ids, probs)
        torch.cuda.synchronize()
    finally:
        pie.pie_destroy(ctx)
    host = logits_dev.cpu()
    stored = host.view(torch.int16).numpy().view(np.uint16) if host.dtype == torch.bfloat16 else host.numpy()
    ids_ref, probs_ref = orc.next_dist(np.ascontiguousarray(stored), K)
    assert np.array_equal(ids.cpu().numpy().astype(np.int64), ids_ref)
    got = probs.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    np.testing.assert_allclose(got, probs_ref, rtol=2e-5, atol=1e-30)
    return got


def _logits(n, V, dtype, seed, scale=2.5):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(n, V, generator=g) * scale
    x[:, ::977] += 9.0                      # a few tokens far ahead of the rest, as in a trained model
    return x.to(dtype)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("n,V,K", [(5, 1000, 7), (3, 128256, 256), (2, 50257, 256), (2, 4096, 1024), (4, 300, 1), (2, 64, 64)])
def test_next_dist_matches_oracle(n, V, K, dtype):
    p = _check(_logits(n, V, dtype, seed=V + K).cuda(), K)
    assert (np.diff(p, axis=1) <= 0).all()
    if K == V:
        np.testing.assert_allclose(p.sum(axis=1), 1.0, rtol=1e-5)


def test_next_dist_with_many_equal_logits_and_masked_vocabulary():
    """Quantised logits (ties everywhere, also across the K-th place), -inf entries (tokens an inferlet has
    excluded), rows that start at unaligned addresses and rows that are further apart than they are long."""
    g = torch.Generator().manual_seed(5)
    x = torch.randint(-6, 7, (4, 20011), generator=g).float() * 0.5
    x[1, 100:15000] = float("-inf")
    x[2, :] = 1.25                                                  # every token equally likely: ids 0 .. K-1
    for dtype in (torch.bfloat16, torch.float32):
        _check(x.to(dtype).cuda(), 256)
        wide = torch.zeros(4, 20011 + 37, dtype=dtype)
        wide[:, 3:3 + 20011] = x.to(dtype)
        _check(wide.cuda()[:, 3:3 + 20011], 300)                   # row stride > vocab, rows not 16-byte aligned
    p = _check(x[2:3].cuda(), 16)
    np.testing.assert_allclose(p, 1.0 / 20011, rtol=1e-5)


def test_next_dist_on_decode_batches_with_a_cluster_of_blocks_per_row():
    """Aligned bf16 rows of at least 8,192 logits in batches up to twice the SM count run with a cluster of thread
    blocks per row (parts of the row in shared memory, candidates gathered through distributed shared memory):
    the benchmark's shape (2 blocks per row), a few rows (4 blocks per row), a vocabulary that is not a multiple
    of 8 inside a wider row stride, and quantised / constant / partly masked rows, where the candidates overflow
    and the first block redoes the row the general way."""
    _check(_logits(64, 128256, torch.bfloat16, seed=11).cuda(), 256)
    _check(_logits(5, 32768, torch.bfloat16, seed=12).cuda(), 256)
    wide = torch.zeros(3, 50264, dtype=torch.bfloat16)
    wide[:, :50260] = _logits(3, 50260, torch.bfloat16, seed=13)
    _check(wide.cuda()[:, :50260], 100)
    g = torch.Generator().manual_seed(6)
    x = torch.randint(-6, 7, (4, 20016), generator=g).float() * 0.5
    x[1, 100:15000] = float("-inf")
    x[2, :] = 1.25
    _check(x.to(torch.bfloat16).cuda(), 256)
    p = _check(x[2:3].to(torch.bfloat16).cuda(), 16)
    np.testing.assert_allclose(p, 1.0 / 20016, rtol=1e-5)
    big = (_logits(4, 32768, torch.float32, seed=14) + 300.0).to(torch.bfloat16)      # logits far from zero
    _check(big.cuda(), 256)
    _check(big.float().cuda(), 256)                                                   # (the one-block kernel)


def test_next_dist_argument_errors():
    import paper_2510_24051_b200 as pie
    ctx = _ctx()
    try:
        x = torch.zeros(2, 100, device="cuda")
        ids = torch.zeros(2, 2000, dtype=torch.int32, device="cuda")
        pr = torch.zeros(2, 2000, device="cuda")
        for K in (0, 101, 1025):
            with pytest.raises(pie.PieError) as e:
                pie.pie_get_next_dist(ctx, x, K, ids, pr)
            assert e.value.status == pie.PIE_ERR_INVALID
        pie.pie_get_next_dist(ctx, x[:0], 5, ids, pr)               # no rows: nothing to do
    finally:
        pie.pie_destroy(ctx)
