"""The N > 1 path on CPU: two gloo ranks shard one batch by request (no data-path collective),
plan their slices with host-only contexts, and reduce tokens / time the way bench.py does."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import paper_2510_24051_b200 as pie
    from paper_2510_24051_b200 import shard
    from workloads import configs
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = configs.small("long_context_policy")
    mi, mb = wl.mask_bytes()
    sh = shard.shard_batch(wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len, world, rank, mi, mb)
    ctx = pie.pie_create(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype, wl.R, wl.T, device=-1)
    pie.pie_alloc_kvpages(ctx, wl.num_pages)
    plan = pie.pie_plan_forward(ctx, sh["qo_indptr"], sh["page_indptr"], sh["page_indices"], sh["last_page_len"],
                                sh["mask_indptr"], sh["mask"])
    info = pie.pie_plan_get_info(plan)
    pie.pie_plan_destroy(plan)
    pie.pie_destroy(ctx)
    tokens, ms = shard.aggregate(info["num_query_tokens"], 10.0 + rank)
    q.put((rank, sh["requests"], info["num_requests"], info["kept_pages"], tokens, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_by_request():
    from paper_2510_24051_b200 import shard
    from workloads import configs
    world, port = 2, 29500 + os.getpid() % 2000
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    wl = configs.small("long_context_policy")
    assert [r[1] for r in res] == [shard.shard_bounds(wl.R, world, k) for k in range(world)]
    assert sum(r[2] for r in res) == wl.R                      # every request on exactly one rank
    assert all(r[4] == wl.T and r[5] == 11.0 for r in res)     # sum of tokens, max of times
    # the slices partition the work: kept pages add up to the single-rank plan
    import paper_2510_24051_b200 as pie
    c = pie.pie_create(wl.num_pages, wl.P, wl.H_q, wl.H_kv, wl.D, wl.dtype, wl.R, wl.T, device=-1)
    pie.pie_alloc_kvpages(c, wl.num_pages)
    mi, mb = wl.mask_bytes()
    plan = pie.pie_plan_forward(c, wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len, mi, mb)
    assert sum(r[3] for r in res) == pie.pie_plan_get_info(plan)["kept_pages"]
    pie.pie_plan_destroy(plan)
    pie.pie_destroy(c)


def test_shard_bounds_cover_everything():
    from paper_2510_24051_b200 import shard
    for n in (0, 1, 7, 64):
        for w in (1, 2, 3, 8):
            b = [shard.shard_bounds(n, w, r) for r in range(w)]
            assert b[0][0] == 0 and b[-1][1] == n
            assert all(b[i][1] == b[i + 1][0] for i in range(w - 1))
            assert max(h - l for l, h in b) - min(h - l for l, h in b) <= 1
