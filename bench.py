#!/usr/bin/env python
"""Benchmark of the batched `forward` attention handler on synthetic workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME|all] [--impl reference]

One "step" is one pass of the whole hot path over one coalesced batch: pie_forward (append of
the new K/V rows, attention, merge of split partials) plus, for the long-context workload, the
pie_copy_kvpage call that follows it.  Plans are built once (host planning time is reported
separately as `plan_ms`); inputs are resident in HBM when the timed region starts.  A timed
region is exactly K steps between two synchronisations, measured with CUDA events; regions are
repeated until a workload has at least `--min-seconds` of device time behind it and the median
region is reported (with the fastest and slowest one beside it).

With no `--workload` the run covers every baseline configuration in one go and prints ONE JSON
line: the top level describes the headline workload (the largest single-GPU configuration,
`long_context_policy`) and `workloads` holds one entry per configuration - each with its own
step time, tokens/s, roofline of its dominant kernel, end-to-end figure, clocks and CPU baseline.

The `e2e` figure goes through pie_forward_host: planning, pinned-host -> device copies of
Q/K/V and the device -> host read of the outputs are inside its timed region.  For decode
workloads it is a decode LOOP - every step appends one token to every request, so page lists,
masks and the plan change from step to step as in a serving loop - and for the others a replay
of the batch with a fresh plan per step.

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank runs its own batch
of the headline shape (requests are independent: no data-path collective); the time is the max
over ranks and `value` counts all ranks' tokens (weak scaling).

`--impl reference` times the fp64 CPU oracle on the same workload shape instead.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "attention tokens/s and achieved HBM GB/s / tensor TFLOPS vs B200 peak"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
HEADLINE = "long_context_policy"
# the default run: the five baseline configurations (config 3 also as its two halves), then
# two entries of our own (a small decode batch, the sample-stage handler)
SUITE = ["long_context_policy", "batched_decode", "mixed_prefill_decode", "mixed_prefill_decode_prefill",
         "mixed_prefill_decode_decode", "shared_prefix_tree", "batched_decode_r16", "next_dist"]

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from one ncu
# capture per workload (not measured in this run: a profiler cannot run inside a timed benchmark)
NCU_TRAFFIC = {
    "batched_decode": (287_950_000, "ncu capture of the split-KV kernel on this workload, two launches"),
    "shared_prefix_tree": (980_300_000, "ncu capture of the row-tile kernel on this workload, two launches"),
    "mixed_prefill_decode_prefill": (82_500_000, "ncu capture of the row-tile kernel on this workload, two launches"),
    "next_dist": (16_480_000, "ncu capture of the cluster kernel on this workload, two launches"),
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    return dict(FALLBACK_PEAKS, source="fallback")


def builder_of(name):
    """(builder, fixed keyword arguments, index for the seed) of a workload name."""
    from workloads import configs
    table = dict(configs.FULL, **configs.EXTRA)
    alias = {
        "mixed_prefill_decode_prefill": ("mixed_prefill_decode", {"only": "prefill"}),
        "mixed_prefill_decode_decode": ("mixed_prefill_decode", {"only": "decode"}),
        "batched_decode_r16": ("batched_decode", {"R": 16}),
    }
    base, fixed = alias.get(name, (name, {}))
    return table[base], dict(fixed), list(table).index(base) + 1


def build_workloads(name, seed_offset=0, params=()):
    """The list of batches a run cycles through (several page placements when one batch's KV is
    small enough to live in L2), plus a note saying how L2 reuse is defeated.  `params` ("key=value"
    strings, --param) override arguments of the workload's builder for shape sweeps."""
    from workloads import configs
    builder, kw, index = builder_of(name)
    seed = configs.SEED0 + index + 1000 * seed_offset
    for kv in params:
        k, v = kv.split("=", 1)
        kw[k] = int(v) if v.lstrip("-").isdigit() else (None if v == "None" else v)
    seed = kw.pop("seed", seed)
    if name.startswith("batched_decode"):
        probe = builder(seed=seed, **kw)
        n_place = max(1, min(16, probe.num_pages // len(probe.page_indices)))
        wls = [builder(seed=seed, placement=i, **kw) for i in range(n_place)]
        note = f"{n_place} rotating page placements ({n_place * probe.algorithmic_bytes()['kv'] / 1e9:.2f} GB of KV) > L2"
    else:
        wls = [builder(seed=seed, **kw)]
        note = f"one placement; KV read per step {wls[0].algorithmic_bytes()['kv'] / 1e9:.2f} GB > L2"
    for wl in wls:
        wl.name = name
    if kw:
        note += "; builder arguments " + ", ".join(f"{k}={v}" for k, v in kw.items())
    return wls, note


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap,clocks.mem,clocks.max.mem,temperature.memory")

    def __init__(self, device):
        self.rows, self.proc, self.device = [], None, device

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.device), f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm, mx, pw, reasons = [], [], [], set()
        mem, mem_max, mem_temp = [], [], []
        for r in self.rows:
            try:
                sm.append(float(r[0])), mx.append(float(r[1]))
                pw.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
            for dst, v in zip((mem, mem_max, mem_temp), r[7:10]):   # (memory clock and temperature: not every driver reports them)
                try:
                    dst.append(float(v))
                except ValueError:
                    pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "sm_min_mhz": min(sm) if sm else None, "power_w_max": max(pw) if pw else None,
                "mem_mhz_min": min(mem) if mem else None, "mem_max_mhz": max(mem_max) if mem_max else None,
                "mem_temp_c_max": max(mem_temp) if mem_temp else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_prepare(wl, budget_s):
    """A bounded sample of the workload for the oracle: a prefix of its requests whose estimated cost fits the
    budget, with every input the oracle will touch generated beforehand (outside any timed region)."""
    from workloads import synth
    qb, kb, vb = (synth.to_numpy_bits(t) for t in (wl.q(), wl.k_new(), wl.v_new()))
    cost = wl.q_lens() * wl.kept_tokens() * wl.H_q * wl.D * 4.0
    rate = 2e9                                        # conservative fp64 flop/s incl. gather overhead
    n, acc = 0, 0.0
    while n < wl.R and (n == 0 or acc + cost[n] / rate <= budget_s):
        acc += cost[n] / rate
        n += 1
    sample = np.arange(n)
    pool = wl.oracle_pool()
    need_pages = []
    for r in sample:                                  # the pages the sampled requests attend to
        m = None if wl.masks is None else wl.masks[r]
        npg = len(wl.pages_of(r))
        if m is None:
            need = np.ones(npg, bool)
        else:
            cols = np.zeros(npg * wl.P, bool)
            cols[:m.shape[1]] = m.any(axis=0)
            need = cols.reshape(npg, wl.P).any(axis=1)
        need_pages.append(wl.pages_of(r)[need])
    kv, ql = wl.kv_lens(), wl.q_lens()
    for r in range(wl.R):                             # pages the append writes (the oracle appends the whole batch)
        need_pages.append(wl.pages_of(r)[(int(kv[r]) - int(ql[r])) // wl.P:])
    pool.prefetch(np.concatenate(need_pages))
    return {"wl": wl, "sample": sample, "pool": pool, "q": qb, "k": kb, "v": vb,
            "desc": f"first {n} of {wl.R} requests of {wl.name}"}


def oracle_pass(prep):
    """One timed pass of the fp64 oracle, as it stands, over the prepared sample.  Returns seconds."""
    from oracle import pie_oracle as orc
    wl = prep["wl"]
    t0 = time.perf_counter()
    orc.forward(prep["pool"], wl.P, wl.H_q, wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len,
                prep["q"], prep["k"], prep["v"], wl.masks, requests=prep["sample"])
    return time.perf_counter() - t0


def oracle_sample(wl, budget_s=20.0):
    """Time the oracle on a bounded sample of the workload's requests.  Returns (tokens, seconds, description,
    cores): cores = CPU time the process spent per second of wall time, i.e. the threads that were actually busy
    (the oracle is one Python thread; only its large matrix products fan out over the BLAS pool)."""
    prep = oracle_prepare(wl, budget_s)
    times = []
    cpu0 = time.process_time()
    while not times or (sum(times) < min(budget_s, 10.0) and len(times) < 20):   # repeat short passes
        times.append(oracle_pass(prep))
    cores = max(1, int(round((time.process_time() - cpu0) / max(sum(times), 1e-9))))
    dt = statistics.mean(times)
    tokens = int(wl.q_lens()[prep["sample"]].sum())
    return tokens, dt, f"{prep['desc']}, mean of {len(times)} passes", cores


def cpu_baseline_of(wl, budget_s):
    tokens, dt, desc, cores = oracle_sample(wl, budget_s=budget_s)
    return {"value": tokens / dt, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": desc, "seconds": dt,
            "threads": "one Python thread; numpy's BLAS pool is used by large matrix products only"}


def run_reference(args):
    """The reference arm: the fp64 CPU oracle, as it stands, on the host cores.  A step is one pass over a bounded
    sample of the headline workload (prepared once, outside the timed passes)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    name = HEADLINE if args.workload == "all" else args.workload
    wls, _ = build_workloads(name, params=args.param)
    wl = wls[0]
    prep = oracle_prepare(wl, budget_s=3.0)
    tokens = int(wl.q_lens()[prep["sample"]].sum())
    t_start = time.perf_counter()
    for _ in range(args.warmup):
        oracle_pass(prep)
        if time.perf_counter() - t_start > 60:        # keep the whole run within a few minutes
            break
    times = []
    cpu0, t0 = time.process_time(), time.perf_counter()
    for _ in range(args.steps):
        times.append(oracle_pass(prep))
        if time.perf_counter() - t_start > 180:
            break
    cores = max(1, int(round((time.process_time() - cpu0) / max(time.perf_counter() - t0, 1e-9))))
    dt = statistics.mean(times)
    val = tokens / dt
    desc = f"{prep['desc']}, {len(times)} timed passes"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": len(times), "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "sample": desc},
        "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


class Env:
    """torch / binding / process-group handles of this rank."""

    def __init__(self):
        import torch
        import torch.distributed as dist
        import paper_2510_24051_b200 as pie
        self.torch, self.dist, self.pie = torch, dist, pie
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
        torch.cuda.set_device(self.local)
        if self.world > 1:
            dist.init_process_group("nccl", device_id=torch.device("cuda", self.local))

    def barrier(self):
        if self.world > 1:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def max_over_ranks(self, x):
        if self.world == 1:
            return x
        t = self.torch.tensor([float(x)], dtype=self.torch.float64, device="cuda")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def close(self):
        if self.world > 1:
            self.dist.destroy_process_group()

    def device_info(self):
        """Which GPU this ran on, and its plain device-to-device copy rate right now (1 GiB, read + write
        bytes, median of 10 after 3 untimed): context for the fractions, which are rated against the pool's
        measured peaks."""
        torch = self.torch
        props = torch.cuda.get_device_properties(self.local)
        x = torch.empty(1 << 30, dtype=torch.uint8, device="cuda")
        y = torch.empty_like(x)
        ts = []
        for i in range(13):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            y.copy_(x)
            b.record()
            torch.cuda.synchronize()
            if i >= 3:
                ts.append(a.elapsed_time(b))
        del x, y
        torch.cuda.empty_cache()
        return {"name": props.name, "uuid": str(getattr(props, "uuid", "")), "sms": props.multi_processor_count,
                "copy_gbs_now": 2 * (1 << 30) / (statistics.median(ts) * 1e-3) / 1e9}


def timed_regions(env, step, steps, min_seconds, max_regions=4000):
    """Regions of exactly `steps` steps, each between a barrier + synchronize on both sides and timed with
    CUDA events on the launching stream (max over ranks), repeated until `min_seconds` of device time
    have been measured.  Returns the per-region milliseconds."""
    torch = env.torch
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    regions, total, i = [], 0.0, 0
    while True:
        env.barrier()
        ev0.record()
        for _ in range(steps):
            step(i)
            i += 1
        ev1.record()
        env.barrier()
        ms = env.max_over_ranks(ev0.elapsed_time(ev1))
        regions.append(ms)
        total += ms
        if total >= min_seconds * 1e3 or len(regions) >= max_regions:
            return regions


def install_context(env, ctx, wl):
    pie, torch = env.pie, env.torch
    used = wl.used_pages()
    for i in range(0, len(used), 4096):
        K, V = wl.context_pages(used[i:i + 4096], "cuda")
        pie.pie_kvpage_write(ctx, used[i:i + 4096], K.contiguous(), V.contiguous())
        torch.cuda.synchronize()
        del K, V


def e2e_decode_loop(env, args, name, wl0, ctx, hbuf, step_ms):
    """End to end as a serving loop would call it: every step appends one token to every request, so
    lengths, page lists, policy masks and therefore the plan change from step to step.  Small batches
    (KV of a step close to the L2 size) run as several independent loops over different requests,
    visited in turn, so that no step finds its pages in L2."""
    from workloads import configs, synth
    pie, torch = env.pie, env.torch
    hq, hk, hv, hout, hlse = hbuf
    n_steps = max(3, min(args.steps, 30 if step_ms > 0.5 else 300))
    own_ctx = None
    if name.startswith("batched_decode"):
        builder, kw, _ = builder_of(name)
        for kv in args.param:
            k, v = kv.split("=", 1)
            if k != "seed":
                kw[k] = int(v) if v.lstrip("-").isdigit() else v
        n_streams = max(2, min(8, int(math.ceil(3 * 126e6 / max(wl0.algorithmic_bytes()["kv"], 1)))))
        visits = (n_steps + n_streams - 1) // n_streams
        n_steps = visits * n_streams
        grow = wl0.R * ((visits + wl0.P - 1) // wl0.P + 1)
        streams, off = [], 0
        sizes = []
        for j in range(n_streams):   # (a first pass for the page counts: each loop has its own lengths)
            probe = builder(seed=wl0.seed + 100 * (j + 1), **kw)
            sizes.append(len(probe.page_indices))
        num_pages = sum(sizes) + n_streams * grow
        perm = synth.permutation(wl0.seed, 10, num_pages)
        for j in range(n_streams):
            wl = builder(seed=wl0.seed + 100 * (j + 1), perm_seed=wl0.seed, page_offset=off, **dict(kw, num_pages=num_pages))
            spare = perm[off + sizes[j]:off + sizes[j] + grow]
            off += sizes[j] + grow
            streams.append((wl, configs.decode_loop(wl, visits, spare)))
        own_ctx = pie.pie_create(num_pages, wl0.P, wl0.H_q, wl0.H_kv, wl0.D, wl0.dtype, wl0.R, wl0.T, env.local)
        pie.pie_alloc_kvpages(own_ctx, num_pages)
        for wl, _ in streams:
            install_context(env, own_ctx, wl)
        ctx = own_ctx
        batches = [streams[s % n_streams][1][s // n_streams] for s in range(n_steps)]
        how = f"decode loop: {n_streams} independent loops of {wl0.R} requests visited in turn, one token appended per visit"
    else:
        # pages the loop may grow into: those of the pool that the batch does not hold (lists may share pages)
        taken = np.zeros(wl0.num_pages, dtype=bool)
        taken[np.asarray(wl0.page_indices)] = True
        total = wl0.meta.get("pages_in_lists", 0)     # (the long-context batch lists only its kept pages: all of a request's pages are its own)
        perm = synth.permutation(wl0.seed, 10, wl0.num_pages)
        taken[perm[:total + (wl0.R if wl0.copies is not None else 0)]] = True
        if wl0.copies is not None:
            taken[np.asarray(wl0.copies["dst"])] = True
        spare = perm[~taken[perm]]
        n_steps = min(n_steps, max(3, (len(spare) // max(wl0.R, 1)) * wl0.P - wl0.P))   # (never more page crossings than spare pages)
        batches = configs.decode_loop(wl0, n_steps, spare)
        how = f"decode loop: one token appended to each of the {wl0.R} requests per step"

    def e2e_step(i):
        b = batches[i % len(batches)]
        pie.pie_forward_host(ctx, b["qo_indptr"], b["page_indptr"], b["page_indices"], b["last_page_len"],
                             hq, hk, hv, hout, hlse, b["mask_indptr"], b["mask"], args.flags)
        if b["copies"] is not None:
            c = b["copies"]
            pie.pie_copy_kvpage(ctx, c["src"], c["dst"], c["src_off"], c["dst_off"], c["ntok"])
            torch.cuda.synchronize()

    for i in range(3):   # (warm-up on the first steps; the timed loop starts over from step 0)
        e2e_step(i)
    env.barrier()
    t0 = time.perf_counter()
    for i in range(n_steps):
        e2e_step(i)
    torch.cuda.synchronize()
    e2e_s = env.max_over_ranks(time.perf_counter() - t0)
    if own_ctx is not None:
        pie.pie_destroy(own_ctx)
    return n_steps, e2e_s, how + "; host planning of every step, pinned H2D of Q/K/V, forward, D2H of O/LSE"


def roofline_of(wl0, name, info, ktimes, ms_per_step, peaks, n_gpus, clocks, region_s):
    """Roofline entry of the workload's dominant kernel: algorithmic bytes (or useful flops) of one launch
    divided by the kernel's live launch duration, against the measured peak."""
    launches_per_step = info["launches"] + (1 if wl0.copies is not None else 0)
    dom = max(("split", "tiles", "simple"), key=lambda k: ktimes[k][0])
    dom_ms = ktimes[dom][0] / max(ktimes[dom][1], 1)
    dom_timing = "events around each launch of the kernel"
    if info.get("side_by_side_sms", 0) > 0:
        # decode and prefill kernels run at the same time on disjoint SM sets: per-kernel events overlap, so the
        # step is rated as a whole against the HBM roofline of its decode part (the prefill part is tensor work)
        dom, dom_ms = "split", ms_per_step
        dom_timing = "timed region / steps (decode and prefill kernels side by side)"
    elif launches_per_step == 1 and n_gpus == 1:
        # the step IS this one kernel: its launch duration is the timed region divided by the launches (the events
        # around single launches keep consecutive launches from overlapping their prologues and report more)
        dom_ms = min(dom_ms, ms_per_step)
        dom_timing = "timed region / launches (one kernel per step)"
    elif n_gpus == 1 and ms_per_step < dom_ms:
        # a kernel cannot take longer than the whole step that contains it: bracketing every launch with events
        # exposes launch latency and prologues that the back-to-back loop overlaps, so the step time is the bound
        dom_ms = ms_per_step
        dom_timing = "timed region / steps (upper bound: the step also contains the other kernels)"
    G = wl0.H_q // wl0.H_kv
    rows = wl0.q_lens() * G
    sel = rows <= 16 if dom == "split" else rows > 16
    b_tok = 2 * wl0.H_kv * wl0.D * wl0.esize
    traffic, traffic_source = NCU_TRAFFIC.get(name, (None, "not captured"))
    common = {"kernel_ms": dom_ms, "timing": dom_timing, "peak_source": peaks["source"], "traffic": traffic,
              "traffic_source": traffic_source}
    if dom == "tiles" and not sel.any():
        # shared-prefix cascade: the row-tile kernel attends gathered decode rows to the shared pages and the
        # split-KV kernel the private pages; together they read every distinct page once
        dom_ms = sum(ktimes[k][0] / max(ktimes[k][1], 1) for k in ("tiles", "split"))
        alg = len(np.unique(wl0.page_indices)) * wl0.P * b_tok + int(wl0.q_lens().sum()) * wl0.H_q * (2 * wl0.D * wl0.esize + 4)
        achieved = alg / (dom_ms * 1e-3) / 1e9
        return dict(common, bound="hbm", kernel="tiles+split (cascade)", achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s",
                    frac=achieved / peaks["hbm_gbs"], algorithmic_bytes=alg, kernel_ms=dom_ms)
    if dom in ("split", "simple"):
        kv_bytes = int(wl0.kept_tokens()[sel].sum()) * b_tok
        qo_bytes = int(wl0.q_lens()[sel].sum()) * wl0.H_q * (2 * wl0.D * wl0.esize + 4)
        mask_bytes = 0 if wl0.masks is None else sum((m.size + 7) // 8 for m, s in zip(wl0.masks, sel) if s and m is not None)
        alg = kv_bytes + qo_bytes + mask_bytes
        if dom == "split" and ktimes["append"][1] == 0:   # fused append: the split-KV kernel also moves the new rows
            alg += int(wl0.q_lens()[sel].sum()) * b_tok * 2
        achieved = alg / (dom_ms * 1e-3) / 1e9
        return dict(common, bound="hbm", kernel=dom, achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s",
                    frac=achieved / peaks["hbm_gbs"], algorithmic_bytes=alg)
    flops = 0
    for r in np.nonzero(sel)[0]:
        m = None if wl0.masks is None else wl0.masks[r]
        ql, kv = int(wl0.q_lens()[r]), int(wl0.kv_lens()[r])
        n = (ql * kv - ql * (ql - 1) // 2) if m is None else int(m.sum())
        flops += 4 * wl0.D * wl0.H_q * n
    achieved = flops / (dom_ms * 1e-3) / 1e12
    burst = peaks["bf16_tflops"]
    sustained = peaks.get("bf16_tflops_sustained", burst)
    # `frac` is always against the dense bf16 peak measured as a burst (cuBLAS at full clocks); the figure against
    # the peak measured over seconds under the power cap is given beside it.  Which regime this run was in
    # follows from the length of the timed region and the clocks sampled during it.
    mhz, mx = (clocks or {}).get("sm_mhz"), (clocks or {}).get("sm_max_mhz")
    regime = "sustained" if (region_s >= 0.5 and mhz and mx and mhz < 0.9 * mx) else "burst"
    return dict(common, bound="tensor", kernel=dom, achieved=achieved, peak=burst, unit="TFLOP/s", frac=achieved / burst,
                peak_sustained=sustained, frac_sustained=achieved / sustained, regime=regime,
                kernel_ms_x_sm_mhz=(dom_ms * mhz if mhz else None), useful_flops=flops,
                peak_source=peaks["source"] + " (bf16_tflops burst; bf16_tflops_sustained beside it)")


def bench_workload(env, args, name, cpu_budget_s):
    """One workload: device-resident timed regions, live per-kernel times, end to end through host buffers,
    the oracle on a bounded sample.  Returns the workload's entry (rank 0; other ranks get None)."""
    pie, torch = env.pie, env.torch
    wls, l2_note = build_workloads(name, seed_offset=env.rank, params=args.param)
    wl0 = wls[0]
    ctx = pie.pie_create(wl0.num_pages, wl0.P, wl0.H_q, wl0.H_kv, wl0.D, wl0.dtype, max(wl0.R, 1), max(wl0.T, 1), env.local)
    ids = pie.pie_alloc_kvpages(ctx, wl0.num_pages)
    assert np.array_equal(ids, np.arange(wl0.num_pages))
    for kv in args.opt:
        k, v = kv.split("=")
        pie.pie_set_option(ctx, int(k), int(v))
    for wl in wls:                                     # install the pre-existing context (device generator)
        install_context(env, ctx, wl)
    plans, plan_ms = [], []
    mask_args = [wl.mask_bytes() for wl in wls]
    for wl, (mi, mb) in zip(wls, mask_args):
        t0 = time.perf_counter()
        plans.append(pie.pie_plan_forward(ctx, wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len,
                                          mi, mb, args.flags))
        plan_ms.append((time.perf_counter() - t0) * 1e3)
    plan_first_ms = statistics.median(plan_ms)       # includes the first allocation of the plan's pinned and device arrays
    plan_ms = []                                     # steady state of a loop that plans every step: plan objects are recycled
    for i in range(6):
        mi, mb = mask_args[0]
        t0 = time.perf_counter()
        extra = pie.pie_plan_forward(ctx, wls[0].qo_indptr, wls[0].page_indptr, wls[0].page_indices, wls[0].last_page_len,
                                     mi, mb, args.flags)
        if i:
            plan_ms.append((time.perf_counter() - t0) * 1e3)
        pie.pie_plan_destroy(extra)
    info = pie.pie_plan_get_info(plans[0])
    q, k_new, v_new = wl0.q("cuda"), wl0.k_new("cuda"), wl0.v_new("cuda")
    out = torch.empty_like(q)
    lse = torch.empty((wl0.T, wl0.H_q), dtype=torch.float32, device="cuda")
    copies = wl0.copies

    def step(i):
        pie.pie_forward(ctx, plans[i % len(plans)], q, k_new, v_new, out, lse)
        if copies is not None:
            pie.pie_copy_kvpage(ctx, copies["src"], copies["dst"], copies["src_off"], copies["dst_off"], copies["ntok"])

    # ---------------------------------------------------------------- device-resident timing
    eager_step = step
    use_graph = args.graph == 1 and copies is None
    if use_graph:
        # pie_forward only enqueues kernels on the caller's stream, so a step is captured once per
        # page placement and replayed: no host launch cost inside the timed loop
        cap = torch.cuda.Stream()
        cap.wait_stream(torch.cuda.current_stream())
        graphs = []
        with torch.cuda.stream(cap):
            for i in range(len(plans)):
                eager_step(i)
            cap.synchronize()
            for i in range(len(plans)):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=cap):
                    eager_step(i)
                graphs.append(g)
        torch.cuda.current_stream().wait_stream(cap)

        def step(i):
            graphs[i % len(graphs)].replay()

    for i in range(args.warmup):
        step(i)
    env.barrier()
    sampler = ClockSampler(env.local)
    if env.rank == 0:
        sampler.start()
    regions = timed_regions(env, step, args.steps, args.min_seconds)
    assert pie.pie_get_last_device_status(ctx) == 0, "a device-side wait timed out"
    ms = statistics.median(regions)
    launches_per_step = info["launches"] + (1 if copies is not None else 0)

    # ---------------------------------------------------------------- per-kernel timing (live)
    pie.pie_set_kernel_timing(ctx, 1)
    for i in range(args.steps):
        eager_step(i)
    torch.cuda.synchronize()
    ktimes = pie.pie_get_kernel_times(ctx)
    pie.pie_set_kernel_timing(ctx, 0)
    clocks = sampler.stop() if env.rank == 0 else None         # covers the timed regions and the per-kernel loop

    # ---------------------------------------------------------------- end to end (host buffers)
    e2e = None
    if not args.no_e2e:
        hq, hk, hv = (t.cpu().pin_memory() for t in (q, k_new, v_new))
        hout = torch.empty_like(hq).pin_memory()
        hlse = torch.empty((wl0.T, wl0.H_q), dtype=torch.float32).pin_memory()
        h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv))
        d2h = hout.numel() * hout.element_size() + hlse.numel() * 4
        decode_only = bool((wl0.q_lens() == 1).all()) and (wl0.masks is None or "window" in wl0.meta)
        if decode_only:
            n_e2e, e2e_s, how = e2e_decode_loop(env, args, name, wl0, ctx, (hq, hk, hv, hout, hlse), ms / args.steps)
        else:
            # (short steps: more of them, so that one hiccup of the host does not move the figure)
            n_e2e = max(3, min(args.steps, 30 if ms / args.steps > 0.5 else 300))

            def e2e_step(i):
                wl = wls[i % len(wls)]
                mi, mb = mask_args[i % len(wls)]
                pie.pie_forward_host(ctx, wl.qo_indptr, wl.page_indptr, wl.page_indices, wl.last_page_len,
                                     hq, hk, hv, hout, hlse, mi, mb, args.flags)

            for i in range(3):
                e2e_step(i)
            env.barrier()
            t0 = time.perf_counter()
            for i in range(n_e2e):
                e2e_step(i)
            torch.cuda.synchronize()
            e2e_s = env.max_over_ranks(time.perf_counter() - t0)
            how = "the same batch every step; host planning of every step, pinned H2D of Q/K/V, forward, D2H of O/LSE"
        e2e = {"value": env.world * wl0.T * n_e2e / e2e_s, "unit": "tokens/s", "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": n_e2e, "ms_per_step": e2e_s / n_e2e * 1e3, "includes": how}

    total_tokens = env.world * wl0.T if env.world > 1 else wl0.T    # every rank runs a batch of the same shape
    for p in plans:
        pie.pie_plan_destroy(p)
    pie.pie_destroy(ctx)
    del q, k_new, v_new, out, lse
    torch.cuda.empty_cache()
    if env.rank != 0:
        return None

    peaks = load_peaks()
    ms_per_step = ms / args.steps
    roof = roofline_of(wl0, name, info, ktimes, ms_per_step, peaks, args.gpus, clocks, sum(regions) * 1e-3)
    cpu = None
    if env.world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline_of(wl0, cpu_budget_s)
    alg_bytes = wl0.algorithmic_bytes()
    return {
        "timed": True, "value": total_tokens / (ms_per_step * 1e-3), "unit": "tokens/s", "ms_per_step": ms_per_step,
        "ms_per_step_min": min(regions) / args.steps, "ms_per_step_max": max(regions) / args.steps,
        "regions": len(regions), "timed_seconds": sum(regions) * 1e-3, "dtype": wl0.dtype,
        "config": {"workload": name, "requests": wl0.R, "query_tokens": wl0.T, "heads": f"{wl0.H_q}/{wl0.H_kv}",
                   "head_dim": wl0.D, "page_size": wl0.P, "pool_pages": wl0.num_pages, "l2": l2_note,
                   "plan_flags": args.flags, "launch": "cuda graph replay" if use_graph else "eager"},
        "hbm_gbs_step": alg_bytes["total"] / (ms_per_step * 1e-3) / 1e9,
        "algorithmic_bytes_step": alg_bytes, "useful_flops_step": wl0.useful_flops(),
        "plan_ms": statistics.median(plan_ms), "plan_first_ms": plan_first_ms, "plan_info": info,
        "kernel_ms": {k: (v[0] / v[1] if v[1] else 0.0) for k, v in ktimes.items()},
        "roofline": roof, "cpu_baseline": cpu, "e2e": e2e,
        "gpu_launches": launches_per_step * args.steps * len(regions), "clocks": clocks,
    }


def bench_next_dist(env, args):
    """The sample stage next to the path (`get_next_dist`, Section 4.2 "Sample API"): one top-K truncated
    distribution per request of the batched-decode workload - 64 rows over the 128,256-entry Llama-3
    vocabulary, bf16 logits ~ N(0, 2.5) with a few tokens far ahead, K = 256.  Buffers rotate so that no
    logits survive in L2 between steps."""
    pie, torch = env.pie, env.torch
    n, V, K = 64, 128256, 256
    nbuf = 20                                                       # 20 x 16.4 MB > L2
    g = torch.Generator(device="cuda").manual_seed(0x50494500 + 99 + 1000 * env.rank)
    bufs = []
    for _ in range(nbuf):
        x = torch.randn(n, V, generator=g, device="cuda") * 2.5
        x[:, ::977] += 9.0
        bufs.append(x.to(torch.bfloat16))
    ctx = pie.pie_create(4, 16, 4, 2, 64, "bf16", 4, 64, env.local)
    ids = torch.empty(n, K, dtype=torch.int32, device="cuda")
    probs = torch.empty(n, K, dtype=torch.float32, device="cuda")

    def eager_step(i):
        pie.pie_get_next_dist(ctx, bufs[i % nbuf], K, ids, probs)

    # The kernel takes about as long as one launch through the Python binding costs on the host, so the timed
    # region replays ONE captured graph that holds its `--steps` launches (the call only enqueues a kernel on
    # the caller's stream): the region is then device time, as for the attention workloads.
    for i in range(max(args.warmup, 3)):
        eager_step(i)
    cap = torch.cuda.Stream()
    cap.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(cap):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=cap):
            for i in range(args.steps):
                eager_step(i)
    torch.cuda.current_stream().wait_stream(cap)

    def step(i):
        if i % args.steps == 0:
            graph.replay()

    for i in range(3):
        step(0)
    env.barrier()
    sampler = ClockSampler(env.local)
    if env.rank == 0:
        sampler.start()
    regions = timed_regions(env, step, args.steps, args.min_seconds)
    clocks = sampler.stop() if env.rank == 0 else None
    ms = statistics.median(regions)
    e2e = None
    if not args.no_e2e:
        host = [b.cpu().pin_memory() for b in bufs[:4]]
        dev = torch.empty_like(bufs[0])
        h_ids, h_probs = torch.empty(n, K, dtype=torch.int32).pin_memory(), torch.empty(n, K).pin_memory()
        n_e2e = max(3, min(args.steps, 30))

        def e2e_step(i):
            dev.copy_(host[i % 4], non_blocking=True)
            pie.pie_get_next_dist(ctx, dev, K, ids, probs)
            h_ids.copy_(ids, non_blocking=True)
            h_probs.copy_(probs, non_blocking=True)
            torch.cuda.synchronize()

        for i in range(3):
            e2e_step(i)
        env.barrier()
        t0 = time.perf_counter()
        for i in range(n_e2e):
            e2e_step(i)
        e2e_s = env.max_over_ranks(time.perf_counter() - t0)
        e2e = {"value": env.world * n * n_e2e / e2e_s, "unit": "tokens/s", "h2d_bytes_per_step": n * V * 2,
               "d2h_bytes_per_step": n * K * 8, "steps": n_e2e, "ms_per_step": e2e_s / n_e2e * 1e3,
               "includes": "pinned H2D of the logits, get_next_dist, D2H of ids and probabilities"}
    cpu = None
    if env.rank == 0 and env.world == 1 and not args.no_cpu_baseline:
        from oracle import pie_oracle as orc
        rows = bufs[0][:8].cpu().view(torch.int16).numpy().view(np.uint16)
        t0 = time.perf_counter()
        orc.next_dist(rows, K)
        dt = time.perf_counter() - t0
        cpu = {"value": len(rows) / dt, "unit": "tokens/s", "cores": 1, "kind": "oracle",
               "sample": f"first {len(rows)} of {n} rows", "seconds": dt}
    pie.pie_destroy(ctx)
    del bufs
    torch.cuda.empty_cache()
    if env.rank != 0:
        return None
    ms_per_step = ms / args.steps
    alg = n * V * 2 + n * K * 8
    peaks = load_peaks()
    achieved = alg / (ms_per_step * 1e-3) / 1e9
    return {
        "timed": True, "value": env.world * n / (ms_per_step * 1e-3), "unit": "tokens/s", "ms_per_step": ms_per_step,
        "ms_per_step_min": min(regions) / args.steps, "ms_per_step_max": max(regions) / args.steps,
        "regions": len(regions), "timed_seconds": sum(regions) * 1e-3, "dtype": "bf16",
        "config": {"workload": "next_dist", "rows": n, "vocab": V, "top_k": K,
                   "l2": f"{nbuf} rotating logit buffers ({nbuf * n * V * 2 / 1e6:.0f} MB) > L2",
                   "launch": "one captured graph of --steps launches per timed region"},
        "hbm_gbs_step": achieved, "algorithmic_bytes_step": {"logits": n * V * 2, "out": n * K * 8, "total": alg},
        "kernel_ms": {"next_dist": ms_per_step},
        "roofline": {"bound": "hbm", "kernel": "next_dist", "achieved": achieved, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC["next_dist"][0],
                     "traffic_source": NCU_TRAFFIC["next_dist"][1],
                     "algorithmic_bytes": alg, "kernel_ms": ms_per_step, "timing": "timed region / launches",
                     "peak_source": peaks["source"]},
        "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": args.steps * len(regions) * args.nd_launches, "clocks": clocks,
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="all",
                    help="one workload by name, or 'all' (default): every baseline configuration in one run")
    ap.add_argument("--min-seconds", type=float, default=0.5, help="device time to collect per workload (regions of --steps steps are repeated)")
    ap.add_argument("--flags", type=int, default=0, help="PIE_PLAN_* flags (debug / A-B runs)")
    ap.add_argument("--opt", action="append", default=[], help="pie_set_option as K=V (tuning runs)")
    ap.add_argument("--graph", type=int, default=0,
                    help="1: replay one captured CUDA graph per step (measured: no gain, the loop is GPU bound), 0: eager launches")
    ap.add_argument("--param", action="append", default=[], help="builder argument of the workload as key=value (shape sweeps)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    args.nd_launches = 1
    if args.impl == "reference":
        return run_reference(args)

    env = Env()
    # N > 1: every rank runs the headline batch (weak scaling); the other entries are single-GPU figures
    names = (SUITE if env.world == 1 else [HEADLINE]) if args.workload == "all" else [args.workload]
    entries = {}
    t_start = time.perf_counter()
    device = env.device_info()
    for name in names:
        t0 = time.perf_counter()
        head = name == names[0]
        if name == "next_dist":
            entry = bench_next_dist(env, args)
        else:
            entry = bench_workload(env, args, name, cpu_budget_s=15.0 if head else 4.0)
        if entry is not None:
            entry["wall_seconds"] = time.perf_counter() - t0
            entries[name] = entry
    if env.rank == 0:
        head = entries[names[0]]
        line = {"metric": METRIC, "value": head["value"], "unit": "tokens/s", "n_gpus": env.world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": head["dtype"], "data": "synthetic"}
        for k in ("config", "hbm_gbs_step", "algorithmic_bytes_step", "useful_flops_step", "plan_ms", "plan_first_ms",
                  "plan_info", "kernel_ms", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks", "regions",
                  "timed_seconds", "ms_per_step_min", "ms_per_step_max"):
            if k in head:
                line[k] = head[k]
        if "shared_prefix_tree" in entries:
            line["roofline_tensor"] = dict(entries["shared_prefix_tree"]["roofline"], workload="shared_prefix_tree")
        if args.workload == "all":
            if env.world == 1:
                entries["tiny_fp32"] = {"timed": False, "note": "correctness-only configuration (fp32, 4 requests): covered by the parity tests"}
            line["workloads"] = entries
        line["device"] = device
        line["wall_seconds"] = time.perf_counter() - t_start
        print(json.dumps(line))
    env.close()


if __name__ == "__main__":
    main()
