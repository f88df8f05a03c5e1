#!/usr/bin/env python
"""Benchmark of the prioritized-replay hot path: one step = sample (indices, IS weights, gather) +
priority update + insert (pearl_prb_update_insert) on one batch of synthetic transitions.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is sampled-and-updated transitions per second through
the whole step with all inputs resident in device memory; `e2e` is the same through the
host-buffer calls (host->device and device->host copies inside the timed region); `roofline`
is the achieved fraction of the measured HBM copy bandwidth of the sample+gather kernel;
`cpu_baseline` is the CPU oracle timed on this machine's host cores on a bounded sample.
With N > 1 every rank runs an independent replica (the buffer does not shard); time is the
maximum over ranks.  `--impl reference` times the CPU oracle instead of the CUDA library.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "PRB sample+update transitions/s at batch B"
UNIT = "transitions/s"
ROTATE = 8           # distinct input/output batch buffers cycled through, so inputs exceed L2 where rows are long
FALLBACK_HBM_GBS = 6650.0
SHORT_REGION_MS = 50.0     # a timed region shorter than this is repeated and the median taken
REGION_REPS = 5


def load_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------------------------------
# CPU oracle arm (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------
def host_available_bytes():
    """Host memory that can still be had (MemAvailable), or a cautious guess."""
    try:
        with open("/proc/meminfo") as f:
            for ln in f:
                if ln.startswith("MemAvailable:"):
                    return int(ln.split()[1]) * 1024
    except Exception:
        pass
    return 8 << 30


def oracle_capacity(wl):
    """Capacity the oracle is timed at: the workload's where its store fits in 60 % of the host memory
    still available (the oracle keeps the whole Data Storage), else the largest power-of-two part that does."""
    room = int(host_available_bytes() * 0.6)
    cap = wl.capacity
    while cap > 1024 and cap * (wl.transition_bytes + 64) > room:
        cap //= 2
    return cap


def oracle_setup(wl, capacity):
    import oracle
    from paper_2311_09445_b200 import workloads as wk
    oracle.build()
    rng = np.random.default_rng(wl.seed)
    o = oracle.OraclePRB(capacity, wl.fanout, wl.obs_bytes, wl.act_bytes)
    plain = wk.scaled(wl, capacity, counter_rows=False)      # same shapes; bytes from numpy (content is irrelevant to time)
    chunk = max(1, min(capacity, (64 << 20) // wl.transition_bytes))
    # one chunk of rows serves the whole prefill (only the priorities are fresh): filling 30 GB with fresh
    # random bytes would take longer than the measurement
    rows = wk.transitions(plain, rng, chunk)
    for first in range(0, capacity, chunk):
        n = min(chunk, capacity - first)
        prio = wk.priorities(plain, rng, n)
        o.insert(rows["obs"][:n], rows["act"][:n], rows["rew"][:n], rows["next_obs"][:n], rows["done"][:n], prio)
    batches = [wk.transitions(plain, rng, max(wl.n_insert, 1)) for _ in range(ROTATE)]
    tds = [wk.td_errors(wl, rng, wl.batch) for _ in range(ROTATE)]
    return o, plain, batches, tds, rng


def oracle_step(o, wl, batches, tds, rng, i):
    from paper_2311_09445_b200 import workloads as wk
    if wl.n_insert:
        b = batches[i % ROTATE]
        o.insert(b["obs"], b["act"], b["rew"], b["next_obs"], b["done"], b["prio"])
    out = o.sample(wl.batch, wl.beta, wl.philox_seed)
    idx = out["idx"]
    if wl.dup_frac:
        idx, _ = wk.update_batch(wl, rng, idx)
    o.update(idx, tds[i % ROTATE], wl.alpha, wl.eps)


def time_oracle(wl, steps, warmup, budget_s=None):
    cap = oracle_capacity(wl)
    o, plain, batches, tds, rng = oracle_setup(wl, cap)
    for i in range(warmup):
        oracle_step(o, wl, batches, tds, rng, i)
    t0 = time.perf_counter()
    done = 0
    for i in range(steps):
        oracle_step(o, wl, batches, tds, rng, i)
        done += 1
        if budget_s is not None and time.perf_counter() - t0 > budget_s:
            break
    dt = time.perf_counter() - t0
    o.close()
    sample = "%d steps of the %s step (insert %d, sample %d, update %d)" % (done, wl.name, wl.n_insert, wl.batch, wl.batch)
    if cap != wl.capacity:
        sample += " at capacity %d of %d (host memory)" % (cap, wl.capacity)
    return done, dt, sample, cap


# ------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index, self.proc = gpu_index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.QUERY,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, watts, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            p = [t.strip() for t in line.split(",")]
            if len(p) < 9:
                continue
            try:
                sm.append(float(p[1])); mx.append(float(p[2]))
            except ValueError:
                continue
            try:
                watts.append(float(p[3]))
            except ValueError:
                pass
            for name, v in zip(names, p[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons),
                # board power while the timed region ran: context for the paper's per-watt figures (Section VI), no more
                "power_w": statistics.median(watts) if watts else None}


# ------------------------------------------------------------------------------------------
# CUDA arm
# ------------------------------------------------------------------------------------------
def device_batches(wl, rng, dev, n, count, first_id):
    """`count` insert batches of n transitions resident on the device."""
    import torch
    from paper_2311_09445_b200 import workloads as wk
    out = []
    for r in range(count):
        if wl.counter_rows:
            small = wk.transitions(wl, rng, n, with_obs=False)
            ids = torch.arange(first_id + r * n, first_id + (r + 1) * n, dtype=torch.int64, device=dev)
            if wl.frame_stack:
                # one frame per slot; an episode start (marker, bit 1 of done) every couple of hundred slots
                d = {"obs": wk.counter_row_bytes(ids, 0, wl.obs_bytes // wl.frame_stack), "next_obs": None}
                small["done"] = np.where(rng.random(n) < 0.005, 2, small["done"] & 1).astype(np.uint8)
            else:
                d = {"obs": wk.counter_row_bytes(ids, 0, wl.obs_bytes), "next_obs": wk.counter_row_bytes(ids, 1, wl.obs_bytes)}
            for k in ("act", "rew", "done", "prio"):
                d[k] = torch.from_numpy(small[k]).to(dev)
        else:
            d = wk.to_device(wk.transitions(wl, rng, n), dev)
        out.append(d)
    return out


def out_buffers(wl, dev, B, pinned=False):
    import torch
    kw = dict(device="cpu", pin_memory=True) if pinned else dict(device=dev)
    return {"idx": torch.zeros(B, dtype=torch.int32, **kw), "w": torch.zeros(B, dtype=torch.float32, **kw),
            "obs": torch.zeros((B, wl.obs_bytes), dtype=torch.uint8, **kw),
            "act": torch.zeros((B, max(wl.act_bytes, 1)), dtype=torch.uint8, **kw),
            "rew": torch.zeros(B, dtype=torch.float32, **kw),
            "next_obs": torch.zeros((B, wl.obs_bytes), dtype=torch.uint8, **kw),
            "done": torch.zeros(B, dtype=torch.uint8, **kw)}


def max_over_ranks(value, device):
    """The maximum of `value` over all ranks of the default process group (every rank gets it)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def time_loop(stream, fn, iters):
    """Milliseconds for `iters` calls of fn(i), CUDA events on `stream`, synchronised on both sides."""
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for i in range(iters):
        fn(i)
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def copy_context(wl, store_rows, dev, stream):
    """Library kernels on the same bytes, for context only (they are not on the product path): a dense
    torch copy of one batch of observation rows, and torch.index_select of B random rows with the
    indices already known.  Microseconds per batch, graphs of ROTATE calls like the per-call timings."""
    import torch
    B, W = wl.batch, wl.obs_bytes
    free, _ = torch.cuda.mem_get_info(dev)
    rows = store_rows if 2 * store_rows * W + (4 << 30) < free + torch.cuda.memory_reserved(dev) else min(store_rows, 1 << 16)
    with torch.cuda.stream(stream):
        store = torch.empty((2, rows, W), dtype=torch.uint8, device=dev).random_(0, 255)
        outs = [torch.empty((2, B, W), dtype=torch.uint8, device=dev) for _ in range(ROTATE)]
        srcs = [torch.empty((2, B, W), dtype=torch.uint8, device=dev).random_(0, 255) for _ in range(ROTATE)]
        idxs = [torch.sort(torch.randint(0, rows, (B,), device=dev))[0] for _ in range(ROTATE)]

        def timed(fn):
            for r in range(ROTATE):
                fn(r)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for r in range(ROTATE):
                    fn(r)
            g.replay()
            return time_loop(stream, lambda i: g.replay(), 25) * 1e3 / (25 * ROTATE)

        def gather(r):
            torch.index_select(store[0], 0, idxs[r], out=outs[r][0])
            torch.index_select(store[1], 0, idxs[r], out=outs[r][1])

        us_copy = timed(lambda r: outs[r].copy_(srcs[r]))
        us_gather = timed(gather)
    nbytes = 4 * B * W
    return {"bytes": nbytes, "torch_dense_copy_us": us_copy, "torch_dense_copy_gbs": nbytes / us_copy / 1e3,
            "torch_index_select_us": us_gather, "torch_index_select_gbs": nbytes / us_gather / 1e3,
            "store_rows": rows,
            "note": "library kernels on the same observation bytes (read+write), indices given; context, not the product path"}


def timed_regions(stream, run_steps, steps, world, dev):
    """Times run_steps(steps) with CUDA events on `stream`, barrier + synchronise on both sides, maximum
    over ranks.  A region shorter than SHORT_REGION_MS is run REGION_REPS times and all times returned
    (the caller takes the median): a sub-millisecond region is at the mercy of one hiccup."""
    import torch.distributed as dist
    times = []
    for rep in range(REGION_REPS):
        if world > 1:
            dist.barrier()
        ms = time_loop(stream, lambda i: run_steps(steps), 1)
        if world > 1:
            dist.barrier()
            ms = max_over_ranks(ms, dev)
        times.append(ms)
        if ms >= SHORT_REGION_MS:
            break
    return times


def measure_workload(wl, steps, warmup, dev, stream, rank=0, world=1, extras=True, e2e=True, use_graph=True, fused=True,
                     min_tree=False):
    """Builds and fills one buffer for workload `wl` and times the step, its calls and the host-buffer step.
    Returns a dict of raw measurements (milliseconds per step / per call)."""
    import torch
    from paper_2311_09445_b200 import PrioritizedReplay
    from paper_2311_09445_b200 import workloads as wk

    rng = np.random.default_rng(wl.seed + 7919 * rank)
    B, n_ins = wl.batch, wl.n_insert
    chunk = 512 if wl.counter_rows else min(wl.capacity, 1 << 16)
    max_batch = max(B, n_ins, chunk)
    m = {}
    with torch.cuda.stream(stream):
        prb = PrioritizedReplay(wl.capacity, wl.fanout, wl.obs_bytes, wl.act_bytes, max_batch, device=dev, stream=stream,
                                frame_stack=wl.frame_stack, min_tree=min_tree)
        # prefill the whole ring through the insert call
        filled = 0
        while filled < wl.capacity:
            n = min(chunk, wl.capacity - filled)
            b = device_batches(wl, rng, dev, n, 1, filled)[0]
            prb.insert(b["obs"], b["act"], b["rew"], b["next_obs"], b["done"], b["prio"])
            filled += n
        torch.cuda.synchronize()
        batches = device_batches(wl, rng, dev, max(n_ins, 1), ROTATE, wl.capacity)
        outs = [out_buffers(wl, dev, B) for _ in range(ROTATE)]
        tds = [torch.from_numpy(wk.td_errors(wl, rng, B)).to(dev) for _ in range(ROTATE)]
        # A workload whose recipe plants duplicates in the update's indices gets its index batches made
        # here, before the timed region, from real sampled batches (so that no library kernel runs
        # inside a timed step); the others update exactly what the step's sample returned.
        n_dup = int(round(wl.dup_frac * B))
        upd_idx = None
        if n_dup:
            upd_idx = []
            for r in range(ROTATE):
                o = outs[r]
                prb.sample(B, wl.beta, wl.philox_seed, o["idx"], o["w"], o["obs"], o["act"] if wl.act_bytes else None,
                           o["rew"], o["next_obs"], o["done"])
                idx = o["idx"].clone()
                pos = torch.from_numpy(rng.choice(B, size=n_dup, replace=False)).to(dev)
                src = torch.from_numpy(rng.integers(0, B, size=n_dup)).to(dev)
                idx[pos] = o["idx"][src]
                upd_idx.append(idx)

        def do_insert(i):
            b = batches[i % ROTATE]
            prb.insert(b["obs"], b["act"], b["rew"], b["next_obs"], b["done"], b["prio"])

        def sample_args(i):
            o = outs[i % ROTATE]
            return (o["idx"], o["w"], o["obs"], o["act"] if wl.act_bytes else None, o["rew"], o["next_obs"], o["done"])

        def do_sample(i):
            prb.sample(B, wl.beta, wl.philox_seed, *sample_args(i))

        def do_update(i):
            idx = upd_idx[i % ROTATE] if upd_idx else outs[i % ROTATE]["idx"]
            prb.update(idx, tds[i % ROTATE], wl.alpha, wl.eps)

        def do_update_insert(i):
            b = batches[i % ROTATE]
            idx = upd_idx[i % ROTATE] if upd_idx else outs[i % ROTATE]["idx"]
            prb.update_insert(idx, tds[i % ROTATE], wl.alpha, wl.eps, b["obs"], b["act"], b["rew"], b["next_obs"],
                              b["done"], b["prio"])

        fused = bool(n_ins) and fused

        def eager_step(i):
            # the paper's schedule (Eq. 7): sample, then update with the insertion running beside it
            do_sample(i)
            if fused:
                do_update_insert(i)
            else:
                do_update(i)
                if n_ins:
                    do_insert(i)

        for i in range(max(warmup, 3)):
            eager_step(i)
        torch.cuda.synchronize()
        status = prb.sync()

        # CUDA graphs (all buffer state lives on the device, so replays advance it): one graph of
        # ROTATE consecutive steps, plus one graph of the remaining K mod ROTATE steps
        l0 = prb.kernel_launches()
        eager_step(0)
        m["kernels_per_step_eager"] = prb.kernel_launches() - l0
        torch.cuda.synchronize()

        def capture(calls):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for c in calls:
                    c()
            return g

        if use_graph:
            l0 = prb.kernel_launches()
            g_all = capture([lambda r=r: eager_step(r) for r in range(ROTATE)])
            m["kernels_per_step"] = (prb.kernel_launches() - l0) / ROTATE
            g_rest = {}          # remainder -> a graph of that many consecutive steps

            def run_steps(k):
                rest = k % ROTATE
                if rest and rest not in g_rest:
                    g_rest[rest] = capture([lambda r=r: eager_step(r) for r in range(rest)])
                for _ in range(k // ROTATE):
                    g_all.replay()
                if rest:
                    g_rest[rest].replay()
        else:
            m["kernels_per_step"] = m["kernels_per_step_eager"]

            def run_steps(k):
                for i in range(k):
                    eager_step(i)
        run_steps(max(warmup, 3))
        if steps % ROTATE:
            run_steps(steps % ROTATE)        # (more warm-up: the remainder's graph is captured here, not in the timed region)
        torch.cuda.synchronize()

        # ---- the timed region: exactly K steps (repeated, median, when it is short) ----------
        clocks = ClockSampler(dev.index or 0)
        if rank == 0:
            clocks.start()
            time.sleep(0.3)
        m["region_ms"] = timed_regions(stream, run_steps, steps, world, dev)
        m["clocks"] = clocks.stop() if rank == 0 else None

        # ---- per-call timings (device resident), used for the roofline and the rates: a graph of
        # ROTATE back-to-back calls of one kind, replayed, so that host launch cost is not in them
        reps = max(3, min(steps, 400) // ROTATE)

        def per_call_ms(fn):
            if not use_graph:
                for i in range(3):
                    fn(i)
                return time_loop(stream, fn, reps * ROTATE) / (reps * ROTATE)
            g = capture([lambda r=r: fn(r) for r in range(ROTATE)])
            g.replay()
            return statistics.median(time_loop(stream, lambda i: g.replay(), reps) / (reps * ROTATE) for _ in range(3))

        m["ms_sample"] = per_call_ms(do_sample)
        m["ms_update"] = per_call_ms(do_update)
        m["ms_insert"] = per_call_ms(do_insert) if n_ins else None
        m["ms_update_insert"] = per_call_ms(do_update_insert) if fused else None
        if extras:
            # the same update with its index batch in random order (the kernel has to sort it)
            shuffled = [(upd_idx[r] if upd_idx else outs[r]["idx"])[torch.randperm(B, device=dev)] for r in range(ROTATE)]
            m["ms_update_shuffled"] = per_call_ms(lambda i: prb.update(shuffled[i % ROTATE], tds[i % ROTATE], wl.alpha, wl.eps))
            # the sample as one kernel, whatever the call before it (the form a sample takes outside a stream
            # capture and right after an update + insertion), through the call that always takes that form
            if B <= 4096:
                m["ms_sample_one_kernel"] = per_call_ms(lambda i: prb.sample_static_scratch(B, wl.beta, wl.philox_seed, *sample_args(i)))
            # the sample issued as 4 sub-batches on 4 streams of the handle (whole call, all joined)
            if B >= 4:
                m["ms_sample_streamed4"] = per_call_ms(lambda i: prb.sample_streamed(B, wl.beta, wl.philox_seed, 4, *sample_args(i)))
            # the sample with weights normalised over the whole buffer
            m["ms_sample_buffer_norm"] = per_call_ms(lambda i: prb.sample_buffer_norm(B, wl.beta, wl.philox_seed, *sample_args(i)))
        status |= prb.sync()

        # ---- end to end through the host-buffer calls ----------------------------------------
        if e2e:
            e2e_steps = max(5, min(steps, 100 if wl.counter_rows else 500))
            hb = [{k: (v.cpu().pin_memory() if v is not None else None) for k, v in batches[r].items()} for r in range(ROTATE)]
            ho = out_buffers(wl, dev, B, pinned=True)
            htd = [t.cpu().pin_memory() for t in tds]

            prb.sample_host(B, wl.beta, wl.philox_seed, ho["idx"], ho["w"], ho["obs"], ho["act"] if wl.act_bytes else None,
                            ho["rew"], ho["next_obs"], ho["done"])

            def e2e_step(i):
                # one iteration through host buffers: the update for the batch sampled last, the new rows, the next batch
                b = hb[i % ROTATE] if n_ins else dict.fromkeys(("obs", "act", "rew", "next_obs", "done", "prio"))
                prb.step_host(ho["idx"], htd[i % ROTATE], wl.alpha, wl.eps, b["obs"], b["act"], b["rew"], b["next_obs"], b["done"],
                              b["prio"], B, wl.beta, wl.philox_seed, ho["idx"], ho["w"], ho["obs"], ho["act"] if wl.act_bytes else None,
                              ho["rew"], ho["next_obs"], ho["done"], n=n_ins)

            for i in range(3):
                e2e_step(i)
            import torch.distributed as dist
            if world > 1:
                dist.barrier()
            ms_e2e = time_loop(stream, e2e_step, e2e_steps)
            if world > 1:
                dist.barrier()
                ms_e2e = max_over_ranks(ms_e2e, dev)
            m["ms_e2e_step"] = ms_e2e / e2e_steps
            m["e2e_steps"] = e2e_steps
            status |= prb.sync()
        m["status"] = status
        m["depth"] = prb.info()[3]
        prb.close()
    return m


def summary_of(wl, m, world=1):
    """One workload's figures: step time, samples/s, updates/s, inserts/s, and the same step through host buffers."""
    B, n_ins = wl.batch, wl.n_insert
    ms_step = statistics.median(m["region_ms"]) / m["steps"]
    out = {"us_step": ms_step * 1e3, "transitions_per_s": world * B / (ms_step * 1e-3),
           "samples_per_s": B / (m["ms_sample"] * 1e-3), "updates_per_s": B / (m["ms_update"] * 1e-3),
           "inserts_per_s": (n_ins / (m["ms_insert"] * 1e-3)) if m.get("ms_insert") else None,
           "us_sample": m["ms_sample"] * 1e3, "us_update": m["ms_update"] * 1e3,
           "us_insert": m["ms_insert"] * 1e3 if m.get("ms_insert") else None,
           "us_update_insert": m["ms_update_insert"] * 1e3 if m.get("ms_update_insert") else None}
    if "ms_e2e_step" in m:
        out["e2e_transitions_per_s"] = world * B / (m["ms_e2e_step"] * 1e-3)
    return out


def run_ours(args, wl, rank, world):
    import torch
    import torch.distributed as dist

    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dev = torch.device("cuda:%d" % local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    stream = torch.cuda.Stream(dev)
    B, n_ins = wl.batch, wl.n_insert
    fused = bool(n_ins) and not args.unfused
    m = measure_workload(wl, args.steps, args.warmup, dev, stream, rank, world, extras=not args.profile,
                         e2e=not args.profile, use_graph=not args.no_graph, fused=fused, min_tree=args.min_tree)
    m["steps"] = args.steps
    ctx = None
    others = None
    if rank == 0 and world == 1 and not args.profile:
        if wl.obs_bytes >= 8192:
            with torch.cuda.stream(stream):
                ctx = copy_context(wl, wl.capacity, dev, stream)
        others = other_workloads(wl, dev, stream)
    if world > 1:
        dist.destroy_process_group()
    if rank != 0:
        return None

    E = wl.transition_bytes
    depth = m["depth"]
    ms = statistics.median(m["region_ms"])
    h2d = (n_ins * (E + 4) if n_ins else 0) + B * 8
    d2h = B * (2 * wl.obs_bytes + wl.act_bytes + 5 + 8)
    peak, peak_kind = load_peak()
    # algorithmic bytes of one sample call: D child groups of K binary32 per stratum, index and
    # weight written, every field of the row read once and written once
    sample_bytes = B * (depth * wl.fanout * 4 + 8 + wl.sample_bytes)
    long_rows = wl.obs_bytes >= 8192 and wl.obs_bytes % 16 == 0 and not wl.frame_stack
    achieved = sample_bytes / (m["ms_sample"] * 1e-3) / 1e9
    rates = summary_of(wl, m, world)
    for k in ("ms_update_shuffled", "ms_sample_one_kernel", "ms_sample_streamed4", "ms_sample_buffer_norm"):
        rates["us" + k[2:]] = m[k] * 1e3 if m.get(k) else None
    line = {
        "metric": METRIC, "value": world * B * args.steps / (ms * 1e-3), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32 tree / f64 targets / u8 rows", "data": "synthetic",
        "config": {"workload": wl.name, "capacity": wl.capacity, "fanout": wl.fanout, "depth": depth, "batch": B,
                   "insert_per_step": n_ins, "transition_bytes": E, "step": "sample(idx,IS,gather) + update_insert" if fused else "sample(idx,IS,gather) + update + insert",
                   "parallelism": "replicas x%d" % world, "cuda_graph": not args.no_graph, "min_tree": bool(args.min_tree),
                   "l2": "inputs/outputs rotate over %d buffers (%d MB per step touched)" % (ROTATE, (2 * (n_ins + B) * E) >> 20)},
        "timed_region": {"repeats": len(m["region_ms"]), "ms_each": m["region_ms"],
                         "value_from": "median" if len(m["region_ms"]) > 1 else "the one region"},
        "rates": rates,
        "roofline": {"kernel": "prb_gather_rows_kernel (+ prb_descend_kernel beside the copy before it)" if long_rows and not args.no_graph
                     else "prb_sample_kernel",
                     "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": "%s copy bandwidth" % peak_kind,
                     "frac_of_8TBs_nominal": achieved / 8000.0, "bytes_per_launch": sample_bytes,
                     "timing": "captured graph of %d consecutive sample calls, replayed; per call" % ROTATE,
                     "traffic": None,
                     "traffic_note": "dram bytes of one launch are in profiles/ (ncu, reduced capacity); not measured in this run"},
        "gpu_launches": int(round(m["kernels_per_step"] * args.steps)),
        "kernels_per_step": m["kernels_per_step"],
        "status_bits": int(m["status"]),
        "clocks": m["clocks"],
    }
    if "ms_e2e_step" in m:
        line["e2e"] = {"value": world * B / (m["ms_e2e_step"] * 1e-3), "unit": UNIT, "steps": m["e2e_steps"],
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
    else:
        line["e2e"] = {"value": None, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
    step_bytes = sample_bytes + (n_ins * (2 * E + 4) if n_ins else 0)
    line["roofline_step"] = {"bound": "hbm", "bytes_per_step": step_bytes, "achieved": step_bytes / (ms / args.steps * 1e-3) / 1e9,
                             "peak": peak, "unit": "GB/s", "frac": step_bytes / (ms / args.steps * 1e-3) / 1e9 / peak}
    if n_ins:
        ins_bytes = n_ins * (2 * E + 4)
        line["roofline_insert"] = {"kernel": "prb_insert_rows_kernel" if long_rows else "prb_insert_kernel", "bound": "hbm",
                                   "bytes_per_launch": ins_bytes,
                                   "achieved": ins_bytes / (m["ms_insert"] * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                                   "frac": ins_bytes / (m["ms_insert"] * 1e-3) / 1e9 / peak}
    if ctx is not None:
        line["roofline"]["context"] = ctx
    if others is not None:
        line["workloads"] = others
    if world == 1 and not args.profile:
        done, dt, sample, cap = time_oracle(wl, 10 ** 9, 2, budget_s=args.cpu_budget)
        line["cpu_baseline"] = {"value": B * done / dt, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
                                "capacity": cap, "host_cpus": os.cpu_count()}
    return line


# the paper's other workloads (Table III shapes), and three cells of the scaling sweep: short runs after the headline's
OTHER_SWEEP_CELLS = [(1 << 20, 16, 1024), (1 << 22, 32, 4096), (1 << 24, 4, 65536)]


def other_workloads(headline, dev, stream):
    import torch
    from paper_2311_09445_b200 import workloads as wk
    out = {}
    todo = [w for name, w in wk.WORKLOADS.items() if name != headline.name]
    todo += [wk.sweep_cell(n, k, b, cell_id=n % 997 + k + b) for n, k, b in OTHER_SWEEP_CELLS]
    for wl in todo:
        free, _ = torch.cuda.mem_get_info(dev)
        if wl.capacity * wl.transition_bytes + (4 << 30) > free + torch.cuda.memory_reserved(dev):
            out[wl.name] = {"skipped": "not enough free device memory"}
            continue
        steps = 200
        m = measure_workload(wl, steps, 3, dev, stream, extras=False, e2e=wl.capacity <= (1 << 20) or wl.frame_stack > 0)
        m["steps"] = steps
        d = summary_of(wl, m)
        d.update(capacity=wl.capacity, fanout=wl.fanout, batch=wl.batch, insert_per_step=wl.n_insert, steps=steps,
                 stored_bytes_per_transition=wl.transition_bytes, gather_bytes_per_sample=wl.sample_bytes,
                 gather_gbs=wl.batch * wl.sample_bytes / (m["ms_sample"] * 1e-3) / 1e9,
                 region_repeats=len(m["region_ms"]), status_bits=int(m["status"]))
        out[wl.name] = d
        torch.cuda.empty_cache()
    return out


# ------------------------------------------------------------------------------------------
# Scaling sweep (capacity x fanout x batch): per-call times of every cell, one process
# ------------------------------------------------------------------------------------------
SWEEP_CAPACITIES = [1 << 16, 1 << 18, 1 << 20, 1 << 22, 1 << 24, 1 << 26]
SWEEP_FANOUTS = [2, 4, 16, 32]
SWEEP_BATCHES = [32, 256, 1024, 4096, 16384, 65536]


def run_sweep(args):
    """Times sample, update, insert and the step (sample + update_insert) on every cell of the scaling
    sweep: 165-byte transitions, LogNormal(0, 2) priorities, 1024 insertions per step.  A buffer is
    created and filled once per (capacity, fanout) and serves all its batch sizes; every timing is a
    captured graph of ROTATE consecutive calls, replayed.  Prints one JSON line with a row per cell."""
    import torch
    from paper_2311_09445_b200 import PrioritizedReplay
    from paper_2311_09445_b200 import workloads as wk

    torch.cuda.set_device(0)
    dev = torch.device("cuda:0")
    stream = torch.cuda.Stream(dev)
    caps = [c for c in SWEEP_CAPACITIES if not args.capacity or c == args.capacity]
    fanouts = [k for k in SWEEP_FANOUTS if not args.sweep_fanout or k == args.sweep_fanout]
    gen = torch.Generator(device=dev)
    rows = []
    clocks = ClockSampler(0)
    clocks.start()
    t_start = time.time()
    with torch.cuda.stream(stream):
        for N in caps:
            for K in fanouts:
                wl = wk.sweep_cell(N, K, 1024, cell_id=0)
                gen.manual_seed(wl.seed + N % 997 + K)
                batches_B = [b for b in SWEEP_BATCHES if b <= N // 2 and (not args.sweep_batch or b == args.sweep_batch)]
                if not batches_B:
                    continue
                chunk = min(N, 1 << 16)
                prb = PrioritizedReplay(N, K, wl.obs_bytes, wl.act_bytes, max(chunk, max(batches_B)), device=dev, stream=stream)

                def lognormal_prio(n):
                    d = torch.exp(2.0 * torch.randn(n, generator=gen, device=dev, dtype=torch.float64))
                    return ((d + 1e-6) ** 0.6).to(torch.float32)

                def make_batch(n):
                    return {"obs": torch.randn((n, wl.obs_bytes // 4), generator=gen, device=dev).view(torch.uint8),
                            "next_obs": torch.randn((n, wl.obs_bytes // 4), generator=gen, device=dev).view(torch.uint8),
                            "act": (torch.rand((n, wl.act_bytes // 4), generator=gen, device=dev) * 2 - 1).view(torch.uint8),
                            "rew": torch.randn(n, generator=gen, device=dev),
                            "done": (torch.rand(n, generator=gen, device=dev) < 0.05).to(torch.uint8)}

                rowsrc = make_batch(chunk)       # the same rows for every prefill chunk, fresh priorities
                for first in range(0, N, chunk):
                    prb.insert(rowsrc["obs"], rowsrc["act"], rowsrc["rew"], rowsrc["next_obs"], rowsrc["done"], lognormal_prio(chunk))
                ins = []
                for r in range(ROTATE):
                    b = make_batch(wl.n_insert)
                    b["prio"] = lognormal_prio(wl.n_insert)
                    ins.append(b)
                for B in batches_B:
                    cw = wk.sweep_cell(N, K, B)
                    outs = [out_buffers(cw, dev, B) for _ in range(ROTATE)]
                    tds = [torch.exp(2.0 * torch.randn(B, generator=gen, device=dev)) for _ in range(ROTATE)]

                    def do_sample(i):
                        o = outs[i % ROTATE]
                        prb.sample(B, cw.beta, cw.philox_seed, o["idx"], o["w"], o["obs"], o["act"], o["rew"], o["next_obs"], o["done"])

                    def do_update(i):
                        prb.update(outs[i % ROTATE]["idx"], tds[i % ROTATE], cw.alpha, cw.eps)

                    def do_insert(i):
                        b = ins[i % ROTATE]
                        prb.insert(b["obs"], b["act"], b["rew"], b["next_obs"], b["done"], b["prio"])

                    def do_update_insert(i):
                        b = ins[i % ROTATE]
                        prb.update_insert(outs[i % ROTATE]["idx"], tds[i % ROTATE], cw.alpha, cw.eps, b["obs"], b["act"], b["rew"],
                                          b["next_obs"], b["done"], b["prio"])

                    def do_step(i):
                        do_sample(i)
                        do_update_insert(i)

                    for i in range(ROTATE):       # every output buffer holds a sampled batch before updates are timed
                        do_step(i)
                    reps = 3 if B >= 16384 else 6

                    def per_call_us(fn):
                        g = torch.cuda.CUDAGraph()
                        with torch.cuda.graph(g, stream=stream):
                            for r in range(ROTATE):
                                fn(r)
                        g.replay()
                        return time_loop(stream, lambda i: g.replay(), reps) / (reps * ROTATE) * 1e3

                    row = {"N": N, "K": K, "B": B, "depth": prb.info()[3],
                           "us_sample": per_call_us(do_sample), "us_update": per_call_us(do_update),
                           "us_insert": per_call_us(do_insert), "us_update_insert": per_call_us(do_update_insert),
                           "us_step": per_call_us(do_step)}
                    row["transitions_per_s"] = B / (row["us_step"] * 1e-6)
                    rows.append(row)
                    print("sweep %6.1f s  %s" % (time.time() - t_start, json.dumps(row)), file=sys.stderr, flush=True)
                    del outs, tds
                status = prb.sync()
                if status & ~0x8:          # anything but CLAMPED (informational)
                    raise RuntimeError("status bits 0x%x in sweep cell N=%d K=%d" % (status, N, K))
                prb.close()
                del prb, rowsrc, ins
                torch.cuda.empty_cache()
    clk = clocks.stop()
    return {"metric": METRIC, "unit": UNIT, "n_gpus": 1, "data": "synthetic",
            "config": {"workload": "sweep", "transition_bytes": 165, "insert_per_step": 1024,
                       "step": "sample(idx,IS,gather) + update_insert", "cuda_graph": True,
                       "timing": "graphs of %d consecutive calls over rotating buffers, CUDA events" % ROTATE},
            "cells": rows, "clocks": clk}


def run_reference(args, wl, rank, world):
    """The CPU oracle as it stands, on this machine's host cores; rank 0 only."""
    if rank != 0:
        return None
    warm = max(args.warmup, 1)
    per_step_guess = 0.03 if wl.counter_rows else 0.001
    steps = max(1, min(args.steps, int(120 / per_step_guess)))
    done, dt, sample, cap = time_oracle(wl, steps, warm, budget_s=150)
    v = wl.batch * done / dt
    return {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": world, "steps": done,
            "warmup": warm, "ms_per_step": dt / done * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32 tree / f64 targets / u8 rows", "data": "synthetic",
            "config": {"workload": wl.name, "capacity": cap, "fanout": wl.fanout, "batch": wl.batch,
                       "insert_per_step": wl.n_insert, "step": "insert+sample(idx,IS,gather)+update"},
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


def relaunch_as_ranks(n):
    """`python bench.py --gpus N` outside a launcher: start N ranks of this script on this node and pass
    their output through (rank 0 prints the one line)."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n), "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="atari_dqn")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--unfused", action="store_true", help="update and insert as two launches instead of pearl_prb_update_insert")
    ap.add_argument("--min-tree", action="store_true",
                    help="the buffer keeps a min-tree (PEARL_OPT_MIN_TREE): rates.us_sample_buffer_norm then has no scan of the leaves")
    ap.add_argument("--cpu-budget", type=float, default=15.0, help="seconds of CPU-oracle work for cpu_baseline")
    ap.add_argument("--sweep", action="store_true",
                    help="time every cell of the capacity x fanout x batch sweep instead (one GPU)")
    prof = ap.add_argument_group("profiling runs (under ncu: the step and its three calls only, a smaller store)")
    prof.add_argument("--profile", action="store_true",
                      help="only the step and its calls: no host-buffer leg, no context timings, no other workloads, no CPU baseline")
    prof.add_argument("--capacity", type=int, default=0, help="override the workload's capacity; with --sweep: this capacity only")
    prof.add_argument("--sweep-fanout", type=int, default=0, help="with --sweep: this fanout only")
    prof.add_argument("--sweep-batch", type=int, default=0, help="with --sweep: this batch size only")
    args = ap.parse_args()

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.sweep:
        sys.exit(relaunch_as_ranks(args.gpus))
    from paper_2311_09445_b200 import workloads as wk
    if args.sweep:
        if int(os.environ.get("RANK", 0)) == 0:
            print(json.dumps(run_sweep(args)), flush=True)
        return
    wl = wk.WORKLOADS[args.workload]
    if args.capacity:
        wl = wk.scaled(wl, args.capacity)
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    line = run_reference(args, wl, rank, world) if args.impl == "reference" else run_ours(args, wl, rank, world)
    if line is not None:
        print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
