"""Benchmark of the paged decode-attention hot path on B200.

One step = one pass of the whole path over one batch: KV append of one token
per sequence, then split-KV attention and the LSE merge over the grown contexts.
The headline value is achieved KV-cache read bandwidth (GB/s): the bytes of K
and V every query must read, divided by the time of the whole step. Inputs are
synthetic, shaped like the paper's rollout workloads (see ``workloads``).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl cuda|reference]

Prints ONE JSON line on rank 0. Without ``--config`` the headline is the largest
single-GPU workload (the multi-turn loop with page allocation) and the other
three target workloads are measured the same way in the same process and
reported under ``per_config``. ``--gpus N`` runs N independent replicas, one
process per GPU: under a launcher that sets WORLD_SIZE the script is one of the
ranks, otherwise it starts the ranks itself. ``--impl reference`` times the CPU
oracle (test infrastructure, run as it stands) on the host cores instead of the
CUDA path.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "decode-attn achieved HBM GB/s (% of B200 peak) and seq-steps/s per layer"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
HEADLINE_CONFIG = 4        # the largest single-GPU workload: the multi-turn loop with page allocation
PER_CONFIG = (1, 2, 3)     # the other target workloads, measured in the same process
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch of the split kernel in the committed ncu
# captures, as a ratio to the algorithmic KV bytes of the captured launch; traffic grows in proportion to the
# pages read, so the ratio of a captured slice of a batch stands for the whole batch.
NCU_TRAFFIC_SOURCE = "profiles/decode_attn_split_traffic_ncu.md"
NCU_TRAFFIC_RATIO = {1: 1.0044, 2: 1.0044, 3: 1.0048, 4: 1.0030}


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    REASONS = {
        0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x10: "sync_boost",
        0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
        0x100: "display_clock_setting",
    }

    def __init__(self, device_index: int, period_s: float = 0.001):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            import torch

            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as e:  # NVML missing: report that instead of clocks
            self.err = repr(e)

    def run(self):
        if not self.ok:
            return
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
                bits = int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self, also=None):
        """Stops sampling and summarises; ``also`` = samplers already stopped whose samples join the summary
        (the clocks of two timed regions of one measurement)."""
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        samples, reasons = list(self.samples), set(self.reasons)
        for other in also or ():
            samples += other.samples
            reasons |= other.reasons
        if not self.ok or not samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["nvml unavailable"]}
        return {"sm_mhz": float(np.median(samples)), "sm_min_mhz": float(np.min(samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(reasons), "samples": len(samples)}


def aggregate_over_ranks(local_ms: float, local_units: float, world_size: int, backend_device=None):
    """Whole-job figures: time = max over ranks, units = sum over ranks (no data-path collective)."""
    if world_size == 1:
        return local_ms, local_units
    import torch
    import torch.distributed as dist

    t = torch.tensor([local_ms], dtype=torch.float64, device=backend_device)
    u = torch.tensor([local_units], dtype=torch.float64, device=backend_device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def workload_config(w, lens, cfg_id):
    return {
        "workload": f"configs[{cfg_id}] {w.name}", "batch": int(len(lens)), "num_q_heads": w.num_q_heads,
        "num_kv_heads": w.num_kv_heads, "head_dim": w.head_dim, "page_size": w.page_size,
        "ctx_tokens_total": int(np.sum(lens)), "ctx_len_min": int(np.min(lens)), "ctx_len_max": int(np.max(lens)),
    }


# ------------------------------------------------------------------------------------------ CUDA arm

def hooked_steps(K: int):
    """Timed steps whose split kernel is bracketed by events: every 4th step of a short run, every 16th of a
    long one, and never fewer than three (or all of them when K < 3)."""
    stride = 4 if K < 48 else 16
    picks = [i for i in range(K) if i % stride == stride // 2]
    if len(picks) < 3:
        picks = sorted({min(K - 1, (2 * j + 1) * K // 6) for j in range(3)})
    return picks


def oracle_sample_size(lens, max_tokens: int = 600_000) -> int:
    """Leading sequences whose cached tokens stay within the CPU baseline's budget (at least one)."""
    csum = np.cumsum(np.asarray(lens, dtype=np.int64))
    return max(1, int(np.searchsorted(csum, max_tokens, side="right")))


def measure_decode(cfg_id, args, rank, world, local_rank, want_cpu_baseline=True):
    """Times one workload: K steps with device-resident inputs, K steps through the host-buffer entry point,
    the split kernel's own duration on a sample of the timed steps, and the oracle on the host cores."""
    import torch

    import paper_2609_35158_b200 as pd
    import workloads as wl

    dev = f"cuda:{local_rank}"
    w = wl.WORKLOADS[cfg_id]
    K, W = args.steps, args.warmup
    # weak scaling: every rank holds its own batch of the same shape (sequences are independent)
    seed = cfg_id + 1000 * rank
    lens0 = wl.context_lengths(cfg_id, seed=seed)
    if args.batch is not None:
        lens0 = lens0[:args.batch]
    B = len(lens0)
    total_steps = 2 * (W + K) + 8  # device-resident loop, then the host-buffer loop
    dynamic_alloc = cfg_id == 4   # pages handed out by the host free list inside the loop
    cache = wl.build_paged_cache(lens0, w.num_kv_heads, w.head_dim, seed=seed, device=dev,
                                 reserve_tokens=total_steps, preassign_reserve=not dynamic_alloc)
    alloc = wl.PageAllocator(cache)
    ctx = pd.pd_create(w.num_q_heads, w.num_kv_heads, w.head_dim, w.page_size, B, cache.page_table.shape[1],
                       cache.num_pages, local_rank)
    R = 4  # rotating activations so no step re-reads the previous step's q / k_new / v_new from L2
    qs = [wl.random_bf16((B, w.num_q_heads, w.head_dim), seed * 100 + 10 + i, dev) for i in range(R)]
    kns = [wl.random_bf16((B, w.num_kv_heads, w.head_dim), seed * 100 + 20 + i, dev) for i in range(R)]
    vns = [wl.random_bf16((B, w.num_kv_heads, w.head_dim), seed * 100 + 30 + i, dev) for i in range(R)]
    out = torch.empty((B, w.num_q_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
    lens = lens0.astype(np.int64).copy()
    bpt = w.kv_bytes_per_token

    # page-table updates of one step travel in one pinned staging row: (sequence, logical page, physical page)
    stage_rows = 2 * (W + K) + 8
    staging = torch.empty((stage_rows, 3, B), dtype=torch.int64).pin_memory() if dynamic_alloc else None
    alloc_calls = [0]
    alloc_seconds = [0.0]

    def allocate_pages():
        if not dynamic_alloc:
            return
        t_alloc = time.perf_counter()
        try:
            need, logical, phys = alloc.assign(lens)
            n = len(need)
            if n:
                row = staging[alloc_calls[0] % stage_rows]
                alloc_calls[0] += 1
                row[0, :n] = torch.from_numpy(need)
                row[1, :n] = torch.from_numpy(logical)
                row[2, :n] = torch.from_numpy(phys.astype(np.int64))
                upd = row[:, :n].to(dev, non_blocking=True)
                cache.page_table[upd[0], upd[1]] = upd[2].to(torch.int32)
        finally:
            alloc_seconds[0] += time.perf_counter() - t_alloc

    def device_step(i):
        nonlocal lens
        allocate_pages()
        if args.step == "fused":
            pd.pd_decode_step(ctx, qs[i % R], kns[i % R], vns[i % R], cache.k_pages, cache.v_pages, cache.page_table,
                              cache.ctx_lens, out, sm_scale=w.sm_scale)
        else:
            pd.pd_kv_append(ctx, kns[i % R], vns[i % R], cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens)
            pd.pd_decode_attn(ctx, qs[i % R], cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out,
                              sm_scale=w.sm_scale)
        lens = lens + 1
        return int(lens.sum()) * bpt  # KV bytes this step's attention must read

    def barrier():
        if world > 1:
            import torch.distributed as dist

            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident loop: the headline value
    for i in range(W):
        device_step(i)
    torch.cuda.synchronize()
    code = pd.pd_device_status(ctx)
    assert code[0] == 0, f"device fault during warm-up: {code}"
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # The library's event hook brackets the split kernel of one step. Two event records cost several
    # microseconds of stream time and switch off launch overlap for that step, so only a sample of the timed
    # steps is hooked.
    hooked = hooked_steps(K)
    befores = {i: torch.cuda.Event(enable_timing=True) for i in hooked}
    afters = {i: torch.cuda.Event(enable_timing=True) for i in hooked}
    sampler = ClockSampler(local_rank)
    launches0 = pd.pd_launch_count(ctx)
    barrier()
    sampler.start()
    t0.record()
    kv_bytes = 0
    hooked_bytes = {}
    alloc_seconds[0] = 0.0
    for i in range(K):
        if i in befores:
            pd.pd_set_profile_events(ctx, befores[i], afters[i])
        step_bytes = device_step(W + i)
        kv_bytes += step_bytes
        if i in befores:
            hooked_bytes[i] = step_bytes
    t1.record()
    barrier()
    clocks = sampler.stop()
    launches = pd.pd_launch_count(ctx) - launches0
    local_ms = t0.elapsed_time(t1)
    alloc_host_us = 1e6 * alloc_seconds[0] / K  # host time of the page allocator per step of the device-resident loop
    split_times = [befores[i].elapsed_time(afters[i]) for i in hooked]
    split_ms = float(np.mean(split_times))
    split_bytes_per_launch = float(np.mean([hooked_bytes[i] for i in hooked]))
    best = int(np.argmin(split_times))
    plan = pd.pd_last_plan(ctx)
    assert pd.pd_device_status(ctx)[0] == 0
    total_ms, total_bytes = aggregate_over_ranks(local_ms, float(kv_bytes), world, dev)
    value_gbs = total_bytes / (total_ms * 1e-3) / 1e9
    bytes_per_step_local = kv_bytes / K

    # ---- host-buffer loop: same step through pd_decode_step_host, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        # one pinned slab per rotation slot, q then k_new then v_new: adjacent host buffers travel in one copy
        hq, hk, hv = [], [], []
        for tq, tk, tv in zip(qs, kns, vns):
            slab = torch.empty(tq.numel() + tk.numel() + tv.numel(), dtype=torch.bfloat16).pin_memory()
            a, b2 = tq.numel(), tq.numel() + tk.numel()
            slab[:a].copy_(tq.reshape(-1)); slab[a:b2].copy_(tk.reshape(-1)); slab[b2:].copy_(tv.reshape(-1))
            hq.append(slab[:a].view(tq.shape)); hk.append(slab[a:b2].view(tk.shape)); hv.append(slab[b2:].view(tv.shape))
        hout = torch.empty((B, w.num_q_heads, w.head_dim), dtype=torch.bfloat16).pin_memory()

        def host_step(i):
            nonlocal lens
            allocate_pages()
            pd.pd_decode_step_host(ctx, hq[i % R], hk[i % R], hv[i % R], cache.k_pages, cache.v_pages, cache.page_table,
                                   cache.ctx_lens, hout, sm_scale=w.sm_scale)
            lens = lens + 1
            return int(lens.sum()) * bpt

        for i in range(W):
            host_step(i)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sampler2 = ClockSampler(local_rank)
        sampler2.start()
        e0.record()
        e2e_bytes = 0
        for i in range(K):
            e2e_bytes += host_step(W + i)
        e1.record()
        barrier()
        clocks = sampler2.stop(also=[sampler])  # samples of both timed regions of this workload
        clocks["regions"] = "device-resident loop + host-buffer loop"
        e2e_ms, e2e_total = aggregate_over_ranks(e0.elapsed_time(e1), float(e2e_bytes), world, dev)
        e2e_gbs = e2e_total / (e2e_ms * 1e-3) / 1e9
        h2d = (hq[0].numel() + hk[0].numel() + hv[0].numel()) * 2
        d2h = hout.numel() * 2
        assert pd.pd_device_status(ctx)[0] == 0
        e2e = {"value": round(e2e_gbs, 2), "unit": "GB/s", "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
               "ms_per_step": round(e2e_ms / K, 5),
               "note": "pd_decode_step_host: q/k_new/v_new from one pinned host slab (one H2D copy), out back to host, "
                       "every step; the KV cache is device-resident state"}

    # ---- CPU baseline: the oracle as it stands, on this machine's host cores (rank 0, N = 1 only)
    cpu_baseline = None
    if want_cpu_baseline and rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = time_oracle_once(w, cache, qs[0], lens)

    peak, peak_kind = measured_hbm_peak()
    achieved = split_bytes_per_launch / (split_ms * 1e-3) / 1e9
    ratio = NCU_TRAFFIC_RATIO.get(cfg_id) if args.batch is None else None
    result = {
        "metric": METRIC, "value": round(value_gbs, 2), "unit": "GB/s", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": round(total_ms / K, 5), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {**workload_config(w, lens0, cfg_id),
                   "ctx_tokens_after_run": int(np.sum(lens)),
                   "l2": f"KV read per step {bytes_per_step_local / 1e9:.2f} GB per GPU >> 126 MB L2; activations rotate over {R} buffers",
                   "parallelism": "1 GPU" if world == 1 else f"{world} independent replicas, sequences sharded by batch, no collective",
                   "plan": plan,
                   **({"page_allocator": f"host free list inside the timed loop, {alloc_host_us:.1f} us of host time per step "
                                         "(one pinned staging row and one index_put per step; it overlaps the previous step's kernels)"}
                      if dynamic_alloc else {})},
        "pct_of_measured_hbm_peak": round(100 * value_gbs / world / peak, 2),
        "pct_of_nominal_8tbs": round(100 * value_gbs / world / NOMINAL_HBM_GBS, 2),
        "seq_steps_per_s": round(B * world * K / (total_ms * 1e-3), 1),
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "decode_attn_split_kernel", "achieved": round(achieved, 2), "peak": peak,
                     "unit": "GB/s", "frac": round(achieved / peak, 4), "peak_kind": f"of {peak_kind}",
                     "traffic": None if ratio is None else int(ratio * split_bytes_per_launch),
                     "traffic_source": None if ratio is None else NCU_TRAFFIC_SOURCE,
                     "algorithmic_bytes_per_launch": int(split_bytes_per_launch), "avg_launch_ms": round(split_ms, 5),
                     "min_launch_ms": round(float(split_times[best]), 5),
                     "achieved_best": round(hooked_bytes[hooked[best]] / (split_times[best] * 1e-3) / 1e9, 2),
                     "launches_timed": len(hooked),
                     "timed": f"CUDA events recorded by the library around the split kernel, {len(hooked)} of the {K} timed launches"},
        "cpu_baseline": cpu_baseline,
    }
    pd.pd_destroy(ctx)
    del cache, qs, kns, vns, out
    torch.cuda.empty_cache()
    return result


def run_cuda(args):
    import torch

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    torch.cuda.set_device(local_rank)
    # default run: the headline is the largest single-GPU workload (the multi-turn loop); the other three
    # target workloads are measured the same way in the same process and reported under per_config
    head_cfg, others = (HEADLINE_CONFIG, PER_CONFIG) if args.config is None else (args.config, ())
    per = {}
    for c in others:
        try:
            r = measure_decode(c, args, rank, world, local_rank)
            per[f"configs[{c}]"] = {k: r[k] for k in ("value", "unit", "ms_per_step", "pct_of_measured_hbm_peak",
                                                     "pct_of_nominal_8tbs", "seq_steps_per_s", "clocks", "e2e", "gpu_launches",
                                                     "roofline", "cpu_baseline", "config")}
        except Exception as e:  # the headline must still be measured
            per[f"configs[{c}]"] = {"error": repr(e)}
    result = measure_decode(head_cfg, args, rank, world, local_rank)
    if others:
        result["per_config"] = per
        if world == 1 and not args.no_next_rows:
            result["next_rows"] = measure_next_rows(args)
    if rank == 0:
        print(json.dumps(result), flush=True)
    if world > 1:
        import torch.distributed as dist

        dist.destroy_process_group()


def measure_next_rows(args):
    """Short runs of the other operations of the library (what `--op prefill`, `--op decode_fp8`, `--op kv_transfer`
    print at length), so that the default line also carries a measurement of each; a failure is reported, not raised."""
    import contextlib
    import copy
    import io

    import torch

    rows = {}
    torch.cuda.empty_cache()  # the headline workload's pools are gone by now; give their memory back first
    jobs = (("prefill", run_prefill, {"steps": 10, "warmup": 3}),
            ("decode_fp8 configs[1]", run_decode_fp8, {"steps": 50, "warmup": 10, "config": 1, "step": "separate"}),
            ("decode_fp8 configs[3]", run_decode_fp8, {"steps": 50, "warmup": 10, "config": 3, "step": "separate"}),
            ("kv_transfer", run_transfer, {"steps": 20, "warmup": 5}))
    for name, fn, overrides in jobs:
        a = copy.copy(args)
        for k, v in overrides.items():
            setattr(a, k, v)
        buf = io.StringIO()
        try:
            with contextlib.redirect_stdout(buf):
                fn(a)
            line = json.loads([ln for ln in buf.getvalue().splitlines() if ln.startswith("{")][-1])
            rows[name] = {k: line[k] for k in ("metric", "value", "unit", "steps", "ms_per_step", "roofline", "clocks")
                          if k in line}
        except Exception as e:
            rows[name] = {"error": repr(e)[:300]}
        torch.cuda.empty_cache()
    return rows


def time_oracle_once(w, cache, q, lens, max_seconds_hint: float = 30.0):
    """Times the oracle on (a prefix of) the batch held in ``cache``; returns the cpu_baseline object."""
    import torch

    import oracle

    cores = os.cpu_count() or 1
    B = len(lens)
    # bounded sample: a prefix of the batch of at most ~600 k cached tokens (2.4 GB of KV at 32/8 heads);
    # the oracle handles roughly 1.5e6 (token x query head) per core-second
    n = oracle_sample_size(lens)
    while n > 1 and float(np.sum(lens[:n])) * w.num_q_heads / (1.5e6 * cores) > max_seconds_hint:
        n //= 2
    # bring only the pages those sequences own to the host, renumbered (the result does not depend on page ids)
    P = cache.k_pages.shape[2]
    table = cache.page_table.detach().cpu().numpy()
    sub_lens = np.asarray(lens, dtype=np.int32)[:n]
    rows = [table[b, :(int(lens[b]) + P - 1) // P] for b in range(n)]
    new_table = np.full((n, table.shape[1]), -1, dtype=np.int32)
    cur = 0
    for i, r in enumerate(rows):
        new_table[i, :len(r)] = np.arange(cur, cur + len(r))
        cur += len(r)
    phys = torch.from_numpy(np.concatenate(rows).astype(np.int64)).to(cache.k_pages.device)
    kp = oracle.bf16_bits(cache.k_pages.index_select(0, phys))
    vp = oracle.bf16_bits(cache.v_pages.index_select(0, phys))
    qb = oracle.bf16_bits(q[:n])
    t = time.perf_counter()
    oracle.decode_attn(qb, kp, vp, new_table, sub_lens, w.sm_scale, nthreads=cores)
    first = time.perf_counter() - t
    # repeat the same step until about 15 core-seconds of CPU work have been timed
    reps = int(min(20, max(1, round(15.0 / max(first * cores, 1e-3)))))
    t = time.perf_counter()
    for _ in range(reps):
        oracle.decode_attn(qb, kp, vp, new_table, sub_lens, w.sm_scale, nthreads=cores)
    dt = (time.perf_counter() - t) / reps
    nbytes = float(np.sum(sub_lens)) * w.kv_bytes_per_token
    return {"value": round(nbytes / dt / 1e9, 4), "unit": "GB/s", "cores": cores, "kind": "oracle",
            "sample": f"attention of the first {n} of {B} sequences ({int(np.sum(sub_lens))} cached tokens, "
                      f"{nbytes / 1e9:.3f} GB of KV per step), {reps} steps, {dt:.2f} s wall per step on "
                      f"{cores} threads",
            "seconds_per_step": round(dt, 3)}


# ------------------------------------------------------------------------------------------ KV transfer op

def run_transfer(args):
    """Gather + scatter of the pages holding every sequence's new tokens (Eq. 3's KV-transfer term).

    Workload: configs[4] geometry (batch 512, 32/8 heads, d = 128); every sequence moves the pages of one
    turn of U{256..2048} new tokens. A step packs them on the source cache and unpacks them into a
    differently placed destination cache. Value = bytes read + written by both kernels / step time."""
    import torch

    import oracle
    import paper_2609_35158_b200 as pd
    import workloads as wl

    dev = "cuda:0"
    torch.cuda.set_device(0)
    w = wl.WORKLOADS[4]
    K, W = args.steps, args.warmup
    rng = np.random.Generator(np.random.PCG64(404))
    new_tokens = rng.integers(256, 2048, size=w.batch, endpoint=True).astype(np.int32)
    src = wl.build_paged_cache(new_tokens, w.num_kv_heads, w.head_dim, seed=41, device=dev)
    dst = wl.build_paged_cache(new_tokens, w.num_kv_heads, w.head_dim, seed=42, device=dev)
    pe = ((new_tokens + 15) // 16).astype(np.int32)
    pb = np.zeros_like(pe)
    off = np.concatenate([[0], np.cumsum(pe)[:-1]]).astype(np.int64)
    total_pages = int(pe.sum())
    page_bytes = 2 * w.num_kv_heads * 16 * w.head_dim * 2
    to_dev = lambda a: torch.from_numpy(a).to(dev)
    d_pb, d_pe, d_off = to_dev(pb), to_dev(pe), to_dev(off)
    packed = torch.empty((total_pages, 2, w.num_kv_heads, 16, w.head_dim), dtype=torch.bfloat16, device=dev)
    ctx_s = pd.pd_create(w.num_q_heads, w.num_kv_heads, w.head_dim, 16, w.batch, src.page_table.shape[1], src.num_pages, 0)
    ctx_d = pd.pd_create(w.num_q_heads, w.num_kv_heads, w.head_dim, 16, w.batch, dst.page_table.shape[1], dst.num_pages, 0)

    def step(buf):
        pd.pd_kv_gather(ctx_s, src.k_pages, src.v_pages, src.page_table, d_pb, d_pe, d_off, buf)
        pd.pd_kv_scatter(ctx_d, buf, d_off, dst.k_pages, dst.v_pages, dst.page_table, d_pb, d_pe)

    for _ in range(W):
        step(packed)
    torch.cuda.synchronize()
    ev = lambda: torch.cuda.Event(enable_timing=True)
    t0, t1 = ev(), ev()
    hooked = [i for i in range(K) if i % 16 == min(8, K - 1)]
    hb, ha = {i: ev() for i in hooked}, {i: ev() for i in hooked}
    sampler = ClockSampler(0)
    sampler.start()
    t0.record()
    for i in range(K):
        if i in hb:
            hb[i].record()
            pd.pd_kv_gather(ctx_s, src.k_pages, src.v_pages, src.page_table, d_pb, d_pe, d_off, packed)
            ha[i].record()
            pd.pd_kv_scatter(ctx_d, packed, d_off, dst.k_pages, dst.v_pages, dst.page_table, d_pb, d_pe)
        else:
            step(packed)
    t1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = t0.elapsed_time(t1) / K
    gather_ms = float(np.mean([hb[i].elapsed_time(ha[i]) for i in hooked]))
    moved = 2 * 2 * total_pages * page_bytes  # two kernels, each reads and writes every page
    assert pd.pd_device_status(ctx_s)[0] == 0 and pd.pd_device_status(ctx_d)[0] == 0

    # host-buffer variant: the packed buffer crosses PCIe in both directions (what a host-staged transport does)
    host = torch.empty(packed.shape, dtype=torch.bfloat16).pin_memory()
    e0, e1 = ev(), ev()
    for i in range(W + K):
        if i == W:
            e0.record()
        pd.pd_kv_gather(ctx_s, src.k_pages, src.v_pages, src.page_table, d_pb, d_pe, d_off, packed)
        host.copy_(packed, non_blocking=True)
        packed.copy_(host, non_blocking=True)
        pd.pd_kv_scatter(ctx_d, packed, d_off, dst.k_pages, dst.v_pages, dst.page_table, d_pb, d_pe)
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1) / K

    # CPU baseline: the oracle's gather + scatter on a prefix of the batch
    n = 64
    sub = list(range(n))
    sk, sv = oracle.bf16_bits(src.k_pages), oracle.bf16_bits(src.v_pages)
    dk, dv = oracle.bf16_bits(dst.k_pages).copy(), oracle.bf16_bits(dst.v_pages).copy()
    sub_off = np.concatenate([[0], np.cumsum(pe[:n])[:-1]]).astype(np.int64)
    t = time.perf_counter()
    reps = 5
    for _ in range(reps):
        pk, _rc = oracle.kv_gather(sk, sv, src.page_table_host[:n], pb[:n], pe[:n], sub_off, int(pe[:n].sum()))
        oracle.kv_scatter(pk, sub_off, dk, dv, dst.page_table_host[:n], pb[:n], pe[:n])
    cpu_s = (time.perf_counter() - t) / reps
    cpu_bytes = 4 * int(pe[:n].sum()) * page_bytes
    peak, peak_kind = measured_hbm_peak()
    value = moved / (ms * 1e-3) / 1e9
    achieved = (moved / 2) / (gather_ms * 1e-3) / 1e9
    result = {
        "metric": "KV page gather+scatter bytes moved (read+write) GB/s", "value": round(value, 2), "unit": "GB/s",
        "n_gpus": 1, "steps": K, "warmup": W, "ms_per_step": round(ms, 5), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": "KV transfer, configs[4] geometry: batch 512, 8 KV heads, d 128, one turn of U{256..2048} new tokens per sequence",
                   "pages_moved": total_pages, "packed_bytes": total_pages * page_bytes,
                   "kv_bytes_per_token_K": w.kv_bytes_per_token,
                   "l2": f"{total_pages * page_bytes / 1e9:.2f} GB packed per step >> 126 MB L2"},
        "clocks": clocks,
        "e2e": {"value": round(moved / (e2e_ms * 1e-3) / 1e9, 2), "unit": "GB/s",
                "h2d_bytes_per_step": total_pages * page_bytes, "d2h_bytes_per_step": total_pages * page_bytes,
                "ms_per_step": round(e2e_ms, 5), "note": "packed buffer staged through pinned host memory between gather and scatter"},
        "gpu_launches": 2 * K,
        "roofline": {"bound": "hbm", "kernel": "kv_transfer_kernel<gather>", "achieved": round(achieved, 2), "peak": peak,
                     "unit": "GB/s", "frac": round(achieved / peak, 4), "peak_kind": f"of {peak_kind}", "traffic": None,
                     "algorithmic_bytes_per_launch": moved // 2, "avg_launch_ms": round(gather_ms, 5)},
        "cpu_baseline": {"value": round(cpu_bytes / cpu_s / 1e9, 3), "unit": "GB/s", "cores": 1, "kind": "oracle",
                         "sample": f"gather + scatter of the first {n} sequences ({int(pe[:n].sum())} pages), {reps} repetitions"},
    }
    pd.pd_destroy(ctx_s)
    pd.pd_destroy(ctx_d)
    print(json.dumps(result), flush=True)


# ------------------------------------------------------------------------------------------ prefill op

def run_prefill(args):
    """Append-prefill of one turn: multi-token append + causal attention of the new tokens over prefix + themselves.

    Workload: Qwen3-8B geometry, 32 sequences whose cached prefix is U{2048..16384} tokens and whose new turn
    is U{256..2048} tokens. Value = attention TFLOP/s of the whole step (append + attention), where the
    attention of query i at position pos costs 4 * H_q * d * (pos + 1) flops."""
    import torch

    import oracle
    import paper_2609_35158_b200 as pd
    import workloads as wl

    dev = "cuda:0"
    torch.cuda.set_device(0)
    w = wl.WORKLOADS[1]
    K, W = args.steps, args.warmup
    B = 32
    rng = np.random.Generator(np.random.PCG64(505))
    q_lens = rng.integers(256, 2048, size=B, endpoint=True).astype(np.int32)
    prefix = rng.integers(2048, 16384, size=B, endpoint=True).astype(np.int32)
    ip = np.concatenate([[0], np.cumsum(q_lens)]).astype(np.int32)
    total_q = int(ip[-1])
    cache = wl.build_paged_cache(prefix, w.num_kv_heads, w.head_dim, seed=51, device=dev,
                                 reserve_tokens=int(q_lens.max()))
    ctx = pd.pd_create(w.num_q_heads, w.num_kv_heads, w.head_dim, 16, B, cache.page_table.shape[1], cache.num_pages, 0)
    q = wl.random_bf16((total_q, w.num_q_heads, w.head_dim), 52, dev)
    kn = wl.random_bf16((total_q, w.num_kv_heads, w.head_dim), 53, dev)
    vn = wl.random_bf16((total_q, w.num_kv_heads, w.head_dim), 54, dev)
    out = torch.empty_like(q)
    ip_dev = torch.from_numpy(ip).to(dev)
    prefix_dev = torch.from_numpy(prefix).to(dev)
    max_q = int(q_lens.max())
    flops = float(sum(4.0 * w.num_q_heads * w.head_dim * (int(n) * int(p0) + int(n) * (int(n) + 1) / 2)
                      for n, p0 in zip(q_lens, prefix)))

    def step():
        cache.ctx_lens.copy_(prefix_dev)  # every step prefills the same turn onto the same prefix
        pd.pd_kv_append_tokens(ctx, kn, vn, ip_dev, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, max_q)
        pd.pd_prefill_attn(ctx, q, ip_dev, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out,
                           max_q_len=max_q, sm_scale=w.sm_scale)

    for _ in range(W):
        step()
    torch.cuda.synchronize()
    assert pd.pd_device_status(ctx)[0] == 0
    ev = lambda: torch.cuda.Event(enable_timing=True)
    t0, t1 = ev(), ev()
    hooked = [i for i in range(K) if i % 4 == min(2, K - 1)]
    hb, ha = {i: ev() for i in hooked}, {i: ev() for i in hooked}
    sampler = ClockSampler(0)
    sampler.start()
    t0.record()
    for i in range(K):
        if i in hb:
            cache.ctx_lens.copy_(prefix_dev)
            pd.pd_kv_append_tokens(ctx, kn, vn, ip_dev, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, max_q)
            hb[i].record()
            pd.pd_prefill_attn(ctx, q, ip_dev, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out,
                               max_q_len=max_q, sm_scale=w.sm_scale)
            ha[i].record()
        else:
            step()
    t1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    assert pd.pd_device_status(ctx)[0] == 0
    ms = t0.elapsed_time(t1) / K
    attn_ms = float(np.mean([hb[i].elapsed_time(ha[i]) for i in hooked]))

    # host-buffer variant: q, k_new, v_new from pinned host memory, out back to the host, every step
    hq, hk, hv = q.cpu().pin_memory(), kn.cpu().pin_memory(), vn.cpu().pin_memory()
    hout = torch.empty(out.shape, dtype=torch.bfloat16).pin_memory()
    e0, e1 = ev(), ev()
    for i in range(W + K):
        if i == W:
            e0.record()
        q.copy_(hq, non_blocking=True)
        kn.copy_(hk, non_blocking=True)
        vn.copy_(hv, non_blocking=True)
        step()
        hout.copy_(out, non_blocking=True)
        torch.cuda.synchronize()
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1) / K

    # CPU baseline: the oracle on a sample of query rows (first, middle, last of a few sequences)
    cores = os.cpu_count() or 1
    kp, vp = oracle.bf16_bits(cache.k_pages), oracle.bf16_bits(cache.v_pages)
    lens_after = (prefix + q_lens).astype(np.int32)
    nseq = 2
    sub_ip = np.concatenate([[0], np.cumsum(q_lens[:nseq])]).astype(np.int32)
    t = time.perf_counter()
    oracle.prefill_attn(oracle.bf16_bits(q[:int(sub_ip[-1])]), sub_ip, kp, vp, cache.page_table_host[:nseq], lens_after[:nseq],
                        w.sm_scale, nthreads=cores)
    cpu_s = time.perf_counter() - t
    cpu_flops = float(sum(4.0 * w.num_q_heads * w.head_dim * (int(n) * int(p0) + int(n) * (int(n) + 1) / 2)
                          for n, p0 in zip(q_lens[:nseq], prefix[:nseq])))
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            peak, peak_kind = float(json.load(f)["bf16_tflops"]), "measured (cuBLAS bf16 burst)"
    except Exception:
        peak, peak_kind = 1590.0, "fallback"
    achieved = flops / (attn_ms * 1e-3) / 1e12
    result = {
        "metric": "append-prefill attention TFLOP/s", "value": round(flops / (ms * 1e-3) / 1e12, 2), "unit": "TFLOP/s",
        "n_gpus": 1, "steps": K, "warmup": W, "ms_per_step": round(ms, 5), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "one prefill turn, Qwen3-8B geometry (32/8 heads, d 128), 32 sequences, prefix U{2048..16384}, new tokens U{256..2048}",
                   "new_tokens_total": total_q, "prefix_tokens_total": int(prefix.sum()), "flops_per_step": flops},
        "clocks": clocks,
        "e2e": {"value": round(flops / (e2e_ms * 1e-3) / 1e12, 2), "unit": "TFLOP/s",
                "h2d_bytes_per_step": int((hq.numel() + hk.numel() + hv.numel()) * 2), "d2h_bytes_per_step": int(hout.numel() * 2),
                "ms_per_step": round(e2e_ms, 5)},
        "gpu_launches": 4 * K,  # append (2 kernels), sequence ordering, attention
        "roofline": {"bound": "tensor", "kernel": "prefill_attn_kernel", "achieved": round(achieved, 2), "peak": peak,
                     "unit": "TFLOP/s", "frac": round(achieved / peak, 4), "peak_kind": f"of {peak_kind}", "traffic": None,
                     "avg_launch_ms": round(attn_ms, 5)},
        "cpu_baseline": {"value": round(cpu_flops / cpu_s / 1e12, 5), "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                         "sample": f"all query rows of the first {nseq} sequences ({int(sub_ip[-1])} new tokens), {cpu_s:.1f} s"},
    }
    pd.pd_destroy(ctx)
    print(json.dumps(result), flush=True)


# ------------------------------------------------------------------------------------------ fitting b

def run_fit_b(args):
    """Measures the decode step (append + attention) at several batch sizes with 8192-token contexts and fits
    step_seconds = A_attn + b * concurrency: b is the per-sequence, per-layer KV-read cost of Eq. 1, as this
    library delivers it on this GPU. The fit feeds pd_decide in an example with assumed remaining parameters."""
    import torch

    import paper_2609_35158_b200 as pd
    import workloads as wl

    dev = "cuda:0"
    torch.cuda.set_device(0)
    w = wl.WORKLOADS[1]
    K, W = args.steps, args.warmup
    ctx_len = 8192
    batches = [8, 16, 32, 64, 128, 256]
    times = []
    for B in batches:
        lens = np.full(B, ctx_len, dtype=np.int32)
        cache = wl.build_paged_cache(lens, w.num_kv_heads, w.head_dim, seed=60 + B, device=dev, reserve_tokens=W + K + 2)
        ctx = pd.pd_create(w.num_q_heads, w.num_kv_heads, w.head_dim, 16, B, cache.page_table.shape[1], cache.num_pages, 0)
        q = wl.random_bf16((B, w.num_q_heads, w.head_dim), 61, dev)
        kn = wl.random_bf16((B, w.num_kv_heads, w.head_dim), 62, dev)
        out = torch.empty_like(q)

        def step():
            pd.pd_kv_append(ctx, kn, kn, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens)
            pd.pd_decode_attn(ctx, q, cache.k_pages, cache.v_pages, cache.page_table, cache.ctx_lens, out, sm_scale=w.sm_scale)

        for _ in range(W):
            step()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t0.record()
        for _ in range(K):
            step()
        t1.record()
        torch.cuda.synchronize()
        times.append(t0.elapsed_time(t1) / K * 1e-3)
        pd.pd_destroy(ctx)
        del cache
    A_attn, b = pd.pd_fit_decode_cost(batches, times)
    layers = 36  # Qwen3-8B has 36 layers (public model card); b per iteration = layers * b per layer
    model = pd.pd_cost_model(64, 10, 200, 1000, 0.5, 0.02, b * layers, 1e-5, 0.01, 5.0, w.kv_bytes_per_token * layers, 50e9,
                             32768.0 * w.kv_bytes_per_token * layers, 120e9, 0)
    tgt = pd.pd_decide(model, 16)
    print(json.dumps({
        "metric": "decode cost per concurrent sequence per layer (b of Eq. 1)", "value": round(b * 1e6, 4), "unit": "us",
        "fixed_us_per_layer": round(A_attn * 1e6, 3), "context_tokens": ctx_len, "batches": batches,
        "step_us": [round(t * 1e6, 2) for t in times],
        "ideal_us_per_sequence_at_measured_copy_bw": round(ctx_len * w.kv_bytes_per_token / measured_hbm_peak()[0] / 1e3, 4),
        "example_decision": {"assumed": "B=64 S=10 r=200 dL=1000 theta=0.5 A=20ms t_prefill=10us T_env=5s BW=50GB/s H_max=120GB, 36 layers",
                             "N_k": 16, "N_P": tgt.N_P, "N_D": tgt.N_D, "N_C": tgt.N_C, "makespan_s": round(tgt.makespan, 3)},
    }), flush=True)


# ------------------------------------------------------------------------------------------ FP8 pages

def run_decode_fp8(args):
    """The decode step over FP8 (e4m3) KV pages: pd_kv_append_fp8 + pd_decode_attn_fp8 (with --step fused the one call
    pd_decode_step_fp8, which enqueues the same three kernels), device-resident inputs.
    Bytes per cached token: one byte per K and V value plus the 16-byte scale record of each (page, KV head)."""
    import torch

    import oracle
    import paper_2609_35158_b200 as pd
    import workloads as wl

    torch.cuda.set_device(0)
    dev = "cuda:0"
    cfg_id = args.config
    w = wl.WORKLOADS[cfg_id]
    K, W = args.steps, args.warmup
    lens0 = wl.context_lengths(cfg_id)
    B = w.batch
    cache = wl.build_paged_cache(lens0, w.num_kv_heads, w.head_dim, seed=cfg_id, device=dev, reserve_tokens=W + K + 2)
    NP, P = cache.num_pages, w.page_size
    ctx = pd.pd_create(w.num_q_heads, w.num_kv_heads, w.head_dim, P, B, cache.page_table.shape[1], NP, 0)
    tip = np.zeros(NP, dtype=np.int32)
    for b, L in enumerate(lens0):
        n = (int(L) + P - 1) // P
        tip[cache.page_table_host[b, :n]] = P
        if L % P:
            tip[cache.page_table_host[b, n - 1]] = L % P
    k8 = torch.empty((NP, w.num_kv_heads, P, w.head_dim), dtype=torch.uint8, device=dev)
    v8 = torch.empty_like(k8)
    sc = torch.empty((NP, w.num_kv_heads, 4), dtype=torch.float32, device=dev)
    pd.pd_kv_quantize_pages(ctx, cache.k_pages, cache.v_pages, torch.from_numpy(tip).to(dev), k8, v8, sc)
    torch.cuda.synchronize()
    R = 4
    qs = [wl.random_bf16((B, w.num_q_heads, w.head_dim), 10 + i, dev) for i in range(R)]
    kns = [wl.random_bf16((B, w.num_kv_heads, w.head_dim), 20 + i, dev) for i in range(R)]
    vns = [wl.random_bf16((B, w.num_kv_heads, w.head_dim), 30 + i, dev) for i in range(R)]
    out = torch.empty((B, w.num_q_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
    lens = lens0.astype(np.int64).copy()
    per_token = 2 * w.num_kv_heads * w.head_dim          # one byte per K and per V value
    per_page = w.num_kv_heads * 16                        # scale records

    def step(i):
        nonlocal lens
        if args.step == "fused":
            pd.pd_decode_step_fp8(ctx, qs[i % R], kns[i % R], vns[i % R], k8, v8, sc, cache.page_table, cache.ctx_lens, out,
                                  sm_scale=w.sm_scale)
        else:
            pd.pd_kv_append_fp8(ctx, kns[i % R], vns[i % R], k8, v8, sc, cache.page_table, cache.ctx_lens)
            pd.pd_decode_attn_fp8(ctx, qs[i % R], k8, v8, sc, cache.page_table, cache.ctx_lens, out, sm_scale=w.sm_scale)
        lens = lens + 1
        return int(lens.sum()) * per_token + int(((lens + P - 1) // P).sum()) * per_page

    for i in range(W):
        step(i)
    torch.cuda.synchronize()
    assert pd.pd_device_status(ctx)[0] == 0
    hooked = [i for i in range(K) if i % 16 == min(8, K - 1)]
    befores = {i: torch.cuda.Event(enable_timing=True) for i in hooked}
    afters = {i: torch.cuda.Event(enable_timing=True) for i in hooked}
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(0)
    torch.cuda.synchronize()
    sampler.start()
    t0.record()
    total = hooked_bytes = 0
    for i in range(K):
        if i in befores:
            pd.pd_set_profile_events(ctx, befores[i], afters[i])
        nb = step(W + i)
        total += nb
        if i in befores:
            hooked_bytes += nb
    t1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    assert pd.pd_device_status(ctx)[0] == 0
    ms = t0.elapsed_time(t1)
    split_ms = float(np.mean([befores[i].elapsed_time(afters[i]) for i in hooked]))
    per_launch = hooked_bytes / len(hooked)
    peak, peak_kind = measured_hbm_peak()
    achieved = per_launch / (split_ms * 1e-3) / 1e9

    # CPU baseline inputs: the oracle's own quantisation of one short and one long sequence of the initial cache (the
    # bf16 pools are untouched by the FP8 steps). Gathered after the timed region: no other kernel runs between
    # pd_create and the timed steps
    sample = [int(np.argmin(lens0)), int(np.argmax(lens0))]
    pages = np.concatenate([cache.page_table_host[b, :(int(lens0[b]) + P - 1) // P] for b in sample])
    idx = torch.from_numpy(pages.astype(np.int64)).to(dev)
    o_k8, o_v8, o_sc = oracle.fp8_quantize_pages(oracle.bf16_bits(cache.k_pages.index_select(0, idx)),
                                                 oracle.bf16_bits(cache.v_pages.index_select(0, idx)), tip[pages])
    o_table = np.full((2, cache.page_table.shape[1]), -1, dtype=np.int32)
    cur = 0
    for i, b in enumerate(sample):
        n = (int(lens0[b]) + P - 1) // P
        o_table[i, :n] = np.arange(cur, cur + n)
        cur += n
    del cache.k_pages, cache.v_pages
    # CPU baseline: the FP8 oracle as it stands on the two sampled sequences
    tc = time.perf_counter()
    oracle.fp8_decode_attn(oracle.bf16_bits(qs[0][torch.tensor(sample, device=dev)]), o_k8, o_v8, o_sc, o_table,
                           lens0[sample].astype(np.int32), w.sm_scale)
    oracle_s = time.perf_counter() - tc
    oracle_bytes = float(lens0[sample].sum()) * per_token
    value = total / (ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": "FP8-page decode-attn achieved HBM GB/s and seq-steps/s per layer", "value": round(value, 2), "unit": "GB/s",
        "n_gpus": 1, "steps": K, "warmup": W, "ms_per_step": round(ms / K, 5), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "e4m3 pages, fp16 products, fp32 accumulation", "data": "synthetic",
        "config": {**workload_config(w, lens, cfg_id), "bytes_per_cached_token": per_token + per_page / P,
                   "l2": f"KV read per step {total / K / 1e9:.2f} GB >> 126 MB L2; activations rotate over {R} buffers"},
        "seq_steps_per_s": round(B * K / (ms * 1e-3), 1), "pct_of_measured_hbm_peak": round(100 * value / peak, 2),
        "clocks": clocks, "gpu_launches": (2 if args.step == "fused" else 3) * K,
        "roofline": {"bound": "hbm", "kernel": "decode_attn_split_fp8_kernel", "achieved": round(achieved, 2), "peak": peak,
                     "unit": "GB/s", "frac": round(achieved / peak, 4), "peak_kind": f"of {peak_kind}", "traffic": None,
                     "algorithmic_bytes_per_launch": int(per_launch), "avg_launch_ms": round(split_ms, 5)},
        "cpu_baseline": {"value": round(oracle_bytes / oracle_s / 1e9, 4), "unit": "GB/s", "cores": os.cpu_count(), "kind": "oracle",
                         "sample": f"FP8 oracle on sequences {sample} ({int(lens0[sample].sum())} cached tokens), {oracle_s:.1f} s"},
    }), flush=True)
    pd.pd_destroy(ctx)


# ------------------------------------------------------------------------------------------ pool toggle

def run_pool_toggle(args):
    """Wall time to release and to restore the physical memory of a KV pool of the multi-turn workload's size
    (the KV-cache share of T_toggle in Eq. 7). Host driver calls, so the clock is the host's."""
    import time

    import torch

    import paper_2609_35158_b200 as pd
    import workloads as wl

    torch.cuda.set_device(0)
    w = wl.WORKLOADS[4]
    lens = wl.context_lengths(4).astype(np.int64) + 128
    pages = int(np.ceil(1.0625 * ((lens + 15) // 16).sum()))
    cap = 2 * pages * w.num_kv_heads * 16 * w.head_dim * 2
    reps = max(3, min(args.steps, 10))
    rows = []
    for chunk in (64 << 20, 256 << 20, 1 << 30):
        pool = pd.pd_pool_create(0, cap, chunk)
        rel, res, touch = [], [], []
        for _ in range(reps):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            pd.pd_pool_resize(pool, pd.pd_pool_capacity(pool))
            t1 = time.perf_counter()
            whole = pd.pool_tensor(pool, 0, (pd.pd_pool_capacity(pool),), torch.uint8)
            whole.zero_()  # first touch of the restored memory
            torch.cuda.synchronize()
            t2 = time.perf_counter()
            del whole
            pd.pd_pool_resize(pool, 0)
            t3 = time.perf_counter()
            res.append(t1 - t0)
            touch.append(t2 - t1)
            rel.append(t3 - t2)
        rows.append({"chunk_mib": pd.pd_pool_chunk_bytes(pool) >> 20, "capacity_gb": round(pd.pd_pool_capacity(pool) / 1e9, 2),
                     "restore_ms": round(1e3 * float(np.median(res)), 2), "first_write_ms": round(1e3 * float(np.median(touch)), 2),
                     "release_ms": round(1e3 * float(np.median(rel)), 2)})
        pd.pd_pool_destroy(pool)
    best = min(rows, key=lambda r: r["restore_ms"] + r["release_ms"])
    t_toggle = (best["restore_ms"] + best["release_ms"]) * 1e-3
    print(json.dumps({
        "metric": "KV pool release + restore wall time (KV share of T_toggle, Eq. 7)", "value": round(t_toggle * 1e3, 2),
        "unit": "ms", "higher_is_better": False, "repetitions": reps, "by_chunk": rows,
        "example_gate": {"assumed": "R/B = 0.25, T_ded = 60 s, T_full = 40 s",
                         "borrow": bool(pd.pd_toggle_gate(16, 64, 60.0, 40.0, t_toggle))},
    }), flush=True)


# ------------------------------------------------------------------------------------------ read ceiling

def run_read_ceiling(args):
    """Read-only HBM ceiling of this GPU: a plain streaming kernel (16-byte loads, nothing stored) over 4 GB,
    best of several grid shapes, set beside the measured copy bandwidth that is the roofline denominator."""
    import torch

    import paper_2609_35158_b200 as pd

    torch.cuda.set_device(0)
    buf = torch.full((4 << 30,), 1, dtype=torch.uint8, device="cuda:0")
    sink = torch.zeros(16, dtype=torch.uint8, device="cuda:0")
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    rows = []
    for per_sm in (2, 4, 8, 16, 32):
        for threads in (256, 512, 1024):
            for _ in range(max(3, args.warmup)):
                pd.pd_read_probe(buf, sms * per_sm, threads, sink)
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            t0.record()
            for _ in range(args.steps):
                pd.pd_read_probe(buf, sms * per_sm, threads, sink)
            t1.record()
            torch.cuda.synchronize()
            rows.append({"blocks_per_sm": per_sm, "threads": threads,
                         "gbs": round(buf.numel() * args.steps / (t0.elapsed_time(t1) * 1e-3) / 1e9, 1)})
    best = max(rows, key=lambda r: r["gbs"])
    peak, kind = measured_hbm_peak()
    print(json.dumps({"metric": "read-only streaming bandwidth (16-byte loads over 4 GB, nothing stored)", "value": best["gbs"],
                      "unit": "GB/s", "best_shape": best, "steps": args.steps, "copy_bandwidth_gbs": peak,
                      "copy_bandwidth_kind": kind, "ratio_to_copy": round(best["gbs"] / peak, 4), "by_shape": rows}), flush=True)


# ------------------------------------------------------------------------------------------ reference arm

def run_reference(args):
    """The CPU oracle timed on the host cores: each step = attention over a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    import workloads as wl

    cfg_id = HEADLINE_CONFIG if args.config is None else args.config
    w = wl.WORKLOADS[cfg_id]
    K, W = args.steps, args.warmup
    cores = os.cpu_count() or 1
    lens_all = wl.context_lengths(cfg_id)
    if args.batch is not None:
        lens_all = lens_all[:args.batch]
    # bounded sample: whole run (K + W steps) within about two minutes. The oracle handles
    # roughly 2e6 (token x query head) per core-second; stay well below that.
    budget_tokens = 120.0 * 1.5e6 * cores / w.num_q_heads / max(1, K + W)
    n = 1
    while n < len(lens_all) and float(np.sum(lens_all[:n + 1])) <= budget_tokens:
        n += 1
    lens = lens_all[:n].copy()
    if float(np.sum(lens)) > budget_tokens:  # a single long sequence: shorten it
        lens[0] = max(16, int(budget_tokens))
    cache = wl.build_paged_cache(lens, w.num_kv_heads, w.head_dim, seed=cfg_id, device="cpu")
    q = oracle.bf16_bits(wl.random_bf16((n, w.num_q_heads, w.head_dim), 100 + cfg_id, "cpu"))
    kp, vp = oracle.bf16_bits(cache.k_pages), oracle.bf16_bits(cache.v_pages)
    nbytes = float(np.sum(lens)) * w.kv_bytes_per_token

    def step():
        oracle.decode_attn(q, kp, vp, cache.page_table_host, lens, w.sm_scale, nthreads=cores)

    for _ in range(W):
        step()
    t = time.perf_counter()
    for _ in range(K):
        step()
    dt = time.perf_counter() - t
    value = nbytes * K / dt / 1e9
    sample = (f"attention of the first {n} of {len(lens_all)} sequences ({int(np.sum(lens))} cached tokens, "
              f"{nbytes / 1e9:.4f} GB of KV per step)")
    result = {
        "impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": "GB/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", str(args.gpus))), "steps": K, "warmup": W,
        "ms_per_step": round(dt / K * 1e3, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        # the workload is the CUDA arm's (same lengths, same totals); `sample` says which part of it a step covers
        "config": {**workload_config(w, lens_all, cfg_id), "sample": sample},
        "cpu_baseline": {"value": round(value, 4), "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": round(value, 4), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(result), flush=True)


# ------------------------------------------------------------------------------------------ replicas

def spawn_replicas(args) -> int:
    """`--gpus N` without a launcher: start N ranks of this script, one process per GPU (RANK = LOCAL_RANK =
    0 .. N-1, rendezvous on 127.0.0.1). The ranks are independent replicas: every one builds its own cache
    (seed + 1000 * rank) and the only communication is the barrier around the timed region and the max / sum
    of two scalars. Rank 0 prints the line."""
    import socket
    import subprocess

    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    procs = []
    for r in range(args.gpus):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(args.gpus), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__), *sys.argv[1:]], env=env))
    rc = 0
    for p in procs:
        try:
            rc = max(rc, abs(p.wait(timeout=3600)))
        except subprocess.TimeoutExpired:
            rc = 1
        if rc:  # one rank failed: the others would wait for it at the barrier
            for other in procs:
                if other.poll() is None:
                    other.kill()
    return rc


def run_stub(args):
    """The multi-rank plumbing with a host stand-in for the step (no GPU, gloo): barrier, K timed 'steps' that
    sleep, max-over-ranks time and summed units, one line from rank 0. It exists so that the spawn path and the
    aggregation can be tested on a machine without GPUs; it measures nothing."""
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    t = time.perf_counter()
    for _ in range(args.steps):
        time.sleep(0.001 * (rank + 1))
    local_ms = (time.perf_counter() - t) * 1e3
    if world > 1:
        dist.barrier()
    ms, units = aggregate_over_ranks(local_ms, float(100 * (rank + 1)), world)
    if rank == 0:
        print(json.dumps({"impl": "stub", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                          "ms_per_step": round(ms / args.steps, 4), "units": units, "scaling": "weak",
                          "seeds": [HEADLINE_CONFIG + 1000 * r for r in range(world)]}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1, help="ranks, one per GPU; without a launcher (no WORLD_SIZE in the "
                    "environment) the script starts them itself")
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", type=int, default=None, choices=[0, 1, 2, 3, 4],
                    help="default: headline on configs[4], configs[1..3] under per_config")
    ap.add_argument("--batch", type=int, default=None, help="only the first N sequences of the workload (small ncu captures)")
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference", "stub"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer loop (small ncu captures)")
    ap.add_argument("--no-next-rows", action="store_true",
                    help="default run only: skip the short prefill / FP8 decode / KV transfer measurements under next_rows")
    ap.add_argument("--step", default=None, choices=["separate", "fused"],
                    help="pd_kv_append + pd_decode_attn (two calls, 3 launches) or pd_decode_step (one call; 2 launches for "
                         "bf16, the same 3 for FP8, which has no fused kernel); default: fused for --op decode, "
                         "separate for --op decode_fp8")
    ap.add_argument("--op", default="decode", choices=["decode", "decode_fp8", "kv_transfer", "prefill", "fit_b", "pool_toggle", "read_ceiling"],
                    help="decode = the headline decode step; kv_transfer = page gather + scatter; "
                         "prefill = one append-prefill turn; fit_b = decode step time over batch size, fitted to A + b * B; "
                         "pool_toggle = release and restore of a KV pool's physical memory; "
                         "decode_fp8 = the decode step over FP8 (e4m3) KV pages; "
                         "read_ceiling = a plain read-only streaming kernel, the practical ceiling of a read-once scan")
    args = ap.parse_args()
    if args.gpus < 1:
        ap.error("--gpus must be >= 1")
    world_env = os.environ.get("WORLD_SIZE")
    if world_env is not None and int(world_env) != args.gpus:
        ap.error(f"--gpus {args.gpus} but the launcher set WORLD_SIZE={world_env}")
    if args.gpus > 1 and world_env is None and args.impl != "reference":
        if args.op != "decode":
            ap.error("--gpus N > 1 runs replicas of the decode step only")
        sys.exit(spawn_replicas(args))
    if args.step is None:
        args.step = "separate" if args.op == "decode_fp8" else "fused"
    if args.warmup < 3 and args.impl == "cuda":
        args.warmup = 3
    if args.op != "decode" and args.config is None:
        args.config = 1
    if args.impl == "cuda":
        # the built library is not tracked: compile it if this checkout has none yet (rank 0 first under torchrun)
        import __graft_entry__ as entry

        if int(os.environ.get("LOCAL_RANK", "0")) == 0:
            entry.ensure_built()
        else:
            for _ in range(600):
                if os.path.exists(os.path.join(ROOT, "paper_2609_35158_b200", "libpd.so")):
                    break
                time.sleep(0.5)
    if args.impl == "reference":
        run_reference(args)
    elif args.impl == "stub":
        run_stub(args)
    elif args.op == "kv_transfer":
        run_transfer(args)
    elif args.op == "prefill":
        run_prefill(args)
    elif args.op == "fit_b":
        run_fit_b(args)
    elif args.op == "decode_fp8":
        run_decode_fp8(args)
    elif args.op == "pool_toggle":
        run_pool_toggle(args)
    elif args.op == "read_ceiling":
        run_read_ceiling(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
