#!/usr/bin/env python
"""Benchmark: one serving step of mixed decode + interrupt-append paged attention on B200.

A step = asynclm_kv_append + asynclm_attn_mixed over one synthetic batch with the Llama-3-8B
attention shape (32 query heads, 8 kv heads, head_dim 128, page 16, 32 sequences, contexts uniform
in [512, 4096], 8 sequences receive an interrupt span of 8..64 tokens, the rest decode one token).
The plan is built once per step on the host (it is shared by all layers of a model) and its cost is
reported separately and inside the end-to-end figure.

Prints ONE JSON line.  `value` is KV GB/s (bytes of K/V the step must read, divided by the step's
device time); `ms_per_step` carries the step time.  Multi-GPU runs are independent replicas (the
path has no cross-GPU exchange).  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "kv_gbps_mixed_decode_interrupt_append"
UNIT = "GB/s"
WORKLOAD = "config2-llama3-8b-mixed-batch"       # the configuration the metric is quoted on (default)
WORKLOADS = {2: WORKLOAD, 3: "config3-large-batch-gqa8", 4: "config4-long-context-split-kv"}
# dram__bytes_read.sum + dram__bytes_write.sum of attn_fused_kernel, one launch on the default
# workload, from an ncu capture; None whenever the kernel has changed since the counters were taken
TRAFFIC_BYTES_PER_LAUNCH = 325_879_808


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int):
        self.samples = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                self.samples.append((time.time(), float(parts[0]), float(parts[1]), parts[2:6]))
            except ValueError:
                pass

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        inside = [s for s in self.samples if t0 <= s[0] <= t1] or self.samples
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        reasons = sorted({self.NAMES[i] for s in inside for i, v in enumerate(s[3])
                          if v.lower().startswith("active")})
        return {"sm_mhz": float(np.median([s[1] for s in inside])), "sm_max_mhz": inside[0][2],
                "reasons": reasons, "samples": len(inside)}


class L2Flush:
    """Evicts the KV pool from L2 between timed steps (untimed): a 256 MiB buffer is rewritten, which
    pushes everything else out, and then another 256 MiB buffer is read, which leaves L2 full of
    clean lines.  Without the read pass L2 would still hold up to 126 MB of the fill's dirty lines,
    and their write-back would ride on the timed step's DRAM traffic (measured: 17 us of a 107 us
    decode-only step)."""
    NOTE = "256 MiB buffer rewritten, then a second 256 MiB buffer read, between timed steps (untimed)"

    def __init__(self, torch):
        self.w = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")     # > 126 MB L2
        self.r = torch.zeros(64 << 20, dtype=torch.int32, device="cuda")

    def fill_(self, v):
        self.w.fill_(v)
        self.r.sum()


# ------------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------------

def oracle_sample_rows(st, budget_pairs: float, seed: int = 0):
    """A seeded subset of token rows whose (row, key) pair count is about `budget_pairs`."""
    n_row = np.repeat(st.kv_len_before.astype(np.int64), st.q_len) + \
        np.concatenate([np.arange(1, q + 1) for q in st.q_len]) if st.total_q else np.zeros(0)
    order = np.random.default_rng(seed).permutation(st.total_q)
    csum = np.cumsum(n_row[order])
    k = int(np.searchsorted(csum, budget_pairs, side="left")) + 1
    rows = np.sort(order[:min(k, st.total_q)])
    return rows, float(n_row[rows].sum()), float(n_row.sum())


def time_oracle(wl, st, seconds_target: float):
    """Times the oracle (as it stands) on a bounded row sample; returns a dict for the report."""
    from oracle import oracle
    from paper_2412_07017_b200 import workload as W
    cores = oracle.num_threads()
    pool = wl.kv_pool.copy()
    t0 = time.perf_counter()
    oracle.kv_append(pool, st.q_indptr, st.kv_len_before, st.page_indptr, st.page_indices,
                     st.k_new, st.v_new)
    t_append = time.perf_counter() - t0
    probe_rows, probe_pairs, total_pairs = oracle_sample_rows(st, 2.0e4 * cores, seed=1)
    t0 = time.perf_counter()
    oracle.attn_mixed(pool, st.q, st.q_indptr, st.kv_len_before, st.page_indptr, st.page_indices,
                      sel_rows=probe_rows)
    rate = probe_pairs / max(time.perf_counter() - t0, 1e-6)       # (row, key) pairs per second
    rows, pairs, total_pairs = oracle_sample_rows(st, rate * seconds_target, seed=2)
    t0 = time.perf_counter()
    oracle.attn_mixed(pool, st.q, st.q_indptr, st.kv_len_before, st.page_indptr, st.page_indices,
                      sel_rows=rows)
    t_attn = time.perf_counter() - t0
    step_seconds = t_append + t_attn * total_pairs / pairs
    kv_bytes = W.algorithmic_bytes(wl.shape, st)["kv"]
    return {"value": kv_bytes / step_seconds / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{len(rows)} of {st.total_q} token rows (seeded), all {wl.shape.num_q_heads} "
                      f"heads, {pairs / total_pairs:.3f} of the step's (row,key) pairs, "
                      f"{t_attn:.1f} s measured, step time extrapolated to {step_seconds:.1f} s",
            "step_seconds": step_seconds}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2412_07017_b200 import workload as W
    wl = W.make_config(2)
    st = wl.steps[0]
    per_step = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    times, last = [], None
    for i in range(args.warmup + args.steps):
        last = time_oracle(wl, st, per_step)
        if i >= args.warmup:
            times.append(last["step_seconds"])
    kv_bytes = W.algorithmic_bytes(wl.shape, st)["kv"]
    sec = float(np.mean(times))
    value = kv_bytes / sec / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": WORKLOAD, "seed": wl.seed},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": last["cores"], "kind": "oracle",
                             "sample": last["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------

def max_over_ranks(x: float) -> float:
    """The largest of the ranks' values (the step time of the slowest replica); identity without a
    process group.  Works on whichever backend the group has (NCCL on GPUs, gloo in the CPU tests)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(x)], device=dev, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(kv_bytes_per_replica: int, world: int, ms_per_step: float) -> float:
    """GB/s of the whole job: every rank runs the same step on its own GPU (no exchange between them),
    and the job's step takes as long as its slowest replica's."""
    return world * kv_bytes_per_replica / (ms_per_step * 1e-3) / 1e9


def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2412_07017_b200 import binding as B
    from paper_2412_07017_b200 import workload as W

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    if args.decode_only:
        # 64 sequences of the Llama-3-8B attention shape, contexts uniform in [1024, 3072], one decode
        # token each: the warp body alone (profiling aid, not the benchmarked workload)
        lens = np.random.default_rng(3).integers(1024, 3073, 64).tolist()
        wl = W.make_single_step("decode-only", W.Shape(32, 8, 128, 16), lens, [1] * 64, seed=11)
    elif args.spans_only:
        # 24 sequences of the same shape, contexts uniform in [1024, 3072], every one with an interrupt
        # span of 64 tokens (256 query rows per kv head): the tensor-core span kernel alone
        lens = np.random.default_rng(4).integers(1024, 3073, 24).tolist()
        wl = W.make_single_step("spans-only", W.Shape(32, 8, 128, 16), lens, [64] * 24, seed=12)
    else:
        wl = W.make_config(args.config)
    st = wl.steps[0]
    shape = wl.shape
    by = W.algorithmic_bytes(shape, st)
    flops = W.algorithmic_flops(shape, st)

    def dev(bits):
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)

    pool = dev(wl.kv_pool)
    q, kn, vn = dev(st.q), dev(st.k_new), dev(st.v_new)
    T = st.total_q
    out = torch.empty((T, shape.num_q_heads, shape.head_dim), dtype=torch.bfloat16, device="cuda")
    flush = L2Flush(torch)
    stream = torch.cuda.current_stream()

    hb, db = B.workspace_size(shape, wl.num_pages, st.batch, T, len(st.page_indices))
    host_ws = torch.empty(hb, dtype=torch.uint8).pin_memory()
    dev_ws = torch.empty(db, dtype=torch.uint8, device="cuda")

    def make_plan():
        return B.asynclm_plan(shape, wl.num_pages, st.q_indptr, st.kv_len_before, st.page_indptr,
                              st.page_indices, host_ws=host_ws, dev_ws=dev_ws)

    plan = make_plan()
    torch.cuda.synchronize()
    launches_per_step = plan.info["launches_append"] + plan.info["launches_attn"]

    def step():
        # the attention kernel is launched with programmatic stream serialization and overlaps its
        # start with the append; the one-call form asynclm_step (append inside the attention kernel)
        # is timed as well and reported beside it (it measures 1-2 us slower)
        B.asynclm_kv_append(plan, kn, vn, pool, stream)
        B.asynclm_attn_mixed(plan, q, pool, out, None, stream)

    sampler = ClockSampler(local) if rank == 0 else None
    for _ in range(max(args.warmup, 3)):
        flush.fill_(1)
        step()
        B.asynclm_step(plan, q, kn, vn, pool, out, None, stream)
    torch.cuda.synchronize()
    assert B.last_device_status(plan) == 0

    # Pass 1 (the reported step time): events around the whole step only, so that the attention kernel
    # may overlap its prologue with the append.
    # The block of K steps is timed `blocks` times in a row, enough for about half a second of timed GPU
    # work, so that the clocks settle; the reported time is that of the median block.
    def timed_block():
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
        for k in range(args.steps):
            flush.fill_(k & 0xff)                 # evict the pool from L2 between steps (untimed)
            ev[k][0].record(stream)
            step()
            ev[k][1].record(stream)
        torch.cuda.synchronize()
        return np.array([e[0].elapsed_time(e[1]) for e in ev])

    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    t_wall0 = time.time()
    first = timed_block()
    blocks = args.blocks if args.blocks > 0 else int(min(100, max(1, np.ceil(500.0 / max(float(first.sum()), 1e-3)))))
    if world > 1:      # every rank times the same number of blocks
        nb = torch.tensor([blocks], device="cuda")
        dist.all_reduce(nb, op=dist.ReduceOp.MAX)
        blocks = int(nb.item())
    all_blocks = [first] + [timed_block() for _ in range(blocks - 1)]
    t_wall1 = time.time()
    if world > 1:
        dist.barrier()
    step_ms = all_blocks[int(np.argsort([b.sum() for b in all_blocks])[len(all_blocks) // 2])]
    total_ms = float(step_ms.sum())
    total_ms = max_over_ranks(total_ms)
    # Pass 2 (roofline of the dominant kernel): the same steps with one more event between the two
    # calls, which gives the duration of asynclm_attn_mixed alone (and serialises it behind the append).
    # Like pass 1 it is repeated block by block and the median block is reported.
    def attn_block():
        ev2 = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
        for k in range(args.steps):
            flush.fill_(k & 0xff)
            B.asynclm_kv_append(plan, kn, vn, pool, stream)
            ev2[k][0].record(stream)
            B.asynclm_attn_mixed(plan, q, pool, out, None, stream)
            ev2[k][1].record(stream)
        torch.cuda.synchronize()
        return np.array([e[0].elapsed_time(e[1]) for e in ev2])

    attn_blocks = [attn_block() for _ in range(blocks)]
    attn_ms = attn_blocks[int(np.argsort([b.sum() for b in attn_blocks])[len(attn_blocks) // 2])]
    t_wall1 = time.time()
    # Pass 3 (context only): no flush between steps.  The pool is larger than L2, so most K/V still
    # comes from DRAM, but the kernels' code and the plan stay cached, as they do between the layers
    # of a model; the reported value stays the flushed one.
    ev3 = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
    for k in range(args.steps):
        ev3[k][0].record(stream)
        step()
        ev3[k][1].record(stream)
    torch.cuda.synchronize()
    t_wall1 = time.time()
    noflush_ms = np.array([e[0].elapsed_time(e[1]) for e in ev3])
    # Pass 4 (context only): the one-call form, asynclm_step
    ev4 = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
    for k in range(args.steps):
        flush.fill_(k & 0xff)
        ev4[k][0].record(stream)
        B.asynclm_step(plan, q, kn, vn, pool, out, None, stream)
        ev4[k][1].record(stream)
    torch.cuda.synchronize()
    t_wall1 = time.time()
    onecall_ms = np.array([e[0].elapsed_time(e[1]) for e in ev4])
    # Read-only ceiling (context): the same K/V blocks, (sequence, kv head) by (sequence, kv head), read
    # with plain loads by a kernel that does nothing else
    ceiling_gbs = None
    if rank == 0:
        n_pg = -(-(st.kv_len_before.astype(np.int64) + st.q_len) // shape.page_size)
        block = shape.page_size * shape.head_dim * 2
        offs = []
        for b in np.nonzero(st.q_len > 0)[0]:
            pages = st.page_indices[st.page_indptr[b]:st.page_indptr[b] + n_pg[b]].astype(np.int64)
            for h in range(shape.num_kv_heads):
                offs.append((pages * 2 * shape.num_kv_heads + h) * block)
        offs_d = torch.from_numpy(np.concatenate(offs)).cuda()
        sink = torch.zeros(1, dtype=torch.int32, device="cuda")
        evc = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(20)]
        for k in range(23):
            flush.fill_(k & 0xff)
            if k >= 3:
                evc[k - 3][0].record(stream)
            B.asynclm_read_ceiling(pool, offs_d, shape.num_kv_heads * block, block, sink, stream)
            if k >= 3:
                evc[k - 3][1].record(stream)
        torch.cuda.synchronize()
        t_wall1 = time.time()
        ceiling_gbs = 2 * block * len(offs_d) / (np.median([e[0].elapsed_time(e[1]) for e in evc]) * 1e-3) / 1e9
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None
    assert B.last_device_status(plan) == 0

    # end to end through the public API: pinned host inputs -> device, plan, append, attention,
    # result back to pinned host memory, every step
    # the step's inputs (q, k_new, v_new) sit back to back in one pinned buffer and go to the device
    # with one copy; the library takes them as three pointers into the device copy
    n_q, n_k = st.q.size, st.k_new.size
    in_h = torch.empty(n_q + 2 * n_k, dtype=torch.int16).pin_memory()
    in_h[:n_q] = torch.from_numpy(st.q.view(np.int16).ravel())
    in_h[n_q:n_q + n_k] = torch.from_numpy(st.k_new.view(np.int16).ravel())
    in_h[n_q + n_k:] = torch.from_numpy(st.v_new.view(np.int16).ravel())
    in_d = torch.empty(n_q + 2 * n_k, dtype=torch.int16, device="cuda")
    q_d = in_d[:n_q].view(torch.bfloat16).view(q.shape)
    kn_d = in_d[n_q:n_q + n_k].view(torch.bfloat16).view(kn.shape)
    vn_d = in_d[n_q + n_k:].view(torch.bfloat16).view(vn.shape)
    out_h = torch.empty((T, shape.num_q_heads, shape.head_dim), dtype=torch.int16).pin_memory()
    e2e_steps = min(args.steps, 200)
    plan_us = []

    def e2e_step():
        in_d.copy_(in_h, non_blocking=True)
        t0 = time.perf_counter()
        p = make_plan()
        plan_us.append((time.perf_counter() - t0) * 1e6)
        B.asynclm_kv_append(p, kn_d, vn_d, pool, stream)
        B.asynclm_attn_mixed(p, q_d, pool, out, None, stream)
        out_h.copy_(out.view(torch.int16), non_blocking=True)
        torch.cuda.synchronize()

    for _ in range(3):
        flush.fill_(2)
        e2e_step()
    plan_us.clear()
    e2e_total = 0.0
    for k in range(e2e_steps):
        flush.fill_(k & 0xff)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        e2e_step()
        e2e_total += time.perf_counter() - t0
    e2e_total = max_over_ranks(e2e_total)
    h2d = in_h.numel() * 2      # + the plan upload (tens of KB)
    d2h = out_h.numel() * 2

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    ms_per_step = total_ms / args.steps
    value = replica_throughput(by["kv"], world, ms_per_step)
    attn_bytes = by["kv"] + by["qo"] + by["page_ids"]
    attn_s = float(attn_ms.mean()) * 1e-3
    achieved = attn_bytes / attn_s / 1e9
    if clocks and clocks.get("sm_mhz"):
        clocks["us_per_step_x_sm_mhz"] = ms_per_step * 1e3 * clocks["sm_mhz"]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": "decode-only-64x[1024,3072]" if args.decode_only else
                        "spans-only-24x[1024,3072]+64" if args.spans_only else WORKLOADS[args.config],
            "seed": wl.seed, "batch": st.batch, "total_q": T,
            "kv_tokens": int(plan.info["total_kv_tokens"]), "replicas": world,
            "l2": L2Flush.NOTE,
            "us_per_step": ms_per_step * 1e3,
            "timed_blocks_of_k_steps": blocks,
            "us_per_step_min_max_over_blocks": [float(min(b.mean() for b in all_blocks)) * 1e3,
                                                float(max(b.mean() for b in all_blocks)) * 1e3],
            "us_per_step_without_l2_flush": float(np.median(noflush_ms)) * 1e3,
            "us_per_step_asynclm_step_one_call": float(onecall_ms.mean()) * 1e3,
            "us_per_step_p10_p50_p90": [float(np.percentile(step_ms, p)) * 1e3 for p in (10, 50, 90)],
            "algorithmic_bytes_per_step": by["total"], "algorithmic_flops_per_step": flops,
            "step_hbm_frac_of_" + peak_kind: by["total"] / (ms_per_step * 1e-3) / 1e9 / peak,
            "step_hbm_frac_of_nominal_8TBps": by["total"] / (ms_per_step * 1e-3) / 1e9 / 8000.0,
            "plan_host_us_median": float(np.median(plan_us)),
            "plan": {k: plan.info[k] for k in ("num_items", "num_split_units", "num_items_tensor",
                                               "kv_chunk_tokens", "num_ctas_cuda", "num_ctas_tensor")},
        },
        "roofline": {"bound": "hbm",
                     "kernel": ("attn_decode_kernel" if args.decode_only else
                                "attn_append_tc_kernel" if args.spans_only else "attn_fused_kernel") +
                               " (asynclm_attn_mixed alone; + lse_merge_kernel if a span unit is split by keys)",
                     "achieved": achieved, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": TRAFFIC_BYTES_PER_LAUNCH if args.config == 2 and not (args.decode_only or args.spans_only) else None,
                     "frac_of_nominal_8TBps": achieved / 8000.0,
                     "read_only_ceiling_gbs": ceiling_gbs,
                     "frac_of_read_only_ceiling": achieved / ceiling_gbs if ceiling_gbs else None,
                     "algorithmic_bytes_per_launch": attn_bytes, "avg_launch_us": attn_s * 1e6},
        "e2e": {"value": world * by["kv"] / (e2e_total / e2e_steps) / 1e9, "unit": UNIT,
                "h2d_bytes_per_step": int(h2d),
                "d2h_bytes_per_step": int(d2h), "us_per_step": e2e_total / e2e_steps * 1e6,
                "steps": e2e_steps, "includes": "H2D of q/k_new/v_new, asynclm_plan (+ its upload), "
                "append, attention, D2H of out"},
        "gpu_launches": int(args.steps * launches_per_step),
        "gpu_launches_note": "pass 1 (timed step); the roofline pass repeats the same launches",
        "clocks": clocks,
    }
    if world == 1 and not args.no_cpu_baseline:
        cb = time_oracle(wl, st, 12.0)
        cb.pop("step_seconds")
        line["cpu_baseline"] = cb
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_replay(args):
    """Config 5: the interrupt-trace replay.  Every step of the trace is planned on the host, appended
    and attended in order (the KV pool grows as the trace goes on); one untimed pass over the trace
    warms up (re-running the appends rewrites the same bytes), the second pass is timed per step."""
    import torch
    from paper_2412_07017_b200 import binding as B
    from paper_2412_07017_b200 import workload as W
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    if int(os.environ.get("RANK", "0")) != 0:
        return
    wl = W.make_config(5)
    shape = wl.shape
    steps = wl.steps[:max(1, min(args.steps, len(wl.steps)))]

    def dev(bits):
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)

    pool = dev(wl.kv_pool)
    dq = [(dev(st.q), dev(st.k_new), dev(st.v_new)) for st in steps]
    max_T = max(st.total_q for st in steps)
    out = torch.empty((max_T, shape.num_q_heads, shape.head_dim), dtype=torch.bfloat16, device="cuda")
    flush = L2Flush(torch)
    stream = torch.cuda.current_stream()
    hb, db = B.workspace_size(shape, wl.num_pages, steps[0].batch, max_T,
                              max(len(st.page_indices) for st in steps))
    host_ws = torch.empty(hb, dtype=torch.uint8).pin_memory()
    dev_ws = torch.empty(db, dtype=torch.uint8, device="cuda")
    sampler = ClockSampler(0)
    plan_us, dev_us, kv_bytes, tot_bytes, spans = [], [], [], [], []
    launches = 0
    for timed in (False, True):
        t_wall0 = time.time()
        for k, st in enumerate(steps):
            t0 = time.perf_counter()
            plan = B.asynclm_plan(shape, wl.num_pages, st.q_indptr, st.kv_len_before, st.page_indptr,
                                  st.page_indices, host_ws=host_ws, dev_ws=dev_ws)
            t1 = time.perf_counter()
            flush.fill_(k & 0xff)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            B.asynclm_kv_append(plan, dq[k][1], dq[k][2], pool, stream)
            B.asynclm_attn_mixed(plan, dq[k][0], pool, out, None, stream)
            e1.record(stream)
            torch.cuda.synchronize()          # the plan workspaces are reused by the next step
            assert B.last_device_status(plan) == 0
            if timed:
                by = W.algorithmic_bytes(shape, st)
                plan_us.append((t1 - t0) * 1e6)
                dev_us.append(e0.elapsed_time(e1) * 1e3)
                kv_bytes.append(by["kv"])
                tot_bytes.append(by["total"])
                spans.append(int((st.q_len > 1).sum()))
                launches += plan.info["launches_append"] + plan.info["launches_attn"]
        t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1)
    peak, peak_kind = measured_peaks()
    dev_us = np.array(dev_us)
    total_s = float(dev_us.sum()) * 1e-6
    line = {
        "metric": METRIC, "value": float(np.sum(kv_bytes)) / total_s / 1e9, "unit": UNIT, "n_gpus": 1,
        "steps": len(steps), "warmup": len(steps), "ms_per_step": float(dev_us.mean()) * 1e-3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": "config5-interrupt-trace-replay", "seed": wl.seed, "batch": steps[0].batch,
            "l2": L2Flush.NOTE,
            "us_per_step_first_median_last": [float(dev_us[0]), float(np.median(dev_us)), float(dev_us[-1])],
            "us_per_step_p10_p90": [float(np.percentile(dev_us, 10)), float(np.percentile(dev_us, 90))],
            "us_per_step_with_interrupts": float(dev_us[np.array(spans) > 0].mean()) if any(spans) else None,
            "us_per_step_decode_only": float(dev_us[np.array(spans) == 0].mean()) if not all(spans) else None,
            "steps_with_interrupts": int((np.array(spans) > 0).sum()),
            "kv_mb_first_last": [kv_bytes[0] / 1e6, kv_bytes[-1] / 1e6],
            "plan_host_us_median": float(np.median(plan_us)),
            "step_hbm_frac_of_" + peak_kind: float(np.sum(tot_bytes)) / total_s / 1e9 / peak,
        },
        "roofline": {"bound": "hbm", "kernel": "whole step (append + attention + merge), all trace steps",
                     "achieved": float(np.sum(tot_bytes)) / total_s / 1e9, "peak": peak, "peak_kind": peak_kind,
                     "unit": "GB/s", "frac": float(np.sum(tot_bytes)) / total_s / 1e9 / peak, "traffic": None},
        "e2e": {"value": float(np.sum(kv_bytes)) / (total_s + float(np.sum(plan_us)) * 1e-6) / 1e9, "unit": UNIT,
                "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                "includes": "asynclm_plan on the host (+ its upload) and the device step; inputs resident"},
        "gpu_launches": int(launches), "clocks": clocks,
    }
    print(json.dumps(line))


def run_timeline(args):
    """Per-CTA timeline of one attention launch of the default workload, from the time-stamp build of
    the library (build.py --trace: -DASYNCLM_TRACE adds a few globaltimer reads per CTA).  Prints one
    JSON line; times are microseconds after the first CTA's entry.  Not a benchmark value."""
    import ctypes
    from paper_2412_07017_b200 import build as lib_build
    os.environ["ASYNCLM_LIBRARY"] = lib_build.build(trace=True)
    import torch
    from paper_2412_07017_b200 import binding as B
    from paper_2412_07017_b200 import workload as W
    torch.cuda.set_device(0)
    if args.spans_only:
        lens = np.random.default_rng(4).integers(1024, 3073, 24).tolist()
        wl = W.make_single_step("spans-only", W.Shape(32, 8, 128, 16), lens, [64] * 24, seed=12)
    else:
        wl = W.make_config(args.config)
    st, shape = wl.steps[0], wl.shape

    def dev(bits):
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)

    pool, q, kn, vn = dev(wl.kv_pool), dev(st.q), dev(st.k_new), dev(st.v_new)
    out = torch.empty((st.total_q, shape.num_q_heads, shape.head_dim), dtype=torch.bfloat16, device="cuda")
    plan = B.asynclm_plan(shape, wl.num_pages, st.q_indptr, st.kv_len_before, st.page_indptr, st.page_indices)
    flush = L2Flush(torch)
    buf = np.zeros((1024, 16), dtype=np.uint64)
    for k in range(6):
        flush.fill_(k)
        B.asynclm_kv_append(plan, kn, vn, pool)
        B.asynclm_attn_mixed(plan, q, pool, out, None)
        torch.cuda.synchronize()
        assert B.load().asynclm_trace_read(ctypes.c_void_p(buf.ctypes.data)) == 0
    n = plan.info["num_ctas_tensor"] if args.spans_only else plan.info["num_ctas_cuda"]
    t = buf[:n].astype(np.int64)
    t0 = t[:, 0].min()
    us = lambda col: (t[:, col] - t0) / 1e3
    span = t[:, 1] > 0
    stats = lambda a: [round(float(x), 1) for x in (a.min(), a.mean(), a.max())] if len(a) else None
    print(json.dumps({
        "workload": "spans-only-24x[1024,3072]+64" if args.spans_only else WORKLOADS.get(args.config, str(args.config)), "ctas": int(n), "span_ctas": int(span.sum()),
        "entry_us_min_mean_max": stats(us(0)),
        "span_body_done_us_min_mean_max": stats(us(1)[span]),
        "first_page_copy_us_mean_ctas_without_span_work": round(float(us(2)[~span].mean()), 1) if (~span).any() else None,
        "consumers_done_us_min_mean_max": stats(us(4)),
        "last_warp_done_us_min_mean_max": stats(us(3)),
        "warp_body_items_per_cta_mean": round(float(t[:, 5].mean()), 1),
        "warp_body_stages_per_cta_mean": round(float(t[:, 6].mean()), 1),
        "split_units_merged_per_cta_mean_max": [round(float(t[:, 7].mean()), 2), int(t[:, 7].max())],
        # span body, SM cycles summed over a CTA's span tiles (CTAs with span work only)
        "span_body_cycles_mean": None if not span.any() else {
            "mma_thread_waits_for_P": round(float(t[span, 8].mean())),
            "mma_thread_waits_for_KV": round(float(t[span, 9].mean())),
            "mma_thread_item_loop": round(float(t[span, 10].mean())),
            "group0_waits_for_S": round(float(t[span, 11].mean())),
            "group1_waits_for_S": round(float(t[span, 15].mean())),
            "group0_softmax_of_tiles": round(float(t[span, 12].mean())),
            "group0_tiles": round(float(t[span, 13].mean()), 1),
            "mma_thread_waits_for_item_start": round(float(t[span, 14].mean())),
            "mma_thread_issues_QK (tensor-only kernel)": round(float(t[span, 2].mean())) if args.spans_only else None,
            "mma_thread_issues_PV (tensor-only kernel)": round(float(t[span, 3].mean())) if args.spans_only else None},
        "plan": {k: plan.info[k] for k in ("num_items", "num_items_tensor", "num_split_units")}}))


def run_trap(args):
    """Trap handler (paper Section 5.4): measures what the keep / swap / recompute rule needs, for one
    layer of the Llama-3-8B attention shape: swap-out + swap-in of a sequence of n tokens through pinned
    host memory (gather kernel, one copy each way) and recomputation of its attention (a span of n
    tokens over an empty context).  Fits swap (linear) and recompute (quadratic) and prints one JSON line
    with the fitted model and the decision table.  Not the benchmarked metric."""
    import torch
    from paper_2412_07017_b200 import binding as B
    from paper_2412_07017_b200 import workload as W
    torch.cuda.set_device(0)
    shape = W.Shape(32, 8, 128, 16)
    lens = [256, 512, 1024, 2048, 4096, 8192]
    num_pages = 2 * max(lens) // 16 + 64
    page_bytes = shape.page_elems * 2
    pool = torch.empty((num_pages, 2, shape.num_kv_heads, 16, shape.head_dim), dtype=torch.bfloat16, device="cuda").normal_()
    perm = np.random.default_rng(1).permutation(num_pages).astype(np.int32)
    stream = torch.cuda.current_stream()
    rows = []
    for n in lens:
        npg = -(-n // 16)
        ids_out, ids_in = perm[:npg], perm[npg:2 * npg]
        staging = torch.empty(B.kv_swap_staging_bytes(shape, num_pages, npg), dtype=torch.uint8, device="cuda")
        image = torch.empty(npg * page_bytes, dtype=torch.uint8).pin_memory()
        q = torch.empty((n, shape.num_q_heads, shape.head_dim), dtype=torch.bfloat16, device="cuda").normal_()
        kn = torch.empty((n, shape.num_kv_heads, shape.head_dim), dtype=torch.bfloat16, device="cuda").normal_()
        out = torch.empty_like(q)
        plan = B.asynclm_plan(shape, num_pages, [0, n], [0], [0, npg], ids_in)
        t_swap, t_gather, t_rec = [], [], []
        for k in range(13):
            e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            e[0].record(stream)
            B.asynclm_kv_swap_out(shape, num_pages, ids_out, pool, staging, image, stream)
            B.asynclm_kv_swap_in(shape, num_pages, ids_in, pool, staging, image, stream)
            e[1].record(stream)
            B.asynclm_step(plan, q, kn, kn, pool, out, None, stream)
            e[2].record(stream)
            torch.cuda.synchronize()
            if k >= 3:
                t_swap.append(e[0].elapsed_time(e[1]) * 1e3)
                t_rec.append(e[1].elapsed_time(e[2]) * 1e3)
        rows.append((n, float(np.median(t_swap)), float(np.median(t_rec)), npg * page_bytes))
    n_arr = np.array([r[0] for r in rows], dtype=np.float64)
    sw = np.polyfit(n_arr, [r[1] for r in rows], 1)
    rc = np.polyfit(n_arr, [r[2] for r in rows], 2)
    model = {"swap_fixed_us": float(sw[1]), "swap_us_per_token": float(sw[0]), "recompute_fixed_us": float(rc[2]),
             "recompute_us_per_token": float(rc[1]), "recompute_us_per_token2": float(rc[0])}
    names = {0: "keep", 1: "swap", 2: "recompute"}
    table = {str(n): {str(w): names[B.asynclm_trap_decide(model, n, w)[0]] for w in (50, 200, 1000, 5000, 100000)}
             for n in (128, 300, 1024, 4096, 16384)}
    print(json.dumps({
        "what": "trap handler: swap-out + swap-in through pinned host memory and attention recompute, one layer, "
                "32/8 heads, head_dim 128 (us per sequence of n tokens)",
        "rows_n_swap_us_recompute_us": [[r[0], round(r[1], 1), round(r[2], 1)] for r in rows],
        "swap_round_trip_gbs": [round(2 * r[3] / (r[1] * 1e-6) / 1e9, 1) for r in rows],
        "model": model, "decision_by_tokens_then_wait_us": table}))


def run_layers(args):
    """A whole decoding step's attention for a model of --layers layers with the Llama-3-8B attention
    shape: one plan per step, then per layer the rotary append into that layer's pool and the mixed
    attention over it (paper Section 4.2 quotes 5-30 ms per output token for whole models; this is the
    attention part).  Every layer has a pool of its own (the default workload's), so a step streams
    layers x 318 MB and nothing of a layer survives in L2 until the next step.  The step is also
    replayed from a CUDA graph.  Prints one JSON line.  Not the benchmarked metric."""
    import torch
    from paper_2412_07017_b200 import binding as B
    from paper_2412_07017_b200 import workload as W
    torch.cuda.set_device(0)
    L = args.layers
    wl = W.make_config(2)
    st, shape = wl.steps[0], wl.shape

    def dev(bits):
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)

    pools = [dev(wl.kv_pool) for _ in range(L)]
    q0, kn, vn = dev(st.q), dev(st.k_new), dev(st.v_new)
    qs = [q0.clone() for _ in range(L)]
    out = torch.empty_like(q0)
    plan = B.asynclm_plan(shape, wl.num_pages, st.q_indptr, st.kv_len_before, st.page_indptr, st.page_indices)
    stream = torch.cuda.current_stream()

    def step(s):
        for l in range(L):
            B.asynclm_kv_append_rope(plan, kn, vn, pools[l], qs[l], 500000.0, s)
            B.asynclm_attn_mixed(plan, qs[l], pools[l], out, None, s)

    def timed(fn, n):
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(n)]
        for k in range(n):
            ev[k][0].record(torch.cuda.current_stream())
            fn()
            ev[k][1].record(torch.cuda.current_stream())
        torch.cuda.synchronize()
        return float(np.median([e[0].elapsed_time(e[1]) for e in ev])) * 1e3

    for _ in range(3):
        step(stream)
    torch.cuda.synchronize()
    eager_us = timed(lambda: step(stream), 20)
    graph_us, graph_note = None, None
    try:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            step(torch.cuda.current_stream())
        g.replay()
        torch.cuda.synchronize()
        graph_us = timed(g.replay, 20)
    except Exception as e:      # capture is an extra; the eager number stands without it
        graph_note = f"capture failed: {type(e).__name__}"
    assert B.last_device_status(plan) == 0
    peak, kind = measured_peaks()
    by = W.algorithmic_bytes(shape, st)
    best = min(x for x in (eager_us, graph_us) if x)
    print(json.dumps({
        "what": f"attention of one decoding step, {L} layers, Llama-3-8B attention shape, default mixed batch",
        "layers": L, "us_per_step_eager": eager_us, "us_per_step_cuda_graph": graph_us, "graph_note": graph_note,
        "us_per_layer": best / L, "kv_gbs": L * by["kv"] / best / 1e3,
        "step_hbm_frac_of_" + kind: L * by["total"] / best / 1e3 / peak,
        "launches_per_step": L * (1 + plan.info["launches_attn"])}))


def run_monitor(args):
    """Token monitor (paper Section 5.1): masked greedy selection + CML state advance over bf16 logits of
    the Llama-3 vocabulary (128 256) for 256 sequences; bound by HBM (one read of the logits).  Prints one
    JSON line.  Not the benchmarked metric."""
    import torch
    from paper_2412_07017_b200 import binding as B
    torch.cuda.set_device(0)
    batch, vocab = 256, 128256
    logits = torch.empty((batch, vocab), dtype=torch.bfloat16, device="cuda").normal_()
    special = {"CALL": 128011, "INTR": 128012, "TRAP": 128013, "END": 128014, "HEAD": 128015}
    # mostly plain text, some sequences inside a function-call block, a few right after [TRAP]
    state = torch.from_numpy(np.random.default_rng(0).choice(4, batch, p=[0.8, 0.08, 0.1, 0.02]).astype(np.int32)).cuda()
    tok, nxt, fl = (torch.empty_like(state) for _ in range(3))
    ws = torch.zeros(B.token_monitor_workspace_bytes(batch), dtype=torch.uint8, device="cuda")
    flush = L2Flush(torch)
    stream = torch.cuda.current_stream()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(50)]
    for k in range(55):
        flush.fill_(k & 0xff)
        if k >= 5:
            ev[k - 5][0].record(stream)
        B.asynclm_token_monitor_step(logits, special, state, tok, nxt, fl, ws, stream)
        if k >= 5:
            ev[k - 5][1].record(stream)
    torch.cuda.synchronize()
    us = float(np.median([e[0].elapsed_time(e[1]) for e in ev])) * 1e3
    peak, kind = measured_peaks()
    nbytes = batch * vocab * 2
    print(json.dumps({"what": "token monitor step, 256 sequences x 128256 bf16 logits", "us_per_step": us,
                      "roofline": {"bound": "hbm", "achieved": nbytes / us / 1e3, "peak": peak, "peak_kind": kind,
                                   "unit": "GB/s", "frac": nbytes / us / 1e3 / peak, "algorithmic_bytes": nbytes},
                      "l2": L2Flush.NOTE}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--blocks", type=int, default=0,
                    help="how many times the block of --steps steps is timed (0 = enough for about 0.5 s of "
                         "timed GPU work; 1 keeps a profiler capture short)")
    ap.add_argument("--config", type=int, default=2, choices=[2, 3, 4, 5],
                    help="synthetic configuration; 2 is the benchmark, 3 and 4 are for reference, "
                         "5 replays the interrupt trace step by step")
    ap.add_argument("--decode-only", action="store_true",
                    help="time a decode-only batch instead (exercises attn_decode_kernel alone)")
    ap.add_argument("--spans-only", action="store_true",
                    help="time a batch in which every sequence gets a 64-token span (attn_append_tc_kernel alone)")
    ap.add_argument("--timeline", action="store_true",
                    help="print a per-CTA timeline of one attention launch (time-stamp build of the library) "
                         "instead of benchmarking")
    ap.add_argument("--trap", action="store_true",
                    help="measure KV swap and attention recompute times and print the trap handler's cost model")
    ap.add_argument("--layers", type=int, default=0,
                    help="time the attention of one decoding step of a model with this many layers instead")
    ap.add_argument("--monitor", action="store_true",
                    help="time the token monitor's masked selection kernel instead")
    args = ap.parse_args()
    if args.layers > 0:
        run_layers(args)
    elif args.monitor:
        run_monitor(args)
    elif args.timeline:
        run_timeline(args)
    elif args.trap:
        run_trap(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.config == 5:
        run_replay(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
