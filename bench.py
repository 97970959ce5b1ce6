#!/usr/bin/env python
"""Benchmark of the sparse MLA decode path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one call of omni_sparse_mla_decode (decode kernel with the split-KV merge: for this
workload the two splits of a request are merged inside the decode kernel, so a step is one
launch) over one batch of the DeepSeek-R1-shaped decode workload (batch 32, 128 heads,
32768-token contexts, 2112 selected tokens per request, shuffled 64-token pages).  Prints ONE
JSON line on rank 0.

Metric: selected-KV bandwidth = 1152 bytes x selected tokens / step time (GB/s), with the step
time in microseconds beside it.  Requests are independent, so with N > 1 every rank runs its own
batch (weak scaling, no collective on the data path) and the value is the sum over ranks divided
by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

KV_ROW_BYTES = 1152
FLOP_PER_TOKEN_HEAD = 2 * (576 + 512)
L2_BYTES = 126 * 1024 * 1024


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm=float(p["hbm_gbs"]), tc_burst=float(p["bf16_tflops"]),
                    tc_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm=6650.0, tc_burst=1590.0, tc_sustained=1400.0, source="fallback")


def _kernel_source_hash():
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2511_22481_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        if not name.endswith(".cuh"):          # device code only: host-side launch logic does not change a kernel
            continue
        if name == "topk_select.cuh":           # the selection producer shares no code with the decode kernels
            continue
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def _recorded_traffic(kernel_hash):
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary, or None if
    there is none or the kernel sources changed since the counters were taken."""
    path = os.path.join(ROOT, "profiles", "dominant_kernel_traffic.json")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        rec = json.load(f)
    if rec.get("kernel_source_hash") != kernel_hash:
        return None
    return rec.get("dram_bytes_per_launch")


class ClockSampler:
    """Samples SM clock and throttle reasons every few milliseconds while the timed region runs
    (NVML from a thread; read-only queries)."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index, period_s=0.02):
        self.index = index
        self.period_s = period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _sample_once(self):
        nv = self.nv
        self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM)))
        try:
            mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
        except Exception:
            mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle)
        for bit, name in self.REASONS.items():
            if mask & bit:
                self.reasons.add(name)

    def _run(self):
        while not self._stop.is_set():
            try:
                self._sample_once()
            except Exception:
                break
            self._stop.wait(self.period_s)

    def start(self):
        if self.nv is None:
            return
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def stop(self):
        if self.nv is None:
            return dict(sm_mhz=None, sm_max_mhz=None, samples=0, reasons=["nvml unavailable"])
        self._stop.set()
        self._thread.join(timeout=2)
        return dict(sm_mhz=statistics.median(self.samples) if self.samples else None, sm_max_mhz=self.max_mhz,
                    samples=len(self.samples), reasons=sorted(self.reasons))


def _oracle_sample(w, target_s=15.0, max_requests=None):
    """Time the CPU oracle, as it stands, on the first requests of the workload (all heads)."""
    import numpy as np
    import torch
    import oracle

    def run(reqs):
        pt = w.page_table[reqs].cpu().numpy()
        si = w.sel_idx[reqs].cpu().numpy()
        sl = w.sel_len[reqs].cpu().numpy()
        rows = oracle.resolve_rows(pt, si, sl, w.page_size, w.num_pages)
        gather = torch.from_numpy(np.where(rows < 0, 0, rows)).to(w.kv_cache.device)
        krows = w.kv_cache.view(-1, w.d_qk)[gather.view(-1)].view(rows.shape[0], -1, w.d_qk).cpu()
        q = w.q[reqs].cpu()
        t0 = time.perf_counter()
        oracle.attend_rows(q, krows, sl, w.d_v, w.scale)
        return time.perf_counter() - t0, int(sl.sum())

    t1, _ = run(slice(0, 1))
    n = max(1, min(w.batch if max_requests is None else max_requests, int(target_s / max(t1, 1e-3))))
    total_t, total_tok, passes = 0.0, 0, 0
    while passes == 0 or (total_t < target_s and passes < 64):
        t, tokens = run(slice(0, n))
        total_t += t
        total_tok += tokens
        passes += 1
    # the float build of the same source, one pass over the same requests (a second CPU figure)
    reqs = slice(0, n)
    pt, si, sl = w.page_table[reqs].cpu().numpy(), w.sel_idx[reqs].cpu().numpy(), w.sel_len[reqs].cpu().numpy()
    rows = oracle.resolve_rows(pt, si, sl, w.page_size, w.num_pages)
    gather = torch.from_numpy(np.where(rows < 0, 0, rows)).to(w.kv_cache.device)
    krows = w.kv_cache.view(-1, w.d_qk)[gather.view(-1)].view(rows.shape[0], -1, w.d_qk).cpu()
    f32_seconds, _, _ = oracle.attend_rows_f32_timed(w.q[reqs].cpu(), krows, sl, w.d_v, w.scale)
    return dict(seconds=total_t, tokens=total_tok, requests=n, passes=passes, cores=oracle.num_threads(),
                f32_seconds=f32_seconds, f32_tokens=int(sl.sum()))


WORKLOAD_HELP = ("config2 (default, the named benchmark) | config1 | config3[:<batch>] | config4 | "
                 "config5:<batch>:<selected>[:dense] (one sweep cell) | "
                 "eq2:<batch>:<n_sink>:<n_recent>[:list] (the paper's sink + recent rule on 32768-token contexts, "
                 "through the range entry point, or with :list through the index-list entry point) | "
                 "rolling:<batch>:<n_sink>:<n_recent> (the same rule over the rolling cache of a compressed layer, "
                 "contexts of one million tokens) | topk_select:<batch>:<ctx>:<k> (the top-k selection producer alone)")


def make_workload(spec, dev, batch):
    """Build a named workload and a one-line description of it.  A trailing ":q8" runs the same
    selection over the 8-bit form of the same pool (omni_sparse_mla_decode_q8)."""
    import numpy as np
    from paper_2511_22481_b200 import workloads as W
    if spec.endswith(":q8"):
        w, text = make_workload(spec[:-3], dev, batch)
        w.meta["entry"] = "q8"
        return w, text + "; 8-bit latent cache (640-byte rows: 512 E4M3 codes + 64 bf16 rope columns, one fp32 scale per row)"
    if spec == "config2":
        w = W.config2_r1(dev, batch=batch)
        text = ("config2 DeepSeek-R1-shaped decode: batch %d/GPU, 128 heads, d_qk 576, d_v 512, ctx 32768, "
                "64-token pages shuffled, 2112 selected tokens/request (page 0 + last 512 + 24 middle pages), seed 1" % batch)
    elif spec == "config1":
        w = W.config1_tiny(dev)
        text = "config1 tiny: batch 1, 16 heads, ctx 4096, identity page table, 832 selected tokens, seed 0"
    elif spec == "config3" or spec.startswith("config3:"):
        n3 = int(spec.split(":")[1]) if ":" in spec else 128          # config3:<batch>: the first requests only (profiling)
        w = W.config3_ragged(dev, batch=n3)
        text = "config3 ragged: batch %d, 128 heads, ctx U[4096,65536], 1/8 of pages selected, seed 2" % n3
    elif spec == "config4":
        w = W.config4_topk(dev)
        text = "config4 token-level top-k: batch 16, 128 heads, ctx 131072, 2048 scattered tokens/request, seed 3"
    elif spec.startswith("config5:"):
        f = spec.split(":")
        w = W.config5_cell(int(f[1]), int(f[2]), dev, dense_variant=(len(f) > 3 and f[3] == "dense"))
        text = "config5 sweep cell: batch %s, %s tokens/request of ctx 65536, 128 heads" % (
            f[1], "all 65536" if len(f) > 3 else f[2])
    elif spec.startswith("eq2:"):
        f = spec.split(":")
        w = W.sink_recent("eq2", 30, int(f[1]), 128, 32768, int(f[2]), int(f[3]), dev)
        w.meta["entry"] = "list" if (len(f) > 4 and f[4] == "list") else "ranges"
        text = ("Eq. 2 selection: batch %s, 128 heads, ctx 32768, N_sink %s + N_recent %s, %s entry point, seed 30"
                % (f[1], f[2], f[3], "index-list" if w.meta["entry"] == "list" else "range"))
    elif spec.startswith("rolling:"):
        from paper_2511_22481_b200 import binding as B
        f = spec.split(":")
        n_sink, n_recent = int(f[2]), int(f[3])
        pages = B.omni_rolling_pages_per_request(n_sink, n_recent)
        # the pool is the whole cache of the layer: pages per request x batch, shuffled; its contents stand
        # for the sink and the last N_recent tokens of a context of one million tokens
        w = W.sink_recent("rolling", 31, int(f[1]), 128, pages * 64, n_sink, n_recent, dev)
        w.ctx_len = np.full(w.batch, 1000000, dtype=np.int64)
        w.meta["entry"] = "rolling"
        text = ("Eq. 2 selection over a rolling cache: batch %s, 128 heads, ctx 1000000, N_sink %d + N_recent %d, "
                "%d pages per request, seed 31" % (f[1], n_sink, n_recent, pages))
    else:
        raise SystemExit("unknown --workload %r; choose %s" % (spec, WORKLOAD_HELP))
    return w, text


def topk_arm(args, spec):
    """`--workload topk_select:<batch>:<ctx>:<k>`: the selection producer alone (one launch per
    step), scores of standard-normal noise, one GPU.  Same JSON shape as the decode arm."""
    import numpy as np
    import torch
    from paper_2511_22481_b200 import binding as B
    from paper_2511_22481_b200 import build as builder

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    parts = spec.split(":")
    batch, ctx, k = (int(parts[1]), int(parts[2]), int(parts[3])) if len(parts) == 4 else (16, 131072, 2048)
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    builder.build()
    B.load()
    score_bytes = batch * ctx * 4
    clones = max(2, -(-3 * L2_BYTES // score_bytes))           # bytes between two uses of a copy: 3 x L2
    gen = torch.Generator(device="cpu").manual_seed(3)
    scores_h = [torch.randn(batch, ctx, generator=gen).pin_memory() for _ in range(min(clones, 4))]
    scores = [scores_h[i % len(scores_h)].to(dev) for i in range(clones)]
    ctx_len = torch.full((batch,), ctx, dtype=torch.int32, device=dev)
    sel_idx = torch.zeros(batch, k, dtype=torch.int32, device=dev)
    sel_len = torch.zeros(batch, dtype=torch.int32, device=dev)
    algo_bytes = score_bytes + batch * 4 + batch * min(k, ctx) * 4 + batch * 4

    def step(i):
        B.omni_topk_select(scores[i % clones], ctx_len, k, sel_idx, sel_len)

    for i in range(args.warmup):
        step(i)
    sampler = ClockSampler(0)
    torch.cuda.synchronize()
    sampler.start()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for i in range(args.steps):
        step(args.warmup + i)
    t1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = t0.elapsed_time(t1) / args.steps

    idx_h = torch.empty(batch, k, dtype=torch.int32).pin_memory()
    len_h = torch.empty(batch, dtype=torch.int32).pin_memory()
    stage = torch.empty(batch, ctx, device=dev)

    def e2e_step(i):
        stage.copy_(scores_h[i % len(scores_h)], non_blocking=True)
        B.omni_topk_select(stage, ctx_len, k, sel_idx, sel_len)
        idx_h.copy_(sel_idx, non_blocking=True)
        len_h.copy_(sel_len, non_blocking=True)

    for i in range(args.warmup):
        e2e_step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2e_steps = min(args.steps, 500)
    e0.record()
    for i in range(e2e_steps):
        e2e_step(i)
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps

    peaks = _peaks()
    achieved = algo_bytes / (ms * 1e-3) / 1e9
    line = {
        "metric": "top-k selection producer: score bytes consumed per second", "value": round(achieved, 2), "unit": "GB/s",
        "us_per_step": round(ms * 1e3, 3), "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": round(ms, 6), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u32 keys of f32 scores", "data": "synthetic",
        "config": {"workload": "topk_select: batch %d, %d scores per request (standard normal, seed 3), k=%d" % (batch, ctx, k),
                   "l2": "cold: %d score copies rotated (%.0f MB per cycle vs %.0f MB L2)"
                         % (clones, clones * score_bytes / 1e6, L2_BYTES / 1e6)},
        "clocks": clocks,
        "e2e": {"value": round(algo_bytes / (e2e_ms * 1e-3) / 1e9, 2), "unit": "GB/s", "us_per_step": round(e2e_ms * 1e3, 3),
                "h2d_bytes_per_step": score_bytes, "d2h_bytes_per_step": batch * k * 4 + batch * 4},
        "gpu_launches": args.steps,
        "roofline": {"bound": "hbm", "achieved": round(achieved, 2), "peak": peaks["hbm"], "unit": "GB/s",
                     "frac": round(achieved / peaks["hbm"], 4), "traffic": None, "peak_source": peaks["source"],
                     "kernel": "topk_select_kernel", "kernel_us_mean": round(ms * 1e3, 3),
                     "algorithmic_bytes_per_launch": algo_bytes},
    }
    if not args.no_cpu_baseline:
        from oracle.topk import topk_batch
        sc = scores_h[0].numpy()
        n, t_begin = 0, time.perf_counter()
        while time.perf_counter() - t_begin < 10.0:
            topk_batch(sc, [ctx] * batch, k)
            n += 1
        secs = time.perf_counter() - t_begin
        line["cpu_baseline"] = {"value": round(n * algo_bytes / secs / 1e9, 5), "unit": "GB/s", "cores": 1, "kind": "oracle",
                                "sample": "oracle top-k (numpy lexsort) on the whole batch, %d passes in %.1f s" % (n, secs)}
    print(json.dumps(line), flush=True)
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--batch", type=int, default=32, help="requests per GPU (32 = the named workload; smaller for profiling)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--kernel", default="tc", choices=["tc", "simt"],
                    help="tc: tensor-core kernel (the product path); simt: plain-FMA bring-up kernel")
    ap.add_argument("--clones", type=int, default=6, help="KV pool copies rotated to keep L2 cold")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-lanes", type=int, default=2,
                    help="end-to-end leg: how many steps are in flight, each on its own stream and buffers")
    ap.add_argument("--workload", default="config2", help=WORKLOAD_HELP)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank != 0:
            return 0
        return reference_arm(args)
    if args.workload.startswith("topk_select"):
        if rank != 0:
            return 0
        return topk_arm(args, args.workload)

    import torch
    import torch.distributed as dist
    from paper_2511_22481_b200 import binding as B
    from paper_2511_22481_b200 import build as builder
    from paper_2511_22481_b200 import workloads as W

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)
    builder.build()
    B.load()

    flags = B.OMNI_FLAG_SIMT if args.kernel == "simt" else 0
    w, workload_text = make_workload(args.workload, dev, args.batch)
    # keep L2 cold: rotate over independent copies of the pool so the bytes touched between two
    # uses of the same copy exceed L2 several times
    clones = max(2, args.clones)
    while clones > 2 and clones * w.kv_cache.numel() * 2 > 40e9:      # keep the rotated copies within 40 GB
        clones -= 1
    q8 = w.meta.get("entry") == "q8"
    if q8:
        # the same pool in its 8-bit form; the bf16 copy is released
        rows = w.kv_cache.view(-1, w.d_qk)
        cache = torch.empty((rows.shape[0], B.OMNI_Q8_ROW_BYTES), dtype=torch.uint8, device=dev)
        scale = torch.empty((rows.shape[0],), dtype=torch.float32, device=dev)
        B.omni_kv_quantize_q8(rows, cache, scale)
        torch.cuda.synchronize()
        w.kv_cache = None
        pools = [(cache, scale)] + [(cache.clone(), scale.clone()) for _ in range(clones - 1)]
    else:
        pools = [w.kv_cache] + [w.kv_cache.clone() for _ in range(clones - 1)]
    plan = B.plan_for(w, flags=flags)
    # algorithmic bytes per selected token: the row as stored (and, for the 8-bit cache, its scale)
    row_bytes = (B.OMNI_Q8_ROW_BYTES + 4) if q8 else KV_ROW_BYTES
    kv_bytes = w.selected_tokens * row_bytes
    flops = w.selected_tokens * w.heads * FLOP_PER_TOKEN_HEAD
    launches_per_step = B.omni_sparse_mla_num_launches(plan.desc)

    ranges = w.meta.get("entry") in ("ranges", "rolling")
    range_entry = (B.omni_sparse_mla_decode_rolling if w.meta.get("entry") == "rolling"
                   else B.omni_sparse_mla_decode_sink_recent)
    ctx_dev = torch.as_tensor(w.ctx_len, dtype=torch.int32).to(dev) if ranges else None

    # The index-list workloads go through the planned entry point: one plan per pool copy, made
    # once (split plan, tensor maps), and the per-step C call with its arguments marshalled once,
    # so that a step costs the host one foreign call and one kernel launch.
    planned = None
    if q8:
        def q8_call(pool):
            cache_i, scale_i = pool
            return lambda: B.omni_sparse_mla_decode_q8(plan.desc, w.q, cache_i, scale_i, w.page_table, w.sel_idx, w.sel_len,
                                                       plan.out, plan.lse, plan.workspace, plan.status)
        planned = [q8_call(pool) for pool in pools]
    elif not ranges:
        stream = torch.cuda.current_stream()
        planned = [B.bind_planned(B.omni_sparse_mla_plan_init(plan.desc, w.q, pool), w.page_table, w.sel_idx,
                                  w.sel_len, plan.out, plan.lse, plan.workspace, plan.status, stream)
                   for pool in pools]

    def step(i, ev=None):
        if ev is not None:
            B.omni_sparse_mla_set_profile_events(ev[0], ev[1])
        if ranges:
            range_entry(plan.desc, w.q, pools[i % clones], w.page_table, ctx_dev, w.meta["n_sink"],
                        w.meta["n_recent"], plan.out, plan.lse, plan.workspace, plan.status)
        else:
            planned[i % clones]()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing --------------------------------------------------------
    sampler = ClockSampler(local_rank)
    sampler.start()                           # before the warm-up, so that short timed regions are sampled too
    for i in range(args.warmup):
        step(i)
    # what the harness itself needs is made before the timed region opens: the events exist (a first
    # record creates them) and the list of per-step calls is built
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_begin.record()
    t_end.record()
    calls = [planned[(args.warmup + i) % clones] for i in range(args.steps)] if planned is not None else None
    barrier()
    t_begin.record()
    host_t0 = time.perf_counter()
    if planned is not None:
        for call in calls:
            call()
    else:
        for i in range(args.steps):
            step(args.warmup + i)
    host_us_per_call = (time.perf_counter() - host_t0) / args.steps * 1e6
    t_end.record()
    barrier()
    # the decode kernel alone, bracketed by its own events, on a few extra steps outside the timed
    # region (an event between two launches stops them from overlapping, so it must not sit there)
    n_bracketed = max(8, min(64, args.steps))
    kern_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_bracketed)]
    for a, b in kern_ev:                      # materialise the events before handing them to C
        a.record()
        b.record()
    for i in range(n_bracketed):
        step(args.warmup + args.steps + i, kern_ev[i])
    barrier()
    B.omni_sparse_mla_set_profile_events(None, None)
    clocks = sampler.stop()
    ms_total = t_begin.elapsed_time(t_end)
    kern_ms = [a.elapsed_time(b) for a, b in kern_ev]
    status = int(plan.status.item())
    if status != 0:
        raise SystemExit("device status word is %d after the timed region" % status)

    # ---- end to end through the host-buffer entry point ---------------------------------
    staging = torch.empty(B.omni_sparse_mla_host_staging_bytes(plan.desc), dtype=torch.uint8, device=dev)
    q_h, pt_h = w.q.cpu().pin_memory(), w.page_table.cpu().pin_memory()
    si_h, sl_h = w.sel_idx.cpu().pin_memory(), w.sel_len.cpu().pin_memory()
    out_h = torch.empty(plan.out.shape, dtype=torch.bfloat16).pin_memory()
    lse_h = torch.empty(plan.lse.shape, dtype=torch.float32).pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in (q_h, pt_h, si_h, sl_h))
    d2h = sum(t.numel() * t.element_size() for t in (out_h, lse_h))

    if q8:
        # no host-buffer entry point for the 8-bit cache: the same copies issued around the device call
        q_d, pt_d, si_d, sl_d = (torch.empty_like(t, device=dev) for t in (q_h, pt_h, si_h, sl_h))

        def e2e_step(i):
            for dst, src in ((q_d, q_h), (pt_d, pt_h), (si_d, si_h), (sl_d, sl_h)):
                dst.copy_(src, non_blocking=True)
            cache_i, scale_i = pools[i % clones]
            B.omni_sparse_mla_decode_q8(plan.desc, q_d, cache_i, scale_i, pt_d, si_d, sl_d, plan.out, plan.lse,
                                        plan.workspace, plan.status)
            out_h.copy_(plan.out, non_blocking=True)
            lse_h.copy_(plan.lse, non_blocking=True)
    else:
        # Two steps in flight: consecutive steps go to two streams in turn, each with its own staging
        # area, host result buffers and workspace, so that the copies out of one step overlap the
        # copies in of the next (PCIe carries both directions at once).  Every step still moves all of
        # its inputs in and all of its results out.
        lanes = []
        for k in range(max(1, args.e2e_lanes)):
            lanes.append({
                "stream": torch.cuda.Stream(device=dev),
                "staging": staging if k == 0 else torch.empty_like(staging),
                "out_h": out_h if k == 0 else torch.empty_like(out_h).pin_memory(),
                "lse_h": lse_h if k == 0 else torch.empty_like(lse_h).pin_memory(),
                "ws": plan.workspace if k == 0 or plan.workspace is None else torch.empty_like(plan.workspace),
            })
        e2e_lanes = len(lanes)

        def e2e_step(i):
            ln = lanes[i % e2e_lanes]
            B.omni_sparse_mla_decode_host(plan.desc, q_h, pools[i % clones], pt_h, si_h, sl_h, ln["out_h"],
                                          ln["lse_h"], ln["staging"], ln["ws"], plan.status, ln["stream"])

    def fork_lanes():
        if not q8:
            for ln in lanes:
                ln["stream"].wait_stream(torch.cuda.current_stream())

    def join_lanes():
        if not q8:
            for ln in lanes:
                torch.cuda.current_stream().wait_stream(ln["stream"])

    e2e_steps = args.steps
    # the PCIe path needs some tens of milliseconds of traffic to reach its steady rate (the first few
    # hundred steps after an idle period run 5 to 40 % slower), so this leg warms up with at least
    # 500 steps whatever W is (untimed, like every warm-up step)
    e2e_warmup = max(args.warmup, 500)
    fork_lanes()
    for i in range(e2e_warmup):
        e2e_step(i)
    join_lanes()
    barrier()
    e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e_begin.record()
    fork_lanes()
    for i in range(e2e_steps):
        e2e_step(args.warmup + i)
    join_lanes()
    e_end.record()
    barrier()
    e2e_ms_total = e_begin.elapsed_time(e_end)

    # ---- reduce over ranks: slowest rank's time, all ranks' bytes ------------------------
    from paper_2511_22481_b200 import dp
    (ms_total, e2e_ms_total), job_bytes = dp.job_throughput([ms_total, e2e_ms_total], kv_bytes, device=dev)
    ms_per_step = ms_total / args.steps
    e2e_ms_per_step = e2e_ms_total / e2e_steps
    value = job_bytes / (ms_per_step * 1e-3) / 1e9
    e2e_value = job_bytes / (e2e_ms_per_step * 1e-3) / 1e9

    if rank == 0:
        peaks = _peaks()
        kbracket = statistics.mean(kern_ms)
        # Average launch duration of the dominant kernel.  When a step is that one launch, the
        # timed region (K back-to-back launches between two events) gives it directly; bracketing
        # single launches with their own events adds the event and launch overhead to each and
        # stops consecutive launches from overlapping, so that figure is kept beside it.  With a
        # separate merge kernel in the step, the bracketed figure is the only per-kernel one.
        kmean = ms_per_step if launches_per_step == 1 else kbracket
        achieved = kv_bytes / (kmean * 1e-3) / 1e9
        khash = _kernel_source_hash()
        tflops = flops / (kmean * 1e-3) / 1e12
        line = {
            "metric": "sparse MLA decode selected-KV bandwidth (us/step beside it)",
            "value": round(value, 2), "unit": "GB/s", "us_per_step": round(ms_per_step * 1e3, 3),
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(ms_per_step, 6), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "e4m3 cache, bf16 q and out, fp32 accumulate" if q8 else "bf16", "data": "synthetic",
            "config": {"workload": workload_text,
                       "selected_tokens_per_gpu": w.selected_tokens, "kv_bytes_per_step_per_gpu": kv_bytes,
                       "kv_bytes_per_token": row_bytes,
                       "splits": plan.splits, "kernel": args.kernel, "launches_per_step": launches_per_step,
                       "entry": ("omni_sparse_mla_decode_q8" if q8 else "omni_sparse_mla_decode_planned" if planned is not None
                                 else "range entry point"),
                       "l2": "cold: %d pool copies rotated (%.0f MB touched per cycle vs %.0f MB L2)"
                             % (clones, clones * kv_bytes / 1e6, L2_BYTES / 1e6),
                       "parallelism": "dp%d (independent requests, no collective)" % world},
            "clocks": clocks,
            "e2e": {"value": round(e2e_value, 2), "unit": "GB/s",
                    "us_per_step": round(e2e_ms_per_step * 1e3, 3),
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "note": "omni_sparse_mla_decode_host: q, page_table, sel_idx, sel_len copied from pinned "
                            "host memory and out, lse copied back every step; the KV cache is persistent "
                            "device state" + ("" if q8 else "; consecutive steps take turns on several "
                                                      "streams (own staging, result buffers and workspace each), so one "
                                                      "step's copies out overlap the next step's copies in"),
                    "steps_in_flight": 1 if q8 else max(1, args.e2e_lanes), "warmup_steps": e2e_warmup},
            "gpu_launches": launches_per_step * args.steps,
            "host_us_per_call": round(host_us_per_call, 3),
            "launch_bound": bool(host_us_per_call > 0.9 * ms_per_step * 1e3),
            "roofline": {"bound": "hbm", "achieved": round(achieved, 2), "peak": peaks["hbm"],
                         "unit": "GB/s", "frac": round(achieved / peaks["hbm"], 4),
                         "traffic": (_recorded_traffic(khash) if args.workload == "config2" and args.batch == 32 else None),
                         "peak_source": peaks["source"],
                         "kernel": "sparse_mla_decode main kernel (128 heads: tc2_decode_cm_kernel where two splits merge inside a cluster, as on the bench workload, else tc2_decode_kernel)", "kernel_us_mean": round(kmean * 1e3, 3),
                         "kernel_us_bracketed_min": round(min(kern_ms) * 1e3, 3),
                         "kernel_us_bracketed_mean": round(kbracket * 1e3, 3),
                         "kernel_us_source": ("timed region / steps (one launch per step)" if launches_per_step == 1
                                              else "events around the decode kernel on extra steps after the timed region"),
                         "algorithmic_bytes_per_launch": kv_bytes,
                         "tensor_tflops": round(tflops, 2),
                         "tensor_frac_of_sustained": round(tflops / peaks["tc_sustained"], 4),
                         "roofline_us": round(max(kv_bytes / peaks["hbm"] / 1e3, flops / peaks["tc_sustained"] / 1e6), 3),
                         "frac_of_slower_bound": round(max(kv_bytes / peaks["hbm"] / 1e3, flops / peaks["tc_sustained"] / 1e6)
                                                       / (kmean * 1e3), 4),
                         "frac_of_nominal_8TBs": round(achieved / 8000.0, 4),
                         "kernel_source_hash": khash},
        }
        if world == 1 and not args.no_cpu_baseline and not q8:
            s = _oracle_sample(w)
            cpu_value = s["tokens"] * KV_ROW_BYTES / s["seconds"] / 1e9
            line["cpu_baseline"] = {
                "value": round(cpu_value, 5), "unit": "GB/s", "cores": s["cores"], "kind": "oracle",
                "sample": "fp64 oracle on the first %d of %d requests, all 128 heads, %d passes (%d selected tokens in all), "
                          "%.1f s; one full step extrapolates to %.0f us"
                          % (s["requests"], w.batch, s["passes"], s["tokens"], s["seconds"],
                             s["seconds"] / s["tokens"] * w.selected_tokens * 1e6),
                "fp32_build": {"value": round(s["f32_tokens"] * KV_ROW_BYTES / s["f32_seconds"] / 1e9, 5), "unit": "GB/s",
                               "note": "the same oracle source compiled with float as its working type, one pass over "
                                       "the same requests; timed only, never a reference"}}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0


def reference_topk_arm(args):
    """The top-k oracle timed on one host core; each step is the whole batch of the workload."""
    import torch
    from oracle.topk import topk_batch
    parts = args.workload.split(":")
    batch, ctx, k = (int(parts[1]), int(parts[2]), int(parts[3])) if len(parts) == 4 else (16, 131072, 2048)
    scores = torch.randn(batch, ctx, generator=torch.Generator().manual_seed(3)).numpy()
    algo_bytes = batch * ctx * 4 + batch * 4 + batch * min(k, ctx) * 4 + batch * 4
    steps = max(1, min(args.steps, 50))
    for _ in range(min(args.warmup, 3)):
        topk_batch(scores, [ctx] * batch, k)
    t0 = time.perf_counter()
    for _ in range(steps):
        topk_batch(scores, [ctx] * batch, k)
    secs = time.perf_counter() - t0
    value = steps * algo_bytes / secs / 1e9
    line = {
        "impl": "reference", "metric": "top-k selection producer: score bytes consumed per second",
        "value": round(value, 5), "unit": "GB/s", "n_gpus": args.gpus, "steps": steps, "warmup": min(args.warmup, 3),
        "ms_per_step": round(secs / steps * 1e3, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32 scores", "data": "synthetic",
        "config": {"workload": "topk_select: batch %d, %d scores per request (standard normal, seed 3), k=%d" % (batch, ctx, k)},
        "cpu_baseline": {"value": round(value, 5), "unit": "GB/s", "cores": 1, "kind": "oracle",
                         "sample": "oracle top-k (numpy lexsort) on the whole batch, %d steps (capped at 50)" % steps},
        "e2e": {"value": round(value, 5), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)
    return 0


def reference_arm(args):
    """The oracle as the reference implementation, timed on host cores on a bounded sample."""
    import torch
    from paper_2511_22481_b200 import workloads as W

    if args.workload.startswith("topk_select"):
        return reference_topk_arm(args)
    # inputs of the same workload; a reduced pool is enough because only selected rows are read
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    w, _ = make_workload(args.workload, dev, args.batch)
    per_step = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    times, tokens = [], 0
    for i in range(args.warmup + args.steps):
        s = _oracle_sample(w, target_s=per_step)
        if i >= args.warmup:
            times.append(s["seconds"])
            tokens += s["tokens"]
    total = sum(times)
    value = tokens * KV_ROW_BYTES / total / 1e9
    ms_per_step_full = total / tokens * w.selected_tokens * 1e3
    line = {
        "impl": "reference", "metric": "sparse MLA decode selected-KV bandwidth (us/step beside it)",
        "value": round(value, 5), "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_per_step_full, 3), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "config2 DeepSeek-R1-shaped decode (same as the CUDA arm); each step is a "
                               "bounded sample of its requests, ms_per_step extrapolated to the full batch"},
        "cpu_baseline": {"value": round(value, 5), "unit": "GB/s", "cores": s["cores"], "kind": "oracle",
                         "sample": "%d requests x 128 heads per step, %.1f s per step" % (s["requests"], total / len(times))},
        "e2e": {"value": round(value, 5), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)
    return 0


if __name__ == "__main__":
    sys.exit(main())
