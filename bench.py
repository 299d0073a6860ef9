#!/usr/bin/env python
"""Benchmark of the sparse decode hot path: decode tokens/s on synthetic Llama-3-8B-shaped workloads.

A "step" is one decode step of the whole path: for each of the L layers, attention over the set gathered
for it, the selection of the next step's set from the speculated token, and the host->HBM gather of a
later layer on the side stream (dd_decode_layer_step). `value` counts output tokens only (B per step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl ours|reference]

N > 1 (under torchrun) runs N independent replicas, one per GPU: the path has no exchange step.
`--impl reference` times the CPU oracle on the host cores instead (a deliberately slow program).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# per-launch traffic from the committed ncu captures (config 2 layer: 64 MiB gathered, 32 MiB of landmarks)
NCU_TRAFFIC = {"gather_dram": 38.7e3 + 9.36e6, "gather_sysmem": 2097152 * 32, "attn_dram": 67.33e6 + 0.95e6,
               "select_dram": 33.68e6}

METRIC = "decode_tokens_per_s"
UNIT = "tok/s"


def log(msg):
    print(f"[bench] {msg}", file=sys.stderr, flush=True)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=32)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=2, help="workload number (2 = batch 8, 32K context, budget 2048)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--phys-layers", type=int, default=0, help="distinct layers kept in the host store (0 = as many as fit)")
    ap.add_argument("--ring-depth", type=int, default=2)
    ap.add_argument("--gather-mode", default="loads", choices=["loads", "bulk"])
    ap.add_argument("--gather-ctas", type=int, default=0)
    ap.add_argument("--attn-splits", type=int, default=0)
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiling of small cases only)")
    ap.add_argument("--batch", type=int, default=0, help="override the batch (profiling of small cases only)")
    ap.add_argument("--correct-misses", action="store_true",
                    help="repair prediction misses on an urgent stream before attention (not the headline path)")
    ap.add_argument("--urgent-fifo", action="store_true",
                    help="with --correct-misses: queue the missing pages on the prefetch stream (single FIFO) instead "
                         "of a high-priority stream of their own")
    ap.add_argument("--spec-fidelity", type=float, default=None,
                    help="override the generator's correlation between a step's speculated query and the next "
                         "step's current query (lower = more prediction misses)")
    ap.add_argument("--landmark-chunk", type=int, default=0,
                    help="tokens per landmark: 0/16 = one per page (default), 8/4/2/1 = several per page")
    ap.add_argument("--no-select-stream", action="store_true",
                    help="run the next-step selection on the compute stream instead of a stream of its own")
    ap.add_argument("--ragged", action="store_true", help="unequal context lengths per request (second workload shape)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-stages", action="store_true")
    return ap.parse_args()


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows, self.proc = [], None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(index)], stdout=subprocess.PIPE, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self) -> dict:
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
            except Exception:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# --------------------------------------------------------------------------------------------------
# CPU oracle legs
# --------------------------------------------------------------------------------------------------
def oracle_sample(w, n_layers_cap=4, min_seconds=10.0, max_steps_per_layer=12):
    """Times the oracle, as it stands, on whole layers of the workload (all requests): selection from the
    speculated token, page gather, attention of both tokens. A few layers' slabs are drawn; each is run
    for several steps of fresh queries until about `min_seconds` of oracle work has been timed. Returns
    tok/s scaled to full steps of w.n_layers layers."""
    import torch
    from oracle import dd_oracle as orc
    from paper_2607_26475_b200 import workloads as wl
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threads = 1
    ctx_len = wl.ctx_lens(w).numpy()
    npg = (ctx_len + w.page_tokens - 1) // w.page_tokens
    n_units, t_total, layers = 0, 0.0, 0
    split = {"select": 0.0, "gather": 0.0, "attn": 0.0}
    while layers < n_layers_cap and (layers == 0 or t_total < min_seconds):
        l = layers
        kv32 = torch.stack([wl.kv_slab(w, l, b) for b in range(w.batch)]).float().numpy()
        lm = orc.build_landmarks(kv32[:, :, :, 0], ctx_len)             # set-up, not timed
        for step in range(max_steps_per_layer):
            q = wl.queries(w, step, l).float().numpy()
            t0 = time.perf_counter()
            idx, _ = orc.select_topk(q[:, 1], lm, npg, w.k_pages, w.forced_recent_pages)
            t1 = time.perf_counter()
            slot = orc.gather_kv(kv32, idx)
            t2 = time.perf_counter()
            orc.sparse_decode_attn(q, slot, idx, ctx_len, w.page_tokens)
            t3 = time.perf_counter()
            split["select"] += t1 - t0
            split["gather"] += t2 - t1
            split["attn"] += t3 - t2
            t_total += t3 - t0
            n_units += 1
            if t_total >= min_seconds:
                break
        layers += 1
        del kv32, lm
    per_layer = t_total / n_units
    value = w.batch / (per_layer * w.n_layers)
    return {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{n_units} layer-steps (all {w.batch} requests; {layers} layer(s) x up to {max_steps_per_layer} "
                      f"steps) of {w.name}, scaled to {w.n_layers} layers per step",
            "us_per_layer": {k: v / n_units * 1e6 for k, v in split.items()}, "seconds": t_total}


def run_reference(args):
    """The oracle arm: each step is one layer (all requests) of the workload through the oracle — selection
    from the speculated token, page gather, attention — scaled to the layers of a full step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    from oracle import dd_oracle as orc
    from paper_2607_26475_b200 import workloads as wl
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threads = 1
    w = wl.CONFIGS[args.config]
    ctx_len = wl.ctx_lens(w).numpy()
    npg = (ctx_len + w.page_tokens - 1) // w.page_tokens
    kv32 = torch.stack([wl.kv_slab(w, 0, b) for b in range(w.batch)]).float().numpy()     # set-up, not timed
    lm = orc.build_landmarks(kv32[:, :, :, 0], ctx_len)
    warm = max(0, min(args.warmup, 2))
    times = []
    t_begin = time.time()
    for step in range(warm + args.steps):
        q = wl.queries(w, step, 0).float().numpy()
        t0 = time.perf_counter()
        idx, _ = orc.select_topk(q[:, 1], lm, npg, w.k_pages, w.forced_recent_pages)
        slot = orc.gather_kv(kv32, idx)
        orc.sparse_decode_attn(q, slot, idx, ctx_len, w.page_tokens)
        dt = time.perf_counter() - t0
        if step >= warm:
            times.append(dt)
        if time.time() - t_begin > 200:
            break
    per_layer = sum(times) / len(times)
    ms = per_layer * w.n_layers * 1e3
    value = w.batch / (ms * 1e-3)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": len(times), "warmup": warm, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "batch": w.batch, "ctx": w.ctx, "budget": w.budget, "layers": w.n_layers,
                       "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim,
                       "page_tokens": w.page_tokens, "parallelism": "host cores only",
                       "generator": {k: v for k, v in w.params().items() if k in (
                           "structure", "planted_frac", "zipf_a", "topic_gain", "planted_noise", "query_topic", "seed")}},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": f"each step = 1 layer x all {w.batch} requests with fresh queries, scaled to "
                                       f"{w.n_layers} layers"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------------
def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    import torch
    import torch.distributed as dist
    from paper_2607_26475_b200 import binding as dd
    from paper_2607_26475_b200 import workloads as wl
    from paper_2607_26475_b200 import replicas
    from paper_2607_26475_b200.store import HostStore, available_host_bytes

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        try:    # keep this replica's threads (and so its pinned store) on the CPUs next to its GPU
            import pynvml
            pynvml.nvmlInit()
            pynvml.nvmlDeviceSetCpuAffinity(pynvml.nvmlDeviceGetHandleByIndex(local_rank))
        except Exception as e:
            log(f"rank {rank}: CPU affinity not set ({e})")
    w = wl.CONFIGS[args.config]
    if args.layers or args.batch:
        w = wl.small(w, n_layers=args.layers or w.n_layers, batch=args.batch or w.batch)
    if args.spec_fidelity is not None:
        w = wl.small(w, spec_fidelity=args.spec_fidelity)
    L, B, K, W = w.n_layers, w.batch, args.steps, max(args.warmup, 0)
    hbm_peak, peak_src = measured_peaks()

    compute = torch.cuda.Stream()
    copy = torch.cuda.Stream(priority=0)
    urgent = None
    if args.correct_misses:
        urgent = copy if args.urgent_fifo else torch.cuda.Stream(priority=-1)
    gm = dd.DD_GATHER_BULK if args.gather_mode == "bulk" else dd.DD_GATHER_LOADS
    ctx = dd.Context(n_layers=L, batch=B, max_pages=w.n_pages, k_pages=w.k_pages,
                     forced_recent_pages=w.forced_recent_pages, ring_depth=args.ring_depth, gather_mode=gm,
                     gather_ctas=args.gather_ctas, attn_splits=args.attn_splits, compute_stream=compute, copy_stream=copy,
                     miss_correction=args.correct_misses, urgent_stream=urgent, landmark_chunk_tokens=args.landmark_chunk,
                     select_stream=None if args.no_select_stream else torch.cuda.Stream())
    budget = replicas.host_budget_per_rank(available_host_bytes(), world)
    store = HostStore(w, ctx, n_phys_layers=args.phys_layers or None, ragged=args.ragged, host_budget_bytes=budget,
                      log=log if rank == 0 else None)
    store.bind(ctx)
    if rank == 0:
        log(f"{w.name}: host store {store.host_bytes / 2**30:.1f} GiB pinned in {store.n_phys} physical layer(s), "
            f"built in {store.build_seconds:.1f} s; ring {ctx.ring_bytes() / 2**20:.0f} MiB, scratch {ctx.scratch_bytes() / 2**20:.1f} MiB")

    # queries of every step (fresh each step), resident in HBM and also in pinned host memory for the e2e leg
    n_q = W + K
    q_host = torch.empty((n_q, L, B, 2, w.n_q_heads, w.head_dim), dtype=torch.bfloat16, pin_memory=True)
    for t in range(n_q):
        for l in range(L):
            q_host[t, l] = wl.queries(w, t, l)
    q_dev = q_host.cuda()
    q_init = torch.stack([wl.queries(w, -1, l)[:, 1] for l in range(L)]).cuda()
    outs = torch.zeros((L, B, 2, w.n_q_heads, w.head_dim), dtype=torch.bfloat16, device="cuda")
    out_host = torch.empty(outs.shape, dtype=torch.bfloat16, pin_memory=True)

    # host-link peak: pinned cudaMemcpyAsync host->device, best of 6 at 256 MiB
    hsrc = torch.empty(256 << 20, dtype=torch.uint8, pin_memory=True)
    hdst = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    link_peak = 0.0
    for _ in range(6):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        hdst.copy_(hsrc, non_blocking=True)
        e1.record()
        torch.cuda.synchronize()
        link_peak = max(link_peak, hsrc.numel() / (e0.elapsed_time(e1) * 1e-3) / 1e9)
    del hsrc, hdst

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def run_steps(t_from, t_to, step_base):
        for t in range(t_from, t_to):
            for l in range(L):
                ctx.decode_layer_step(step_base + t - t_from, l, q_dev[t, l], outs[l])

    # ---- device-resident run: W warm-up steps, then exactly K timed steps
    sampler = ClockSampler(local_rank) if rank == 0 else None
    ctx.prime(q_init)
    run_steps(0, W, 0)
    barrier()
    if sampler:
        t_wait = time.time()
        while not sampler.rows and time.time() - t_wait < 3.0:     # nvidia-smi takes a moment to start
            time.sleep(0.05)
        sampler.rows.clear()                                       # keep only samples of the timed region
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    x0, x1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    tail = torch.cuda.Event()
    ev0.record(compute)
    x0.record(copy)
    run_steps(W, W + K, W)
    x1.record(copy)
    tail.record(copy)
    compute.wait_event(tail)          # the timed region ends when both streams are done
    ev1.record(compute)
    barrier()
    clocks = sampler.stop() if sampler else None
    ms_total = ev0.elapsed_time(ev1)
    copy_ms = x0.elapsed_time(x1)
    code, detail = ctx.device_error()
    if code != 0:
        raise RuntimeError(f"device error {code} (detail {detail}) during the timed run")
    miss = ctx.miss_stats(reset=True) if args.correct_misses else None
    ms_total, tokens = replicas.aggregate(ms_total, B * K, device="cuda")
    ms_per_step = ms_total / K
    value = tokens / (ms_total * 1e-3)
    n_gathers = K * L
    gather_bytes = w.gathered_bytes_per_layer
    gather_ms_live = copy_ms / n_gathers

    # ---- traced pass (outside the timed region): where the compute stream waits, how long the live gathers take
    trace_steps = min(K, 4)
    ctx.sync()
    ctx.prime(q_init)
    run_steps(0, W, 0)
    ctx.trace_begin(trace_steps * L)
    run_steps(W, W + trace_steps, W)
    tr = ctx.trace_end()
    pipeline_trace = None
    if len(tr) > 2 * L:
        import numpy as np
        t = tr[L:]                                   # drop the first traced step (pipeline refill after the sync)
        stall, attn_t, step_t, gath = t[:, 1] - t[:, 0], t[:, 2] - t[:, 1], t[:, 3] - t[:, 0], t[:, 5] - t[:, 4]
        period = np.diff(t[:, 2])                    # attention-done to attention-done = layer period
        pipeline_trace = {
            "layer_steps": int(len(t)),
            "compute_stall_on_transfer_us": {"median": float(np.median(stall)), "p90": float(np.percentile(stall, 90))},
            "attention_us": float(np.median(attn_t)),
            "gather_us_live": {"median": float(np.median(gath)), "p90": float(np.percentile(gath, 90))},
            "layer_period_us": float(np.median(period)),
            "exposed_transfer_fraction_of_period": float(np.median(stall) / np.median(period)),
        }

    # ---- end-to-end run: every step copies its queries from pinned host memory, reads the outputs back
    ctx.sync()
    ctx.prime(q_init)
    done = torch.cuda.Event()
    for t in range(W):
        ctx.decode_step_host(t, q_host[t], out_host)
        done.record(compute)
        done.synchronize()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(compute)
    for t in range(W, W + K):
        ctx.decode_step_host(t, q_host[t], out_host)      # host queries in, host outputs out, through the C ABI
        done.record(compute)
        done.synchronize()                                # the caller needs the step's result before the next step
    tail.record(copy)
    compute.wait_event(tail)
    e1.record(compute)
    barrier()
    e2e_value = replicas.throughput(e0.elapsed_time(e1), B * K, device="cuda")
    q_bytes = q_host[0].numel() * 2
    o_bytes = outs.numel() * 2

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "batch": B, "ctx": w.ctx, "budget": w.budget, "layers": L,
                   "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim,
                   "page_tokens": w.page_tokens, "ring_depth": args.ring_depth, "ragged_contexts": args.ragged, "select_stream": not args.no_select_stream, "landmark_chunk_tokens": args.landmark_chunk or w.page_tokens, "gather_mode": args.gather_mode,
                   "host_store_gib": store.host_bytes / 2**30, "phys_layers": store.n_phys,
                   "parallelism": "replicas only" if world > 1 else "single GPU",
                   "l2": "inputs larger than L2: each layer streams its own 32 MiB of landmarks and 64 MiB of "
                         "freshly gathered pages; the host store is never cached",
                   "generator": {k: v for k, v in w.params().items() if k in (
                       "structure", "planted_frac", "zipf_a", "topic_gain", "planted_noise", "query_topic", "seed")}},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": q_bytes + L * gather_bytes,
                "d2h_bytes_per_step": o_bytes,
                "note": "dd_decode_step_host: queries from pinned host memory and outputs back to it every step, the host "
                        "waits for each step; the KV gather from the host store is part of the path in both numbers"},
        # per layer step: attention, selection, prefetch gather (+ true-index selection, diff, missing-page gather)
        "gpu_launches": K * L * (6 if args.correct_misses else 3),
        "clocks": clocks,
        "pipeline_trace": pipeline_trace,
    }

    if w.structure in ("needle_q", "needle_topic"):
        # plausibility statistic, not a gate: share of the planted needles' pages inside the set that the
        # speculated token of (step 0, layer 0) selects
        ctx.sync()
        sel = torch.empty((B, w.n_kv_heads, w.k_pages), dtype=torch.int32, device="cuda")
        ctx.select_topk_chunked(wl.queries(w, 0, 0).cuda(), 1, store.landmarks[0], store.n_pages_dev, store.ctx_len_dev, sel)
        torch.cuda.synchronize()
        sel = sel.cpu()
        hit = tot = 0
        for b in range(B):
            pages = wl.needle_positions(w, 0, b) // w.page_tokens
            for g in range(w.n_kv_heads):
                chosen = set(sel[b, g].tolist())
                want = set(pages[g].tolist())
                hit += len(want & chosen)
                tot += len(want)
        line["needle_page_recall"] = hit / max(1, tot)
    if miss is not None:
        line["miss_correction"] = {"missing_pages": miss[0], "selected_pages": miss[1],
                                   "miss_rate": miss[0] / max(1, miss[1]),
                                   "urgent_queue": "fifo behind the prefetches" if args.urgent_fifo else "own high-priority stream",
                                   "spec_fidelity": w.spec_fidelity,
                                   "extra_link_bytes_per_layer": miss[0] * w.page_bytes / max(1, (W + K) * L),
                                   "note": "attention runs over the set selected from the current token; the pages the "
                                           "prediction missed cross the link on the urgent stream (counts include warm-up)"}
    if rank == 0:
        us_layer = ms_per_step / L * 1e3
        link_time_us = gather_bytes / (link_peak * 1e9) * 1e6
        hbm_bytes = (B * w.n_kv_heads * w.n_pages * 256) + 2 * gather_bytes
        hbm_time_us = hbm_bytes / (hbm_peak * 1e9) * 1e6
        line["roofline"] = {
            "kernel": "dd_gather_loads_kernel" if args.gather_mode == "loads" else "dd_gather_bulk_kernel",
            "bound": "host_link", "achieved": gather_bytes / (gather_ms_live * 1e-3) / 1e9, "peak": link_peak,
            "unit": "GB/s", "frac": gather_bytes / (gather_ms_live * 1e-3) / 1e9 / link_peak,
            "traffic": NCU_TRAFFIC["gather_dram"] * gather_bytes / (64 << 20),
            "link_traffic": NCU_TRAFFIC["gather_sysmem"] * gather_bytes / (64 << 20),
            "traffic_source": "ncu capture of a 64 MiB launch (summary committed under profiles/), scaled by gathered "
                              "bytes: `traffic` = DRAM read+write (the slot stays in L2), `link_traffic` = sysmem sectors x 32 B",
            "peak_source": "pinned cudaMemcpyAsync host->device, 256 MiB, best of 6, measured in this run",
            "how": "gathered bytes per launch / (copy-stream span of the timed region / launches)",
        }
        line["layer_step"] = {"us_per_layer": us_layer, "roofline_us": max(link_time_us, hbm_time_us),
                              "frac_of_roofline": max(link_time_us, hbm_time_us) / us_layer,
                              "link_us": link_time_us, "hbm_us": hbm_time_us, "hbm_peak_gbs": hbm_peak,
                              "hbm_peak_source": peak_src}
        if not args.no_stages and not args.correct_misses:
            line["stages"] = stage_timings(torch, dd, ctx, store, w, q_dev, outs, hbm_peak, link_peak, args, K, W)
            st = line["stages"]
            t_c = st["compute_only_us_per_layer"]
            t_g = st["gather_us"]
            line["layer_step"].update({
                "exposed_transfer_us_per_layer": us_layer - t_c,
                "hidden_fraction_raw": 1.0 - (us_layer - t_c) / t_g,
                "hidden_fraction_bound": min(1.0, t_c / t_g),
                "overlap_efficiency": (t_c + t_g - us_layer) / min(t_c, t_g)})
            line["roofline_kernels"] = st.pop("roofline_kernels")
    ctx.sync()
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        log("timing the CPU oracle on a sample of the workload ...")
        line["cpu_baseline"] = oracle_sample(w)
    if rank == 0:
        print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def stage_timings(torch, dd, ctx, store, w, q_dev, outs, hbm_peak, link_peak, args, K, W):
    """Each kernel alone, CUDA events on its stream around batches of launches (the split of a layer into
    select / gather / attention and the per-kernel rooflines). Selection and gather rotate over the layers
    (every launch reads landmarks / host pages no earlier launch left in L2); attention is timed both on an
    L2-warm slot and with L2 flushed before every launch."""
    L, B = w.n_layers, w.batch
    cs, xs = ctx.compute_stream, ctx.copy_stream
    ctx.sync()
    reps = max(8, min(64, 2 * L))
    idx = torch.stack([ctx.get_indices(0, l) for l in range(L)])
    tmp_idx = torch.empty_like(idx[0])
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def timed(stream, fn, pre=None):
        """Average device time of fn over `reps` launches enqueued back to back on `stream` (no host
        synchronisation in between, as in the pipeline); `pre` runs before every launch and its own cost,
        measured the same way, is subtracted."""
        def batch(with_fn):
            for i in range(3):
                if pre:
                    pre(i)
                if with_fn:
                    fn(i)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for i in range(reps):
                if pre:
                    pre(i)
                if with_fn:
                    fn(i)
            e1.record(stream)
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) * 1e3 / reps
        total = batch(True)
        return total - (batch(False) if pre else 0.0)

    sel_us = timed(cs, lambda i: ctx.select_topk_chunked(q_dev[i % q_dev.shape[0], i % L], 1, store.landmarks[i % L],
                                                         store.n_pages_dev, store.ctx_len_dev, tmp_idx, None, stream=cs))
    gat_us = timed(xs, lambda i: ctx.gather_kv_from_host(store.kv[i % L], idx[i % L], store.n_pages_dev,
                                                         i % args.ring_depth, stream=xs))
    ctx.gather_kv_from_host(store.kv[0], idx[0], store.n_pages_dev, 0, stream=cs)

    def flush_l2(i):
        with torch.cuda.stream(cs):
            flush.fill_(i & 255)

    attn = lambda i: ctx.sparse_decode_attn(q_dev[0, 0], 0, idx[0], store.ctx_len_dev, outs[0], None, stream=cs)
    att_warm = timed(cs, attn)
    att_cold = timed(cs, attn, pre=flush_l2)
    # load-only twins: what the memory system delivers for the same launch shape and size without any arithmetic
    att_loads = timed(cs, lambda i: ctx.probe_attn_loads(0, stream=cs), pre=flush_l2)
    sel_loads = timed(cs, lambda i: ctx.probe_select_loads(store.landmarks[i % L], store.n_pages_dev, stream=cs))
    # compute-only step: attention + selection of every layer with the slot already filled
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_rep = 4
    ss = ctx.select_stream
    fork, join = torch.cuda.Event(), torch.cuda.Event()
    for r in range(n_rep + 1):
        if r == 1:
            e0.record(cs)
        for l in range(L):
            if ss is not None:            # as in the pipelined step: selection next to the attention, joined afterwards
                fork.record(cs)
                ss.wait_event(fork)
            ctx.select_topk_chunked(q_dev[0, l], 1, store.landmarks[l], store.n_pages_dev, store.ctx_len_dev, tmp_idx,
                                    None, stream=ss if ss is not None else cs)
            ctx.sparse_decode_attn(q_dev[0, l], 0, idx[0], store.ctx_len_dev, outs[l], None, stream=cs)
            if ss is not None:
                join.record(ss)
                cs.wait_event(join)
    e1.record(cs)
    torch.cuda.synchronize()
    compute_only = e0.elapsed_time(e1) * 1e3 / (n_rep * L)
    lm_bytes = B * w.n_kv_heads * w.n_pages * 256 * (w.page_tokens // args.landmark_chunk if args.landmark_chunk else 1)
    sel_bytes = float(lm_bytes)           # landmarks once; the fused kernel keeps the logits in shared memory
    gb = w.gathered_bytes_per_layer
    return {
        "select_us": sel_us, "gather_us": gat_us, "attn_us_l2_warm": att_warm, "attn_us_l2_flushed": att_cold,
        "select_loads_only_us": sel_loads, "attn_loads_only_us_l2_flushed": att_loads,
        "compute_only_us_per_layer": compute_only, "reps": reps,
        "roofline_kernels": {
            "dd_select_fused_kernel": {"bound": "hbm", "achieved": sel_bytes / (sel_us * 1e-6) / 1e9,
                                       "peak": hbm_peak, "unit": "GB/s",
                                       "frac": sel_bytes / (sel_us * 1e-6) / 1e9 / hbm_peak,
                                       "traffic": NCU_TRAFFIC["select_dram"] * lm_bytes / (32 << 20),
                                       "frac_of_load_only_kernel": sel_loads / sel_us},
            "dd_attn_kernel(l2 flushed)": {"bound": "hbm", "achieved": gb / (att_cold * 1e-6) / 1e9, "peak": hbm_peak,
                                           "unit": "GB/s", "frac": gb / (att_cold * 1e-6) / 1e9 / hbm_peak,
                                           "traffic": NCU_TRAFFIC["attn_dram"] * gb / (64 << 20),
                                           "frac_of_load_only_kernel": att_loads / att_cold},
            "gather(alone)": {"bound": "host_link", "achieved": gb / (gat_us * 1e-6) / 1e9, "peak": link_peak,
                              "unit": "GB/s", "frac": gb / (gat_us * 1e-6) / 1e9 / link_peak},
        },
    }


if __name__ == "__main__":
    main()
