#!/usr/bin/env python
"""Benchmark of the sparse decode hot path: decode tokens/s on synthetic Llama-3-8B-shaped workloads.

A "step" is one decode step of the whole path: for each of the L layers, attention over the set gathered
for it, the selection of the next step's set from the speculated token, and the host->HBM gather of a
later layer on the side stream (dd_decode_layer_step). `value` counts output tokens only (B per step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl ours|reference]

The headline line is the batch-8 / 32K-context workload with its own 64 decode steps. The same line carries,
measured in the same run: the gather engines side by side (`gather_modes`, with the run-length histogram of the
selected sets), one pass with miss correction (`miss_correction`), and compact results of the other
workloads (`other_configs`). `--sweeps` adds a ring-depth sweep, a gather-grid sweep and miss correction against the miss rate.

N > 1 runs N independent replicas, one per GPU (the path has no exchange step): under torchrun as launched,
otherwise this script starts the N ranks itself. `--impl reference` times the CPU oracle on the host cores
instead (a deliberately slow program).
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# Per-launch traffic of the three kernels, NOT measured in this run: taken from the ncu captures whose
# summaries are committed under profiles/ (a layer of the batch-8 / 32K workload: 64 MiB gathered, 32 MiB of
# landmarks) and scaled by bytes for other sizes.
NCU_TRAFFIC = {"gather_dram": 38.7e3 + 9.36e6, "gather_sysmem": 2097152 * 32, "attn_dram": 67.33e6 + 0.95e6,
               "select_dram": 33.68e6}
NCU_TRAFFIC_NOTE = "from the ncu captures summarised under profiles/ (64 MiB / 32 MiB launches), scaled by bytes; " \
                   "not measured in this run"

METRIC = "decode_tokens_per_s"
UNIT = "tok/s"
GEN_KEYS = ("structure", "planted_frac", "zipf_a", "topic_gain", "planted_noise", "query_topic", "seed")


def log(msg):
    print(f"[bench] {msg}", file=sys.stderr, flush=True)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0, help="timed decode steps (0 = the workload's own count: 64 for config 2)")
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--config", type=int, default=2, help="workload number (2 = batch 8, 32K context, budget 2048)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--phys-layers", type=int, default=0, help="distinct layers kept in the host store (0 = as many as fit)")
    ap.add_argument("--ring-depth", type=int, default=2)
    ap.add_argument("--gather-mode", default="loads", choices=["loads", "bulk", "staged"])
    ap.add_argument("--gather-ctas", type=int, default=0)
    ap.add_argument("--stage-min-run", type=int, default=0, help="staged gather: shortest run the copy engine takes (0 = 8)")
    ap.add_argument("--stage-block", type=int, default=0, help="staged gather: aligned block size in pages (0 = exact runs)")
    ap.add_argument("--attn-splits", type=int, default=0)
    ap.add_argument("--attn-mode", default="auto", choices=["auto", "split", "stream", "tc"],
                    help="attention kernel: split-KV with cluster merge, or TMA-fed streaming (auto = library default)")
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
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the gather-engine comparison, the miss-correction pass and the other workloads")
    ap.add_argument("--sweeps", action="store_true", help="add ring_depth_sweep, gather_ctas_sweep and miss_rate_sweep to the line")
    ap.add_argument("--cpu-stub", action="store_true",
                    help="multi-rank plumbing only: no CUDA, gloo backend, a made-up per-rank measurement (used by the tests)")
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

    def wait_started(self):
        t_wait = time.time()
        while self.proc and not self.rows and time.time() - t_wait < 3.0:     # nvidia-smi takes a moment to start
            time.sleep(0.05)
        self.rows.clear()                                                      # keep only samples taken from now on

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


L2_NOTE = ("inputs larger than L2: each layer streams its own landmarks and freshly gathered pages; the host store is "
           "never cached")


def config_dict(w, n_ranks=1, **extra):
    """The workload description; both arms print exactly the same dictionary."""
    d = {"workload": w.name, "batch": w.batch, "ctx": w.ctx, "budget": w.budget, "layers": w.n_layers,
         "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim, "page_tokens": w.page_tokens,
         "forced_recent_pages": w.forced_recent_pages, "config_steps": w.steps,
         "generator": {k: v for k, v in w.params().items() if k in GEN_KEYS},
         "parallelism": "replicas only" if n_ranks > 1 else "single GPU", "l2": L2_NOTE}
    d.update(extra)
    return d


# --------------------------------------------------------------------------------------------------
# CPU oracle legs
# --------------------------------------------------------------------------------------------------
def _blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        return 1


def _oracle_layer(orc, w, q, lm, kv32, npg, ctx_len):
    """One layer (all requests) through the oracle as it stands: selection from the speculated token, page
    gather, attention of both tokens. Returns the three durations."""
    t0 = time.perf_counter()
    idx, _ = orc.select_topk(q[:, 1], lm, npg, w.k_pages, w.forced_recent_pages)
    t1 = time.perf_counter()
    slot = orc.gather_kv(kv32, idx)
    t2 = time.perf_counter()
    orc.sparse_decode_attn(q, slot, idx, ctx_len, w.page_tokens)
    t3 = time.perf_counter()
    return t1 - t0, t2 - t1, t3 - t2


def oracle_sample(w, n_layers_cap=4, min_seconds=10.0, max_steps_per_layer=12):
    """Times the oracle on whole layers of the workload (all requests). A few layers' slabs are drawn; each is
    run for several steps of fresh queries until about `min_seconds` of oracle work has been timed. Returns
    tok/s scaled to full steps of w.n_layers layers. `cores` is what the program really used: process CPU time
    over wall time (the oracle is Python loops around small numpy calls, so it is close to one)."""
    import torch
    from oracle import dd_oracle as orc
    from paper_2607_26475_b200 import workloads as wl
    ctx_len = wl.ctx_lens(w).numpy()
    npg = (ctx_len + w.page_tokens - 1) // w.page_tokens
    n_units, t_total, cpu_total, layers = 0, 0.0, 0.0, 0
    split = {"select": 0.0, "gather": 0.0, "attn": 0.0}
    while layers < n_layers_cap and (layers == 0 or t_total < min_seconds):
        l = layers
        kv32 = torch.stack([wl.kv_slab(w, l, b) for b in range(w.batch)]).float().numpy()
        lm = orc.build_landmarks(kv32[:, :, :, 0], ctx_len)             # set-up, not timed
        for step in range(max_steps_per_layer):
            q = wl.queries(w, step, l).float().numpy()
            c0 = time.process_time()
            a, b, c = _oracle_layer(orc, w, q, lm, kv32, npg, ctx_len)
            cpu_total += time.process_time() - c0
            split["select"] += a
            split["gather"] += b
            split["attn"] += c
            t_total += a + b + c
            n_units += 1
            if t_total >= min_seconds:
                break
        layers += 1
        del kv32, lm
    per_layer = t_total / n_units
    value = w.batch / (per_layer * w.n_layers)
    return {"value": value, "unit": UNIT, "cores": max(1, round(cpu_total / t_total)), "kind": "oracle",
            "cpu_seconds_over_wall_seconds": cpu_total / t_total, "blas_pool_threads": _blas_threads(),
            "host_cores": len(os.sched_getaffinity(0)),
            "sample": f"{n_units} layer-steps (all {w.batch} requests; {layers} layer(s) x up to {max_steps_per_layer} "
                      f"steps) of {w.name}, scaled to {w.n_layers} layers per step",
            "us_per_layer": {k: v / n_units * 1e6 for k, v in split.items()}, "seconds": t_total}


def run_reference(args):
    """The oracle arm: each step is one layer (all requests) of the workload through the oracle, with fresh
    queries; ms_per_step and value are that layer time scaled to the layers of a full step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    from oracle import dd_oracle as orc
    from paper_2607_26475_b200 import workloads as wl
    w = wl.CONFIGS[args.config]
    K = args.steps or 8
    W = max(args.warmup, 0)
    ctx_len = wl.ctx_lens(w).numpy()
    npg = (ctx_len + w.page_tokens - 1) // w.page_tokens
    kv32 = torch.stack([wl.kv_slab(w, 0, b) for b in range(w.batch)]).float().numpy()     # set-up, not timed
    lm = orc.build_landmarks(kv32[:, :, :, 0], ctx_len)
    times, cpu = [], 0.0
    t_begin = time.time()
    budget_s = 150.0
    done_warm = 0
    for step in range(W + K):
        q = wl.queries(w, step, 0).float().numpy()
        c0 = time.process_time()
        dt = sum(_oracle_layer(orc, w, q, lm, kv32, npg, ctx_len))
        if step >= W:
            times.append(dt)
            cpu += time.process_time() - c0
        else:
            done_warm += 1
        if time.time() - t_begin > budget_s and times:
            break
    per_layer = sum(times) / len(times)
    ms = per_layer * w.n_layers * 1e3
    value = w.batch / (ms * 1e-3)
    cores = max(1, round(cpu / sum(times)))
    sample = (f"each step = 1 layer x all {w.batch} requests with fresh queries through the oracle, scaled to "
              f"{w.n_layers} layers")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": len(times), "warmup": done_warm, "ms_per_step": ms, "extrapolated_from_layers": 1,
            "measured_ms_per_layer": per_layer * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(w, n_ranks=args.gpus),
            "engine": {"what": "CPU oracle on the host cores (numpy, fp64); no GPU work"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                             "cpu_seconds_over_wall_seconds": cpu / sum(times), "host_cores": len(os.sched_getaffinity(0))},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------------
# GPU arm: one workload on one GPU (store, queries, contexts, timed runs)
# --------------------------------------------------------------------------------------------------
class Bench:
    """A workload resident on this rank's GPU and host: pinned KV store, landmarks, queries of every step. Contexts
    with different engine settings are created over the same store."""

    def __init__(self, mods, w, args, rank, world, steps, warmup, phys_layers=None, quiet=False):
        torch, dd, wl, replicas, HostStore, available_host_bytes = mods
        self.torch, self.dd, self.wl, self.replicas = torch, dd, wl, replicas
        self.w, self.args, self.rank, self.world = w, args, rank, world
        self.K, self.W = steps, warmup
        self.compute = torch.cuda.Stream()
        self.copy = torch.cuda.Stream(priority=0)
        self.select = None if args.no_select_stream else torch.cuda.Stream()
        self.ctx = self.make_ctx()
        budget = replicas.host_budget_per_rank(available_host_bytes(), world)
        self.store = HostStore(w, self.ctx, n_phys_layers=phys_layers, ragged=args.ragged, host_budget_bytes=budget,
                               log=log if rank == 0 and not quiet else None)
        self.store.bind(self.ctx)
        L, B = w.n_layers, w.batch
        n_q = self.W + self.K
        self.q_host = torch.empty((n_q, L, B, 2, w.n_q_heads, w.head_dim), dtype=torch.bfloat16, pin_memory=True)
        for t in range(n_q):
            for l in range(L):
                self.q_host[t, l] = wl.queries(w, t, l)
        self.q_dev = self.q_host.cuda()
        self.q_init = torch.stack([wl.queries(w, -1, l)[:, 1] for l in range(L)]).cuda()
        self.outs = torch.zeros((L, B, 2, w.n_q_heads, w.head_dim), dtype=torch.bfloat16, device="cuda")
        self.out_host = torch.empty(self.outs.shape, dtype=torch.bfloat16, pin_memory=True)

    def make_ctx(self, **over):
        a, w, dd = self.args, self.w, self.dd
        mode = over.pop("gather_mode", a.gather_mode)
        kw = dict(n_layers=w.n_layers, batch=w.batch, max_pages=w.n_pages, k_pages=w.k_pages,
                  forced_recent_pages=w.forced_recent_pages, ring_depth=a.ring_depth,
                  gather_mode={"loads": dd.DD_GATHER_LOADS, "bulk": dd.DD_GATHER_BULK, "staged": dd.DD_GATHER_STAGED}[mode],
                  gather_ctas=a.gather_ctas, attn_splits=a.attn_splits, compute_stream=self.compute,
                  copy_stream=self.copy, landmark_chunk_tokens=a.landmark_chunk, select_stream=self.select,
                  stage_min_run_pages=a.stage_min_run, stage_block_pages=a.stage_block,
                  attn_mode={"auto": dd.DD_ATTN_AUTO, "split": dd.DD_ATTN_SPLIT, "stream": dd.DD_ATTN_STREAM,
                             "tc": dd.DD_ATTN_TC}[a.attn_mode])
        if over.pop("correct", a.correct_misses):
            fifo = over.pop("urgent_fifo", a.urgent_fifo)
            kw.update(miss_correction=True, urgent_stream=self.copy if fifo else self.torch.cuda.Stream(priority=-1))
        kw.update(over)
        return dd.Context(**kw)

    def barrier(self):
        self.torch.cuda.synchronize()
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
        self.torch.cuda.synchronize()

    def run_steps(self, ctx, t_from, t_to, step_base):
        L = self.w.n_layers
        for t in range(t_from, t_to):
            for l in range(L):
                ctx.decode_layer_step(step_base + t - t_from, l, self.q_dev[t, l], self.outs[l])

    def timed(self, ctx, K=None, W=None, sampler=None):
        """W warm-up steps, then exactly K timed steps with the queries resident in HBM. Returns milliseconds of the
        compute stream (closing on an event that also waits for the copy stream) and of the copy stream."""
        torch = self.torch
        K = self.K if K is None else K
        W = self.W if W is None else W
        ctx.sync()
        ctx.prime(self.q_init)
        self.run_steps(ctx, 0, W, 0)
        self.barrier()
        if sampler:
            sampler.wait_started()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        x0, x1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        tail = torch.cuda.Event()
        ev0.record(self.compute)
        x0.record(self.copy)
        self.run_steps(ctx, W, W + K, W)
        x1.record(self.copy)
        tail.record(self.copy)
        self.compute.wait_event(tail)          # the timed region ends when both streams are done
        ev1.record(self.compute)
        self.barrier()
        code, detail = ctx.device_error()
        if code != 0:
            raise RuntimeError(f"device error {code} (detail {detail}) during the timed run")
        return ev0.elapsed_time(ev1), x0.elapsed_time(x1)

    def e2e(self, ctx, K=None, W=None):
        """The same steps through dd_decode_step_host: queries from pinned host memory and outputs back to it every
        step, the host waits for each step's result. Returns milliseconds."""
        torch = self.torch
        K = self.K if K is None else K
        W = self.W if W is None else W
        ctx.sync()
        ctx.prime(self.q_init)
        done = torch.cuda.Event()
        for t in range(W):
            ctx.decode_step_host(t, self.q_host[t], self.out_host)
            done.record(self.compute)
            done.synchronize()
        self.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        tail = torch.cuda.Event()
        e0.record(self.compute)
        for t in range(W, W + K):
            ctx.decode_step_host(t, self.q_host[t], self.out_host)
            done.record(self.compute)
            done.synchronize()                                # the caller needs the step's result before the next step
        tail.record(self.copy)
        self.compute.wait_event(tail)
        e1.record(self.compute)
        self.barrier()
        return e0.elapsed_time(e1)

    def trace(self, ctx, steps):
        """A traced pass outside any timed region: where the compute stream waits, how long the live gathers take."""
        import numpy as np
        L = self.w.n_layers
        steps = min(steps, self.K)
        ctx.sync()
        ctx.prime(self.q_init)
        self.run_steps(ctx, 0, self.W, 0)
        ctx.trace_begin(steps * L)
        self.run_steps(ctx, self.W, self.W + steps, self.W)
        tr = ctx.trace_end()
        if len(tr) <= 2 * L:
            return None
        t = tr[L:]                                   # drop the first traced step (pipeline refill after the sync)
        stall, attn_t, gath = t[:, 1] - t[:, 0], t[:, 2] - t[:, 1], t[:, 5] - t[:, 4]
        period = np.diff(t[:, 2])                    # attention-done to attention-done = layer period
        return {
            "layer_steps": int(len(t)),
            "compute_stall_on_transfer_us": {"median": float(np.median(stall)), "p90": float(np.percentile(stall, 90))},
            "attention_us": float(np.median(attn_t)),
            "gather_us_live": {"median": float(np.median(gath)), "p90": float(np.percentile(gath, 90))},
            "layer_period_us": float(np.median(period)),
            "exposed_transfer_fraction_of_period": float(np.median(stall) / np.median(period)),
        }

    def link_peak(self, mib=256, reps=6):
        """Pinned cudaMemcpyAsync host->device: the copy engine's rate on this machine, every repetition reported."""
        torch = self.torch
        hsrc = torch.empty(mib << 20, dtype=torch.uint8, pin_memory=True)
        hdst = torch.empty(mib << 20, dtype=torch.uint8, device="cuda")
        rates = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            hdst.copy_(hsrc, non_blocking=True)
            e1.record()
            torch.cuda.synchronize()
            rates.append(hsrc.numel() / (e0.elapsed_time(e1) * 1e-3) / 1e9)
        return max(rates), {"min": min(rates), "median": statistics.median(rates), "max": max(rates), "reps": reps,
                            "mib": mib}

    def run_length_histogram(self, ctx, layers=4):
        """Runs of adjacent selected pages in the sets the pipeline last selected (first `layers` layers, both
        parities): what a copy engine could move with one copy each."""
        import numpy as np
        w = self.w
        runs = []
        for par in (0, 1):
            for l in range(min(layers, w.n_layers)):
                idx = ctx.get_indices(par, l).cpu().numpy().reshape(-1, w.k_pages)
                for row in idx:
                    brk = np.flatnonzero(np.diff(row) != 1)
                    ends = np.concatenate([brk + 1, [len(row)]])
                    starts = np.concatenate([[0], brk + 1])
                    runs.append(ends - starts)
        runs = np.concatenate(runs)
        tot = float(runs.sum())
        out = {"sets": int(2 * min(layers, w.n_layers) * w.batch * w.n_kv_heads), "pages": int(tot), "runs": int(len(runs)),
               "mean_run_pages": float(runs.mean()), "max_run_pages": int(runs.max())}
        for thr in (2, 4, 8, 16, 32):
            sel = runs[runs >= thr]
            out[f"runs_ge{thr}"] = {"runs_per_set": float(len(sel) / out["sets"]), "share_of_pages": float(sel.sum() / tot)}
        return out

    def close(self):
        self.ctx.close()


def load_modules():
    import torch
    from paper_2607_26475_b200 import binding as dd
    from paper_2607_26475_b200 import replicas
    from paper_2607_26475_b200 import workloads as wl
    from paper_2607_26475_b200.store import HostStore, available_host_bytes
    return torch, dd, wl, replicas, HostStore, available_host_bytes


def compare_gather_modes(b, link_peak, steps=6, warm=2):
    """The gather engines side by side over the same store and queries: short pipelined runs (tok/s, live GB/s on
    the copy stream), plus what the staged engine did with the selected sets. Not a timed headline region."""
    w = b.w
    gb, L = w.gathered_bytes_per_layer, w.n_layers
    steps = min(steps, b.K)
    warm = min(warm, b.W)
    out = {}
    variants = [("loads", dict(gather_mode="loads")), ("bulk", dict(gather_mode="bulk")),
                ("staged_runs_ge8", dict(gather_mode="staged", stage_min_run_pages=8, stage_block_pages=0)),
                ("staged_runs_ge2", dict(gather_mode="staged", stage_min_run_pages=2, stage_block_pages=0)),
                ("staged_all_runs", dict(gather_mode="staged", stage_min_run_pages=1, stage_block_pages=0)),
                ("staged_blocks_4", dict(gather_mode="staged", stage_block_pages=4)),
                ("staged_blocks_8", dict(gather_mode="staged", stage_block_pages=8))]
    for name, kw in variants:
        ctx = b.make_ctx(correct=False, **kw)
        b.store.bind(ctx)
        ms, copy_ms = b.timed(ctx, K=steps, W=warm)
        r = {"tok_s": w.batch * steps / (ms * 1e-3), "us_per_layer": ms / (steps * L) * 1e3,
             "gather_gb_s_live": gb / (copy_ms / (steps * L) * 1e-3) / 1e9,
             "frac_of_link_peak": gb / (copy_ms / (steps * L) * 1e-3) / 1e9 / link_peak}
        if kw["gather_mode"] == "staged":
            st = ctx.gather_stats()
            n = max(1, st["gathers"])
            r.update({"copies_per_layer": st["copies"] / n, "link_bytes_over_algorithmic":
                      (st["copied_bytes"] + st["pages_zero_copy"] * w.page_bytes) / (n * gb),
                      "share_of_pages_through_copy_engine": st["pages_staged"] / max(1, st["pages_staged"] + st["pages_zero_copy"]),
                      "host_issue_us_per_layer": st["host_issue_us"] / n, "host_wait_us_per_layer": st["host_wait_us"] / n})
        out[name] = r
        if name == "loads":
            out["run_length_histogram"] = b.run_length_histogram(ctx)
        ctx.close()
    out["steps"] = steps
    out["note"] = ("same store and queries, ring depth as configured; staged_* = copy engine for runs of adjacent selected "
                   "pages (>= 8 / >= 2 / all) or for aligned 4- / 8-page blocks that hold a selected page, zero-copy "
                   "kernel for the rest")
    return out


def correction_pass(b, link_peak, steps=8, warm=2):
    """One pass with miss correction on an urgent high-priority stream (not the headline path)."""
    w = b.w
    steps, warm = min(steps, b.K), min(warm, b.W)
    ctx = b.make_ctx(correct=True, urgent_fifo=False)
    b.store.bind(ctx)
    ms, copy_ms = b.timed(ctx, K=steps, W=warm)
    miss = ctx.miss_stats(reset=True)
    ctx.close()
    us_layer = ms / (steps * w.n_layers) * 1e3
    rate = miss[0] / max(1, miss[1])
    gb = w.gathered_bytes_per_layer
    link_us = gb * (1.0 + rate) / (link_peak * 1e9) * 1e6
    return {"tok_s": w.batch * steps / (ms * 1e-3), "us_per_layer": us_layer, "steps": steps, "miss_rate": rate,
            "missing_pages": miss[0], "selected_pages": miss[1], "spec_fidelity": w.spec_fidelity,
            "urgent_queue": "own high-priority stream",
            "roofline": {"bound": "host_link", "bytes_per_layer": gb * (1.0 + rate), "roofline_us": link_us,
                         "frac": link_us / us_layer, "peak": link_peak, "unit": "GB/s",
                         "note": "prefetched pages plus the missing pages cross the same link"},
            "gpu_launches_per_layer": 6,
            "note": "attention runs over the set selected from the current token; counts include warm-up"}


def miss_rate_sweep(b, link_peak, fidelities=(0.995, 0.97, 0.9, 0.8, 0.6, 0.3), steps=4, warm=2):
    """Miss correction against the miss rate (Sec. 6.4's priority-scheduling experiment, on synthetic queries): for
    every fidelity of the speculated query the same steps run with the missing pages on a high-priority stream of
    their own and with the missing pages queued behind the prefetches on the copy stream (FIFO)."""
    torch, wl, w0 = b.torch, b.wl, b.w
    steps, warm = min(steps, b.K), min(warm, b.W)
    keep = (b.w, b.q_dev, b.q_init)
    out = {}
    try:
        for f in fidelities:
            w = wl.small(w0, spec_fidelity=f)
            q = torch.stack([torch.stack([wl.queries(w, t, l) for l in range(w.n_layers)]) for t in range(steps + warm)])
            b.w, b.q_dev = w, q.cuda()
            b.q_init = torch.stack([wl.queries(w, -1, l)[:, 1] for l in range(w.n_layers)]).cuda()
            row = {}
            for name, fifo in (("priority", False), ("fifo", True)):
                ctx = b.make_ctx(correct=True, urgent_fifo=fifo)
                b.store.bind(ctx)
                ms, _ = b.timed(ctx, K=steps, W=warm)
                miss = ctx.miss_stats(reset=True)
                ctx.close()
                rate = miss[0] / max(1, miss[1])
                us_layer = ms / (steps * w.n_layers) * 1e3
                link_us = w.gathered_bytes_per_layer * (1.0 + rate) / (link_peak * 1e9) * 1e6
                row["miss_rate"] = rate
                row[name] = {"ms_per_step": ms / steps, "us_per_layer": us_layer, "tok_s": w.batch * steps / (ms * 1e-3),
                             "frac_of_link_roofline": link_us / us_layer}
            out[str(f)] = row
    finally:
        b.w, b.q_dev, b.q_init = keep
    out["note"] = ("spec_fidelity = correlation of a step's speculated query with the next step's current query; priority = "
                   "missing pages on their own high-priority stream, fifo = queued behind the prefetches on the copy stream")
    return out


def measure_other_config(mods, n, args, rank, world, hbm_peak, link_peak):
    """A compact measurement of another workload: pipelined tok/s, e2e, per-kernel times and roofline fractions.
    The host store keeps two physical layers (logical layer l uses l mod 2; per-layer bytes, page scatter and the
    uncached host link are unchanged by the aliasing)."""
    import copy as _copy
    torch, dd, wl = mods[0], mods[1], mods[2]
    w = wl.CONFIGS[n]
    a = _copy.copy(args)
    a.correct_misses, a.ragged, a.landmark_chunk, a.gather_mode = False, False, 0, "loads"
    a.ring_depth, a.gather_ctas, a.attn_splits, a.stage_min_run, a.stage_block = 2, 0, 0, 0, 0
    steps = w.steps if n != 1 else 256          # config 1 is one 40-microsecond step: repeat it to get a stable time
    warm = 3 if n != 1 else 16
    phys = min(2, w.n_layers)
    t0 = time.time()
    b = Bench(mods, w, a, rank, world, steps, warm, phys_layers=phys, quiet=True)
    ms, copy_ms = b.timed(b.ctx)
    e2e_ms = b.e2e(b.ctx)
    L, gb = w.n_layers, w.gathered_bytes_per_layer
    us_layer = ms / (steps * L) * 1e3
    link_us = gb / (link_peak * 1e9) * 1e6
    hbm_us = (w.batch * w.n_kv_heads * w.n_pages * 256 + 2 * gb) / (hbm_peak * 1e9) * 1e6
    st = stage_timings(torch, dd, b.ctx, b.store, w, b.q_dev, b.outs, hbm_peak, link_peak, a, steps, warm)
    rk = st["roofline_kernels"]
    out = {"workload": w.name, "steps": steps, "warmup": warm, "phys_layers": b.store.n_phys,
           "host_store_gib": b.store.host_bytes / 2**30,
           "tok_s": w.batch * steps / (ms * 1e-3), "e2e_tok_s": w.batch * steps / (e2e_ms * 1e-3),
           "ms_per_step": ms / steps, "us_per_layer": us_layer,
           "roofline_us": max(link_us, hbm_us), "frac_of_roofline": max(link_us, hbm_us) / us_layer,
           "gather_gb_s_live": gb / (copy_ms / (steps * L) * 1e-3) / 1e9,
           "select_us": st["select_us"], "select_frac_of_hbm": rk["dd_select_fused_kernel"]["frac"],
           "gather_us": st["gather_us"], "gather_frac_of_link": rk["gather(alone)"]["frac"],
           "attn_us_l2_flushed": st["attn_us_l2_flushed"], "attn_frac_of_hbm": rk["dd_attn_kernel(l2 flushed)"]["frac"],
           "compute_only_us_per_layer": st["compute_only_us_per_layer"], "seconds": None}
    if w.structure in ("needle_q", "needle_topic"):
        out["needle_page_recall"] = needle_recall(torch, wl, b)
    b.close()
    del b
    out["seconds"] = time.time() - t0
    return out


def needle_recall(torch, wl, b):
    """Plausibility statistic, not a gate: share of the planted needles' pages inside the set that the speculated
    token of (step 0, layer 0) selects."""
    w = b.w
    b.ctx.sync()
    sel = torch.empty((w.batch, w.n_kv_heads, w.k_pages), dtype=torch.int32, device="cuda")
    b.ctx.select_topk_chunked(wl.queries(w, 0, 0).cuda(), 1, b.store.landmarks[0], b.store.n_pages_dev, b.store.ctx_len_dev, sel)
    torch.cuda.synchronize()
    sel = sel.cpu()
    hit = tot = 0
    for r in range(w.batch):
        pages = wl.needle_positions(w, 0, r) // w.page_tokens
        for g in range(w.n_kv_heads):
            want = set(pages[g].tolist())
            hit += len(want & set(sel[r, g].tolist()))
            tot += len(want)
    return hit / max(1, tot)


def run_gpu(args):
    mods = load_modules()
    torch, dd, wl, replicas = mods[0], mods[1], mods[2], mods[3]
    import torch.distributed as dist
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
    L, B = w.n_layers, w.batch
    K = args.steps if args.steps > 0 else w.steps
    W = max(args.warmup, 3)
    hbm_peak, peak_src = measured_peaks()

    b = Bench(mods, w, args, rank, world, K, W, phys_layers=args.phys_layers or None)
    ctx, store = b.ctx, b.store
    if rank == 0:
        log(f"{w.name}: host store {store.host_bytes / 2**30:.1f} GiB pinned in {store.n_phys} physical layer(s), "
            f"built in {store.build_seconds:.1f} s; ring {ctx.ring_bytes() / 2**20:.0f} MiB, scratch {ctx.scratch_bytes() / 2**20:.1f} MiB")
    link_peak, link_spread = b.link_peak()

    # ---- device-resident run: W warm-up steps, then exactly K timed steps
    sampler = ClockSampler(local_rank) if rank == 0 else None
    ms_local, copy_ms = b.timed(ctx, sampler=sampler)
    clocks = sampler.stop() if sampler else None
    miss = ctx.miss_stats(reset=True) if args.correct_misses else None
    per_rank_tok_s = replicas.gather_per_rank(B * K / (ms_local * 1e-3))
    gather_bytes = w.gathered_bytes_per_layer
    gather_ms_live = copy_ms / (K * L)
    per_rank_gather = replicas.gather_per_rank(gather_bytes / (gather_ms_live * 1e-3) / 1e9)
    ms_total, tokens = replicas.aggregate(ms_local, B * K, device="cuda")
    ms_per_step = ms_total / K
    value = tokens / (ms_total * 1e-3)

    pipeline_trace = b.trace(ctx, 4)
    e2e_value = replicas.throughput(b.e2e(ctx), B * K, device="cuda")
    q_bytes = b.q_host[0].numel() * 2
    o_bytes = b.outs.numel() * 2
    mode_kernel = {"loads": "dd_gather_loads_kernel", "bulk": "dd_gather_bulk_kernel",
                   "staged": "copy engine + dd_assemble_kernel + dd_gather_list_kernel"}[args.gather_mode]

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": config_dict(w, n_ranks=world),
        "engine": {"ring_depth": args.ring_depth, "ragged_contexts": args.ragged, "select_stream": not args.no_select_stream,
                   "landmark_chunk_tokens": args.landmark_chunk or w.page_tokens, "gather_mode": args.gather_mode,
                   "attn_mode": args.attn_mode, "host_store_gib": store.host_bytes / 2**30, "phys_layers": store.n_phys},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": q_bytes + L * gather_bytes,
                "d2h_bytes_per_step": o_bytes,
                "note": "dd_decode_step_host: queries from pinned host memory and outputs back to it every step, the host "
                        "waits for each step; the KV gather from the host store is part of the path in both numbers"},
        # per layer step: attention, selection, prefetch gather (+ true-index selection, diff, missing-page gather)
        "gpu_launches": K * L * (6 if args.correct_misses else 3),
        "clocks": clocks,
        "pipeline_trace": pipeline_trace,
    }
    if world > 1:
        line["per_rank"] = {"tok_s": per_rank_tok_s, "gather_gb_s": per_rank_gather}
    if w.structure in ("needle_q", "needle_topic"):
        line["needle_page_recall"] = needle_recall(torch, wl, b)
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
        achieved = gather_bytes / (gather_ms_live * 1e-3) / 1e9
        line["roofline"] = {
            "kernel": mode_kernel, "bound": "host_link", "achieved": achieved, "peak": link_peak,
            "unit": "GB/s", "frac": achieved / link_peak,
            "traffic": NCU_TRAFFIC["gather_dram"] * gather_bytes / (64 << 20),
            "link_traffic": NCU_TRAFFIC["gather_sysmem"] * gather_bytes / (64 << 20),
            "traffic_source": NCU_TRAFFIC_NOTE + "; `traffic` = DRAM read+write of the zero-copy kernel (the slot stays in "
                              "L2), `link_traffic` = sysmem sectors x 32 B",
            "peak_source": "pinned cudaMemcpyAsync host->device measured in this run (MEASURED_PEAKS.json has no host-link "
                           "figure); best of the repetitions in peak_spread",
            "peak_spread": link_spread,
            "frac_of_pcie_gen5_x16_nominal_64": achieved / 64.0,
            "how": "gathered bytes per launch / (copy-stream span of the timed region / launches)",
        }
        line["layer_step"] = {"us_per_layer": us_layer, "roofline_us": max(link_time_us, hbm_time_us),
                              "frac_of_roofline": max(link_time_us, hbm_time_us) / us_layer,
                              "link_us": link_time_us, "hbm_us": hbm_time_us, "hbm_peak_gbs": hbm_peak,
                              "hbm_peak_source": peak_src}
        if not args.no_stages and not args.correct_misses:
            line["stages"] = stage_timings(torch, dd, ctx, store, w, b.q_dev, b.outs, hbm_peak, link_peak, args, K, W)
            st = line["stages"]
            t_c = st["compute_only_us_per_layer"]
            t_g = st["gather_us"]
            line["layer_step"].update({
                "exposed_transfer_us_per_layer": us_layer - t_c,
                "hidden_fraction_raw": 1.0 - (us_layer - t_c) / t_g,
                "hidden_fraction_bound": min(1.0, t_c / t_g),
                "hidden_fraction_target_0.9_met": bool(1.0 - (us_layer - t_c) / t_g >= 0.9),
                "overlap_efficiency": (t_c + t_g - us_layer) / min(t_c, t_g),
                "overlap_efficiency_is": "(compute + gather - layer time) / min(compute, gather): how much of the "
                                         "shorter of the two ran under the other; NOT the hidden fraction of the transfer (a value a few percent "
                                         "above 1 is timing noise: the gather alone and the pipelined layer differ by < 0.3%)"})
            line["roofline_kernels"] = st.pop("roofline_kernels")
    ctx.sync()
    extras = rank == 0 and world == 1 and not args.no_extras and not args.correct_misses
    if extras:
        log("comparing the gather engines ...")
        line["gather_modes"] = compare_gather_modes(b, link_peak)
        log("one pass with miss correction ...")
        line["miss_correction"] = correction_pass(b, link_peak)
    if rank == 0 and world == 1 and args.sweeps:
        line["ring_depth_sweep"] = sweep(b, "ring_depth", [2, 3, 4], link_peak)
        line["gather_ctas_sweep"] = sweep(b, "gather_ctas", [8, 12, 16, 24, 32], link_peak)
        log("miss correction against the miss rate ...")
        line["miss_rate_sweep"] = miss_rate_sweep(b, link_peak)
    b.close()
    if extras and args.config == 2 and not (args.layers or args.batch):
        del b, ctx, store
        line["other_configs"] = {}
        for n in (1, 3, 4, 5):
            log(f"workload {n} ...")
            line["other_configs"][str(n)] = measure_other_config(mods, n, args, rank, world, hbm_peak, link_peak)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        log("timing the CPU oracle on a sample of the workload ...")
        line["cpu_baseline"] = oracle_sample(w)
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def sweep(b, key, values, link_peak, steps=6, warm=2):
    """Short pipelined runs over one context setting, with the live attention and gather times from a trace."""
    w = b.w
    out = {}
    for v in values:
        ctx = b.make_ctx(correct=False, **{key: v})
        b.store.bind(ctx)
        ms, copy_ms = b.timed(ctx, K=min(steps, b.K), W=min(warm, b.W))
        n = min(steps, b.K) * w.n_layers
        tr = b.trace(ctx, 3)
        out[str(v)] = {"tok_s": w.batch * min(steps, b.K) / (ms * 1e-3),
                       "gather_gb_s_live": w.gathered_bytes_per_layer / (copy_ms / n * 1e-3) / 1e9,
                       "attention_us_live": tr["attention_us"] if tr else None,
                       "gather_us_live": tr["gather_us_live"]["median"] if tr else None}
        ctx.close()
    return out


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

    def timed(stream, fn, pre=None, ahead=True):
        """Average device time of fn over `reps` launches enqueued back to back on `stream` (no host
        synchronisation in between, as in the pipeline; the stream is kept busy while the host enqueues, so
        that host launch cost is not in the number); `pre` runs before every launch and its own cost,
        measured the same way, is subtracted."""
        def batch(with_fn):
            spin = ahead
            for i in range(3):
                if pre:
                    pre(i)
                if with_fn:
                    fn(i)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            try:                                   # ~1.5 ms of device idle-spin: the host queues the launches ahead,
                if spin:                           # so the events bracket device time, not host enqueue time
                    with torch.cuda.stream(stream):
                        torch.cuda._sleep(3_000_000)
            except Exception:
                pass
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
                                                         i % args.ring_depth, stream=xs), ahead=False)   # milliseconds each
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
                                       "traffic_source": NCU_TRAFFIC_NOTE,
                                       "frac_of_load_only_kernel": sel_loads / sel_us},
            "dd_attn_kernel(l2 flushed)": {"bound": "hbm", "achieved": gb / (att_cold * 1e-6) / 1e9, "peak": hbm_peak,
                                           "unit": "GB/s", "frac": gb / (att_cold * 1e-6) / 1e9 / hbm_peak,
                                           "traffic": NCU_TRAFFIC["attn_dram"] * gb / (64 << 20),
                                           "traffic_source": NCU_TRAFFIC_NOTE,
                                           "frac_of_load_only_kernel": att_loads / att_cold},
            "gather(alone)": {"bound": "host_link", "achieved": gb / (gat_us * 1e-6) / 1e9, "peak": link_peak,
                              "unit": "GB/s", "frac": gb / (gat_us * 1e-6) / 1e9 / link_peak},
        },
    }


# --------------------------------------------------------------------------------------------------
# several GPUs: N independent replicas
# --------------------------------------------------------------------------------------------------
def free_port() -> int:
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(args) -> int:
    """`--gpus N` without a launcher: start the N ranks with torch.distributed.run (one process per GPU) and pass
    this command line on. Rank 0 of the children prints the JSON line."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__), *sys.argv[1:]]
    env = dict(os.environ)
    if not args.cpu_stub:
        env.setdefault("NCCL_DEBUG", "INFO")           # the communicator log shows the rank count of the barrier
        env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    log(f"starting {args.gpus} ranks: {' '.join(cmd)}")
    return subprocess.run(cmd, env=env).returncode


def run_stub(args):
    """The multi-rank plumbing without a GPU (gloo): every rank reports a made-up measurement through the same
    aggregation as the real run, and rank 0 prints a line of the same shape. Used by the CPU tests only."""
    import torch.distributed as dist
    from paper_2607_26475_b200 import replicas
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    K, B = args.steps or 2, 8
    ms_local = 10.0 * K * (1.0 + 0.1 * rank)               # rank r is 10 r % slower
    per_rank = replicas.gather_per_rank(B * K / (ms_local * 1e-3))
    ms_total, tokens = replicas.aggregate(ms_local, B * K)
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": tokens / (ms_total * 1e-3), "unit": UNIT, "n_gpus": world,
                          "steps": K, "warmup": args.warmup, "ms_per_step": ms_total / K, "higher_is_better": True,
                          "scaling": "weak", "data": "stub", "per_rank": {"tok_s": per_rank}}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    if args.cpu_stub:
        run_stub(args)
        return
    run_gpu(args)


if __name__ == "__main__":
    main()
