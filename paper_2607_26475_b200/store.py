"""Host-resident KV store and GPU-resident landmarks of a synthetic workload.

The store is what the method keeps in host memory: for every layer a pinned bf16 tensor
[B, Hkv, P, 2, T, d] (a page = 4 KiB of K followed by 4 KiB of V). Slabs are drawn on the GPU by
the seeded generators, the landmarks are built there by the library's set-up kernel, and the slab is
then copied into the pinned store. When the host cannot hold every layer, `n_phys_layers` distinct
layers are generated and logical layer l uses physical layer l % n_phys_layers (its landmarks alias
the same way); per-layer bytes, page scatter and the absence of any cache on the host link are
unchanged by the aliasing.
"""
from __future__ import annotations

import time

import torch

from . import workloads as wl


def available_host_bytes() -> int:
    for line in open("/proc/meminfo"):
        if line.startswith("MemAvailable:"):
            return int(line.split()[1]) * 1024
    return 0


class HostStore:
    def __init__(self, w: wl.Workload, ctx, n_phys_layers: int | None = None, ragged: bool = False,
                 host_budget_bytes: int | None = None, log=None):
        """`ctx` is a binding.Context of matching geometry (used for dd_build_landmarks only)."""
        self.w = w
        L, B = w.n_layers, w.batch
        layer_bytes = w.slab_bytes * B
        if n_phys_layers is None:
            budget = host_budget_bytes if host_budget_bytes is not None else int(available_host_bytes() * 0.6)
            n_phys_layers = max(1, min(L, budget // layer_bytes))
        self.n_phys = int(n_phys_layers)
        self.layer_bytes = layer_bytes
        self.ctx_len = wl.ctx_lens(w, ragged=ragged)
        self.n_pages = ((self.ctx_len + w.page_tokens - 1) // w.page_tokens).to(torch.int32)
        self.ctx_len_dev = self.ctx_len.cuda()
        self.n_pages_dev = self.n_pages.cuda()
        t0 = time.time()
        self.phys_kv, self.phys_lm = [], []
        for l in range(self.n_phys):
            host = torch.empty((B, w.n_kv_heads, w.n_pages, 2, w.page_tokens, w.head_dim), dtype=torch.bfloat16,
                               pin_memory=True)
            R = w.page_tokens // ctx.cfg.landmark_chunk_tokens if ctx.cfg.landmark_chunk_tokens else 1
            lm = torch.empty((B, w.n_kv_heads, w.n_pages * R, w.head_dim), dtype=torch.bfloat16, device="cuda")
            for b in range(B):
                slab = wl.kv_slab(w, l, b, device="cuda")
                # landmarks of one request at a time: view the request as a batch of one
                ctx_b = self.ctx_len_dev[b:b + 1]
                self._landmarks_one(ctx, slab, ctx_b, lm[b])
                host[b].copy_(slab)
                del slab
            torch.cuda.synchronize()
            self.phys_kv.append(host)
            self.phys_lm.append(lm)
            if log and (l == 0 or (l + 1) % 8 == 0 or l + 1 == self.n_phys):
                log(f"store: {l + 1}/{self.n_phys} physical layers, {time.time() - t0:.1f} s")
        self.kv = [self.phys_kv[l % self.n_phys] for l in range(L)]
        self.landmarks = [self.phys_lm[l % self.n_phys] for l in range(L)]
        self.build_seconds = time.time() - t0

    def _landmarks_one(self, ctx, slab, ctx_b, lm_b):
        if ctx.cfg.batch == 1:
            ctx.build_landmarks(slab, ctx_b, lm_b)
        else:
            self._lm_ctx(ctx).build_landmarks(slab, ctx_b, lm_b)

    def _lm_ctx(self, ctx):
        if not hasattr(self, "_one"):
            from . import binding
            c = ctx.cfg
            self._one = binding.Context(n_layers=1, batch=1, max_pages=c.max_pages, k_pages=1,
                                        n_q_heads=c.n_q_heads, n_kv_heads=c.n_kv_heads,
                                        landmark_chunk_tokens=c.landmark_chunk_tokens)
        return self._one

    @property
    def host_bytes(self) -> int:
        return self.n_phys * self.layer_bytes

    def bind(self, ctx):
        ctx.bind(self.landmarks, self.kv, self.n_pages_dev, self.ctx_len_dev)
