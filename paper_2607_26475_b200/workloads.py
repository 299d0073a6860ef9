"""Seeded synthetic inputs for the sparse decode hot path.

This module only draws numbers: it holds none of the method's arithmetic (no
landmarks, scores, selection, gather or attention) and is the one module that
both the CUDA path's callers and the CPU checker's callers may share.

The workloads stand in for the long-context serving workloads of the paper's
evaluation (Sec. 6.1): only shapes (Llama-3-8B attention geometry, contexts 4K
to 1M tokens, 16-token pages) and sparsity structure (a few high-score tokens
scattered in a long context) are taken from there; no benchmark item is
reproduced. All tensors are torch tensors on the device asked for; the same
(seed, config, layer, request) always gives the same bits on the same device
type, and CPU and CUDA generators give different (equally distributed) bits.
"""
from __future__ import annotations

import dataclasses
import math

import torch

HQ, HKV, HEAD_DIM, PAGE_TOKENS = 32, 8, 128, 16


@dataclasses.dataclass(frozen=True)
class Workload:
    """One benchmark / parity configuration. `budget` and `recent_window` are in tokens per KV head."""
    name: str
    n_layers: int
    batch: int
    ctx: int
    budget: int
    steps: int
    structure: str            # "needle_q" | "zipf_topic" | "windows" | "needle_topic" | "iid"
    recent_window: int = 0
    n_q_heads: int = HQ
    n_kv_heads: int = HKV
    head_dim: int = HEAD_DIM
    page_tokens: int = PAGE_TOKENS
    seed: int = 0
    # generator parameters (recorded with every result)
    planted_frac: float = 0.01
    zipf_a: float = 1.1
    topic_gain: float = math.sqrt(HEAD_DIM)
    planted_noise: float = 0.25
    query_topic: float = 0.5
    spec_fidelity: float = 0.97   # correlation of step t's speculated query with step t+1's current query
    window_tokens: int = 64
    window_frac: float = 0.10
    window_norm: float = 2.0
    n_needles: int = 8
    needle_gain: float = 4.0

    @property
    def n_pages(self) -> int:
        return (self.ctx + self.page_tokens - 1) // self.page_tokens

    @property
    def k_pages(self) -> int:
        return self.budget // self.page_tokens

    @property
    def forced_recent_pages(self) -> int:
        return (self.recent_window + self.page_tokens - 1) // self.page_tokens

    @property
    def page_bytes(self) -> int:
        return 2 * self.page_tokens * self.head_dim * 2

    @property
    def slab_bytes(self) -> int:
        """Bytes of one (layer, request) slab [Hkv, P, 2, T, d] bf16."""
        return self.n_kv_heads * self.n_pages * self.page_bytes

    @property
    def gathered_bytes_per_layer(self) -> int:
        return self.batch * self.n_kv_heads * self.k_pages * self.page_bytes

    def params(self) -> dict:
        return dataclasses.asdict(self)


CONFIGS = {
    1: Workload("c1_needle_4k", 1, 1, 4096, 256, 1, "needle_q", n_needles=8),
    2: Workload("c2_llama8b_b8_32k", 32, 8, 32768, 2048, 64, "zipf_topic"),
    3: Workload("c3_llama8b_b32_32k", 32, 32, 32768, 1024, 16, "zipf_topic"),
    4: Workload("c4_llama8b_b8_128k", 32, 8, 131072, 4096, 32, "windows", recent_window=128),
    5: Workload("c5_llama8b_b1_1m", 32, 1, 1048576, 8192, 16, "needle_topic", n_needles=256),
}


def small(w: Workload, **kw) -> Workload:
    """A reduced copy of a configuration (fewer layers / requests / tokens) for parity tests."""
    return dataclasses.replace(w, **kw)


def _gen(device, *key: int) -> torch.Generator:
    g = torch.Generator(device=device)
    s = 0x9E3779B97F4A7C15
    for k in key:
        s = ((s ^ (int(k) + 0x632BE59BD9B4E019)) * 0xD6E8FEB86659FD93) & 0x7FFFFFFFFFFFFFFF
    g.manual_seed(s)
    return g


def topic(w: Workload, layer: int, b: int, device="cpu") -> torch.Tensor:
    """Unit 'topic' directions u [Hkv, d] fp32 of one (layer, request)."""
    g = _gen("cpu", w.seed, 11, layer, b)
    u = torch.randn(w.n_kv_heads, w.head_dim, generator=g, dtype=torch.float32)
    u = u / u.norm(dim=-1, keepdim=True)
    return u.to(device)


def config1_queries(w: Workload) -> torch.Tensor:
    """Config 1's two query tokens [B=1, 2, Hq, d] bf16 (token 0 current, 1 speculated), CPU seed 0."""
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed)
    q = torch.randn(1, 2, w.n_q_heads, w.head_dim, generator=g, dtype=torch.float32)
    return q.to(torch.bfloat16)


def queries(w: Workload, step: int, layer: int, device="cpu") -> torch.Tensor:
    """Queries of one (step, layer): [B, 2, Hq, d] bf16, token 0 = current, token 1 = speculated.

    step = -1 gives the queries of the priming selection (only token 1 is used).
    Topic workloads mix the (layer, request, KV head) topic direction into both
    tokens, which is what makes the speculated token's selection resemble the
    current token's."""
    if w.structure == "needle_q":
        q = config1_queries(w)
        if step > 0 or step < 0:
            g = _gen("cpu", w.seed, 13, step + 1, layer)
            q = torch.randn(q.shape, generator=g, dtype=torch.float32).to(torch.bfloat16)
        return q.to(device)
    B, Hq, d, G = w.batch, w.n_q_heads, w.head_dim, w.n_q_heads // w.n_kv_heads

    def spec_noise(t):
        return torch.randn(B, 1, Hq, d, generator=_gen("cpu", w.seed, 17, t + 1, layer), dtype=torch.float32)

    # The speculated token of a step stands for the next step's real token (Sec. 4.1): the current token of
    # step t is the speculated token of step t-1 seen through noise. The first step's current token pairs
    # with the priming query (step -1).
    rho = w.spec_fidelity
    fresh = torch.randn(B, 1, Hq, d, generator=_gen("cpu", w.seed, 31, step + 1, layer), dtype=torch.float32)
    cur = rho * spec_noise(step - 1) + math.sqrt(1.0 - rho * rho) * fresh if step >= 0 else fresh
    noise = torch.cat([cur, spec_noise(step)], dim=1)
    if w.structure == "iid" or w.structure == "windows":
        return noise.to(torch.bfloat16).to(device)
    u = torch.stack([topic(w, layer, b) for b in range(B)])            # [B, Hkv, d]
    u = u.repeat_interleave(G, dim=1)[:, None]                          # [B, 1, Hq, d]
    q = w.query_topic * math.sqrt(d) * u + math.sqrt(1.0 - w.query_topic ** 2) * noise
    return q.to(torch.bfloat16).to(device)


def kv_slab(w: Workload, layer: int, b: int, device="cpu") -> torch.Tensor:
    """K and V of one (layer, request): [Hkv, P, 2, T, d] bf16, [:, :, 0] = K, [:, :, 1] = V.

    Tokens at positions >= ctx inside the last page are drawn like any other
    (the path must ignore them)."""
    Hkv, P, T, d = w.n_kv_heads, w.n_pages, w.page_tokens, w.head_dim
    g = _gen(device, w.seed, 19, layer, b)
    chunk_pages = max(1, min(P, (64 << 20) // (Hkv * 2 * T * d * 4)))
    slab = torch.empty(Hkv, P, 2, T, d, dtype=torch.bfloat16, device=device)
    for p0 in range(0, P, chunk_pages):
        p1 = min(P, p0 + chunk_pages)
        slab[:, p0:p1] = torch.randn(Hkv, p1 - p0, 2, T, d, generator=g, dtype=torch.float32,
                                     device=device).to(torch.bfloat16)

    def put_keys(h, pos, val):                         # token position -> (page, offset) of the K half
        slab[h, pos // T, 0, pos % T] = val.to(torch.bfloat16)

    def get_keys(h, pos):
        return slab[h, pos // T, 0, pos % T].float()

    gc = _gen("cpu", w.seed, 23, layer, b)
    if w.structure == "needle_q":
        q = config1_queries(w)[0, 1].float()            # speculated token [Hq, d]
        G = w.n_q_heads // Hkv
        for h in range(Hkv):
            qm = q[h * G:(h + 1) * G].mean(dim=0)
            qhat = (qm / qm.norm()).to(device)
            pos = torch.randperm(w.ctx, generator=gc)[: w.n_needles].to(device)
            put_keys(h, pos, (w.needle_gain * qhat).expand(pos.numel(), d))
    elif w.structure == "needle_topic":
        u = topic(w, layer, b, device)
        for h in range(Hkv):
            pos = torch.randperm(w.ctx, generator=gc)[: w.n_needles].to(device)
            put_keys(h, pos, (w.needle_gain * u[h]).expand(pos.numel(), d))
    elif w.structure == "zipf_topic":
        u = topic(w, layer, b, device)
        n_plant = max(1, int(round(w.planted_frac * w.ctx)))
        weights = torch.arange(1, w.ctx + 1, dtype=torch.float64).pow(-w.zipf_a)
        for h in range(Hkv):
            # distinct distances z from the end of the context, Zipf-weighted (no collisions)
            z = torch.multinomial(weights, n_plant, replacement=False, generator=gc) + 1
            pos = (w.ctx - z).to(device)
            nz = torch.randn(n_plant, d, generator=g, dtype=torch.float32, device=device)
            put_keys(h, pos, w.topic_gain * u[h] + w.planted_noise * nz)
    elif w.structure == "windows":
        n_win_slots = w.ctx // w.window_tokens
        n_win = max(1, int(round(w.window_frac * w.ctx / w.window_tokens)))
        for h in range(Hkv):
            starts = torch.randperm(n_win_slots, generator=gc)[:n_win].to(device) * w.window_tokens
            pos = (starts[:, None] + torch.arange(w.window_tokens, device=device)[None, :]).reshape(-1)
            put_keys(h, pos, get_keys(h, pos) * w.window_norm)
    elif w.structure != "iid":
        raise ValueError(w.structure)
    return slab


def needle_positions(w: Workload, layer: int, b: int) -> torch.Tensor:
    """Token positions [Hkv, n_needles] of the needles `kv_slab` plants in a needle workload (same draws)."""
    if w.structure not in ("needle_q", "needle_topic"):
        raise ValueError("not a needle workload")
    gc = _gen("cpu", w.seed, 23, layer, b)
    return torch.stack([torch.randperm(w.ctx, generator=gc)[: w.n_needles] for _ in range(w.n_kv_heads)])


def ctx_lens(w: Workload, ragged: bool = False) -> torch.Tensor:
    """Context length of every request [B] int32. `ragged` shortens the requests
    unequally (to non-multiples of the page size) for the parity tests."""
    n = torch.full((w.batch,), w.ctx, dtype=torch.int32)
    if ragged:
        g = _gen("cpu", w.seed, 29)
        lo = max(w.budget + 1, w.ctx // 2)
        n = torch.randint(lo, w.ctx + 1, (w.batch,), generator=g, dtype=torch.int32)
        n[0] = w.ctx - 5 if w.ctx - 5 >= lo else w.ctx
    return n
