"""The seeded input generators: shapes, determinism and the structure each configuration plants."""
import dataclasses

import torch

from paper_2607_26475_b200 import workloads as wl


def test_config_table_matches_the_benchmark_shapes():
    c = wl.CONFIGS
    assert (c[1].n_pages, c[1].k_pages) == (256, 16)
    assert (c[2].n_pages, c[2].k_pages, c[2].batch, c[2].n_layers, c[2].steps) == (2048, 128, 8, 32, 64)
    assert (c[3].k_pages, c[3].batch) == (64, 32)
    assert (c[4].n_pages, c[4].k_pages, c[4].forced_recent_pages) == (8192, 256, 8)
    assert (c[5].n_pages, c[5].k_pages, c[5].batch) == (65536, 512, 1)
    assert c[2].page_bytes == 8192
    assert c[2].slab_bytes * c[2].batch * c[2].n_layers == 32 << 30
    assert c[2].gathered_bytes_per_layer == 64 << 20


def test_slabs_and_queries_are_deterministic_and_distinct():
    w = wl.small(wl.CONFIGS[2], n_layers=2, batch=2, ctx=1024, budget=128)
    a = wl.kv_slab(w, 1, 0)
    b = wl.kv_slab(w, 1, 0)
    c = wl.kv_slab(w, 1, 1)
    assert a.shape == (8, 64, 2, 16, 128) and a.dtype == torch.bfloat16
    assert torch.equal(a, b) and not torch.equal(a, c)
    q0, q1 = wl.queries(w, 0, 1), wl.queries(w, 0, 1)
    assert q0.shape == (2, 2, 32, 128) and torch.equal(q0, q1)
    assert not torch.equal(q0, wl.queries(w, 1, 1))
    assert not torch.equal(q0, wl.queries(w, -1, 1))


def test_config1_needles_are_four_times_the_normalised_query_direction():
    w = wl.CONFIGS[1]
    slab = wl.kv_slab(w, 0, 0)
    q = wl.config1_queries(w)[0, 1].float()
    keys = slab[:, :, 0].reshape(8, 4096, 128).float()
    for g in range(8):
        qm = q[4 * g:4 * g + 4].mean(0)
        needle = (4.0 * qm / qm.norm()).to(torch.bfloat16).float()
        hits = (keys[g] == needle).all(dim=-1)
        assert hits.sum().item() == 8
        assert sorted(hits.nonzero().flatten().tolist()) == sorted(wl.needle_positions(w, 0, 0)[g].tolist())


def test_zipf_planted_tokens_crowd_the_recent_end():
    w = wl.small(wl.CONFIGS[2], n_layers=1, batch=1, ctx=8192, budget=256)
    slab = wl.kv_slab(w, 0, 0)
    u = wl.topic(w, 0, 0)
    keys = slab[:, :, 0].reshape(8, 8192, 128).float()
    align = torch.einsum("gtd,gd->gt", keys, u)
    planted = align > 6.0                       # topic gain sqrt(128) = 11.3 vs N(0,1) noise
    n = planted.sum(dim=1)
    assert torch.all((n >= 75) & (n <= 90))     # 1% of 8192 = 82
    assert planted[:, 4096:].sum() > 3 * planted[:, :4096].sum()


def test_windows_have_elevated_norm_and_ragged_lengths_keep_the_budget_feasible():
    w = wl.small(wl.CONFIGS[4], n_layers=1, batch=3, ctx=4096, budget=512)
    slab = wl.kv_slab(w, 0, 0)
    norms = slab[:, :, 0].reshape(8, 4096, 128).float().norm(dim=-1)
    frac = (norms > 17.0).float().mean().item()  # ordinary keys have norm ~11.3, elevated ~22.6
    assert 0.08 < frac < 0.12
    n = wl.ctx_lens(w, ragged=True)
    assert n.dtype == torch.int32 and int(n[0]) == 4091
    assert all(int(x) > w.budget and int(x) <= w.ctx for x in n)
    assert torch.equal(wl.ctx_lens(w), torch.full((3,), 4096, dtype=torch.int32))
    assert dataclasses.asdict(w)["recent_window"] == 128
