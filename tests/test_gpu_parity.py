"""GPU parity: every kernel of the C-ABI library against the CPU oracle on the same seeded inputs.

Integer and byte results (gathered pages, landmarks' bits) must be identical. Selected sets must obey
the band rule: exact wherever the k-th and (k+1)-th scores differ by more than 1e-3 relative.
Attention (bf16 in, fp32 accumulate, bf16 out): max-abs <= 2e-2, mean-abs <= 2e-3.
"""
import numpy as np
import pytest
import torch

from oracle import dd_oracle as orc
from paper_2607_26475_b200 import workloads as wl
from tests._util import check_attention, check_selection, f32, raw16

pytestmark = pytest.mark.gpu

HQ, HKV, D, T = 32, 8, 128, 16


@pytest.fixture(scope="module")
def dd():
    from paper_2607_26475_b200 import binding
    return binding


@pytest.fixture(params=["stream", "split", "tc"])
def attn_mode(request, dd):
    """All three attention kernels serve the same entry points."""
    return {"stream": dd.DD_ATTN_STREAM, "split": dd.DD_ATTN_SPLIT, "tc": dd.DD_ATTN_TC}[request.param]


def _layer_store(w, layer, pinned=True):
    """One layer of the host store [B, Hkv, P, 2, T, d] bf16 (pinned) from the seeded generator."""
    kv = torch.stack([wl.kv_slab(w, layer, b) for b in range(w.batch)])
    return kv.pin_memory() if pinned else kv


def _select_case(dd, B, P, k, forced, n_pages, seed, G=4, Tq=2, scale=1.0, select_mode=0):
    Hq = HKV * G
    g = torch.Generator().manual_seed(seed)
    lm = torch.randn(B, HKV, P, D, generator=g).mul(scale).to(torch.bfloat16)
    q = torch.randn(B, Tq, Hq, D, generator=g).to(torch.bfloat16)
    npg = torch.tensor(n_pages, dtype=torch.int32)
    ctx = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=k, n_q_heads=Hq, n_kv_heads=HKV,
                     forced_recent_pages=forced, n_q_tokens=Tq, select_mode=select_mode)
    idx = torch.full((B, HKV, k), -7, dtype=torch.int32, device="cuda")
    scores = torch.full((B, HKV, P), -1.0, dtype=torch.float32, device="cuda")
    qt = Tq - 1
    ctx.select_topk(q.cuda(), qt, lm.cuda(), npg.cuda(), idx, scores)
    assert ctx.device_error() == (0, 0)
    want_idx, want_scores = orc.select_topk(f32(q)[:, qt], f32(lm), npg.numpy(), k, forced)
    got, got_sc = idx.cpu().numpy(), scores.cpu().numpy()
    n_exact = 0
    for b in range(B):
        n = int(npg[b])
        np.testing.assert_allclose(got_sc[b, :, :n], want_scores[b], rtol=2e-4, atol=1e-30)
        assert np.all(got_sc[b, :, n:] == -1.0), "scores beyond n_pages must not be written"
        for h in range(HKV):
            n_exact += check_selection(got[b, h], want_scores[b][h], k, forced)
    ctx.close()
    return n_exact, B * HKV, got, want_idx


def test_landmarks_bit_exact_from_pinned_and_device_memory(dd):
    w = wl.small(wl.CONFIGS[2], n_layers=1, batch=3, ctx=16 * 37, budget=64)
    kv = _layer_store(w, 0)
    ctx_len = torch.tensor([16 * 37, 16 * 37 - 5, 16 * 20 + 1], dtype=torch.int32)
    c = dd.Context(n_layers=1, batch=3, max_pages=37, k_pages=4)
    want = orc.build_landmarks(f32(kv[:, :, :, 0]), ctx_len.numpy())
    for src in (kv, kv.cuda()):
        lm = torch.full((3, HKV, 37, D), 9.0, dtype=torch.bfloat16, device="cuda")
        c.build_landmarks(src, ctx_len.cuda(), lm)
        torch.cuda.synchronize()
        assert np.array_equal(f32(lm), want)
    c.close()


def test_select_config1_shape_needles(dd):
    """Config 1: 4096-token context, 256 pages, budget 256 tokens = 16 pages, planted needles."""
    w = wl.CONFIGS[1]
    kv = _layer_store(w, 0, pinned=False)
    q = wl.queries(w, 0, 0)
    ctx_len = wl.ctx_lens(w)
    lm = torch.from_numpy(orc.build_landmarks(f32(kv[:, :, :, 0]), ctx_len.numpy())).to(torch.bfloat16)
    npg = torch.tensor([w.n_pages], dtype=torch.int32)
    c = dd.Context(n_layers=1, batch=1, max_pages=w.n_pages, k_pages=w.k_pages)
    idx = torch.empty((1, HKV, w.k_pages), dtype=torch.int32, device="cuda")
    sc = torch.empty((1, HKV, w.n_pages), dtype=torch.float32, device="cuda")
    c.select_topk(q.cuda(), 1, lm.cuda(), npg.cuda(), idx, sc)
    assert c.device_error() == (0, 0)
    _, want_sc = orc.select_topk(f32(q)[:, 1], f32(lm), npg.numpy(), w.k_pages)
    for h in range(HKV):
        check_selection(idx.cpu().numpy()[0, h], want_sc[0][h], w.k_pages, 0)
    np.testing.assert_allclose(sc.cpu().numpy()[0], want_sc[0], rtol=2e-4)
    c.close()


@pytest.mark.parametrize("B,P,k,forced,n_pages,G,Tq", [
    (3, 700, 37, 3, [700, 655, 129], 4, 2),        # several tiles, ragged tails, forced recent pages
    (2, 128, 128, 0, [128, 128], 4, 2),            # budget = every page
    (2, 300, 40, 40, [300, 41], 4, 1),             # every slot forced; one request barely larger than k
    (1, 2048, 128, 0, [2048], 4, 2),               # config 2's per-request shape
    (1, 8192, 256, 8, [8192], 4, 2),               # config 4's per-request shape
    (2, 517, 16, 0, [517, 300], 1, 2),             # G = 1 (MHA), odd page count
    (2, 260, 9, 1, [260, 259], 8, 1),              # G = 8
])
@pytest.mark.parametrize("select_mode", [0, 1], ids=["fused", "two_kernels"])
def test_select_band_rule_and_scores(dd, B, P, k, forced, n_pages, G, Tq, select_mode):
    n_exact, n_all, got, _ = _select_case(dd, B, P, k, forced, n_pages, seed=P + k, G=G, Tq=Tq, select_mode=select_mode)
    assert n_exact >= 1 or n_all == 0
    if select_mode == 0:       # both kernels take the decision in the same arithmetic: same sets, bit for bit
        _, _, got2, _ = _select_case(dd, B, P, k, forced, n_pages, seed=P + k, G=G, Tq=Tq, select_mode=1)
        assert np.array_equal(got, got2)


def test_select_well_separated_scores_are_bit_exact(dd):
    """Sharper landmarks spread the scores, so nearly every (request, head) must match the oracle exactly."""
    for mode in (0, 1):
        n_exact, n_all, got, want = _select_case(dd, 4, 1000, 20, 2, [1000, 990, 512, 77], seed=5, scale=3.0,
                                                 select_mode=mode)
        assert n_exact >= n_all - 2
        assert (got == want).mean() > 0.98


def test_select_long_request_uses_the_global_key_path(dd):
    """More pages than fit in shared memory (config 5's regime, reduced): keys live in global scratch."""
    for mode in (0, 1):
        n_exact, n_all, _, _ = _select_case(dd, 1, 20000, 300, 0, [19997], seed=11, select_mode=mode)
        assert n_all == HKV


def test_select_ties_go_to_the_lower_page(dd):
    """Identical landmarks give identical scores: the set must be the first k pages (plus the forced ones)."""
    B, P, k, forced = 1, 200, 10, 2
    lm = torch.randn(1, HKV, 1, D).expand(1, HKV, P, D).contiguous().to(torch.bfloat16)
    q = torch.randn(1, 2, HQ, D).to(torch.bfloat16)
    for mode in (0, 1):
        c = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=k, forced_recent_pages=forced, select_mode=mode)
        idx = torch.empty((B, HKV, k), dtype=torch.int32, device="cuda")
        c.select_topk(q.cuda(), 1, lm.cuda(), torch.tensor([P], dtype=torch.int32).cuda(), idx)
        assert c.device_error() == (0, 0)
        want = list(range(k - forced)) + [P - 2, P - 1]
        assert all(idx.cpu().numpy()[0, h].tolist() == want for h in range(HKV))
        c.close()


@pytest.mark.parametrize("mode", ["loads", "bulk"])
def test_gather_is_a_bit_copy_and_leaves_canaries_alone(dd, mode):
    w = wl.small(wl.CONFIGS[2], n_layers=1, batch=3, ctx=16 * 211, budget=16 * 37)
    kv = _layer_store(w, 0)
    P, k = w.n_pages, w.k_pages
    g = torch.Generator().manual_seed(3)
    idx = torch.stack([torch.stack([torch.randperm(P, generator=g)[:k].sort().values for _ in range(HKV)])
                       for _ in range(w.batch)]).to(torch.int32)
    guard = 4096
    gm = dd.DD_GATHER_BULK if mode == "bulk" else dd.DD_GATHER_LOADS
    probe = dd.Context(n_layers=1, batch=w.batch, max_pages=P, k_pages=k, ring_depth=3)
    ring_bytes = probe.ring_bytes()
    slot_bytes = probe.slot_bytes()
    probe.close()
    assert slot_bytes == w.batch * HKV * k * 8192 and ring_bytes == 3 * slot_bytes
    big = torch.full((guard + ring_bytes + guard,), 0xAB, dtype=torch.uint8, device="cuda")
    c = dd.Context(n_layers=1, batch=w.batch, max_pages=P, k_pages=k, ring_depth=3, gather_mode=gm,
                   ring=big[guard:guard + ring_bytes])
    c.gather_kv_from_host(kv, idx.cuda(), None, 1)
    assert c.device_error() == (0, 0)
    want = orc.gather_kv(raw16(kv), idx.numpy())
    assert np.array_equal(raw16(c.slot_tensor(1)), want)
    host = big.cpu().numpy()
    assert np.all(host[:guard] == 0xAB) and np.all(host[guard + ring_bytes:] == 0xAB)
    assert np.all(host[guard:guard + slot_bytes] == 0xAB)                      # slot 0 untouched
    assert np.all(host[guard + 2 * slot_bytes:guard + ring_bytes] == 0xAB)     # slot 2 untouched
    # the same gather from a device-resident copy of the store
    c.gather_kv_from_host(kv.cuda(), idx.cuda(), None, 2)
    torch.cuda.synchronize()
    assert np.array_equal(raw16(c.slot_tensor(2)), want)
    c.close()


def test_gather_rejects_pageable_memory_and_clamps_bad_indices(dd):
    B, P, k = 1, 40, 4
    c = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=k)
    kv = torch.randn(B, HKV, P, 2, T, D).to(torch.bfloat16)
    idx = torch.tensor([0, 1, 2, 3], dtype=torch.int32).repeat(B, HKV, 1)
    with pytest.raises(dd.DDError) as e:
        c.gather_kv_from_host(kv, idx.cuda(), None, 0)                # pageable host memory
    assert e.value.code == dd.DD_ERR_NOT_PINNED
    with pytest.raises(dd.DDError) as e:
        c.gather_kv_from_host(kv.pin_memory(), idx.cuda(), None, 2)   # slot outside the ring
    assert e.value.code == dd.DD_ERR_INVALID_ARG
    with pytest.raises(dd.DDError) as e:
        c.gather_kv_from_host(kv.pin_memory(), idx, None, 0)          # idx must be device memory
    assert e.value.code == dd.DD_ERR_INVALID_ARG
    bad = idx.clone()
    bad[0, 3, 2] = P + 5                                              # beyond the store: clamped, reported
    pinned = kv.pin_memory()
    c.gather_kv_from_host(pinned, bad.cuda(), None, 0)
    code, detail = c.device_error()
    assert (code, detail) == (dd.DD_ERR_INDEX_RANGE, P + 5)
    fixed = bad.clone()
    fixed[0, 3, 2] = P - 1
    assert np.array_equal(raw16(c.slot_tensor(0)), orc.gather_kv(raw16(pinned), fixed.numpy()))
    assert c.device_error() == (0, 0)                                 # the error word was cleared
    # with n_pages given, the limit is the request's own page count
    c.gather_kv_from_host(pinned, idx.cuda(), torch.tensor([3], dtype=torch.int32).cuda(), 0)
    assert c.device_error() == (dd.DD_ERR_INDEX_RANGE, 3)
    c.close()


def _attn_case(dd, B, P, k, ctx_len, Tq, splits, seed, G=4, sharp=1.0, attn_mode=0):
    Hq = HKV * G
    g = torch.Generator().manual_seed(seed)
    kv = torch.randn(B, HKV, P, 2, T, D, generator=g).to(torch.bfloat16).pin_memory()
    q = (torch.randn(B, Tq, Hq, D, generator=g) * sharp).to(torch.bfloat16)
    idx = torch.stack([torch.stack([torch.randperm(P, generator=g)[:k].sort().values for _ in range(HKV)])
                       for _ in range(B)]).to(torch.int32)
    cl = torch.tensor(ctx_len, dtype=torch.int32)
    for b in range(B):                       # make sure the last (possibly partial) page is in some sets
        last = (int(cl[b]) - 1) // T
        idx[b, ::2, -1] = last
        idx[b] = idx[b].clamp(max=last)
        for h in range(HKV):                 # clamping may duplicate: rebuild as a sorted unique set
            s = sorted(set(idx[b, h].tolist()))
            fill = [p for p in range(last + 1) if p not in s]
            idx[b, h] = torch.tensor(sorted(s + fill[:k - len(s)]), dtype=torch.int32)
    c = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=k, n_q_heads=Hq, n_q_tokens=Tq, attn_splits=splits,
                   attn_mode=attn_mode)
    c.gather_kv_from_host(kv, idx.cuda(), None, 0)
    out = torch.full((B, Tq, Hq, D), 7.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((B, Tq, Hq), dtype=torch.float32, device="cuda")
    c.sparse_decode_attn(q.cuda(), 0, idx.cuda(), cl.cuda(), out, lse)
    assert c.device_error() == (0, 0)
    slot = orc.gather_kv(f32(kv), idx.numpy())
    want, want_lse = orc.sparse_decode_attn(f32(q), slot, idx.numpy(), cl.numpy(), T)
    check_attention(out, want)
    np.testing.assert_allclose(lse.cpu().numpy(), want_lse, atol=2e-3, rtol=1e-4)
    c.close()


@pytest.mark.parametrize("B,P,k,ctx_len,Tq,splits", [
    (1, 256, 16, [4096], 2, 0),                    # config 1 shape
    (2, 100, 23, [1600, 1589], 2, 1),              # one split, ragged last page
    (2, 100, 23, [1600, 1589], 2, 5),              # splits that do not divide k
    (3, 300, 128, [4800, 4799, 2049], 2, 0),       # config 2's budget, automatic splits
    (2, 64, 3, [1024, 1000], 1, 3),                # fewer pages than warps; single query token
    (1, 40, 40, [633], 2, 7),                      # full budget, partial last page
])
def test_attention_matches_oracle(dd, attn_mode, B, P, k, ctx_len, Tq, splits):
    _attn_case(dd, B, P, k, ctx_len, Tq, splits, seed=B * 1000 + k, attn_mode=attn_mode)


def test_attention_sharp_queries_and_other_group_sizes(dd, attn_mode):
    _attn_case(dd, 2, 128, 32, [2048, 2040], 2, 0, seed=1, sharp=4.0, attn_mode=attn_mode)     # peaked soft-max
    _attn_case(dd, 2, 128, 32, [2048, 2040], 2, 0, seed=2, G=2, attn_mode=attn_mode)
    _attn_case(dd, 2, 128, 32, [2048, 2040], 1, 4, seed=3, G=8, attn_mode=attn_mode)
    _attn_case(dd, 1, 128, 32, [2048], 2, 2, seed=4, G=1, attn_mode=attn_mode)


@pytest.mark.parametrize("mode", ["stream", "tc"])
def test_streaming_attention_when_blocks_cut_units_at_every_offset(dd, mode):
    """Shapes whose flat page list is cut into per-block runs that start and end inside units, cover several whole
    units, or hold fewer pages than consumer warps (or than a tile): many requests with few pages, one with many."""
    attn_mode = dd.DD_ATTN_STREAM if mode == "stream" else dd.DD_ATTN_TC
    for B, P, k, seed in [(16, 40, 5, 1), (9, 64, 7, 2), (1, 4096, 1200, 3), (5, 200, 66, 4), (32, 64, 64, 5)]:
        _attn_case(dd, B, P, k, [P * 16 - (3 * b) % 15 for b in range(B)], 2, 0, seed=seed, attn_mode=attn_mode)


def test_full_budget_equals_dense_attention(dd):
    """Budget = context: selection returns every page and the result is dense GQA attention (torch SDPA)."""
    B, P = 2, 48
    w = wl.small(wl.CONFIGS[2], n_layers=1, batch=B, ctx=P * T, budget=P * T)
    kv = _layer_store(w, 0)
    q = wl.queries(w, 0, 0)
    cl = torch.tensor([P * T, P * T - 9], dtype=torch.int32)
    npg = torch.tensor([P, P], dtype=torch.int32)
    lm = torch.from_numpy(orc.build_landmarks(f32(kv[:, :, :, 0]), cl.numpy())).to(torch.bfloat16)
    c = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=P)
    idx = torch.empty((B, HKV, P), dtype=torch.int32, device="cuda")
    c.select_topk(q.cuda(), 1, lm.cuda(), npg.cuda(), idx)
    c.gather_kv_from_host(kv, idx, npg.cuda(), 0)
    out = torch.empty((B, 2, HQ, D), dtype=torch.bfloat16, device="cuda")
    c.sparse_decode_attn(q.cuda(), 0, idx, cl.cuda(), out)
    assert c.device_error() == (0, 0)
    assert np.array_equal(idx.cpu().numpy(), np.tile(np.arange(P, dtype=np.int32), (B, HKV, 1)))
    for b in range(B):
        n = int(cl[b])
        K = kv[b, :, :, 0].reshape(HKV, P * T, D)[:, :n].double().repeat_interleave(4, dim=0)
        V = kv[b, :, :, 1].reshape(HKV, P * T, D)[:, :n].double().repeat_interleave(4, dim=0)
        Q = q[b].double().permute(1, 0, 2)
        ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V).permute(1, 0, 2).numpy()
        check_attention(out[b], ref)
    c.close()


@pytest.mark.parametrize("B,P,k,ctx_len,Tq,splits,G", [
    (2, 100, 23, [1600, 1589], 2, 0, 4),
    (2, 100, 23, [1600, 1589], 2, 5, 4),           # several clusters: the tail enters through the global merge
    (1, 256, 16, [4096], 2, 1, 4),
    (2, 64, 8, [1024, 1001], 1, 2, 8),             # one query token: it sees only its own new entry
    (3, 300, 128, [4800, 4799, 2049], 2, 0, 2),
])
def test_attention_with_causal_tail_matches_oracle(dd, attn_mode, B, P, k, ctx_len, Tq, splits, G):
    Hq = HKV * G
    g = torch.Generator().manual_seed(B * 77 + k)
    kv = torch.randn(B, HKV, P, 2, T, D, generator=g).to(torch.bfloat16).pin_memory()
    q = torch.randn(B, Tq, Hq, D, generator=g).to(torch.bfloat16)
    k_new = torch.randn(B, Tq, HKV, D, generator=g).to(torch.bfloat16)
    v_new = (torch.randn(B, Tq, HKV, D, generator=g) * 3).to(torch.bfloat16)
    k_new[0, 0, 0] = (4.0 * q[0, 0, 0].float()).to(torch.bfloat16)     # one new key that dominates its row
    cl = torch.tensor(ctx_len, dtype=torch.int32)
    idx = torch.empty((B, HKV, k), dtype=torch.int32)
    for b in range(B):
        last = (int(cl[b]) - 1) // T
        for h in range(HKV):
            s = torch.randperm(last, generator=g)[:k - 1].tolist() + [last]
            idx[b, h] = torch.tensor(sorted(s), dtype=torch.int32)
    c = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=k, n_q_heads=Hq, n_q_tokens=Tq, attn_splits=splits,
                   attn_mode=attn_mode)
    c.gather_kv_from_host(kv, idx.cuda(), None, 0)
    out = torch.full((B, Tq, Hq, D), 7.0, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((B, Tq, Hq), dtype=torch.float32, device="cuda")
    c.sparse_decode_attn_causal(q.cuda(), 0, idx.cuda(), cl.cuda(), k_new.cuda(), v_new.cuda(), out, lse)
    assert c.device_error() == (0, 0)
    slot = orc.gather_kv(f32(kv), idx.numpy())
    want, want_lse = orc.sparse_decode_attn_causal(f32(q), slot, idx.numpy(), cl.numpy(), T, f32(k_new), f32(v_new))
    check_attention(out, want)
    np.testing.assert_allclose(lse.cpu().numpy(), want_lse, atol=2e-3, rtol=1e-4)
    base, _ = orc.sparse_decode_attn(f32(q), slot, idx.numpy(), cl.numpy(), T)
    assert np.abs(want - base).max() > 0.1          # the tail matters in this case
    c.close()


def test_select_precondition_violation_is_reported_and_stays_in_range(dd):
    """A request with fewer pages than the budget violates k <= n_pages: no trap, the error word is set, and the
    indices written stay inside the request (the valid pages first, then the last valid page repeated)."""
    B, P, k = 2, 64, 20
    g = torch.Generator().manual_seed(2)
    lm = torch.randn(B, HKV, P, D, generator=g).to(torch.bfloat16).cuda()
    q = torch.randn(B, 2, HQ, D, generator=g).to(torch.bfloat16).cuda()
    for mode in (0, 1):
        c = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=k, select_mode=mode)
        idx = torch.full((B, HKV, k), -1, dtype=torch.int32, device="cuda")
        c.select_topk(q, 1, lm, torch.tensor([64, 7], dtype=torch.int32).cuda(), idx)
        code, detail = c.device_error()
        assert (code, detail) == (dd.DD_ERR_INDEX_RANGE, 7)
        got = idx.cpu().numpy()
        assert np.all(np.diff(got[0], axis=-1) > 0)                      # the healthy request is unaffected
        assert all(got[1, h].tolist() == list(range(7)) + [6] * (k - 7) for h in range(HKV))
        # a request that claims more pages than the layout holds is clamped to the layout
        c.select_topk(q, 1, lm, torch.tensor([64, 1000], dtype=torch.int32).cuda(), idx)
        assert c.device_error() == (dd.DD_ERR_INDEX_RANGE, 1000)
        assert idx.max().item() < P and idx.min().item() >= 0
        c.close()


def test_smallest_geometry(dd):
    """One request, one KV head, one query head, one query token, one page selected out of one."""
    kv = torch.randn(1, 1, 1, 2, T, D).to(torch.bfloat16).pin_memory()
    q = torch.randn(1, 1, 1, D).to(torch.bfloat16)
    cl = torch.tensor([11], dtype=torch.int32)
    npg = torch.tensor([1], dtype=torch.int32)
    c = dd.Context(n_layers=1, batch=1, max_pages=1, k_pages=1, n_q_heads=1, n_kv_heads=1, n_q_tokens=1)
    lm = torch.empty((1, 1, 1, D), dtype=torch.bfloat16, device="cuda")
    c.build_landmarks(kv, cl.cuda(), lm)
    idx = torch.full((1, 1, 1), 9, dtype=torch.int32, device="cuda")
    c.select_topk(q.cuda(), 0, lm, npg.cuda(), idx)
    c.gather_kv_from_host(kv, idx, npg.cuda(), 0)
    out = torch.empty((1, 1, 1, D), dtype=torch.bfloat16, device="cuda")
    c.sparse_decode_attn(q.cuda(), 0, idx, cl.cuda(), out)
    assert c.device_error() == (0, 0)
    assert idx.item() == 0
    assert np.array_equal(f32(lm), orc.build_landmarks(f32(kv[:, :, :, 0]), cl.numpy()))
    slot = orc.gather_kv(f32(kv), idx.cpu().numpy())
    want, _ = orc.sparse_decode_attn(f32(q), slot, idx.cpu().numpy(), cl.numpy(), T)
    check_attention(out, want)
    c.close()
