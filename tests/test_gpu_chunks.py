"""GPU parity of finer landmarks: several chunk landmarks per page, a page scoring as its best chunk."""
import numpy as np
import pytest
import torch

from oracle import dd_oracle as orc
from paper_2607_26475_b200 import workloads as wl
from tests._util import check_attention, check_selection, f32

pytestmark = pytest.mark.gpu

HQ, HKV, D, T = 32, 8, 128, 16


@pytest.fixture(scope="module")
def dd():
    from paper_2607_26475_b200 import binding
    return binding


@pytest.mark.parametrize("c", [8, 4, 1])
def test_chunk_landmarks_and_selection_match_the_oracle(dd, c):
    R = T // c
    w = wl.small(wl.CONFIGS[2], n_layers=1, batch=3, ctx=16 * 150, budget=16 * 12)
    kv = torch.stack([wl.kv_slab(w, 0, b) for b in range(w.batch)]).pin_memory()
    ctx_len = torch.tensor([16 * 150, 16 * 150 - 7, 16 * 90 + 1], dtype=torch.int32)
    npg = ((ctx_len + T - 1) // T).to(torch.int32)
    n_chunks = ((ctx_len + c - 1) // c).numpy()
    q = wl.queries(w, 0, 0)
    ctx = dd.Context(n_layers=1, batch=w.batch, max_pages=w.n_pages, k_pages=w.k_pages, forced_recent_pages=2,
                     landmark_chunk_tokens=c)
    lm = torch.full((w.batch, HKV, w.n_pages * R, D), 5.0, dtype=torch.bfloat16, device="cuda")
    ctx.build_landmarks(kv, ctx_len.cuda(), lm)
    torch.cuda.synchronize()
    want_lm = orc.build_landmarks(f32(kv[:, :, :, 0]), ctx_len.numpy(), chunk_tokens=c)
    assert np.array_equal(f32(lm), want_lm)
    idx = torch.empty((w.batch, HKV, w.k_pages), dtype=torch.int32, device="cuda")
    sc = torch.full((w.batch, HKV, w.n_pages), -1.0, dtype=torch.float32, device="cuda")
    with pytest.raises(dd.DDError):                       # the page-level call needs ctx_len on such a context
        ctx.select_topk(q.cuda(), 1, lm, npg.cuda(), idx)
    ctx.select_topk_chunked(q.cuda(), 1, lm, npg.cuda(), ctx_len.cuda(), idx, sc)
    assert ctx.device_error() == (0, 0)
    _, want_sc = orc.select_topk(f32(q)[:, 1], want_lm, npg.numpy(), w.k_pages, 2, chunks_per_page=R, n_chunks=n_chunks)
    got = idx.cpu().numpy()
    for b in range(w.batch):
        n = int(npg[b])
        np.testing.assert_allclose(sc.cpu().numpy()[b, :, :n], want_sc[b], rtol=2e-4)
        for h in range(HKV):
            check_selection(got[b, h], want_sc[b][h], w.k_pages, 2)
    ctx.close()


def test_whole_page_chunks_equal_the_page_level_path(dd):
    B, P, k = 2, 200, 16
    g = torch.Generator().manual_seed(3)
    lm = torch.randn(B, HKV, P, D, generator=g).to(torch.bfloat16).cuda()
    q = torch.randn(B, 2, HQ, D, generator=g).to(torch.bfloat16).cuda()
    cl = torch.tensor([P * T, P * T - 20], dtype=torch.int32).cuda()
    npg = torch.tensor([P, P - 1], dtype=torch.int32).cuda()
    a = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=k)
    b = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=k, landmark_chunk_tokens=16)
    ia = torch.empty((B, HKV, k), dtype=torch.int32, device="cuda")
    ib = torch.empty_like(ia)
    a.select_topk(q, 1, lm, npg, ia)
    b.select_topk_chunked(q, 1, lm, npg, cl, ib)
    torch.cuda.synchronize()
    assert torch.equal(ia, ib)
    a.close(); b.close()


def test_pipeline_with_two_chunks_per_page(dd):
    S, c = 2, 8
    R = T // c
    w = wl.small(wl.CONFIGS[2], n_layers=2, batch=2, ctx=16 * 80, budget=16 * 10)
    L, B = w.n_layers, w.batch
    store = [torch.stack([wl.kv_slab(w, l, b) for b in range(B)]).pin_memory() for l in range(L)]
    ctx_len = wl.ctx_lens(w, ragged=True)
    npg = ((ctx_len + T - 1) // T).to(torch.int32)
    n_chunks = ((ctx_len + c - 1) // c).numpy()
    lms = [orc.build_landmarks(f32(store[l][:, :, :, 0]), ctx_len.numpy(), chunk_tokens=c) for l in range(L)]
    q_init = torch.stack([wl.queries(w, -1, l)[:, 1] for l in range(L)])
    q_steps = torch.stack([torch.stack([wl.queries(w, t, l) for l in range(L)]) for t in range(S)])
    cx = dd.Context(n_layers=L, batch=B, max_pages=w.n_pages, k_pages=w.k_pages, landmark_chunk_tokens=c)
    cx.bind([torch.from_numpy(x).to(torch.bfloat16).cuda() for x in lms], store, npg.cuda(), ctx_len.cuda())
    cx.prime(q_init.cuda())
    qd = q_steps.cuda()
    outs = torch.zeros_like(qd)
    idxs = []
    for t in range(S):
        idxs.append(torch.stack([cx.get_indices(t & 1, l) for l in range(L)]).cpu().numpy())
        for l in range(L):
            cx.decode_layer_step(t, l, qd[t, l], outs[t, l])
    cx.sync()
    assert cx.device_error() == (0, 0)
    for t in range(S):
        for l in range(L):
            qsel = f32(q_init[l]) if t == 0 else f32(q_steps[t - 1, l][:, 1])
            _, sc = orc.select_topk(qsel, lms[l], npg.numpy(), w.k_pages, chunks_per_page=R, n_chunks=n_chunks)
            for b in range(B):
                for h in range(HKV):
                    check_selection(idxs[t][l][b, h], sc[b][h], w.k_pages, 0)
            slot = orc.gather_kv(f32(store[l]), idxs[t][l])
            want, _ = orc.sparse_decode_attn(f32(q_steps[t, l]), slot, idxs[t][l], ctx_len.numpy(), T)
            check_attention(outs[t, l], want)
    cx.close()


def test_chunked_selection_on_long_requests_with_forced_pages(dd):
    """Config 4's per-request shape (8192 pages, 256 selected, 8 forced) with four landmarks per page and a context
    that ends inside a page: several blocks per cluster, 64 KiB of logits per block."""
    B, P, k, forced, c = 1, 8192, 256, 8, 4
    R = T // c
    g = torch.Generator().manual_seed(9)
    lm = torch.randn(B, HKV, P * R, D, generator=g).to(torch.bfloat16)
    q = torch.randn(B, 2, HQ, D, generator=g).to(torch.bfloat16)
    ctx_len = torch.tensor([P * T - 9], dtype=torch.int32)        # the last page has two of its four chunks
    npg = torch.tensor([P], dtype=torch.int32)
    n_chunks = ((ctx_len + c - 1) // c).numpy()
    lm[:, :, int(n_chunks[0]):] = 50.0                            # chunks that do not exist must not matter
    cx = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=k, forced_recent_pages=forced, landmark_chunk_tokens=c)
    idx = torch.empty((B, HKV, k), dtype=torch.int32, device="cuda")
    sc = torch.empty((B, HKV, P), dtype=torch.float32, device="cuda")
    cx.select_topk_chunked(q.cuda(), 1, lm.cuda(), npg.cuda(), ctx_len.cuda(), idx, sc)
    assert cx.device_error() == (0, 0)
    _, want_sc = orc.select_topk(f32(q)[:, 1], f32(lm), npg.numpy(), k, forced, chunks_per_page=R, n_chunks=n_chunks)
    np.testing.assert_allclose(sc.cpu().numpy()[0], want_sc[0], rtol=2e-4)
    for h in range(HKV):
        check_selection(idx.cpu().numpy()[0, h], want_sc[0][h], k, forced)
    cx.close()
