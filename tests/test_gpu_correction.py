"""GPU parity of the miss correction (urgent-stream repair of the predicted set) against the oracle."""
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


def test_diff_and_fetch_match_the_oracle_bit_for_bit(dd):
    B, P, k = 3, 300, 41
    g = torch.Generator().manual_seed(7)
    kv = torch.randn(B, HKV, P, 2, T, D, generator=g).to(torch.bfloat16).pin_memory()

    def rand_sets(overlap):
        out = torch.empty((B, HKV, k), dtype=torch.int32)
        for b in range(B):
            for h in range(HKV):
                out[b, h] = torch.randperm(P, generator=g)[:k].sort().values
        return out
    pred = rand_sets(0)
    true = rand_sets(0)
    true[0, 0] = pred[0, 0]                       # no miss at all
    true[0, 1, :-1] = pred[0, 1, :-1]             # at most one miss
    true[0, 1, -1] = P - 1 if int(pred[0, 1, -1]) != P - 1 else int(pred[0, 1, -2]) + 1
    true[0, 1] = true[0, 1].sort().values
    c = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=k, ring_depth=2)
    for slot in (1, 0):
        merged = torch.full((B, HKV, k), -1, dtype=torch.int32, device="cuda")
        c.gather_kv_from_host(kv, pred.cuda(), None, slot)
        c.diff_indices(pred.cuda(), true.cuda(), slot, merged)
        c.fetch_missing_from_host(kv, slot)
        assert c.device_error() == (0, 0)
        want_merged, fixes, n_miss = orc.correct_misses(pred.numpy(), true.numpy())
        assert np.array_equal(merged.cpu().numpy(), want_merged)
        assert np.array_equal(raw16(c.slot_tensor(slot)), orc.gather_kv(raw16(kv), want_merged))
    missing, selected = c.miss_stats(reset=True)
    assert missing == 2 * int(n_miss.sum()) and selected == 2 * B * HKV * k
    assert int(n_miss[0, 0]) == 0 and int(n_miss[0, 1]) <= 1
    assert c.miss_stats() == (0, 0)
    c.close()


def _inputs(w, S):
    L, B = w.n_layers, w.batch
    store = [torch.stack([wl.kv_slab(w, l, b) for b in range(B)]).pin_memory() for l in range(L)]
    ctx_len = wl.ctx_lens(w, ragged=True)
    npg = ((ctx_len + T - 1) // T).to(torch.int32)
    lms = [torch.from_numpy(orc.build_landmarks(f32(store[l][:, :, :, 0]), ctx_len.numpy())).to(torch.bfloat16)
           for l in range(L)]
    q_init = torch.stack([wl.queries(w, -1, l)[:, 1] for l in range(L)])
    q_steps = torch.stack([torch.stack([wl.queries(w, t, l) for l in range(L)]) for t in range(S)])
    return store, lms, ctx_len, npg, q_init, q_steps


def _run(dd, w, S, inp, depth, correct, read=True, side_select=False):
    store, lms, ctx_len, npg, q_init, q_steps = inp
    L, B = w.n_layers, w.batch
    c = dd.Context(n_layers=L, batch=B, max_pages=w.n_pages, k_pages=w.k_pages,
                   forced_recent_pages=w.forced_recent_pages, ring_depth=depth, miss_correction=correct,
                   select_stream=torch.cuda.Stream() if side_select else None)
    c.bind([x.cuda() for x in lms], store, npg.cuda(), ctx_len.cuda())
    c.prime(q_init.cuda())
    qd = q_steps.cuda()
    outs = torch.zeros_like(qd)
    merged = np.zeros((S, L, B, HKV, w.k_pages), dtype=np.int32)
    for t in range(S):
        for l in range(L):
            c.decode_layer_step(t, l, qd[t, l], outs[t, l])
            if correct and read:
                merged[t, l] = c.get_merged_indices((t * L + l) % depth).cpu().numpy()
    c.sync()
    assert c.device_error() == (0, 0)
    stats = c.miss_stats() if correct else (0, 0)
    c.close()
    return outs, merged, stats


def test_corrected_chain_attends_the_true_sets(dd):
    """Whatever was predicted, the repaired slot holds the set selected from the current token and the output
    is attention over it; the result does not depend on ring depth, host reads in between, or the priming query."""
    S = 3
    w = wl.small(wl.CONFIGS[2], n_layers=3, batch=2, ctx=16 * 120, budget=16 * 14)
    inp = _inputs(w, S)
    store, lms, ctx_len, npg, q_init, q_steps = inp
    outs, merged, (missing, selected) = _run(dd, w, S, inp, depth=2, correct=True)
    assert selected == S * w.n_layers * w.batch * HKV * w.k_pages
    assert 0 < missing < selected                               # the prediction is useful but not perfect
    for t in range(S):
        for l in range(w.n_layers):
            _, sc = orc.select_topk(f32(q_steps[t, l][:, 0]), f32(lms[l]), npg.numpy(), w.k_pages)
            for b in range(w.batch):
                for h in range(HKV):
                    assert len(set(merged[t, l, b, h].tolist())) == w.k_pages
                    check_selection(np.sort(merged[t, l, b, h]), sc[b][h], w.k_pages, 0)   # = a valid TRUE set
            slot = orc.gather_kv(f32(store[l]), merged[t, l])
            want, _ = orc.sparse_decode_attn(f32(q_steps[t, l]), slot, merged[t, l], ctx_len.numpy(), T)
            check_attention(outs[t, l], want)
    # oracle chain with correction: identical when every true set matched exactly
    o_outs, _, o_true, o_miss = orc.decode_chain_corrected(f32(q_init), f32(q_steps), [f32(x) for x in lms],
                                                           [f32(x) for x in store], npg.numpy(), ctx_len.numpy(),
                                                           w.k_pages, T)
    if np.array_equal(np.sort(merged, axis=-1), o_true):
        check_attention(outs, o_outs)
        assert missing == int(o_miss.sum())
    # same sets and (to rounding: the buffer order differs) same outputs for other ring depths and priming queries
    for depth, shift in [(3, 0.0), (2, 2.5)]:
        inp2 = (store, lms, ctx_len, npg, (q_init.float() + shift).to(torch.bfloat16), q_steps)
        o2, m2, _ = _run(dd, w, S, inp2, depth=depth, correct=True)
        assert np.array_equal(np.sort(m2, axis=-1), np.sort(merged, axis=-1))
        assert np.abs(f32(o2) - f32(outs)).max() <= 2e-2
    # the next-step selection on its own stream changes nothing
    o4, m4, _ = _run(dd, w, S, inp, depth=2, correct=True, side_select=True)
    assert np.array_equal(m4, merged) and np.array_equal(raw16(o4), raw16(outs))
    # without correction the outputs are those of the predicted sets: they differ
    o3, _, _ = _run(dd, w, S, inp, depth=2, correct=False)
    assert np.abs(f32(o3) - f32(outs)).max() > 1e-3


def test_corrected_chain_and_causal_tail_at_the_headline_request_shape(dd):
    """The same two paths at the per-request shape of the batch-8 / 32K-context workload (2048 pages, 128
    selected per KV head), not only at toy sizes: one request, two layers, two steps."""
    S = 2
    w = wl.small(wl.CONFIGS[2], n_layers=2, batch=1)
    assert w.n_pages == 2048 and w.k_pages == 128
    inp = _inputs(w, S)
    store, lms, ctx_len, npg, q_init, q_steps = inp
    outs, merged, (missing, selected) = _run(dd, w, S, inp, depth=2, correct=True)
    assert 0 < missing < selected
    for t in range(S):
        for l in range(w.n_layers):
            _, sc = orc.select_topk(f32(q_steps[t, l][:, 0]), f32(lms[l]), npg.numpy(), w.k_pages)
            for h in range(HKV):
                check_selection(np.sort(merged[t, l, 0, h]), sc[0][h], w.k_pages, 0)
            slot = orc.gather_kv(f32(store[l]), merged[t, l])
            want, _ = orc.sparse_decode_attn(f32(q_steps[t, l]), slot, merged[t, l], ctx_len.numpy(), T)
            check_attention(outs[t, l], want)
    # causal tail through the pipelined call, same shape
    g = torch.Generator().manual_seed(9)
    k_new = torch.randn(S, w.n_layers, 1, 2, HKV, D, generator=g).to(torch.bfloat16)
    v_new = torch.randn(S, w.n_layers, 1, 2, HKV, D, generator=g).to(torch.bfloat16)
    c = dd.Context(n_layers=w.n_layers, batch=1, max_pages=w.n_pages, k_pages=w.k_pages)
    c.bind([x.cuda() for x in lms], store, npg.cuda(), ctx_len.cuda())
    c.prime(q_init.cuda())
    qd, kd, vd = q_steps.cuda(), k_new.cuda(), v_new.cuda()
    o = torch.zeros_like(qd)
    idxs = []
    for t in range(S):
        idxs.append([c.get_indices(t & 1, l).cpu().numpy() for l in range(w.n_layers)])
        for l in range(w.n_layers):
            c.decode_layer_step_causal(t, l, qd[t, l], kd[t, l], vd[t, l], o[t, l])
    c.sync()
    assert c.device_error() == (0, 0)
    c.close()
    for t in range(S):
        for l in range(w.n_layers):
            slot = orc.gather_kv(f32(store[l]), idxs[t][l])
            want, _ = orc.sparse_decode_attn_causal(f32(q_steps[t, l]), slot, idxs[t][l], ctx_len.numpy(), T,
                                                    f32(k_new[t, l]), f32(v_new[t, l]))
            check_attention(o[t, l], want)
