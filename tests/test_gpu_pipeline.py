"""GPU parity of the pipelined layer step (ring + events) against the oracle's multi-step chain,
its invariance to ring depth and gather engine, its call-order checks, and a sampled check at
config 2's full launch configuration (32 layers, batch 8, 2048 pages, 128 selected)."""
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


def _inputs(w, S, ragged=True):
    L, B = w.n_layers, w.batch
    store = [torch.stack([wl.kv_slab(w, l, b) for b in range(B)]).pin_memory() for l in range(L)]
    ctx_len = wl.ctx_lens(w, ragged=ragged)
    npg = ((ctx_len + T - 1) // T).to(torch.int32)
    lms = [torch.from_numpy(orc.build_landmarks(f32(store[l][:, :, :, 0]), ctx_len.numpy())).to(torch.bfloat16)
           for l in range(L)]
    q_init = torch.stack([wl.queries(w, -1, l)[:, 1] for l in range(L)])                   # [L, B, Hq, d]
    q_steps = torch.stack([torch.stack([wl.queries(w, t, l) for l in range(L)]) for t in range(S)])
    return store, lms, ctx_len, npg, q_init, q_steps


def _run(dd, w, S, inp, depth, mode=0, read_idx=True, one_stream=False, side_select=False, ctx_kw=None):
    store, lms, ctx_len, npg, q_init, q_steps = inp
    L, B = w.n_layers, w.batch
    streams = {}
    if one_stream:                # fully synchronous schedule: gathers, attention and selection on one stream
        st = torch.cuda.Stream()
        streams = dict(compute_stream=st, copy_stream=st)
    if side_select:               # the next-step selection on a stream of its own, next to the attention
        streams = dict(select_stream=torch.cuda.Stream())
    c = dd.Context(n_layers=L, batch=B, max_pages=w.n_pages, k_pages=w.k_pages,
                   forced_recent_pages=w.forced_recent_pages, ring_depth=depth, gather_mode=mode, **streams,
                   **(ctx_kw or {}))
    lm_dev = [x.cuda() for x in lms]
    c.bind(lm_dev, store, npg.cuda(), ctx_len.cuda())
    c.prime(q_init.cuda())
    qd = q_steps.cuda()
    outs = torch.zeros_like(qd)
    idxs = []
    for t in range(S):
        if read_idx:
            idxs.append(torch.stack([c.get_indices(t & 1, l) for l in range(L)]).cpu().numpy())
        for l in range(L):
            c.decode_layer_step(t, l, qd[t, l], outs[t, l])
    c.sync()
    assert c.device_error() == (0, 0)
    c.close()
    return outs, (np.stack(idxs) if read_idx else None)


def test_chain_matches_oracle_and_is_invariant_to_ring_depth_and_engine(dd):
    S = 3
    w = wl.small(wl.CONFIGS[4], n_layers=3, batch=2, ctx=16 * 90, budget=16 * 12, recent_window=32)
    inp = _inputs(w, S)
    store, lms, ctx_len, npg, q_init, q_steps = inp
    outs, idxs = _run(dd, w, S, inp, depth=2)
    # selection of every (step, layer): band rule against the oracle's scores for the query that produced it
    for t in range(S):
        for l in range(w.n_layers):
            qsel = f32(q_init[l]) if t == 0 else f32(q_steps[t - 1, l][:, 1])
            _, sc = orc.select_topk(qsel, f32(lms[l]), npg.numpy(), w.k_pages, w.forced_recent_pages)
            for b in range(w.batch):
                for h in range(HKV):
                    check_selection(idxs[t, l, b, h], sc[b][h], w.k_pages, w.forced_recent_pages)
            # attention over the GPU's own set
            slot = orc.gather_kv(f32(store[l]), idxs[t, l])
            want, _ = orc.sparse_decode_attn(f32(q_steps[t, l]), slot, idxs[t, l], ctx_len.numpy(), T)
            check_attention(outs[t, l], want)
    # the whole chain in the oracle, when every set matched exactly
    o_outs, o_idxs = orc.decode_chain(f32(q_init), f32(q_steps), [f32(x) for x in lms], [f32(x) for x in store],
                                      npg.numpy(), ctx_len.numpy(), w.k_pages, T, w.forced_recent_pages)
    if np.array_equal(o_idxs[:S], idxs):
        check_attention(outs, o_outs)
    # same bits whatever the ring depth, the gather engine, with no host reads in between, and with the whole
    # schedule serialised on a single stream
    for depth, mode, read, one in [(3, 0, True, False), (4, 0, False, False), (2, 1, False, False), (2, 0, False, False),
                                   (2, 0, False, True), (2, 0, False, "side")]:
        o2, i2 = _run(dd, w, S, inp, depth=depth, mode=mode, read_idx=read, one_stream=one is True,
                      side_select=one == "side")
        assert np.array_equal(raw16(o2), raw16(outs)), (depth, mode, one)
        if read:
            assert np.array_equal(i2, idxs)


@pytest.mark.parametrize("mode", ["stream", "tc"])
def test_chain_with_the_streaming_attention_kernel(dd, mode):
    """The pipelined step with the TMA-fed attention kernels (mma.sync consumers, or tcgen05 with accumulators in tensor
    memory): same index sets, outputs equal to the split-KV kernel's up to rounding (partial results are merged in
    different orders) and within tolerance of the oracle."""
    attn_mode = dd.DD_ATTN_STREAM if mode == "stream" else dd.DD_ATTN_TC
    S = 3
    w = wl.small(wl.CONFIGS[4], n_layers=3, batch=2, ctx=16 * 90, budget=16 * 12, recent_window=32)
    inp = _inputs(w, S)
    store, lms, ctx_len, npg, q_init, q_steps = inp
    want, want_idx = _run(dd, w, S, inp, depth=2)
    for depth in (2, 3):
        got, got_idx = _run(dd, w, S, inp, depth=depth, ctx_kw=dict(attn_mode=attn_mode))
        assert np.array_equal(got_idx, want_idx)
        assert np.abs(f32(got) - f32(want)).max() <= 2e-2
        for t in range(S):
            for l in range(w.n_layers):
                slot = orc.gather_kv(f32(store[l]), got_idx[t, l])
                ref, _ = orc.sparse_decode_attn(f32(q_steps[t, l]), slot, got_idx[t, l], ctx_len.numpy(), T)
                check_attention(got[t, l], ref)


def test_single_layer_model_with_a_deeper_ring(dd):
    """Config 1's shape: one layer, two slots; the next step's gather is released by this step's selection."""
    S = 4
    w = wl.small(wl.CONFIGS[1], steps=S)
    inp = _inputs(w, S, ragged=False)
    store, lms, ctx_len, npg, q_init, q_steps = inp
    outs, idxs = _run(dd, w, S, inp, depth=2)
    for t in range(S):
        slot = orc.gather_kv(f32(store[0]), idxs[t, 0])
        want, _ = orc.sparse_decode_attn(f32(q_steps[t, 0]), slot, idxs[t, 0], ctx_len.numpy(), T)
        check_attention(outs[t, 0], want)
        qsel = f32(q_init[0]) if t == 0 else f32(q_steps[t - 1, 0][:, 1])
        _, sc = orc.select_topk(qsel, f32(lms[0]), npg.numpy(), w.k_pages)
        for h in range(HKV):
            check_selection(idxs[t, 0, 0, h], sc[0][h], w.k_pages, 0)


def test_layer_step_with_causal_tail(dd):
    """The pipelined step with the tokens' own new KV entries appended (output token first, then the
    speculated token, which also sees the output token's entry)."""
    S = 2
    w = wl.small(wl.CONFIGS[2], n_layers=2, batch=2, ctx=16 * 70, budget=16 * 9)
    store, lms, ctx_len, npg, q_init, q_steps = _inputs(w, S)
    g = torch.Generator().manual_seed(5)
    k_new = torch.randn(S, w.n_layers, w.batch, 2, HKV, D, generator=g).to(torch.bfloat16)
    v_new = torch.randn(S, w.n_layers, w.batch, 2, HKV, D, generator=g).to(torch.bfloat16)
    c = dd.Context(n_layers=w.n_layers, batch=w.batch, max_pages=w.n_pages, k_pages=w.k_pages)
    c.bind([x.cuda() for x in lms], store, npg.cuda(), ctx_len.cuda())
    c.prime(q_init.cuda())
    qd, kd, vd = q_steps.cuda(), k_new.cuda(), v_new.cuda()
    outs = torch.zeros_like(qd)
    idxs = []
    for t in range(S):
        idxs.append(torch.stack([c.get_indices(t & 1, l) for l in range(w.n_layers)]).cpu().numpy())
        for l in range(w.n_layers):
            c.decode_layer_step_causal(t, l, qd[t, l], kd[t, l], vd[t, l], outs[t, l])
    c.sync()
    assert c.device_error() == (0, 0)
    for t in range(S):
        for l in range(w.n_layers):
            slot = orc.gather_kv(f32(store[l]), idxs[t][l])
            want, _ = orc.sparse_decode_attn_causal(f32(q_steps[t, l]), slot, idxs[t][l], ctx_len.numpy(), T,
                                                    f32(k_new[t, l]), f32(v_new[t, l]))
            check_attention(outs[t, l], want)
    c.close()


def test_timeline_api(dd):
    """Trace capacity, row shape and the state checks of the timeline calls (the schedule rules themselves are
    replayed in test_gpu_schedule.py)."""
    S = 3
    w = wl.small(wl.CONFIGS[2], n_layers=4, batch=2, ctx=16 * 200, budget=16 * 40)
    store, lms, ctx_len, npg, q_init, q_steps = _inputs(w, S)
    L = w.n_layers
    c = dd.Context(n_layers=L, batch=w.batch, max_pages=w.n_pages, k_pages=w.k_pages)
    with pytest.raises(dd.DDError) as e:
        c.trace_end()
    assert e.value.code == dd.DD_ERR_STATE
    c.bind([x.cuda() for x in lms], store, npg.cuda(), ctx_len.cuda())
    c.prime(q_init.cuda())
    qd = q_steps.cuda()
    outs = torch.zeros_like(qd)
    c.trace_begin(S * L - 2)                       # capacity smaller than the run: the rest is not recorded
    for t in range(S):
        for l in range(L):
            c.decode_layer_step(t, l, qd[t, l], outs[t, l])
    tr = c.trace_end()
    assert tr.shape == (S * L - 2, dd.DD_TRACE_FIELDS)
    assert tr[0, 0] >= 0.0
    assert np.all(tr[:, 6:] == -1.0)                           # no urgent stream without miss correction
    assert np.all(np.diff(tr[:, :4], axis=1) >= 0.0)          # points 0..3 are ordered within a call
    assert np.all(tr[:, 5] > tr[:, 4])                         # a gather takes time
    c.close()


def test_whole_step_from_host_buffers(dd):
    """dd_decode_step_host gives the same bits as the layer-by-layer calls on device tensors."""
    S = 2
    w = wl.small(wl.CONFIGS[2], n_layers=3, batch=2, ctx=16 * 60, budget=16 * 8)
    inp = _inputs(w, S)
    store, lms, ctx_len, npg, q_init, q_steps = inp
    want, _ = _run(dd, w, S, inp, depth=2, read_idx=False)
    c = dd.Context(n_layers=w.n_layers, batch=w.batch, max_pages=w.n_pages, k_pages=w.k_pages)
    c.bind([x.cuda() for x in lms], store, npg.cuda(), ctx_len.cuda())
    c.prime(q_init.cuda())
    qh = q_steps.pin_memory()
    oh = torch.zeros_like(q_steps).pin_memory()
    for t in range(S):
        c.decode_step_host(t, qh[t], oh[t])
    c.sync()
    assert c.device_error() == (0, 0)
    assert np.array_equal(raw16(oh), raw16(want))
    with pytest.raises(dd.DDError) as e:
        c.decode_step_host(S, q_steps[0].clone(), oh[0])          # pageable queries
    assert e.value.code == dd.DD_ERR_NOT_PINNED
    c.close()


def test_call_order_is_checked(dd):
    w = wl.small(wl.CONFIGS[2], n_layers=2, batch=1, ctx=16 * 40, budget=16 * 4)
    inp = _inputs(w, 1, ragged=False)
    store, lms, ctx_len, npg, q_init, q_steps = inp
    c = dd.Context(n_layers=2, batch=1, max_pages=40, k_pages=4)
    q = q_steps[0, 0].cuda()
    out = torch.empty_like(q)
    with pytest.raises(dd.DDError) as e:
        c.prime(q_init.cuda())
    assert e.value.code == dd.DD_ERR_STATE
    with pytest.raises(dd.DDError) as e:
        c.decode_layer_step(0, 0, q, out)
    assert e.value.code == dd.DD_ERR_STATE
    with pytest.raises(dd.DDError) as e:
        c.bind([x.cuda() for x in lms], [s.clone() for s in store], npg.cuda(), ctx_len.cuda())   # not pinned
    assert e.value.code == dd.DD_ERR_NOT_PINNED
    c.bind([x.cuda() for x in lms], store, npg.cuda(), ctx_len.cuda())
    c.prime(q_init.cuda())
    with pytest.raises(dd.DDError) as e:
        c.decode_layer_step(0, 1, q, out)          # layer 0 comes first
    assert e.value.code == dd.DD_ERR_STATE
    c.decode_layer_step(0, 0, q, out)
    c.decode_layer_step(0, 1, q, out)
    with pytest.raises(dd.DDError) as e:
        c.decode_layer_step(0, 1, q, out)          # already done
    assert e.value.code == dd.DD_ERR_STATE
    c.decode_layer_step(1, 0, q, out)
    c.sync()
    assert c.device_error() == (0, 0)
    c.close()


def test_invalid_configurations_are_rejected(dd):
    for kw in (dict(head_dim=64), dict(page_tokens=32), dict(k_pages=50), dict(ring_depth=1), dict(n_q_heads=30),
               dict(forced_recent_pages=9), dict(n_q_heads=64, n_q_tokens=2), dict(gather_mode=5)):
        args = dict(n_layers=1, batch=1, max_pages=40, k_pages=8)
        args.update(kw)
        with pytest.raises(dd.DDError) as e:
            dd.Context(**args)
        assert e.value.code == dd.DD_ERR_INVALID_ARG


@pytest.mark.parametrize("cfg,n_phys,samples", [
    (2, 2, [(0, 0, 0), (0, 17, 7), (1, 31, 3), (1, 16, 0)]),
    (3, 1, [(0, 5, 31), (1, 30, 0)]),
    (4, 1, [(0, 0, 7), (1, 31, 2)]),
    (5, 1, [(0, 3, 0), (1, 28, 0)]),
])
def test_full_launch_configuration_sampled(dd, cfg, n_phys, samples):
    """Configs 2-5 as the benchmark launches them (32 layers, full batch, full context and budget, ring depth
    2). The host store aliases `n_phys` physical layers to stay small; sampled (step, layer, request)
    outputs are checked one by one against the oracle."""
    w = wl.CONFIGS[cfg]
    L, B, P, k, S, F = w.n_layers, w.batch, w.n_pages, w.k_pages, 2, w.forced_recent_pages
    ctx_len = wl.ctx_lens(w)
    npg = torch.full((B,), P, dtype=torch.int32)
    c = dd.Context(n_layers=L, batch=B, max_pages=P, k_pages=k, forced_recent_pages=F)
    one = dd.Context(n_layers=1, batch=1, max_pages=P, k_pages=1)
    phys, lms = [], []
    for l in range(n_phys):
        host = torch.empty((B, HKV, P, 2, T, D), dtype=torch.bfloat16, pin_memory=True)
        lm = torch.empty((B, HKV, P, D), dtype=torch.bfloat16, device="cuda")
        for b in range(B):
            dev = wl.kv_slab(w, l, b, device="cuda")
            one.build_landmarks(dev, ctx_len[b:b + 1].cuda(), lm[b])
            host[b].copy_(dev)
            del dev
        phys.append(host)
        lms.append(lm)
    torch.cuda.synchronize()
    one.close()
    store = [phys[l % n_phys] for l in range(L)]
    lm_l = [lms[l % n_phys] for l in range(L)]
    q_init = torch.stack([wl.queries(w, -1, l)[:, 1] for l in range(L)])
    q_steps = torch.stack([torch.stack([wl.queries(w, t, l) for l in range(L)]) for t in range(S)])
    c.bind(lm_l, store, npg.cuda(), ctx_len.cuda())
    c.prime(q_init.cuda())
    qd = q_steps.cuda()
    outs = torch.zeros_like(qd)
    idxs = []
    for t in range(S):
        idxs.append(torch.stack([c.get_indices(t & 1, l) for l in range(L)]).cpu().numpy())
        for l in range(L):
            c.decode_layer_step(t, l, qd[t, l], outs[t, l])
    c.sync()
    assert c.device_error() == (0, 0)
    n_exact = n_all = 0
    for t, l, b in samples:
        kv_b = store[l][b:b + 1]
        lm_want = orc.build_landmarks(f32(kv_b[:, :, :, 0]), ctx_len[b:b + 1].numpy())
        assert np.array_equal(f32(lm_l[l][b:b + 1]), lm_want), "device-built landmarks differ from the oracle's"
        qsel = f32(q_init[l][b:b + 1]) if t == 0 else f32(q_steps[t - 1, l][b:b + 1, 1])
        _, sc = orc.select_topk(qsel, lm_want, npg[b:b + 1].numpy(), k, F)
        got = idxs[t][l][b:b + 1]
        for h in range(HKV):
            n_exact += check_selection(got[0, h], sc[0][h], k, F)
            n_all += 1
        slot_bits = orc.gather_kv(raw16(kv_b), got)                     # bit copy of the selected pages only
        slot = (slot_bits.astype(np.uint32) << 16).view(np.float32)
        want, _ = orc.sparse_decode_attn(f32(q_steps[t, l][b:b + 1]), slot, got, ctx_len[b:b + 1].numpy(), T)
        check_attention(outs[t, l][b:b + 1], want)
    print(f"config {cfg}: exact index sets {n_exact}/{n_all}")
    c.close()
