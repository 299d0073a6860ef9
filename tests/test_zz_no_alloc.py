"""The allocation-free attention entry point against the context-based one and against the CPU oracle.

Callers that may not allocate device memory (they run inside someone else's memory plan, or must not
trigger the device synchronisation an allocation can cause) use dd_sparse_decode_attn_static, whose
scratch is a fixed array inside the library. It must give the same result as dd_sparse_decode_attn on
the same gathered slot, call after call, although every call reuses (and finds the leftovers of the
previous call in) the same array. Collected last on purpose: a run that stops at the first failure has
then already run every other test.
"""
import numpy as np
import pytest
import torch

from tests._util import ATTN_MAX_ABS, ATTN_MEAN_ABS, check_attention, f32

pytestmark = pytest.mark.gpu

HKV, D, T = 8, 128, 16


def _case(dd, seed, B, P, k, splits_ctx, splits_static, ctx_len):
    g = torch.Generator().manual_seed(seed)
    kv = torch.randn(B, HKV, P, 2, T, D, generator=g).to(torch.bfloat16).pin_memory()
    q = torch.randn(B, 2, 32, D, generator=g).to(torch.bfloat16).cuda()
    idx = torch.stack([torch.stack([torch.randperm(P, generator=g)[:k].sort().values for _ in range(HKV)])
                       for _ in range(B)]).to(torch.int32).cuda()
    cl = torch.tensor(ctx_len, dtype=torch.int32).cuda()
    c = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=k, attn_splits=splits_ctx)
    c.gather_kv_from_host(kv, idx, None, 0)
    want = torch.empty((B, 2, 32, D), dtype=torch.bfloat16, device="cuda")
    want_lse = torch.empty((B, 2, 32), dtype=torch.float32, device="cuda")
    c.sparse_decode_attn(q, 0, idx, cl, want, want_lse)
    slot = c.slot_tensor(0)                               # the caller of the static entry point owns the slot
    got = torch.full_like(want, 3.0)
    got_lse = torch.zeros_like(want_lse)
    dd.sparse_decode_attn_static(q, slot, idx, cl, got, got_lse, n_splits=splits_static)
    torch.cuda.synchronize()
    assert c.device_error() == (0, 0)
    c.close()
    err = np.abs(f32(got).astype(np.float64) - f32(want).astype(np.float64))
    assert err.max() <= ATTN_MAX_ABS and err.mean() <= ATTN_MEAN_ABS, (err.max(), err.mean())
    np.testing.assert_allclose(got_lse.cpu().numpy(), want_lse.cpu().numpy(), atol=2e-3, rtol=1e-4)
    # and directly against the oracle, on the slot the caller handed in
    from oracle import dd_oracle as orc
    ref, ref_lse = orc.sparse_decode_attn(f32(q), f32(slot), idx.cpu().numpy(), np.asarray(ctx_len), T)
    check_attention(got, ref)
    np.testing.assert_allclose(got_lse.cpu().numpy(), ref_lse, atol=2e-3, rtol=1e-4)
    return err.max()


def test_static_entry_point_matches_the_context_entry_point_on_consecutive_calls():
    from paper_2607_26475_b200 import binding as dd
    assert dd.lib.dd_static_scratch_capacity() == 8 << 20
    # two calls in a row with different shapes and split counts: the second finds the first one's leftovers
    e1 = _case(dd, 1, B=3, P=200, k=64, splits_ctx=5, splits_static=5, ctx_len=[3200, 3190, 1700])
    e2 = _case(dd, 2, B=2, P=150, k=37, splits_ctx=1, splits_static=5, ctx_len=[2400, 2399])
    e3 = _case(dd, 3, B=3, P=200, k=64, splits_ctx=5, splits_static=5, ctx_len=[3200, 3190, 1700])
    assert e1 == 0.0 and e3 == 0.0          # same split geometry (no clusters) gives the same bits as the context path
    assert e2 <= ATTN_MAX_ABS


def test_static_entry_point_rejects_what_does_not_fit():
    from paper_2607_26475_b200 import binding as dd
    B, k = 64, 128
    q = torch.zeros((B, 2, 32, D), dtype=torch.bfloat16, device="cuda")
    idx = torch.zeros((B, HKV, k), dtype=torch.int32, device="cuda")
    cl = torch.full((B,), k * T, dtype=torch.int32, device="cuda")
    slot = torch.zeros((1,), dtype=torch.bfloat16, device="cuda")       # never touched: the call must fail first
    with pytest.raises(dd.DDError) as e:
        dd.sparse_decode_attn_static(q, slot, idx, cl, q.clone(), n_splits=8)   # 64 * 8 * 8 * 4160 B > 8 MiB
    assert e.value.code == dd.DD_ERR_INVALID_ARG and "8388608" in str(e.value)
    with pytest.raises(dd.DDError) as e:
        dd.sparse_decode_attn_static(q, slot, idx, cl, q.clone(), n_splits=k + 1)
    assert e.value.code == dd.DD_ERR_INVALID_ARG


def test_static_entry_point_rejects_memory_the_device_cannot_use():
    """Pageable host memory (or a misaligned pointer) for any tensor is an error code before anything is
    enqueued, never a device fault: the checks run on the host and launch nothing."""
    from paper_2607_26475_b200 import binding as dd
    B, k = 2, 16
    q = torch.zeros((B, 2, 32, D), dtype=torch.bfloat16, device="cuda")
    idx = torch.arange(k, dtype=torch.int32).repeat(B, HKV, 1).contiguous().cuda()
    cl = torch.full((B,), k * T, dtype=torch.int32, device="cuda")
    slot = torch.zeros((B, HKV, 2, k * T, D), dtype=torch.bfloat16, device="cuda")
    out = torch.full_like(q, 7.0)
    good = dict(q=q, slot=slot, idx=idx, ctx_len=cl, out=out)
    for name in ("q", "slot", "idx", "ctx_len", "out"):
        args = dict(good)
        args[name] = good[name].cpu()                                    # pageable host memory
        with pytest.raises(dd.DDError) as e:
            dd.sparse_decode_attn_static(args["q"], args["slot"], args["idx"], args["ctx_len"], args["out"], n_splits=2)
        assert e.value.code == dd.DD_ERR_INVALID_ARG and name in str(e.value)
    with pytest.raises(dd.DDError) as e:
        dd.sparse_decode_attn_static(q, slot, idx, cl, out, torch.zeros((B, 2, 32), dtype=torch.float32), n_splits=2)
    assert e.value.code == dd.DD_ERR_INVALID_ARG and "out_lse" in str(e.value)
    with pytest.raises(dd.DDError) as e:                                 # bf16 tensors must be 16-byte aligned
        q_off = torch.zeros(q.numel() + 8, dtype=torch.bfloat16, device="cuda")[1:1 + q.numel()].view(q.shape)
        dd.sparse_decode_attn_static(q_off, slot, idx, cl, out, n_splits=2)
    assert e.value.code == dd.DD_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())                                      # nothing ran
    dd.sparse_decode_attn_static(q, slot, idx, cl, out, n_splits=2)      # the device is still usable
    torch.cuda.synchronize()
    assert bool((out == 0.0).all())


def test_static_entry_point_inside_a_cuda_graph():
    """The call allocates nothing and is ordered by its stream only, so it can be captured: a graph that holds two
    calls (different split counts, the second finds the first one's leftovers in the scratch array) is replayed on
    fresh inputs written into the captured buffers and must give the eager call's bits."""
    from paper_2607_26475_b200 import binding as dd
    B, P, k = 2, 160, 48
    g = torch.Generator().manual_seed(9)
    idx = torch.stack([torch.stack([torch.randperm(P, generator=g)[:k].sort().values for _ in range(HKV)])
                       for _ in range(B)]).to(torch.int32).cuda()
    cl = torch.tensor([P * T, P * T - 5], dtype=torch.int32).cuda()
    q = torch.zeros(B, 2, 32, D, dtype=torch.bfloat16, device="cuda")
    slot = torch.zeros(B, HKV, 2, k * T, D, dtype=torch.bfloat16, device="cuda")
    out_a, out_b = torch.zeros_like(q), torch.zeros_like(q)
    lse_a = torch.zeros(B, 2, 32, dtype=torch.float32, device="cuda")
    # the first call on the device looks up the scratch array: before the capture begins
    dd.sparse_decode_attn_static(q, slot, idx, cl, out_a, lse_a, n_splits=1)
    torch.cuda.synchronize()
    s = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=s):
        dd.sparse_decode_attn_static(q, slot, idx, cl, out_a, lse_a, n_splits=6, stream=s)
        dd.sparse_decode_attn_static(q, slot, idx, cl, out_b, None, n_splits=3, stream=s)
    for rep in range(3):
        q.copy_(torch.randn(q.shape, generator=g).to(torch.bfloat16))
        slot.copy_(torch.randn(slot.shape, generator=g).to(torch.bfloat16))
        out_a.fill_(7.0)
        out_b.fill_(7.0)
        graph.replay()
        torch.cuda.synchronize()
        want_a, want_b = torch.zeros_like(q), torch.zeros_like(q)
        want_lse = torch.zeros_like(lse_a)
        dd.sparse_decode_attn_static(q, slot, idx, cl, want_a, want_lse, n_splits=6)
        dd.sparse_decode_attn_static(q, slot, idx, cl, want_b, None, n_splits=3)
        torch.cuda.synchronize()
        assert torch.equal(out_a, want_a) and torch.equal(out_b, want_b) and torch.equal(lse_a, want_lse)
        from oracle import dd_oracle as orc
        ref, _ = orc.sparse_decode_attn(f32(q), f32(slot), idx.cpu().numpy(), cl.cpu().numpy(), T)
        check_attention(out_a, ref)
        check_attention(out_b, ref)
