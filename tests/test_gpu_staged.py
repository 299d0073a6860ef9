"""The staged gather (copy engine -> staging region -> assembly kernel, short runs by zero-copy loads):
bit-exact against the oracle's page copy for exact runs, for every run threshold and for aligned-block
over-fetch; canaries intact; host-side index checks; and the pipelined chain gives the same bits as with
the direct gather."""
import numpy as np
import pytest
import torch

from oracle import dd_oracle as orc
from paper_2607_26475_b200 import workloads as wl
from tests._util import raw16
from tests.test_gpu_pipeline import _inputs, _run

pytestmark = pytest.mark.gpu

HKV, D, T = 8, 128, 16


@pytest.fixture(scope="module")
def dd():
    from paper_2607_26475_b200 import binding
    return binding


def _index_sets_with_runs(B, P, k, seed):
    """Ascending sets that mix isolated pages with runs of 2..12 adjacent pages (and one run that ends at
    the last page of the request)."""
    g = torch.Generator().manual_seed(seed)
    out = torch.empty((B, HKV, k), dtype=torch.int32)
    for b in range(B):
        for h in range(HKV):
            chosen = set()
            if (b + h) % 3 == 0:
                chosen.update(range(P - 5, P))
            while len(chosen) < k:
                start = int(torch.randint(0, P, (1,), generator=g))
                run = int(torch.randint(1, 13, (1,), generator=g)) if torch.rand(1, generator=g) < 0.3 else 1
                for p in range(start, min(P, start + run)):
                    if len(chosen) < k:
                        chosen.add(p)
            out[b, h] = torch.tensor(sorted(chosen), dtype=torch.int32)
    return out


@pytest.mark.parametrize("min_run,block", [(0, 0), (1, 0), (4, 0), (1000, 0), (0, 4), (0, 8), (0, 32)])
def test_staged_gather_is_a_bit_copy(dd, min_run, block):
    B, P, k = 3, 211, 61
    g = torch.Generator().manual_seed(11)
    kv = torch.randn(B, HKV, P, 2, T, D, generator=g).to(torch.bfloat16).pin_memory()
    idx = _index_sets_with_runs(B, P, k, seed=5)
    guard = 4096
    probe = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=k, ring_depth=3)
    ring_bytes, slot_bytes = probe.ring_bytes(), probe.slot_bytes()
    probe.close()
    big = torch.full((guard + ring_bytes + guard,), 0xAB, dtype=torch.uint8, device="cuda")
    c = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=k, ring_depth=3, gather_mode=dd.DD_GATHER_STAGED,
                   stage_min_run_pages=min_run, stage_block_pages=block, ring=big[guard:guard + ring_bytes])
    want = orc.gather_kv(raw16(kv), idx.numpy())
    for rep in range(2):                       # the second call reuses staging region and descriptor buffers
        c.gather_kv_from_host(kv, idx.cuda(), None, 1)
        assert c.device_error() == (0, 0)
        assert np.array_equal(raw16(c.slot_tensor(1)), want)
    host = big.cpu().numpy()
    assert np.all(host[:guard] == 0xAB) and np.all(host[guard + ring_bytes:] == 0xAB)
    assert np.all(host[guard:guard + slot_bytes] == 0xAB)
    assert np.all(host[guard + 2 * slot_bytes:guard + ring_bytes] == 0xAB)
    st = c.gather_stats()
    total = B * HKV * k
    assert st["gathers"] == 2 and st["pages_staged"] + st["pages_zero_copy"] == 2 * total
    if block:
        assert st["pages_zero_copy"] == 0 and st["copied_bytes"] >= 2 * total * 8192
    elif min_run == 1:
        assert st["pages_zero_copy"] == 0 and st["copied_bytes"] == 2 * total * 8192
    elif min_run == 1000:
        assert st["pages_staged"] == 0 and st["copies"] == 0
    else:
        assert st["copied_bytes"] == st["pages_staged"] * 8192 and st["copies"] > 0 and st["pages_zero_copy"] > 0
    # more than DD_STAGE_LISTS gathers in a row: the descriptor buffers are recycled behind their events
    idx2 = _index_sets_with_runs(B, P, k, seed=6)
    for rep in range(10):
        c.gather_kv_from_host(kv, (idx if rep % 2 else idx2).cuda(), None, rep % 3)
    torch.cuda.synchronize()
    assert np.array_equal(raw16(c.slot_tensor(0)), orc.gather_kv(raw16(kv), idx.numpy()))      # rep 9 -> slot 0
    assert np.array_equal(raw16(c.slot_tensor(2)), orc.gather_kv(raw16(kv), idx2.numpy()))     # rep 8 -> slot 2
    c.close()


def test_staged_gather_checks_indices_on_the_host(dd):
    B, P, k = 1, 40, 4
    kv = torch.randn(B, HKV, P, 2, T, D).to(torch.bfloat16).pin_memory()
    idx = torch.tensor([0, 1, 2, 3], dtype=torch.int32).repeat(B, HKV, 1)
    for block in (0, 8):
        c = dd.Context(n_layers=1, batch=B, max_pages=P, k_pages=k, gather_mode=dd.DD_GATHER_STAGED,
                       stage_min_run_pages=2, stage_block_pages=block)
        bad = idx.clone()
        bad[0, 3, 3] = P + 5
        c.gather_kv_from_host(kv, bad.cuda(), None, 0)
        assert c.last_device_error() == (dd.DD_ERR_INDEX_RANGE, P + 5)      # visible without synchronising
        assert c.device_error() == (dd.DD_ERR_INDEX_RANGE, P + 5)
        fixed = bad.clone()
        fixed[0, 3, 3] = P - 1
        assert np.array_equal(raw16(c.slot_tensor(0)), orc.gather_kv(raw16(kv), fixed.numpy()))
        assert c.device_error() == (0, 0) and c.last_device_error() == (0, 0)
        c.gather_kv_from_host(kv, idx.cuda(), torch.tensor([3], dtype=torch.int32).cuda(), 0)
        assert c.device_error() == (dd.DD_ERR_INDEX_RANGE, 3)
        c.close()
    with pytest.raises(dd.DDError) as e:
        dd.Context(n_layers=1, batch=1, max_pages=40, k_pages=4, gather_mode=dd.DD_GATHER_STAGED, stage_block_pages=3)
    assert e.value.code == dd.DD_ERR_INVALID_ARG


@pytest.mark.parametrize("depth,kw", [(2, dict(stage_min_run_pages=2)), (3, dict(stage_min_run_pages=1)),
                                      (4, dict(stage_block_pages=4)), (2, dict(stage_min_run_pages=2, side=True))])
def test_chain_with_the_staged_gather_equals_the_direct_gather(dd, depth, kw):
    """Ring invariance extended to the staged engine: same output bits and same index sets as the zero-copy
    gather, for ring depths 2..4, exact runs and aligned blocks, with and without a selection stream."""
    S = 3
    w = wl.small(wl.CONFIGS[4], n_layers=3, batch=2, ctx=16 * 90, budget=16 * 12, recent_window=32)
    inp = _inputs(w, S)
    kw = dict(kw)
    side = kw.pop("side", False)
    want, want_idx = _run(dd, w, S, inp, depth=2)
    got, got_idx = _run(dd, w, S, inp, depth=depth, mode=dd.DD_GATHER_STAGED, side_select=side, ctx_kw=kw)
    assert np.array_equal(raw16(got), raw16(want))
    assert np.array_equal(got_idx, want_idx)
    # one layer and a deeper ring: the host needs the set selected in the same call
    w1 = wl.small(wl.CONFIGS[1], steps=S)
    inp1 = _inputs(w1, S, ragged=False)
    a, ai = _run(dd, w1, S, inp1, depth=2)
    b, bi = _run(dd, w1, S, inp1, depth=2, mode=dd.DD_GATHER_STAGED, ctx_kw=dict(stage_min_run_pages=1))
    assert np.array_equal(raw16(a), raw16(b)) and np.array_equal(ai, bi)


def test_whole_step_from_host_buffers_with_the_staged_gather(dd):
    """dd_decode_step_host on a context with the staged gather: same bits as the layer-by-layer calls with the
    direct gather, and the counters show that both the copy engine and the zero-copy kernel carried pages."""
    S = 3
    w = wl.small(wl.CONFIGS[2], n_layers=3, batch=2, ctx=16 * 80, budget=16 * 20)
    inp = _inputs(w, S)
    store, lms, ctx_len, npg, q_init, q_steps = inp
    want, _ = _run(dd, w, S, inp, depth=2, read_idx=False)
    c = dd.Context(n_layers=w.n_layers, batch=w.batch, max_pages=w.n_pages, k_pages=w.k_pages,
                   gather_mode=dd.DD_GATHER_STAGED, stage_min_run_pages=2)
    c.bind([x.cuda() for x in lms], store, npg.cuda(), ctx_len.cuda())
    c.prime(q_init.cuda())
    qh = q_steps.pin_memory()
    oh = torch.zeros_like(q_steps).pin_memory()
    for t in range(S):
        c.decode_step_host(t, qh[t], oh[t])
    c.sync()
    assert c.device_error() == (0, 0)
    assert np.array_equal(raw16(oh), raw16(want))
    st = c.gather_stats()
    assert st["gathers"] >= S * w.n_layers and st["pages_staged"] > 0 and st["pages_zero_copy"] > 0
    c.close()
