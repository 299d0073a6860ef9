"""The host's part of the staged gather (forming copy-engine copies from an index set), checked without a GPU against
a brute-force replay: every selected page must reach its slot item exactly once, either through a copy (whose bytes
are laid out as the map says) or through the zero-copy list; copies follow the run / aligned-block rules."""
import ctypes as C

import numpy as np
import pytest


@pytest.fixture(scope="module")
def lib():
    from paper_2607_26475_b200 import build
    build.build()
    from paper_2607_26475_b200 import binding
    return binding.lib


def plan(lib, idx, P, min_run, block, n_pages=None, capacity=None, max_copies=None):
    B, Hkv, k = idx.shape
    total = B * Hkv * k
    capacity = total * max(1, block) if capacity is None else capacity
    max_copies = total if max_copies is None else max_copies
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    copies = np.zeros(3 * max(1, max_copies), dtype=np.int64)
    mp = np.full(max(1, capacity), -7, dtype=np.int32)
    strag = np.full(total, -7, dtype=np.int32)
    nc, ns, nt = C.c_longlong(), C.c_longlong(), C.c_longlong()
    bad = np.zeros(2, dtype=np.int32)
    npg = None if n_pages is None else np.ascontiguousarray(n_pages, dtype=np.int32)
    rc = lib.dd_test_stage_plan(idx.ctypes.data, None if npg is None else npg.ctypes.data, B, Hkv, P, k, min_run, block,
                                capacity, copies.ctypes.data, max_copies, C.addressof(nc), mp.ctypes.data, C.addressof(ns),
                                strag.ctypes.data, C.addressof(nt), bad.ctypes.data)
    return rc, copies[:3 * nc.value].reshape(-1, 3), mp[:ns.value], strag[:nt.value], bad


def replay(idx, P, copies, mp, strag, n_pages=None):
    """Which global page (unit * P + page) ends up in every slot item."""
    B, Hkv, k = idx.shape
    got = np.full(B * Hkv * k, -1, dtype=np.int64)
    staged_src = np.full(len(mp), -1, dtype=np.int64)
    for src, dst, n in copies:
        assert n >= 1 and np.all(staged_src[dst:dst + n] == -1), "copies overlap in the staging region"
        staged_src[dst:dst + n] = src + np.arange(n)
        assert src // P == (src + n - 1) // P, "a copy crosses into the next (request, KV head)"
    assert np.all(staged_src >= 0), "a staged page is covered by no copy"
    for s, item in enumerate(mp):
        if item >= 0:
            assert got[item] == -1, "a slot item is written twice"
            got[item] = staged_src[s]
    flat = idx.reshape(-1, k)
    for item in strag:
        assert got[item] == -1, "a slot item is both staged and left to the zero-copy kernel"
        u, j = divmod(int(item), k)
        p = int(flat[u, j])
        lim = P if n_pages is None else min(P, int(n_pages[u // Hkv]))
        p = 0 if p < 0 else (max(lim - 1, 0) if p >= lim else p)
        got[item] = u * P + p
    return got


def sets_with_runs(B, Hkv, P, k, seed):
    rng = np.random.default_rng(seed)
    out = np.zeros((B, Hkv, k), dtype=np.int32)
    for b in range(B):
        for h in range(Hkv):
            chosen = set()
            if (b + h) % 3 == 0:
                chosen.update(range(P - 5, P))
            while len(chosen) < k:
                start = int(rng.integers(0, P))
                run = int(rng.integers(1, 13)) if rng.random() < 0.3 else 1
                chosen.update(range(start, min(P, start + run)))
            out[b, h] = sorted(chosen)[:k] if len(chosen) > k else sorted(chosen)
    return out


@pytest.mark.parametrize("min_run,block", [(1, 0), (2, 0), (8, 0), (1000, 0), (1, 2), (1, 4), (1, 8), (1, 32)])
def test_every_selected_page_reaches_its_slot_item_once(lib, min_run, block):
    B, Hkv, P, k = 3, 4, 211, 61
    idx = sets_with_runs(B, Hkv, P, k, seed=min_run * 7 + block)
    rc, copies, mp, strag, bad = plan(lib, idx, P, min_run, block)
    assert rc == 0 and bad[0] == 0
    got = replay(idx, P, copies, mp, strag)
    want = (np.arange(B * Hkv)[:, None] * P + idx.reshape(-1, k)).reshape(-1)
    assert np.array_equal(got, want)
    flat = idx.reshape(-1, k)
    if block == 0:
        # exact runs: a copy is a maximal run of adjacent selected pages of at least min_run pages; nothing else is staged
        assert np.all(mp >= 0) and len(mp) + len(strag) == B * Hkv * k
        assert all(n >= min_run for _, _, n in copies)
        for u in range(B * Hkv):
            row = flat[u]
            brk = np.flatnonzero(np.diff(row) != 1)
            starts = np.concatenate([[0], brk + 1])
            ends = np.concatenate([brk + 1, [k]])
            long_runs = {(u * P + int(row[a]), int(e - a)) for a, e in zip(starts, ends) if e - a >= min_run}
            mine = {(int(s), int(n)) for s, _, n in copies if s // P == u}
            assert mine == long_runs
    else:
        # aligned blocks: every copy starts on a block boundary, ends on one (or at the end of the store), holds a
        # selected page in every block, and two copies of a unit are never adjacent
        assert len(strag) == 0
        for s, _, n in copies:
            page0, page1 = int(s % P), int(s % P + n)
            assert page0 % block == 0 and (page1 % block == 0 or page1 == P)
            u = int(s // P)
            sel = set(flat[u].tolist())
            for blk in range(page0 // block, (page1 + block - 1) // block):
                assert sel & set(range(blk * block, min(P, (blk + 1) * block))), "a block without a selected page was copied"
        for u in range(B * Hkv):
            spans = sorted((int(s % P), int(s % P + n)) for s, _, n in copies if s // P == u)
            assert all(a[1] < b[0] for a, b in zip(spans, spans[1:])), "adjacent or overlapping copies were not merged"
        staged = sum(int(n) for _, _, n in copies)
        assert staged == len(mp) and staged >= B * Hkv * k and int((mp >= 0).sum()) == B * Hkv * k


def test_bad_indices_are_clamped_and_reported_and_limits_are_respected(lib):
    P, k = 40, 4
    idx = np.array([[[0, 1, 2, P + 5], [3, 4, 5, 6]]], dtype=np.int32)
    for block in (0, 8):
        rc, copies, mp, strag, bad = plan(lib, idx, P, 2, block)
        assert rc == 0 and bad.tolist() == [1, P + 5]
        got = replay(idx, P, copies, mp, strag)
        assert got.tolist() == [0, 1, 2, P - 1, P + 3, P + 4, P + 5, P + 6]
    # the request's own page count is the limit when given: 3 is out of range for a request of 3 pages
    short = np.array([[[0, 1, 2, 3]]], dtype=np.int32)
    rc, copies, mp, strag, bad = plan(lib, short, P, 2, 0, n_pages=[3])
    assert rc == 0 and bad.tolist() == [1, 3]
    assert replay(short, P, copies, mp, strag, n_pages=[3]).tolist() == [0, 1, 2, 2]
    # a plan that does not fit the staging region or the copy list is refused
    full = np.arange(k, dtype=np.int32)[None, None, :]
    assert plan(lib, full, P, 1, 0, capacity=k - 1)[0] != 0
    assert plan(lib, np.array([[[0, 2, 4, 6]]], dtype=np.int32), P, 1, 0, max_copies=3)[0] != 0
    assert plan(lib, full, P, 1, 0, capacity=k)[0] == 0
    # a set that is not ascending still reaches its items (runs are only formed from ascending neighbours)
    odd = np.array([[[5, 4, 3, 10]]], dtype=np.int32)
    for block in (0, 4):
        rc, copies, mp, strag, bad = plan(lib, odd, P, 1, block)
        assert rc == 0 and replay(odd, P, copies, mp, strag).tolist() == [5, 4, 3, 10]
