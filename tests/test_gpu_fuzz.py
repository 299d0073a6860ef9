"""Seeded random launch shapes for the selection and the attention kernels against the oracle: page counts that are
no multiple of any tile, budgets from one page to every page, unequal requests, every group size, forced pages."""
import numpy as np
import pytest

from tests.test_gpu_parity import _attn_case, _select_case

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dd():
    from paper_2607_26475_b200 import binding
    return binding


def _select_shapes(n, seed):
    rng = np.random.default_rng(seed)
    for i in range(n):
        B = int(rng.integers(1, 5))
        P = int(rng.choice([rng.integers(17, 200), rng.integers(200, 1500), rng.integers(1500, 6000)]))
        k = int(rng.choice([1, rng.integers(1, min(P, 300) + 1), min(P, 128), P if P <= 400 else 64]))
        forced = int(rng.choice([0, 0, rng.integers(0, k + 1)]))
        n_pages = [int(rng.integers(k, P + 1)) for _ in range(B)]
        n_pages[int(rng.integers(0, B))] = P
        G = int(rng.choice([1, 2, 4, 8]))
        Tq = int(rng.choice([1, 2])) if G < 8 else 1          # the library takes at most 8 query rows per KV head
        yield B, P, k, forced, n_pages, G, Tq, 1000 * seed + i


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_selection_on_random_shapes(dd, seed):
    for B, P, k, forced, n_pages, G, Tq, s in _select_shapes(6, seed):
        _, _, fused, _ = _select_case(dd, B, P, k, forced, n_pages, seed=s, G=G, Tq=Tq, select_mode=0)
        _, _, two, _ = _select_case(dd, B, P, k, forced, n_pages, seed=s, G=G, Tq=Tq, select_mode=1)
        assert np.array_equal(fused, two), (B, P, k, forced, n_pages, G, Tq)
        for b in range(B):                       # ascending, in range, distinct
            assert np.all(np.diff(fused[b], axis=-1) > 0) and fused[b].min() >= 0 and fused[b].max() < n_pages[b]


def _attn_shapes(n, seed):
    rng = np.random.default_rng(seed)
    for i in range(n):
        B = int(rng.integers(1, 5))
        P = int(rng.integers(8, 400))
        k = int(rng.choice([1, rng.integers(1, P + 1), min(P, 128)]))
        ctx_len = []
        for b in range(B):
            pages = int(rng.integers(k, P + 1))
            ctx_len.append(pages * 16 - int(rng.integers(0, 16)))
        G = int(rng.choice([1, 2, 4, 8]))
        Tq = int(rng.choice([1, 2])) if G < 8 else 1
        splits = int(rng.choice([0, 0, 1, rng.integers(1, min(k, 16) + 1)]))
        yield B, P, k, ctx_len, Tq, splits, 1000 * seed + i, G


@pytest.mark.parametrize("seed", [1, 2, 3])
@pytest.mark.parametrize("mode", ["split", "stream", "tc"])
def test_attention_on_random_shapes(dd, seed, mode):
    attn_mode = {"stream": dd.DD_ATTN_STREAM, "split": dd.DD_ATTN_SPLIT, "tc": dd.DD_ATTN_TC}[mode]
    for B, P, k, ctx_len, Tq, splits, s, G in _attn_shapes(6, seed):
        _attn_case(dd, B, P, k, ctx_len, Tq, splits, seed=s, G=G, attn_mode=attn_mode)
