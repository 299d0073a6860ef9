"""Helpers shared by the GPU parity tests: conversions and the selection comparator."""
import numpy as np
import torch

TAU = 1e-3            # relative band around the k-th score inside which either choice is correct
ATTN_MAX_ABS = 2e-2   # bf16 output, fp32 accumulation
ATTN_MEAN_ABS = 2e-3


def f32(t: torch.Tensor) -> np.ndarray:
    """Exact fp32 numpy copy of a (bf16) tensor."""
    return t.detach().float().cpu().numpy()


def raw16(t: torch.Tensor) -> np.ndarray:
    """The bits of a bf16 tensor as uint16 (for bitwise comparisons)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def check_selection(got: np.ndarray, score: np.ndarray, k: int, forced: int, tau: float = TAU):
    """Band rule for one (request, KV head): `got` [k] from the GPU, `score` [n_pages] from the oracle.
    Returns True when the set equals the oracle's exact set."""
    n = score.shape[0]
    assert got.shape == (k,)
    assert np.all(np.diff(got) > 0), "indices must be strictly ascending"
    assert got[0] >= 0 and got[-1] < n, "index outside the request's pages"
    sel = np.zeros(n, dtype=bool)
    sel[got] = True
    assert sel[n - forced:].all(), "a forced recent page is missing"
    k_free, n_free = k - forced, n - forced
    exact = True
    if k_free > 0:
        free = score[:n_free]
        order = np.argsort(-free, kind="stable")
        hi = free[order[k_free - 1]]
        must = free > hi * (1 + tau)
        must_not = free < hi * (1 - tau)
        assert sel[:n_free][must].all(), "a page clearly above the k-th score was not selected"
        assert not sel[:n_free][must_not].any(), "a page clearly below the k-th score was selected"
        want = np.zeros(n_free, dtype=bool)
        want[order[:k_free]] = True
        exact = bool(np.array_equal(want, sel[:n_free]))
    else:
        assert not sel[:n_free].any()
    return exact


def check_attention(got_bf16: torch.Tensor, want: np.ndarray):
    err = np.abs(f32(got_bf16).astype(np.float64) - want)
    assert err.max() <= ATTN_MAX_ABS, f"max abs error {err.max():.4g}"
    assert err.mean() <= ATTN_MEAN_ABS, f"mean abs error {err.mean():.4g}"
    return err.max(), err.mean()
