"""Plain CPU oracle of the per-layer sparse decode hot path (DualDecoder).

TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and the CPU legs
of the benchmark; never by the product package, and it never calls the CUDA
library. Slow on purpose: every function is the definition written out in
numpy, in fp64 unless a storage rounding is part of the definition.

The paper defines the path in prose only (no equation, no listing):

* retrieval index = f(token query, static GPU-resident chunk landmarks)
  (Sec. 2.2 "Dynamic Sparse KV Cache", Sec. 4.1 "KV Retrieval Predictability");
* the index used for step i+1 is predicted from the speculated token of step i
  (Sec. 4.1 "Retrieval index prediction");
* selected KV blocks are moved from host memory into a layer-scoped GPU buffer
  in attention layout (Sec. 5.3, Sec. 5.4 "GPU-side sparse KV assembly");
* attention runs over exactly that sparse set (Sec. 4.2, Sec. 5.4).

Readings taken where the paper is silent (each is listed in the design notes):
landmark = per-page mean key, stored in bf16; score = scaled dot product,
softmax over the request's valid pages per query head, then maximum over the
query heads that share a KV head; ties go to the lower page; the selected set
is emitted in ascending page order; the last `forced_recent` valid pages are
always selected and count inside the budget.

Parity with numbers printed in the paper: UNPINNED for every function (the
paper prints no worked example). Correctness is pinned by closed forms, brute
force, invariants and library special cases in tests/test_oracle_*.py.

Array conventions (numpy):
  q        [B, Tq, Hq, d]   queries, token 0 = current, token 1 = speculated
  lm       [B, Hkv, P, d]   landmarks (bf16-representable values)
  kv       [B, Hkv, P, 2, T, d]  one layer of the host store, [..,0,..]=K, [..,1,..]=V
  idx      [B, Hkv, k]      selected pages, ascending
  slot     [B, Hkv, 2, k*T, d]   gathered buffer in attention layout
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "round_to_bf16",
    "build_landmarks",
    "page_scores",
    "topk_pages",
    "select_topk",
    "gather_kv",
    "sparse_decode_attn",
    "sparse_decode_attn_causal",
    "decode_chain",
    "correct_misses",
    "decode_chain_corrected",
]


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); returns fp32.

    bf16 is the upper 16 bits of an IEEE fp32, so rounding adds half of the
    dropped field (plus the parity of the kept LSB) and truncates.
    NaN is not expected on this path.
    """
    a = np.ascontiguousarray(x, dtype=np.float32)
    bits = a.view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    bits = (bits + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return bits.astype(np.uint32).view(np.float32).reshape(a.shape)


def build_landmarks(k_pages: np.ndarray, ctx_len: np.ndarray, chunk_tokens: int | None = None) -> np.ndarray:
    """Landmark of a chunk = mean of its valid keys (Sec. 2.2: chunks of adjacent
    KV entries with compressed landmarks; Sec. 4.1: built before decoding, fixed).

    k_pages [B, Hkv, P, T, d] bf16-valued; ctx_len [B] tokens. A chunk is
    `chunk_tokens` consecutive tokens of a page (default: the whole page, T);
    the result is [B, Hkv, P * T / chunk_tokens, d], chunks of a page adjacent.
    A chunk with no valid token gets a zero landmark (it is never scored). The
    storage format is part of the definition: sum in fp32 in token order, divide
    in fp32, round to bf16, so that the same bits can be produced by any
    implementation.
    """
    k_pages = np.asarray(k_pages, dtype=np.float32)
    B, Hkv, P, T, d = k_pages.shape
    c = T if chunk_tokens is None else int(chunk_tokens)
    assert T % c == 0
    toks = k_pages.reshape(B, Hkv, P * T, d)
    n_chunks = P * T // c
    out = np.zeros((B, Hkv, n_chunks, d), dtype=np.float32)
    for b in range(B):
        n_tok = int(ctx_len[b])
        for ch in range(n_chunks):
            cnt = min(c, n_tok - ch * c)
            if cnt <= 0:
                continue
            acc = np.zeros((Hkv, d), dtype=np.float32)
            for i in range(cnt):
                acc = acc + toks[b, :, ch * c + i, :]
            out[b, :, ch, :] = acc / np.float32(cnt)
    return round_to_bf16(out)


def page_scores(q_tok: np.ndarray, lm: np.ndarray, n_pages: int, group_reduce: str = "softmax_max",
                chunks_per_page: int = 1, n_chunks: int | None = None):
    """Scores of one request's pages for every KV head (Sec. 4.1).

    q_tok [Hq, d] (the scoring token's per-head queries), lm [Hkv, P, d].
    Returns (score [Hkv, n_pages] in (0, 1], logit s [Hq, n_pages], lse [Hq]).

      s[h, p]  = <q[h], lm[g(h), p]> / sqrt(d),  g(h) = h // (Hq / Hkv)
      lse[h]   = log sum_p exp(s[h, p])          over the valid pages
      score[g, p] = max_{h in group g} exp(s[h, p] - lse[h])

    `group_reduce` other than "softmax_max" exists only to show sensitivity to
    the reading ("logit_max", "logit_mean"); the contract is "softmax_max".

    With finer landmarks (chunks_per_page = R > 1, lm [Hkv, P * R, d], the first
    n_chunks chunks of the request exist) the soft-max runs over the existing
    chunks and a page takes the maximum over its chunks as well:
      score[g, p] = max_{h in group g, r < R} exp(s[h, p * R + r] - lse[h]);
    s and lse are then returned per chunk.
    """
    if chunks_per_page != 1:
        R = int(chunks_per_page)
        nc = int(n_chunks)
        assert (n_pages - 1) * R < nc <= n_pages * R
        chunk_score, s, lse = page_scores(q_tok, lm, nc, "softmax_max")
        padded = np.zeros((chunk_score.shape[0], n_pages * R), dtype=np.float64)
        padded[:, :nc] = chunk_score
        return padded.reshape(-1, n_pages, R).max(axis=2), s, lse
    q_tok = np.asarray(q_tok, dtype=np.float64)
    lm = np.asarray(lm, dtype=np.float64)
    Hq, d = q_tok.shape
    Hkv = lm.shape[0]
    assert Hq % Hkv == 0
    G = Hq // Hkv
    s = np.empty((Hq, n_pages), dtype=np.float64)
    for h in range(Hq):
        s[h] = lm[h // G, :n_pages, :] @ q_tok[h] / np.sqrt(float(d))
    m = s.max(axis=1, keepdims=True)
    lse = (m + np.log(np.exp(s - m).sum(axis=1, keepdims=True)))[:, 0]
    if group_reduce == "softmax_max":
        per_head = np.exp(s - lse[:, None])
        score = per_head.reshape(Hkv, G, n_pages).max(axis=1)
    elif group_reduce == "logit_max":
        score = s.reshape(Hkv, G, n_pages).max(axis=1)
    elif group_reduce == "logit_mean":
        score = s.reshape(Hkv, G, n_pages).mean(axis=1)
    else:
        raise ValueError(group_reduce)
    return score, s, lse


def topk_pages(score: np.ndarray, k: int, forced_recent: int = 0) -> np.ndarray:
    """The k pages of largest score, by full sort; ties go to the lower page; the
    last `forced_recent` pages are always in the set and count inside k. Output
    ascending. score [n_pages]."""
    n = score.shape[0]
    if not (0 < k <= n) or not (0 <= forced_recent <= k):
        raise ValueError("need 0 < k <= n_pages and 0 <= forced_recent <= k")
    key = np.array(score, dtype=np.float64, copy=True)
    if forced_recent:
        key[n - forced_recent:] = np.inf
    # stable sort of the negated key: equal keys stay in ascending page order
    order = np.argsort(-key, kind="stable")
    return np.sort(order[:k]).astype(np.int32)


def select_topk(q_tok: np.ndarray, lm: np.ndarray, n_pages: np.ndarray, k: int,
                forced_recent: int = 0, group_reduce: str = "softmax_max", chunks_per_page: int = 1,
                n_chunks: np.ndarray | None = None):
    """Per-KV-head critical set of every request (Sec. 2.2, Sec. 4.1).

    q_tok [B, Hq, d], lm [B, Hkv, P * chunks_per_page, d], n_pages [B] (and n_chunks [B], the existing
    chunks of every request, when chunks_per_page > 1).
    Returns (idx [B, Hkv, k] int32 ascending, scores: list of [Hkv, n_pages[b]])."""
    B = q_tok.shape[0]
    Hkv = lm.shape[1]
    idx = np.empty((B, Hkv, k), dtype=np.int32)
    scores = []
    for b in range(B):
        sc, _, _ = page_scores(q_tok[b], lm[b], int(n_pages[b]), group_reduce, chunks_per_page,
                               None if n_chunks is None else int(n_chunks[b]))
        scores.append(sc)
        for g in range(Hkv):
            idx[b, g] = topk_pages(sc[g], k, forced_recent)
    return idx, scores


def gather_kv(kv_layer: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """Copy the selected pages into attention layout (Sec. 5.4 assembly; the bits
    are unchanged). kv_layer [B, Hkv, P, 2, T, d] (any dtype), idx [B, Hkv, k]
    → slot [B, Hkv, 2, k*T, d]."""
    B, Hkv, P, two, T, d = kv_layer.shape
    k = idx.shape[2]
    slot = np.empty((B, Hkv, 2, k * T, d), dtype=kv_layer.dtype)
    for b in range(B):
        for g in range(Hkv):
            for j in range(k):
                p = int(idx[b, g, j])
                slot[b, g, 0, j * T:(j + 1) * T, :] = kv_layer[b, g, p, 0]
                slot[b, g, 1, j * T:(j + 1) * T, :] = kv_layer[b, g, p, 1]
    return slot


def sparse_decode_attn(q: np.ndarray, slot: np.ndarray, idx: np.ndarray, ctx_len: np.ndarray,
                       page_tokens: int, return_weights: bool = False):
    """Scaled-dot-product GQA attention of every query token over the gathered
    set only (Sec. 4.2, Sec. 5.4: attention observes the layer's sparse KV set).

    q [B, Tq, Hq, d]; slot [B, Hkv, 2, k*T, d]; idx [B, Hkv, k]; ctx_len [B].
    Gathered token (j, i) sits at context position idx[j]*T + i and is masked
    out when that position is >= ctx_len[b]. Both query tokens see the same set.
    Returns (out [B, Tq, Hq, d] fp64, lse [B, Tq, Hq] fp64[, weights])."""
    q = np.asarray(q, dtype=np.float64)
    slot = np.asarray(slot, dtype=np.float64)
    B, Tq, Hq, d = q.shape
    Hkv = slot.shape[1]
    G = Hq // Hkv
    n_tok = slot.shape[3]
    T = page_tokens
    out = np.zeros((B, Tq, Hq, d), dtype=np.float64)
    lse = np.zeros((B, Tq, Hq), dtype=np.float64)
    weights = np.zeros((B, Tq, Hq, n_tok), dtype=np.float64) if return_weights else None
    for b in range(B):
        for g in range(Hkv):
            pos = (idx[b, g].astype(np.int64)[:, None] * T + np.arange(T)[None, :]).reshape(-1)
            valid = pos < int(ctx_len[b])
            keys = slot[b, g, 0]
            vals = slot[b, g, 1]
            for t in range(Tq):
                for h in range(g * G, (g + 1) * G):
                    z = keys @ q[b, t, h] / np.sqrt(float(d))
                    z = np.where(valid, z, -np.inf)
                    m = z.max()
                    e = np.exp(z - m)
                    den = e.sum()
                    w = e / den
                    out[b, t, h] = w @ vals
                    lse[b, t, h] = m + np.log(den)
                    if return_weights:
                        weights[b, t, h] = w
    if return_weights:
        return out, lse, weights
    return out, lse


def sparse_decode_attn_causal(q: np.ndarray, slot: np.ndarray, idx: np.ndarray, ctx_len: np.ndarray,
                              page_tokens: int, k_new: np.ndarray, v_new: np.ndarray):
    """Attention of the step's tokens over the gathered set plus the step's own new KV entries, with the
    dual-token mask (Sec. 5.2 "Dual-token decoding": output token and speculated token of a request are
    concatenated along the sequence, and the output token must not see the speculated token).

    Query token t (0 = output token, 1 = speculated token) sees every valid gathered token and the new
    entries j <= t, i.e. itself and the tokens before it. k_new, v_new [B, Tq, Hkv, d] are the keys and
    values of the step's tokens (context positions ctx_len[b] + j). Returns (out [B, Tq, Hq, d], lse)."""
    q = np.asarray(q, dtype=np.float64)
    slot = np.asarray(slot, dtype=np.float64)
    k_new = np.asarray(k_new, dtype=np.float64)
    v_new = np.asarray(v_new, dtype=np.float64)
    B, Tq, Hq, d = q.shape
    Hkv = slot.shape[1]
    G = Hq // Hkv
    T = page_tokens
    out = np.zeros((B, Tq, Hq, d), dtype=np.float64)
    lse = np.zeros((B, Tq, Hq), dtype=np.float64)
    for b in range(B):
        for g in range(Hkv):
            pos = (idx[b, g].astype(np.int64)[:, None] * T + np.arange(T)[None, :]).reshape(-1)
            valid = pos < int(ctx_len[b])
            for t in range(Tq):
                keys = np.concatenate([slot[b, g, 0][valid], k_new[b, :t + 1, g]], axis=0)
                vals = np.concatenate([slot[b, g, 1][valid], v_new[b, :t + 1, g]], axis=0)
                for h in range(g * G, (g + 1) * G):
                    z = keys @ q[b, t, h] / np.sqrt(float(d))
                    m = z.max()
                    e = np.exp(z - m)
                    den = e.sum()
                    out[b, t, h] = (e / den) @ vals
                    lse[b, t, h] = m + np.log(den)
    return out, lse


def decode_chain(q_init: np.ndarray, q_steps: np.ndarray, lm_layers, kv_layers, n_pages: np.ndarray,
                 ctx_len: np.ndarray, k: int, page_tokens: int, forced_recent: int = 0):
    """Several decode steps of every layer (Sec. 4.1, Sec. 5.2, Sec. 5.3):

      idx[0][l]   = select(q_init[l])                      (stand-in for the pre-decode step)
      out[t][l]   = attn(q_steps[t][l], gather(idx[t][l]))  (both tokens)
      idx[t+1][l] = select(speculated token of q_steps[t][l])

    q_init [L, B, Hq, d]; q_steps [S, L, B, 2, Hq, d]; lm_layers[l] [B, Hkv, P, d];
    kv_layers[l] [B, Hkv, P, 2, T, d]. Returns (outs [S, L, B, 2, Hq, d], idxs [S+1, L, B, Hkv, k])."""
    S, L = q_steps.shape[0], q_steps.shape[1]
    B = q_steps.shape[2]
    Hkv = lm_layers[0].shape[1]
    idxs = np.empty((S + 1, L, B, Hkv, k), dtype=np.int32)
    outs = np.empty(q_steps.shape, dtype=np.float64)
    for l in range(L):
        idxs[0, l], _ = select_topk(q_init[l], lm_layers[l], n_pages, k, forced_recent)
    for t in range(S):
        for l in range(L):
            slot = gather_kv(kv_layers[l], idxs[t, l])
            outs[t, l], _ = sparse_decode_attn(q_steps[t, l], slot, idxs[t, l], ctx_len, page_tokens)
            idxs[t + 1, l], _ = select_topk(q_steps[t, l][:, 1], lm_layers[l], n_pages, k, forced_recent)
    return outs, idxs


def correct_misses(pred_idx: np.ndarray, true_idx: np.ndarray):
    """Repair of a predicted set once the true index is known (Sec. 5.3 "Prioritized missing KV transfer":
    the pages the prediction missed are fetched before attention so that the result is the one computed
    with the true retrieval index; Sec. 5.4: the assembly step merges them into the layer's buffer).

    pred_idx, true_idx [B, Hkv, k] ascending. The pages of the true set the prediction lacks
    (missing = true minus predicted, ascending) take the buffer positions of the pages the true set does not
    want (victims = predicted minus true, in ascending position). Returns
      merged  [B, Hkv, k]  page held by every buffer position after the repair (as a set = the true set),
      fixes   list over (b, g) of (positions, pages) arrays,
      n_miss  [B, Hkv]."""
    B, Hkv, k = pred_idx.shape
    merged = np.array(pred_idx, dtype=np.int32, copy=True)
    fixes = []
    n_miss = np.zeros((B, Hkv), dtype=np.int32)
    for b in range(B):
        for g in range(Hkv):
            pred = [int(x) for x in pred_idx[b, g]]
            true = [int(x) for x in true_idx[b, g]]
            pred_set, true_set = set(pred), set(true)
            missing = [p for p in true if p not in pred_set]
            victims = [j for j, p in enumerate(pred) if p not in true_set]
            assert len(missing) == len(victims)
            for j, p in zip(victims, missing):
                merged[b, g, j] = p
            fixes.append((np.array(victims, dtype=np.int32), np.array(missing, dtype=np.int32)))
            n_miss[b, g] = len(missing)
    return merged, fixes, n_miss


def decode_chain_corrected(q_init: np.ndarray, q_steps: np.ndarray, lm_layers, kv_layers, n_pages: np.ndarray,
                           ctx_len: np.ndarray, k: int, page_tokens: int, forced_recent: int = 0):
    """The chain with miss correction: the set prefetched for step t is predicted from the speculated token
    of step t-1 (or q_init), the true set comes from the current token of step t, and attention runs over
    the repaired buffer, i.e. over the true set (Sec. 4.2: prediction does not change the attention result).
    Returns (outs [S, L, B, 2, Hq, d], pred [S+1, L, B, Hkv, k], true [S, L, B, Hkv, k], n_miss [S, L, B, Hkv])."""
    S, L, B = q_steps.shape[0], q_steps.shape[1], q_steps.shape[2]
    Hkv = lm_layers[0].shape[1]
    pred = np.empty((S + 1, L, B, Hkv, k), dtype=np.int32)
    true = np.empty((S, L, B, Hkv, k), dtype=np.int32)
    n_miss = np.empty((S, L, B, Hkv), dtype=np.int32)
    outs = np.empty(q_steps.shape, dtype=np.float64)
    for l in range(L):
        pred[0, l], _ = select_topk(q_init[l], lm_layers[l], n_pages, k, forced_recent)
    for t in range(S):
        for l in range(L):
            true[t, l], _ = select_topk(q_steps[t, l][:, 0], lm_layers[l], n_pages, k, forced_recent)
            merged, _, n_miss[t, l] = correct_misses(pred[t, l], true[t, l])
            slot = gather_kv(kv_layers[l], merged)
            outs[t, l], _ = sparse_decode_attn(q_steps[t, l], slot, merged, ctx_len, page_tokens)
            pred[t + 1, l], _ = select_topk(q_steps[t, l][:, 1], lm_layers[l], n_pages, k, forced_recent)
    return outs, pred, true, n_miss
