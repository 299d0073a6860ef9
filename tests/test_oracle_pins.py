"""Pins of the CPU oracle against things other than itself: closed forms worked
by hand, brute force written as Python loops, library special cases (torch SDPA,
struct-level bf16 rounding) and invariants. The paper prints no worked example,
so none of these is a value quoted from it."""
import math
import struct

import numpy as np
import pytest
import torch

from oracle import dd_oracle as orc


# ----------------------------------------------------------------------------- bf16 rounding
def _bf16_bits_via_struct(x: float) -> int:
    """Round-to-nearest-even on the raw bits, one value at a time (independent of numpy)."""
    (u,) = struct.unpack("<I", struct.pack("<f", x))
    upper, lower = u >> 16, u & 0xFFFF
    if lower > 0x8000 or (lower == 0x8000 and (upper & 1)):
        upper += 1
    return upper & 0xFFFF


def test_round_to_bf16_matches_bitwise_rne_and_torch():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(2000).astype(np.float32) * 3,
                        np.array([1.0, 1.00390625, 1.01171875, -1.00390625, 0.0, 65504.0, 1e-30], np.float32)])
    got = orc.round_to_bf16(x)
    for xi, gi in zip(x, got):
        want_bits = _bf16_bits_via_struct(float(xi))
        (gb,) = struct.unpack("<I", struct.pack("<f", float(gi)))
        assert gb == want_bits << 16
    want = torch.from_numpy(x).to(torch.bfloat16).float().numpy()
    assert np.array_equal(got, want)
    # ties: 1 + 2^-8 is halfway between 1 and 1 + 2^-7 -> even (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    assert got[-6] == 1.0 and got[-5] == np.float32(1.015625)


# ----------------------------------------------------------------------------- landmarks
def test_landmark_of_identical_keys_is_that_key_and_partial_page():
    B, Hkv, P, T, d = 1, 2, 3, 4, 8
    rng = np.random.default_rng(2)
    key = orc.round_to_bf16(rng.standard_normal((Hkv, d)).astype(np.float32))
    k = np.zeros((B, Hkv, P, T, d), np.float32)
    k[0, :, 0] = key[:, None, :]                  # page 0: four copies of one key
    k[0, :, 1, 0] = 2.0                           # page 1: 2, 4, then garbage beyond ctx
    k[0, :, 1, 1] = 4.0
    k[0, :, 1, 2:] = 1000.0
    k[0, :, 2] = 77.0                             # page 2 entirely beyond ctx
    lm = orc.build_landmarks(k, np.array([6]))
    assert np.array_equal(lm[0, :, 0], key)
    assert np.all(lm[0, :, 1] == 3.0)             # mean of the two valid tokens only
    assert np.all(lm[0, :, 2] == 0.0)


def test_landmark_close_to_fp64_mean_within_one_bf16_ulp():
    rng = np.random.default_rng(3)
    k = orc.round_to_bf16(rng.standard_normal((2, 2, 5, 16, 32)).astype(np.float32))
    lm = orc.build_landmarks(k, np.array([80, 80]))
    ref = k.astype(np.float64).mean(axis=3)
    ulp = np.maximum(np.abs(ref), 2.0 ** -126) * 2.0 ** -8
    assert np.all(np.abs(lm - ref) <= ulp)


# ----------------------------------------------------------------------------- scoring
def test_score_closed_form_two_heads_two_pages():
    """d = 4 (sqrt d = 2), one KV head shared by two query heads, two pages.
    Head A sees logits (ln 3, 0) -> probabilities (3/4, 1/4); head B sees (0, ln 4)
    -> (1/5, 4/5). Group maximum: page 0 -> 3/4, page 1 -> 4/5. Dropping 1/sqrt(d),
    the softmax, or using a mean over the group would each give other numbers."""
    a, b = math.log(3.0), math.log(4.0)
    lm = np.zeros((1, 2, 4))
    lm[0, 0] = [1, 0, 0, 0]
    lm[0, 1] = [0, 1, 0, 0]
    q = np.zeros((2, 4))
    q[0] = [2 * a, 0, 0, 0]
    q[1] = [0, 2 * b, 0, 0]
    score, s, lse = orc.page_scores(q, lm, 2)
    assert score.shape == (1, 2)
    np.testing.assert_allclose(score[0], [0.75, 0.8], rtol=1e-14)
    np.testing.assert_allclose(s, [[a, 0.0], [0.0, b]], atol=1e-15)
    np.testing.assert_allclose(lse, [math.log(4.0), math.log(5.0)], rtol=1e-14)


def test_score_head_to_kv_head_mapping_is_block_wise():
    """Query head h reads KV head h // G: a signal on head 5 (G = 4) must raise a
    page of KV head 1, not of KV head 5 % 2 or any other."""
    Hq, Hkv, P, d = 8, 2, 6, 16
    rng = np.random.default_rng(4)
    lm = rng.standard_normal((Hkv, P, d)) * 0.01
    q = rng.standard_normal((Hq, d)) * 0.01
    lm[1, 4] = 0.0
    lm[1, 4, 3] = 5.0
    q[5, 3] = 8.0
    score, _, _ = orc.page_scores(q, lm, P)
    assert int(np.argmax(score[1])) == 4
    assert score[1, 4] > 0.99
    assert score[0].max() < 0.5


def test_softmax_probabilities_sum_to_one_and_ignore_pages_beyond_n_pages():
    rng = np.random.default_rng(5)
    Hq, Hkv, P, d = 8, 2, 40, 32
    q = rng.standard_normal((Hq, d))
    lm = rng.standard_normal((Hkv, P, d))
    n = 33
    score, s, lse = orc.page_scores(q, lm, n)
    np.testing.assert_allclose(np.exp(s - lse[:, None]).sum(axis=1), 1.0, rtol=1e-12)
    lm2 = lm.copy()
    lm2[:, n:] = 1e3                               # pages that do not exist must not matter
    score2, _, _ = orc.page_scores(q, lm2, n)
    assert np.array_equal(score, score2)
    assert score.shape == (Hkv, n) and np.all(score > 0) and np.all(score <= 1)


def test_single_head_group_reduces_to_topk_of_raw_dot_products():
    """With G = 1 the softmax is monotone, so the set is the top-k of <q, landmark>."""
    rng = np.random.default_rng(6)
    H, P, d, k = 3, 50, 16, 7
    q = rng.standard_normal((1, H, d))
    lm = rng.standard_normal((1, H, P, d))
    idx, _ = orc.select_topk(q, lm, np.array([P]), k)
    for h in range(H):
        dots = [sum(q[0, h, c] * lm[0, h, p, c] for c in range(d)) for p in range(P)]
        want = sorted(sorted(range(P), key=lambda p: -dots[p])[:k])
        assert idx[0, h].tolist() == want
    # positive scaling of the query keeps each head's order
    idx2, _ = orc.select_topk(q * 3.7, lm, np.array([P]), k)
    assert np.array_equal(idx, idx2)


def test_one_token_pages_select_the_top_attention_logits():
    """Page = 1 token makes the landmark the key itself, so selection must be the
    brute-force token-level top-k of the attention logits."""
    rng = np.random.default_rng(7)
    ctx, d, k = 37, 8, 5
    keys = orc.round_to_bf16(rng.standard_normal((1, 1, ctx, 1, d)).astype(np.float32))
    lm = orc.build_landmarks(keys, np.array([ctx]))
    assert np.array_equal(lm[0, 0], keys[0, 0, :, 0])
    q = rng.standard_normal((1, 1, d))
    idx, _ = orc.select_topk(q, lm, np.array([ctx]), k)
    logits = (keys[0, 0, :, 0].astype(np.float64) @ q[0, 0]) / math.sqrt(d)
    want = sorted(np.argsort(-logits)[:k].tolist())
    assert idx[0, 0].tolist() == want


# ----------------------------------------------------------------------------- top-k
def _brute_topk(score, k, forced):
    n = len(score)
    chosen = list(range(n - forced, n))
    rest = [p for p in range(n - forced)]
    while len(chosen) < k:
        best = None
        for p in rest:                              # first maximum = lowest page among equals
            if best is None or score[p] > score[best]:
                best = p
        chosen.append(best)
        rest.remove(best)
    return sorted(chosen)


@pytest.mark.parametrize("n,k,forced", [(1, 1, 0), (9, 3, 0), (9, 9, 0), (17, 5, 2), (17, 5, 5), (40, 13, 3)])
def test_topk_equals_brute_force_selection(n, k, forced):
    rng = np.random.default_rng(100 + n + k)
    for trial in range(20):
        score = rng.random(n)
        if trial % 3 == 0:                          # heavy ties
            score = np.round(score * 4) / 4
        got = orc.topk_pages(score, k, forced)
        assert got.tolist() == _brute_topk(score.tolist(), k, forced)
        assert got.dtype == np.int32
        assert np.all(np.diff(got) > 0) and got.min() >= 0 and got.max() < n


def test_topk_ties_go_to_lower_page_and_full_budget_returns_everything():
    assert orc.topk_pages(np.array([0.5, 0.5, 0.5, 0.5]), 2).tolist() == [0, 1]
    assert orc.topk_pages(np.array([0.1, 0.9, 0.9, 0.1]), 3).tolist() == [0, 1, 2]
    assert orc.topk_pages(np.array([0.3, 0.2, 0.1]), 3).tolist() == [0, 1, 2]
    # the forced recent pages displace better-scored ones
    assert orc.topk_pages(np.array([0.9, 0.8, 0.7, 0.0, 0.0]), 3, forced_recent=2).tolist() == [0, 3, 4]
    with pytest.raises(ValueError):
        orc.topk_pages(np.array([0.3, 0.2]), 3)
    with pytest.raises(ValueError):
        orc.topk_pages(np.array([0.3, 0.2]), 1, forced_recent=2)


# ----------------------------------------------------------------------------- gather
def test_gather_bitwise_against_python_loops_and_identity():
    rng = np.random.default_rng(8)
    B, Hkv, P, T, d, k = 2, 3, 7, 4, 8, 3
    kv = rng.integers(0, 2 ** 16, size=(B, Hkv, P, 2, T, d), dtype=np.uint16)
    idx = np.stack([np.stack([np.sort(rng.choice(P, k, replace=False)) for _ in range(Hkv)]) for _ in range(B)])
    slot = orc.gather_kv(kv, idx.astype(np.int32))
    assert slot.shape == (B, Hkv, 2, k * T, d) and slot.dtype == np.uint16
    for b in range(B):
        for g in range(Hkv):
            for j in range(k):
                for i in range(T):
                    for c in range(d):
                        assert slot[b, g, 0, j * T + i, c] == kv[b, g, idx[b, g, j], 0, i, c]
                        assert slot[b, g, 1, j * T + i, c] == kv[b, g, idx[b, g, j], 1, i, c]
    ident = np.tile(np.arange(P, dtype=np.int32), (B, Hkv, 1))
    full = orc.gather_kv(kv, ident)
    assert np.array_equal(full[:, :, 0], kv[:, :, :, 0].reshape(B, Hkv, P * T, d))
    assert np.array_equal(full[:, :, 1], kv[:, :, :, 1].reshape(B, Hkv, P * T, d))


# ----------------------------------------------------------------------------- attention
def _setup_attn(seed, B=2, Tq=2, Hq=8, Hkv=2, P=6, T=4, d=16):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((B, Tq, Hq, d))
    kv = rng.standard_normal((B, Hkv, P, 2, T, d))
    return rng, q, kv


def test_full_budget_equals_dense_attention_from_torch_sdpa():
    """Budget = whole context: the sparse path must equal dense GQA attention, here
    computed by torch's scaled_dot_product_attention in fp64 (a library routine,
    with the KV heads expanded to the query heads by hand)."""
    B, Tq, Hq, Hkv, P, T, d = 2, 2, 8, 2, 6, 4, 16
    _, q, kv = _setup_attn(9, B, Tq, Hq, Hkv, P, T, d)
    ident = np.tile(np.arange(P, dtype=np.int32), (B, Hkv, 1))
    ctx = np.array([P * T, P * T - 3])              # second request: ragged last page
    slot = orc.gather_kv(kv, ident)
    out, lse, w = orc.sparse_decode_attn(q, slot, ident, ctx, T, return_weights=True)
    np.testing.assert_allclose(w.sum(axis=-1), 1.0, rtol=1e-12)
    G = Hq // Hkv
    for b in range(B):
        n = int(ctx[b])
        K = torch.from_numpy(kv[b, :, :, 0].reshape(Hkv, P * T, d)[:, :n]).repeat_interleave(G, dim=0)
        V = torch.from_numpy(kv[b, :, :, 1].reshape(Hkv, P * T, d)[:, :n]).repeat_interleave(G, dim=0)
        Q = torch.from_numpy(q[b]).permute(1, 0, 2)                    # [Hq, Tq, d]
        ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V)  # no mask: both tokens see all
        np.testing.assert_allclose(out[b], ref.permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)
        ref_lse = torch.logsumexp(Q @ K.transpose(1, 2) / math.sqrt(d), dim=-1).permute(1, 0).numpy()
        np.testing.assert_allclose(lse[b], ref_lse, rtol=1e-12)
        assert np.all(w[b][..., n:] == 0.0)


def test_attention_over_a_subset_equals_dense_attention_restricted_to_it():
    """Brute force in Python loops on a strict subset of pages, checking the GQA head map too."""
    B, Tq, Hq, Hkv, P, T, d = 1, 2, 4, 2, 5, 2, 4
    _, q, kv = _setup_attn(10, B, Tq, Hq, Hkv, P, T, d)
    idx = np.array([[[1, 4], [0, 2]]], dtype=np.int32)
    slot = orc.gather_kv(kv, idx)
    out, _ = orc.sparse_decode_attn(q, slot, idx, np.array([P * T]), T)
    for t in range(Tq):
        for h in range(Hq):
            g = h // (Hq // Hkv)
            toks = [(p, i) for p in idx[0, g] for i in range(T)]
            z = [sum(q[0, t, h, c] * kv[0, g, p, 0, i, c] for c in range(d)) / math.sqrt(d) for p, i in toks]
            zmax = max(z)
            e = [math.exp(v - zmax) for v in z]
            den = sum(e)
            want = [sum(e[n] / den * kv[0, g, p, 1, i, c] for n, (p, i) in enumerate(toks)) for c in range(d)]
            np.testing.assert_allclose(out[0, t, h], want, rtol=1e-12, atol=1e-14)


def test_attention_invariants():
    B, Tq, Hq, Hkv, P, T, d = 1, 2, 8, 2, 8, 4, 16
    rng, q, kv = _setup_attn(11, B, Tq, Hq, Hkv, P, T, d)
    ctx = np.array([P * T])
    idx = np.array([[[0, 2, 5, 7], [1, 2, 3, 6]]], dtype=np.int32)
    out, _ = orc.sparse_decode_attn(q, orc.gather_kv(kv, idx), idx, ctx, T)
    # order of the set does not matter
    perm = idx[:, :, ::-1].copy()
    out_p, _ = orc.sparse_decode_attn(q, orc.gather_kv(kv, perm), perm, ctx, T)
    np.testing.assert_allclose(out, out_p, rtol=1e-12, atol=1e-14)
    # equal keys -> plain mean of the values
    kv_eq = kv.copy()
    kv_eq[:, :, :, 0] = kv[:, :, :1, 0, :1]
    out_eq, _ = orc.sparse_decode_attn(q, orc.gather_kv(kv_eq, idx), idx, ctx, T)
    mean_v = orc.gather_kv(kv_eq, idx)[:, :, 1].mean(axis=2)             # [B, Hkv, d]
    np.testing.assert_allclose(out_eq, np.broadcast_to(np.repeat(mean_v, Hq // Hkv, axis=1)[:, None], out_eq.shape),
                               rtol=1e-12, atol=1e-14)
    # constant values -> that constant
    kv_c = kv.copy()
    kv_c[:, :, :, 1] = 2.5
    out_c, _ = orc.sparse_decode_attn(q, orc.gather_kv(kv_c, idx), idx, ctx, T)
    np.testing.assert_allclose(out_c, 2.5, rtol=1e-13)
    # one dominant key -> its value
    kv_d = kv.copy()
    kv_d[0, 0, 5, 0, 2] = 200.0 * q[0, 0, 1] / np.linalg.norm(q[0, 0, 1])
    out_d, _ = orc.sparse_decode_attn(q, orc.gather_kv(kv_d, idx), idx, ctx, T)
    np.testing.assert_allclose(out_d[0, 0, 1], kv_d[0, 0, 5, 1, 2], rtol=1e-9, atol=1e-9)
    # masking: tokens at or beyond ctx_len are ignored whatever they hold
    kv_m = kv.copy()
    kv_m[0, :, 7, :, 2:] = 1e4
    short = np.array([7 * T + 2])
    o1, _ = orc.sparse_decode_attn(q, orc.gather_kv(kv, idx), idx, short, T)
    o2, _ = orc.sparse_decode_attn(q, orc.gather_kv(kv_m, idx), idx, short, T)
    assert np.array_equal(o1, o2)
    assert not np.allclose(o1, out)


# ----------------------------------------------------------------------------- chain
def test_chain_uses_the_speculated_token_of_the_previous_step():
    rng = np.random.default_rng(12)
    S, L, B, Hq, Hkv, P, T, d, k = 3, 2, 2, 4, 2, 10, 2, 8, 3
    ctx = np.array([P * T, P * T - 1])
    npg = np.array([P, P])
    kv = [orc.round_to_bf16(rng.standard_normal((B, Hkv, P, 2, T, d)).astype(np.float32)) for _ in range(L)]
    lm = [orc.build_landmarks(kv[l][:, :, :, 0], ctx) for l in range(L)]
    q_init = rng.standard_normal((L, B, Hq, d))
    q_steps = rng.standard_normal((S, L, B, 2, Hq, d))
    outs, idxs = orc.decode_chain(q_init, q_steps, lm, kv, npg, ctx, k, T)
    assert outs.shape == q_steps.shape and idxs.shape == (S + 1, L, B, Hkv, k)
    for l in range(L):
        want0, _ = orc.select_topk(q_init[l], lm[l], npg, k)
        assert np.array_equal(idxs[0, l], want0)
        for t in range(S):
            want, _ = orc.select_topk(q_steps[t, l][:, 1], lm[l], npg, k)     # token 1 = speculated
            assert np.array_equal(idxs[t + 1, l], want)
            o, _ = orc.sparse_decode_attn(q_steps[t, l], orc.gather_kv(kv[l], idxs[t, l]), idxs[t, l], ctx, T)
            assert np.array_equal(outs[t, l], o)
    # the current token must not influence the next index
    q2 = q_steps.copy()
    q2[:, :, :, 0] += 5.0
    _, idxs2 = orc.decode_chain(q_init, q2, lm, kv, npg, ctx, k, T)
    assert np.array_equal(idxs, idxs2)


# ----------------------------------------------------------------------------- miss correction
def test_correction_hand_example_and_set_identities():
    """Predicted {1,4,6,9}, true {2,4,9,11}: pages 2 and 11 are missing, the victims are positions 0 and 2
    (pages 1 and 6). After the repair the buffer holds [2, 4, 11, 9]."""
    pred = np.array([[[1, 4, 6, 9]]], dtype=np.int32)
    true = np.array([[[2, 4, 9, 11]]], dtype=np.int32)
    merged, fixes, n_miss = orc.correct_misses(pred, true)
    assert merged.tolist() == [[[2, 4, 11, 9]]]
    assert fixes[0][0].tolist() == [0, 2] and fixes[0][1].tolist() == [2, 11]
    assert n_miss.tolist() == [[1 * 2]]
    rng = np.random.default_rng(20)
    for _ in range(30):
        P, k = 60, 17
        a = np.sort(rng.choice(P, k, replace=False)).astype(np.int32)[None, None]
        b = np.sort(rng.choice(P, k, replace=False)).astype(np.int32)[None, None]
        merged, fixes, n_miss = orc.correct_misses(a, b)
        assert set(merged[0, 0].tolist()) == set(b[0, 0].tolist())            # the buffer holds the true set
        keep = [j for j in range(k) if a[0, 0, j] in set(b[0, 0].tolist())]
        assert all(merged[0, 0, j] == a[0, 0, j] for j in keep)                # common pages do not move
        assert n_miss[0, 0] == len(set(b[0, 0].tolist()) - set(a[0, 0].tolist()))
        assert np.all(np.diff(fixes[0][0]) > 0) and np.all(np.diff(fixes[0][1]) > 0)
    same, fixes, n_miss = orc.correct_misses(pred, pred)
    assert np.array_equal(same, pred) and n_miss.sum() == 0 and fixes[0][0].size == 0


def test_corrected_chain_equals_attention_over_the_true_sets():
    """With correction the prediction must not change the result: every output equals attention over the
    set selected from the current token, whatever was predicted."""
    rng = np.random.default_rng(21)
    S, L, B, Hq, Hkv, P, T, d, k = 2, 2, 2, 4, 2, 12, 2, 8, 4
    ctx = np.array([P * T, P * T - 1])
    npg = np.array([P, P])
    kv = [orc.round_to_bf16(rng.standard_normal((B, Hkv, P, 2, T, d)).astype(np.float32)) for _ in range(L)]
    lm = [orc.build_landmarks(kv[l][:, :, :, 0], ctx) for l in range(L)]
    q_init = rng.standard_normal((L, B, Hq, d))
    q_steps = rng.standard_normal((S, L, B, 2, Hq, d))
    outs, pred, true, n_miss = orc.decode_chain_corrected(q_init, q_steps, lm, kv, npg, ctx, k, T)
    assert n_miss.sum() > 0                                    # independent tokens: the prediction does miss
    for t in range(S):
        for l in range(L):
            want_true, _ = orc.select_topk(q_steps[t, l][:, 0], lm[l], npg, k)      # token 0 = current
            assert np.array_equal(true[t, l], want_true)
            o, _ = orc.sparse_decode_attn(q_steps[t, l], orc.gather_kv(kv[l], want_true), want_true, ctx, T)
            np.testing.assert_allclose(outs[t, l], o, rtol=1e-12, atol=1e-14)
    # another priming query changes the first prediction but not a single output
    outs2, pred2, _, _ = orc.decode_chain_corrected(q_init + 3.0, q_steps, lm, kv, npg, ctx, k, T)
    assert not np.array_equal(pred[0], pred2[0])
    np.testing.assert_allclose(outs, outs2, rtol=1e-12, atol=1e-14)


# ----------------------------------------------------------------------------- dual-token causal tail
def test_causal_tail_equals_dense_causal_attention_over_the_extended_sequence():
    """Full budget: context of n tokens, then the output token, then the speculated token. The result must be
    dense attention over [context, new tokens] with the causal mask, computed here by torch SDPA with an
    explicit boolean mask (the output token does not see the speculated token; both see the whole context)."""
    rng = np.random.default_rng(30)
    B, Tq, Hq, Hkv, P, T, d = 2, 2, 8, 2, 5, 4, 16
    q = rng.standard_normal((B, Tq, Hq, d))
    kv = rng.standard_normal((B, Hkv, P, 2, T, d))
    k_new = rng.standard_normal((B, Tq, Hkv, d))
    v_new = rng.standard_normal((B, Tq, Hkv, d))
    ident = np.tile(np.arange(P, dtype=np.int32), (B, Hkv, 1))
    ctx = np.array([P * T, P * T - 2])
    out, lse = orc.sparse_decode_attn_causal(q, orc.gather_kv(kv, ident), ident, ctx, T, k_new, v_new)
    G = Hq // Hkv
    for b in range(B):
        n = int(ctx[b])
        K = np.concatenate([kv[b, :, :, 0].reshape(Hkv, P * T, d)[:, :n], k_new[b].transpose(1, 0, 2)], axis=1)
        V = np.concatenate([kv[b, :, :, 1].reshape(Hkv, P * T, d)[:, :n], v_new[b].transpose(1, 0, 2)], axis=1)
        Kt = torch.from_numpy(K).repeat_interleave(G, dim=0)
        Vt = torch.from_numpy(V).repeat_interleave(G, dim=0)
        Q = torch.from_numpy(q[b]).permute(1, 0, 2)
        mask = torch.ones(Tq, n + Tq, dtype=torch.bool)
        mask[0, n + 1] = False                                        # output token does not see the speculated one
        ref = torch.nn.functional.scaled_dot_product_attention(Q, Kt, Vt, attn_mask=mask).permute(1, 0, 2).numpy()
        np.testing.assert_allclose(out[b], ref, rtol=1e-10, atol=1e-12)
    # the speculated token's own entry matters to it and not to the output token
    k2, v2 = k_new.copy(), v_new.copy()
    k2[:, 1] += 1.0
    v2[:, 1] -= 2.0
    out2, _ = orc.sparse_decode_attn_causal(q, orc.gather_kv(kv, ident), ident, ctx, T, k2, v2)
    assert np.array_equal(out2[:, 0], out[:, 0]) and not np.allclose(out2[:, 1], out[:, 1])
    # merging by log-sum-exp: the tail result is the lse-weighted mix of the set-only result and the tail's own
    o_set, lse_set = orc.sparse_decode_attn(q, orc.gather_kv(kv, ident), ident, ctx, T)
    b, t, h = 1, 1, 5
    g = h // G
    z_tail = k_new[b, :t + 1, g] @ q[b, t, h] / math.sqrt(d)
    w_set = math.exp(lse_set[b, t, h] - lse[b, t, h])
    w_tail = np.exp(z_tail - lse[b, t, h])
    np.testing.assert_allclose(out[b, t, h], w_set * o_set[b, t, h] + w_tail @ v_new[b, :t + 1, g], rtol=1e-10)
    assert abs(w_set + w_tail.sum() - 1.0) < 1e-12


# ----------------------------------------------------------------------------- finer landmarks
def test_chunk_landmarks_and_chunked_page_scores():
    rng = np.random.default_rng(40)
    B, Hkv, Hq, P, T, d, c = 1, 2, 4, 6, 8, 16, 2
    R = T // c
    ctx = np.array([P * T - 3])                                  # last chunk of the last page is missing, one is partial
    keys = orc.round_to_bf16(rng.standard_normal((B, Hkv, P, T, d)).astype(np.float32))
    lm_c = orc.build_landmarks(keys, ctx, chunk_tokens=c)
    assert lm_c.shape == (B, Hkv, P * R, d)
    toks = keys.reshape(B, Hkv, P * T, d).astype(np.float64)
    for ch in range(P * R):
        lo, hi = ch * c, min((ch + 1) * c, int(ctx[0]))
        want = toks[0, :, lo:hi].mean(axis=1) if hi > lo else np.zeros((Hkv, d))
        assert np.all(np.abs(lm_c[0, :, ch] - want) <= np.maximum(np.abs(want), 1e-30) * 2.0 ** -8)
    assert np.all(lm_c[0, :, -1] == 0.0)
    # whole-page chunks are the page landmarks, bit for bit
    assert np.array_equal(orc.build_landmarks(keys, ctx, chunk_tokens=T), orc.build_landmarks(keys, ctx))
    # chunked page score = brute force over chunks: soft-max over the existing chunks, max over heads and chunks
    q = rng.standard_normal((Hq, d))
    n_chunks = -(-int(ctx[0]) // c)
    score, s, lse = orc.page_scores(q, lm_c[0], P, chunks_per_page=R, n_chunks=n_chunks)
    G = Hq // Hkv
    for g in range(Hkv):
        for p in range(P):
            best = 0.0
            for h in range(g * G, (g + 1) * G):
                z = [sum(q[h, x] * lm_c[0, g, ch, x] for x in range(d)) / math.sqrt(d) for ch in range(n_chunks)]
                den = sum(math.exp(v) for v in z)
                for r in range(R):
                    ch = p * R + r
                    if ch < n_chunks:
                        best = max(best, math.exp(z[ch]) / den)
            assert abs(score[g, p] - best) <= 1e-12 * best
    # R = 1 is the page-level definition
    lm_p = orc.build_landmarks(keys, ctx)
    a, _, _ = orc.page_scores(q, lm_p[0], P)
    b2, _, _ = orc.page_scores(q, lm_p[0], P, chunks_per_page=1)
    assert np.array_equal(a, b2)
    # one-token chunks: a page scores as its best token does
    lm_1 = orc.build_landmarks(keys, ctx, chunk_tokens=1)
    sc1, _, _ = orc.page_scores(q[:2], lm_1[0][:1], P, chunks_per_page=T, n_chunks=int(ctx[0]))
    logits = toks[0, 0, :int(ctx[0])] @ q[0] / math.sqrt(d)
    prob = np.exp(logits - logits.max()); prob /= prob.sum()
    logits1 = toks[0, 0, :int(ctx[0])] @ q[1] / math.sqrt(d)
    prob1 = np.exp(logits1 - logits1.max()); prob1 /= prob1.sum()
    both = np.maximum(prob, prob1)
    pad = np.zeros(P * T); pad[:int(ctx[0])] = both
    np.testing.assert_allclose(sc1[0], pad.reshape(P, T).max(axis=1), rtol=1e-10)
