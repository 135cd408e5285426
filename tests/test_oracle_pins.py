"""Pins for the CPU oracle: every check here is fixed by the paper or by mathematics, not by
the oracle's own formulae.  Closed forms, hand-built cases, brute force on tiny inputs, library
routines on the special cases that reduce to them, and the invariants of Eq. 4.
"""
import os

import numpy as np
import pytest
import torch

from oracle import budget
from oracle import vscan_oracle as vo

RNG = np.random.default_rng(1234)


# ------------------------------------------------------------------ paper-printed values
def _rows(path):
    for line in open(path):
        line = line.strip()
        if line and not line.startswith("#"):
            yield [c.strip() for c in line.split("|")]


def test_budget_values_printed_in_paper(golden_dir):
    n = 0
    for kind, inputs, expected, tol, _cite in _rows(os.path.join(golden_dir, "budget_paper_values.txt")):
        a = inputs.split()
        if kind == "avg_rate":
            got = budget.average_retention(float(a[0]), float(a[1]), int(a[2]), int(a[3]))
        else:
            got = budget.average_tokens(int(a[0]), int(a[1]), int(a[2]), int(a[3]))
        assert abs(got - float(expected)) <= float(tol) + 1e-12, (kind, inputs, got)
        n += 1
    assert n == 9


def test_eq6_flops_values_printed_in_paper(golden_dir):
    n = 0
    for tokens, expected, tol, _cite in _rows(os.path.join(golden_dir, "flops_paper_values.txt")):
        got = budget.prefill_flops([int(tokens)] * 32, d=4096, m=11008) / 1e12
        assert abs(got - float(expected)) <= float(tol), (tokens, got)
        n += 1
    assert n == 7
    # two-stage schedule averages to the same count the paper quotes (App. B.1)
    per_layer = budget.vscan_tokens_per_layer(96, 32, 16, 32)
    assert sum(per_layer) / 32 == 64


# ------------------------------------------------------------------ Eq. 2: head mean
def test_score_row_one_hot_heads_closed_form():
    # Head h puts all its mass on patch p[h]; the head mean is (#heads on j)/H.  The [CLS] entry
    # (index 0) takes the mass of one head and must be skipped, not shifted into patch 0.
    H, N = 5, 7
    target = [0, 3, 3, 6, None]            # None: mass on [CLS]
    attn = np.zeros((H, N + 1))
    for h, t in enumerate(target):
        attn[h, 0 if t is None else 1 + t] = 1.0
    s = vo.score_row(attn, 1)
    expect = np.zeros(N)
    expect[0], expect[3], expect[6] = 1 / 5, 2 / 5, 1 / 5
    np.testing.assert_allclose(s, expect, atol=1e-15)
    assert abs(s.sum() - 4 / 5) < 1e-15      # not renormalised after dropping [CLS]
    # without [CLS] nothing is skipped
    s0 = vo.score_row(attn, 0)
    assert s0.shape == (N + 1,) and abs(s0[0] - 1 / 5) < 1e-15


def test_score_row_uniform_and_linear():
    H, L = 4, 10
    np.testing.assert_allclose(vo.score_row(np.full((H, L), 1 / L), 1), np.full(L - 1, 1 / L))
    # head h holds h * ramp -> mean is mean(h) * ramp
    ramp = np.arange(L, dtype=np.float64)
    attn = np.stack([h * ramp for h in range(H)])
    np.testing.assert_allclose(vo.score_row(attn, 1), 1.5 * ramp[1:])


def test_cls_attention_rows_eq1():
    # planted distribution: q = e_0 / scale, K_j = log(p_j) e_0  ->  the softmax returns p
    H, L, d, scale = 3, 6, 4, 0.5
    p = RNG.random((H, L)); p /= p.sum(1, keepdims=True)
    q = np.zeros((H, d)); q[:, 0] = 1 / scale
    k = np.zeros((H, L, d)); k[:, :, 0] = np.log(p)
    np.testing.assert_allclose(vo.cls_attention_rows(q, k, scale), p, atol=1e-14)
    # library special case, and Eq. 1 -> Eq. 2 equals the Eq. 5 form with the softmax over all keys
    q2 = RNG.standard_normal((H, d)); k2 = RNG.standard_normal((H, L, d))
    ref = torch.softmax(torch.from_numpy(0.7 * np.einsum("hd,hld->hl", q2, k2)), dim=-1).numpy()
    rows = vo.cls_attention_rows(q2, k2, 0.7)
    np.testing.assert_allclose(rows, ref, atol=1e-15)
    np.testing.assert_allclose(vo.score_row(rows, 1), vo.score_qk(q2, k2, 1, L - 1, 0.7, vo.SPAN_FULL), atol=1e-15)


def test_received_attention_excludes_self():
    # Two heads, three tokens.  Head 0: every query attends only to itself -> receives 0 from
    # others.  Head 1: every query attends uniformly -> each token receives 1/3 from each of the
    # two others -> mean 1/3.
    eye = np.eye(3)
    uni = np.full((3, 3), 1 / 3)
    r = vo.received_attention(np.stack([eye, uni]))
    np.testing.assert_allclose(r[0], 0.0)
    np.testing.assert_allclose(r[1], 1 / 3)
    # a column-specific case: everyone attends to token 2 only
    p = np.zeros((1, 3, 3))
    p[0, :, 2] = 1.0
    np.testing.assert_allclose(vo.received_attention(p)[0], [0, 0, 1.0])


# ------------------------------------------------------------------ exact top-k
def _rank_count_topk(s, k, cand):
    """Definition: i is kept iff fewer than k candidates beat it (higher score, or equal score and
    lower index)."""
    out = []
    for i in cand:
        beats = sum(1 for j in cand if s[j] > s[i] or (s[j] == s[i] and j < i))
        if beats < k:
            out.append(i)
    return sorted(out)


def test_topk_matches_rank_count_definition_with_ties():
    for trial in range(200):
        n = int(RNG.integers(1, 14))
        s = RNG.integers(0, 4, size=n).astype(np.float64)      # many ties
        cand = sorted(RNG.choice(n, size=int(RNG.integers(1, n + 1)), replace=False).tolist())
        k = int(RNG.integers(0, len(cand) + 1))
        got = vo.topk_lowest_index(s, k, np.array(cand)).tolist()
        assert got == _rank_count_topk(s, k, cand), (s, cand, k)


def test_topk_uniform_scores_select_first_k():
    s = np.full(20, 0.25)
    assert vo.topk_lowest_index(s, 7).tolist() == list(range(7))
    assert vo.topk_lowest_index(s, 0).tolist() == []
    assert vo.topk_lowest_index(s, 20).tolist() == list(range(20))


def test_topk_distinct_scores_match_torch_topk():
    s = RNG.permutation(500).astype(np.float64) / 500
    for k in (1, 17, 499):
        ref = torch.topk(torch.from_numpy(s), k).indices.sort().values.numpy()
        np.testing.assert_array_equal(vo.topk_lowest_index(s, k), ref)


def test_topk_negative_and_signed_zero():
    s = np.array([-1.0, 0.0, -0.0, -3.0, 0.0])
    assert vo.topk_lowest_index(s, 2).tolist() == [1, 2]       # -0.0 ties with 0.0 -> lowest index


# ------------------------------------------------------------------ windows and selection
def test_window_map_hand_enumerated():
    # 4x6 grid, 2x3 windows, two frames.  Enumerate windows by nested loops (frame, window row,
    # window column, inner row, inner column): an independent construction of the partition.
    F, Gh, Gw, wh, ww = 2, 4, 6, 2, 3
    expect = {}
    w = 0
    for f in range(F):
        for wr in range(Gh // wh):
            for wc in range(Gw // ww):
                for r in range(wh):
                    for c in range(ww):
                        expect[f * Gh * Gw + (wr * wh + r) * Gw + wc * ww + c] = w
                w += 1
    assert w == 8
    for t in range(F * Gh * Gw):
        assert vo.window_of(t, F, Gh, Gw, wh, ww) == expect[t]
    # spot values typed by hand: token 9 = row 1, col 3 -> window 1; token 24+13 = frame 1,
    # row 2, col 1 -> window 4 + 2 = 6
    assert vo.window_of(9, F, Gh, Gw, wh, ww) == 1
    assert vo.window_of(37, F, Gh, Gw, wh, ww) == 6


def test_select_hand_example():
    # 2x4 grid, windows 2x2 -> window 0 = tokens {0,1,4,5}, window 1 = {2,3,6,7}.
    s_l = np.array([.1, .9, .2, .2, .8, .3, .1, .0])
    s_g = np.array([.5, .6, .7, .1, .9, .4, .3, .2])
    kept, local, glob = vo.select_global_local(s_g, s_l, 1, 2, 4, 2, 2, k_w=1, k_g=2)
    assert local.tolist() == [1, 2]          # window 1 ties .2/.2 -> token 2 (lowest index)
    # global over the rest {0,3,4,5,6,7}: best are 4 (.9) and 0 (.5); token 2 (.7) is already local
    assert glob.tolist() == [0, 4]
    assert kept.tolist() == [0, 1, 2, 4]


def test_select_invariants_random():
    for trial in range(30):
        F = int(RNG.integers(1, 3)); wh, ww = int(RNG.integers(1, 4)), int(RNG.integers(1, 4))
        Gh, Gw = wh * int(RNG.integers(1, 4)), ww * int(RNG.integers(1, 4))
        N = F * Gh * Gw
        W = F * (Gh // wh) * (Gw // ww)
        k_w = int(RNG.integers(0, wh * ww + 1))
        k_g = int(RNG.integers(0, N - W * k_w + 1))
        s_g = RNG.integers(0, 5, N) / 4.0
        s_l = RNG.integers(0, 5, N) / 4.0
        kept, local, glob = vo.select_global_local(s_g, s_l, F, Gh, Gw, wh, ww, k_w, k_g)
        assert len(kept) == W * k_w + k_g                      # exactly K1 survivors
        assert np.all(np.diff(kept) > 0)                        # strictly ascending, no duplicates
        assert set(local).isdisjoint(glob)
        per_win = np.bincount([vo.window_of(t, F, Gh, Gw, wh, ww) for t in local], minlength=W)
        assert np.all(per_win == k_w)                           # uniform budget per window
        # brute force: global set by the rank-count definition over the complement
        rest = [t for t in range(N) if t not in set(local.tolist())]
        assert glob.tolist() == _rank_count_topk(s_g, k_g, rest)
        # brute force: local set per window
        for w in range(W):
            members = [t for t in range(N) if vo.window_of(t, F, Gh, Gw, wh, ww) == w]
            assert sorted(set(local.tolist()) & set(members)) == _rank_count_topk(s_l, k_w, members)


def test_select_uniform_scores_first_indices():
    F, Gh, Gw, wh, ww = 1, 4, 4, 2, 2
    s = np.full(16, 0.5)
    kept, local, glob = vo.select_global_local(s, s, F, Gh, Gw, wh, ww, k_w=2, k_g=3)
    assert local.tolist() == [0, 1, 2, 3, 8, 9, 10, 11]        # first two of each window
    assert glob.tolist() == [4, 5, 6]                            # first three of the remainder


def test_select_global_only_and_local_only():
    s_g = RNG.random(36); s_l = RNG.random(36)
    kept, local, glob = vo.select_global_local(s_g, s_l, 1, 6, 6, 3, 3, k_w=0, k_g=10)
    assert local.size == 0
    np.testing.assert_array_equal(kept, np.sort(np.argsort(-s_g)[:10]))
    kept, local, glob = vo.select_global_local(s_g, s_l, 1, 6, 6, 3, 3, k_w=9, k_g=0)
    assert kept.tolist() == list(range(36))


# ------------------------------------------------------------------ Eq. 4: merging
def test_merge_orthogonal_basis_closed_form():
    # Kept tokens are scaled basis vectors a_s * e_s, so cos(u, kept_s) = u_s / |u|: the argmax is
    # the largest coordinate of u whatever the scales a_s (a missing normalisation would favour
    # the long kept vector instead).
    D = 4
    x = np.zeros((6, D))
    x[0] = 100.0 * np.eye(D)[0]      # kept slot 0, very long
    x[2] = 0.01 * np.eye(D)[1]       # kept slot 1, very short
    x[5] = 1.0 * np.eye(D)[2]        # kept slot 2
    x[1] = [0.5, 0.6, 0.1, 0.0]      # -> slot 1
    x[3] = [0.2, 0.1, 0.9, 3.0]      # -> slot 2 (coordinate 3 has no kept token)
    x[4] = [2.0, 1.0, 1.0, 0.0]      # -> slot 0
    merged, assign, counts = vo.merge(x, 0, np.array([0, 2, 5]))
    assert assign.tolist() == [0, 1, 1, 2, 0, 2]
    assert counts.tolist() == [2, 2, 2]
    np.testing.assert_allclose(merged[0], (x[0] + x[4]) / 2)
    np.testing.assert_allclose(merged[1], (x[2] + x[1]) / 2)
    np.testing.assert_allclose(merged[2], (x[5] + x[3]) / 2)


def test_merge_negative_cosine_and_tie_lowest_slot():
    x = np.array([[1.0, 0.0], [0.0, 1.0], [-1.0, -1.0], [1.0, 1.0]])
    # token 2 has cos = -0.707 with both kept tokens -> tie -> slot 0; token 3 ties at +0.707 -> 0
    _, assign, counts = vo.merge(x, 0, np.array([0, 1]))
    assert assign.tolist() == [0, 1, 0, 0] and counts.tolist() == [3, 1]


def test_merge_cls_row_is_never_read():
    x = RNG.standard_normal((9, 5))
    kept = np.array([1, 4, 6])
    a = vo.merge(x, 1, kept)
    x2 = x.copy(); x2[0] = 1e6
    b = vo.merge(x2, 1, kept)
    np.testing.assert_array_equal(a[0], b[0]); np.testing.assert_array_equal(a[1], b[1])


def test_merge_matches_torch_cosine_similarity_argmax():
    x = RNG.standard_normal((40, 16))
    kept = np.sort(RNG.choice(40, 7, replace=False))
    _, assign, _ = vo.merge(x, 0, kept)
    xt = torch.from_numpy(x)
    cos = torch.nn.functional.cosine_similarity(xt[:, None, :], xt[kept][None, :, :], dim=-1)
    ref = cos.argmax(dim=1).numpy()
    unsel = np.setdiff1d(np.arange(40), kept)
    np.testing.assert_array_equal(assign[unsel], ref[unsel])
    np.testing.assert_array_equal(assign[kept], np.arange(7))


def test_merge_invariants():
    L, D, c = 31, 6, 1
    x = RNG.standard_normal((L, D))
    kept = np.sort(RNG.choice(L - c, 5, replace=False))
    merged, assign, counts = vo.merge(x, c, kept)
    # every output token times its group size sums to the token sum over its group (Eq. 4)
    np.testing.assert_allclose((merged * counts[:, None]).sum(0), x[c:].sum(0), atol=1e-12)
    assert counts.sum() == L - c
    for s in range(5):
        members = np.nonzero(assign == s)[0]
        np.testing.assert_allclose(merged[s] * counts[s], x[c + members].sum(0), atol=1e-12)
    # keep-all makes the merge the identity
    m_all, a_all, c_all = vo.merge(x, c, np.arange(L - c))
    np.testing.assert_array_equal(m_all, x[c:]); assert np.all(c_all == 1)
    # a single kept token receives everything: the mean of all tokens
    m1, _, c1 = vo.merge(x, c, np.array([7]))
    np.testing.assert_allclose(m1[0], x[c:].mean(0), atol=1e-13); assert c1[0] == L - c
    # an unselected token identical to a kept token goes to it
    x2 = x.copy(); x2[c + 3] = 2.5 * x2[c + kept[2]] if 3 not in kept else x2[c + 3]
    if 3 not in kept:
        assert vo.merge(x2, c, kept)[1][3] == 2


def test_merge_permuting_unselected_permutes_assign_only():
    L, D = 20, 5
    x = RNG.standard_normal((L, D))
    kept = np.array([2, 9, 15])
    merged, assign, counts = vo.merge(x, 0, kept)
    unsel = np.setdiff1d(np.arange(L), kept)
    perm = RNG.permutation(unsel)
    x2 = x.copy(); x2[unsel] = x[perm]
    merged2, assign2, counts2 = vo.merge(x2, 0, kept)
    np.testing.assert_array_equal(assign2[unsel], assign[perm])
    np.testing.assert_allclose(merged2, merged, atol=1e-12)
    np.testing.assert_array_equal(counts2, counts)


def test_merge_separate_metric():
    x = RNG.standard_normal((6, 3))
    metric = np.array([[1, 0], [0, 1], [0.9, 0.1], [0.1, 0.9], [1, 0.2], [0.3, 1]], dtype=float)
    merged, assign, _ = vo.merge(x, 0, np.array([0, 1]), metric=metric)
    assert assign.tolist() == [0, 1, 0, 1, 0, 1]
    np.testing.assert_allclose(merged[0], x[[0, 2, 4]].mean(0))


# ------------------------------------------------------------------ Eq. 5: text attention
def test_score_qk_recovers_planted_distribution():
    # q = e_0 / scale and K_j = log(p_j) e_0 make the logits log p_j, so the softmax is p exactly.
    Hq, Hkv, S, d, scale = 4, 2, 9, 6, 0.37
    n_sys, n_vis = 2, 5
    p = RNG.random((Hkv, n_vis)); p /= p.sum(1, keepdims=True)
    k = RNG.standard_normal((Hkv, S, d))
    q = np.zeros((Hq, d)); q[:, 0] = 1 / scale
    for g in range(Hkv):
        k[g, n_sys:n_sys + n_vis] = 0
        k[g, n_sys:n_sys + n_vis, 0] = np.log(p[g])
    s = vo.score_qk(q, k, n_sys, n_vis, scale, vo.SPAN_ONLY)
    # heads 0,1 read KV head 0; heads 2,3 read KV head 1 (grouped-query mapping)
    np.testing.assert_allclose(s, (2 * p[0] + 2 * p[1]) / 4, atol=1e-14)
    assert abs(s.sum() - 1) < 1e-14


def test_score_qk_gqa_mapping_distinguishes_heads():
    # Hq=6, Hkv=3: query heads (0,1)->0, (2,3)->1, (4,5)->2.  Only query head 4 is non-zero, and only
    # KV head 2 has structure, so any other mapping returns the uniform distribution.
    Hq, Hkv, n, d = 6, 3, 4, 3
    q = np.zeros((Hq, d)); q[4] = [1, 0, 0]
    k = np.zeros((Hkv, n, d)); k[2, :, 0] = np.log([1, 2, 3, 4.0])
    s = vo.score_qk(q, k, 0, n, 1.0)
    expect = (5 * np.full(n, 0.25) + np.array([1, 2, 3, 4.0]) / 10) / 6
    np.testing.assert_allclose(s, expect, atol=1e-15)


def test_score_qk_full_span_mass():
    Hq, S, d = 2, 7, 4
    q = RNG.standard_normal((Hq, d)); k = RNG.standard_normal((Hq, S, d))
    full = vo.score_qk(q, k, 2, 3, 0.5, vo.SPAN_FULL)
    ref = torch.softmax(torch.from_numpy(0.5 * np.einsum("hd,hsd->hs", q, k)), dim=-1).mean(0).numpy()
    np.testing.assert_allclose(full, ref[2:5], atol=1e-15)
    only = vo.score_qk(q, k, 2, 3, 0.5, vo.SPAN_ONLY)
    ref2 = torch.softmax(torch.from_numpy(0.5 * np.einsum("hd,hsd->hs", q, k[:, 2:5])), dim=-1).mean(0).numpy()
    np.testing.assert_allclose(only, ref2, atol=1e-15)
    assert full.sum() < 1 and abs(only.sum() - 1) < 1e-14


def test_score_qk_equal_keys_uniform_and_large_logits_stable():
    q = RNG.standard_normal((3, 5)); k = np.tile(RNG.standard_normal((1, 1, 5)), (3, 8, 1))
    np.testing.assert_allclose(vo.score_qk(q, k, 1, 6, 1.0), 1 / 6, atol=1e-15)
    qb = np.array([[1000.0]]); kb = np.array([[[1.0], [2.0], [2.0]]])
    np.testing.assert_allclose(vo.score_qk(qb, kb, 0, 3, 1.0), [0, .5, .5], atol=1e-12)


# ------------------------------------------------------------------ Sec. 4.2: compaction
def test_llm_prune_hand_example():
    n_sys, n_vis, n_txt, d = 1, 4, 2, 2
    S = 7
    q = np.array([[1.0, 0.0]])
    k = np.zeros((1, S, d)); k[0, n_sys:n_sys + n_vis, 0] = [0.1, 0.4, 0.3, 0.4]
    v = np.arange(S * d, dtype=float).reshape(1, S, d)
    hidden = np.arange(S * 3, dtype=float).reshape(S, 3)
    pos = np.stack([np.arange(S), 10 * np.arange(S)])
    out = vo.llm_prune(q, k, v, hidden, pos, n_sys, n_vis, n_txt, 2, 1.0)
    assert out["kept_vis"].tolist() == [1, 3]                 # the two 0.4 keys
    assert out["rows"].tolist() == [0, 2, 4, 5, 6]
    np.testing.assert_array_equal(out["hidden"], hidden[[0, 2, 4, 5, 6]])
    np.testing.assert_array_equal(out["v"], v[:, [0, 2, 4, 5, 6]])
    np.testing.assert_array_equal(out["pos"], pos[:, [0, 2, 4, 5, 6]])    # original ids, no renumbering
    out1 = vo.llm_prune(q, k, v, hidden, pos, n_sys, n_vis, n_txt, 1, 1.0)
    assert out1["kept_vis"].tolist() == [1]                    # tie .4/.4 -> lowest index


def test_compaction_matches_index_select_and_keeps_order():
    n_sys, n_vis, n_txt = 3, 10, 4
    kept = np.array([0, 2, 3, 9])
    rows = vo.compaction_rows(n_sys, n_vis, n_txt, kept)
    assert rows.tolist() == [0, 1, 2, 3, 5, 6, 12, 13, 14, 15, 16]
    h = torch.arange(17 * 2).reshape(17, 2)
    np.testing.assert_array_equal(h.index_select(0, torch.from_numpy(rows)).numpy(), h.numpy()[rows])
    assert np.all(np.diff(rows) > 0)


# ------------------------------------------------------------------ helpers the parity tests lean on
def test_mean_merge_hand_example_and_agreement_with_merge():
    # five tokens in one dimension, tokens 1 and 3 kept; groups decided by hand: {1, 0, 2} and {3, 4}
    x = np.array([[2.0], [4.0], [9.0], [10.0], [30.0]])
    merged, counts = vo.mean_merge(x, 0, np.array([1, 3]), np.array([0, 0, 0, 1, 1]))
    assert merged[:, 0].tolist() == [(4.0 + 2.0 + 9.0) / 3, (10.0 + 30.0) / 2] and counts.tolist() == [3, 2]
    # a [CLS] row in front shifts the rows, not the token numbering
    xc = np.concatenate([[[1000.0]], x])
    assert np.array_equal(vo.mean_merge(xc, 1, np.array([1, 3]), np.array([0, 0, 0, 1, 1]))[0], merged)
    # merge() = cosine arg-max followed by exactly this function
    xr = RNG.standard_normal((41, 12))
    kept = np.array([3, 8, 20, 33])
    m, a, c = vo.merge(xr, 1, kept)
    m2, c2 = vo.mean_merge(xr, 1, kept, a)
    assert np.array_equal(m, m2) and np.array_equal(c, c2)


def test_topk_boundary_gap_hand_values():
    s = np.array([0.5, 0.1, 0.9, 0.4, 0.7])
    assert vo.topk_boundary_gap(s, 2) == pytest.approx(0.7 - 0.5)
    assert vo.topk_boundary_gap(s, 4) == pytest.approx(0.4 - 0.1)
    assert vo.topk_boundary_gap(s, 1, np.array([1, 3, 4])) == pytest.approx(0.7 - 0.4)   # candidates only
    assert vo.topk_boundary_gap(s, 0) == float("inf") and vo.topk_boundary_gap(s, 5) == float("inf")
    assert vo.topk_boundary_gap(np.array([1.0, 1.0, 0.0]), 1) == 0.0                     # an exact tie at the cut


# ------------------------------------------------------------------ planted mistakes are caught
@pytest.mark.parametrize("mistake", ["no_norm", "shift_cls", "gqa_mod", "tie_high"])
def test_pins_detect_planted_oracle_mistakes(monkeypatch, mistake):
    """Each plausible slip, planted into the oracle, must fail at least one pin above."""
    if mistake == "no_norm":
        monkeypatch.setattr(vo, "cosine_matrix", lambda xu, xs: xu @ xs.T)
        with pytest.raises(AssertionError):
            test_merge_orthogonal_basis_closed_form()
    elif mistake == "shift_cls":
        orig = vo.score_row
        monkeypatch.setattr(vo, "score_row", lambda a, c: orig(np.asarray(a)[:, :np.asarray(a).shape[1] - c], 0))
        with pytest.raises(AssertionError):
            test_score_row_one_hot_heads_closed_form()
    elif mistake == "gqa_mod":
        def bad(q, k, b, n, scale, span=vo.SPAN_ONLY):
            q = np.asarray(q, float); k = np.asarray(k, float)
            tot = np.zeros(n)
            for h in range(q.shape[0]):
                z = scale * (k[h % k.shape[0], b:b + n] @ q[h]); p = np.exp(z - z.max()); tot += p / p.sum()
            return tot / q.shape[0]
        monkeypatch.setattr(vo, "score_qk", bad)
        with pytest.raises(AssertionError):
            test_score_qk_gqa_mapping_distinguishes_heads()
    else:
        def bad_topk(s, k, candidates=None):
            s = np.asarray(s, float); cand = np.arange(len(s)) if candidates is None else np.asarray(candidates)
            rev = cand[::-1]                                   # ties now go to the highest index
            return np.sort(rev[np.argsort(-s[rev], kind="stable")[:k]])
        monkeypatch.setattr(vo, "topk_lowest_index", bad_topk)
        with pytest.raises(AssertionError):
            test_select_hand_example()
