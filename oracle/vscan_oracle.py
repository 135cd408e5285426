"""CPU oracle for the VScan two-stage visual-token reduction (TEST INFRASTRUCTURE).

This file is test infrastructure, not product code: only the test-suite, the
smoke check and the benchmark's CPU-baseline leg may import it.  It shares no
code with the CUDA library and never calls it.

Everything is evaluated in float64 with numpy, one instance (one crop of one
image, or one LLM sequence) at a time, in the order and notation of the paper.
The method does not approximate anything: its results are exact top-k sets, an
exact argmax and exact means, so each function is that definition written out.

Pins (tests marked "not gpu"): closed forms, hand-built cases with known
answers, brute-force rank counting on tiny inputs, library routines on the
special cases that reduce to them, and the conservation invariants of Eq. 4.
End-task accuracy (all result tables of the paper) is "parity unpinned": it
needs model weights and datasets that are not available offline.

Readings taken where the paper is silent (each listed in the design notes):
ties resolve to the lowest index; survivors are listed in ascending original
index; the [CLS] entry is never a candidate and the row is not renormalised
after skipping it; cosine similarity clamps norms at 1e-12; grouped-query
attention maps query head h to KV head floor(h * Hkv / Hq).
"""
from __future__ import annotations

import numpy as np

SPAN_ONLY = 0   # Eq. 5 literally: softmax over the visual keys only
SPAN_FULL = 1   # softmax over every key of the sequence ("vanilla attention", Sec. 4.2 remarks)

_EPS = 1e-12


# --------------------------------------------------------------------------- Stage 1: scores
def score_row(attn: np.ndarray, cls_offset: int) -> np.ndarray:
    """Eq. 2: S_avg[j] = (1/H) * sum_h S^h[c + j] for one instance.

    attn: [H, L] per-head attention probabilities of the [CLS] query (Eq. 1), or, for encoders
    without [CLS], the per-head attention each token receives (Sec. 4.1, after Eq. 2), c = 0.
    Returns [N] float64 with N = L - c.
    """
    a = np.asarray(attn, dtype=np.float64)
    H = a.shape[0]
    total = np.zeros(a.shape[1] - cls_offset, dtype=np.float64)
    for h in range(H):                       # h ascending, as in the sum of Eq. 2
        total += a[h, cls_offset:]
    return total / H


def cls_attention_rows(q_cls: np.ndarray, k: np.ndarray, scale: float) -> np.ndarray:
    """Eq. 1 for one instance: S^h = Softmax(scale * Q_cls^h K^h^T) over all L keys of the layer
    ([CLS] itself included), one row per head.  q_cls: [H, d], k: [H, L, d].  Returns [H, L]."""
    q = np.asarray(q_cls, dtype=np.float64)
    kk = np.asarray(k, dtype=np.float64)
    rows = np.empty(kk.shape[:2])
    for h in range(q.shape[0]):
        z = scale * (kk[h] @ q[h])
        z = z - z.max()
        e = np.exp(z)
        rows[h] = e / e.sum()
    return rows


def received_attention(probs: np.ndarray) -> np.ndarray:
    """Sec. 4.1 (text after Eq. 2): for an encoder without [CLS], the score source is the average
    attention each token receives from the *other* tokens.

    probs: [H, n, n] with probs[h, i, j] = attention of query i on key j.  Returns [H, n]:
    mean over i != j.  (Small-size helper: the library takes these rows as input.)
    """
    p = np.asarray(probs, dtype=np.float64)
    H, n, _ = p.shape
    out = np.zeros((H, n))
    for h in range(H):
        col = p[h].sum(axis=0) - np.diagonal(p[h])
        out[h] = col / max(n - 1, 1)
    return out


# --------------------------------------------------------------------------- exact top-k
def topk_lowest_index(scores: np.ndarray, k: int, candidates: np.ndarray | None = None) -> np.ndarray:
    """The k candidates with the largest score; equal scores go to the lower index (Sec. 4.1, text
    after Eq. 2: the threshold tau is whatever value leaves the wanted count).  Returns ascending indices.

    A stable sort on descending score keeps equal scores in index order, so the first k entries
    are exactly the set {i : #{j : s_j > s_i or (s_j == s_i and j < i)} < k}.
    """
    s = np.asarray(scores, dtype=np.float64)
    cand = np.arange(s.shape[0]) if candidates is None else np.asarray(candidates, dtype=np.int64)
    if k < 0 or k > cand.shape[0]:
        raise ValueError("k out of range")
    order = np.argsort(-s[cand], kind="stable")
    return np.sort(cand[order[:k]])


# --------------------------------------------------------------------------- Stage 1: selection
def window_of(t: int, frames: int, grid_h: int, grid_w: int, win_h: int, win_w: int) -> int:
    """Window index of token t = f*Gh*Gw + r*Gw + c for non-overlapping win_h x win_w windows
    (Sec. 4.1 "Local Scan"); windows are numbered frame-major, then row-major."""
    per_frame = grid_h * grid_w
    f, rem = divmod(t, per_frame)
    r, c = divmod(rem, grid_w)
    wpr = grid_w // win_w
    wpf = (grid_h // win_h) * wpr
    return f * wpf + (r // win_h) * wpr + (c // win_w)


def select_global_local(scores_global: np.ndarray, scores_local: np.ndarray, frames: int,
                        grid_h: int, grid_w: int, win_h: int, win_w: int, k_w: int, k_g: int):
    """Sec. 4.1: local scan (Eq. 3) first, then global scan (Eq. 2) over the tokens the local scan
    did not take (footnote to Sec. 4.1: local tokens have priority and are excluded from the global
    selection), then the union.  Returns (kept ascending, local ascending, global ascending)."""
    N = frames * grid_h * grid_w
    if grid_h % win_h or grid_w % win_w:
        raise ValueError("window must divide the grid")
    s_g = np.asarray(scores_global, dtype=np.float64)
    s_l = np.asarray(scores_local, dtype=np.float64)
    assert s_g.shape == (N,) and s_l.shape == (N,)
    win = np.array([window_of(t, frames, grid_h, grid_w, win_h, win_w) for t in range(N)])
    W = frames * (grid_h // win_h) * (grid_w // win_w)
    local = []
    for w in range(W):
        members = np.nonzero(win == w)[0]          # ascending token index
        local.append(topk_lowest_index(s_l, k_w, members))
    local = np.sort(np.concatenate(local)) if local else np.zeros(0, dtype=np.int64)
    taken = np.zeros(N, dtype=bool)
    taken[local] = True
    rest = np.nonzero(~taken)[0]
    glob = topk_lowest_index(s_g, k_g, rest)
    kept = np.sort(np.concatenate([local, glob])).astype(np.int64)
    return kept, local.astype(np.int64), glob.astype(np.int64)


# --------------------------------------------------------------------------- Stage 1: merging
def cosine_matrix(xu: np.ndarray, xs: np.ndarray) -> np.ndarray:
    """cos(x_u, x_s) for every (unselected, selected) pair, norms clamped at 1e-12."""
    nu = np.maximum(np.sqrt((xu * xu).sum(axis=1)), _EPS)
    ns = np.maximum(np.sqrt((xs * xs).sum(axis=1)), _EPS)
    return (xu @ xs.T) / nu[:, None] / ns[None, :]


def merge(x: np.ndarray, cls_offset: int, kept_idx: np.ndarray, metric: np.ndarray | None = None):
    """Sec. 4.1 "Token Merging", Eq. 4, for one instance.

    x: [L, D] features (row c + t is patch token t).  kept_idx: [K1] ascending token indices.
    metric: optional [L, Dm] representation the cosine similarity is taken on (default: x).
    Each unselected token u goes to a(u) = argmax_s cos(x_u, x_s) (first maximum = lowest slot);
    merged[s] = (x_s + sum_{a(u)=s} x_u) / (|U^s| + 1).
    Returns merged [K1, D] float64 (unrounded), assign [N] (slot of every token; a kept token maps
    to its own slot), counts [K1] (group size including the kept token itself).
    """
    x = np.asarray(x, dtype=np.float64)
    m = x if metric is None else np.asarray(metric, dtype=np.float64)
    N = x.shape[0] - cls_offset
    kept = np.asarray(kept_idx, dtype=np.int64)
    K1 = kept.shape[0]
    is_kept = np.zeros(N, dtype=bool)
    is_kept[kept] = True
    unsel = np.nonzero(~is_kept)[0]
    assign = np.empty(N, dtype=np.int64)
    assign[kept] = np.arange(K1)
    if unsel.size:
        cos = cosine_matrix(m[cls_offset + unsel], m[cls_offset + kept])
        assign[unsel] = np.argmax(cos, axis=1)       # first maximum: lowest slot on ties
    merged, counts = mean_merge(x, cls_offset, kept, assign)
    return merged, assign, counts


def mean_merge(x: np.ndarray, cls_offset: int, kept_idx: np.ndarray, assign: np.ndarray):
    """Eq. 4 alone, for groups that are already decided: assign[u] is the kept slot of token u (a kept
    token holds its own slot).  merged[s] = (x_s + sum_{u in U^s} x_u) / (|U^s| + 1).
    Returns merged [K1, D] float64 (unrounded) and counts [K1] (|U^s| + 1)."""
    x = np.asarray(x, dtype=np.float64)
    kept = np.asarray(kept_idx, dtype=np.int64)
    N, K1 = x.shape[0] - cls_offset, kept.shape[0]
    is_kept = np.zeros(N, dtype=bool)
    is_kept[kept] = True
    merged = x[cls_offset + kept].copy()
    counts = np.ones(K1, dtype=np.int64)
    for u in np.nonzero(~is_kept)[0]:                 # sum over U^s in token order, then divide
        merged[assign[u]] += x[cls_offset + u]
        counts[assign[u]] += 1
    merged /= counts[:, None]
    return merged, counts


# --------------------------------------------------------------------------- Stage 2
def score_qk(q: np.ndarray, k: np.ndarray, span_begin: int, span_len: int, scale: float,
             softmax_span: int = SPAN_ONLY) -> np.ndarray:
    """Eq. 5 for one sequence: per query head h, softmax_j(scale * q_h . K_{g(h), j}); the result is
    the mean over the Hq query heads of the probabilities on the span [span_begin, span_begin+n).

    q: [Hq, d] query of the last instruction token; k: [Hkv, S, d] keys of the layer.
    SPAN_ONLY normalises over the span's keys (Eq. 5: K_V holds the visual tokens only);
    SPAN_FULL over all S keys (the last token sees every key).  g(h) = floor(h * Hkv / Hq).
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    Hq, Hkv, S = q.shape[0], k.shape[0], k.shape[1]
    lo, hi = (span_begin, span_begin + span_len) if softmax_span == SPAN_ONLY else (0, S)
    total = np.zeros(span_len)
    for h in range(Hq):
        g = (h * Hkv) // Hq
        z = scale * (k[g, lo:hi] @ q[h])
        z = z - z.max()
        p = np.exp(z)
        p = p / p.sum()
        total += p[span_begin - lo: span_begin - lo + span_len]
    return total / Hq


def compaction_rows(n_sys: int, n_vis: int, n_txt: int, kept_vis: np.ndarray) -> np.ndarray:
    """Sec. 4.2 remarks: after pruning, the sequence holds the system tokens, the surviving visual
    tokens and the text tokens, in their original order."""
    kv = np.asarray(kept_vis, dtype=np.int64)
    return np.concatenate([np.arange(n_sys), n_sys + kv, np.arange(n_sys + n_vis, n_sys + n_vis + n_txt)])


def llm_prune(q_last, k, v, hidden, pos_ids, n_sys: int, n_vis: int, n_txt: int, k_keep: int,
              scale: float, softmax_span: int = SPAN_ONLY):
    """Sec. 4.2 for one sequence: score the visual span by Eq. 5, keep the k_keep highest, and keep
    only their rows (plus all system / text rows) of hidden states, K, V and position ids.

    k, v: [Hkv, S, d]; hidden: [S, Dh]; pos_ids: [P, S].  Returns a dict.
    """
    scores = score_qk(q_last, k, n_sys, n_vis, scale, softmax_span)
    kept_vis = topk_lowest_index(scores, k_keep)
    rows = compaction_rows(n_sys, n_vis, n_txt, kept_vis)
    return {"scores": scores, "kept_vis": kept_vis, "rows": rows,
            "hidden": np.asarray(hidden)[rows], "k": np.asarray(k)[:, rows],
            "v": np.asarray(v)[:, rows], "pos": np.asarray(pos_ids)[:, rows]}


# --------------------------------------------------------------------------- helpers for tests
def topk_boundary_gap(scores: np.ndarray, k: int, candidates: np.ndarray | None = None) -> float:
    """Score difference between the k-th and (k+1)-th best candidate (inf when nothing is cut)."""
    s = np.asarray(scores, dtype=np.float64)
    cand = np.arange(s.shape[0]) if candidates is None else np.asarray(candidates)
    if k <= 0 or k >= cand.shape[0]:
        return float("inf")
    v = np.sort(s[cand])[::-1]
    return float(v[k - 1] - v[k])
