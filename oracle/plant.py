"""Margin planting for parity inputs (TEST INFRASTRUCTURE, see package note).

Bit-exact index parity is only meaningful where the fp64 oracle's decision is
not a near-tie.  These helpers take generated inputs and nudge them, using the
oracle alone, until every k-boundary (Eq. 2, Eq. 3, Sec. 4.2 top-k) has a score
gap above `margin` and every unselected token's best and second-best cosine
(Sec. 4.1 "Token Merging") differ by more than `margin`.  All arrays stay
representable in the workload's I/O dtype.
"""
from __future__ import annotations

import numpy as np

from synth import VScanConfig, redraw_token, round_to_dtype

from . import vscan_oracle as vo

DEFAULT_MARGIN = 1.5e-4


def _windows(cfg: VScanConfig):
    win = np.array([vo.window_of(t, cfg.frames, cfg.grid_h, cfg.grid_w, cfg.win_h, cfg.win_w)
                    for t in range(cfg.N)])
    return [np.nonzero(win == w)[0] for w in range(cfg.W)]


def _lift(attn: np.ndarray, cfg: VScanConfig, cand: np.ndarray, k: int, margin: float) -> bool:
    """Raise, on every head, the entries of the top-k candidates that sit closer than `margin`
    to the (k+1)-th score.  Returns True when nothing had to change."""
    if k <= 0 or k >= cand.size:
        return True
    s = vo.score_row(attn, cfg.cls)
    top = vo.topk_lowest_index(s, k, cand)
    rest = np.setdiff1d(cand, top)
    thr = s[rest].max()
    low = top[s[top] < thr + margin]
    if low.size == 0:
        return True
    for t in low:
        attn[:, cfg.cls + t] += np.float32((thr + 1.3 * margin - s[t]) * 1.02)
    attn[:] = round_to_dtype(attn, cfg.dtype)
    return False


def plant_stage1_scores(cfg: VScanConfig, attn_g: np.ndarray, attn_l: np.ndarray,
                        margin: float = DEFAULT_MARGIN, max_rounds: int = 50):
    """In place.  Local tensor first (per window), then the global tensor over the complement."""
    wins = _windows(cfg)
    for b in range(attn_g.shape[0]):
        for _ in range(max_rounds):
            if all([_lift(attn_l[b], cfg, m, cfg.k_w, margin) for m in wins]):
                break
        else:
            raise RuntimeError("local margins did not settle")
        s_l = vo.score_row(attn_l[b], cfg.cls)
        local = np.concatenate([vo.topk_lowest_index(s_l, cfg.k_w, m) for m in wins]) \
            if cfg.k_w else np.zeros(0, dtype=np.int64)
        rest = np.setdiff1d(np.arange(cfg.N), local)
        for _ in range(max_rounds):
            if _lift(attn_g[b], cfg, rest, cfg.k_g, margin):
                break
        else:
            raise RuntimeError("global margins did not settle")
    return attn_g, attn_l


def cosine_gaps(x_inst: np.ndarray, cls: int, kept: np.ndarray):
    """(unselected token ids, best-minus-second-best cosine per unselected token)."""
    N = x_inst.shape[0] - cls
    mask = np.ones(N, dtype=bool)
    mask[kept] = False
    unsel = np.nonzero(mask)[0]
    if kept.size < 2 or unsel.size == 0:
        return unsel, np.full(unsel.size, np.inf)
    x = x_inst.astype(np.float64)
    cos = vo.cosine_matrix(x[cls + unsel], x[cls + kept])
    part = np.partition(cos, cos.shape[1] - 2, axis=1)
    return unsel, part[:, -1] - part[:, -2]


def plant_merge(cfg: VScanConfig, x: np.ndarray, kept_idx: np.ndarray, seed: int = 0,
                margin: float = DEFAULT_MARGIN, max_attempts: int = 64):
    """In place: re-draw the noise of every unselected token whose two best cosines are closer
    than `margin`."""
    for b in range(x.shape[0]):
        kept = np.asarray(kept_idx[b], dtype=np.int64)
        xs = x[b].astype(np.float64)[cfg.cls + kept]
        unsel, gaps = cosine_gaps(x[b], cfg.cls, kept)
        for u in unsel[gaps <= margin]:
            for attempt in range(max_attempts):
                x[b, cfg.cls + u] = redraw_token(cfg, seed, b, cfg.cls + int(u), x[b], attempt)
                c = vo.cosine_matrix(x[b, cfg.cls + u].astype(np.float64)[None, :], xs)[0]
                c.sort()
                if c[-1] - c[-2] > margin:
                    break
            else:
                raise RuntimeError("merge margin did not settle")
    return x


def plant_stage2(cfg: VScanConfig, q_last: np.ndarray, k: np.ndarray, scale: float,
                 softmax_span: int = vo.SPAN_ONLY, margin: float = DEFAULT_MARGIN,
                 n_vis: int | None = None, k_keep: int | None = None):
    """In place: push the keys of the oracle's top-k set along the mean query direction of their
    KV group until the k-boundary gap exceeds `margin`."""
    n_vis = cfg.n_vis if n_vis is None else n_vis
    k_keep = cfg.k2 if k_keep is None else k_keep
    if k_keep <= 0 or k_keep >= n_vis:
        return k
    rep = cfg.Hq // cfg.Hkv
    for b in range(q_last.shape[0]):
        s = vo.score_qk(q_last[b], k[b], cfg.n_sys, n_vis, scale, softmax_span)
        if vo.topk_boundary_gap(s, k_keep) > margin:
            continue
        top = vo.topk_lowest_index(s, k_keep)
        base = k[b].copy()
        beta = 0.25
        for _ in range(12):
            k[b] = base
            for g in range(cfg.Hkv):
                m = q_last[b, g * rep:(g + 1) * rep].astype(np.float64).mean(axis=0)
                m /= max(np.linalg.norm(m), 1e-12)
                k[b, g, cfg.n_sys + top] = base[g, cfg.n_sys + top] + np.float32(beta) * m.astype(np.float32)
            k[b] = round_to_dtype(k[b], cfg.dtype)
            s = vo.score_qk(q_last[b], k[b], cfg.n_sys, n_vis, scale, softmax_span)
            if vo.topk_boundary_gap(s, k_keep) > margin:
                break
            beta *= 2
        else:
            raise RuntimeError("stage-2 margin did not settle")
    return k
