"""Shared pieces of the GPU parity tests: planted inputs, the oracle run over a batch, casts."""
from __future__ import annotations

import numpy as np
import torch

from oracle import plant
from oracle import vscan_oracle as vo
from synth import stage1_inputs, stage2_inputs

TOL_MERGED = {"f32": 1e-4, "bf16": 2e-2}     # max-abs bar on floating-point outputs
TOL_SCORE = 2e-6                               # fp32 head means of probabilities (values <= 1)


def torch_dtype(name):
    return torch.float32 if name == "f32" else torch.bfloat16


def dev(a: np.ndarray, dtype: str | None = None):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(torch_dtype(dtype)) if dtype is not None else t


def stage1_case(cfg, seed=0, instances=None, planted=True):
    """Inputs (numpy, representable in cfg.dtype) and the oracle's results for every instance."""
    n = cfg.instances if instances is None else instances
    d = stage1_inputs(cfg, seed, n)
    if planted:
        plant.plant_stage1_scores(cfg, d["attn_g"], d["attn_l"])
    sg = np.stack([vo.score_row(d["attn_g"][b], cfg.cls) for b in range(n)])
    sl = np.stack([vo.score_row(d["attn_l"][b], cfg.cls) for b in range(n)])
    kept = np.stack([vo.select_global_local(sg[b], sl[b], cfg.frames, cfg.grid_h, cfg.grid_w, cfg.win_h,
                                            cfg.win_w, cfg.k_w, cfg.k_g)[0] for b in range(n)])
    if planted:
        plant.plant_merge(cfg, d["x"], kept, seed)
    merged, assign, counts = [], [], []
    for b in range(n):
        m, a, c = vo.merge(d["x"][b], cfg.cls, kept[b])
        merged.append(m); assign.append(a); counts.append(c)
    d.update(scores_g=sg, scores_l=sl, kept=kept, merged=np.stack(merged), assign=np.stack(assign),
             counts=np.stack(counts))
    return d


def stage2_case(cfg, seed=0, batch=None, planted=True, softmax_span=vo.SPAN_ONLY):
    n = cfg.B if batch is None else batch
    d = stage2_inputs(cfg, seed, n)
    if planted:
        plant.plant_stage2(cfg, d["q_last"], d["k"], d["scale"], softmax_span)
    outs = [vo.llm_prune(d["q_last"][b], d["k"][b], d["v"][b], d["hidden"][b], d["pos_ids"][:, b], cfg.n_sys,
                         cfg.n_vis, cfg.n_txt, cfg.k2, d["scale"], softmax_span) for b in range(n)]
    d["oracle"] = {
        "scores": np.stack([o["scores"] for o in outs]),
        "kept_vis": np.stack([o["kept_vis"] for o in outs]),
        "hidden": np.stack([o["hidden"] for o in outs]),
        "k": np.stack([o["k"] for o in outs]),
        "v": np.stack([o["v"] for o in outs]),
        "pos": np.stack([o["pos"] for o in outs], axis=1),
    }
    return d


def bf16_half_ulp(ref: np.ndarray) -> np.ndarray:
    """Half a bf16 unit in the last place at the magnitude of `ref` (8 significand bits)."""
    mag = np.maximum(np.abs(ref), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(mag)) - 8)


def check_merged(got: torch.Tensor, ref: np.ndarray, dtype: str):
    g = got.float().cpu().numpy().astype(np.float64)
    err = np.abs(g - ref)
    assert err.max() <= TOL_MERGED[dtype], f"max-abs {err.max()}"
    if dtype == "bf16":
        # one rounding of an fp32 mean: within half a bf16 ulp of the exact mean (+ fp32 slack)
        assert np.all(err <= bf16_half_ulp(ref) * 1.02 + 2e-5), float((err - bf16_half_ulp(ref)).max())
    return float(err.max())


# ------------------------------------------------------------------ inputs without planted margins
NEAR_TIE = 1e-4     # a decision whose fp64 margin is below this may fall either way on the GPU


def check_topk_unplanted(got, scores, k, candidates=None) -> int:
    """Exact top-k on scores that were not margin-planted.  `got` (ascending indices) must have exactly k
    distinct candidates; it may differ from the oracle's set only by tokens whose fp64 score lies within
    NEAR_TIE of the oracle's k-th largest, everything else must be the oracle's choice.  Returns the
    number of tokens in which the two sets differ."""
    s = np.asarray(scores, dtype=np.float64)
    cand = np.arange(s.shape[0]) if candidates is None else np.asarray(candidates)
    ref = vo.topk_lowest_index(s, k, cand)
    got = np.asarray(got, dtype=np.int64)
    assert got.shape == ref.shape and np.all(np.diff(got) > 0) and np.isin(got, cand).all()
    diff = np.setxor1d(got, ref)
    if diff.size:
        kth = np.sort(s[cand])[::-1][k - 1]
        assert np.all(np.abs(s[diff] - kth) < NEAR_TIE), (diff, s[diff], kth)
    return int(diff.size)


def check_merge_unplanted(x, cls, kept, merged, assign, counts, dtype) -> int:
    """Merge results on features that were not margin-planted.  A token's assignment may differ from the
    oracle's only where the oracle's best and second-best cosine are closer than NEAR_TIE, and then only
    to a slot whose cosine is within NEAR_TIE of the best; every other assignment is the oracle's.
    Counts and merged rows are then checked against Eq. 4 evaluated on the assignment the GPU took.
    Returns the number of assignments that differ."""
    x64 = np.asarray(x, dtype=np.float64)
    kept = np.asarray(kept, dtype=np.int64)
    _, a_ref, _ = vo.merge(x64, cls, kept)
    a = assign.cpu().numpy().astype(np.int64)
    np.testing.assert_array_equal(a[kept], np.arange(kept.size))
    differ = np.nonzero(a != a_ref)[0]
    if differ.size:
        cos = vo.cosine_matrix(x64[cls + differ], x64[cls + kept])
        best = cos.max(axis=1)
        taken = cos[np.arange(differ.size), a[differ]]
        assert np.all(best - taken < NEAR_TIE), (differ, best - taken)
    m_ref, c_ref = vo.mean_merge(x64, cls, kept, a)
    np.testing.assert_array_equal(counts.cpu().numpy(), c_ref)
    check_merged(merged, m_ref, dtype)
    return int(differ.size)
