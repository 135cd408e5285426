"""Ragged batches: instances and sequences of different sizes in one library call (dynamic-resolution encoders,
Sec. 5.1 "Models": 4 to 16384 visual tokens per image).  Every unit's result is compared with the oracle run on
that unit alone, bit for bit where the result is an index or a copy."""
import numpy as np
import pytest
import torch

import paper_2505_22654_b200 as vs
from oracle import plant
from oracle import vscan_oracle as vo
from synth import CONFIGS, round_to_dtype

from helpers import check_merged, dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_stage1_mixed_sizes_in_one_call(dtype):
    rng = np.random.default_rng(21)
    H, D, c, wh, ww = 4, 128, 1, 2, 2
    # (frames, grid_h, grid_w), k_per_window, k_global: 4 tokens up to 16384; three equal neighbours form one run
    units = [((1, 2, 2), 1, 1), ((1, 24, 24), 1, 20), ((1, 24, 24), 1, 20), ((1, 24, 24), 1, 20), ((1, 12, 18), 0, 37),
             ((16, 32, 32), 0, 96), ((1, 6, 10), 2, 0), ((1, 24, 24), 0, 64)]
    ag, al, xs, kept_ref = [], [], [], []
    for (F, gh, gw), kw, kg in units:
        N = F * gh * gw
        cfg = CONFIGS[2].with_(name="ragged", config_id=60, dtype=dtype, frames=F, grid_h=gh, grid_w=gw, cls=c, D=D, H=H,
                               win_h=wh, win_w=ww, k_w=kw, k_g=kg, B=1, C=1)
        a_g = round_to_dtype(rng.random((1, H, N + c)).astype(np.float32) / N, dtype)
        a_l = round_to_dtype(rng.random((1, H, N + c)).astype(np.float32) / N, dtype)
        plant.plant_stage1_scores(cfg, a_g, a_l)
        x = round_to_dtype(rng.standard_normal((1, N + c, D)).astype(np.float32), dtype)
        kept = vo.select_global_local(vo.score_row(a_g[0], c), vo.score_row(a_l[0], c), F, gh, gw, wh, ww, kw, kg)[0]
        plant.plant_merge(cfg, x, kept[None, :])
        ag.append(a_g[0]); al.append(a_l[0]); xs.append(x[0]); kept_ref.append(kept)
    kept_v, merged_v, ws = vs.vscan_stage1_ragged([dev(a, dtype) for a in ag], [dev(a, dtype) for a in al],
                                                  [dev(x, dtype) for x in xs], c, [u[0] for u in units], wh, ww,
                                                  [u[1] for u in units], [u[2] for u in units])
    assert vs.vscan_check(ws) == 0
    for i in range(len(units)):
        np.testing.assert_array_equal(kept_v[i].cpu().numpy(), kept_ref[i])
        m, _, _ = vo.merge(xs[i], c, kept_ref[i])
        check_merged(merged_v[i], m, dtype)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_llm_prune_mixed_lengths_in_one_call(dtype):
    rng = np.random.default_rng(22)
    Hq, Hkv, d, Dh = 8, 2, 64, 96
    # n_sys, n_vis, n_txt, k_keep per sequence: equal neighbours form one run; an empty survivor list is legal
    seqs = [(3, 4, 5, 2), (35, 320, 64, 160), (35, 320, 64, 160), (0, 1000, 7, 333), (2, 50, 0, 0), (5, 64, 9, 64)]
    B = len(seqs)
    scale = float(d ** -0.5)
    q = round_to_dtype(rng.standard_normal((B, Hq, d)).astype(np.float32), dtype)
    ks, vs_, hs, ps, refs = [], [], [], [], []
    cfg = CONFIGS[2].with_(name="ragged2", config_id=61, dtype=dtype, Hq=Hq, Hkv=Hkv, d=d, Dh=Dh)
    for b, (ns, nv, nt, kk) in enumerate(seqs):
        S = ns + nv + nt
        k = round_to_dtype(rng.standard_normal((1, Hkv, S, d)).astype(np.float32), dtype)
        v = round_to_dtype(rng.standard_normal((Hkv, S, d)).astype(np.float32), dtype)
        h = round_to_dtype(rng.standard_normal((S, Dh)).astype(np.float32), dtype)
        pos = (np.arange(S, dtype=np.int32) * 3 + b)
        plant.plant_stage2(cfg.with_(n_sys=ns), q[b:b + 1], k, scale, vo.SPAN_ONLY, n_vis=nv, k_keep=kk)
        ks.append(k[0]); vs_.append(v); hs.append(h); ps.append(pos)
        refs.append(vo.llm_prune(q[b], k[0], v, h, pos[None, :], ns, nv, nt, kk, scale))
    outs, ws = vs.vscan_llm_prune_ragged(dev(q, dtype), [dev(k, dtype) for k in ks], [dev(v, dtype) for v in vs_],
                                         [dev(h, dtype) for h in hs], [dev(p) for p in ps], [s[0] for s in seqs],
                                         [s[1] for s in seqs], [s[2] for s in seqs], [s[3] for s in seqs], scale)
    assert vs.vscan_check(ws) == 0
    for b in range(B):
        r, o = refs[b], outs[b]
        np.testing.assert_array_equal(o["kept_vis"].cpu().numpy(), r["kept_vis"])
        np.testing.assert_array_equal(o["hidden"].float().cpu().numpy(), r["hidden"])
        np.testing.assert_array_equal(o["k"].float().cpu().numpy(), r["k"])
        np.testing.assert_array_equal(o["v"].float().cpu().numpy(), r["v"])
        np.testing.assert_array_equal(o["pos"].cpu().numpy(), r["pos"][0])
