"""Generator properties (determinism, dtype representability, prefix stability) and the margin
planting that the parity tests rely on."""
import numpy as np
import torch

from oracle import plant
from oracle import vscan_oracle as vo
from synth import CONFIGS, stage1_inputs, stage2_inputs, sweep_config, tiny_config


def _small(dtype="bf16"):
    # 12x12 grid, 4 windows of 6x6: same structure as the LLaVA shapes, small enough for CPU.
    return CONFIGS[2].with_(name="small", B=2, C=2, grid_h=12, grid_w=12, D=64, H=4, k_w=2, k_g=8,
                            n_clusters=8, n_txt=8, Dh=64, Hq=8, Hkv=4, d=32, k2=16, dtype=dtype)


def test_config_shapes_match_workloads():
    c0, c1, c2, c3 = (CONFIGS[i] for i in range(4))
    assert (c0.N, c0.L, c0.W, c0.K1, c0.S, c0.S_out) == (576, 577, 16, 64, 139, 107)
    assert (c1.K1, c1.n_vis, c1.S, c1.S_out) == (192, 192, 291, 195)
    assert (c2.K1, c2.n_vis, c2.S, c2.S_out, c2.instances) == (64, 320, 419, 259, 160)
    assert (c3.N, c3.W, c3.K1, c3.S, c3.S_out) == (16384, 256, 2048, 2176, 1152)
    s = sweep_config(8, "25%")
    assert (s.K1, s.n_vis, s.k2) == (144, 720, 360)
    assert sweep_config(1, "5.5%").K1 == 32


def test_generator_is_seeded_and_prefix_stable():
    cfg = _small()
    a = stage1_inputs(cfg, seed=0)
    b = stage1_inputs(cfg, seed=0, instances=2)
    c = stage1_inputs(cfg, seed=1, instances=2)
    for name in ("x", "attn_g", "attn_l"):
        np.testing.assert_array_equal(a[name][:2], b[name])
        assert not np.array_equal(b[name], c[name])
    assert a["x"].shape == (4, cfg.L, cfg.D) and a["attn_g"].shape == (4, cfg.H, cfg.L)
    s2 = stage2_inputs(cfg)
    assert s2["k"].shape == (cfg.B, cfg.Hkv, cfg.S, cfg.d) and s2["pos_ids"].shape == (1, cfg.B, cfg.S)


def test_generated_values_are_representable_in_io_dtype():
    cfg = _small("bf16")
    d = stage1_inputs(cfg, instances=1)
    for name in ("x", "attn_g", "attn_l"):
        t = torch.from_numpy(d[name])
        assert torch.equal(t.to(torch.bfloat16).to(torch.float32), t)
    assert np.abs(d["x"]).max() < 8
    np.testing.assert_allclose(d["attn_g"].sum(-1), 1.0, atol=2e-2)   # probabilities (bf16-rounded)


def test_planted_margins_hold():
    cfg = _small("bf16")
    s1 = stage1_inputs(cfg)
    plant.plant_stage1_scores(cfg, s1["attn_g"], s1["attn_l"])
    kept_all = []
    for b in range(cfg.instances):
        s_g = vo.score_row(s1["attn_g"][b], cfg.cls)
        s_l = vo.score_row(s1["attn_l"][b], cfg.cls)
        kept, local, glob = vo.select_global_local(s_g, s_l, cfg.frames, cfg.grid_h, cfg.grid_w,
                                                   cfg.win_h, cfg.win_w, cfg.k_w, cfg.k_g)
        for members in plant._windows(cfg):
            assert vo.topk_boundary_gap(s_l, cfg.k_w, members) > 1e-4
        rest = np.setdiff1d(np.arange(cfg.N), local)
        assert vo.topk_boundary_gap(s_g, cfg.k_g, rest) > 1e-4
        kept_all.append(kept)
    kept_all = np.stack(kept_all)
    plant.plant_merge(cfg, s1["x"], kept_all)
    for b in range(cfg.instances):
        _, gaps = plant.cosine_gaps(s1["x"][b], cfg.cls, kept_all[b])
        assert gaps.min() > 1e-4
    t = torch.from_numpy(s1["x"])
    assert torch.equal(t.to(torch.bfloat16).to(torch.float32), t)
    s2 = stage2_inputs(cfg)
    plant.plant_stage2(cfg, s2["q_last"], s2["k"], s2["scale"])
    for b in range(cfg.B):
        s = vo.score_qk(s2["q_last"][b], s2["k"][b], cfg.n_sys, cfg.n_vis, s2["scale"])
        assert vo.topk_boundary_gap(s, cfg.k2) > 1e-4


def test_tiny_config_is_consistent():
    t = tiny_config()
    assert t.N == 24 and t.W == 4 and t.K1 == 7 and t.n_vis == 14


def test_schedule_points_follow_the_printed_settings():
    """Table 1's (k, R2) pairs average 75 % of the Stage-1 set over 32 layers (App. B.1's rule), the
    Table 6(a) pairs all average 11.1 %, and every schedule point is a legal call."""
    from oracle import budget
    from synth import schedule_points
    from synth.configs import TABLE1_SETTINGS
    for k, r2 in TABLE1_SETTINGS:
        assert abs(budget.average_retention(1.0, r2 / 100, k, 32) - 0.75) < 1e-3
    pts = schedule_points()
    assert len(pts) == 12 + 5 + 5 + 1
    for label, cfg, s1 in pts:
        assert 0 <= cfg.k2 <= cfg.n_vis and cfg.k_w <= cfg.win_h * cfg.win_w and 0 <= cfg.k_g <= cfg.N - cfg.W * cfg.k_w
        if label.startswith("table6a"):
            assert abs(budget.average_tokens(cfg.K1, cfg.k2 // cfg.C, 16, 32) / cfg.N - 0.111) < 2e-3
        if label.startswith("table6b"):
            assert cfg.K1 == 96
        if not s1:
            assert cfg.n_vis == cfg.C * cfg.N
