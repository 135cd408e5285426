"""Stage 1 -> Stage 2 parity at the full sizes of the named workloads, in the launch
configuration the benchmark times (VScanReducer, preallocated buffers, one stream).

Kept indices and assignments must match the oracle bit for bit (margins are planted), floating
point outputs within the stated max-abs bars.  Where a batch is too large to generate and check on
the host (the 256- and 512-image sweep points) a small generated batch is tiled on the device to the
full launch size and the oracle checks sampled images of it.
"""
import numpy as np
import pytest
import torch

import paper_2505_22654_b200 as vs
from synth import CONFIGS, sweep_config

from helpers import TOL_SCORE, check_merged, dev, stage1_case, stage2_case

pytestmark = pytest.mark.gpu


def run_and_check(cfg, gen_instances=None, gen_batch=None, sample=None):
    """gen_*: how many distinct instances / sequences to generate (tiled up to the config's size)."""
    n_inst = cfg.instances if gen_instances is None else gen_instances
    n_seq = cfg.B if gen_batch is None else gen_batch
    s1 = stage1_case(cfg, instances=n_inst)
    s2 = stage2_case(cfg, batch=n_seq)

    def tile(a, total, axis=0):
        reps = -(-total // a.shape[axis])
        idx = [slice(None)] * a.dim()
        out = torch.cat([a] * reps, dim=axis)
        idx[axis] = slice(0, total)
        return out[tuple(idx)].contiguous()

    dt = cfg.dtype
    attn_g, attn_l, x = (tile(dev(s1[n], dt), cfg.instances) for n in ("attn_g", "attn_l", "x"))
    q, k, v, h = (tile(dev(s2[n], dt), cfg.B) for n in ("q_last", "k", "v", "hidden"))
    pos = tile(dev(s2["pos_ids"]), cfg.B, axis=1)
    red = vs.VScanReducer.from_config(cfg)
    red.run(attn_g, attn_l, x, q, k, v, h, pos)
    torch.cuda.synchronize()

    inst_ids = range(cfg.instances) if sample is None else sample(cfg.instances)
    sg, sl = red.scores_g.cpu().numpy(), red.scores_l.cpu().numpy()
    kept = red.kept_idx.cpu().numpy()
    for i in inst_ids:
        j = i % n_inst
        assert np.abs(sg[i] - s1["scores_g"][j]).max() <= TOL_SCORE
        assert np.abs(sl[i] - s1["scores_l"][j]).max() <= TOL_SCORE
        np.testing.assert_array_equal(kept[i], s1["kept"][j])
        check_merged(red.merged[i], s1["merged"][j], dt)
    # properties that hold at any size, checked on every instance
    assert kept.shape == (cfg.instances, cfg.K1)
    assert np.all(np.diff(kept, axis=1) > 0) and kept.min() >= 0 and kept.max() < cfg.N

    o = s2["oracle"]
    seq_ids = range(cfg.B) if sample is None else sample(cfg.B)
    kv = red.out2["kept_vis"].cpu().numpy()
    assert np.all(np.diff(kv, axis=1) > 0)
    for b in seq_ids:
        j = b % n_seq
        np.testing.assert_array_equal(kv[b], o["kept_vis"][j])
        for name in ("hidden", "k", "v"):
            np.testing.assert_array_equal(red.out2[name][b].float().cpu().numpy(), o[name][j])
        np.testing.assert_array_equal(red.out2["pos"][:, b].cpu().numpy(), o["pos"][:, j])
    return red


def test_config0_llava15_b1_fp32():
    run_and_check(CONFIGS[0])


def test_config1_llava15_b256_bf16():
    run_and_check(CONFIGS[1])


def test_config2_llavanext_b32_bf16():
    red = run_and_check(CONFIGS[2])
    # assignments and group sizes too, through the optional outputs
    cfg = CONFIGS[2]
    s1 = stage1_case(cfg, instances=10)
    merged, assign, counts = vs.vscan_merge(dev(s1["x"], "bf16"), cfg.cls, dev(s1["kept"].astype(np.int32)),
                                            want_assign=True, want_counts=True)
    np.testing.assert_array_equal(assign.cpu().numpy(), s1["assign"])
    np.testing.assert_array_equal(counts.cpu().numpy(), s1["counts"])
    assert int(counts.sum(dim=1).min()) == cfg.N == int(counts.sum(dim=1).max())
    # each output token times its group size sums to the token sum of the instance (Eq. 4)
    lhs = (merged.double() * counts.double()[..., None]).sum(1).cpu().numpy()
    rhs = s1["x"][:, cfg.cls:].astype(np.float64).sum(1)
    assert np.abs(lhs - rhs).max() <= 0.02 * cfg.N ** 0.5 * 8


def test_config3_long_frames_b4_bf16():
    run_and_check(CONFIGS[3])


@pytest.mark.parametrize("retention", ["25%", "11.1%", "5.5%"])
def test_config4_sweep_b8(retention):
    run_and_check(sweep_config(8, retention))


@pytest.mark.parametrize("batch,retention", [(1, "11.1%"), (64, "25%"), (256, "5.5%"), (512, "11.1%")])
def test_config4_sweep_batches(batch, retention):
    cfg = sweep_config(batch, retention)
    g = min(batch, 4)
    run_and_check(cfg, gen_instances=g * cfg.C, gen_batch=g,
                  sample=lambda n: sorted(set(np.linspace(0, n - 1, 9).astype(int).tolist())))


def test_host_stream_of_batches_matches_device_runs():
    """run_host_many overlaps uploads, passes and downloads of neighbouring batches; every batch's
    results must equal those of a plain device-resident run on the same inputs."""
    cfg = CONFIGS[2].with_(name="host_stream", B=3, C=2, k2=64)
    red = vs.VScanReducer.from_config(cfg)
    batches = []
    for seed in range(4):
        s1, s2 = stage1_case(cfg, seed=seed, planted=False), stage2_case(cfg, seed=seed, planted=False)
        batches.append({"attn_g": dev(s1["attn_g"], cfg.dtype), "attn_l": dev(s1["attn_l"], cfg.dtype),
                        "x": dev(s1["x"], cfg.dtype), "q_last": dev(s2["q_last"], cfg.dtype), "k": dev(s2["k"], cfg.dtype),
                        "v": dev(s2["v"], cfg.dtype), "hidden": dev(s2["hidden"], cfg.dtype), "pos_ids": dev(s2["pos_ids"])})
    expect = []
    for d in batches:
        red.run(**d)
        torch.cuda.synchronize()
        expect.append({"merged": red.merged.cpu().clone(), **{k: red.out2[k].cpu().clone() for k in ("kept_vis", "hidden", "k", "v", "pos")}})
    host_ins = [{k: v.cpu().pin_memory() for k, v in d.items()} for d in batches]
    host_outs = [{k: torch.empty_like(v).pin_memory() for k, v in e.items()} for e in expect]
    slots = [{k: torch.empty_like(v) for k, v in batches[0].items()} for _ in range(2)]
    red.run_host_many(host_ins, host_outs, slots)
    torch.cuda.synchronize()
    for got, ref in zip(host_outs, expect):
        for name in ref:
            assert torch.equal(got[name], ref[name]), name
