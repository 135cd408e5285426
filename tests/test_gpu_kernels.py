"""Per-call parity of the CUDA library against the CPU oracle on small and edge-case shapes
(several tiles plus ragged tails).  Everything goes through the C ABI via the ctypes binding."""
import numpy as np
import pytest
import torch

import paper_2505_22654_b200 as vs
from oracle import plant
from oracle import vscan_oracle as vo
from synth import CONFIGS, round_to_dtype

from helpers import TOL_SCORE, check_merge_unplanted, check_merged, dev, stage1_case, stage2_case

pytestmark = pytest.mark.gpu
RNG = np.random.default_rng(7)


def small_cfg(dtype, **kw):
    base = CONFIGS[2].with_(name="small", config_id=50, B=2, C=3, grid_h=12, grid_w=18, D=72, H=5, k_w=2,
                            k_g=9, n_clusters=6, n_sys=3, n_txt=5, Dh=72, Hq=6, Hkv=3, d=40, k2=17, dtype=dtype)
    return base.with_(**kw)


# ------------------------------------------------------------------ vscan_score, ROW mode
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,H,L,c", [(1, 1, 9, 1), (3, 16, 577, 1), (2, 7, 300, 0), (2, 3, 1031, 1)])
def test_score_row(dtype, B, H, L, c):
    attn = round_to_dtype(RNG.random((B, H, L)).astype(np.float32) / L, dtype)
    got = vs.vscan_score_row(dev(attn, dtype), c).cpu().numpy()
    ref = np.stack([vo.score_row(attn[b], c) for b in range(B)])
    assert got.shape == ref.shape
    assert np.abs(got - ref).max() <= TOL_SCORE


def test_score_row_partial_row_and_empty_batch():
    attn = RNG.random((2, 4, 50)).astype(np.float32)
    got = vs.vscan_score_row(dev(attn, "f32"), 2, n_tokens=40).cpu().numpy()
    ref = np.stack([vo.score_row(attn[b][:, :42], 2) for b in range(2)])
    assert np.abs(got - ref).max() <= 1e-6
    empty = torch.empty((0, 4, 50), device="cuda")
    assert vs.vscan_score_row(empty, 1).shape == (0, 49)


# ------------------------------------------------------------------ vscan_select_global_local
SELECT_SHAPES = [  # F, Gh, Gw, wh, ww, k_w, k_g
    (1, 24, 24, 6, 6, 2, 32), (1, 24, 24, 6, 6, 6, 96), (1, 24, 24, 6, 6, 0, 64), (1, 24, 24, 6, 6, 3, 0),
    (1, 24, 24, 24, 24, 10, 5), (2, 4, 6, 2, 3, 1, 3), (1, 1, 1, 1, 1, 1, 0), (1, 5, 7, 1, 1, 0, 35),
    (3, 10, 10, 5, 2, 4, 100), (16, 32, 32, 8, 8, 4, 1024), (1, 24, 24, 6, 6, 36, 0), (4, 16, 16, 16, 16, 37, 11),
    # above 2048 tokens a cluster of CTAs shares an instance: uneven band counts per CTA, windows above 64 tokens,
    # no local or no global scan, a global scan that takes everything left
    (5, 24, 24, 6, 6, 2, 300), (3, 30, 30, 10, 30, 0, 500), (1, 64, 48, 2, 48, 50, 0), (7, 20, 20, 4, 5, 1, 2000),
    (16, 32, 32, 32, 32, 9, 16240), (1, 128, 128, 64, 128, 3, 77),
]


@pytest.mark.parametrize("shape", SELECT_SHAPES)
@pytest.mark.parametrize("ties", [False, True])
def test_select_bit_exact(shape, ties):
    F, Gh, Gw, wh, ww, k_w, k_g = shape
    N, B = F * Gh * Gw, 3
    if ties:   # few distinct values, signed zeros and negatives: the tie rule decides nearly everything
        sg = RNG.integers(-2, 3, (B, N)).astype(np.float32) * 0.25
        sl = RNG.integers(0, 3, (B, N)).astype(np.float32) * 0.5
        sg[:, ::7] = -0.0
    else:
        sg = RNG.random((B, N)).astype(np.float32)
        sl = RNG.standard_normal((B, N)).astype(np.float32)
    got, mask = vs.vscan_select_global_local(dev(sg), dev(sl), F, Gh, Gw, wh, ww, k_w, k_g, want_mask=True)
    got, mask = got.cpu().numpy(), mask.cpu().numpy()
    for b in range(B):
        ref = vo.select_global_local(sg[b], sl[b], F, Gh, Gw, wh, ww, k_w, k_g)[0]
        np.testing.assert_array_equal(got[b], ref)
        m = np.zeros(N, dtype=np.uint8); m[ref] = 1
        np.testing.assert_array_equal(mask[b], m)


def test_select_uniform_scores_take_first_indices_and_aliasing():
    s = dev(np.full((2, 576), 0.125, dtype=np.float32))
    got = vs.vscan_select_global_local(s, s, 1, 24, 24, 6, 6, 2, 32).cpu().numpy()
    ref = vo.select_global_local(np.full(576, 0.125), np.full(576, 0.125), 1, 24, 24, 6, 6, 2, 32)[0]
    np.testing.assert_array_equal(got[0], ref); np.testing.assert_array_equal(got[1], ref)
    # window w starts at row 6*(w//4), column 6*(w%4): its first two tokens are kept
    assert {0, 1, 6, 7, 144, 145}.issubset(set(got[0].tolist()))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", [(1, 24, 24, 6, 6, 2, 32, 1, 16), (2, 6, 8, 3, 4, 5, 20, 0, 5),
                                   (1, 16, 16, 16, 16, 40, 9, 1, 3), (16, 32, 32, 8, 8, 4, 1024, 0, 16),
                                   (5, 24, 24, 6, 6, 2, 300, 1, 16), (3, 30, 30, 10, 30, 7, 500, 0, 5)])
def test_score_select_fused_matches_oracle(dtype, shape):
    F, Gh, Gw, wh, ww, k_w, k_g, c, H = shape
    N, B = F * Gh * Gw, 2
    cfg = small_cfg(dtype, frames=F, grid_h=Gh, grid_w=Gw, win_h=wh, win_w=ww, k_w=k_w, k_g=k_g, cls=c, H=H, C=1, B=B)
    ag = round_to_dtype(RNG.random((B, H, N + c)).astype(np.float32) / N, dtype)
    al = round_to_dtype(RNG.random((B, H, N + c)).astype(np.float32) / N, dtype)
    plant.plant_stage1_scores(cfg, ag, al)
    sg = torch.empty((B, N), dtype=torch.float32, device="cuda"); sl = torch.empty_like(sg)
    kept = vs.vscan_score_select(dev(ag, dtype), dev(al, dtype), c, F, Gh, Gw, wh, ww, k_w, k_g,
                                 scores_global=sg, scores_local=sl).cpu().numpy()
    for b in range(B):
        rg, rl = vo.score_row(ag[b], c), vo.score_row(al[b], c)
        assert np.abs(sg[b].cpu().numpy() - rg).max() <= TOL_SCORE and np.abs(sl[b].cpu().numpy() - rl).max() <= TOL_SCORE
        np.testing.assert_array_equal(kept[b], vo.select_global_local(rg, rl, F, Gh, Gw, wh, ww, k_w, k_g)[0])
    # same buffer for both scans, no score outputs: the decisions are taken on the kernel's own fp32
    # head means (returned above), so the oracle fed with exactly those values must agree bit for bit
    kept2 = vs.vscan_score_select(dev(ag, dtype), dev(ag, dtype), c, F, Gh, Gw, wh, ww, k_w, k_g).cpu().numpy()
    for b in range(B):
        g32 = sg[b].cpu().numpy()
        np.testing.assert_array_equal(kept2[b], vo.select_global_local(g32, g32, F, Gh, Gw, wh, ww, k_w, k_g)[0])


# ------------------------------------------------------------------ vscan_merge
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("path", ["simt", "auto"])
def test_merge_small_planted(dtype, path):
    cfg = small_cfg(dtype)
    case = stage1_case(cfg)
    x, kept = dev(case["x"], dtype), dev(case["kept"].astype(np.int32))
    merged, assign, counts = vs.vscan_merge(x, cfg.cls, kept, want_assign=True, want_counts=True,
                                            path=vs.MERGE_SIMT if path == "simt" else vs.MERGE_AUTO)
    np.testing.assert_array_equal(assign.cpu().numpy(), case["assign"])
    np.testing.assert_array_equal(counts.cpu().numpy(), case["counts"])
    check_merged(merged, case["merged"], dtype)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_merge_edge_shapes(dtype):
    D, L, c = 264, 131, 1
    N = L - c
    x = round_to_dtype(RNG.standard_normal((2, L, D)).astype(np.float32), dtype)
    xd = dev(x, dtype)
    # keep-all: identity, bit for bit
    kept_all = np.tile(np.arange(N, dtype=np.int32), (2, 1))
    merged, counts = vs.vscan_merge(xd, c, dev(kept_all), want_counts=True)
    assert torch.equal(merged, xd[:, c:]) and int(counts.min()) == 1 == int(counts.max())
    # a single kept token receives the mean of everything
    one = np.array([[5], [77]], dtype=np.int32)
    merged, assign, counts = vs.vscan_merge(xd, c, dev(one), want_assign=True, want_counts=True)
    assert int(assign.abs().max()) == 0 and counts.flatten().tolist() == [N, N]
    ref = x[:, c:].astype(np.float64).mean(axis=1, keepdims=True)
    check_merged(merged, ref, dtype)
    # ragged kept count (not a multiple of the tile) with margins planted
    cfg = small_cfg(dtype, grid_h=10, grid_w=13, win_h=10, win_w=13, k_w=0, k_g=67, D=264, C=1, B=2)
    x2 = round_to_dtype(RNG.standard_normal((2, cfg.L, D)).astype(np.float32), dtype)
    kept = np.stack([np.sort(RNG.choice(cfg.N, 67, replace=False)) for _ in range(2)])
    plant.plant_merge(cfg, x2, kept)
    merged, assign, counts = vs.vscan_merge(dev(x2, dtype), cfg.cls, dev(kept.astype(np.int32)),
                                            want_assign=True, want_counts=True)
    for b in range(2):
        m, a, cn = vo.merge(x2[b], cfg.cls, kept[b])
        np.testing.assert_array_equal(assign[b].cpu().numpy(), a)
        np.testing.assert_array_equal(counts[b].cpu().numpy(), cn)
        check_merged(merged[b], m, dtype)


def test_merge_exact_ties_and_duplicates():
    # identical tokens: every cosine ties at 1 -> lowest slot; kept duplicates keep their own slot
    x = np.tile(RNG.standard_normal((1, 1, 16)).astype(np.float32), (1, 40, 1))
    kept = np.array([[3, 10, 25]], dtype=np.int32)
    merged, assign, counts = vs.vscan_merge(dev(x, "f32"), 0, dev(kept), want_assign=True, want_counts=True)
    ref_m, ref_a, ref_c = vo.merge(x[0], 0, kept[0])
    np.testing.assert_array_equal(assign[0].cpu().numpy(), ref_a)
    assert counts[0].tolist() == ref_c.tolist() == [38, 1, 1]
    # a zero vector has cosine 0 with everything -> slot 0
    x2 = RNG.standard_normal((1, 12, 8)).astype(np.float32); x2[0, 4] = 0
    kept2 = np.array([[1, 7]], dtype=np.int32)
    _, a2 = vs.vscan_merge(dev(x2, "f32"), 0, dev(kept2), want_assign=True)
    np.testing.assert_array_equal(a2[0].cpu().numpy(), vo.merge(x2[0], 0, kept2[0])[1])
    assert int(a2[0, 4]) == 0


@pytest.mark.parametrize("N,D,K1,c", [(576, 1024, 64, 1), (576, 1024, 192, 1), (300, 72, 17, 0), (130, 264, 130, 1),
                                      (1000, 1280, 300, 0), (128, 64, 1, 1), (129, 128, 16, 0),
                                      (1500, 256, 800, 1), (1300, 128, 1100, 0)])
@pytest.mark.parametrize("path", ["tensor", "interleaved"])
def test_merge_tensor_path_matches_oracle(N, D, K1, c, path):
    """The tcgen05 path on its own (path = TENSOR): tile tails, kept counts that are not multiples of
    16, more than 256 kept tokens (several accumulator rounds on CTA pairs), more than 768 (the kept set scanned in
    two shares whose results are combined by whichever finishes last), feature dims that are not multiples of 64."""
    cfg = small_cfg("bf16", grid_h=1, grid_w=N, win_h=1, win_w=N, k_w=0, k_g=K1, D=D, C=1, B=2, cls=c)
    x = round_to_dtype(RNG.standard_normal((2, N + c, D)).astype(np.float32), "bf16")
    kept = np.stack([np.sort(RNG.choice(N, K1, replace=False)) for _ in range(2)])
    plant.plant_merge(cfg, x, kept)
    if path == "interleaved" and K1 > 256:
        with pytest.raises(vs.VScanError) as e:
            vs.vscan_merge(dev(x, "bf16"), c, dev(kept.astype(np.int32)), path=vs.MERGE_INTERLEAVED)
        assert e.value.status == 2       # more kept tokens than one accumulator holds: not this path
        return
    ws = vs.Workspace(8 << 20)
    merged, assign, counts = vs.vscan_merge(dev(x, "bf16"), c, dev(kept.astype(np.int32)), want_assign=True,
                                            want_counts=True, workspace=ws,
                                            path={"tensor": vs.MERGE_TENSOR, "interleaved": vs.MERGE_INTERLEAVED}[path])
    assert vs.vscan_check(ws) == 0
    for b in range(2):
        m, a, cn = vo.merge(x[b], c, kept[b])
        np.testing.assert_array_equal(assign[b].cpu().numpy(), a)
        np.testing.assert_array_equal(counts[b].cpu().numpy(), cn)
        check_merged(merged[b], m, "bf16")


@pytest.mark.parametrize("B,N,D,K1,c", [(2, 576, 1024, 64, 1), (3, 300, 512, 17, 0), (2, 130, 256, 40, 1), (1, 1000, 1024, 33, 0),
                                        (170, 576, 1024, 64, 1), (90, 200, 512, 9, 1)])
def test_merge_one_pass_cluster_path(B, N, D, K1, c):
    """The one-pass merge (a cluster of D / 256 CTAs per instance exchanging partial dot products through distributed
    shared memory): cluster sizes 1, 2 and 4, ragged last tiles, kept counts that are not multiples of 16, and more
    instances than clusters fit on the GPU at once (persistent loop, buffer rotation across instances)."""
    cfg = small_cfg("bf16", grid_h=1, grid_w=N, win_h=1, win_w=N, k_w=0, k_g=K1, D=D, C=1, B=B, cls=c)
    rng = np.random.default_rng(B * 7 + N)
    x = round_to_dtype(rng.standard_normal((B, N + c, D)).astype(np.float32), "bf16")
    kept = np.stack([np.sort(rng.choice(N, K1, replace=False)) for _ in range(B)])
    check = range(B) if B <= 3 else (0, 1, B // 2, B - 2, B - 1)
    for b in check:
        plant.plant_merge(cfg, x[b:b + 1], kept[b:b + 1])
    ws = vs.Workspace(64 << 20)
    merged, assign, counts = vs.vscan_merge(dev(x, "bf16"), c, dev(kept.astype(np.int32)), want_assign=True,
                                            want_counts=True, workspace=ws, path=vs.MERGE_CLUSTER)
    assert vs.vscan_check(ws) == 0
    for b in check:
        m, a, cn = vo.merge(x[b], c, kept[b])
        np.testing.assert_array_equal(assign[b].cpu().numpy(), a)
        np.testing.assert_array_equal(counts[b].cpu().numpy(), cn)
        check_merged(merged[b], m, "bf16")


@pytest.mark.parametrize("B,N,D,K1", [(150, 200, 64, 20), (97, 131, 128, 7), (40, 576, 1024, 64)])
def test_merge_interleaved_many_instances(B, N, D, K1):
    """More instances than the block-order distance between an instance's assignment CTAs and its mean
    CTAs (head, steady part and tail of the block order all occur); two calls on one workspace (the
    counters are cleared by every call); same result as the two-kernel tensor path, checked against
    the oracle on sampled instances."""
    rng = np.random.default_rng(B * 1000 + N)
    x = round_to_dtype(rng.standard_normal((B, N, D)).astype(np.float32), "bf16")
    kept = np.stack([np.sort(rng.choice(N, K1, replace=False)) for _ in range(B)]).astype(np.int32)
    xd, kd = dev(x, "bf16"), dev(kept)
    ws = vs.Workspace(8 << 20)
    ref = vs.vscan_merge(xd, 0, kd, want_assign=True, want_counts=True, path=vs.MERGE_TENSOR)
    for _ in range(2):
        out = vs.vscan_merge(xd, 0, kd, want_assign=True, want_counts=True, workspace=ws, path=vs.MERGE_INTERLEAVED)
        assert vs.vscan_check(ws) == 0
        same = (ref[1] == out[1]).all(dim=1)      # (the two paths round the kept-row norms in different orders:
        assert same.float().mean() > 0.9          #  a near-tie may fall the other way)
        assert (ref[1] == out[1]).float().mean() > 0.999
        assert torch.equal(ref[1][same], out[1][same]) and torch.equal(ref[2][same], out[2][same])
        # the two paths add a group's rows in different orders (tensor-core sums against ordered fp32 sums):
        # the same means up to the last bf16 digit
        a, c = ref[0][same].float(), out[0][same].float()
        assert bool(((a - c).abs() <= 2.0 ** -7 * torch.maximum(a.abs(), c.abs()) + 1e-6).all())
    for b in (0, B // 2, B - 1):                  # unplanted inputs: the near-tie rule decides what may differ
        n_band = check_merge_unplanted(x[b], 0, kept[b], out[0][b], out[1][b], out[2][b], "bf16")
        assert n_band <= N // 20


@pytest.mark.parametrize("K1", [144, 192])
@pytest.mark.parametrize("path", ["auto", "interleaved"])
def test_merge_calls_back_to_back_on_one_workspace(K1, path):
    """Three vscan_merge calls enqueued on one stream and one workspace with nothing between them (no
    vscan_check, no synchronisation, different inputs and outputs per call).  The kernels of one call are
    launched so that they may start while the previous kernel drains; a call must not disturb the counters,
    packed rows or status word an earlier call is still using.  Every result is checked against the oracle."""
    B, N, D, calls = 40, 576, 1024, 3
    cfg = small_cfg("bf16", grid_h=1, grid_w=N, win_h=1, win_w=N, k_w=0, k_g=K1, D=D, C=1, B=B, cls=1)
    rng = np.random.default_rng(K1)
    xs, kepts = [], []
    for c in range(calls):
        x = round_to_dtype(rng.standard_normal((B, N + 1, D)).astype(np.float32), "bf16")
        kept = np.stack([np.sort(rng.choice(N, K1, replace=False)) for _ in range(B)])
        plant.plant_merge(cfg, x, kept, seed=c)
        xs.append(x); kepts.append(kept)
    xd = [dev(x, "bf16") for x in xs]
    kd = [dev(k.astype(np.int32)) for k in kepts]
    outs = [(torch.empty((B, K1, D), dtype=torch.bfloat16, device="cuda"),) for _ in range(calls)]
    ws = vs.Workspace(64 << 20)
    code = vs.MERGE_AUTO if path == "auto" else vs.MERGE_INTERLEAVED
    torch.cuda.synchronize()
    res = [vs.vscan_merge(xd[c], 1, kd[c], want_assign=True, want_counts=True, workspace=ws, path=code, out=outs[c][0])
           for c in range(calls)]
    assert vs.vscan_check(ws) == 0
    for c in range(calls):
        merged, assign, counts = res[c]
        for b in (0, 17, B - 1):
            m, a, cn = vo.merge(xs[c][b], 1, kepts[c][b])
            np.testing.assert_array_equal(assign[b].cpu().numpy(), a)
            np.testing.assert_array_equal(counts[b].cpu().numpy(), cn)
            check_merged(merged[b], m, "bf16")


def test_merge_tensor_path_refuses_fp32():
    x = torch.randn((1, 40, 16), device="cuda")
    kept = torch.tensor([[1, 5]], dtype=torch.int32, device="cuda")
    with pytest.raises(vs.VScanError) as e:
        vs.vscan_merge(x, 0, kept, path=vs.MERGE_TENSOR)
    assert e.value.status == 2


def test_merge_separate_metric():
    x = RNG.standard_normal((2, 50, 24)).astype(np.float32)
    metric = RNG.standard_normal((2, 50, 16)).astype(np.float32)
    kept = np.stack([np.sort(RNG.choice(50, 6, replace=False)) for _ in range(2)]).astype(np.int32)
    merged, assign = vs.vscan_merge(dev(x, "f32"), 0, dev(kept), metric=dev(metric, "f32"), want_assign=True)
    for b in range(2):
        m, a, _ = vo.merge(x[b], 0, kept[b], metric=metric[b])
        np.testing.assert_array_equal(assign[b].cpu().numpy(), a)
        check_merged(merged[b], m, "f32")


# ------------------------------------------------------------------ vscan_score, QK mode
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("span", [vo.SPAN_ONLY, vo.SPAN_FULL])
@pytest.mark.parametrize("B,Hq,Hkv,S,d,b0,n", [(2, 6, 3, 70, 40, 3, 51), (1, 32, 32, 139, 128, 35, 64),
                                               (2, 28, 4, 300, 128, 0, 257), (1, 4, 1, 9, 8, 8, 1)])
def test_score_qk(dtype, span, B, Hq, Hkv, S, d, b0, n):
    q = round_to_dtype(RNG.standard_normal((B, Hq, d)).astype(np.float32), dtype)
    k = round_to_dtype(RNG.standard_normal((B, Hkv, S, d)).astype(np.float32), dtype)
    scale = 1.0 / np.sqrt(d)
    got = vs.vscan_score_qk(dev(q, dtype), dev(k, dtype), b0, n, scale, span).cpu().numpy()
    ref = np.stack([vo.score_qk(q[b], k[b], b0, n, float(np.float32(scale)), span) for b in range(B)])
    assert np.abs(got - ref).max() <= TOL_SCORE
    if span == vo.SPAN_ONLY:
        np.testing.assert_allclose(got.sum(-1), 1.0, atol=1e-5)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_cls_scores_from_q_and_k_eq1_eq2(dtype):
    """Eq. 1 + Eq. 2 without materialised attention rows: the QK mode with the [CLS] query of an encoder
    layer (softmax over all keys, span = the patches) gives the same scores as the head mean of the
    Eq. 1 rows, and feeds the selection directly."""
    B, H, N, d = 3, 16, 576, 64
    q = round_to_dtype(RNG.standard_normal((B, H, d)).astype(np.float32), dtype)
    k = round_to_dtype(RNG.standard_normal((B, H, N + 1, d)).astype(np.float32), dtype)
    scale = float(np.float32(d ** -0.5))
    got = vs.vscan_score_qk(dev(q, dtype), dev(k, dtype), 1, N, scale, vs.SPAN_FULL)
    ref = np.stack([vo.score_row(vo.cls_attention_rows(q[b], k[b], scale), 1) for b in range(B)])
    assert np.abs(got.cpu().numpy() - ref).max() <= TOL_SCORE
    kept = vs.vscan_select_global_local(got, got, 1, 24, 24, 6, 6, 2, 32).cpu().numpy()
    g32 = got.cpu().numpy()
    for b in range(B):
        np.testing.assert_array_equal(kept[b], vo.select_global_local(g32[b], g32[b], 1, 24, 24, 6, 6, 2, 32)[0])
    # The other reading of Eq. 1 (K_V = the patch keys only, [CLS] left out of the softmax) is the same
    # call with SPAN_ONLY: each head's row is the full-softmax row renormalised over the patches.
    alt = vs.vscan_score_qk(dev(q, dtype), dev(k, dtype), 1, N, scale, vs.SPAN_ONLY).cpu().numpy()
    for b in range(B):
        rows = vo.cls_attention_rows(q[b], k[b], scale)[:, 1:]
        ref_alt = (rows / rows.sum(axis=1, keepdims=True)).mean(axis=0)
        assert np.abs(alt[b] - ref_alt).max() <= TOL_SCORE
        assert abs(alt[b].sum() - 1.0) < 1e-5


@pytest.mark.parametrize("B,H,N,d", [(2, 3, 300, 64), (1, 4, 2048, 128), (1, 2, 129, 64), (3, 1, 128, 128), (2, 2, 1, 64)])
def test_received_attention_scores_from_q_and_k(B, H, N, d):
    """Sec. 4.1 (text after Eq. 2): for encoders without [CLS] the score of a token is the head mean of the average
    attention it receives from the other tokens.  The library computes it from q and k block by block; the oracle
    builds every head's full softmax matrix in float64 and takes its column means without the diagonal.  Tolerance:
    the scores are means of probabilities (<= 1) accumulated in fp32 from base-2 exponentials whose argument carries
    a relative rounding error of 2^-24 on values of up to a few tens: relative error of a probability about 2e-6,
    far below the 2e-6 absolute bar for values of the order 1/N."""
    rng = np.random.default_rng(N + d)
    q = round_to_dtype(rng.standard_normal((B, H, N, d)).astype(np.float32), "bf16")
    k = round_to_dtype(rng.standard_normal((B, H, N, d)).astype(np.float32), "bf16")
    scale = float(d ** -0.5)
    ws = vs.Workspace(0)
    got, rows = vs.vscan_score_received(dev(q, "bf16"), dev(k, "bf16"), scale, want_head_rows=True, workspace=None)
    got, rows = got.cpu().numpy(), rows.cpu().numpy()
    for b in range(B):
        z = scale * np.einsum("hid,hjd->hij", q[b].astype(np.float64), k[b].astype(np.float64))
        z -= z.max(axis=2, keepdims=True)
        p = np.exp(z)
        p /= p.sum(axis=2, keepdims=True)
        ref_rows = vo.received_attention(p)
        assert np.abs(rows[b] - ref_rows).max() <= TOL_SCORE
        assert np.abs(got[b] - vo.score_row(ref_rows, 0)).max() <= TOL_SCORE
    if N > 1:   # every query's attention sums to one, so the received attention sums to (N - diag mass) / (N - 1) <= N / (N - 1)
        assert np.all(got.sum(axis=1) <= N / (N - 1) + 1e-4)
    del ws


def test_received_attention_feeds_the_selection():
    """The received-attention scores go straight into the selection (the 16384-token workload without handed-in rows,
    at a size the oracle can follow): kept indices equal the oracle's on the library's own fp32 scores."""
    rng = np.random.default_rng(5)
    B, H, N, d = 2, 4, 1024, 64
    q = round_to_dtype(rng.standard_normal((B, H, N, d)).astype(np.float32), "bf16")
    k = round_to_dtype(rng.standard_normal((B, H, N, d)).astype(np.float32), "bf16")
    s = vs.vscan_score_received(dev(q, "bf16"), dev(k, "bf16"), float(d ** -0.5))
    kept = vs.vscan_select_global_local(s, s, 1, 32, 32, 8, 8, 2, 64).cpu().numpy()
    s32 = s.cpu().numpy()
    for b in range(B):
        np.testing.assert_array_equal(kept[b], vo.select_global_local(s32[b], s32[b], 1, 32, 32, 8, 8, 2, 64)[0])


# ------------------------------------------------------------------ vscan_llm_prune
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("span", [vo.SPAN_ONLY, vo.SPAN_FULL])
def test_llm_prune_small_planted(dtype, span):
    cfg = small_cfg(dtype, pos_planes=3)
    case = stage2_case(cfg, softmax_span=span)
    case["pos_ids"][1] *= 3; case["pos_ids"][2] += 100            # planes differ
    out = vs.vscan_llm_prune(dev(case["q_last"], dtype), dev(case["k"], dtype), dev(case["v"], dtype),
                             dev(case["hidden"], dtype), dev(case["pos_ids"]), cfg.n_sys, cfg.n_vis, cfg.n_txt,
                             cfg.k2, case["scale"], span, want_scores=True)
    o = case["oracle"]
    assert np.abs(out["scores"].cpu().numpy() - o["scores"]).max() <= TOL_SCORE
    np.testing.assert_array_equal(out["kept_vis"].cpu().numpy(), o["kept_vis"])
    for name in ("hidden", "k", "v"):
        np.testing.assert_array_equal(out[name].float().cpu().numpy(), o[name])      # bit-exact copies
    for b in range(cfg.B):
        rows = vo.compaction_rows(cfg.n_sys, cfg.n_vis, cfg.n_txt, o["kept_vis"][b])
        np.testing.assert_array_equal(out["pos"][:, b].cpu().numpy(), case["pos_ids"][:, b][:, rows])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("span", [vo.SPAN_ONLY, vo.SPAN_FULL])
@pytest.mark.parametrize("n_sys,n_vis,n_txt", [(5, 1100, 9), (0, 2048, 0), (300, 513, 260)])
def test_llm_prune_long_sequences_share_a_head_between_ctas(dtype, span, n_sys, n_vis, n_txt):
    """A few long sequences: several CTAs take contiguous shares of one head's keys and the last to finish rescales
    the row (Eq. 5 is unchanged: the softmax over the span from the shares' maxima and sums).  Shares that straddle
    the span's ends, a span that is the whole sequence, text and system keys that only enter the denominator."""
    B, Hq, Hkv, d, Dh, k_keep = 2, 6, 3, 64, 32, 200
    S = n_sys + n_vis + n_txt
    q = round_to_dtype(RNG.standard_normal((B, Hq, d)).astype(np.float32), dtype)
    k = round_to_dtype(RNG.standard_normal((B, Hkv, S, d)).astype(np.float32), dtype)
    h = round_to_dtype(RNG.standard_normal((B, S, Dh)).astype(np.float32), dtype)
    pos = np.tile(np.arange(S, dtype=np.int32), (1, B, 1))
    scale = 0.5
    out = vs.vscan_llm_prune(dev(q, dtype), dev(k, dtype), None, dev(h, dtype), dev(pos), n_sys, n_vis, n_txt, k_keep,
                             scale, span, want_scores=True)
    s32 = out["scores"].cpu().numpy()
    for b in range(B):
        ref = vo.score_qk(q[b], k[b], n_sys, n_vis, scale, span)
        assert np.abs(s32[b] - ref).max() <= TOL_SCORE
        kept = out["kept_vis"][b].cpu().numpy()
        np.testing.assert_array_equal(kept, vo.topk_lowest_index(s32[b], k_keep))   # decided on the kernel's fp32 scores
        rows = vo.compaction_rows(n_sys, n_vis, n_txt, kept)
        np.testing.assert_array_equal(out["hidden"][b].float().cpu().numpy(), h[b][rows])
        np.testing.assert_array_equal(out["k"][b].float().cpu().numpy(), k[b][:, rows])


def test_multi_turn_reselection_from_the_same_pool():
    """App. B "multi-turn conversations": a new question re-scores and re-selects from the existing
    token pool.  The library is stateless, so this is a second call with the new last-token query on
    the same keys; each turn must match the oracle on its own."""
    cfg = small_cfg("bf16")
    base = stage2_case(cfg)
    kd, vd, hd, pd = dev(base["k"], "bf16"), dev(base["v"], "bf16"), dev(base["hidden"], "bf16"), dev(base["pos_ids"])
    ws = vs.Workspace(1 << 20)
    kept_turns = []
    for turn in range(3):
        q = round_to_dtype(RNG.standard_normal(base["q_last"].shape).astype(np.float32) * 4, "bf16")
        out = vs.vscan_llm_prune(dev(q, "bf16"), kd, vd, hd, pd, cfg.n_sys, cfg.n_vis, cfg.n_txt, cfg.k2, base["scale"],
                                 want_scores=True, workspace=ws)
        s32 = out["scores"].cpu().numpy()
        for b in range(cfg.B):
            ref = vo.score_qk(q[b], base["k"][b], cfg.n_sys, cfg.n_vis, base["scale"])
            assert np.abs(s32[b] - ref).max() <= TOL_SCORE
            # selection is decided on the kernel's fp32 scores: feed exactly those to the oracle
            np.testing.assert_array_equal(out["kept_vis"][b].cpu().numpy(), vo.topk_lowest_index(s32[b], cfg.k2))
            rows = vo.compaction_rows(cfg.n_sys, cfg.n_vis, cfg.n_txt, out["kept_vis"][b].cpu().numpy())
            np.testing.assert_array_equal(out["hidden"][b].float().cpu().numpy(), base["hidden"][b][rows])
        kept_turns.append(out["kept_vis"].cpu().numpy().copy())
    assert any(not np.array_equal(kept_turns[0], k) for k in kept_turns[1:])     # different questions, different sets


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_prune_schedule_over_several_layers(dtype):
    """Stage 2 applied at three LLM layers in a row on the shrinking sequence (the multi-layer schedules
    App. B.1 compares with): each layer brings its own q / K / V for the current sequence, while hidden
    states and position ids are the previous call's output.  Every call is checked against the oracle run
    on the oracle's previous output, bit for bit, and the position ids end up naming the original tokens."""
    cfg = small_cfg(dtype, B=3, pos_planes=3, n_sys=4, n_txt=6)
    rng = np.random.default_rng(11)
    n_vis, keeps = cfg.n_vis, (31, 16, 5)
    S = cfg.n_sys + n_vis + cfg.n_txt
    hidden = round_to_dtype(rng.standard_normal((cfg.B, S, cfg.Dh)).astype(np.float32), dtype)
    pos = np.broadcast_to(np.arange(S, dtype=np.int32), (3, cfg.B, S)).copy()
    pos[1] *= 2
    h_ref, p_ref = hidden, pos
    h_gpu, p_gpu = dev(hidden, dtype), dev(pos)
    scale = float(cfg.d ** -0.5)
    for layer, k_keep in enumerate(keeps):
        S = cfg.n_sys + n_vis + cfg.n_txt
        q = round_to_dtype(rng.standard_normal((cfg.B, cfg.Hq, cfg.d)).astype(np.float32), dtype)
        k = round_to_dtype(rng.standard_normal((cfg.B, cfg.Hkv, S, cfg.d)).astype(np.float32), dtype)
        v = round_to_dtype(rng.standard_normal((cfg.B, cfg.Hkv, S, cfg.d)).astype(np.float32), dtype)
        plant.plant_stage2(cfg, q, k, scale, vo.SPAN_ONLY, n_vis=n_vis, k_keep=k_keep)
        ref = [vo.llm_prune(q[b], k[b], v[b], h_ref[b], p_ref[:, b], cfg.n_sys, n_vis, cfg.n_txt, k_keep, scale)
               for b in range(cfg.B)]
        out = vs.vscan_llm_prune(dev(q, dtype), dev(k, dtype), dev(v, dtype), h_gpu, p_gpu, cfg.n_sys, n_vis,
                                 cfg.n_txt, k_keep, scale)
        h_ref = np.stack([r["hidden"] for r in ref])
        p_ref = np.stack([r["pos"] for r in ref], axis=1)
        np.testing.assert_array_equal(out["kept_vis"].cpu().numpy(), np.stack([r["kept_vis"] for r in ref]))
        np.testing.assert_array_equal(out["hidden"].float().cpu().numpy(), h_ref)
        np.testing.assert_array_equal(out["k"].float().cpu().numpy(), np.stack([r["k"] for r in ref]))
        np.testing.assert_array_equal(out["v"].float().cpu().numpy(), np.stack([r["v"] for r in ref]))
        np.testing.assert_array_equal(out["pos"].cpu().numpy(), p_ref)
        h_gpu, p_gpu, n_vis = out["hidden"], out["pos"], k_keep
    # plane 0 still holds original sequence positions: strictly increasing, system and text spans intact
    final = p_gpu[0].cpu().numpy()
    assert final.shape == (cfg.B, cfg.n_sys + keeps[-1] + cfg.n_txt) and np.all(np.diff(final, axis=1) > 0)
    assert np.array_equal(final[:, :cfg.n_sys], np.tile(np.arange(cfg.n_sys), (cfg.B, 1)))
    np.testing.assert_array_equal(p_gpu[1].cpu().numpy(), 2 * final)


@pytest.mark.parametrize("k_keep,n_sys,n_txt", [(0, 3, 4), (20, 3, 4), (7, 0, 0), (20, 0, 5), (1, 2, 0)])
def test_llm_prune_edges(k_keep, n_sys, n_txt):
    n_vis, Hq, Hkv, d, Dh, B = 20, 4, 2, 16, 24, 2
    S = n_sys + n_vis + n_txt
    q = RNG.standard_normal((B, Hq, d)).astype(np.float32)
    k = RNG.standard_normal((B, Hkv, S, d)).astype(np.float32)
    v = RNG.standard_normal((B, Hkv, S, d)).astype(np.float32)
    h = RNG.standard_normal((B, S, Dh)).astype(np.float32)
    pos = np.tile(np.arange(S, dtype=np.int32) * 2, (1, B, 1))
    out = vs.vscan_llm_prune(dev(q), dev(k), dev(v), dev(h), dev(pos), n_sys, n_vis, n_txt, k_keep, 0.25)
    for b in range(B):
        o = vo.llm_prune(q[b], k[b], v[b], h[b], pos[:, b], n_sys, n_vis, n_txt, k_keep, 0.25)
        np.testing.assert_array_equal(out["kept_vis"][b].cpu().numpy(), o["kept_vis"])
        np.testing.assert_array_equal(out["hidden"][b].cpu().numpy(), o["hidden"])
        np.testing.assert_array_equal(out["k"][b].cpu().numpy(), o["k"])
        np.testing.assert_array_equal(out["v"][b].cpu().numpy(), o["v"])
        np.testing.assert_array_equal(out["pos"][:, b].cpu().numpy(), o["pos"])
        assert np.all(np.diff(out["pos"][0, b].cpu().numpy()) > 0)
    # K only (no V, hidden or position ids)
    out2 = vs.vscan_llm_prune(dev(q), dev(k), None, None, None, n_sys, n_vis, n_txt, k_keep, 0.25)
    assert torch.equal(out2["k"], out["k"]) and "v" not in out2


def test_workspace_too_small_and_status_word():
    cfg = small_cfg("bf16")
    case = stage2_case(cfg, planted=False)
    args = (dev(case["q_last"], "bf16"), dev(case["k"], "bf16"), None, None, None, cfg.n_sys, cfg.n_vis,
            cfg.n_txt, cfg.k2, case["scale"])
    with pytest.raises(vs.VScanError) as e:
        vs.vscan_llm_prune(*args, workspace=vs.Workspace(256))
    assert e.value.status == 3
    ws = vs.Workspace(1 << 20)
    ws.buf.fill_(0xFF)
    vs.vscan_llm_prune(*args, workspace=ws)
    assert vs.vscan_check(ws) == 0
    assert vs.kernel_launches() > 0


# ------------------------------------------------------------------ failure path of the device-side waits
def test_bounded_wait_runs_out_and_reports_timeout():
    """A wait on a flag that nothing sets gives up after its bound, the status word says so, and the
    context is still usable: the next call on the same workspace succeeds and clears the status."""
    ws = vs.Workspace(8 << 20)
    vs.vscan_selftest_bounded_wait(ws, polls=2000)          # about 0.2 ms
    assert vs.vscan_check(ws) == 5                          # VSCAN_ERR_TIMEOUT
    assert vs.status_string(5)
    x = torch.randn((1, 40, 16), device="cuda")
    kept = torch.tensor([[1, 5]], dtype=torch.int32, device="cuda")
    merged = vs.vscan_merge(x, 0, kept, workspace=ws)
    assert vs.vscan_check(ws) == 0
    assert torch.isfinite(merged).all()
    with pytest.raises(vs.VScanError):
        vs.vscan_selftest_bounded_wait(ws, polls=0)
