"""The C-ABI library loads without a GPU, exports every symbol the header declares, its structs
have the layout the ctypes binding assumes, and argument validation rejects bad calls on the host
(before anything could be launched)."""
import ctypes as C
import os
import re
import subprocess
import sys
import tempfile

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "vscan.h")

from paper_2505_22654_b200 import binding as vb  # noqa: E402
from paper_2505_22654_b200 import _build  # noqa: E402


@pytest.fixture(scope="module")
def L():
    _build.build()
    return vb.lib()


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vscan_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = _declared_functions()
    assert {"vscan_score", "vscan_select_global_local", "vscan_merge", "vscan_llm_prune"} <= set(names)
    for n in names:
        assert hasattr(L, n), n
    assert L.vscan_version() == 100
    assert vb.status_string(vb.ERR_WORKSPACE).startswith("workspace")


def test_struct_layout_matches_header():
    prog = r'''
#include <stdio.h>
#include <stddef.h>
#include "vscan.h"
#define P(s, f) printf(#s "." #f " %zu\n", offsetof(s, f))
int main(void) {
  printf("vscan_score_desc %zu\n", sizeof(vscan_score_desc));
  P(vscan_score_desc, attn); P(vscan_score_desc, q); P(vscan_score_desc, batch); P(vscan_score_desc, scale); P(vscan_score_desc, scores); P(vscan_score_desc, head_rows);
  printf("vscan_select_desc %zu\n", sizeof(vscan_select_desc));
  P(vscan_select_desc, instances); P(vscan_select_desc, kept_idx); P(vscan_select_desc, kept_mask);
  printf("vscan_merge_desc %zu\n", sizeof(vscan_merge_desc));
  P(vscan_merge_desc, x); P(vscan_merge_desc, instances); P(vscan_merge_desc, n_kept); P(vscan_merge_desc, merged); P(vscan_merge_desc, counts);
  printf("vscan_prune_desc %zu\n", sizeof(vscan_prune_desc));
  P(vscan_prune_desc, q_last); P(vscan_prune_desc, batch); P(vscan_prune_desc, k_keep); P(vscan_prune_desc, scale); P(vscan_prune_desc, kept_vis); P(vscan_prune_desc, scores);
  printf("vscan_stage1_ragged_desc %zu\n", sizeof(vscan_stage1_ragged_desc));
  P(vscan_stage1_ragged_desc, attn_global); P(vscan_stage1_ragged_desc, merged); P(vscan_stage1_ragged_desc, frames); P(vscan_stage1_ragged_desc, kept_offset);
  printf("vscan_prune_ragged_desc %zu\n", sizeof(vscan_prune_ragged_desc));
  P(vscan_prune_ragged_desc, scale); P(vscan_prune_ragged_desc, q_last); P(vscan_prune_ragged_desc, pos_out); P(vscan_prune_ragged_desc, n_sys); P(vscan_prune_ragged_desc, kept_offset);
  return 0;
}'''
    with tempfile.TemporaryDirectory() as td:
        src, exe = os.path.join(td, "layout.c"), os.path.join(td, "layout")
        open(src, "w").write(prog)
        subprocess.run(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"), src, "-o", exe], check=True)
        out = subprocess.run([exe], capture_output=True, text=True, check=True).stdout
    got = dict(line.rsplit(" ", 1) for line in out.strip().splitlines())
    structs = {"vscan_score_desc": vb.ScoreDesc, "vscan_select_desc": vb.SelectDesc,
               "vscan_merge_desc": vb.MergeDesc, "vscan_prune_desc": vb.PruneDesc,
               "vscan_stage1_ragged_desc": vb.Stage1RaggedDesc, "vscan_prune_ragged_desc": vb.PruneRaggedDesc}
    for key, val in got.items():
        if "." in key:
            s, f = key.split(".")
            assert getattr(structs[s], f).offset == int(val), key
        else:
            assert C.sizeof(structs[key]) == int(val), key


FAKE = 0x10000  # a non-null, 16-byte aligned address that is never dereferenced on the host


def test_select_validation_is_host_side(L):
    def call(**kw):
        base = dict(scores_global=FAKE, scores_local=FAKE, instances=1, frames=1, grid_h=4, grid_w=4,
                    win_h=2, win_w=2, k_per_window=1, k_global=2, kept_idx=FAKE + 0x10000)
        base.update(kw)
        d = vb.SelectDesc(**base)
        return L.vscan_select_global_local(C.byref(d), None, 0, None)
    assert call(scores_global=None) == vb.ERR_INVALID_ARG
    assert call(win_h=3) == vb.ERR_INVALID_ARG                  # window must divide the grid
    assert call(k_per_window=5) == vb.ERR_INVALID_ARG           # more than the window holds
    assert call(k_global=13) == vb.ERR_INVALID_ARG              # more than the complement holds
    assert call(k_global=-1) == vb.ERR_INVALID_ARG
    assert call(kept_idx=FAKE + 4) == vb.ERR_INVALID_ARG        # misaligned / overlapping output
    assert call(frames=64, grid_h=32, grid_w=32, win_h=8, win_w=8) == vb.ERR_UNSUPPORTED   # N > 16384
    assert call(instances=0) == vb.OK                           # empty batch: nothing to do


def test_score_validation_is_host_side(L):
    d = vb.ScoreDesc(mode=vb.SCORE_ROW, dtype=vb.BF16, attn=FAKE, instances=1, heads=4, row_len=8,
                     cls_offset=1, n_tokens=8, scores=FAKE + 0x10000)
    assert L.vscan_score(C.byref(d), None, 0, None) == vb.ERR_INVALID_ARG      # row too short
    d = vb.ScoreDesc(mode=7, dtype=vb.BF16, scores=FAKE)
    assert L.vscan_score(C.byref(d), None, 0, None) == vb.ERR_INVALID_ARG
    d = vb.ScoreDesc(mode=vb.SCORE_QK, dtype=vb.BF16, q=FAKE, k=FAKE + 0x100000, batch=1, q_heads=6, kv_heads=4,
                     seq_len=16, head_dim=64, span_begin=0, span_len=16, scale=1.0, scores=FAKE + 0x800000)
    assert L.vscan_score(C.byref(d), None, 0, None) == vb.ERR_INVALID_ARG      # 6 heads over 4 KV heads
    d.q_heads = 8
    d.head_dim = 60
    assert L.vscan_score(C.byref(d), None, 0, None) == vb.ERR_INVALID_ARG      # head_dim % 8
    d.head_dim = 64
    assert L.vscan_score_workspace_bytes(C.byref(d)) >= 256 + 8 * 16 * 4
    assert L.vscan_score(C.byref(d), None, 0, None) == vb.ERR_WORKSPACE       # no workspace given
    d.span_len = 17
    assert L.vscan_score(C.byref(d), None, 0, None) == vb.ERR_INVALID_ARG      # span leaves the sequence
    d.span_begin, d.span_len = 2 ** 31 - 1, 16                                # the sum must not wrap around
    assert L.vscan_score(C.byref(d), None, 0, None) == vb.ERR_INVALID_ARG
    assert L.vscan_score_qk_static(C.byref(d), None) == vb.ERR_INVALID_ARG
    d.span_begin = 0
    d.scores = FAKE + 0x100000                                                # output on top of the keys
    assert L.vscan_score(C.byref(d), None, 0, None) == vb.ERR_INVALID_ARG
    assert L.vscan_score_qk_static(C.byref(d), None) == vb.ERR_INVALID_ARG    # same checks in the static variant
    d.scores = FAKE + 0x800000


def test_received_mode_validation(L):
    d = vb.ScoreDesc(mode=vb.SCORE_RECEIVED, dtype=vb.BF16, q=FAKE, k=FAKE + 0x1000000, batch=2, q_heads=4, kv_heads=4,
                     seq_len=300, head_dim=64, scale=0.125, scores=FAKE + 0x2000000)
    assert L.vscan_score_workspace_bytes(C.byref(d)) >= 256 + 8 * 384 * 4 + 8 * 300 * 4
    assert L.vscan_score(C.byref(d), None, 0, None) == vb.ERR_WORKSPACE        # legal: next check is the workspace
    d.kv_heads = 2
    assert L.vscan_score(C.byref(d), None, 0, None) == vb.ERR_INVALID_ARG      # every head has its own keys here
    d.kv_heads, d.head_dim = 4, 80
    assert L.vscan_score(C.byref(d), None, 0, None) == vb.ERR_UNSUPPORTED      # head_dim 64 or 128 in this build
    d.head_dim, d.dtype = 64, vb.F32
    assert L.vscan_score(C.byref(d), None, 0, None) == vb.ERR_UNSUPPORTED      # tensor-core path: bf16 only
    d.dtype, d.batch = vb.BF16, 20000
    assert L.vscan_score(C.byref(d), None, 0, None) == vb.ERR_UNSUPPORTED      # batch * heads beyond the grid limit
    d.batch, d.scores = 2, FAKE
    assert L.vscan_score(C.byref(d), None, 0, None) == vb.ERR_INVALID_ARG      # output on top of q


def test_shape_limits_are_refused_before_anything_is_enqueued(L):
    """Limits of the build come back as UNSUPPORTED from the host-side checks (no stream, no workspace
    and fake pointers here: a launch or a memset would fail differently)."""
    d = vb.ScoreDesc(mode=vb.SCORE_ROW, dtype=vb.BF16, attn=FAKE, instances=70000, heads=2, row_len=8,
                     cls_offset=0, n_tokens=8, scores=FAKE + 0x10000000)
    assert L.vscan_score(C.byref(d), None, 0, None) == vb.ERR_UNSUPPORTED      # grid.y limit
    q = vb.ScoreDesc(mode=vb.SCORE_QK, dtype=vb.BF16, q=FAKE, k=FAKE + 0x100000, batch=70000, q_heads=2,
                     kv_heads=2, seq_len=16, head_dim=64, span_begin=0, span_len=16, scale=1.0,
                     scores=FAKE + 0x40000000)
    assert L.vscan_score(C.byref(q), None, 0, None) == vb.ERR_UNSUPPORTED
    q.batch, q.seq_len, q.span_len = 1, 70000, 70000                          # softmax row beyond shared memory
    assert L.vscan_score(C.byref(q), None, 0, None) == vb.ERR_UNSUPPORTED
    assert L.vscan_score_qk_static(C.byref(q), None) == vb.ERR_UNSUPPORTED
    m = vb.MergeDesc(dtype=vb.BF16, path=vb.MERGE_AUTO, x=FAKE, kept_idx=FAKE + 0x40000000, instances=1,
                     row_len=30000, cls_offset=0, n_tokens=30000, dim=8, n_kept=4, merged=FAKE + 0x50000000)
    assert L.vscan_merge(C.byref(m), None, 0, None) == vb.ERR_UNSUPPORTED      # member list beyond shared memory
    m.n_tokens = m.row_len = 29054
    assert L.vscan_merge(C.byref(m), None, 0, None) == vb.ERR_WORKSPACE       # legal: next check is the workspace


def test_merge_and_prune_validation_is_host_side(L):
    m = vb.MergeDesc(dtype=vb.BF16, path=vb.MERGE_AUTO, x=FAKE, kept_idx=FAKE + 0x100000, instances=1, row_len=17,
                     cls_offset=1, n_tokens=16, dim=64, n_kept=4, merged=FAKE + 0x200000)
    assert L.vscan_merge(C.byref(m), None, 0, None) == vb.ERR_WORKSPACE
    assert L.vscan_merge_workspace_bytes(C.byref(m)) >= 256 + 16 + 64
    m.n_kept = 0
    assert L.vscan_merge(C.byref(m), None, 0, None) == vb.ERR_INVALID_ARG
    m.n_kept = 17
    assert L.vscan_merge(C.byref(m), None, 0, None) == vb.ERR_INVALID_ARG
    m.n_kept, m.dim = 4, 60
    assert L.vscan_merge(C.byref(m), None, 0, None) == vb.ERR_INVALID_ARG
    m.dim, m.merged = 64, FAKE                                              # output on top of the input
    assert L.vscan_merge(C.byref(m), None, 0, None) == vb.ERR_INVALID_ARG
    m.merged, m.path = FAKE + 0x200000, 9
    assert L.vscan_merge(C.byref(m), None, 0, None) == vb.ERR_INVALID_ARG

    p = vb.PruneDesc(dtype=vb.BF16, q_last=FAKE, k=FAKE + 0x100000, batch=1, q_heads=4, kv_heads=2, head_dim=32,
                     n_sys=2, n_vis=8, n_txt=2, k_keep=9, scale=1.0, kept_vis=FAKE + 0x300000,
                     k_out=FAKE + 0x400000)
    assert L.vscan_llm_prune(C.byref(p), None, 0, None) == vb.ERR_INVALID_ARG  # k_keep > n_vis
    p.k_keep = 4
    assert L.vscan_llm_prune(C.byref(p), None, 0, None) == vb.ERR_WORKSPACE
    p.v = FAKE + 0x500000                                                    # v without v_out
    assert L.vscan_llm_prune(C.byref(p), None, 0, None) == vb.ERR_INVALID_ARG
    p.v = None
    p.n_vis, p.k_keep = 20000, 4
    assert L.vscan_llm_prune(C.byref(p), None, 0, None) == vb.ERR_UNSUPPORTED


def test_ragged_validation_is_host_side(L):
    """Sizes, budgets and offsets of a ragged call are host arrays: everything is checked before a launch."""
    def stage1(**kw):
        n = 2
        base = dict(dtype=vb.BF16, merge_path=vb.MERGE_AUTO, instances=n, heads=4, cls_offset=1, dim=64, win_h=2, win_w=2,
                    attn_global=FAKE, attn_local=FAKE, x=FAKE + 0x100000, kept_idx=FAKE + 0x200000, merged=FAKE + 0x300000,
                    frames=[1, 1], grid_h=[4, 6], grid_w=[4, 6], k_per_window=[1, 1], k_global=[2, 2],
                    attn_offset=[0, 72], x_offset=[0, 17 * 64], kept_offset=[0, 8])
        base.update(kw)
        arrays = {k: (vb._host_i64(v) if k.endswith("offset") else vb._host_i32(v)) for k, v in base.items() if isinstance(v, list)}
        base.update(arrays)
        d = vb.Stage1RaggedDesc(**base)
        return L.vscan_stage1_ragged(C.byref(d), None, 0, None), L.vscan_stage1_ragged_workspace_bytes(C.byref(d))
    st, need = stage1()
    assert st == vb.ERR_WORKSPACE and need > 256                 # legal call: next check is the workspace
    assert stage1(grid_h=[4, 5])[0] == vb.ERR_INVALID_ARG         # window does not divide the second grid
    assert stage1(attn_offset=[0, 69])[0] == vb.ERR_WORKSPACE     # (alignment is checked after the workspace)
    assert stage1(instances=0)[0] == vb.OK
    assert stage1(frames=None)[0] == vb.ERR_INVALID_ARG
    p = vb.PruneRaggedDesc(dtype=vb.BF16, batch=1, q_heads=4, kv_heads=2, head_dim=32, hidden_dim=0, pos_planes=0, scale=1.0,
                           q_last=FAKE, k=FAKE + 0x100000, kept_vis=FAKE + 0x200000, k_out=FAKE + 0x300000,
                           n_sys=vb._host_i32([2]), n_vis=vb._host_i32([8]), n_txt=vb._host_i32([2]), k_keep=vb._host_i32([9]),
                           kv_offset=vb._host_i64([0]), kv_out_offset=vb._host_i64([0]), kept_offset=vb._host_i64([0]))
    assert L.vscan_llm_prune_ragged(C.byref(p), None, 0, None) == vb.ERR_INVALID_ARG   # k_keep > n_vis
    p.k_keep = vb._host_i32([4])
    assert L.vscan_llm_prune_ragged(C.byref(p), None, 0, None) == vb.ERR_WORKSPACE


def test_stale_library_is_rebuilt_or_refused(monkeypatch, tmp_path):
    """A library that does not match the sources on disk is never loaded silently."""
    assert not _build._stale()                     # the fixture `L` loaded (and, if needed, rebuilt) it
    stamp = tmp_path / "stamp"
    stamp.write_text("0" * 64 + "\n")              # a digest of other sources
    monkeypatch.setattr(_build, "STAMP_PATH", str(stamp))
    assert _build._stale()
    monkeypatch.setattr(vb, "_LIB", None)
    monkeypatch.setattr(_build, "have_nvcc", lambda: False)
    with pytest.raises(RuntimeError, match="does not match the sources"):
        vb.lib()
    calls = []
    monkeypatch.setattr(_build, "have_nvcc", lambda: True)
    monkeypatch.setattr(_build, "build", lambda force=False, **k: calls.append(force) or _build.LIB_PATH)
    assert vb.lib().vscan_version() > 0 and calls == [False]


def test_no_cpu_fallback_when_library_missing(monkeypatch, tmp_path):
    """The product path must fail loudly, not route around a missing CUDA library."""
    monkeypatch.setattr(vb, "_LIB", None)
    monkeypatch.setattr(_build, "LIB_PATH", str(tmp_path / "nope.so"))
    monkeypatch.setattr(_build, "build", lambda *a, **k: (_ for _ in ()).throw(RuntimeError("nvcc not found")))
    with pytest.raises(RuntimeError):
        vb.lib()
    src = open(os.path.join(ROOT, "paper_2505_22654_b200", "binding.py")).read() + \
        open(os.path.join(ROOT, "paper_2505_22654_b200", "pipeline.py")).read()
    assert "oracle" not in src
