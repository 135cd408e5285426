"""vscan_score_qk_static: the entry point for callers that cannot allocate device memory.

Collected last on purpose (file name), so a run that stops at the first failure has already been
through every other test.  The scores are checked twice over: against the library's own workspace-based
entry point on the same inputs (same arithmetic, so they must agree within the score tolerance used
everywhere else) and against the CPU oracle's Eq. 5, on two calls in a row (the second one finds the
first one's leftovers in the built-in scratch and must not be disturbed by them).
"""
import ctypes as C

import numpy as np
import pytest
import torch

import paper_2505_22654_b200 as vs
from paper_2505_22654_b200 import binding as vb

from oracle import vscan_oracle as vo

from helpers import TOL_SCORE

pytestmark = pytest.mark.gpu


def _inputs(seed, B, Hq, Hkv, S, d, dtype):
    g = torch.Generator(device="cpu").manual_seed(seed)
    q = torch.randn((B, Hq, d), generator=g).to(dtype).cuda()
    k = torch.randn((B, Hkv, S, d), generator=g).to(dtype).cuda()
    return q, k


def _oracle(q, k, b0, n, scale, span=vo.SPAN_ONLY):
    qn, kn = q.float().cpu().numpy(), k.float().cpu().numpy()
    return np.stack([vo.score_qk(qn[b], kn[b], b0, n, scale, span) for b in range(qn.shape[0])])


def test_static_scratch_matches_workspace_entry_point_twice_in_a_row():
    # first call: the 2880-token LLM shape (32 sequences, 32 heads, 320 visual keys), bf16
    q, k = _inputs(1, 32, 32, 32, 419, 128, torch.bfloat16)
    out = torch.empty((32, 320), dtype=torch.float32, device="cuda")     # the caller brings the output
    out2 = torch.empty((3, 257), dtype=torch.float32, device="cuda")
    out3 = torch.empty((32, 320), dtype=torch.float32, device="cuda")
    got1 = vs.vscan_score_qk_static(q, k, 35, 320, 128 ** -0.5, out)
    ref1 = vs.vscan_score_qk(q, k, 35, 320, 128 ** -0.5)
    # second call straight after, other shape, grouped heads, softmax over the whole sequence, fp32:
    # the scratch still holds the first call's probabilities
    q2, k2 = _inputs(2, 3, 28, 4, 300, 64, torch.float32)
    got2 = vs.vscan_score_qk_static(q2, k2, 7, 257, 0.125, out2, vs.SPAN_FULL)
    ref2 = vs.vscan_score_qk(q2, k2, 7, 257, 0.125, vs.SPAN_FULL)
    torch.cuda.synchronize()
    assert got1.data_ptr() == out.data_ptr()
    assert float((got1 - ref1).abs().max()) <= TOL_SCORE
    assert float((got2 - ref2).abs().max()) <= TOL_SCORE
    np.testing.assert_allclose(got1.sum(-1).cpu().numpy(), 1.0, atol=1e-5)
    # the same two results against the CPU oracle (Eq. 5 in float64 on the same rounded inputs)
    assert np.abs(got1.cpu().numpy() - _oracle(q, k, 35, 320, 128 ** -0.5)).max() <= TOL_SCORE
    assert np.abs(got2.cpu().numpy() - _oracle(q2, k2, 7, 257, 0.125, vo.SPAN_FULL)).max() <= TOL_SCORE
    # and the first shape once more gives the first answer again
    got3 = vs.vscan_score_qk_static(q, k, 35, 320, 128 ** -0.5, out3)
    assert float((got3 - ref1).abs().max()) <= TOL_SCORE


def test_static_scratch_rejects_sizes_beyond_its_capacity():
    L = vb.lib()
    cap = L.vscan_score_qk_static_capacity()
    assert cap == 1 << 20
    q, k = _inputs(3, 2, 8, 8, 40, 32, torch.bfloat16)
    out = torch.zeros((2, 40), dtype=torch.float32, device="cuda")
    d = vb.score_qk_desc(q, k, 0, 40, 1.0, vb.SPAN_ONLY, out)
    d.batch = 4096                       # 4096 * 8 * 40 floats > 1 Mi: refused before any launch
    assert L.vscan_score_qk_static(C.byref(d), None) == vb.ERR_UNSUPPORTED
    d.batch, d.mode = 2, vb.SCORE_ROW    # only the QK mode has a static variant
    assert L.vscan_score_qk_static(C.byref(d), None) == vb.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert float(out.abs().max()) == 0.0
