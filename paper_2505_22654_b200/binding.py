"""ctypes binding of libvscan.so: argument marshalling only.

Each function mirrors one entry point of include/vscan.h, takes CUDA torch tensors (used purely
as device memory) and enqueues the library's kernels on torch's current stream.  There is no
fallback of any kind: if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import _build

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)
F32, BF16 = 0, 1
SCORE_ROW, SCORE_QK, SCORE_RECEIVED = 0, 1, 2
SPAN_ONLY, SPAN_FULL = 0, 1
MERGE_AUTO, MERGE_SIMT, MERGE_TENSOR, MERGE_CLUSTER, MERGE_INTERLEAVED = 0, 1, 2, 3, 4

_vp, _i32, _f32 = C.c_void_p, C.c_int32, C.c_float


class ScoreDesc(C.Structure):
    _fields_ = [("mode", _i32), ("dtype", _i32), ("attn", _vp), ("instances", _i32), ("heads", _i32),
                ("row_len", _i32), ("cls_offset", _i32), ("n_tokens", _i32), ("q", _vp), ("k", _vp),
                ("batch", _i32), ("q_heads", _i32), ("kv_heads", _i32), ("seq_len", _i32),
                ("head_dim", _i32), ("span_begin", _i32), ("span_len", _i32), ("softmax_span", _i32),
                ("scale", _f32), ("scores", _vp), ("head_rows", _vp)]


class SelectDesc(C.Structure):
    _fields_ = [("scores_global", _vp), ("scores_local", _vp), ("instances", _i32), ("frames", _i32),
                ("grid_h", _i32), ("grid_w", _i32), ("win_h", _i32), ("win_w", _i32),
                ("k_per_window", _i32), ("k_global", _i32), ("kept_idx", _vp), ("kept_mask", _vp)]


class ScoreSelectDesc(C.Structure):
    _fields_ = [("dtype", _i32), ("attn_global", _vp), ("attn_local", _vp), ("heads", _i32), ("row_len", _i32),
                ("cls_offset", _i32), ("select", SelectDesc)]


class MergeDesc(C.Structure):
    _fields_ = [("dtype", _i32), ("path", _i32), ("x", _vp), ("metric", _vp), ("kept_idx", _vp),
                ("instances", _i32), ("row_len", _i32), ("cls_offset", _i32), ("n_tokens", _i32),
                ("dim", _i32), ("metric_dim", _i32), ("n_kept", _i32), ("merged", _vp), ("assign", _vp),
                ("counts", _vp)]


class PruneDesc(C.Structure):
    _fields_ = [("dtype", _i32), ("q_last", _vp), ("k", _vp), ("v", _vp), ("hidden", _vp),
                ("pos_ids", _vp), ("batch", _i32), ("q_heads", _i32), ("kv_heads", _i32),
                ("head_dim", _i32), ("hidden_dim", _i32), ("pos_planes", _i32), ("n_sys", _i32),
                ("n_vis", _i32), ("n_txt", _i32), ("k_keep", _i32), ("softmax_span", _i32),
                ("scale", _f32), ("kept_vis", _vp), ("hidden_out", _vp), ("k_out", _vp), ("v_out", _vp),
                ("pos_out", _vp), ("scores", _vp)]


_i64p, _i32p = C.POINTER(C.c_int64), C.POINTER(C.c_int32)


class Stage1RaggedDesc(C.Structure):
    _fields_ = [("dtype", _i32), ("merge_path", _i32), ("instances", _i32), ("heads", _i32), ("cls_offset", _i32),
                ("dim", _i32), ("win_h", _i32), ("win_w", _i32), ("attn_global", _vp), ("attn_local", _vp), ("x", _vp),
                ("kept_idx", _vp), ("merged", _vp), ("frames", _i32p), ("grid_h", _i32p), ("grid_w", _i32p),
                ("k_per_window", _i32p), ("k_global", _i32p), ("attn_offset", _i64p), ("x_offset", _i64p),
                ("kept_offset", _i64p)]


class PruneRaggedDesc(C.Structure):
    _fields_ = [("dtype", _i32), ("batch", _i32), ("q_heads", _i32), ("kv_heads", _i32), ("head_dim", _i32),
                ("hidden_dim", _i32), ("pos_planes", _i32), ("softmax_span", _i32), ("scale", _f32), ("q_last", _vp),
                ("k", _vp), ("v", _vp), ("hidden", _vp), ("pos_ids", _vp), ("kept_vis", _vp), ("hidden_out", _vp),
                ("k_out", _vp), ("v_out", _vp), ("pos_out", _vp), ("n_sys", _i32p), ("n_vis", _i32p), ("n_txt", _i32p),
                ("k_keep", _i32p), ("kv_offset", _i64p), ("kv_out_offset", _i64p), ("hidden_offset", _i64p),
                ("hidden_out_offset", _i64p), ("pos_offset", _i64p), ("pos_out_offset", _i64p), ("kept_offset", _i64p)]


class VScanError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status}, cuda error {lib().vscan_last_cuda_error()})")


_LIB = None


def lib() -> C.CDLL:
    """Load libvscan.so, building it first when it is missing or was built from other sources than the
    ones on disk.  Raises if it is unavailable, or stale with no compiler to rebuild it: a library that
    does not match its sources is never loaded silently."""
    global _LIB
    if _LIB is None:
        path = _build.LIB_PATH
        force = os.environ.get("VSCAN_REBUILD") == "1"
        if force or _build._stale():
            if not _build.have_nvcc():
                raise RuntimeError(f"{path} is missing or does not match the sources under csrc/, and nvcc is "
                                   "not available to rebuild it")
            path = _build.build(force=force)
        L = C.CDLL(path)
        for name, desc in (("score", ScoreDesc), ("select", SelectDesc), ("merge", MergeDesc),
                           ("llm_prune", PruneDesc)):
            ws = getattr(L, f"vscan_{name}_workspace_bytes")
            ws.restype, ws.argtypes = C.c_size_t, [C.POINTER(desc)]
        for fn, desc in (("vscan_score", ScoreDesc), ("vscan_select_global_local", SelectDesc),
                         ("vscan_merge", MergeDesc), ("vscan_llm_prune", PruneDesc)):
            f = getattr(L, fn)
            f.restype, f.argtypes = _i32, [C.POINTER(desc), _vp, C.c_size_t, _vp]
        for name, desc in (("stage1_ragged", Stage1RaggedDesc), ("llm_prune_ragged", PruneRaggedDesc)):
            ws = getattr(L, f"vscan_{name}_workspace_bytes")
            ws.restype, ws.argtypes = C.c_size_t, [C.POINTER(desc)]
            f = getattr(L, f"vscan_{name}")
            f.restype, f.argtypes = _i32, [C.POINTER(desc), _vp, C.c_size_t, _vp]
        L.vscan_score_select.restype = _i32
        L.vscan_score_select.argtypes = [C.POINTER(ScoreSelectDesc), _vp]
        L.vscan_version.restype = _i32
        L.vscan_status_string.restype, L.vscan_status_string.argtypes = C.c_char_p, [_i32]
        L.vscan_check.restype, L.vscan_check.argtypes = _i32, [_vp, _vp]
        L.vscan_last_cuda_error.restype = _i32
        L.vscan_kernel_launches.restype = C.c_uint64
        L.vscan_profile_begin.restype, L.vscan_profile_begin.argtypes = _i32, [_i32]
        L.vscan_profile_end.restype = _i32
        L.vscan_profile_end.argtypes = [C.c_char_p, C.POINTER(C.c_float), _i32]
        L.vscan_selftest_bounded_wait.restype = _i32
        L.vscan_selftest_bounded_wait.argtypes = [_vp, C.c_size_t, C.c_uint32, _vp]
        L.vscan_selftest_fma_rate.restype = _i32
        L.vscan_selftest_fma_rate.argtypes = [_vp, C.c_size_t, _i32, _i32, C.POINTER(C.c_double), _vp]
        L.vscan_score_qk_static_capacity.restype = C.c_size_t
        L.vscan_score_qk_static.restype = _i32
        L.vscan_score_qk_static.argtypes = [C.POINTER(ScoreDesc), _vp]
        _LIB = L
    return _LIB


def status_string(status: int) -> str:
    return lib().vscan_status_string(status).decode()


def kernel_launches() -> int:
    return int(lib().vscan_kernel_launches())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("tensors must be contiguous CUDA tensors")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


class Workspace:
    """A reusable device scratch buffer (256-byte aligned by the torch allocator)."""

    def __init__(self, nbytes: int = 0, device="cuda"):
        self.device = device
        self.buf = None
        self.reserve(nbytes)

    def reserve(self, nbytes: int):
        if self.buf is None or self.buf.numel() < nbytes:
            self.buf = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=self.device)
        return self

    @property
    def ptr(self):
        return self.buf.data_ptr()

    @property
    def nbytes(self):
        return self.buf.numel()


def _call(fn_name, desc, ws_fn_name, workspace):
    L = lib()
    need = getattr(L, ws_fn_name)(C.byref(desc))
    if workspace is None:
        workspace = Workspace(need)
    elif workspace.nbytes < need:
        raise VScanError(ERR_WORKSPACE, f"{fn_name}: workspace of {workspace.nbytes} B < {need} B")
    st = getattr(L, fn_name)(C.byref(desc), workspace.ptr, workspace.nbytes, _stream())
    if st != OK:
        raise VScanError(st, fn_name)
    return workspace


# ------------------------------------------------------------------------------------------ API
def score_row_desc(attn, cls_offset, n_tokens, scores) -> ScoreDesc:
    B, H, L = attn.shape
    return ScoreDesc(mode=SCORE_ROW, dtype=_dtype_code(attn), attn=_ptr(attn), instances=B, heads=H,
                     row_len=L, cls_offset=cls_offset, n_tokens=n_tokens, scores=_ptr(scores))


def vscan_score_row(attn: torch.Tensor, cls_offset: int, n_tokens: int | None = None,
                    out: torch.Tensor | None = None) -> torch.Tensor:
    """Eq. 2: head mean of attention rows.  attn [B', H, L] -> scores [B', N] float32."""
    n = attn.shape[2] - cls_offset if n_tokens is None else n_tokens
    if out is None:
        out = torch.empty((attn.shape[0], n), dtype=torch.float32, device=attn.device)
    d = score_row_desc(attn, cls_offset, n, out)
    st = lib().vscan_score(C.byref(d), None, 0, _stream())
    if st != OK:
        raise VScanError(st, "vscan_score")
    return out


def score_qk_desc(q, k, span_begin, span_len, scale, softmax_span, scores) -> ScoreDesc:
    B, Hq, d = q.shape
    _, Hkv, S, _ = k.shape
    return ScoreDesc(mode=SCORE_QK, dtype=_dtype_code(k), q=_ptr(q), k=_ptr(k), batch=B, q_heads=Hq,
                     kv_heads=Hkv, seq_len=S, head_dim=d, span_begin=span_begin, span_len=span_len,
                     softmax_span=softmax_span, scale=scale, scores=_ptr(scores))


def vscan_score_qk(q, k, span_begin, span_len, scale, softmax_span=SPAN_ONLY, out=None, workspace=None):
    """Eq. 5: head mean of softmax(scale * q . K) on a span.  -> scores [B, span_len] float32."""
    if out is None:
        out = torch.empty((q.shape[0], span_len), dtype=torch.float32, device=q.device)
    d = score_qk_desc(q, k, span_begin, span_len, scale, softmax_span, out)
    _call("vscan_score", d, "vscan_score_workspace_bytes", workspace)
    return out


def vscan_score_received(q, k, scale, out=None, want_head_rows=False, workspace=None):
    """Sec. 4.1 (text after Eq. 2): head mean of the attention every token receives from the others, from
    q, k [B', H, N, d] without the N x N matrix.  -> scores [B', N] float32 (and the per-head rows [B', H, N])."""
    B, H, N, d = q.shape
    if out is None:
        out = torch.empty((B, N), dtype=torch.float32, device=q.device)
    rows = torch.empty((B, H, N), dtype=torch.float32, device=q.device) if want_head_rows else None
    desc = ScoreDesc(mode=SCORE_RECEIVED, dtype=_dtype_code(q), q=_ptr(q), k=_ptr(k), batch=B, q_heads=H, kv_heads=H,
                     seq_len=N, head_dim=d, scale=scale, scores=_ptr(out), head_rows=_ptr(rows))
    _call("vscan_score", desc, "vscan_score_workspace_bytes", workspace)
    return (out, rows) if want_head_rows else out


def vscan_score_qk_static(q, k, span_begin, span_len, scale, out, softmax_span=SPAN_ONLY):
    """Same scores as vscan_score_qk, for callers that may not allocate device memory: the scratch
    is a fixed 4 MiB array inside the library instead of a workspace, and nothing is allocated here
    either, so the caller brings `out` ([B, span_len] float32).  Raises VScanError(ERR_UNSUPPORTED)
    when B * Hq * span_len exceeds the built-in capacity.  Calls on one GPU share the scratch: do not
    let two of them overlap."""
    d = score_qk_desc(q, k, span_begin, span_len, scale, softmax_span, out)
    st = lib().vscan_score_qk_static(C.byref(d), _stream())
    if st != OK:
        raise VScanError(st, "vscan_score_qk_static")
    return out


def vscan_select_global_local(scores_global, scores_local, frames, grid_h, grid_w, win_h, win_w,
                              k_per_window, k_global, out=None, want_mask=False):
    """Sec. 4.1 selection.  -> kept_idx [B', K1] int32 ascending (and the optional uint8 mask)."""
    B = scores_global.shape[0]
    windows = frames * (grid_h // max(win_h, 1)) * (grid_w // max(win_w, 1))
    k1 = windows * k_per_window + k_global
    if out is None:
        out = torch.empty((B, max(k1, 0)), dtype=torch.int32, device=scores_global.device)
    mask = torch.empty((B, frames * grid_h * grid_w), dtype=torch.uint8, device=out.device) if want_mask else None
    d = SelectDesc(scores_global=_ptr(scores_global), scores_local=_ptr(scores_local), instances=B,
                   frames=frames, grid_h=grid_h, grid_w=grid_w, win_h=win_h, win_w=win_w,
                   k_per_window=k_per_window, k_global=k_global, kept_idx=_ptr(out), kept_mask=_ptr(mask))
    st = lib().vscan_select_global_local(C.byref(d), None, 0, _stream())
    if st != OK:
        raise VScanError(st, "vscan_select_global_local")
    return (out, mask) if want_mask else out


def vscan_score_select(attn_global, attn_local, cls_offset, frames, grid_h, grid_w, win_h, win_w, k_per_window,
                       k_global, out=None, scores_global=None, scores_local=None):
    """Eq. 2 + Eq. 3 in one launch: head means of the two attention tensors and the selection.
    -> kept_idx [B', K1] int32.  scores_global / scores_local, if given, receive the head means."""
    B, H, L = attn_global.shape
    windows = frames * (grid_h // max(win_h, 1)) * (grid_w // max(win_w, 1))
    k1 = windows * k_per_window + k_global
    if out is None:
        out = torch.empty((B, max(k1, 0)), dtype=torch.int32, device=attn_global.device)
    sd = SelectDesc(scores_global=_ptr(scores_global), scores_local=_ptr(scores_local), instances=B, frames=frames,
                    grid_h=grid_h, grid_w=grid_w, win_h=win_h, win_w=win_w, k_per_window=k_per_window,
                    k_global=k_global, kept_idx=_ptr(out), kept_mask=None)
    d = ScoreSelectDesc(dtype=_dtype_code(attn_global), attn_global=_ptr(attn_global), attn_local=_ptr(attn_local),
                        heads=H, row_len=L, cls_offset=cls_offset, select=sd)
    st = lib().vscan_score_select(C.byref(d), _stream())
    if st != OK:
        raise VScanError(st, "vscan_score_select")
    return out


def vscan_merge(x, cls_offset, kept_idx, n_tokens=None, metric=None, path=MERGE_AUTO, out=None,
                want_assign=False, want_counts=False, workspace=None):
    """Eq. 4.  x [B', L, D], kept_idx [B', K1] -> merged [B', K1, D] (+ assign, counts)."""
    B, L, D = x.shape
    n = L - cls_offset if n_tokens is None else n_tokens
    K1 = kept_idx.shape[1]
    if out is None:
        out = torch.empty((B, K1, D), dtype=x.dtype, device=x.device)
    assign = torch.empty((B, n), dtype=torch.int32, device=x.device) if want_assign else None
    counts = torch.empty((B, K1), dtype=torch.int32, device=x.device) if want_counts else None
    d = MergeDesc(dtype=_dtype_code(x), path=path, x=_ptr(x), metric=_ptr(metric), kept_idx=_ptr(kept_idx),
                  instances=B, row_len=L, cls_offset=cls_offset, n_tokens=n, dim=D,
                  metric_dim=0 if metric is None else metric.shape[2], n_kept=K1, merged=_ptr(out),
                  assign=_ptr(assign), counts=_ptr(counts))
    _call("vscan_merge", d, "vscan_merge_workspace_bytes", workspace)
    res = [out]
    if want_assign:
        res.append(assign)
    if want_counts:
        res.append(counts)
    return res[0] if len(res) == 1 else tuple(res)


def vscan_llm_prune(q_last, k, v, hidden, pos_ids, n_sys, n_vis, n_txt, k_keep, scale,
                    softmax_span=SPAN_ONLY, want_scores=False, out=None, workspace=None):
    """Sec. 4.2.  Returns a dict with kept_vis, hidden, k, v, pos (and scores)."""
    B, Hq, d_ = q_last.shape
    Hkv = k.shape[1]
    S = n_sys + n_vis + n_txt
    So = S - n_vis + k_keep
    dev = k.device
    o = out or {}
    o.setdefault("kept_vis", torch.empty((B, k_keep), dtype=torch.int32, device=dev))
    o.setdefault("k", torch.empty((B, Hkv, So, d_), dtype=k.dtype, device=dev))
    if v is not None:
        o.setdefault("v", torch.empty((B, Hkv, So, d_), dtype=v.dtype, device=dev))
    if hidden is not None:
        o.setdefault("hidden", torch.empty((B, So, hidden.shape[2]), dtype=hidden.dtype, device=dev))
    if pos_ids is not None:
        o.setdefault("pos", torch.empty((pos_ids.shape[0], B, So), dtype=torch.int32, device=dev))
    if want_scores:
        o.setdefault("scores", torch.empty((B, n_vis), dtype=torch.float32, device=dev))
    desc = PruneDesc(dtype=_dtype_code(k), q_last=_ptr(q_last), k=_ptr(k), v=_ptr(v), hidden=_ptr(hidden),
                     pos_ids=_ptr(pos_ids), batch=B, q_heads=Hq, kv_heads=Hkv, head_dim=d_,
                     hidden_dim=0 if hidden is None else hidden.shape[2],
                     pos_planes=0 if pos_ids is None else pos_ids.shape[0], n_sys=n_sys, n_vis=n_vis,
                     n_txt=n_txt, k_keep=k_keep, softmax_span=softmax_span, scale=scale,
                     kept_vis=_ptr(o["kept_vis"]), hidden_out=_ptr(o.get("hidden")), k_out=_ptr(o["k"]),
                     v_out=_ptr(o.get("v")), pos_out=_ptr(o.get("pos")), scores=_ptr(o.get("scores")))
    _call("vscan_llm_prune", desc, "vscan_llm_prune_workspace_bytes", workspace)
    return o


# ------------------------------------------------------------------------------------------ ragged batches
def _host_i32(values):
    return (C.c_int32 * len(values))(*[int(v) for v in values])


def _host_i64(values):
    return (C.c_int64 * len(values))(*[int(v) for v in values])


def _aligned_offsets(sizes, align_elems):
    """Element offsets of consecutive blocks, each block starting on a multiple of `align_elems`."""
    offs, cur = [], 0
    for n in sizes:
        cur = -(-cur // align_elems) * align_elems
        offs.append(cur)
        cur += int(n)
    return offs, cur


def vscan_stage1_ragged(attn_g_list, attn_l_list, x_list, cls_offset, grids, win_h, win_w, k_per_window, k_global,
                        path=MERGE_AUTO, workspace=None):
    """Stage 1 for instances of different sizes in one library call.  attn_*_list[i]: [H, c + N_i], x_list[i]:
    [c + N_i, D] (CUDA tensors); grids[i] = (frames, grid_h, grid_w); k_per_window / k_global: per-instance lists.
    Packs the inputs (argument marshalling only) and returns ([kept_idx_i], [merged_i]) as views of the packed
    outputs, plus the workspace (for vscan_check)."""
    n = len(x_list)
    dt, dev = x_list[0].dtype, x_list[0].device
    e_align = 16 // x_list[0].element_size()
    H, D = attn_g_list[0].shape[0], x_list[0].shape[1]
    a_off, a_total = _aligned_offsets([t.numel() for t in attn_g_list], e_align)
    x_off, x_total = _aligned_offsets([t.numel() for t in x_list], e_align)
    k1 = [f * (gh // win_h) * (gw // win_w) * kw + kg for (f, gh, gw), kw, kg in zip(grids, k_per_window, k_global)]
    # kept lists are int32 (4 per 16 bytes); merged rows start at kept_offset * D, so 4-entry alignment covers both
    k_off, k_total = _aligned_offsets(k1, 4 if (4 * D * x_list[0].element_size()) % 16 == 0 else 16)
    ag = torch.zeros(a_total, dtype=dt, device=dev)
    al = torch.zeros(a_total, dtype=dt, device=dev)
    x = torch.zeros(x_total, dtype=dt, device=dev)
    for i in range(n):
        ag[a_off[i]:a_off[i] + attn_g_list[i].numel()] = attn_g_list[i].reshape(-1)
        al[a_off[i]:a_off[i] + attn_l_list[i].numel()] = attn_l_list[i].reshape(-1)
        x[x_off[i]:x_off[i] + x_list[i].numel()] = x_list[i].reshape(-1)
    kept = torch.full((max(k_total, 1),), -1, dtype=torch.int32, device=dev)
    merged = torch.zeros((max(k_total, 1) * D,), dtype=dt, device=dev)
    keep_alive = [_host_i32([g[0] for g in grids]), _host_i32([g[1] for g in grids]), _host_i32([g[2] for g in grids]),
                  _host_i32(k_per_window), _host_i32(k_global), _host_i64(a_off), _host_i64(x_off), _host_i64(k_off)]
    d = Stage1RaggedDesc(dtype=_dtype_code(x), merge_path=path, instances=n, heads=H, cls_offset=cls_offset, dim=D,
                         win_h=win_h, win_w=win_w, attn_global=_ptr(ag), attn_local=_ptr(al), x=_ptr(x),
                         kept_idx=_ptr(kept), merged=_ptr(merged), frames=keep_alive[0], grid_h=keep_alive[1],
                         grid_w=keep_alive[2], k_per_window=keep_alive[3], k_global=keep_alive[4],
                         attn_offset=keep_alive[5], x_offset=keep_alive[6], kept_offset=keep_alive[7])
    workspace = _call("vscan_stage1_ragged", d, "vscan_stage1_ragged_workspace_bytes", workspace)
    kept_views = [kept[k_off[i]:k_off[i] + k1[i]] for i in range(n)]
    merged_views = [merged[k_off[i] * D:(k_off[i] + k1[i]) * D].view(k1[i], D) for i in range(n)]
    return kept_views, merged_views, workspace


def vscan_llm_prune_ragged(q_last, k_list, v_list, hidden_list, pos_list, n_sys, n_vis, n_txt, k_keep, scale,
                           softmax_span=SPAN_ONLY, workspace=None):
    """Stage 2 for sequences of different lengths in one library call.  q_last [B, Hq, d]; k_list[i], v_list[i]:
    [Hkv, S_i, d]; hidden_list[i]: [S_i, Dh]; pos_list[i]: [S_i] int32; n_sys .. k_keep: per-sequence lists.
    Returns a list of dicts (kept_vis, hidden, k, v, pos) of views into the packed outputs, plus the workspace."""
    B, Hq, d_ = q_last.shape
    Hkv, Dh = k_list[0].shape[0], hidden_list[0].shape[1]
    dt, dev = k_list[0].dtype, k_list[0].device
    e_align = 16 // k_list[0].element_size()
    S = [a + b + c for a, b, c in zip(n_sys, n_vis, n_txt)]
    So = [s - b + kk for s, b, kk in zip(S, n_vis, k_keep)]
    kv_off, kv_total = _aligned_offsets([Hkv * s * d_ for s in S], e_align)
    kvo_off, kvo_total = _aligned_offsets([Hkv * s * d_ for s in So], e_align)
    h_off, h_total = _aligned_offsets([s * Dh for s in S], e_align)
    ho_off, ho_total = _aligned_offsets([s * Dh for s in So], e_align)
    p_off, p_total = _aligned_offsets(S, 4)
    po_off, po_total = _aligned_offsets(So, 4)
    kp_off, kp_total = _aligned_offsets(k_keep, 4)
    k = torch.zeros(kv_total, dtype=dt, device=dev); v = torch.zeros(kv_total, dtype=dt, device=dev)
    hidden = torch.zeros(h_total, dtype=dt, device=dev); pos = torch.zeros(p_total, dtype=torch.int32, device=dev)
    for i in range(B):
        k[kv_off[i]:kv_off[i] + k_list[i].numel()] = k_list[i].reshape(-1)
        v[kv_off[i]:kv_off[i] + v_list[i].numel()] = v_list[i].reshape(-1)
        hidden[h_off[i]:h_off[i] + hidden_list[i].numel()] = hidden_list[i].reshape(-1)
        pos[p_off[i]:p_off[i] + S[i]] = pos_list[i]
    k_out = torch.zeros(max(kvo_total, 1), dtype=dt, device=dev); v_out = torch.zeros(max(kvo_total, 1), dtype=dt, device=dev)
    h_out = torch.zeros(max(ho_total, 1), dtype=dt, device=dev); pos_out = torch.zeros(max(po_total, 1), dtype=torch.int32, device=dev)
    kept = torch.full((max(kp_total, 1),), -1, dtype=torch.int32, device=dev)
    keep_alive = [_host_i32(n_sys), _host_i32(n_vis), _host_i32(n_txt), _host_i32(k_keep), _host_i64(kv_off),
                  _host_i64(kvo_off), _host_i64(h_off), _host_i64(ho_off), _host_i64(p_off), _host_i64(po_off),
                  _host_i64(kp_off)]
    desc = PruneRaggedDesc(dtype=_dtype_code(k), batch=B, q_heads=Hq, kv_heads=Hkv, head_dim=d_, hidden_dim=Dh,
                           pos_planes=1, softmax_span=softmax_span, scale=scale, q_last=_ptr(q_last), k=_ptr(k), v=_ptr(v),
                           hidden=_ptr(hidden), pos_ids=_ptr(pos), kept_vis=_ptr(kept), hidden_out=_ptr(h_out),
                           k_out=_ptr(k_out), v_out=_ptr(v_out), pos_out=_ptr(pos_out), n_sys=keep_alive[0],
                           n_vis=keep_alive[1], n_txt=keep_alive[2], k_keep=keep_alive[3], kv_offset=keep_alive[4],
                           kv_out_offset=keep_alive[5], hidden_offset=keep_alive[6], hidden_out_offset=keep_alive[7],
                           pos_offset=keep_alive[8], pos_out_offset=keep_alive[9], kept_offset=keep_alive[10])
    workspace = _call("vscan_llm_prune_ragged", desc, "vscan_llm_prune_ragged_workspace_bytes", workspace)
    outs = []
    for i in range(B):
        outs.append({"kept_vis": kept[kp_off[i]:kp_off[i] + k_keep[i]],
                     "k": k_out[kvo_off[i]:kvo_off[i] + Hkv * So[i] * d_].view(Hkv, So[i], d_),
                     "v": v_out[kvo_off[i]:kvo_off[i] + Hkv * So[i] * d_].view(Hkv, So[i], d_),
                     "hidden": h_out[ho_off[i]:ho_off[i] + So[i] * Dh].view(So[i], Dh),
                     "pos": pos_out[po_off[i]:po_off[i] + So[i]]})
    return outs, workspace


def profile_begin(capacity: int = 4096):
    st = lib().vscan_profile_begin(capacity)
    if st != OK:
        raise VScanError(st, "vscan_profile_begin")


def profile_end(capacity: int = 4096):
    """-> list of (kernel name, milliseconds) in launch order."""
    names = C.create_string_buffer(capacity * 32)
    ms = (C.c_float * capacity)()
    n = lib().vscan_profile_end(names, ms, capacity)
    if n < 0:
        raise VScanError(ERR_INVALID_ARG, "vscan_profile_end")
    raw = names.raw
    return [(raw[i * 32:(i + 1) * 32].split(b"\0", 1)[0].decode(), float(ms[i])) for i in range(n)]


def fma_rate_tflops(blocks: int = 148 * 16, iters: int = 1 << 15, repeats: int = 5) -> float:
    """Measured fp32 FMA rate of the GPU in TFLOP/s (best of `repeats` launches of vscan_selftest_fma_rate)."""
    scratch = torch.empty(blocks * 256, dtype=torch.float32, device="cuda")
    flops = C.c_double(0.0)
    best = 0.0
    for _ in range(repeats + 1):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        st = lib().vscan_selftest_fma_rate(scratch.data_ptr(), scratch.numel(), blocks, iters, C.byref(flops), _stream())
        e1.record()
        if st != OK:
            raise VScanError(st, "vscan_selftest_fma_rate")
        e1.synchronize()
        best = max(best, flops.value / (e0.elapsed_time(e1) * 1e-3) / 1e12)
    return best


def vscan_check(workspace: Workspace) -> int:
    return int(lib().vscan_check(workspace.ptr, _stream()))


def vscan_selftest_bounded_wait(workspace: Workspace, polls: int = 2000) -> None:
    """One CTA waits `polls` polls on a flag nothing sets; vscan_check(workspace) then reports the timeout."""
    workspace.reserve(512)
    st = lib().vscan_selftest_bounded_wait(workspace.ptr, C.c_size_t(workspace.buf.numel()), C.c_uint32(polls), _stream())
    if st != 0:
        raise VScanError(st, "vscan_selftest_bounded_wait")
