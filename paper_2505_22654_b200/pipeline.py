"""Chained Stage 1 + Stage 2 reduction with preallocated buffers (argument marshalling only).

`VScanReducer` owns the output tensors and workspaces for one fixed shape so that a pass makes no
allocation and can be captured in a CUDA graph.  `run_host` is the end-to-end form: inputs arrive
in pinned host memory, results are returned in pinned host memory.
"""
from __future__ import annotations

import torch

from . import binding as vb


class VScanReducer:
    def __init__(self, *, dtype, instances, frames, grid_h, grid_w, cls, D, H, win_h, win_w, k_w, k_g,
                 B, n_sys, n_vis, n_txt, Dh, Hq, Hkv, d, k2, pos_planes=1, scale=None,
                 softmax_span=vb.SPAN_ONLY, merge_path=vb.MERGE_AUTO, fused_select=True, overlap_stages=False,
                 run_stage1=True, device="cuda"):
        self.dtype = torch.float32 if dtype in ("f32", torch.float32) else torch.bfloat16
        self.instances, self.frames, self.grid_h, self.grid_w, self.cls = instances, frames, grid_h, grid_w, cls
        self.D, self.H, self.win_h, self.win_w, self.k_w, self.k_g = D, H, win_h, win_w, k_w, k_g
        self.N = frames * grid_h * grid_w
        self.L = self.N + cls
        self.W = frames * (grid_h // win_h) * (grid_w // win_w)
        self.K1 = k_g + self.W * k_w
        self.B, self.n_sys, self.n_vis, self.n_txt = B, n_sys, n_vis, n_txt
        self.Dh, self.Hq, self.Hkv, self.d, self.k2, self.P = Dh, Hq, Hkv, d, k2, pos_planes
        self.S = n_sys + n_vis + n_txt
        self.S_out = self.S - n_vis + k2
        self.scale = float(scale if scale is not None else d ** -0.5)
        self.softmax_span, self.merge_path, self.fused_select = softmax_span, merge_path, fused_select
        dev, dt = device, self.dtype
        self.scores_g = torch.empty((instances, self.N), dtype=torch.float32, device=dev)
        self.scores_l = torch.empty((instances, self.N), dtype=torch.float32, device=dev)
        self.kept_idx = torch.empty((instances, self.K1), dtype=torch.int32, device=dev)
        self.merged = torch.empty((instances, self.K1, D), dtype=dt, device=dev)
        self.out2 = {
            "kept_vis": torch.empty((B, k2), dtype=torch.int32, device=dev),
            "hidden": torch.empty((B, self.S_out, Dh), dtype=dt, device=dev),
            "k": torch.empty((B, Hkv, self.S_out, d), dtype=dt, device=dev),
            "v": torch.empty((B, Hkv, self.S_out, d), dtype=dt, device=dev),
            "pos": torch.empty((pos_planes, B, self.S_out), dtype=torch.int32, device=dev),
        }
        self.ws_merge = vb.Workspace(64 << 10, dev)
        self.ws_prune = vb.Workspace(64 << 10, dev)
        self.overlap_stages, self._side, self.run_stage1 = overlap_stages, None, run_stage1
        self._reserve()

    @classmethod
    def from_config(cls_, cfg, **kw):
        return cls_(dtype=cfg.dtype, instances=cfg.instances, frames=cfg.frames, grid_h=cfg.grid_h,
                    grid_w=cfg.grid_w, cls=cfg.cls, D=cfg.D, H=cfg.H, win_h=cfg.win_h, win_w=cfg.win_w,
                    k_w=cfg.k_w, k_g=cfg.k_g, B=cfg.B, n_sys=cfg.n_sys, n_vis=cfg.n_vis, n_txt=cfg.n_txt,
                    Dh=cfg.Dh, Hq=cfg.Hq, Hkv=cfg.Hkv, d=cfg.d, k2=cfg.k2, pos_planes=cfg.pos_planes, **kw)

    # ---- device-resident pass: the four library calls on the current stream
    def stage1(self, attn_g, attn_l, x):
        if self.fused_select:      # Eq. 2 and Eq. 3 in one launch; the head means are still written out
            vb.vscan_score_select(attn_g, attn_l, self.cls, self.frames, self.grid_h, self.grid_w, self.win_h,
                                  self.win_w, self.k_w, self.k_g, out=self.kept_idx, scores_global=self.scores_g,
                                  scores_local=self.scores_l)
        else:
            vb.vscan_score_row(attn_g, self.cls, self.N, out=self.scores_g)
            vb.vscan_score_row(attn_l, self.cls, self.N, out=self.scores_l)
            vb.vscan_select_global_local(self.scores_g, self.scores_l, self.frames, self.grid_h, self.grid_w,
                                         self.win_h, self.win_w, self.k_w, self.k_g, out=self.kept_idx)
        vb.vscan_merge(x, self.cls, self.kept_idx, n_tokens=self.N, path=self.merge_path, out=self.merged,
                       workspace=self.ws_merge)
        return self.merged

    def stage2(self, q_last, k, v, hidden, pos_ids):
        return vb.vscan_llm_prune(q_last, k, v, hidden, pos_ids, self.n_sys, self.n_vis, self.n_txt, self.k2,
                                  self.scale, self.softmax_span, out=self.out2, workspace=self.ws_prune)

    def run(self, attn_g, attn_l, x, q_last, k, v, hidden, pos_ids):
        if not self.run_stage1:      # schedules that prune inside the LLM only
            return self.stage2(q_last, k, v, hidden, pos_ids)
        if not self.overlap_stages:
            self.stage1(attn_g, attn_l, x)
            return self.stage2(q_last, k, v, hidden, pos_ids)
        # The two stages of one pass have no data in common (Stage 2 reads the LLM's layer-k tensors,
        # Stage 1 the encoder's), so they are enqueued as two branches that fork from and join back into
        # the current stream; captured in a CUDA graph they are two parallel branches of the one graph.
        # Stage 1 (a few hundred long-lived CTAs that leave DRAM half idle) goes to a high-priority stream,
        # so that its CTAs take SM slots as the thousands of short row-copy CTAs of Stage 2 retire.
        cur = torch.cuda.current_stream()
        if self._side is None:
            self._side = torch.cuda.Stream(device=self.merged.device, priority=-1)
        self._side.wait_stream(cur)
        with torch.cuda.stream(self._side):
            self.stage1(attn_g, attn_l, x)
        out = self.stage2(q_last, k, v, hidden, pos_ids)
        cur.wait_stream(self._side)
        return out

    def check(self) -> int:
        """Synchronises the current stream and reads the device status words of both workspaces: 0, or
        the status a bounded device-side wait left there (binding.ERR_TIMEOUT).  A pass that timed out has
        unwritten output rows, so callers that time or trust a pass call this after it."""
        used = [self.ws_prune] + ([self.ws_merge] if self.run_stage1 else [])   # an unused workspace holds no status
        return max(vb.vscan_check(w) for w in used)

    def _reserve(self):
        import ctypes as C
        L = vb.lib()
        code = vb.F32 if self.dtype == torch.float32 else vb.BF16
        md = vb.MergeDesc(dtype=code, instances=self.instances, n_kept=self.K1, n_tokens=self.N,
                          dim=self.D, row_len=self.L, cls_offset=self.cls)
        self.ws_merge.reserve(L.vscan_merge_workspace_bytes(C.byref(md)))
        pd = vb.PruneDesc(batch=self.B, q_heads=self.Hq, n_vis=self.n_vis)
        self.ws_prune.reserve(L.vscan_llm_prune_workspace_bytes(C.byref(pd)))

    # ---- end to end: pinned host buffers in, pinned host buffers out
    def run_host(self, host_in: dict, host_out: dict, dev_in: dict):
        """host_in / dev_in: same keys (attn_g, attn_l, x, q_last, k, v, hidden, pos_ids); host_out:
        merged, kept_vis, hidden, k, v, pos.  Copies in, runs the pass, copies out, all on the
        current stream; the caller synchronises."""
        for name, t in host_in.items():
            dev_in[name].copy_(t, non_blocking=True)
        self.run(**dev_in)
        host_out["merged"].copy_(self.merged, non_blocking=True)
        for name in ("kept_vis", "hidden", "k", "v", "pos"):
            host_out[name].copy_(self.out2[name], non_blocking=True)
        return host_out

    def run_host_many(self, host_ins, host_outs, dev_sets):
        """A stream of batches from pinned host memory: the upload of batch i+1 and the download of
        batch i-1 overlap the pass over batch i (three streams, `dev_sets` >= 2 device input sets used
        in turn; outputs are single-buffered, so a pass waits for the previous download).  Everything
        is enqueued asynchronously; the caller synchronises the current stream, which ends up ordered
        after the last download."""
        cur = torch.cuda.current_stream()
        if not hasattr(self, "_s_in"):
            self._s_in, self._s_out = torch.cuda.Stream(), torch.cuda.Stream()
        n_slots = len(dev_sets)
        ev_in = [torch.cuda.Event() for _ in range(n_slots)]
        ev_done = [None] * n_slots          # pass that last used the slot
        ev_out = None                       # last download
        self._s_in.wait_stream(cur)
        self._s_out.wait_stream(cur)
        for i, (hin, hout) in enumerate(zip(host_ins, host_outs)):
            slot = i % n_slots
            with torch.cuda.stream(self._s_in):
                if ev_done[slot] is not None:
                    self._s_in.wait_event(ev_done[slot])
                for name, t in hin.items():
                    dev_sets[slot][name].copy_(t, non_blocking=True)
                ev_in[slot].record(self._s_in)
            cur.wait_event(ev_in[slot])
            if ev_out is not None:
                cur.wait_event(ev_out)
            self.run(**dev_sets[slot])
            ev_done[slot] = torch.cuda.Event()
            ev_done[slot].record(cur)
            with torch.cuda.stream(self._s_out):
                self._s_out.wait_event(ev_done[slot])
                hout["merged"].copy_(self.merged, non_blocking=True)
                for name in ("kept_vis", "hidden", "k", "v", "pos"):
                    hout[name].copy_(self.out2[name], non_blocking=True)
                ev_out = torch.cuda.Event()
                ev_out.record(self._s_out)
        if ev_out is not None:
            cur.wait_event(ev_out)
        return host_outs
