"""VScan two-stage visual-token reduction for NVIDIA B200 (sm_100a).

Thin Python face of libvscan.so (see include/vscan.h).  Every step runs in the library's CUDA
kernels; torch is used for device memory and streams only.  Importing this package does not load
the shared library; the first call does, and raises if it cannot.
"""
from .binding import (BF16, F32, MERGE_AUTO, MERGE_CLUSTER, MERGE_INTERLEAVED, MERGE_SIMT, MERGE_TENSOR, SPAN_FULL, SPAN_ONLY, VScanError,
                      Workspace, kernel_launches, lib, status_string, vscan_check, vscan_llm_prune, vscan_llm_prune_ragged, vscan_selftest_bounded_wait,
                      vscan_stage1_ragged,
                      vscan_merge, vscan_score_qk, vscan_score_qk_static, vscan_score_received, vscan_score_row, vscan_score_select,
                      vscan_select_global_local)
from .pipeline import VScanReducer

__all__ = ["BF16", "F32", "MERGE_AUTO", "MERGE_CLUSTER", "MERGE_INTERLEAVED", "MERGE_SIMT", "MERGE_TENSOR", "SPAN_FULL", "SPAN_ONLY",
           "VScanError", "Workspace", "kernel_launches", "lib", "status_string", "vscan_check", "vscan_selftest_bounded_wait",
           "vscan_llm_prune", "vscan_llm_prune_ragged", "vscan_stage1_ragged", "vscan_merge", "vscan_score_qk", "vscan_score_qk_static", "vscan_score_received", "vscan_score_row", "vscan_score_select",
           "vscan_select_global_local", "VScanReducer"]
