// Internal declarations of the merge step (Sec. 4.1 "Token Merging", Eq. 4).
#pragma once

#include "common.cuh"

namespace vscan {

struct MergeParams {
  const void* x;        // [instances][row_len][dim]
  const void* metric;   // [instances][row_len][metric_dim] (== x when no separate metric)
  const int32_t* kept;  // [instances][n_kept]
  float* inv_norm;      // [instances][n_kept]   1 / max(|m_kept|, 1e-12)       (workspace)
  int32_t* assign;      // [instances][n_tokens]                                  (workspace or output)
  void* merged;         // [instances][n_kept][dim]
  int32_t* counts;      // optional
  void* kept_packed;    // [instances][n_kept rounded up to 256, or to 16 when <= 256][metric_dim] copy of the kept rows   (workspace;
                        // feeds the tensor paths with plain tile loads: kept sets above 128, and the persistent path)
  int* counters;        // [instances + 1] counters of the persistent path                              (workspace)
  int32_t* order;       // [instances][n_tokens] tokens ordered by slot, long instances only            (workspace)
  int32_t* order_start; // [instances][n_kept + 1] segment starts of `order`                            (workspace)
  float2* partial;      // [2][instances][n_tokens] (value, slot) per share of the kept set, kept sets above 768 (workspace)
  int* tickets;         // [instances][ceil(n_tokens / 128)] shares of a tile that have finished                  (workspace)
  int clear_status;     // this launch resets the status word (first launch of a call)
  uint32_t* status;     // device status word
  int instances, row_len, cls_offset, n_tokens, dim, metric_dim, n_kept;
};

// Similarity contraction + arg-max on CUDA cores (fp32 FMA).  Works for both dtypes.
vscan_status launch_assign_simt(int dtype, const MergeParams& p, cudaStream_t stream);
// Same result on the tensor cores (bf16 only).  Returns VSCAN_ERR_UNSUPPORTED for shapes it
// cannot take.
vscan_status launch_assign_tensor(const MergeParams& p, cudaStream_t stream);
bool assign_tensor_supported(int dtype, const MergeParams& p);
// Tensor-core assignment and group means in one launch (bf16, kept sets small enough for two or three
// CTAs per SM): the mean CTAs of an instance follow its assignment CTAs in block order and re-read the
// features from L2.  Clears the status word and uses the inv_norm region of the workspace for counters.
vscan_status launch_merge_interleaved(const MergeParams& p, cudaStream_t stream);
bool merge_interleaved_supported(int dtype, const MergeParams& p);
// Group sums of Eq. 4 as one-hot matrix products on the tensor cores (bf16, at most 256 kept tokens, feature dim a
// multiple of 128, no unused rows after the last token).  Reads `assign`, writes merged / counts.
vscan_status launch_group_sum_tensor(const MergeParams& p, cudaStream_t stream);
bool group_sum_tensor_supported(int dtype, const MergeParams& p);

// Assignment and group sums in one pass over the features: a cluster of dim / 256 CTAs per instance exchanges partial
// dot products through distributed shared memory (bf16, at most 64 kept tokens, dim 256 / 512 / 1024, no separate metric).
vscan_status launch_merge_cluster(const MergeParams& p, cudaStream_t stream);
bool merge_cluster_supported(int dtype, const MergeParams& p);

}  // namespace vscan
