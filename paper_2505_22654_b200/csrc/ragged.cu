// Ragged batches: one call for instances (Stage 1) or sequences (Stage 2) of different sizes, as dynamic-resolution
// encoders produce them (Sec. 5.1 "Models": 4 to 16384 visual tokens per image).  Sizes and offsets are HOST arrays:
// the caller knows them from the image resolutions.  The library cuts the batch into runs of consecutive units with
// the same shape and regularly spaced blocks and hands every run to the uniform entry points, all on the caller's
// stream; a run gets its own slice of the workspace, and a last small kernel folds the runs' status words into the
// first word of the workspace, where vscan_check looks.
#include <vector>

#include "common.cuh"

namespace vscan {

__global__ void fold_status_kernel(uint32_t* main_word, const unsigned char* first, size_t stride, int runs) {
  uint32_t acc = 0;
  for (int r = threadIdx.x; r < runs; r += 32) acc |= *reinterpret_cast<const uint32_t*>(first + static_cast<size_t>(r) * stride);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc |= __shfl_xor_sync(0xffffffffu, acc, o);
  if (threadIdx.x == 0) *main_word = acc ? static_cast<uint32_t>(VSCAN_ERR_TIMEOUT) : 0u;
}

struct Run { int first, count; };

static long long tokens_of(const vscan_stage1_ragged_desc* d, int i) {
  return 1ll * d->frames[i] * d->grid_h[i] * d->grid_w[i];
}
static long long kept_of(const vscan_stage1_ragged_desc* d, int i) {
  const long long windows = 1ll * d->frames[i] * (d->grid_h[i] / d->win_h) * (d->grid_w[i] / d->win_w);
  return windows * d->k_per_window[i] + d->k_global[i];
}

static vscan_status stage1_runs(const vscan_stage1_ragged_desc* d, std::vector<Run>& runs) {
  if (!d || d->instances < 0) return VSCAN_ERR_INVALID_ARG;
  if (d->instances == 0) return VSCAN_OK;
  if (!d->frames || !d->grid_h || !d->grid_w || !d->k_per_window || !d->k_global || !d->attn_offset || !d->x_offset ||
      !d->kept_offset || d->win_h <= 0 || d->win_w <= 0 || d->heads <= 0 || d->dim <= 0 || d->cls_offset < 0)
    return VSCAN_ERR_INVALID_ARG;
  for (int i = 0; i < d->instances; ++i) {
    if (d->frames[i] <= 0 || d->grid_h[i] <= 0 || d->grid_w[i] <= 0 || d->grid_h[i] % d->win_h || d->grid_w[i] % d->win_w ||
        d->attn_offset[i] < 0 || d->x_offset[i] < 0 || d->kept_offset[i] < 0)
      return VSCAN_ERR_INVALID_ARG;
    const long long n = tokens_of(d, i), row = d->cls_offset + n;
    bool joins = false;
    if (!runs.empty()) {
      const int p = i - 1;
      joins = d->frames[p] == d->frames[i] && d->grid_h[p] == d->grid_h[i] && d->grid_w[p] == d->grid_w[i] &&
              d->k_per_window[p] == d->k_per_window[i] && d->k_global[p] == d->k_global[i] &&
              d->attn_offset[i] - d->attn_offset[p] == 1ll * d->heads * row && d->x_offset[i] - d->x_offset[p] == row * d->dim &&
              d->kept_offset[i] - d->kept_offset[p] == kept_of(d, i);
    }
    if (joins) ++runs.back().count;
    else runs.push_back({i, 1});
  }
  return VSCAN_OK;
}

// the uniform merge call of one run
static vscan_merge_desc merge_desc_of(const vscan_stage1_ragged_desc* d, const Run& r) {
  const int i = r.first;
  const size_t e = dtype_bytes(d->dtype);
  vscan_merge_desc m = {};
  m.dtype = d->dtype; m.path = d->merge_path;
  m.x = static_cast<const char*>(d->x) + d->x_offset[i] * e;
  m.kept_idx = d->kept_idx + d->kept_offset[i];
  m.instances = r.count; m.n_tokens = static_cast<int32_t>(tokens_of(d, i)); m.cls_offset = d->cls_offset;
  m.row_len = m.cls_offset + m.n_tokens; m.dim = d->dim; m.n_kept = static_cast<int32_t>(kept_of(d, i));
  m.merged = static_cast<char*>(d->merged) + d->kept_offset[i] * d->dim * e;
  return m;
}

static size_t stage1_stride(const vscan_stage1_ragged_desc* d, const std::vector<Run>& runs) {
  size_t stride = kStatusBytes;
  for (const Run& r : runs) {
    const vscan_merge_desc m = merge_desc_of(d, r);
    stride = std::max(stride, round_up(vscan_merge_workspace_bytes(&m), 256));
  }
  return stride;
}

struct Run2 { int first, count; };

static vscan_status stage2_runs(const vscan_prune_ragged_desc* d, std::vector<Run>& runs) {
  if (!d || d->batch < 0) return VSCAN_ERR_INVALID_ARG;
  if (d->batch == 0) return VSCAN_OK;
  if (!d->n_sys || !d->n_vis || !d->n_txt || !d->k_keep || !d->kv_offset || !d->kv_out_offset || !d->kept_offset ||
      d->q_heads <= 0 || d->kv_heads <= 0 || d->head_dim <= 0)
    return VSCAN_ERR_INVALID_ARG;
  if ((d->hidden != nullptr) != (d->hidden_out != nullptr) || (d->hidden && (!d->hidden_offset || !d->hidden_out_offset || d->hidden_dim <= 0)))
    return VSCAN_ERR_INVALID_ARG;
  if ((d->pos_ids != nullptr) != (d->pos_out != nullptr) || (d->pos_ids && (!d->pos_offset || !d->pos_out_offset || d->pos_planes != 1)))
    return VSCAN_ERR_INVALID_ARG;   // packed position ids are one plane per sequence block
  for (int i = 0; i < d->batch; ++i) {
    if (d->n_sys[i] < 0 || d->n_vis[i] < 0 || d->n_txt[i] < 0 || d->k_keep[i] < 0 || d->k_keep[i] > d->n_vis[i]) return VSCAN_ERR_INVALID_ARG;
    const long long S = 1ll * d->n_sys[i] + d->n_vis[i] + d->n_txt[i], So = S - d->n_vis[i] + d->k_keep[i];
    bool joins = false;
    if (!runs.empty()) {
      const int p = i - 1;
      joins = d->n_sys[p] == d->n_sys[i] && d->n_vis[p] == d->n_vis[i] && d->n_txt[p] == d->n_txt[i] && d->k_keep[p] == d->k_keep[i] &&
              d->kv_offset[i] - d->kv_offset[p] == 1ll * d->kv_heads * S * d->head_dim &&
              d->kv_out_offset[i] - d->kv_out_offset[p] == 1ll * d->kv_heads * So * d->head_dim &&
              d->kept_offset[i] - d->kept_offset[p] == d->k_keep[i] &&
              (!d->hidden || (d->hidden_offset[i] - d->hidden_offset[p] == S * d->hidden_dim &&
                              d->hidden_out_offset[i] - d->hidden_out_offset[p] == So * d->hidden_dim)) &&
              (!d->pos_ids || (d->pos_offset[i] - d->pos_offset[p] == S && d->pos_out_offset[i] - d->pos_out_offset[p] == So));
    }
    if (joins) ++runs.back().count;
    else runs.push_back({i, 1});
  }
  return VSCAN_OK;
}

static vscan_prune_desc prune_desc_of(const vscan_prune_ragged_desc* d, const Run& r) {
  const int i = r.first;
  const size_t e = dtype_bytes(d->dtype);
  vscan_prune_desc p = {};
  p.dtype = d->dtype;
  p.q_last = static_cast<const char*>(d->q_last) + static_cast<size_t>(i) * d->q_heads * d->head_dim * e;
  p.k = static_cast<const char*>(d->k) + d->kv_offset[i] * e;
  p.v = d->v ? static_cast<const char*>(d->v) + d->kv_offset[i] * e : nullptr;
  p.hidden = d->hidden ? static_cast<const char*>(d->hidden) + d->hidden_offset[i] * e : nullptr;
  p.pos_ids = d->pos_ids ? d->pos_ids + d->pos_offset[i] : nullptr;
  p.batch = r.count; p.q_heads = d->q_heads; p.kv_heads = d->kv_heads; p.head_dim = d->head_dim; p.hidden_dim = d->hidden_dim;
  p.pos_planes = d->pos_ids ? 1 : 0;
  p.n_sys = d->n_sys[i]; p.n_vis = d->n_vis[i]; p.n_txt = d->n_txt[i]; p.k_keep = d->k_keep[i];
  p.softmax_span = d->softmax_span; p.scale = d->scale;
  p.kept_vis = d->kept_vis ? d->kept_vis + d->kept_offset[i] : nullptr;
  p.hidden_out = d->hidden_out ? static_cast<char*>(d->hidden_out) + d->hidden_out_offset[i] * e : nullptr;
  p.k_out = static_cast<char*>(d->k_out) + d->kv_out_offset[i] * e;
  p.v_out = d->v_out ? static_cast<char*>(d->v_out) + d->kv_out_offset[i] * e : nullptr;
  p.pos_out = d->pos_out ? d->pos_out + d->pos_out_offset[i] : nullptr;
  return p;
}

static size_t stage2_stride(const vscan_prune_ragged_desc* d, const std::vector<Run>& runs) {
  size_t stride = kStatusBytes;
  for (const Run& r : runs) {
    const vscan_prune_desc p = prune_desc_of(d, r);
    stride = std::max(stride, round_up(vscan_llm_prune_workspace_bytes(&p), 256));
  }
  return stride;
}

}  // namespace vscan

using namespace vscan;

extern "C" size_t vscan_stage1_ragged_workspace_bytes(const vscan_stage1_ragged_desc* d) {
  std::vector<Run> runs;
  if (stage1_runs(d, runs) != VSCAN_OK || runs.empty()) return kStatusBytes;
  return kStatusBytes + runs.size() * stage1_stride(d, runs);
}

extern "C" vscan_status vscan_stage1_ragged(const vscan_stage1_ragged_desc* d, void* workspace, size_t workspace_bytes,
                                            void* stream_) {
  std::vector<Run> runs;
  vscan_status st = stage1_runs(d, runs);
  if (st != VSCAN_OK) return st;
  if (runs.empty()) return VSCAN_OK;
  if (d->dtype != VSCAN_F32 && d->dtype != VSCAN_BF16) return VSCAN_ERR_INVALID_ARG;
  if (!d->attn_global || !d->attn_local || !d->x || !d->kept_idx || !d->merged) return VSCAN_ERR_INVALID_ARG;
  const size_t stride = stage1_stride(d, runs);
  if (!workspace || !aligned256(workspace) || workspace_bytes < kStatusBytes + runs.size() * stride) return VSCAN_ERR_WORKSPACE;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const size_t e = dtype_bytes(d->dtype);
  // every run is checked before the first one is launched: on a validation error nothing is enqueued
  std::vector<vscan_score_select_desc> selects(runs.size());
  std::vector<vscan_merge_desc> merges(runs.size());
  for (size_t r = 0; r < runs.size(); ++r) {
    const int i = runs[r].first;
    vscan_score_select_desc& s = selects[r];
    s = vscan_score_select_desc{};
    s.dtype = d->dtype;
    s.attn_global = static_cast<const char*>(d->attn_global) + d->attn_offset[i] * e;
    s.attn_local = static_cast<const char*>(d->attn_local) + d->attn_offset[i] * e;
    s.heads = d->heads; s.cls_offset = d->cls_offset;
    s.row_len = static_cast<int32_t>(d->cls_offset + tokens_of(d, i));
    s.select.instances = runs[r].count; s.select.frames = d->frames[i]; s.select.grid_h = d->grid_h[i]; s.select.grid_w = d->grid_w[i];
    s.select.win_h = d->win_h; s.select.win_w = d->win_w; s.select.k_per_window = d->k_per_window[i]; s.select.k_global = d->k_global[i];
    s.select.kept_idx = d->kept_idx + d->kept_offset[i];
    merges[r] = merge_desc_of(d, runs[r]);
    if (tokens_of(d, i) > 16384) return VSCAN_ERR_UNSUPPORTED;
    if (kept_of(d, i) < 1 || kept_of(d, i) > tokens_of(d, i) || d->dim % 8) return VSCAN_ERR_INVALID_ARG;
    if (!aligned16(s.attn_global) || !aligned16(s.attn_local) || !aligned16(merges[r].x) || !aligned16(merges[r].kept_idx) ||
        !aligned16(merges[r].merged))
      return VSCAN_ERR_INVALID_ARG;   // every instance's blocks start on 16 bytes
  }
  char* ws = static_cast<char*>(workspace);
  for (size_t r = 0; r < runs.size(); ++r) {
    st = vscan_score_select(&selects[r], stream_);
    if (st != VSCAN_OK) return st;
    st = vscan_merge(&merges[r], ws + kStatusBytes + r * stride, stride, stream_);
    if (st != VSCAN_OK) return st;
  }
  VSCAN_LAUNCH("fold_status", stream,
               (fold_status_kernel<<<1, 32, 0, stream>>>(static_cast<uint32_t*>(workspace),
                                                         reinterpret_cast<const unsigned char*>(ws + kStatusBytes), stride,
                                                         static_cast<int>(runs.size()))));
  return VSCAN_OK;
}

extern "C" size_t vscan_llm_prune_ragged_workspace_bytes(const vscan_prune_ragged_desc* d) {
  std::vector<Run> runs;
  if (stage2_runs(d, runs) != VSCAN_OK || runs.empty()) return kStatusBytes;
  return kStatusBytes + runs.size() * stage2_stride(d, runs);
}

extern "C" vscan_status vscan_llm_prune_ragged(const vscan_prune_ragged_desc* d, void* workspace, size_t workspace_bytes,
                                               void* stream_) {
  std::vector<Run> runs;
  vscan_status st = stage2_runs(d, runs);
  if (st != VSCAN_OK) return st;
  if (runs.empty()) return VSCAN_OK;
  if (d->dtype != VSCAN_F32 && d->dtype != VSCAN_BF16) return VSCAN_ERR_INVALID_ARG;
  if (!d->q_last || !d->k || !d->k_out || (d->v == nullptr) != (d->v_out == nullptr)) return VSCAN_ERR_INVALID_ARG;
  const size_t stride = stage2_stride(d, runs);
  if (!workspace || !aligned256(workspace) || workspace_bytes < kStatusBytes + runs.size() * stride) return VSCAN_ERR_WORKSPACE;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  std::vector<vscan_prune_desc> descs(runs.size());
  for (size_t r = 0; r < runs.size(); ++r) {
    descs[r] = prune_desc_of(d, runs[r]);
    const vscan_prune_desc& p = descs[r];
    if (p.n_vis > 16384) return VSCAN_ERR_UNSUPPORTED;
    const void* ptrs[] = {p.q_last, p.k, p.v, p.hidden, p.pos_ids, p.kept_vis, p.hidden_out, p.k_out, p.v_out, p.pos_out};
    for (const void* ptr : ptrs)
      if (ptr && !aligned16(ptr)) return VSCAN_ERR_INVALID_ARG;   // every sequence's blocks start on 16 bytes
  }
  char* ws = static_cast<char*>(workspace);
  for (size_t r = 0; r < runs.size(); ++r) {
    st = vscan_llm_prune(&descs[r], ws + kStatusBytes + r * stride, stride, stream_);
    if (st != VSCAN_OK) return st;
  }
  VSCAN_LAUNCH("fold_status", stream,
               (fold_status_kernel<<<1, 32, 0, stream>>>(static_cast<uint32_t*>(workspace),
                                                         reinterpret_cast<const unsigned char*>(ws + kStatusBytes), stride,
                                                         static_cast<int>(runs.size()))));
  return VSCAN_OK;
}
