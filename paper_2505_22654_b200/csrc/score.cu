// vscan_score: head-mean of attention rows (ROW mode, Eq. 2) and of softmax(q.K) (QK mode, Eq. 5).
#include "score.cuh"

namespace vscan {

// ROW mode.  grid = (ceil(n_tokens / blockDim), instances); one thread per token, heads ascending.
template <typename T>
__global__ void __launch_bounds__(256) row_mean_kernel(const T* __restrict__ attn, float* __restrict__ scores,
                                                       int heads, int row_len, int cls_offset, int n_tokens) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n_tokens) return;
  const T* base = attn + static_cast<size_t>(blockIdx.y) * heads * row_len + cls_offset + j;
  float acc = 0.f;
  int h = 0;
  for (; h + 8 <= heads; h += 8) {   // eight independent loads in flight, added in head order
    float a[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) a[u] = to_float(base[static_cast<size_t>(h + u) * row_len]);
#pragma unroll
    for (int u = 0; u < 8; ++u) acc += a[u];
  }
  for (; h < heads; ++h) acc += to_float(base[static_cast<size_t>(h) * row_len]);
  scores[static_cast<size_t>(blockIdx.y) * n_tokens + j] = acc / static_cast<float>(heads);
}

template <typename T>
static vscan_status launch_qk_typed(const QkParams& p, int batch, size_t smem, cudaStream_t stream) {
  constexpr int E = Vec16<T>::kElems;
  dim3 grid(p.q_heads, batch);
  const int vecs = p.head_dim / E;
  // small CTAs keep every (head, sequence) pair of a typical batch resident at once; the top-k tail
  // needs at most 64 keys per thread
  const int threads = p.span_len <= 8192 ? 128 : 256;
#define VSCAN_QK_CASE(VPS)                                                                          \
  do {                                                                                              \
    VSCAN_CUDA_TRY(allow_smem(qk_softmax_kernel<T, VPS>, smem));                                    \
    VSCAN_LAUNCH("qk_softmax", stream, (qk_softmax_kernel<T, VPS><<<grid, threads, smem, stream>>>(p))); \
    return VSCAN_OK;                                                                                \
  } while (0)
  if (vecs == 16) VSCAN_QK_CASE(2);
  if (vecs == 32) VSCAN_QK_CASE(4);
  if (vecs == 8) VSCAN_QK_CASE(1);
  VSCAN_QK_CASE(0);
#undef VSCAN_QK_CASE
}

vscan_status launch_qk_softmax(int dtype, const QkParams& p, int batch, cudaStream_t stream) {
  const size_t smem = qk_smem_bytes(p.head_dim, p.soft_n);
  if (smem > kMaxDynamicSmem) return VSCAN_ERR_UNSUPPORTED;
  if (batch > 65535) return VSCAN_ERR_UNSUPPORTED;
  return dtype == VSCAN_F32 ? launch_qk_typed<float>(p, batch, smem, stream)
                            : launch_qk_typed<__nv_bfloat16>(p, batch, smem, stream);
}

}  // namespace vscan

namespace vscan {

// Argument checks shared by vscan_score and vscan_score_qk_static.  Shape limits of this build are refused
// here (VSCAN_ERR_UNSUPPORTED), before anything is enqueued.
vscan_status validate_score(const vscan_score_desc* d) {
  if (!d || !d->scores) return VSCAN_ERR_INVALID_ARG;
  if (d->dtype != VSCAN_F32 && d->dtype != VSCAN_BF16) return VSCAN_ERR_INVALID_ARG;
  if (!aligned16(d->scores)) return VSCAN_ERR_INVALID_ARG;
  const size_t e = dtype_bytes(d->dtype);
  if (d->mode == VSCAN_SCORE_ROW) {
    if (!d->attn || !aligned16(d->attn)) return VSCAN_ERR_INVALID_ARG;
    if (d->instances < 0 || d->heads <= 0 || d->n_tokens < 0 || d->cls_offset < 0 ||
        static_cast<long long>(d->row_len) < static_cast<long long>(d->cls_offset) + d->n_tokens)
      return VSCAN_ERR_INVALID_ARG;
    if (d->instances > 65535) return VSCAN_ERR_UNSUPPORTED;
    if (overlaps(d->scores, static_cast<size_t>(d->instances) * d->n_tokens * 4, d->attn,
                 static_cast<size_t>(d->instances) * d->heads * d->row_len * e))
      return VSCAN_ERR_INVALID_ARG;
    return VSCAN_OK;
  }
  if (d->mode == VSCAN_SCORE_QK) {
    if (!d->q || !d->k || !aligned16(d->q) || !aligned16(d->k)) return VSCAN_ERR_INVALID_ARG;
    if (d->batch < 0 || d->q_heads <= 0 || d->kv_heads <= 0 || d->q_heads % d->kv_heads ||
        d->seq_len <= 0 || d->head_dim <= 0 || d->span_begin < 0 || d->span_len < 0 ||
        static_cast<long long>(d->span_begin) + d->span_len > static_cast<long long>(d->seq_len))
      return VSCAN_ERR_INVALID_ARG;
    if (d->softmax_span != VSCAN_SPAN_ONLY && d->softmax_span != VSCAN_SPAN_FULL)
      return VSCAN_ERR_INVALID_ARG;
    if (d->head_dim % 8 || d->head_dim > 256) return VSCAN_ERR_INVALID_ARG;
    if (d->batch > 65535) return VSCAN_ERR_UNSUPPORTED;
    const int soft_n = d->softmax_span == VSCAN_SPAN_ONLY ? d->span_len : d->seq_len;
    if (qk_smem_bytes(d->head_dim, soft_n) > kMaxDynamicSmem) return VSCAN_ERR_UNSUPPORTED;
    if (overlaps(d->scores, static_cast<size_t>(d->batch) * d->span_len * 4, d->k,
                 static_cast<size_t>(d->batch) * d->kv_heads * d->seq_len * d->head_dim * e) ||
        overlaps(d->scores, static_cast<size_t>(d->batch) * d->span_len * 4, d->q,
                 static_cast<size_t>(d->batch) * d->q_heads * d->head_dim * e))
      return VSCAN_ERR_INVALID_ARG;
    return VSCAN_OK;
  }
  if (d->mode == VSCAN_SCORE_RECEIVED) {
    if (!d->q || !d->k || !aligned16(d->q) || !aligned16(d->k)) return VSCAN_ERR_INVALID_ARG;
    if (d->head_rows && !aligned16(d->head_rows)) return VSCAN_ERR_INVALID_ARG;
    if (d->batch < 0 || d->q_heads <= 0 || d->kv_heads != d->q_heads || d->seq_len <= 0 || d->head_dim <= 0 || d->head_dim % 8)
      return VSCAN_ERR_INVALID_ARG;
    if (1ll * d->batch * d->q_heads > 65535) return VSCAN_ERR_UNSUPPORTED;
    if (!received_supported(d)) return VSCAN_ERR_UNSUPPORTED;   // bf16, head_dim 64 or 128
    const size_t qk = static_cast<size_t>(d->batch) * d->q_heads * d->seq_len * d->head_dim * e;
    const size_t rows = static_cast<size_t>(d->batch) * d->q_heads * d->seq_len * 4, sc = static_cast<size_t>(d->batch) * d->seq_len * 4;
    if (overlaps(d->scores, sc, d->q, qk) || overlaps(d->scores, sc, d->k, qk) || overlaps(d->head_rows, rows, d->q, qk) ||
        overlaps(d->head_rows, rows, d->k, qk) || overlaps(d->head_rows, rows, d->scores, sc))
      return VSCAN_ERR_INVALID_ARG;
    return VSCAN_OK;
  }
  return VSCAN_ERR_INVALID_ARG;
}

}  // namespace vscan

using namespace vscan;

extern "C" size_t vscan_score_workspace_bytes(const vscan_score_desc* d) {
  if (d && d->mode == VSCAN_SCORE_RECEIVED && d->batch > 0 && d->q_heads > 0 && d->seq_len > 0) return received_workspace_bytes(d);
  if (!d || d->mode != VSCAN_SCORE_QK || d->batch <= 0 || d->q_heads <= 0 || d->span_len <= 0) return 0;
  return kStatusBytes + round_up(static_cast<size_t>(d->batch) * sizeof(int), 256) +
         round_up(static_cast<size_t>(d->batch) * d->q_heads * d->span_len * sizeof(float), 256);
}

extern "C" vscan_status vscan_score(const vscan_score_desc* d, void* workspace, size_t workspace_bytes,
                                    void* stream_) {
  if (d && ((d->mode == VSCAN_SCORE_ROW && d->instances == 0) || ((d->mode == VSCAN_SCORE_QK || d->mode == VSCAN_SCORE_RECEIVED) && d->batch == 0)))
    return VSCAN_OK;  // empty batch: nothing to read or write
  vscan_status st = validate_score(d);
  if (st != VSCAN_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (d->mode == VSCAN_SCORE_ROW) {
    if (d->instances == 0 || d->n_tokens == 0) return VSCAN_OK;
    dim3 grid((d->n_tokens + 255) / 256, d->instances);
    if (d->dtype == VSCAN_F32)
      VSCAN_LAUNCH("row_mean", stream,
                   row_mean_kernel<float><<<grid, 256, 0, stream>>>(static_cast<const float*>(d->attn), d->scores,
                                                                    d->heads, d->row_len, d->cls_offset, d->n_tokens));
    else
      VSCAN_LAUNCH("row_mean", stream,
                   row_mean_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(
                       static_cast<const __nv_bfloat16*>(d->attn), d->scores, d->heads, d->row_len, d->cls_offset,
                       d->n_tokens));
    return VSCAN_OK;
  }
  if (d->mode == VSCAN_SCORE_RECEIVED) {
    const size_t need = vscan_score_workspace_bytes(d);
    if (!workspace || !aligned256(workspace) || workspace_bytes < need) return VSCAN_ERR_WORKSPACE;
    const size_t bh = static_cast<size_t>(d->batch) * d->q_heads;
    float* rows = d->head_rows ? d->head_rows
                               : reinterpret_cast<float*>(static_cast<char*>(workspace) + kStatusBytes +
                                                          round_up(bh * round_up(d->seq_len, 128) * sizeof(float), 256));
    st = launch_received(d, workspace, rows, stream);
    if (st != VSCAN_OK) return st;
    // Eq. 2 on the per-head rows
    dim3 grid((d->seq_len + 255) / 256, d->batch);
    VSCAN_LAUNCH("row_mean", stream,
                 row_mean_kernel<float><<<grid, 256, 0, stream>>>(rows, d->scores, d->q_heads, d->seq_len, 0, d->seq_len));
    return VSCAN_OK;
  }
  if (d->batch == 0 || d->span_len == 0) return VSCAN_OK;
  const size_t need = vscan_score_workspace_bytes(d);
  if (!workspace || !aligned256(workspace) || workspace_bytes < need) return VSCAN_ERR_WORKSPACE;
  // workspace: status word | per-sequence arrival counters | per-head probabilities
  char* ws = static_cast<char*>(workspace);
  const size_t counter_bytes = round_up(static_cast<size_t>(d->batch) * sizeof(int), 256);
  QkParams p;
  p.q = d->q; p.k = d->k;
  p.status = static_cast<uint32_t*>(workspace);
  p.counters = reinterpret_cast<int*>(ws + kStatusBytes);
  p.probs = reinterpret_cast<float*>(ws + kStatusBytes + counter_bytes);
  p.scores = d->scores;
  p.q_heads = d->q_heads; p.kv_heads = d->kv_heads; p.seq_len = d->seq_len; p.head_dim = d->head_dim;
  p.span_begin = d->span_begin; p.span_len = d->span_len; p.scale = d->scale;
  if (d->softmax_span == VSCAN_SPAN_ONLY) { p.soft_lo = d->span_begin; p.soft_n = d->span_len; }
  else { p.soft_lo = 0; p.soft_n = d->seq_len; }
  VSCAN_CUDA_TRY(cudaMemsetAsync(p.counters, 0, counter_bytes, stream));
  st = launch_qk_softmax(d->dtype, p, d->batch, stream);
  if (st != VSCAN_OK) return st;
  return VSCAN_OK;
}
