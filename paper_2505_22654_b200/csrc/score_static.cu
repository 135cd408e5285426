// vscan_score_qk_static: the QK-mode score (Eq. 5 arithmetic, unchanged) for callers that cannot
// hand over a workspace because they cannot allocate device memory at all.  Its scratch, the per-head
// probabilities, lives in a fixed array that is part of the loaded library image on every GPU.
#include <mutex>

#include "score.cuh"

namespace vscan {

// Capacity of the built-in scratch: batch * q_heads * span_len floats.  4 MiB per GPU, held from the
// moment the library is loaded on that GPU until the process exits.
constexpr size_t kStaticProbFloats = size_t(1) << 20;
static __device__ __align__(256) float g_static_probs[kStaticProbFloats];

// In host code `g_static_probs` is only a handle for the runtime, not a device address, so the address
// is asked for once per device and cached here.
constexpr int kMaxDevices = 64;
static std::mutex g_static_mutex;
static float* g_static_ptr[kMaxDevices] = {};

static vscan_status static_scratch(float** out) {
  int dev = -1;
  VSCAN_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return VSCAN_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_ptr[dev]) {
    void* ptr = nullptr;
    VSCAN_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_probs));
    g_static_ptr[dev] = static_cast<float*>(ptr);
  }
  *out = g_static_ptr[dev];
  return VSCAN_OK;
}

// scores[b][j] = (1/q_heads) * sum_h probs[b][h][j], h ascending, reading the built-in scratch.
__global__ void __launch_bounds__(256) static_head_mean_kernel(float* __restrict__ scores, int q_heads, int span_len) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= span_len) return;
  const float* base = g_static_probs + static_cast<size_t>(blockIdx.y) * q_heads * span_len + j;
  float acc = 0.f;
  int h = 0;
  for (; h + 8 <= q_heads; h += 8) {   // eight independent loads in flight, added in head order
    float a[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) a[u] = base[static_cast<size_t>(h + u) * span_len];
#pragma unroll
    for (int u = 0; u < 8; ++u) acc += a[u];
  }
  for (; h < q_heads; ++h) acc += base[static_cast<size_t>(h) * span_len];
  scores[static_cast<size_t>(blockIdx.y) * span_len + j] = acc / static_cast<float>(q_heads);
}

}  // namespace vscan

using namespace vscan;

extern "C" size_t vscan_score_qk_static_capacity(void) { return kStaticProbFloats; }

extern "C" vscan_status vscan_score_qk_static(const vscan_score_desc* d, void* stream_) {
  if (!d || d->mode != VSCAN_SCORE_QK) return VSCAN_ERR_INVALID_ARG;
  if (d->batch == 0) return VSCAN_OK;
  // the built-in scratch has a fixed size: refuse anything that does not fit, before looking any further
  if (d->batch > 0 && d->q_heads > 0 && d->span_len > 0 &&
      static_cast<size_t>(d->batch) * d->q_heads * d->span_len > kStaticProbFloats)
    return VSCAN_ERR_UNSUPPORTED;
  vscan_status st = validate_score(d);   // the same checks as vscan_score, output/input overlap included
  if (st != VSCAN_OK) return st;
  if (d->span_len == 0) return VSCAN_OK;
  float* probs = nullptr;
  st = static_scratch(&probs);
  if (st != VSCAN_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  QkParams p;
  p.q = d->q; p.k = d->k; p.probs = probs; p.status = nullptr;
  p.q_heads = d->q_heads; p.kv_heads = d->kv_heads; p.seq_len = d->seq_len; p.head_dim = d->head_dim;
  p.span_begin = d->span_begin; p.span_len = d->span_len; p.scale = d->scale;
  if (d->softmax_span == VSCAN_SPAN_ONLY) { p.soft_lo = d->span_begin; p.soft_n = d->span_len; }
  else { p.soft_lo = 0; p.soft_n = d->seq_len; }
  // every float of the scratch that the second kernel reads is written by the first one in this same
  // call, so nothing has to be cleared even though the array still holds the previous call's values
  st = launch_qk_softmax(d->dtype, p, d->batch, stream);
  if (st != VSCAN_OK) return st;
  dim3 grid((d->span_len + 255) / 256, d->batch);
  VSCAN_LAUNCH("static_head_mean", stream,
               static_head_mean_kernel<<<grid, 256, 0, stream>>>(d->scores, d->q_heads, d->span_len));
  return VSCAN_OK;
}
