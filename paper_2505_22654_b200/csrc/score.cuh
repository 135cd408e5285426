// Device code shared by vscan_score (QK mode) and vscan_llm_prune: Eq. 5.
#pragma once

#include "common.cuh"

namespace vscan {

struct QkParams {
  const void* q;     // [batch][q_heads][head_dim]
  const void* k;     // [batch][kv_heads][seq_len][head_dim]
  float* probs;      // [batch][q_heads][span_len]  per-head probabilities on the span (workspace)
  uint32_t* status;  // device status word of the workspace, cleared by the first CTA
  int q_heads, kv_heads, seq_len, head_dim, span_begin, span_len;
  int soft_lo, soft_n;  // keys the softmax runs over: [soft_lo, soft_lo + soft_n)
  float scale;
};

// One CTA per (query head, sequence).  Dynamic shared memory: q[head_dim] floats | z[soft_n] floats.
// Eight lanes share one key row (each lane 16-byte pieces, fp32 accumulate, 3 shuffles).
template <typename T>
__global__ void __launch_bounds__(256) qk_softmax_kernel(QkParams p) {
  extern __shared__ __align__(16) float smem_f[];
  float* qs = smem_f;
  float* z = smem_f + p.head_dim;
  __shared__ float red[33];
  constexpr int E = Vec16<T>::kElems;
  const int h = blockIdx.x, b = blockIdx.y;
  if (h == 0 && b == 0 && threadIdx.x == 0 && p.status) *p.status = 0u;
  const int g = static_cast<int>((static_cast<long long>(h) * p.kv_heads) / p.q_heads);
  const T* qh = static_cast<const T*>(p.q) + (static_cast<size_t>(b) * p.q_heads + h) * p.head_dim;
  for (int i = threadIdx.x; i < p.head_dim; i += blockDim.x) qs[i] = to_float(qh[i]);
  __syncthreads();

  const T* kb = static_cast<const T*>(p.k) +
                ((static_cast<size_t>(b) * p.kv_heads + g) * p.seq_len + p.soft_lo) * p.head_dim;
  const int vecs = p.head_dim / E;           // 16-byte pieces per key row
  const int sub = threadIdx.x & 7;           // lane within the 8-lane group
  const int grp = threadIdx.x >> 3, ngrp = blockDim.x >> 3;
  float local_max = -INFINITY;
  for (int j0 = 0; j0 < p.soft_n; j0 += ngrp) {   // uniform trip count: shuffles stay converged
    const int j = j0 + grp;
    float acc = 0.f;
    if (j < p.soft_n) {
      const uint4* row = reinterpret_cast<const uint4*>(kb + static_cast<size_t>(j) * p.head_dim);
      for (int v = sub; v < vecs; v += 8) {
        float kv[E];
        Vec16<T>::unpack(ld_nc_16(row + v), kv);
#pragma unroll
        for (int e = 0; e < E; ++e) acc = fmaf(kv[e], qs[v * E + e], acc);
      }
    }
    acc += __shfl_xor_sync(0xffffffffu, acc, 1);
    acc += __shfl_xor_sync(0xffffffffu, acc, 2);
    acc += __shfl_xor_sync(0xffffffffu, acc, 4);
    if (j < p.soft_n) {
      acc *= p.scale;
      if (sub == 0) z[j] = acc;
      local_max = fmaxf(local_max, acc);
    }
  }
  // block max
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  float m = warp_max(local_max);
  if (lane == 0) red[warp] = m;
  __syncthreads();
  if (warp == 0) {
    float t = lane < nwarps ? red[lane] : -INFINITY;
    t = warp_max(t);
    if (lane == 0) red[32] = t;
  }
  __syncthreads();
  const float zmax = red[32];
  float local_sum = 0.f;
  for (int j = threadIdx.x; j < p.soft_n; j += blockDim.x) {
    float e = expf(z[j] - zmax);
    z[j] = e;
    local_sum += e;
  }
  float s = warp_sum(local_sum);
  __syncthreads();
  if (lane == 0) red[warp] = s;
  __syncthreads();
  if (warp == 0) {
    float t = lane < nwarps ? red[lane] : 0.f;
    t = warp_sum(t);
    if (lane == 0) red[32] = t;
  }
  __syncthreads();
  const float inv = 1.f / red[32];
  float* out = p.probs + (static_cast<size_t>(b) * p.q_heads + h) * p.span_len;
  const int off = p.span_begin - p.soft_lo;
  for (int j = threadIdx.x; j < p.span_len; j += blockDim.x) out[j] = z[off + j] * inv;
}

inline size_t qk_smem_bytes(int head_dim, int soft_n) {
  return (static_cast<size_t>(head_dim) + soft_n) * sizeof(float) + 16;
}

// Host-side launch shared by both entry points.
vscan_status launch_qk_softmax(int dtype, const QkParams& p, int batch, cudaStream_t stream);

// scores[b][j] = (1/q_heads) * sum_h probs[b][h][j], h ascending.
__global__ void head_mean_kernel(const float* probs, float* scores, int q_heads, int span_len);

}  // namespace vscan
