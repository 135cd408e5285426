// Device code shared by vscan_score (QK mode) and vscan_llm_prune: Eq. 5.
#pragma once

#include "common.cuh"
#include "topk.cuh"

namespace vscan {

struct QkParams {
  const void* q = nullptr;     // [batch][q_heads][head_dim]
  const void* k = nullptr;     // [batch][kv_heads][seq_len][head_dim]
  float* probs = nullptr;      // [batch][q_heads][span_len]  per-head probabilities on the span (scratch)
  uint32_t* status = nullptr;  // device status word of the workspace, cleared by the first CTA
  int q_heads = 0, kv_heads = 0, seq_len = 0, head_dim = 0, span_begin = 0, span_len = 0;
  int soft_lo = 0, soft_n = 0;  // keys the softmax runs over: [soft_lo, soft_lo + soft_n)
  float scale = 0.f;
  // Tail run by the last CTA of a sequence to finish (all null/zero: no tail):
  int* counters = nullptr;     // [batch], zero before the launch
  float* scores = nullptr;     // [batch][span_len] head mean (optional)
  int32_t* kept = nullptr;     // [batch][k_keep] top-k of the head mean, ascending (optional)
  int k_keep = 0;
  int* ready = nullptr;        // [batch] set to 1 once `kept` of the sequence is written (optional)
  // Split form (few long sequences): `nsplit` CTAs share the keys of one (head, sequence); each leaves its part of
  // the row unnormalised with (max, sum) in `stats`, and the last of them to finish (ticket) rescales the row.
  int nsplit = 1;
  float2* stats = nullptr;     // [batch][q_heads][nsplit]
  int* head_tickets = nullptr; // [batch][q_heads], zero before the launch
};

// One CTA per (query head, sequence), or `nsplit` of them, each on a contiguous share of the keys.
// Dynamic shared memory: q[head_dim] floats | z[soft_n] floats.
// Eight lanes share one key row (16-byte pieces, fp32 accumulate, 3 shuffles); each 8-lane group has
// four rows in flight.  VPS = 16-byte pieces per lane and row when that is a compile-time constant
// (head_dim / (8 lanes * elements per piece)), 0 for any other head_dim.
// With `counters` set, the CTA that finishes a sequence last sums the per-head probabilities in head
// order (the same fixed order whichever CTA it is), writes the head mean and/or its exact top-k.
template <typename T, int VPS>
__device__ __forceinline__ void qk_softmax_role(const QkParams& p, const int h, const int b, float* smem_f, const int split = 0) {
  float* qs = smem_f;
  float* z = smem_f + p.head_dim;
  __shared__ float red[33];
  __shared__ SelectScratch sc;
  __shared__ int is_last;
  constexpr int E = Vec16<T>::kElems;
  constexpr int R = VPS > 0 && VPS <= 2 ? 8 : 4;   // key rows in flight per 8-lane group
  if (h == 0 && b == 0 && threadIdx.x == 0 && p.status) *p.status = 0u;
  const int g = static_cast<int>((static_cast<long long>(h) * p.kv_heads) / p.q_heads);
  const T* qh = static_cast<const T*>(p.q) + (static_cast<size_t>(b) * p.q_heads + h) * p.head_dim;
  for (int i = threadIdx.x; i < p.head_dim; i += blockDim.x) qs[i] = to_float(qh[i]);
  __syncthreads();

  // this CTA's share of the softmax keys: [c_lo, c_lo + n_here) relative to soft_lo
  const int chunk = (p.soft_n + p.nsplit - 1) / p.nsplit;
  const int c_lo = min(p.soft_n, split * chunk), n_here = min(p.soft_n, c_lo + chunk) - c_lo;
  const T* kb = static_cast<const T*>(p.k) +
                ((static_cast<size_t>(b) * p.kv_heads + g) * p.seq_len + p.soft_lo + c_lo) * p.head_dim;
  const int vecs = p.head_dim / E;           // 16-byte pieces per key row
  const int sub = threadIdx.x & 7;           // lane within the 8-lane group
  const int grp = threadIdx.x >> 3, ngrp = blockDim.x >> 3;
  float local_max = -INFINITY;
  for (int j0 = 0; j0 < n_here; j0 += R * ngrp) {   // uniform trip count: shuffles stay converged
    float acc[R];
    if constexpr (VPS > 0) {
      uint4 raw[R][VPS];
#pragma unroll
      for (int u = 0; u < R; ++u) {
        const int j = j0 + u * ngrp + grp;
        const uint4* row = reinterpret_cast<const uint4*>(kb + static_cast<size_t>(min(j, n_here - 1)) * p.head_dim);
#pragma unroll
        for (int i = 0; i < VPS; ++i) raw[u][i] = ld_nc_16(row + sub + 8 * i);
      }
#pragma unroll
      for (int u = 0; u < R; ++u) {
        acc[u] = 0.f;
#pragma unroll
        for (int i = 0; i < VPS; ++i) {
          float kv[E];
          Vec16<T>::unpack(raw[u][i], kv);
#pragma unroll
          for (int e = 0; e < E; ++e) acc[u] = fmaf(kv[e], qs[(sub + 8 * i) * E + e], acc[u]);
        }
      }
    } else {
#pragma unroll
      for (int u = 0; u < R; ++u) {
        const int j = j0 + u * ngrp + grp;
        acc[u] = 0.f;
        if (j < n_here) {
          const uint4* row = reinterpret_cast<const uint4*>(kb + static_cast<size_t>(j) * p.head_dim);
          for (int v = sub; v < vecs; v += 8) {
            float kv[E];
            Vec16<T>::unpack(ld_nc_16(row + v), kv);
#pragma unroll
            for (int e = 0; e < E; ++e) acc[u] = fmaf(kv[e], qs[v * E + e], acc[u]);
          }
        }
      }
    }
#pragma unroll
    for (int u = 0; u < R; ++u) {
      const int j = j0 + u * ngrp + grp;
      float a = acc[u];
      a += __shfl_xor_sync(0xffffffffu, a, 1);
      a += __shfl_xor_sync(0xffffffffu, a, 2);
      a += __shfl_xor_sync(0xffffffffu, a, 4);
      if (j < n_here) {
        a *= p.scale;
        if (sub == 0) z[j] = a;
        local_max = fmaxf(local_max, a);
      }
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
  for (int j = threadIdx.x; j < n_here; j += blockDim.x) {
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
  float* out = p.probs + (static_cast<size_t>(b) * p.q_heads + h) * p.span_len;
  const int off = p.span_begin - p.soft_lo;
  if (p.nsplit == 1) {
    const float inv = 1.f / red[32];
    for (int j = threadIdx.x; j < p.span_len; j += blockDim.x) out[j] = z[off + j] * inv;
  } else {
    // leave exp(z - max of this share) for the span keys of the share, and the share's (max, sum)
    const int j_lo = max(c_lo, off), j_hi = min(c_lo + n_here, off + p.span_len);
    for (int j = j_lo + threadIdx.x; j < j_hi; j += blockDim.x) out[j - off] = z[j - c_lo];
    float2* st = p.stats + (static_cast<size_t>(b) * p.q_heads + h) * p.nsplit;
    if (threadIdx.x == 0) st[split] = make_float2(n_here > 0 ? zmax : -INFINITY, n_here > 0 ? red[32] : 0.f);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(&p.head_tickets[b * p.q_heads + h], 1) == p.nsplit - 1);
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // the row's max and denominator from the shares; every share is rescaled by exp(its max - row max) / denominator
    float row_max = -INFINITY;
    for (int c = 0; c < p.nsplit; ++c) row_max = fmaxf(row_max, __ldcg(&st[c].x));
    float denom = 0.f;
    for (int c = 0; c < p.nsplit; ++c) {
      const float2 sc2 = __ldcg(&st[c]);
      denom += sc2.y > 0.f ? sc2.y * expf(sc2.x - row_max) : 0.f;
    }
    const float inv = 1.f / denom;
    for (int j = threadIdx.x; j < p.span_len; j += blockDim.x) {
      const int c = (j + off) / chunk;
      out[j] = __ldcg(out + j) * (expf(__ldcg(&st[c].x) - row_max) * inv);
    }
    __syncthreads();   // is_last is reused below
  }

  if (!p.counters) return;
  // ---- tail: whoever finishes this sequence last reduces over the heads
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(&p.counters[b], 1) == p.q_heads - 1);
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  uint32_t* keys = reinterpret_cast<uint32_t*>(z);   // span_len <= soft_n entries fit
  const float* base = p.probs + static_cast<size_t>(b) * p.q_heads * p.span_len;
  if ((p.span_len & 3) == 0) {
    // four columns per thread and load: the rows start on 16-byte boundaries; same additions in the same order
    const int n4 = p.span_len >> 2;
    const float4* base4 = reinterpret_cast<const float4*>(base);
    const float rq = static_cast<float>(p.q_heads);
    for (int j = threadIdx.x; j < n4; j += blockDim.x) {
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      int hh = 0;
      for (; hh + 8 <= p.q_heads; hh += 8) {   // eight 16-byte loads in flight, added in head order
        float4 a[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) a[u] = __ldcg(base4 + static_cast<size_t>(hh + u) * n4 + j);
#pragma unroll
        for (int u = 0; u < 8; ++u) { acc.x += a[u].x; acc.y += a[u].y; acc.z += a[u].z; acc.w += a[u].w; }
      }
      for (; hh < p.q_heads; ++hh) {
        const float4 a = __ldcg(base4 + static_cast<size_t>(hh) * n4 + j);
        acc.x += a.x; acc.y += a.y; acc.z += a.z; acc.w += a.w;
      }
      acc.x /= rq; acc.y /= rq; acc.z /= rq; acc.w /= rq;
      if (p.scores) reinterpret_cast<float4*>(p.scores + static_cast<size_t>(b) * p.span_len)[j] = acc;
      keys[4 * j + 0] = float_to_key(acc.x); keys[4 * j + 1] = float_to_key(acc.y);
      keys[4 * j + 2] = float_to_key(acc.z); keys[4 * j + 3] = float_to_key(acc.w);
    }
  } else
  for (int j = threadIdx.x; j < p.span_len; j += blockDim.x) {
    float acc = 0.f;
    int hh = 0;
    for (; hh + 16 <= p.q_heads; hh += 16) {   // sixteen loads in flight, added in head order
      float a[16];
#pragma unroll
      for (int u = 0; u < 16; ++u) a[u] = __ldcg(base + static_cast<size_t>(hh + u) * p.span_len + j);
#pragma unroll
      for (int u = 0; u < 16; ++u) acc += a[u];
    }
    for (; hh + 4 <= p.q_heads; hh += 4) {
      float a[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) a[u] = __ldcg(base + static_cast<size_t>(hh + u) * p.span_len + j);
#pragma unroll
      for (int u = 0; u < 4; ++u) acc += a[u];
    }
    for (; hh < p.q_heads; ++hh) acc += __ldcg(base + static_cast<size_t>(hh) * p.span_len + j);
    acc /= static_cast<float>(p.q_heads);
    if (p.scores) p.scores[static_cast<size_t>(b) * p.span_len + j] = acc;
    keys[j] = float_to_key(acc);
  }
  __syncthreads();
  if (p.kept && p.k_keep > 0)
    block_topk_emit(keys, p.span_len, p.k_keep, sc, p.kept + static_cast<size_t>(b) * p.k_keep);
  if (p.ready) {   // publish: the survivor list of sequence b is complete
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) atomicExch(&p.ready[b], 1);
  }
}

template <typename T, int VPS>
__global__ void __launch_bounds__(256) qk_softmax_kernel(QkParams p) {
  extern __shared__ __align__(16) float smem_f[];
  grid_dependency_launch();
  qk_softmax_role<T, VPS>(p, blockIdx.x, blockIdx.y, smem_f);
}

inline size_t qk_smem_bytes(int head_dim, int soft_n) {
  return (static_cast<size_t>(head_dim) + soft_n) * sizeof(float) + 16;
}

// Host-side argument checks and launch shared by the entry points.
vscan_status validate_score(const vscan_score_desc* d);
vscan_status launch_qk_softmax(int dtype, const QkParams& p, int batch, cudaStream_t stream);
// RECEIVED mode (Sec. 4.1, text after Eq. 2): per-head received attention from Q and K on the tensor cores.
bool received_supported(const vscan_score_desc* d);
size_t received_workspace_bytes(const vscan_score_desc* d);
vscan_status launch_received(const vscan_score_desc* d, void* workspace, float* rows_out, cudaStream_t stream);

}  // namespace vscan
