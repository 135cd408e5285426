// vscan_llm_prune: Stage 2 (Sec. 4.2).  Eq. 5 scores -> exact top-k -> compaction of hidden states,
// K, V and position ids to [system | surviving visual | text].
#include "score.cuh"
#include "topk.cuh"

namespace vscan {

struct CompactParams {
  const int32_t* kept_vis;  // [batch][k_keep]
  const uint4* hidden; uint4* hidden_out;
  const uint4* k; uint4* k_out;
  const uint4* v; uint4* v_out;
  const int32_t* pos; int32_t* pos_out;
  int batch, kv_heads, seq_len, seq_out, n_sys, n_vis, k_keep, pos_planes;
  int hidden_vecs;  // 16-byte pieces per hidden row
  int kv_vecs;      // 16-byte pieces per (head, token) row of K or V
};

// One CTA per output row (b, r).  The row's source position is decoded once; then the CTA moves
// the hidden row and the kv_heads rows of K and of V with 16-byte accesses, all loads of a round in
// flight before the first store.
constexpr int kCompactThreads = 256;
constexpr int kCompactUnroll = 4;

__device__ __forceinline__ void copy_run(const uint4* __restrict__ src, uint4* __restrict__ dst, int n) {
  // n pieces, contiguous on both sides
  for (int i0 = threadIdx.x; i0 < n; i0 += kCompactThreads * kCompactUnroll) {
    uint4 r[kCompactUnroll];
#pragma unroll
    for (int u = 0; u < kCompactUnroll; ++u) {
      int i = i0 + u * kCompactThreads;
      if (i < n) r[u] = ld_nc_16(src + i);
    }
#pragma unroll
    for (int u = 0; u < kCompactUnroll; ++u) {
      int i = i0 + u * kCompactThreads;
      if (i < n) st_16(dst + i, r[u]);
    }
  }
}

__global__ void __launch_bounds__(kCompactThreads) compact_kernel(CompactParams p) {
  const int r = blockIdx.x, b = blockIdx.y;
  grid_dependency_wait();   // the survivor list comes from the kernel before this one
  int src;
  if (r < p.n_sys) src = r;
  else if (r < p.n_sys + p.k_keep) {
    int kv = p.kept_vis[static_cast<size_t>(b) * p.k_keep + (r - p.n_sys)];
    kv = min(max(kv, 0), p.n_vis - 1);
    src = p.n_sys + kv;
  } else src = r + (p.n_vis - p.k_keep);

  if (p.hidden) {
    copy_run(p.hidden + (static_cast<size_t>(b) * p.seq_len + src) * p.hidden_vecs,
             p.hidden_out + (static_cast<size_t>(b) * p.seq_out + r) * p.hidden_vecs, p.hidden_vecs);
  }
  // K and V: kv_heads rows of kv_vecs pieces, strided by the sequence length
  const int total = p.kv_heads * p.kv_vecs;
  const size_t src_head = static_cast<size_t>(p.seq_len) * p.kv_vecs, dst_head = static_cast<size_t>(p.seq_out) * p.kv_vecs;
  const size_t src0 = (static_cast<size_t>(b) * p.kv_heads * p.seq_len + src) * p.kv_vecs;
  const size_t dst0 = (static_cast<size_t>(b) * p.kv_heads * p.seq_out + r) * p.kv_vecs;
  for (int i0 = threadIdx.x; i0 < total; i0 += kCompactThreads * kCompactUnroll) {
    uint4 rk[kCompactUnroll], rv[kCompactUnroll];
    size_t so[kCompactUnroll], dof[kCompactUnroll];
#pragma unroll
    for (int u = 0; u < kCompactUnroll; ++u) {
      int i = i0 + u * kCompactThreads;
      if (i < total) {
        int head = i / p.kv_vecs, vec = i - head * p.kv_vecs;
        so[u] = src0 + head * src_head + vec;
        dof[u] = dst0 + head * dst_head + vec;
        rk[u] = ld_nc_16(p.k + so[u]);
        if (p.v) rv[u] = ld_nc_16(p.v + so[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < kCompactUnroll; ++u) {
      int i = i0 + u * kCompactThreads;
      if (i < total) {
        st_16(p.k_out + dof[u], rk[u]);
        if (p.v) st_16(p.v_out + dof[u], rv[u]);
      }
    }
  }
  if (p.pos && threadIdx.x < p.pos_planes) {
    const int pl = threadIdx.x;
    p.pos_out[(static_cast<size_t>(pl) * p.batch + b) * p.seq_out + r] =
        p.pos[(static_cast<size_t>(pl) * p.batch + b) * p.seq_len + src];
  }
}

}  // namespace vscan

using namespace vscan;

static vscan_status validate_prune(const vscan_prune_desc* d) {
  if (!d || !d->q_last || !d->k || !d->k_out) return VSCAN_ERR_INVALID_ARG;
  if (!d->kept_vis && d->k_keep > 0) return VSCAN_ERR_INVALID_ARG;  // an empty survivor list may be NULL
  if (d->dtype != VSCAN_F32 && d->dtype != VSCAN_BF16) return VSCAN_ERR_INVALID_ARG;
  if ((d->v == nullptr) != (d->v_out == nullptr) || (d->hidden == nullptr) != (d->hidden_out == nullptr) ||
      (d->pos_ids == nullptr) != (d->pos_out == nullptr))
    return VSCAN_ERR_INVALID_ARG;
  if (d->batch < 0 || d->q_heads <= 0 || d->kv_heads <= 0 || d->q_heads % d->kv_heads || d->head_dim <= 0 ||
      d->n_sys < 0 || d->n_vis < 0 || d->n_txt < 0 || d->k_keep < 0 || d->k_keep > d->n_vis)
    return VSCAN_ERR_INVALID_ARG;
  if (d->softmax_span != VSCAN_SPAN_ONLY && d->softmax_span != VSCAN_SPAN_FULL) return VSCAN_ERR_INVALID_ARG;
  if (d->head_dim % 8 || d->head_dim > 256) return VSCAN_ERR_INVALID_ARG;
  const size_t e = dtype_bytes(d->dtype);
  if (d->hidden && (d->hidden_dim <= 0 || (d->hidden_dim * e) % 16)) return VSCAN_ERR_INVALID_ARG;
  if (d->pos_ids && d->pos_planes <= 0) return VSCAN_ERR_INVALID_ARG;
  if (d->pos_ids && d->pos_planes > vscan::kCompactThreads) return VSCAN_ERR_UNSUPPORTED;
  if (d->n_vis > 16384) return VSCAN_ERR_UNSUPPORTED;
  const void* ptrs[] = {d->q_last, d->k, d->v, d->hidden, d->pos_ids, d->kept_vis, d->hidden_out,
                        d->k_out, d->v_out, d->pos_out, d->scores};
  for (const void* ptr : ptrs)
    if (ptr && !aligned16(ptr)) return VSCAN_ERR_INVALID_ARG;
  const size_t S = static_cast<size_t>(d->n_sys) + d->n_vis + d->n_txt, So = S - d->n_vis + d->k_keep;
  const size_t B = d->batch;
  struct Rng { const void* p; size_t n; };
  const Rng ins[] = {{d->q_last, B * d->q_heads * d->head_dim * e}, {d->k, B * d->kv_heads * S * d->head_dim * e},
                     {d->v, B * d->kv_heads * S * d->head_dim * e}, {d->hidden, B * S * d->hidden_dim * e},
                     {d->pos_ids, static_cast<size_t>(d->pos_planes) * B * S * 4}};
  const Rng outs[] = {{d->kept_vis, B * d->k_keep * 4}, {d->hidden_out, B * So * d->hidden_dim * e},
                      {d->k_out, B * d->kv_heads * So * d->head_dim * e}, {d->v_out, B * d->kv_heads * So * d->head_dim * e},
                      {d->pos_out, static_cast<size_t>(d->pos_planes) * B * So * 4}, {d->scores, B * d->n_vis * 4}};
  for (const Rng& o : outs) {
    for (const Rng& i : ins)
      if (overlaps(o.p, o.n, i.p, i.n)) return VSCAN_ERR_INVALID_ARG;
    for (const Rng& o2 : outs)
      if (o.p != o2.p && overlaps(o.p, o.n, o2.p, o2.n)) return VSCAN_ERR_INVALID_ARG;
  }
  return VSCAN_OK;
}

extern "C" size_t vscan_llm_prune_workspace_bytes(const vscan_prune_desc* d) {
  if (!d || d->batch <= 0 || d->q_heads <= 0 || d->n_vis <= 0) return kStatusBytes;
  return kStatusBytes + round_up(static_cast<size_t>(d->batch) * sizeof(int), 256) +
         round_up(static_cast<size_t>(d->batch) * d->q_heads * d->n_vis * sizeof(float), 256);
}

extern "C" vscan_status vscan_llm_prune(const vscan_prune_desc* d, void* workspace, size_t workspace_bytes,
                                        void* stream_) {
  if (d && d->batch == 0) return VSCAN_OK;  // empty batch
  vscan_status st = validate_prune(d);
  if (st != VSCAN_OK) return st;
  if (d->batch == 0) return VSCAN_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const size_t need = vscan_llm_prune_workspace_bytes(d);
  if (!workspace || !aligned256(workspace) || workspace_bytes < need) return VSCAN_ERR_WORKSPACE;
  const int seq_len = d->n_sys + d->n_vis + d->n_txt, seq_out = seq_len - d->n_vis + d->k_keep;
  // workspace: status word | per-sequence arrival counters | per-head probabilities
  char* ws = static_cast<char*>(workspace);
  const size_t counter_bytes = round_up(static_cast<size_t>(d->batch) * sizeof(int), 256);

  if (d->n_vis > 0) {
    QkParams p;
    p.q = d->q_last; p.k = d->k; p.status = static_cast<uint32_t*>(workspace);
    p.counters = reinterpret_cast<int*>(ws + kStatusBytes);
    p.probs = reinterpret_cast<float*>(ws + kStatusBytes + counter_bytes);
    p.scores = d->scores; p.kept = d->kept_vis; p.k_keep = d->k_keep;
    p.q_heads = d->q_heads; p.kv_heads = d->kv_heads; p.seq_len = seq_len; p.head_dim = d->head_dim;
    p.span_begin = d->n_sys; p.span_len = d->n_vis; p.scale = d->scale;
    if (d->softmax_span == VSCAN_SPAN_ONLY) { p.soft_lo = d->n_sys; p.soft_n = d->n_vis; }
    else { p.soft_lo = 0; p.soft_n = seq_len; }
    // score and top-k in one launch: the last CTA of each sequence reduces over the heads and selects
    VSCAN_CUDA_TRY(cudaMemsetAsync(p.counters, 0, counter_bytes, stream));
    st = launch_qk_softmax(d->dtype, p, d->batch, stream);
    if (st != VSCAN_OK) return st;
  } else {
    VSCAN_CUDA_TRY(cudaMemsetAsync(workspace, 0, kStatusBytes, stream));
  }
  if (seq_out == 0) return VSCAN_OK;
  const size_t e = dtype_bytes(d->dtype);
  CompactParams c;
  c.kept_vis = d->kept_vis;
  c.hidden = static_cast<const uint4*>(d->hidden); c.hidden_out = static_cast<uint4*>(d->hidden_out);
  c.k = static_cast<const uint4*>(d->k); c.k_out = static_cast<uint4*>(d->k_out);
  c.v = static_cast<const uint4*>(d->v); c.v_out = static_cast<uint4*>(d->v_out);
  c.pos = d->pos_ids; c.pos_out = d->pos_out;
  c.batch = d->batch; c.kv_heads = d->kv_heads; c.seq_len = seq_len; c.seq_out = seq_out;
  c.n_sys = d->n_sys; c.n_vis = d->n_vis; c.k_keep = d->k_keep; c.pos_planes = d->pos_planes;
  c.hidden_vecs = d->hidden ? static_cast<int>(d->hidden_dim * e / 16) : 0;
  c.kv_vecs = static_cast<int>(d->head_dim * e / 16);
  dim3 grid(seq_out, d->batch);
  VSCAN_LAUNCH("compact", stream, (void)launch_dependent(compact_kernel, grid, dim3(kCompactThreads), 0, stream, c));
  return VSCAN_OK;
}
