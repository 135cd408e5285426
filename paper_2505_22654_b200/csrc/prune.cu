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

template <int THREADS>
__device__ __forceinline__ void copy_run(const uint4* __restrict__ src, uint4* __restrict__ dst, int n) {
  // n pieces, contiguous on both sides
  for (int i0 = threadIdx.x; i0 < n; i0 += THREADS * kCompactUnroll) {
    uint4 r[kCompactUnroll];
#pragma unroll
    for (int u = 0; u < kCompactUnroll; ++u) {
      int i = i0 + u * THREADS;
      if (i < n) r[u] = ld_nc_16(src + i);
    }
#pragma unroll
    for (int u = 0; u < kCompactUnroll; ++u) {
      int i = i0 + u * THREADS;
      if (i < n) st_16(dst + i, r[u]);
    }
  }
}

// Moves output row r of sequence b: hidden row, the kv_heads rows of K and of V, position ids.
template <int THREADS>
__device__ __forceinline__ void compact_row(const CompactParams& p, const int r, const int b) {
  int src;
  if (r < p.n_sys) src = r;
  else if (r < p.n_sys + p.k_keep) {
    int kv = __ldcg(p.kept_vis + static_cast<size_t>(b) * p.k_keep + (r - p.n_sys));
    kv = min(max(kv, 0), p.n_vis - 1);
    src = p.n_sys + kv;
  } else src = r + (p.n_vis - p.k_keep);

  if (p.hidden) {
    copy_run<THREADS>(p.hidden + (static_cast<size_t>(b) * p.seq_len + src) * p.hidden_vecs,
             p.hidden_out + (static_cast<size_t>(b) * p.seq_out + r) * p.hidden_vecs, p.hidden_vecs);
  }
  // K and V: kv_heads rows of kv_vecs pieces, strided by the sequence length
  const int total = p.kv_heads * p.kv_vecs;
  const size_t src_head = static_cast<size_t>(p.seq_len) * p.kv_vecs, dst_head = static_cast<size_t>(p.seq_out) * p.kv_vecs;
  const size_t src0 = (static_cast<size_t>(b) * p.kv_heads * p.seq_len + src) * p.kv_vecs;
  const size_t dst0 = (static_cast<size_t>(b) * p.kv_heads * p.seq_out + r) * p.kv_vecs;
  for (int i0 = threadIdx.x; i0 < total; i0 += THREADS * kCompactUnroll) {
    uint4 rk[kCompactUnroll], rv[kCompactUnroll];
    size_t so[kCompactUnroll], dof[kCompactUnroll];
#pragma unroll
    for (int u = 0; u < kCompactUnroll; ++u) {
      int i = i0 + u * THREADS;
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
      int i = i0 + u * THREADS;
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

__global__ void __launch_bounds__(kCompactThreads) compact_kernel(CompactParams p) {
  grid_dependency_wait();   // the survivor list comes from the kernel before this one
  compact_row<kCompactThreads>(p, blockIdx.x, blockIdx.y);
}

// Score, top-k and compaction of Stage 2 in ONE launch.  n_score CTAs are the (head, sequence)
// scoring CTAs of qk_softmax_role; the others each move one output row.  Rows of the system and text
// spans do not depend on the selection: they come first in block order, interleaved with the scoring
// CTAs; a row of the visual span waits, with a bound, until the scoring CTA that finished its
// sequence last has published the survivor list.  Blocks are dispatched in index order and every
// scoring CTA has a lower index than any waiting CTA, so every scoring CTA is running or done
// before a waiting CTA can occupy a slot.
constexpr int kPruneThreads = 128;
constexpr unsigned kReadySpinLimit = 1u << 22;

template <typename T, int VPS>
__global__ void __launch_bounds__(kPruneThreads, 8) prune_fused_kernel(QkParams q, CompactParams c, int n_score) {
  extern __shared__ __align__(16) float smem_f[];
  // Block order: the scoring CTAs and the rows that do not depend on the selection are dealt out together, one
  // scoring CTA per `period` blocks (scoring is bound by latency, the row copies by bandwidth: side by side they
  // keep the memory pipe busy from the start); the rows that wait for a survivor list come after all of them.
  const int fixed_rows = c.seq_out - c.k_keep;           // system + text rows per sequence
  const int n_fixed = c.batch * fixed_rows, n_indep = n_score + n_fixed;
  const int blk = blockIdx.x;
  int idx;                                                // row index: first the independent rows, then the dependent ones
  if (blk < n_indep) {
    const int period = n_score > 0 ? n_indep / n_score : 1;
    const int qd = blk / period, rm = blk - qd * period;
    if (qd < n_score && rm == 0) {
      const int unit = qd / q.nsplit;   // (sequence, head), heads fastest; the shares of a unit are neighbours
      qk_softmax_role<T, VPS>(q, unit % q.q_heads, unit / q.q_heads, smem_f, qd - unit * q.nsplit);
      return;
    }
    idx = qd < n_score ? qd * (period - 1) + (rm - 1) : n_score * (period - 1) + (blk - n_score * period);
  } else {
    idx = blk - n_score;
  }
  int r, b;
  bool dependent;
  if (idx < n_fixed) {
    b = idx / fixed_rows;
    const int i = idx - b * fixed_rows;
    r = i < c.n_sys ? i : i + c.k_keep;
    dependent = false;
  } else {
    idx -= n_fixed;
    b = idx / c.k_keep;
    r = c.n_sys + (idx - b * c.k_keep);
    dependent = true;
  }
  if (dependent) {
    __shared__ int ok;
    if (threadIdx.x == 0) {
      ok = wait_flag_bounded(q.ready + b, 1, kReadySpinLimit);
      if (!ok && q.status) atomicExch(q.status, static_cast<uint32_t>(VSCAN_ERR_TIMEOUT));
      __threadfence();
    }
    __syncthreads();
    if (!ok) return;
  }
  compact_row<kPruneThreads>(c, r, b);
}

template <typename T>
static vscan_status launch_prune_fused(const QkParams& q, const CompactParams& c, size_t smem, cudaStream_t stream) {
  constexpr int E = Vec16<T>::kElems;
  const int n_score = c.batch * q.q_heads * q.nsplit;
  const unsigned blocks = static_cast<unsigned>(n_score) + static_cast<unsigned>(c.batch) * c.seq_out;
  const int vecs = q.head_dim / E;
#define VSCAN_PRUNE_CASE(VPS)                                                                                  \
  do {                                                                                                         \
    VSCAN_CUDA_TRY(allow_smem(prune_fused_kernel<T, VPS>, smem));                                              \
    VSCAN_LAUNCH("prune_fused", stream,                                                                        \
                 (prune_fused_kernel<T, VPS><<<blocks, kPruneThreads, smem, stream>>>(q, c, n_score)));        \
    return VSCAN_OK;                                                                                           \
  } while (0)
  if (vecs == 16) VSCAN_PRUNE_CASE(2);
  if (vecs == 32) VSCAN_PRUNE_CASE(4);
  if (vecs == 8) VSCAN_PRUNE_CASE(1);
  VSCAN_PRUNE_CASE(0);
#undef VSCAN_PRUNE_CASE
}

// One CTA that waits, the way a row-copy CTA waits for its sequence's survivor list, on a flag nobody sets.
__global__ void __launch_bounds__(32) selftest_wait_kernel(uint32_t* status, int* flag, unsigned limit) {
  if (threadIdx.x == 0 && !wait_flag_bounded(flag, 1, limit)) atomicExch(status, static_cast<uint32_t>(VSCAN_ERR_TIMEOUT));
}

}  // namespace vscan

using namespace vscan;

extern "C" vscan_status vscan_selftest_bounded_wait(void* workspace, size_t workspace_bytes, uint32_t polls, void* stream_) {
  if (!workspace || !aligned256(workspace) || workspace_bytes < 2 * kStatusBytes) return VSCAN_ERR_WORKSPACE;
  if (polls == 0 || polls > (1u << 24)) return VSCAN_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  VSCAN_CUDA_TRY(cudaMemsetAsync(workspace, 0, 2 * kStatusBytes, stream));   // status word and the flag
  int* flag = reinterpret_cast<int*>(static_cast<char*>(workspace) + kStatusBytes);
  VSCAN_LAUNCH("selftest_wait", stream,
               (selftest_wait_kernel<<<1, 32, 0, stream>>>(static_cast<uint32_t*>(workspace), flag, polls)));
  return VSCAN_OK;
}

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
  if (d->pos_ids && d->pos_planes > vscan::kPruneThreads) return VSCAN_ERR_UNSUPPORTED;
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

// CTAs that share the keys of one (head, sequence) in the scoring part: one per 256 keys, at most 8, and only while
// the scoring CTAs of the whole batch stay within what the SMs hold at once (a few long sequences).
static int score_splits(const vscan_prune_desc* d) {
  const long long soft_n = d->softmax_span == VSCAN_SPAN_ONLY ? d->n_vis : 1ll * d->n_sys + d->n_vis + d->n_txt;
  long long n = soft_n / 256;
  n = n > 8 ? 8 : n;
  const long long units = 1ll * d->batch * d->q_heads;
  while (n > 1 && units * n > 1184) --n;   // 8 scoring CTAs per SM
  return n < 1 ? 1 : static_cast<int>(n);
}
// per-sequence arrival counters and ready flags, per-(sequence, head) tickets of the split form
static size_t prune_counter_bytes(const vscan_prune_desc* d) {
  return round_up((2 + static_cast<size_t>(d->q_heads)) * d->batch * sizeof(int), 256);
}
static size_t prune_stats_bytes(const vscan_prune_desc* d) {
  return round_up(static_cast<size_t>(d->batch) * d->q_heads * 8 * sizeof(float2), 256);
}

extern "C" size_t vscan_llm_prune_workspace_bytes(const vscan_prune_desc* d) {
  if (!d || d->batch <= 0 || d->q_heads <= 0 || d->n_vis <= 0) return kStatusBytes;
  return kStatusBytes + prune_counter_bytes(d) + prune_stats_bytes(d) +
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
  // workspace: status word | per-sequence arrival counters, per-sequence ready flags, per-head tickets |
  //            (max, sum) of the key shares | per-head probabilities
  char* ws = static_cast<char*>(workspace);
  const size_t counter_bytes = prune_counter_bytes(d);
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

  bool fused = false;
  if (d->n_vis > 0) {
    QkParams p;
    p.q = d->q_last; p.k = d->k; p.status = static_cast<uint32_t*>(workspace);
    p.counters = reinterpret_cast<int*>(ws + kStatusBytes);
    p.ready = p.counters + d->batch;
    p.head_tickets = p.ready + d->batch;
    p.stats = reinterpret_cast<float2*>(ws + kStatusBytes + counter_bytes);
    p.probs = reinterpret_cast<float*>(ws + kStatusBytes + counter_bytes + prune_stats_bytes(d));
    p.scores = d->scores; p.kept = d->kept_vis; p.k_keep = d->k_keep;
    p.q_heads = d->q_heads; p.kv_heads = d->kv_heads; p.seq_len = seq_len; p.head_dim = d->head_dim;
    p.span_begin = d->n_sys; p.span_len = d->n_vis; p.scale = d->scale;
    if (d->softmax_span == VSCAN_SPAN_ONLY) { p.soft_lo = d->n_sys; p.soft_n = d->n_vis; }
    else { p.soft_lo = 0; p.soft_n = seq_len; }
    VSCAN_CUDA_TRY(cudaMemsetAsync(p.counters, 0, counter_bytes, stream));
    // one launch for score, top-k and compaction when the top-k fits the 128-thread scoring CTAs
    const int nsplit = score_splits(d);
    const long long blocks = 1ll * d->batch * d->q_heads * nsplit + 1ll * d->batch * seq_out;
    const size_t smem = qk_smem_bytes(p.head_dim, p.soft_n);
    if (d->n_vis <= 8192 && seq_out > 0 && blocks < (1ll << 31) && smem <= kMaxDynamicSmem) {
      p.nsplit = nsplit;
      st = d->dtype == VSCAN_F32 ? launch_prune_fused<float>(p, c, smem, stream)
                                 : launch_prune_fused<__nv_bfloat16>(p, c, smem, stream);
      if (st != VSCAN_OK) return st;
      fused = true;
    } else {
      p.ready = nullptr;
      st = launch_qk_softmax(d->dtype, p, d->batch, stream);
      if (st != VSCAN_OK) return st;
    }
  } else {
    VSCAN_CUDA_TRY(cudaMemsetAsync(workspace, 0, kStatusBytes, stream));
  }
  if (fused || seq_out == 0) return VSCAN_OK;
  dim3 grid(seq_out, d->batch);
  VSCAN_LAUNCH("compact", stream, (void)launch_dependent(compact_kernel, grid, dim3(kCompactThreads), 0, stream, c));
  return VSCAN_OK;
}
