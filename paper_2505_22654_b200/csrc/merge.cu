// vscan_merge: cosine arg-max assignment of the unselected tokens and mean merge (Eq. 4).
//   kept_inv_norm_kernel   1 / max(|m_s|, eps) of every kept token
//   assign (SIMT or tensor) a(u) = argmax_s (m_u . m_s) * inv_norm[s]   (|m_u| is constant along a
//                           row of the similarity matrix and cannot change the arg-max)
//   group_mean_kernel      members of every slot in ascending token order, fp32 sum, one rounding
#include "merge.cuh"
#include "merge_mean.cuh"

namespace vscan {

// ------------------------------------------------------------------ norms of the kept tokens
// One warp per kept token.  grid = (ceil(n_kept / 8), instances), 256 threads.
template <typename T>
__global__ void __launch_bounds__(256) kept_inv_norm_kernel(MergeParams p) {
  constexpr int E = Vec16<T>::kElems;
  const int b = blockIdx.y, s = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (p.clear_status && blockIdx.x == 0 && b == 0 && threadIdx.x == 0) *p.status = 0u;
  if (s >= p.n_kept) return;
  int t = p.kept[static_cast<size_t>(b) * p.n_kept + s];
  t = min(max(t, 0), p.n_tokens - 1);
  const uint4* row = reinterpret_cast<const uint4*>(
      static_cast<const T*>(p.metric) + (static_cast<size_t>(b) * p.row_len + p.cls_offset + t) * p.metric_dim);
  const int vecs = p.metric_dim / E;
  float ss = 0.f;
  for (int v = lane; v < vecs; v += 32) {
    float f[E];
    Vec16<T>::unpack(ld_nc_16(row + v), f);
#pragma unroll
    for (int e = 0; e < E; ++e) ss = fmaf(f[e], f[e], ss);
  }
  ss = warp_sum(ss);
  if (lane == 0) p.inv_norm[static_cast<size_t>(b) * p.n_kept + s] = 1.f / fmaxf(sqrtf(ss), 1e-12f);
}

// ------------------------------------------------------------------ assignment on CUDA cores
// CTA tile: 64 tokens x 64 kept, 32-wide slices of the feature dim, 4x4 outputs per thread.
constexpr int kTileT = 64, kTileS = 64, kTileK = 32, kPad = 4;

template <typename T>
__global__ void __launch_bounds__(256) assign_simt_kernel(MergeParams p) {
  constexpr int E = Vec16<T>::kElems;
  constexpr int kVecPerRow = kTileK / E;
  __shared__ __align__(16) float As[kTileK][kTileT + kPad];
  __shared__ __align__(16) float Bs[kTileK][kTileS + kPad];
  __shared__ int kept_row[kTileS];
  __shared__ float kept_scale[kTileS];
  __shared__ int best_slot[kTileT];

  const int b = blockIdx.y, t0 = blockIdx.x * kTileT;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const T* mb = static_cast<const T*>(p.metric) + (static_cast<size_t>(b) * p.row_len + p.cls_offset) * p.metric_dim;
  const int32_t* kept = p.kept + static_cast<size_t>(b) * p.n_kept;
  const float* inv_norm = p.inv_norm + static_cast<size_t>(b) * p.n_kept;

  float run_val[4];
  int run_idx[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) { run_val[i] = -INFINITY; run_idx[i] = 0; }

  for (int s0 = 0; s0 < p.n_kept; s0 += kTileS) {
    __syncthreads();
    if (threadIdx.x < kTileS) {
      int s = s0 + threadIdx.x;
      int t = s < p.n_kept ? min(max(kept[s], 0), p.n_tokens - 1) : -1;
      kept_row[threadIdx.x] = t;
      kept_scale[threadIdx.x] = s < p.n_kept ? inv_norm[s] : 0.f;
    }
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int k0 = 0; k0 < p.metric_dim; k0 += kTileK) {
      __syncthreads();
      for (int idx = threadIdx.x; idx < kTileT * kVecPerRow; idx += 256) {
        const int row = idx / kVecPerRow, vec = idx % kVecPerRow, kk = k0 + vec * E;
        float fa[E], fb[E];
#pragma unroll
        for (int e = 0; e < E; ++e) { fa[e] = 0.f; fb[e] = 0.f; }
        const int t = t0 + row;
        if (t < p.n_tokens && kk < p.metric_dim)
          Vec16<T>::unpack(ld_nc_16(mb + static_cast<size_t>(t) * p.metric_dim + kk), fa);
        const int tk = kept_row[row];
        if (tk >= 0 && kk < p.metric_dim)
          Vec16<T>::unpack(ld_nc_16(mb + static_cast<size_t>(tk) * p.metric_dim + kk), fb);
#pragma unroll
        for (int e = 0; e < E; ++e) { As[vec * E + e][row] = fa[e]; Bs[vec * E + e][row] = fb[e]; }
      }
      __syncthreads();
#pragma unroll
      for (int k = 0; k < kTileK; ++k) {
        const float4 a = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
        const float4 c = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
        const float av[4] = {a.x, a.y, a.z, a.w}, cv[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], cv[j], acc[i][j]);
      }
    }
    // arg-max of this kept tile, lowest slot on ties
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float bv = -INFINITY;
      int bi = 0x7fffffff;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int s = s0 + tx * 4 + j;
        if (s < p.n_kept) {
          const float v = acc[i][j] * kept_scale[tx * 4 + j];
          if (v > bv) { bv = v; bi = s; }
        }
      }
#pragma unroll
      for (int o = 1; o < 16; o <<= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
      }
      if (bv > run_val[i]) { run_val[i] = bv; run_idx[i] = bi; }
    }
  }
  if (tx == 0) {
#pragma unroll
    for (int i = 0; i < 4; ++i) best_slot[ty * 4 + i] = run_idx[i] == 0x7fffffff ? 0 : run_idx[i];
  }
  __syncthreads();
  // a kept token belongs to its own slot
  for (int s = threadIdx.x; s < p.n_kept; s += 256) {
    const int t = min(max(kept[s], 0), p.n_tokens - 1);
    if (t >= t0 && t < t0 + kTileT) best_slot[t - t0] = s;
  }
  __syncthreads();
  if (threadIdx.x < kTileT && t0 + threadIdx.x < p.n_tokens)
    p.assign[static_cast<size_t>(b) * p.n_tokens + t0 + threadIdx.x] = best_slot[threadIdx.x];
}

vscan_status launch_assign_simt(int dtype, const MergeParams& p, cudaStream_t stream) {
  dim3 grid((p.n_tokens + kTileT - 1) / kTileT, p.instances);
  if (dtype == VSCAN_F32) VSCAN_LAUNCH("assign_simt", stream, assign_simt_kernel<float><<<grid, 256, 0, stream>>>(p));
  else VSCAN_LAUNCH("assign_simt", stream, assign_simt_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(p));
  return VSCAN_OK;
}

// ------------------------------------------------------------------ group means
// One CTA per (group of slots, instance), one warp per slot: 4 slots per CTA for short instances, 16
// for long ones (the list-building prologue is O(n_tokens) per CTA); warp w owns slot s0 + w.  The CTA first lists, in
// ascending token order, the tokens assigned to its slots; each warp then walks that list and adds
// its members' rows in that order (fp32), R rows in flight.  Small CTAs keep a large group from
// holding the resources of many finished warps.
// dynamic shared memory: list[n_tokens] of (local slot << 24 | token), then assign[n_tokens]
template <typename T, int VPL, int R, int kSlotsPerCta>
__global__ void __launch_bounds__(kSlotsPerCta * 32) group_mean_kernel(MergeParams p) {
  extern __shared__ __align__(16) uint32_t list[];
  __shared__ int warp_sums[33];
  grid_dependency_wait();   // the assignments come from the kernel before this one
  group_mean_body<T, VPL, R, kSlotsPerCta, kSlotsPerCta>(p, gridDim.y - 1 - blockIdx.y, blockIdx.x * kSlotsPerCta, list, warp_sums,
                                                         static_cast<int>(threadIdx.x), CtaSync());
}

template <typename T, int VPL, int R>
__global__ void __launch_bounds__(128) group_mean_bits_kernel(MergeParams p) {
  extern __shared__ __align__(16) unsigned char smem_bits[];
  grid_dependency_wait();   // the assignments come from the kernel before this one
  group_mean_bits_body<T, VPL, R>(p, gridDim.y - 1 - blockIdx.y, blockIdx.x * 4, smem_bits);
}

// ---- long instances (more than 2048 tokens): members by counting sort, segments put in order, then the sums.
// order_kernel, one CTA per instance: histogram of the assignments over the kept slots (shared-memory atomics),
// exclusive scan -> start[instance][n_kept + 1], then every token is dropped into its slot's segment of
// order[instance][n_tokens] (segment cursors are shared-memory atomics, so the order inside a segment is arbitrary).
__global__ void __launch_bounds__(1024) order_kernel(MergeParams p, int32_t* order, int32_t* start) {
  extern __shared__ __align__(16) int hist[];          // n_kept + 1 cursors
  __shared__ int warp_sums[33];
  grid_dependency_wait();                               // the assignments come from the kernel before this one
  const int b = blockIdx.x;
  const int32_t* ag = p.assign + static_cast<size_t>(b) * p.n_tokens;
  for (int s = threadIdx.x; s <= p.n_kept; s += blockDim.x) hist[s] = 0;
  __syncthreads();
  for (int i = threadIdx.x; i < p.n_tokens; i += blockDim.x) atomicAdd(&hist[min(max(__ldcg(ag + i), 0), p.n_kept - 1)], 1);
  __syncthreads();
  // exclusive scan of the n_kept counts, a contiguous run of slots per thread
  const int per = (p.n_kept + blockDim.x - 1) / blockDim.x;
  const int lo = min(p.n_kept, static_cast<int>(threadIdx.x) * per), hi = min(p.n_kept, lo + per);
  int mine = 0;
  for (int s = lo; s < hi; ++s) mine += hist[s];
  int total;
  int run = block_exclusive_scan(mine, warp_sums, total);
  int32_t* st = start + static_cast<size_t>(b) * (p.n_kept + 1);
  for (int s = lo; s < hi; ++s) { const int c = hist[s]; hist[s] = run; st[s] = run; run += c; }
  if (threadIdx.x == 0) st[p.n_kept] = total;
  __syncthreads();
  int32_t* od = order + static_cast<size_t>(b) * p.n_tokens;
  for (int i = threadIdx.x; i < p.n_tokens; i += blockDim.x) od[atomicAdd(&hist[min(max(__ldcg(ag + i), 0), p.n_kept - 1)], 1)] = i;
}

// sort_segments_kernel: one warp per kept slot puts its segment of `order` into ascending token order, in place:
// up to 32 members by rank counting in registers, up to kSortMax by a bitonic network in the warp's shared memory,
// beyond that (one slot holding thousands of tokens) by repeated minimum search.
constexpr int kSortMax = 2048;
__global__ void __launch_bounds__(256) sort_segments_kernel(MergeParams p, int32_t* order, const int32_t* start) {
  extern __shared__ __align__(16) int32_t sort_all[];
  grid_dependency_wait();
  const int b = blockIdx.y, w = threadIdx.x >> 5, lane = threadIdx.x & 31, s = blockIdx.x * 8 + w;
  if (s >= p.n_kept) return;
  const int32_t* st = start + static_cast<size_t>(b) * (p.n_kept + 1);
  const int seg0 = __ldcg(st + s), count = __ldcg(st + s + 1) - seg0;
  int32_t* seg = order + static_cast<size_t>(b) * p.n_tokens + seg0;
  if (count <= 1) return;
  if (count <= 32) {
    const int mine = lane < count ? __ldcg(seg + lane) : 0x7fffffff;
    int rank = 0;
#pragma unroll
    for (int l = 0; l < 32; ++l) rank += __shfl_sync(0xffffffffu, mine, l) < mine;   // ids are distinct
    if (lane < count) seg[rank] = mine;
    return;
  }
  if (count <= kSortMax) {
    int32_t* a = sort_all + w * kSortMax;
    int n = 64;
    while (n < count) n <<= 1;
    for (int i = lane; i < n; i += 32) a[i] = i < count ? __ldcg(seg + i) : 0x7fffffff;
    __syncwarp();
    for (int k = 2; k <= n; k <<= 1)
      for (int jj = k >> 1; jj > 0; jj >>= 1) {
        for (int idx = lane; idx < n / 2; idx += 32) {
          const int l = ((idx / jj) * 2 * jj) + (idx % jj), r = l + jj;
          const int x = a[l], y = a[r];
          const bool up = (l & k) == 0;
          if ((x > y) == up) { a[l] = y; a[r] = x; }
        }
        __syncwarp();
      }
    for (int i = lane; i < count; i += 32) seg[i] = a[i];
    return;
  }
  // oversized segment: selection sort with warp-wide minimum search (quadratic, for the pathological case only)
  for (int k = 0; k < count - 1; ++k) {
    int best = 0x7fffffff, at = -1;
    for (int i = k + lane; i < count; i += 32) { const int t = seg[i]; if (t < best) { best = t; at = i; } }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const int ob = __shfl_xor_sync(0xffffffffu, best, o), oa = __shfl_xor_sync(0xffffffffu, at, o);
      if (ob < best) { best = ob; at = oa; }
    }
    if (lane == 0 && at != k) { const int t = seg[k]; seg[k] = best; seg[at] = t; }
    __syncwarp();
  }
}

// group_mean_sorted_kernel: one warp per (kept slot, chunk of 32 * VPL 16-byte column pieces).  The warp walks the
// slot's ordered segment and adds the rows' chunk in that order, R rows in flight: the same additions in the same
// order as the other CUDA-core group means.  Splitting the columns over warps keeps a slot with hundreds of members
// from becoming one long chain.
template <typename T, int VPL, int R>
__global__ void __launch_bounds__(256) group_mean_sorted_kernel(MergeParams p, const int32_t* order, const int32_t* start, int chunks) {
  constexpr int E = Vec16<T>::kElems;
  grid_dependency_wait();
  const int b = gridDim.y - 1 - blockIdx.y, lane = threadIdx.x & 31;   // last instance first: the assignment pass has just read it
  const int task = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int s = task / chunks, v0 = (task - s * chunks) * 32 * VPL;
  if (s >= p.n_kept) return;
  const int32_t* st = start + static_cast<size_t>(b) * (p.n_kept + 1);
  const int seg0 = __ldcg(st + s), count = __ldcg(st + s + 1) - seg0;
  const int32_t* seg = order + static_cast<size_t>(b) * p.n_tokens + seg0;
  const int vecs = p.dim / E;
  const T* xb = static_cast<const T*>(p.x) + (static_cast<size_t>(b) * p.row_len + p.cls_offset) * p.dim;
  T* out = static_cast<T*>(p.merged) + (static_cast<size_t>(b) * p.n_kept + s) * p.dim;
  float acc[VPL][E];
#pragma unroll
  for (int i = 0; i < VPL; ++i)
#pragma unroll
    for (int e = 0; e < E; ++e) acc[i][e] = 0.f;
  for (int k0 = 0; k0 < count; k0 += 32) {
    const int mine = k0 + lane < count ? min(max(__ldcg(seg + k0 + lane), 0), p.n_tokens - 1) : -1;   // 32 members per round of ids
    const int here = min(32, count - k0);
    for (int k = 0; k < here; k += R) {
      uint4 raw[R][VPL];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const int tok = __shfl_sync(0xffffffffu, mine, min(k + r, 31));
        if (k + r < here) {
          const uint4* row = reinterpret_cast<const uint4*>(xb + static_cast<size_t>(tok) * p.dim);
#pragma unroll
          for (int i = 0; i < VPL; ++i) {
            const int v = v0 + lane + 32 * i;
            if (v < vecs) raw[r][i] = ld_nc_16(row + v);
          }
        }
      }
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if (k + r < here) {
#pragma unroll
          for (int i = 0; i < VPL; ++i) {
            const int v = v0 + lane + 32 * i;
            if (v < vecs) {
              float f[E];
              Vec16<T>::unpack(raw[r][i], f);
#pragma unroll
              for (int e = 0; e < E; ++e) acc[i][e] += f[e];
            }
          }
        }
      }
    }
  }
  const float inv = 1.f / static_cast<float>(max(count, 1));
#pragma unroll
  for (int i = 0; i < VPL; ++i) {
    const int v = v0 + lane + 32 * i;
    if (v < vecs) {
      float f[E];
#pragma unroll
      for (int e = 0; e < E; ++e) f[e] = acc[i][e] * inv;
      st_16(reinterpret_cast<uint4*>(out) + v, Vec16<T>::pack(f));
    }
  }
  if (v0 == 0 && lane == 0 && p.counts) p.counts[static_cast<size_t>(b) * p.n_kept + s] = count;
}

template <typename T>
static vscan_status launch_group_mean_sorted(const MergeParams& p, cudaStream_t stream) {
  constexpr int E = Vec16<T>::kElems, VPL = 1, R = 8;
  const size_t smem_order = (static_cast<size_t>(p.n_kept) + 1) * sizeof(int);
  VSCAN_CUDA_TRY(allow_smem(order_kernel, smem_order));
  VSCAN_LAUNCH("order_members", stream,
               (void)launch_dependent(order_kernel, dim3(p.instances), dim3(1024), smem_order, stream, p, p.order, p.order_start));
  const size_t smem_sort = 8 * kSortMax * sizeof(int32_t);
  VSCAN_CUDA_TRY(allow_smem(sort_segments_kernel, smem_sort));
  dim3 sgrid((p.n_kept + 7) / 8, p.instances);
  VSCAN_LAUNCH("order_members", stream,
               (void)launch_dependent(sort_segments_kernel, sgrid, dim3(256), smem_sort, stream, p, p.order,
                                      static_cast<const int32_t*>(p.order_start)));
  const int chunks = (p.dim / E + 32 * VPL - 1) / (32 * VPL);
  dim3 grid((static_cast<unsigned>(p.n_kept) * chunks + 7) / 8, p.instances);
  VSCAN_LAUNCH("group_mean", stream,
               (void)launch_dependent(group_mean_sorted_kernel<T, VPL, R>, grid, dim3(256), 0, stream, p,
                                      static_cast<const int32_t*>(p.order), static_cast<const int32_t*>(p.order_start), chunks));
  return VSCAN_OK;
}

template <typename T, int VPL, int R>
static vscan_status launch_group_mean_bits(const MergeParams& p, cudaStream_t stream) {
  const size_t chunks = (static_cast<size_t>(p.n_tokens) + 31) / 32;
  const size_t smem = 4 * chunks * 4 + 4 * static_cast<size_t>(p.n_tokens) * 2 + 16;
  dim3 grid((p.n_kept + 3) / 4, p.instances);
  VSCAN_CUDA_TRY(allow_smem(group_mean_bits_kernel<T, VPL, R>, smem));
  VSCAN_LAUNCH("group_mean", stream,
               (void)launch_dependent(group_mean_bits_kernel<T, VPL, R>, grid, dim3(128), smem, stream, p));
  return VSCAN_OK;
}

template <typename T, int VPL, int R, int SLOTS>
static vscan_status launch_group_mean_as(const MergeParams& p, size_t smem, cudaStream_t stream) {
  dim3 grid((p.n_kept + SLOTS - 1) / SLOTS, p.instances);
  VSCAN_CUDA_TRY(allow_smem(group_mean_kernel<T, VPL, R, SLOTS>, smem));
  VSCAN_LAUNCH("group_mean", stream,
               (void)launch_dependent(group_mean_kernel<T, VPL, R, SLOTS>, grid, dim3(SLOTS * 32), smem, stream, p));
  return VSCAN_OK;
}

template <typename T>
static vscan_status launch_group_mean(const MergeParams& p, cudaStream_t stream) {
  constexpr int E = Vec16<T>::kElems;
  const size_t smem = static_cast<size_t>(p.n_tokens) * 8 + 16;   // member list + staged assignments
  if (smem > kMaxDynamicSmem) return VSCAN_ERR_UNSUPPORTED;
  const bool wide = p.dim / E > 128, long_instance = p.n_tokens > 2048;
  // 512-thread CTAs have 128 registers per thread: wide rows are then summed in two column passes
  // (4 pieces per lane each) rather than with 8 pieces per lane, which would spill
  // long instances: counting sort + one warp per slot while groups are small on average (each warp orders its
  // own members); with few slots the groups are long lists, which the CTA-wide ordered listing handles better
  if (long_instance && static_cast<long long>(p.n_kept) * 64 >= p.n_tokens && p.order) return launch_group_mean_sorted<T>(p, stream);
  if (long_instance) return launch_group_mean_as<T, 4, 4, 16>(p, smem, stream);
  if (!wide) return launch_group_mean_bits<T, 2, 4>(p, stream);   // two column passes, few registers: more CTAs per SM
  return launch_group_mean_as<T, 8, 2, 4>(p, smem, stream);
}

}  // namespace vscan

using namespace vscan;

static vscan_status validate_merge(const vscan_merge_desc* d) {
  if (!d || !d->x || !d->kept_idx || !d->merged) return VSCAN_ERR_INVALID_ARG;
  if (d->dtype != VSCAN_F32 && d->dtype != VSCAN_BF16) return VSCAN_ERR_INVALID_ARG;
  if (d->path != VSCAN_MERGE_AUTO && d->path != VSCAN_MERGE_SIMT && d->path != VSCAN_MERGE_TENSOR &&
      d->path != VSCAN_MERGE_INTERLEAVED && d->path != VSCAN_MERGE_CLUSTER)
    return VSCAN_ERR_INVALID_ARG;
  if (d->instances < 0 || d->n_tokens <= 0 || d->cls_offset < 0 || d->row_len < d->cls_offset + d->n_tokens ||
      d->dim <= 0 || d->dim % 8 || d->n_kept < 1 || d->n_kept > d->n_tokens)
    return VSCAN_ERR_INVALID_ARG;
  if (d->metric && (d->metric_dim <= 0 || d->metric_dim % 8)) return VSCAN_ERR_INVALID_ARG;
  // the group-mean kernels stage one instance's member list and assignments in shared memory
  if (static_cast<size_t>(d->n_tokens) * 8 + 16 > kMaxDynamicSmem) return VSCAN_ERR_UNSUPPORTED;
  if (d->instances > 65535) return VSCAN_ERR_UNSUPPORTED;
  const void* ptrs[] = {d->x, d->metric, d->kept_idx, d->merged, d->assign, d->counts};
  for (const void* ptr : ptrs)
    if (ptr && !aligned16(ptr)) return VSCAN_ERR_INVALID_ARG;
  const size_t e = dtype_bytes(d->dtype), B = d->instances;
  struct Rng { const void* p; size_t n; };
  const Rng ins[] = {{d->x, B * d->row_len * d->dim * e},
                     {d->metric, d->metric ? B * d->row_len * d->metric_dim * e : 0},
                     {d->kept_idx, B * d->n_kept * 4}};
  const Rng outs[] = {{d->merged, B * d->n_kept * d->dim * e}, {d->assign, B * d->n_tokens * 4},
                      {d->counts, B * d->n_kept * 4}};
  for (const Rng& o : outs) {
    for (const Rng& i : ins)
      if (overlaps(o.p, o.n, i.p, i.n)) return VSCAN_ERR_INVALID_ARG;
    for (const Rng& o2 : outs)
      if (o.p != o2.p && overlaps(o.p, o.n, o2.p, o2.n)) return VSCAN_ERR_INVALID_ARG;
  }
  return VSCAN_OK;
}

// rows per instance of the packed copy of the kept rows: whole 256-row rounds for large kept sets, else
// the kept count rounded up to the MMA's granularity of 16
// kept sets above this size (at least four rounds of 256) are scanned in two shares by the CTA-pair assignment
constexpr int kSplitKept = 768;
static size_t packed_rows(int n_kept) { return n_kept > 256 ? round_up(n_kept, 256) : round_up(n_kept, 16); }

extern "C" size_t vscan_merge_workspace_bytes(const vscan_merge_desc* d) {
  if (!d || d->instances <= 0 || d->n_kept <= 0 || d->n_tokens <= 0) return kStatusBytes;
  size_t bytes = kStatusBytes;
  bytes += round_up(static_cast<size_t>(d->instances) * d->n_kept * sizeof(float), 256);    // inv_norm
  bytes += round_up(static_cast<size_t>(d->instances) * d->n_tokens * sizeof(int32_t), 256);  // assign
  if (d->n_tokens > 2048) {   // long instances: tokens ordered by slot, segment starts
    bytes += round_up(static_cast<size_t>(d->instances) * d->n_tokens * sizeof(int32_t), 256);
    bytes += round_up(static_cast<size_t>(d->instances) * (static_cast<size_t>(d->n_kept) + 1) * sizeof(int32_t), 256);
  }
  if (d->dtype == VSCAN_BF16) {   // packed copy of the kept rows for the tensor paths
    const size_t md = d->metric ? d->metric_dim : d->dim;
    bytes += round_up(static_cast<size_t>(d->instances) * packed_rows(d->n_kept) * md * 2, 256);
    bytes += round_up((static_cast<size_t>(d->instances) + 1) * sizeof(int), 256);   // counters of the persistent path
    if (d->n_kept > kSplitKept) {   // the kept set is scanned in two shares: their partial results and the tiles' tickets
      bytes += round_up(2 * static_cast<size_t>(d->instances) * d->n_tokens * sizeof(float2), 256);
      bytes += round_up(static_cast<size_t>(d->instances) * ((d->n_tokens + 127) / 128) * sizeof(int), 256);
    }
  }
  return bytes;
}

extern "C" vscan_status vscan_merge(const vscan_merge_desc* d, void* workspace, size_t workspace_bytes,
                                    void* stream_) {
  if (d && d->instances == 0) return VSCAN_OK;  // empty batch
  vscan_status st = validate_merge(d);
  if (st != VSCAN_OK) return st;
  if (d->instances == 0) return VSCAN_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const size_t need = vscan_merge_workspace_bytes(d);
  if (!workspace || !aligned256(workspace) || workspace_bytes < need) return VSCAN_ERR_WORKSPACE;

  MergeParams p;
  p.x = d->x;
  p.metric = d->metric ? d->metric : d->x;
  p.metric_dim = d->metric ? d->metric_dim : d->dim;
  p.kept = d->kept_idx;
  char* ws = static_cast<char*>(workspace);
  p.status = reinterpret_cast<uint32_t*>(ws);
  p.inv_norm = reinterpret_cast<float*>(ws + kStatusBytes);
  int32_t* ws_assign = reinterpret_cast<int32_t*>(
      ws + kStatusBytes + round_up(static_cast<size_t>(d->instances) * d->n_kept * sizeof(float), 256));
  p.assign = d->assign ? d->assign : ws_assign;
  char* ws_next = reinterpret_cast<char*>(ws_assign) + round_up(static_cast<size_t>(d->instances) * d->n_tokens * sizeof(int32_t), 256);
  p.order = nullptr; p.order_start = nullptr;
  if (d->n_tokens > 2048) {
    p.order = reinterpret_cast<int32_t*>(ws_next);
    ws_next += round_up(static_cast<size_t>(d->instances) * d->n_tokens * sizeof(int32_t), 256);
    p.order_start = reinterpret_cast<int32_t*>(ws_next);
    ws_next += round_up(static_cast<size_t>(d->instances) * (static_cast<size_t>(d->n_kept) + 1) * sizeof(int32_t), 256);
  }
  p.kept_packed = d->dtype == VSCAN_BF16 ? static_cast<void*>(ws_next) : nullptr;
  p.counters = p.kept_packed ? reinterpret_cast<int*>(static_cast<char*>(p.kept_packed) +
                                                      round_up(static_cast<size_t>(d->instances) * packed_rows(d->n_kept) * p.metric_dim * 2, 256))
                             : nullptr;
  p.partial = nullptr; p.tickets = nullptr;
  if (p.counters && d->n_kept > kSplitKept) {
    char* after = reinterpret_cast<char*>(p.counters) + round_up((static_cast<size_t>(d->instances) + 1) * sizeof(int), 256);
    p.partial = reinterpret_cast<float2*>(after);
    p.tickets = reinterpret_cast<int*>(after + round_up(2 * static_cast<size_t>(d->instances) * d->n_tokens * sizeof(float2), 256));
  }
  p.merged = d->merged; p.counts = d->counts;
  p.instances = d->instances; p.row_len = d->row_len; p.cls_offset = d->cls_offset;
  p.n_tokens = d->n_tokens; p.dim = d->dim; p.n_kept = d->n_kept;
  p.clear_status = 1;

  // one pass over the features, a cluster per instance: on request only (see the measurements in the design notes)
  if (d->path == VSCAN_MERGE_CLUSTER) {
    if (!merge_cluster_supported(d->dtype, p)) return VSCAN_ERR_UNSUPPORTED;
    return launch_merge_cluster(p, stream);
  }

  // assignment and group means in one persistent launch: on request only.  (It was the choice for kept sets of
  // 129-256 until the assignment on CTA pairs, which takes packed kept rows at any size above 128: 230 us against
  // 103 + 79 us for 256 instances with 192 kept tokens.)
  if (d->path == VSCAN_MERGE_INTERLEAVED) {
    if (merge_interleaved_supported(d->dtype, p)) {
      st = launch_merge_interleaved(p, stream);
      if (st != VSCAN_ERR_UNSUPPORTED || d->path == VSCAN_MERGE_INTERLEAVED) return st;
    } else if (d->path == VSCAN_MERGE_INTERLEAVED) {
      return VSCAN_ERR_UNSUPPORTED;
    }
  }

  bool tensor = false;
  if (d->path == VSCAN_MERGE_TENSOR) {
    if (!assign_tensor_supported(d->dtype, p)) return VSCAN_ERR_UNSUPPORTED;
    tensor = true;
  } else if (d->path == VSCAN_MERGE_AUTO) {
    tensor = assign_tensor_supported(d->dtype, p);
  }

  // the tensor path takes the norms of the kept rows itself; the CUDA-core path gets them from a
  // small kernel of its own
  st = VSCAN_ERR_UNSUPPORTED;
  if (tensor) {
    st = launch_assign_tensor(p, stream);   // clears the status word itself
    if (st != VSCAN_OK && (st != VSCAN_ERR_UNSUPPORTED || d->path != VSCAN_MERGE_AUTO)) return st;
  }
  if (st == VSCAN_ERR_UNSUPPORTED) {   // CUDA cores (asked for, or a shape the tensor path cannot take)
    dim3 ngrid((d->n_kept + 7) / 8, d->instances);
    if (d->dtype == VSCAN_F32) VSCAN_LAUNCH("kept_inv_norm", stream, kept_inv_norm_kernel<float><<<ngrid, 256, 0, stream>>>(p));
    else VSCAN_LAUNCH("kept_inv_norm", stream, kept_inv_norm_kernel<__nv_bfloat16><<<ngrid, 256, 0, stream>>>(p));
    st = launch_assign_simt(d->dtype, p, stream);
    if (st != VSCAN_OK) return st;
  }
  // (Cutting the batch into runs of instances small enough for L2, so that the group-mean pass of a
  // run finds its features there, was measured slower: the smaller grids are latency-bound.)
  if (d->dtype == VSCAN_F32) return launch_group_mean<float>(p, stream);
  // after a tensor-core assignment the sums run on the tensor cores too where the shape allows
  if (tensor && group_sum_tensor_supported(d->dtype, p)) return launch_group_sum_tensor(p, stream);
  return launch_group_mean<__nv_bfloat16>(p, stream);
}
