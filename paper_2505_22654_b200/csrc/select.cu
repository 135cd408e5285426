// vscan_select_global_local: local scan (Eq. 3), global scan (Eq. 2) over the complement, union.
// One CTA per encoder instance; all state of the instance lives in shared memory.
#include <type_traits>

#include "topk.cuh"

namespace vscan {

struct SelectParams {
  const float* scores_global;
  const float* scores_local;
  // fused form: the scores are the head means of these attention rows (Eq. 2), taken here
  const void* attn_global;
  const void* attn_local;
  float* scores_global_out;   // optional
  float* scores_local_out;    // optional
  int heads, row_len, cls_offset;
  int32_t* kept_idx;
  uint8_t* kept_mask;
  int n, frames, grid_h, grid_w, win_h, win_w, k_w, k_g, windows, wins_per_row, wins_per_frame;
};

// Head mean of one token's attention entries, heads ascending (same arithmetic as the ROW-mode score).
template <typename T>
__device__ __forceinline__ float head_mean_of(const T* base, int heads, int row_len) {
  float acc = 0.f;
  int h = 0;
  for (; h + 16 <= heads; h += 16) {   // sixteen independent loads in flight, added in head order
    T a[16];
#pragma unroll
    for (int u = 0; u < 16; ++u) a[u] = base[static_cast<size_t>(h + u) * row_len];
#pragma unroll
    for (int u = 0; u < 16; ++u) acc += to_float(a[u]);
  }
  for (; h + 4 <= heads; h += 4) {
    T a[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) a[u] = base[static_cast<size_t>(h + u) * row_len];
#pragma unroll
    for (int u = 0; u < 4; ++u) acc += to_float(a[u]);
  }
  for (; h < heads; ++h) acc += to_float(base[static_cast<size_t>(h) * row_len]);
  return acc / static_cast<float>(heads);
}

// dynamic shared memory: keys_g[n] | keys_l[n] | taken[n] (bytes)
// T = void: scores are read; T = element type: scores are computed from the attention rows.
template <typename T>
__global__ void __launch_bounds__(1024) select_kernel(SelectParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint32_t* keys_g = reinterpret_cast<uint32_t*>(smem_raw);
  uint32_t* keys_l = keys_g + p.n;
  uint8_t* taken = reinterpret_cast<uint8_t*>(keys_l + p.n);
  __shared__ SelectScratch sc;
  grid_dependency_launch();

  const int b = blockIdx.x;
  if constexpr (std::is_void<T>::value) {
    const float* sg = p.scores_global + static_cast<size_t>(b) * p.n;
    const float* sl = p.scores_local + static_cast<size_t>(b) * p.n;
    for (int i = threadIdx.x; i < p.n; i += blockDim.x) {
      keys_g[i] = float_to_key(sg[i]);
      keys_l[i] = float_to_key(sl[i]);
      taken[i] = 0;
    }
  } else {
    const size_t inst = static_cast<size_t>(b) * p.heads * p.row_len + p.cls_offset;
    const T* ag = static_cast<const T*>(p.attn_global) + inst;
    const T* al = static_cast<const T*>(p.attn_local) + inst;
    for (int i = threadIdx.x; i < p.n; i += blockDim.x) {
      const bool same = p.attn_local == p.attn_global;
      float g, l;
      if (!same && p.heads == 16) {   // the common head count: all 32 loads of the token in flight at once
        T a[16], c[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) { a[u] = ag[i + static_cast<size_t>(u) * p.row_len]; c[u] = al[i + static_cast<size_t>(u) * p.row_len]; }
        g = 0.f; l = 0.f;
#pragma unroll
        for (int u = 0; u < 16; ++u) { g += to_float(a[u]); l += to_float(c[u]); }
        g /= 16.f; l /= 16.f;
      } else {
        g = head_mean_of(ag + i, p.heads, p.row_len);
        l = same ? g : head_mean_of(al + i, p.heads, p.row_len);
      }
      if (p.scores_global_out) p.scores_global_out[static_cast<size_t>(b) * p.n + i] = g;
      if (p.scores_local_out) p.scores_local_out[static_cast<size_t>(b) * p.n + i] = l;
      keys_g[i] = float_to_key(g);
      keys_l[i] = float_to_key(l);
      taken[i] = 0;
    }
  }
  __syncthreads();

  // ---- local scan: one warp per window, windows dealt round-robin
  if (p.k_w > 0) {
    const int warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int m = p.win_h * p.win_w;
    for (int w = warp; w < p.windows; w += nwarps) {
      const int f = w / p.wins_per_frame, wr = (w % p.wins_per_frame) / p.wins_per_row,
                wc = w % p.wins_per_row;
      const int base = f * p.grid_h * p.grid_w + wr * p.win_h * p.grid_w + wc * p.win_w;
      const int win_w = p.win_w, grid_w = p.grid_w;
      auto token_of = [=](int q) { return base + (q / win_w) * grid_w + (q % win_w); };
      if (m <= 64) warp_rank_mark(keys_l, m, p.k_w, token_of, taken);
      else warp_select_mark(keys_l, m, p.k_w, token_of, taken);
    }
  }
  __syncthreads();

  // ---- global scan over the tokens the local scan left
  uint32_t thr = 0;
  int need = 0;
  if (p.k_g > 0) block_radix_select(keys_g, taken, p.n, p.k_g, sc, thr, need);

  // ---- union, ascending.  Each thread owns a contiguous run of tokens.
  const int per = (p.n + blockDim.x - 1) / blockDim.x;
  const int lo = min(p.n, static_cast<int>(threadIdx.x) * per), hi = min(p.n, lo + per);
  int eq_before = 0;
  {
    int eq_local = 0;
    if (p.k_g > 0)
      for (int i = lo; i < hi; ++i) eq_local += (!taken[i] && keys_g[i] == thr);
    int total;
    eq_before = block_exclusive_scan(eq_local, sc.warp_sums, total);
  }
  int kept_local = 0;
  for (int i = lo; i < hi; ++i) {
    bool keep = taken[i];
    if (!keep && p.k_g > 0) {
      uint32_t key = keys_g[i];
      if (key > thr) keep = true;
      else if (key == thr) { keep = eq_before < need; ++eq_before; }
    }
    // reuse keys_l as the flag array (local keys are no longer needed)
    keys_l[i] = keep ? 1u : 0u;
    kept_local += keep;
  }
  int total_kept;
  int pos = block_exclusive_scan(kept_local, sc.warp_sums, total_kept);
  const int k1 = p.windows * p.k_w + p.k_g;
  int32_t* out = p.kept_idx + static_cast<size_t>(b) * k1;
  for (int i = lo; i < hi; ++i)
    if (keys_l[i]) { if (pos < k1) out[pos] = i; ++pos; }
  if (p.kept_mask) {
    __syncthreads();
    uint8_t* mk = p.kept_mask + static_cast<size_t>(b) * p.n;
    for (int i = threadIdx.x; i < p.n; i += blockDim.x) mk[i] = static_cast<uint8_t>(keys_l[i]);
  }
}

}  // namespace vscan

using namespace vscan;

extern "C" size_t vscan_select_workspace_bytes(const vscan_select_desc*) { return 0; }

static vscan_status validate_grid(const vscan_select_desc* d, long long* n_out, int* windows_out, long long* k1_out) {
  if (d->instances < 0 || d->frames <= 0 || d->grid_h <= 0 || d->grid_w <= 0 || d->win_h <= 0 || d->win_w <= 0)
    return VSCAN_ERR_INVALID_ARG;
  if (d->grid_h % d->win_h || d->grid_w % d->win_w) return VSCAN_ERR_INVALID_ARG;
  const long long n = 1ll * d->frames * d->grid_h * d->grid_w;
  if (n > 16384) return VSCAN_ERR_UNSUPPORTED;
  if (d->instances > 65535) return VSCAN_ERR_UNSUPPORTED;
  const int windows = d->frames * (d->grid_h / d->win_h) * (d->grid_w / d->win_w);
  if (d->k_per_window < 0 || d->k_per_window > d->win_h * d->win_w) return VSCAN_ERR_INVALID_ARG;
  const long long local_total = 1ll * windows * d->k_per_window;
  if (d->k_global < 0 || d->k_global > n - local_total) return VSCAN_ERR_INVALID_ARG;
  *n_out = n; *windows_out = windows; *k1_out = local_total + d->k_global;
  return VSCAN_OK;
}

static void fill_params(SelectParams& p, const vscan_select_desc* d, long long n, int windows) {
  p = SelectParams{};
  p.scores_global = d->scores_global; p.scores_local = d->scores_local;
  p.kept_idx = d->kept_idx; p.kept_mask = d->kept_mask;
  p.n = static_cast<int>(n); p.frames = d->frames; p.grid_h = d->grid_h; p.grid_w = d->grid_w;
  p.win_h = d->win_h; p.win_w = d->win_w; p.k_w = d->k_per_window; p.k_g = d->k_global;
  p.windows = windows; p.wins_per_row = d->grid_w / d->win_w;
  p.wins_per_frame = (d->grid_h / d->win_h) * p.wins_per_row;
}

// One warp per window while there are enough windows to fill the block.
static int select_threads(long long n, int windows) {
  if (n > 2048) return 1024;
  // a thread per token where that is possible, so that the scores of an instance are read in one round of loads
  if (n > 512 && n <= 1024) return static_cast<int>((n + 31) / 32 * 32);
  return windows > 8 || n > 256 ? 512 : 256;
}

extern "C" vscan_status vscan_select_global_local(const vscan_select_desc* d, void* /*workspace*/,
                                                  size_t /*workspace_bytes*/, void* stream) {
  if (d && d->instances == 0) return VSCAN_OK;  // empty batch
  if (!d || !d->scores_global || !d->scores_local || !d->kept_idx) return VSCAN_ERR_INVALID_ARG;
  long long n, k1;
  int windows;
  vscan_status vs = validate_grid(d, &n, &windows, &k1);
  if (vs != VSCAN_OK) return vs;
  if (!aligned16(d->scores_global) || !aligned16(d->scores_local) || !aligned16(d->kept_idx))
    return VSCAN_ERR_INVALID_ARG;
  const size_t sbytes = static_cast<size_t>(d->instances) * n * 4, obytes = static_cast<size_t>(d->instances) * k1 * 4;
  const size_t mbytes = static_cast<size_t>(d->instances) * n;
  if (overlaps(d->kept_idx, obytes, d->scores_global, sbytes) || overlaps(d->kept_idx, obytes, d->scores_local, sbytes) ||
      overlaps(d->kept_mask, mbytes, d->scores_global, sbytes) || overlaps(d->kept_mask, mbytes, d->scores_local, sbytes) ||
      overlaps(d->kept_mask, mbytes, d->kept_idx, obytes))
    return VSCAN_ERR_INVALID_ARG;

  SelectParams p;
  fill_params(p, d, n, windows);
  const size_t smem = static_cast<size_t>(n) * 9 + 16;
  VSCAN_CUDA_TRY(allow_smem(select_kernel<void>, smem));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  VSCAN_LAUNCH("select", st, select_kernel<void><<<d->instances, select_threads(n, windows), smem, st>>>(p));
  return VSCAN_OK;
}

extern "C" vscan_status vscan_score_select(const vscan_score_select_desc* d, void* stream) {
  if (d && d->select.instances == 0) return VSCAN_OK;  // empty batch
  if (!d || !d->attn_global || !d->attn_local || !d->select.kept_idx) return VSCAN_ERR_INVALID_ARG;
  if (d->dtype != VSCAN_F32 && d->dtype != VSCAN_BF16) return VSCAN_ERR_INVALID_ARG;
  const vscan_select_desc* sd = &d->select;
  long long n, k1;
  int windows;
  vscan_status vs = validate_grid(sd, &n, &windows, &k1);
  if (vs != VSCAN_OK) return vs;
  if (d->heads <= 0 || d->cls_offset < 0 || d->row_len < d->cls_offset + n) return VSCAN_ERR_INVALID_ARG;
  const void* ptrs[] = {d->attn_global, d->attn_local, sd->kept_idx, sd->scores_global, sd->scores_local};
  for (const void* ptr : ptrs)
    if (ptr && !aligned16(ptr)) return VSCAN_ERR_INVALID_ARG;
  const size_t abytes = static_cast<size_t>(sd->instances) * d->heads * d->row_len * dtype_bytes(d->dtype);
  const size_t sbytes = static_cast<size_t>(sd->instances) * n * 4, obytes = static_cast<size_t>(sd->instances) * k1 * 4;
  const size_t mbytes = static_cast<size_t>(sd->instances) * n;
  struct Rng { const void* p; size_t n; };
  const Rng outs[] = {{sd->kept_idx, obytes}, {sd->kept_mask, mbytes}, {sd->scores_global, sbytes}, {sd->scores_local, sbytes}};
  for (const Rng& o : outs) {
    if (overlaps(o.p, o.n, d->attn_global, abytes) || overlaps(o.p, o.n, d->attn_local, abytes)) return VSCAN_ERR_INVALID_ARG;
    for (const Rng& o2 : outs)
      if (o.p != o2.p && overlaps(o.p, o.n, o2.p, o2.n)) return VSCAN_ERR_INVALID_ARG;
  }
  if (sd->scores_global && sd->scores_global == sd->scores_local && d->attn_global != d->attn_local)
    return VSCAN_ERR_INVALID_ARG;

  SelectParams p;
  fill_params(p, sd, n, windows);
  p.scores_global = nullptr; p.scores_local = nullptr;
  p.attn_global = d->attn_global; p.attn_local = d->attn_local;
  p.scores_global_out = const_cast<float*>(sd->scores_global);
  p.scores_local_out = const_cast<float*>(sd->scores_local);
  p.heads = d->heads; p.row_len = d->row_len; p.cls_offset = d->cls_offset;
  const size_t smem = static_cast<size_t>(n) * 9 + 16;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int threads = select_threads(n, windows);
  if (d->dtype == VSCAN_F32) {
    VSCAN_CUDA_TRY(allow_smem(select_kernel<float>, smem));
    VSCAN_LAUNCH("score_select", st, select_kernel<float><<<sd->instances, threads, smem, st>>>(p));
  } else {
    VSCAN_CUDA_TRY(allow_smem(select_kernel<__nv_bfloat16>, smem));
    VSCAN_LAUNCH("score_select", st, select_kernel<__nv_bfloat16><<<sd->instances, threads, smem, st>>>(p));
  }
  return VSCAN_OK;
}
