// vscan_select_global_local: local scan (Eq. 3), global scan (Eq. 2) over the complement, union.
// One CTA per encoder instance; all state of the instance lives in shared memory.
#include "topk.cuh"

namespace vscan {

struct SelectParams {
  const float* scores_global;
  const float* scores_local;
  int32_t* kept_idx;
  uint8_t* kept_mask;
  int n, frames, grid_h, grid_w, win_h, win_w, k_w, k_g, windows, wins_per_row, wins_per_frame;
};

// dynamic shared memory: keys_g[n] | keys_l[n] | taken[n] (bytes)
__global__ void __launch_bounds__(1024) select_kernel(SelectParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint32_t* keys_g = reinterpret_cast<uint32_t*>(smem_raw);
  uint32_t* keys_l = keys_g + p.n;
  uint8_t* taken = reinterpret_cast<uint8_t*>(keys_l + p.n);
  __shared__ SelectScratch sc;

  const int b = blockIdx.x;
  const float* sg = p.scores_global + static_cast<size_t>(b) * p.n;
  const float* sl = p.scores_local + static_cast<size_t>(b) * p.n;
  for (int i = threadIdx.x; i < p.n; i += blockDim.x) {
    keys_g[i] = float_to_key(sg[i]);
    keys_l[i] = float_to_key(sl[i]);
    taken[i] = 0;
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
      warp_select_mark(keys_l, m, p.k_w,
                       [=](int q) { return base + (q / win_w) * grid_w + (q % win_w); }, taken);
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

extern "C" vscan_status vscan_select_global_local(const vscan_select_desc* d, void* /*workspace*/,
                                                  size_t /*workspace_bytes*/, void* stream) {
  if (d && d->instances == 0) return VSCAN_OK;  // empty batch
  if (!d || !d->scores_global || !d->scores_local || !d->kept_idx) return VSCAN_ERR_INVALID_ARG;
  if (d->instances < 0 || d->frames <= 0 || d->grid_h <= 0 || d->grid_w <= 0 || d->win_h <= 0 ||
      d->win_w <= 0)
    return VSCAN_ERR_INVALID_ARG;
  if (d->grid_h % d->win_h || d->grid_w % d->win_w) return VSCAN_ERR_INVALID_ARG;
  const long long n = 1ll * d->frames * d->grid_h * d->grid_w;
  if (n > 16384) return VSCAN_ERR_UNSUPPORTED;
  const int windows = d->frames * (d->grid_h / d->win_h) * (d->grid_w / d->win_w);
  if (d->k_per_window < 0 || d->k_per_window > d->win_h * d->win_w) return VSCAN_ERR_INVALID_ARG;
  const long long local_total = 1ll * windows * d->k_per_window;
  if (d->k_global < 0 || d->k_global > n - local_total) return VSCAN_ERR_INVALID_ARG;
  const long long k1 = local_total + d->k_global;
  if (!aligned16(d->scores_global) || !aligned16(d->scores_local) || !aligned16(d->kept_idx))
    return VSCAN_ERR_INVALID_ARG;
  const size_t sbytes = static_cast<size_t>(d->instances) * n * 4, obytes = static_cast<size_t>(d->instances) * k1 * 4;
  if (overlaps(d->kept_idx, obytes, d->scores_global, sbytes) ||
      overlaps(d->kept_idx, obytes, d->scores_local, sbytes) ||
      overlaps(d->kept_mask, static_cast<size_t>(d->instances) * n, d->scores_global, sbytes) ||
      overlaps(d->kept_mask, static_cast<size_t>(d->instances) * n, d->scores_local, sbytes) ||
      overlaps(d->kept_mask, static_cast<size_t>(d->instances) * n, d->kept_idx, obytes))
    return VSCAN_ERR_INVALID_ARG;
  if (d->instances == 0) return VSCAN_OK;

  SelectParams p;
  p.scores_global = d->scores_global; p.scores_local = d->scores_local;
  p.kept_idx = d->kept_idx; p.kept_mask = d->kept_mask;
  p.n = static_cast<int>(n); p.frames = d->frames; p.grid_h = d->grid_h; p.grid_w = d->grid_w;
  p.win_h = d->win_h; p.win_w = d->win_w; p.k_w = d->k_per_window; p.k_g = d->k_global;
  p.windows = windows; p.wins_per_row = d->grid_w / d->win_w;
  p.wins_per_frame = (d->grid_h / d->win_h) * p.wins_per_row;
  const size_t smem = static_cast<size_t>(n) * 9 + 16;
  VSCAN_CUDA_TRY(allow_smem(select_kernel, smem));
  const int threads = n <= 2048 ? 256 : 1024;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  VSCAN_LAUNCH("select", st, select_kernel<<<d->instances, threads, smem, st>>>(p));
  return VSCAN_OK;
}
