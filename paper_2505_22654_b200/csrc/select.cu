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
  // ceil(2^32 / d) for d = tokens per frame, grid_w, win_h, win_w: umulhi(x, rcp) == x / d for x * d < 2^32
  uint32_t rcp_frame, rcp_grid_w, rcp_win_h, rcp_win_w;
  // cluster form: window-row bands (win_h grid rows of one frame) handled by each CTA of a cluster
  int bands_per_cta;
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

// ---------------------------------------------------------------------------------------------
// Instances of at most 1024 tokens: one thread per token, keys in registers.
//   loads   fused form: the instance's [heads][row_len] block of each attention tensor is one contiguous run
//           of memory; when it is 16-byte aligned it comes in as one bulk copy per tensor (mbarrier with
//           transaction count) and the head means are taken out of shared memory, else (or if the copy does
//           not arrive within the wait's bound) with one strided load per head as in the large kernel
//   local   one warp per window, rank counting in registers (or the 32-step bit select for windows above 64)
//   global  the k_g-th largest key of the complement by binary search on the key's bits, one
//           barrier-with-count per varying bit (bits that all candidates share are skipped)
//   union   warp ballots and one exchange of per-warp counts: position = kept tokens before mine
// dynamic shared memory: keys_l[n] | taken[n] bytes (padded to 16) | staging for the two attention blocks
// x / d through the host's ceil(2^32 / d) (d = 1 has no 32-bit reciprocal)
__device__ __forceinline__ int quot(int x, int d, uint32_t rcp) {
  return d == 1 ? x : static_cast<int>(__umulhi(static_cast<uint32_t>(x), rcp));
}

struct SmallScratch {
  int warp_sure[32], warp_eq[32];
  uint32_t bits_or, bits_and;
  unsigned long long mbar;
};

template <typename T>
__global__ void __launch_bounds__(1024) select_small_kernel(SelectParams p, int stage_bytes) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint32_t* keys_l = reinterpret_cast<uint32_t*>(smem_raw);
  uint8_t* taken = reinterpret_cast<uint8_t*>(keys_l + p.n);
  __shared__ SmallScratch sc;
  grid_dependency_launch();

  const int b = blockIdx.x, i = threadIdx.x, lane = i & 31, warp = i >> 5, nwarps = blockDim.x >> 5;
  const bool live = i < p.n;
  float g = 0.f, l = 0.f;
  if constexpr (std::is_void<T>::value) {
    if (live) {
      g = p.scores_global[static_cast<size_t>(b) * p.n + i];
      l = p.scores_local[static_cast<size_t>(b) * p.n + i];
    }
  } else {
    const size_t block_elems = static_cast<size_t>(p.heads) * p.row_len;
    const T* ag = static_cast<const T*>(p.attn_global) + static_cast<size_t>(b) * block_elems;
    const T* al = static_cast<const T*>(p.attn_local) + static_cast<size_t>(b) * block_elems;
    const bool same = p.attn_local == p.attn_global;
    bool staged = false;
    if (stage_bytes > 0) {
      unsigned char* stage = smem_raw + ((static_cast<size_t>(p.n) * 5 + 15) / 16) * 16;
      const uint32_t bar = static_cast<uint32_t>(__cvta_generic_to_shared(&sc.mbar));
      if (i == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(same ? stage_bytes : 2 * stage_bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(stage))), "l"(ag), "r"(stage_bytes), "r"(bar) : "memory");
        if (!same)
          asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                       ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(stage + stage_bytes))), "l"(al), "r"(stage_bytes), "r"(bar) : "memory");
      }
      __syncthreads();   // the barrier is initialised before anyone polls it
      uint32_t done = 0;
      for (uint32_t spin = 0; spin < (1u << 20) && !done; ++spin)
        asm volatile("{\n\t.reg .pred q;\n\tmbarrier.try_wait.parity.shared::cta.b64 q, [%1], 0;\n\tselp.u32 %0, 1, 0, q;\n\t}"
                     : "=r"(done) : "r"(bar) : "memory");
      staged = __syncthreads_and(done != 0) != 0;   // all or nobody: a copy that did not arrive is not relied on
      if (staged && live) {
        const T* sg = reinterpret_cast<const T*>(stage) + p.cls_offset + i;
        const T* sl = same ? sg : reinterpret_cast<const T*>(stage + stage_bytes) + p.cls_offset + i;
        for (int h = 0; h < p.heads; ++h) g += to_float(sg[static_cast<size_t>(h) * p.row_len]);
        g /= static_cast<float>(p.heads);
        if (same) l = g;
        else {
          for (int h = 0; h < p.heads; ++h) l += to_float(sl[static_cast<size_t>(h) * p.row_len]);
          l /= static_cast<float>(p.heads);
        }
      }
    }
    if (!staged && live) {
      g = head_mean_of(ag + p.cls_offset + i, p.heads, p.row_len);
      l = same ? g : head_mean_of(al + p.cls_offset + i, p.heads, p.row_len);
    }
    if (live) {
      if (p.scores_global_out) p.scores_global_out[static_cast<size_t>(b) * p.n + i] = g;
      if (p.scores_local_out) p.scores_local_out[static_cast<size_t>(b) * p.n + i] = l;
    }
  }
  const uint32_t key = float_to_key(g);
  if (live) { keys_l[i] = float_to_key(l); taken[i] = 0; }
  if (i == 0) { sc.bits_or = 0u; sc.bits_and = 0xFFFFFFFFu; }
  __syncthreads();

  // ---- local scan.  Windows of up to 128 tokens: every thread ranks its own token among the tokens of its
  // window (kept iff fewer than k_w of them beat it: larger key, or equal key and lower index), all warps busy
  // and no warp-wide chain.  Larger windows: one warp per window with the 32-step bit select.
  bool mine_taken = false;
  if (p.k_w > 0) {
    const int m = p.win_h * p.win_w;
    if (m <= 128) {
      if (live) {
        // quotients by multiplication with the host's rounded-up reciprocals (exact for these ranges)
        const int per_frame = p.grid_h * p.grid_w;
        const int f = quot(i, per_frame, p.rcp_frame), rem = i - f * per_frame;
        const int r = quot(rem, p.grid_w, p.rcp_grid_w), c = rem - r * p.grid_w;
        const int wr = quot(r, p.win_h, p.rcp_win_h), wc = quot(c, p.win_w, p.rcp_win_w);
        const int base = f * per_frame + wr * p.win_h * p.grid_w + wc * p.win_w;
        const uint32_t mykey = keys_l[i];
        int rank = 0;
        for (int wy = 0; wy < p.win_h; ++wy) {
          const int row = base + wy * p.grid_w;
          for (int wx0 = 0; wx0 < p.win_w; wx0 += 8) {     // eight independent loads per round
            uint32_t kt[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) kt[u] = wx0 + u < p.win_w ? keys_l[row + wx0 + u] : 0u;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const int t = row + wx0 + u;
              rank += (wx0 + u < p.win_w) && ((kt[u] > mykey) || (kt[u] == mykey && t < i));
            }
          }
        }
        mine_taken = rank < p.k_w;
      }
    } else {
      for (int w = warp; w < p.windows; w += nwarps) {
        const int f = w / p.wins_per_frame, wr = (w % p.wins_per_frame) / p.wins_per_row, wc = w % p.wins_per_row;
        const int base = f * p.grid_h * p.grid_w + wr * p.win_h * p.grid_w + wc * p.win_w;
        const int win_w = p.win_w, grid_w = p.grid_w;
        auto token_of = [=](int q) { return base + (q / win_w) * grid_w + (q % win_w); };
        warp_select_mark(keys_l, m, p.k_w, token_of, taken);
      }
      __syncthreads();
      mine_taken = live && taken[i];
    }
  }
  const bool cand = live && !mine_taken;

  // ---- global scan: threshold = k_g-th largest candidate key, need = how many keys equal to it belong to the set
  uint32_t thr = 0;
  int need = 0;
  if (p.k_g > 0) {
    // bits on which all candidates agree cannot decide anything: start below them
    const uint32_t wo = __reduce_or_sync(0xffffffffu, cand ? key : 0u);
    const uint32_t wa = __reduce_and_sync(0xffffffffu, cand ? key : 0xFFFFFFFFu);
    if (lane == 0) { atomicOr(&sc.bits_or, wo); atomicAnd(&sc.bits_and, wa); }
    __syncthreads();
    const uint32_t differ = sc.bits_or ^ sc.bits_and;
    const int top = differ ? 31 - __clz(differ) : -1;            // highest bit that varies
    // the leading bits all candidates share (all 32 when no bit varies: the threshold is that one key)
    thr = top < 0 ? sc.bits_and : (top == 31 ? 0u : (sc.bits_and & ~((2u << top) - 1u)));
    for (int bit = top; bit >= 0; --bit) {
      const uint32_t t = thr | (1u << bit);
      if (__syncthreads_count(cand && key >= t) >= p.k_g) thr = t;
    }
    need = p.k_g - __syncthreads_count(cand && key > thr);
  }

  // ---- union, ascending: a token's position is the number of kept tokens before it
  const bool sure = mine_taken || (cand && p.k_g > 0 && key > thr);
  const bool eq = cand && p.k_g > 0 && key == thr;
  const unsigned b_sure = __ballot_sync(0xffffffffu, sure), b_eq = __ballot_sync(0xffffffffu, eq);
  if (lane == 0) { sc.warp_sure[warp] = __popc(b_sure); sc.warp_eq[warp] = __popc(b_eq); }
  __syncthreads();
  int ws = lane < nwarps ? sc.warp_sure[lane] : 0, we = lane < nwarps ? sc.warp_eq[lane] : 0;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int a = __shfl_up_sync(0xffffffffu, ws, o), c = __shfl_up_sync(0xffffffffu, we, o);
    if (lane >= o) { ws += a; we += c; }
  }
  const int sure_warps = warp > 0 ? __shfl_sync(0xffffffffu, ws, warp - 1) : 0;   // inclusive sums of the warps before mine
  const int eq_warps = warp > 0 ? __shfl_sync(0xffffffffu, we, warp - 1) : 0;
  const unsigned lt = (1u << lane) - 1u;
  const int eq_rank = eq_warps + __popc(b_eq & lt);                 // equal keys before mine, in index order
  const bool keep = sure || (eq && eq_rank < need);
  const int pos = sure_warps + __popc(b_sure & lt) + min(eq_rank, need);
  const int k1 = p.windows * p.k_w + p.k_g;
  if (keep && pos < k1) p.kept_idx[static_cast<size_t>(b) * k1 + pos] = i;
  if (p.kept_mask && live) p.kept_mask[static_cast<size_t>(b) * p.n + i] = keep ? 1 : 0;
}

// ---------------------------------------------------------------------------------------------
// Long instances: a thread-block cluster per instance.  The instance is cut into contiguous runs of whole
// window-row bands (win_h grid rows of a frame: every window lies inside one band), one run per CTA.
//   scores, local scan   on the CTA's own tokens only, as in select_kernel
//   global scan          radix select over the cluster: every CTA histograms its own candidates, a cluster barrier,
//                        then every CTA adds up the histograms of all CTAs through distributed shared memory and
//                        takes the same decision; one histogram per pass, so one cluster barrier per pass
//   union                every CTA publishes (tokens surely kept, candidates equal to the threshold); the counts
//                        of the CTAs before it give the rank of its first equal key and its first output position
// All CTAs of a cluster run the same number of cluster barriers whatever their token count; the last one keeps
// every CTA's shared memory alive until the neighbours' remote reads are done.
// dynamic shared memory: keys_g[cap] | keys_l[cap] | taken[cap] (bytes), cap = tokens per CTA
struct ClusterScratch {
  int hist[4][256];
  int sum[4][256];      // the cluster's histogram of each pass, added up locally
  int totals[2];        // tokens of this CTA kept for sure; its candidates equal to the threshold
  int all_totals[8][2];
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared-memory variable in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t peer_smem(const void* local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(static_cast<uint32_t>(__cvta_generic_to_shared(local))), "r"(rank));
  return r;
}
__device__ __forceinline__ int4 ld_peer4(uint32_t addr) {
  int4 v;
  asm volatile("ld.shared::cluster.v4.s32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ int2 ld_peer2(uint32_t addr) {
  int2 v;
  asm volatile("ld.shared::cluster.v2.s32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr) : "memory");
  return v;
}

template <typename T>
__global__ void __launch_bounds__(1024) select_cluster_kernel(SelectParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int band_tokens = p.win_h * p.grid_w;
  const int cap = p.bands_per_cta * band_tokens;
  uint32_t* keys_g = reinterpret_cast<uint32_t*>(smem_raw);
  uint32_t* keys_l = keys_g + cap;
  uint8_t* taken = reinterpret_cast<uint8_t*>(keys_l + cap);
  __shared__ SelectScratch sc;
  __shared__ __align__(16) ClusterScratch cs;
  grid_dependency_launch();

  const uint32_t csize = cluster_nctarank(), rank = cluster_ctarank();
  const int b = blockIdx.x / csize;
  const int t_lo = min(p.n, static_cast<int>(rank) * cap), t_hi = min(p.n, t_lo + cap), cnt = t_hi - t_lo;

  for (int i = threadIdx.x; i < 8 * 256; i += blockDim.x) (&cs.hist[0][0])[i] = 0;   // hist and sum
  if constexpr (std::is_void<T>::value) {
    const float* sg = p.scores_global + static_cast<size_t>(b) * p.n + t_lo;
    const float* sl = p.scores_local + static_cast<size_t>(b) * p.n + t_lo;
    for (int i = threadIdx.x; i < cnt; i += blockDim.x) {
      keys_g[i] = float_to_key(sg[i]);
      keys_l[i] = float_to_key(sl[i]);
      taken[i] = 0;
    }
  } else {
    const size_t inst = static_cast<size_t>(b) * p.heads * p.row_len + p.cls_offset + t_lo;
    const T* ag = static_cast<const T*>(p.attn_global) + inst;
    const T* al = static_cast<const T*>(p.attn_local) + inst;
    const bool same = p.attn_local == p.attn_global;
    for (int i = threadIdx.x; i < cnt; i += blockDim.x) {
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
      if (p.scores_global_out) p.scores_global_out[static_cast<size_t>(b) * p.n + t_lo + i] = g;
      if (p.scores_local_out) p.scores_local_out[static_cast<size_t>(b) * p.n + t_lo + i] = l;
      keys_g[i] = float_to_key(g);
      keys_l[i] = float_to_key(l);
      taken[i] = 0;
    }
  }
  __syncthreads();

  // ---- local scan over the windows of this CTA's bands: one warp per window
  if (p.k_w > 0 && cnt > 0) {
    const int warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int m = p.win_h * p.win_w;
    const int my_windows = (cnt / band_tokens) * p.wins_per_row;
    for (int w = warp; w < my_windows; w += nwarps) {
      const int band = w / p.wins_per_row, wc = w - band * p.wins_per_row;
      const int base = band * band_tokens + wc * p.win_w;      // relative to t_lo
      const int win_w = p.win_w, grid_w = p.grid_w;
      auto token_of = [=](int q) { return base + (q / win_w) * grid_w + (q % win_w); };
      if (m <= 64) warp_rank_mark(keys_l, m, p.k_w, token_of, taken);
      else warp_select_mark(keys_l, m, p.k_w, token_of, taken);
    }
  }
  __syncthreads();

  // ---- global scan over the cluster's candidates
  uint32_t thr = 0;
  int need = 0;
  if (p.k_g > 0) {
    uint32_t prefix = 0, mask = 0;
    int k_rem = p.k_g;
    int pass = 0;
    for (int shift = 24; shift >= 0; shift -= 8, ++pass) {
      radix_hist_add(keys_g, taken, cnt, shift, prefix, mask, cs.hist[pass]);
      cluster_barrier();                     // every CTA's histogram of this pass is complete and visible
      {   // warp c fetches the histogram of CTA c (all remote reads in flight together) and adds it to the local sum
        const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        if (warp < csize) {
          const uint32_t addr = peer_smem(&cs.hist[pass][lane * 8], warp);
          const int4 lo4 = ld_peer4(addr), hi4 = ld_peer4(addr + 16);
          int* dst = &cs.sum[pass][lane * 8];
          atomicAdd(dst + 0, lo4.x); atomicAdd(dst + 1, lo4.y); atomicAdd(dst + 2, lo4.z); atomicAdd(dst + 3, lo4.w);
          atomicAdd(dst + 4, hi4.x); atomicAdd(dst + 5, hi4.y); atomicAdd(dst + 6, hi4.z); atomicAdd(dst + 7, hi4.w);
        }
      }
      __syncthreads();
      if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        int local[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) local[j] = cs.sum[pass][lane * 8 + j];
        radix_pick(local, lane, k_rem, prefix, shift, sc);
      }
      __syncthreads();
      prefix = sc.threshold;
      k_rem = sc.need;
      mask |= 0xFFu << shift;
      __syncthreads();
    }
    thr = prefix;
    need = k_rem;
  }

  // ---- union, ascending.  Each thread owns a contiguous run of this CTA's tokens.
  const int per = (cnt + blockDim.x - 1) / blockDim.x;
  const int lo = min(cnt, static_cast<int>(threadIdx.x) * per), hi = min(cnt, lo + per);
  int sure_local = 0, eq_local = 0;
  for (int i = lo; i < hi; ++i) {
    const bool cand = !taken[i] && p.k_g > 0;
    sure_local += taken[i] || (cand && keys_g[i] > thr);
    eq_local += cand && keys_g[i] == thr;
  }
  int sure_total, eq_total;
  int sure_before = block_exclusive_scan(sure_local, sc.warp_sums, sure_total);
  int eq_before = block_exclusive_scan(eq_local, sc.warp_sums, eq_total);
  if (threadIdx.x == 0) { cs.totals[0] = sure_total; cs.totals[1] = eq_total; }
  cluster_barrier();
  if (threadIdx.x < csize) {
    const int2 t = ld_peer2(peer_smem(&cs.totals[0], threadIdx.x));
    cs.all_totals[threadIdx.x][0] = t.x; cs.all_totals[threadIdx.x][1] = t.y;
  }
  __syncthreads();
  int eq_base = 0, pos_base = 0;
  for (uint32_t c = 0; c < rank; ++c) {
    const int e = cs.all_totals[c][1];
    pos_base += cs.all_totals[c][0] + min(max(need - eq_base, 0), e);
    eq_base += e;
  }
  eq_before += eq_base;
  // position of this thread's first kept token: the sure ones before it plus the equal keys before it that made it
  int pos = pos_base + sure_before + (min(eq_before, need) - min(eq_base, need));
  const int k1 = p.windows * p.k_w + p.k_g;
  int32_t* out = p.kept_idx + static_cast<size_t>(b) * k1;
  uint8_t* mk = p.kept_mask ? p.kept_mask + static_cast<size_t>(b) * p.n + t_lo : nullptr;
  for (int i = lo; i < hi; ++i) {
    bool keep = taken[i];
    if (!keep && p.k_g > 0) {
      const uint32_t key = keys_g[i];
      if (key > thr) keep = true;
      else if (key == thr) { keep = eq_before < need; ++eq_before; }
    }
    if (keep) { if (pos < k1) out[pos] = t_lo + i; ++pos; }
    if (mk) mk[i] = keep ? 1 : 0;
  }
  cluster_barrier();   // nobody leaves while a neighbour may still read its histograms or counts
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
  auto rcp = [](long long v) { return v <= 1 ? 0u : static_cast<uint32_t>(((1ull << 32) + v - 1) / v); };
  p.rcp_frame = rcp(1ll * d->grid_h * d->grid_w); p.rcp_grid_w = rcp(d->grid_w);
  p.rcp_win_h = rcp(d->win_h); p.rcp_win_w = rcp(d->win_w);
}

// One warp per window while there are enough windows to fill the block.
static int select_threads(long long n, int windows) {
  if (n > 2048) return 1024;
  // a thread per token where that is possible, so that the scores of an instance are read in one round of loads
  if (n > 512 && n <= 1024) return static_cast<int>((n + 31) / 32 * 32);
  return windows > 8 || n > 256 ? 512 : 256;
}

// ---- the one-thread-per-token kernel
constexpr long long kSmallSelect = 1024;
static int small_threads(long long n) { return static_cast<int>((n + 31) / 32 * 32); }
// keys_l + taken flags, then (fused form) the staged attention blocks
static size_t small_smem(long long n, size_t stage_bytes, bool two) {
  return (static_cast<size_t>(n) * 5 + 15) / 16 * 16 + stage_bytes * (two ? 2 : 1);
}
// Bytes of one instance's [heads][row_len] block when it can come in as one bulk copy: every block starts on a
// 16-byte boundary, its size is a multiple of 16 bytes, and both blocks fit beside the keys.  Else 0.
static size_t stage_block_bytes(const vscan_score_select_desc* d, long long n) {
  const size_t bytes = static_cast<size_t>(d->heads) * d->row_len * dtype_bytes(d->dtype);
  if (bytes % 16 != 0 || bytes >= (1u << 20)) return 0;
  const bool two = d->attn_global != d->attn_local;
  if (small_smem(n, bytes, two) > 160 * 1024) return 0;
  return bytes;
}

// ---- the cluster kernel: instances above kClusterSelect tokens that have at least two window-row bands
constexpr long long kClusterSelect = 2048;
constexpr int kMaxSelectCluster = 8;      // the portable cluster size (16, non-portable, measured no faster)
// CTAs per instance: enough that a CTA holds about a thousand tokens, at most one per band.  0 = not applicable.
static int select_cluster_size(const vscan_select_desc* d, long long n, int max_size, int* bands_per_cta) {
  if (n <= kClusterSelect) return 0;
  const int bands = d->frames * (d->grid_h / d->win_h);
  if (bands < 2) return 0;
  int c = static_cast<int>((n + 1023) / 1024);
  if (c > max_size) c = max_size;
  if (c > bands) c = bands;
  const int per = (bands + c - 1) / c;
  c = (bands + per - 1) / per;             // no CTA without a band
  *bands_per_cta = per;
  return c >= 2 ? c : 0;
}

template <typename T>
static vscan_status launch_select_cluster(const char* name, SelectParams& p, const vscan_select_desc* d, cudaStream_t st) {
  const int instances = d->instances;
  const int csize = select_cluster_size(d, p.n, kMaxSelectCluster, &p.bands_per_cta);
  const size_t cap = static_cast<size_t>(p.bands_per_cta) * p.win_h * p.grid_w;
  const size_t smem = cap * 9 + 16;
  if (smem > kMaxDynamicSmem) return VSCAN_ERR_UNSUPPORTED;
  VSCAN_CUDA_TRY(allow_smem(select_cluster_kernel<T>, smem));
  cudaLaunchConfig_t cfg = {};
  int threads = static_cast<int>((cap + 31) / 32 * 32);
  threads = threads > 1024 ? 1024 : (threads < 256 ? 256 : threads);
  cfg.gridDim = dim3(static_cast<unsigned>(instances) * csize);
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = csize; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  VSCAN_LAUNCH(name, st, (void)cudaLaunchKernelEx(&cfg, select_cluster_kernel<T>, p));
  return VSCAN_OK;
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
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (n <= kSmallSelect) {
    VSCAN_LAUNCH("select", st, select_small_kernel<void><<<d->instances, small_threads(n), small_smem(n, 0, false), st>>>(p, 0));
    return VSCAN_OK;
  }
  int unused;
  if (select_cluster_size(d, n, kMaxSelectCluster, &unused)) return launch_select_cluster<void>("select", p, d, st);
  const size_t smem = static_cast<size_t>(n) * 9 + 16;
  VSCAN_CUDA_TRY(allow_smem(select_kernel<void>, smem));
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
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (n <= kSmallSelect) {
    const size_t stage = stage_block_bytes(d, n);
    const size_t sm = small_smem(n, stage, d->attn_global != d->attn_local);
    if (d->dtype == VSCAN_F32) {
      VSCAN_CUDA_TRY(allow_smem(select_small_kernel<float>, sm));
      VSCAN_LAUNCH("score_select", st, select_small_kernel<float><<<sd->instances, small_threads(n), sm, st>>>(p, static_cast<int>(stage)));
    } else {
      VSCAN_CUDA_TRY(allow_smem(select_small_kernel<__nv_bfloat16>, sm));
      VSCAN_LAUNCH("score_select", st, select_small_kernel<__nv_bfloat16><<<sd->instances, small_threads(n), sm, st>>>(p, static_cast<int>(stage)));
    }
    return VSCAN_OK;
  }
  int unused;
  if (select_cluster_size(sd, n, kMaxSelectCluster, &unused)) {
    if (d->dtype == VSCAN_F32) return launch_select_cluster<float>("score_select", p, sd, st);
    return launch_select_cluster<__nv_bfloat16>("score_select", p, sd, st);
  }
  const size_t smem = static_cast<size_t>(n) * 9 + 16;
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
