// The merge step (Sec. 4.1 "Token Merging", Eq. 4) in ONE pass over the features: cosine arg-max assignment and
// group sums of an instance from the same token tiles in shared memory, so that the features cross DRAM once.
//
// One cluster of C = dim / 256 CTAs per instance (persistent: cluster c takes instances c, c + clusters, ...).
// CTA r owns feature columns [256 r, 256 r + 256): it holds that slice of the kept rows, streams that slice of the
// token tiles (32 tokens at a time), and accumulates that slice of the group sums in tensor memory.  The dot products
// of a token with the kept rows need all columns, so the CTAs exchange partial sums through distributed shared memory:
//   warp 0      TMA producer: kept-row slice (row gathers, once per instance), then the token tiles
//   warp 1      MMA issuer:   S^T[slots x tokens] = kept_slice . tile_slice^T      (partial dot products, M = 64, N = 32)
//                             acc[slots x columns] += onehot_tile . tile_slice       (group sums, token tile as MN-major B)
//   warps 2-5   read S^T out of tensor memory (one kept slot per thread) and scatter it: the 8 tokens CTA r' owns go
//               into the exchange buffer of CTA r' (remote stores, then a remote arrive on its mbarrier); at the start
//               of an instance the same threads exchange the partial squared norms of the kept rows
//   warps 6-7   for the CTA's own 8 tokens of the tile: add the C partial sums in rank order, scale by 1 / |m_s|,
//               arg-max (lowest slot on ties; a kept token takes its own slot), and send the 8 assignments to all CTAs
//   warp 8      with the tile's 32 assignments: sets the one-hot tile (slots x tokens, bf16), counts the groups,
//               writes the optional assign output
//   warps 9-12  per instance: accumulator -> x 1/count -> bf16 -> merged rows (16-byte stores)
// Every wait is bounded; on expiry the CTA records VSCAN_ERR_TIMEOUT and falls through to the common exit, where the
// cluster meets once more so that no CTA leaves while a neighbour may still write into its shared memory.
#include "merge.cuh"
#include "tc_common.cuh"

namespace vscan {
namespace cl {

using namespace tc;

constexpr int kThreads = 13 * 32;
constexpr int kSlots = 64;                 // rows of both MMAs: kept slots, padded
constexpr int kTok = 32;                   // tokens per tile
constexpr int kCols = 256;                 // feature columns per CTA
constexpr int kBox = kTok * 128;           // [32 tokens x 64 columns] box: 4 KB
constexpr int kStageBytes = 4 * kBox;      // 16 KB
constexpr int kKeptBytes = 4 * kSlots * 128;   // kept slice: four [64 rows x 64 columns] chunks, 32 KB
constexpr int kOneHotBytes = kSlots * 128; // one-hot tile: 64 rows of 128 bytes (the first 64 bytes hold the 32 tokens)
constexpr int kStages = 6;
constexpr int kXDepth = 4;                 // exchange buffers in rotation
constexpr int kADepth = 8;                 // assignment buffers in rotation
constexpr int kMaxC = 4;
constexpr int kLag = 3;                    // the sums of a tile are issued this many tiles after its dot products

struct Params {
  MergeParams m;
  int c;            // CTAs per cluster
  int tiles;        // token tiles per instance
  int clusters;     // clusters in the grid
};

struct Shared {
  uint64_t full[kStages], empty[kStages];
  uint64_t kfull[2], kempty[2];
  uint64_t sfull[2], sempty[2];
  uint64_t xfull[kXDepth];
  uint64_t xfree[kXDepth];   // every CTA of the cluster has read what this CTA sent into that exchange buffer
  uint64_t afull[kADepth];
  uint64_t pfull[2], pempty[2];
  uint64_t accfull, accempty;
  uint64_t nfull[2];
  uint32_t tmem_base;
  int abort_flag;
  int assign_buf[kADepth][kTok];
  float norm_buf[2][kMaxC][kSlots];
  float inv_norm[2][kSlots];
  int kept_list[2][kSlots];
  int counts[2][kSlots];
  float inv_count[kSlots];
  float cand_val[2][kTok];
  int cand_idx[2][kTok];
  int built;          // token tiles whose one-hot tile this CTA has finished (written by the builder warp)
};

__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, int rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
// Stores into another CTA's shared memory that count their bytes on an mbarrier of that CTA: the receiver arms the
// barrier with the bytes it expects, no thread of the sender has to arrive on it.
__device__ __forceinline__ void remote_store4(uint32_t cluster_addr, uint32_t cluster_bar, float a, float b, float c, float d) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
               ::"r"(cluster_addr), "r"(__float_as_uint(a)), "r"(__float_as_uint(b)), "r"(__float_as_uint(c)), "r"(__float_as_uint(d)),
                 "r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void remote_arrive(uint32_t cluster_bar) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void remote_store1(uint32_t cluster_addr, uint32_t cluster_bar, uint32_t v) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];"
               ::"r"(cluster_addr), "r"(v), "r"(cluster_bar) : "memory");
}
// Bounded wait that also acquires what other CTAs of the cluster wrote before their arrive.
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    if (ok) return true;
    if ((i & 1023u) == 1023u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
// Bounded wait (whole warp) until the builder's tile counter has reached `target`.
__device__ __forceinline__ bool wait_built(const volatile int* built, int target, volatile int* abort_flag) {
  bool ok = true;
  for (uint32_t i = 0; *built < target; ++i) {
    if (i >= kSpinLimit) { *abort_flag = 1; ok = false; break; }
    if ((i & 255u) == 255u && *abort_flag) { ok = false; break; }
    __nanosleep(40);
  }
  return __all_sync(0xffffffffu, ok);
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}

__device__ __forceinline__ uint64_t desc_mn_sw128(uint32_t smem_addr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= 1ull << 46;
  d |= 2ull << 61;
  return d;
}
__device__ __forceinline__ uint32_t onehot_offset(int s, int j) {
  return static_cast<uint32_t>(s) * 128u + (((static_cast<uint32_t>(j) >> 3) ^ (static_cast<uint32_t>(s) & 7u)) << 4) +
         ((static_cast<uint32_t>(j) & 7u) << 1);
}

// map_x: 3-D [column][row][instance], box 64 x 32 (token tiles); map_rows: 2-D [column][all rows], box 64 x 1 (row gathers)
template <int C>
__global__ void __launch_bounds__(kThreads, 1) merge_cluster_kernel(const __grid_constant__ CUtensorMap map_x,
                                                                    const __grid_constant__ CUtensorMap map_rows, Params p) {
  extern __shared__ unsigned char smem_dyn[];
  __shared__ Shared sh;
  unsigned char* base = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  unsigned char* kept_sm = base;                                   // [2] kept-row slices
  unsigned char* stage_sm = kept_sm + 2 * kKeptBytes;              // [kStages] token tiles
  unsigned char* onehot_sm = stage_sm + kStages * kStageBytes;     // [2] one-hot tiles
  float* xbuf = reinterpret_cast<float*>(onehot_sm + 2 * kOneHotBytes);   // [kXDepth][C][64 slots][8 tokens]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const MergeParams& m = p.m;
  const int rank = static_cast<int>(cluster_rank());
  const int cluster_id = blockIdx.x / C;
  const int col0 = rank * kCols;
  constexpr int own = kTok / C;                                     // tokens of a tile this CTA finalises
  volatile int* abort_flag = &sh.abort_flag;
  constexpr int xbuf_floats = kSlots * kTok;                            // per exchange buffer: [source][slot][own tokens]

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&sh.kfull[a], 1); mbar_init(&sh.kempty[a], 1);
      mbar_init(&sh.sfull[a], 1); mbar_init(&sh.sempty[a], 4);
      mbar_init(&sh.pfull[a], 1); mbar_init(&sh.pempty[a], 1);
      mbar_init(&sh.nfull[a], 1);
    }
    // the three exchange barriers complete on bytes: the receiving warp arms them with what it expects
    for (int a = 0; a < kXDepth; ++a) { mbar_init(&sh.xfull[a], 1); mbar_init(&sh.xfree[a], C); }
    for (int a = 0; a < kADepth; ++a) mbar_init(&sh.afull[a], 1);
    mbar_init(&sh.accfull, 1); mbar_init(&sh.accempty, 4);
    sh.abort_flag = 0;
    sh.built = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)), "n"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  for (int i = threadIdx.x; i < 2 * kOneHotBytes / 16; i += kThreads) reinterpret_cast<uint4*>(onehot_sm)[i] = make_uint4(0u, 0u, 0u, 0u);
  for (int i = threadIdx.x; i < 2 * kSlots; i += kThreads) (&sh.counts[0][0])[i] = 0;
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  cluster_sync_all();          // every CTA's barriers exist before anyone arrives on them remotely
  const uint32_t tmem_s = sh.tmem_base;            // S^T: two buffers of 32 columns
  const uint32_t tmem_acc = sh.tmem_base + 64;     // group sums: 256 columns
  grid_dependency_wait();      // the kept list comes from the kernel before this one

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    bool ok = true;
    int it = 0, i = 0;
    for (int b = cluster_id; b < m.instances && ok; b += p.clusters, ++i) {
      const int kb = i & 1;
      if (i >= 2) ok = mbar_wait_warp(&sh.kempty[kb], ((i >> 1) - 1) & 1, abort_flag);
      if (!ok) break;
      {   // kept-row slice: lane l < 16 gathers rows 4l .. 4l + 3 of every 64-column chunk; padding repeats the first row
        const int32_t* kept = m.kept + static_cast<size_t>(b) * m.n_kept;
        const int row_base = b * m.row_len + m.cls_offset;
        int rows[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int s_idx = lane * 4 + j;
          rows[j] = row_base + min(max(kept[(lane < 16 && s_idx < m.n_kept) ? s_idx : 0], 0), m.n_tokens - 1);
        }
        if (lane == 0) mbar_arrive_expect_tx(&sh.kfull[kb], kKeptBytes);
        __syncwarp();
        if (lane < 16)
          for (int kc = 0; kc < 4; ++kc)
            tma_gather4(kept_sm + kb * kKeptBytes + kc * (kSlots * 128) + lane * 512, &map_rows, &sh.kfull[kb], col0 + kc * 64,
                        rows[0], rows[1], rows[2], rows[3]);
      }
      for (int t = 0; t < p.tiles && ok; ++t, ++it) {
        const int s = it % kStages, round = it / kStages;
        if (round > 0) ok = mbar_wait_warp(&sh.empty[s], (round - 1) & 1, abort_flag);
        if (!ok) break;
        if (lane == 0) {
          unsigned char* st = stage_sm + s * kStageBytes;
          mbar_arrive_expect_tx(&sh.full[s], kStageBytes);
          for (int c = 0; c < 4; ++c) tma_load_3d(st + c * kBox, &map_x, &sh.full[s], col0 + c * 64, m.cls_offset + t * kTok, b);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kTok >> 3) << 17) | (static_cast<uint32_t>(kSlots >> 4) << 24);
      const uint32_t idesc_a = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (static_cast<uint32_t>(kCols >> 3) << 17) | (static_cast<uint32_t>(kSlots >> 4) << 24);
      int n_inst = 0;
      for (int b = cluster_id; b < m.instances; b += p.clusters) ++n_inst;
      const int total = n_inst * p.tiles;
      bool ok = true;
      // g: tile whose dot products are issued now; h = g - kLag: tile whose sums are issued now
      for (int g = 0; g < total + kLag && ok && !*abort_flag; ++g) {
        if (g < total) {
          const int i = g / p.tiles, t = g - i * p.tiles, s = g % kStages, sb = g & 1;
          if (t == 0 && !mbar_wait(&sh.kfull[i & 1], (i >> 1) & 1, abort_flag)) { ok = false; break; }
          if (!mbar_wait(&sh.full[s], (g / kStages) & 1, abort_flag)) { ok = false; break; }
          if (g >= 2 && !mbar_wait(&sh.sempty[sb], ((g >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = smem_u32(kept_sm + (i & 1) * kKeptBytes), b_addr = smem_u32(stage_sm + s * kStageBytes);
          for (int kc = 0; kc < 4; ++kc) {
            const uint64_t da = smem_desc_sw128(a_addr + kc * (kSlots * 128)), db = smem_desc_sw128(b_addr + kc * kBox);
#pragma unroll
            for (int k = 0; k < 4; ++k) umma_bf16(tmem_s + sb * kTok, da + 2u * k, db + 2u * k, idesc_s, kc > 0 || k > 0);
          }
          umma_commit(&sh.sfull[sb]);
          if (t == p.tiles - 1) umma_commit(&sh.kempty[i & 1]);
        }
        const int h = g - kLag;
        if (h >= 0) {
          const int i = h / p.tiles, t = h - i * p.tiles, s = h % kStages, pb = h & 1;
          if (t == 0 && i > 0 && !mbar_wait(&sh.accempty, (i - 1) & 1, abort_flag)) { ok = false; break; }
          if (!mbar_wait(&sh.pfull[pb], (h >> 1) & 1, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint64_t da = smem_desc_sw128(smem_u32(onehot_sm + pb * kOneHotBytes));
          const uint32_t st_addr = smem_u32(stage_sm + s * kStageBytes);
#pragma unroll
          for (int k = 0; k < kTok / 16; ++k)
            umma_bf16(tmem_acc, da + 2u * k, desc_mn_sw128(st_addr + k * 2048, kBox), idesc_a, t > 0 || k > 0);
          umma_commit(&sh.empty[s]);
          umma_commit(&sh.pempty[pb]);
          if (t == p.tiles - 1) umma_commit(&sh.accfull);
        }
      }
    }
    __syncwarp();
  } else if (warp < 6) {
    // ------------------------------------------------------------ S^T readers: thread (quarter, lane < 16) owns slot 16 * quarter + lane
    const int quarter = warp & 3, slot = quarter * 16 + lane;
    const bool live = lane < 16;
    const uint32_t xbuf_local = smem_u32(xbuf), norm_local = smem_u32(&sh.norm_buf[0][0][0]);
    bool ok = true;
    int g = 0, i = 0;
    for (int b = cluster_id; b < m.instances; b += p.clusters, ++i) {
      const int kb = i & 1;
      // the first tile of the instance reuses the exchange buffer of tile g - kXDepth: once every CTA has read that
      // one, every finaliser of the cluster is at least kXDepth tiles into the previous instance and has long taken
      // the norms of the instance before it, whose buffer the norms below overwrite
      if (ok && g >= kXDepth) ok = mbar_wait_warp(&sh.xfree[g % kXDepth], ((g / kXDepth) - 1) & 1, abort_flag);
      if (ok) ok = mbar_wait_warp(&sh.kfull[kb], (i >> 1) & 1, abort_flag);
      if (ok && live) {
        // partial squared norm of the slot's kept row over this CTA's 256 columns
        float ss = 0.f;
        const unsigned char* kr = kept_sm + kb * kKeptBytes + slot * 128;
#pragma unroll
        for (int kc = 0; kc < 4; ++kc)
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            float f[8];
            Vec16<__nv_bfloat16>::unpack(*reinterpret_cast<const uint4*>(kr + kc * (kSlots * 128) + ((j ^ (slot & 7)) << 4)), f);
#pragma unroll
            for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
          }
        for (int r = 0; r < C; ++r)
          remote_store1(map_to_cta(norm_local + ((kb * kMaxC + rank) * kSlots + slot) * 4, r), map_to_cta(smem_u32(&sh.nfull[kb]), r),
                        __float_as_uint(ss));
      }
      for (int t = 0; t < p.tiles; ++t, ++g) {
        const int sb = g & 1, xb = g % kXDepth;
        // the buffer's previous contents (tile g - kXDepth) have been read by every CTA they went to
        if (ok && g >= kXDepth) ok = mbar_wait_warp(&sh.xfree[xb], ((g / kXDepth) - 1) & 1, abort_flag);
        if (ok) ok = mbar_wait_warp(&sh.sfull[sb], (g >> 1) & 1, abort_flag);
        if (!ok) continue;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        uint32_t v[32];
        tmem_ld32(tmem_s + (static_cast<uint32_t>(quarter * 32) << 16) + sb * kTok, v);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.sempty[sb]);
        if (live) {
#pragma unroll
          for (int r = 0; r < C; ++r) {
            // the tokens CTA r finalises: own * r .. own * r + own - 1 of the tile
            const uint32_t dst = map_to_cta(xbuf_local + (xb * xbuf_floats + (rank * kSlots + slot) * own) * 4, r);
            const uint32_t bar = map_to_cta(smem_u32(&sh.xfull[xb]), r);
#pragma unroll
            for (int q4 = 0; q4 < own / 4; ++q4)
              remote_store4(dst + q4 * 16, bar, __uint_as_float(v[own * r + q4 * 4]), __uint_as_float(v[own * r + q4 * 4 + 1]),
                            __uint_as_float(v[own * r + q4 * 4 + 2]), __uint_as_float(v[own * r + q4 * 4 + 3]));
          }
        }
      }
    }
  } else if (warp < 8) {
    // ------------------------------------------------------------ finalisers: thread f = (slot group f / 8, token f % 8)
    // own tokens x (64 / own) slot groups of `own` slots each
    const int f = threadIdx.x - 6 * 32, j = f % own, sg = f / own, fw = warp - 6;
    const uint32_t abuf_local = smem_u32(&sh.assign_buf[0][0]);
    bool ok = true;
    int g = 0, i = 0;
    for (int b = cluster_id; b < m.instances; b += p.clusters, ++i) {
      const int kb = i & 1;
      if (f == 0) mbar_arrive_expect_tx(&sh.nfull[kb], C * kSlots * 4);     // the partial norms of the C slices
      if (ok) ok = mbar_wait_cluster(&sh.nfull[kb], (i >> 1) & 1, abort_flag);
      {   // 1 / |m_s| from the C partial squared norms, added in rank order; the kept list for the own-slot rule
        float ss = 0.f;
        for (int r = 0; r < C; ++r) ss += sh.norm_buf[kb][r][f];
        sh.inv_norm[kb][f] = f < m.n_kept ? 1.f / fmaxf(sqrtf(ss), 1e-12f) : 0.f;
        sh.kept_list[kb][f] = f < m.n_kept ? min(max(m.kept[static_cast<size_t>(b) * m.n_kept + f], 0), m.n_tokens - 1) : 0x7fffffff;
      }
      asm volatile("bar.sync 3, 64;" ::: "memory");
      for (int t = 0; t < p.tiles; ++t, ++g) {
        const int xb = g % kXDepth, ab = g % kADepth;
        if (f == 0) mbar_arrive_expect_tx(&sh.xfull[xb], kSlots * kTok * 4);   // own tokens x 64 slots x C sources
        if (ok) ok = mbar_wait_cluster(&sh.xfull[xb], (g / kXDepth) & 1, abort_flag);
        float best = -INFINITY;
        int best_s = 0x7fffffff;
        float dot[own];
        {
          const float* xb_p = xbuf + static_cast<size_t>(xb) * xbuf_floats + sg * own * own + j;
#pragma unroll
          for (int u = 0; u < own; ++u) {
            dot[u] = 0.f;
#pragma unroll
            for (int r = 0; r < C; ++r) dot[u] += xb_p[(r * kSlots + u) * own];   // rank order: the sum does not depend on who adds
          }
        }
        // all 64 threads have their values: the sources may reuse the buffer (one arrive per source from this CTA)
        asm volatile("bar.sync 3, 64;" ::: "memory");
        if (f < C && ok) remote_arrive(map_to_cta(smem_u32(&sh.xfree[xb]), f));
        if (ok) {
#pragma unroll
          for (int u = 0; u < own; ++u) {
            const int s = sg * own + u;
            const float val = dot[u] * sh.inv_norm[kb][s];
            if (s < m.n_kept && val > best) { best = val; best_s = s; }
          }
        }
        // combine the slot groups of a token: lanes own, 2 * own, ... apart within the warp, then the two warps
#pragma unroll
        for (int o = own; o <= 16; o <<= 1) {
          const float ov = __shfl_xor_sync(0xffffffffu, best, o);
          const int os = __shfl_xor_sync(0xffffffffu, best_s, o);
          if (ov > best || (ov == best && os < best_s)) { best = ov; best_s = os; }
        }
        if (lane < own) { sh.cand_val[fw][lane] = best; sh.cand_idx[fw][lane] = best_s; }
        asm volatile("bar.sync 3, 64;" ::: "memory");
        if (f < own && ok) {
          // (with 32 own tokens each warp holds one slot group of every token; else warp 1 holds the higher groups)
          float v0 = sh.cand_val[0][f], v1 = sh.cand_val[1][f];
          int s0 = sh.cand_idx[0][f], s1 = sh.cand_idx[1][f];
          int a = (v1 > v0 || (v1 == v0 && s1 < s0)) ? s1 : s0;
          const int tok = t * kTok + rank * own + f;
          if (tok >= m.n_tokens) a = -1;
          else {
            if (a == 0x7fffffff) a = 0;
            // a kept token belongs to its own slot: binary search of the ascending kept list
            int lo = 0, hi = m.n_kept - 1;
            while (lo < hi) { const int mid = (lo + hi) >> 1; if (sh.kept_list[kb][mid] < tok) lo = mid + 1; else hi = mid; }
            if (sh.kept_list[kb][lo] == tok) a = lo;
          }
          for (int r = 0; r < C; ++r)
            remote_store1(map_to_cta(abuf_local + (ab * kTok + rank * own + f) * 4, r), map_to_cta(smem_u32(&sh.afull[ab]), r),
                          static_cast<uint32_t>(a));
        }
        asm volatile("bar.sync 3, 64;" ::: "memory");   // the candidate buffers are free for the next tile
      }
    }
  } else if (warp == 8) {
    // ------------------------------------------------------------ one-hot builder: lane = token of the tile
    int prev0 = -1, prev1 = -1;
    bool ok = true;
    int g = 0, i = 0;
    for (int b = cluster_id; b < m.instances; b += p.clusters, ++i) {
      for (int t = 0; t < p.tiles; ++t, ++g) {
        const int ab = g % kADepth, pb = g & 1;
        if (lane == 0) mbar_arrive_expect_tx(&sh.afull[ab], kTok * 4);   // the tile's 32 assignments
        if (ok) ok = mbar_wait_cluster(&sh.afull[ab], (g / kADepth) & 1, abort_flag);
        if (ok && g >= 2) ok = mbar_wait_warp(&sh.pempty[pb], ((g >> 1) - 1) & 1, abort_flag);
        if (ok) {
          const int a = min(sh.assign_buf[ab][lane], m.n_kept - 1);
          unsigned char* tile = onehot_sm + pb * kOneHotBytes;
          const int prev = pb ? prev1 : prev0;
          if (prev >= 0) *reinterpret_cast<uint16_t*>(tile + onehot_offset(prev, lane)) = 0u;
          if (a >= 0) {
            *reinterpret_cast<uint16_t*>(tile + onehot_offset(a, lane)) = 0x3F80u;   // bf16 1.0
            atomicAdd(&sh.counts[i & 1][a], 1);
            if (rank == 0 && m.assign) m.assign[static_cast<size_t>(b) * m.n_tokens + t * kTok + lane] = a;
          }
          if (pb) prev1 = a; else prev0 = a;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0 && ok) {
          mbar_arrive(&sh.pfull[pb]);
          *reinterpret_cast<volatile int*>(&sh.built) = g + 1;
        }
      }
    }
  } else {
    // ------------------------------------------------------------ read-back (warps 9-12): thread (quarter, lane < 16) owns slot 16 * quarter + lane
    const int quarter = warp & 3, slot = quarter * 16 + lane, tid9 = threadIdx.x - 9 * 32;
    bool ok = true;
    int i = 0;
    for (int b = cluster_id; b < m.instances; b += p.clusters, ++i) {
      if (ok) ok = mbar_wait_warp(&sh.accfull, i & 1, abort_flag);
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      for (int s = tid9; s < kSlots; s += 128) {
        const int c = sh.counts[i & 1][s];
        sh.inv_count[s] = 1.f / static_cast<float>(max(c, 1));
        if (rank == 0 && m.counts && s < m.n_kept && ok) m.counts[static_cast<size_t>(b) * m.n_kept + s] = c;
        sh.counts[i & 1][s] = 0;
      }
      asm volatile("bar.sync 2, 128;" ::: "memory");
      if (ok) {
        const bool mine = lane < 16 && slot < m.n_kept;
        const float inv = mine ? sh.inv_count[slot] : 0.f;
        uint4* out = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(m.merged) +
                                              (static_cast<size_t>(b) * m.n_kept + (mine ? slot : 0)) * m.dim + col0);
        const uint32_t taddr = tmem_acc + (static_cast<uint32_t>(quarter * 32) << 16);
        for (int c0 = 0; c0 < kCols; c0 += 32) {
          uint32_t v[32];
          tmem_ld32(taddr + c0, v);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          if (mine) {
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
              float fl[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) fl[e] = __uint_as_float(v[q4 * 8 + e]) * inv;
              st_16(out + c0 / 8 + q4, Vec16<__nv_bfloat16>::pack(fl));
            }
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      asm volatile("bar.sync 2, 128;" ::: "memory");    // inv_count is read by all four warps before the next instance overwrites it
      if (lane == 0 && ok) mbar_arrive(&sh.accempty);
    }
  }

  // ------------------------------------------------------------ common exit
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (sh.abort_flag) {
    if (threadIdx.x == 0) atomicExch(m.status, static_cast<uint32_t>(VSCAN_ERR_TIMEOUT));
    for (int i = 0; i < 64; ++i) __nanosleep(2000);   // copies still in flight land before the memory is released
    __syncthreads();
  }
  cluster_sync_all();          // nobody leaves while a neighbour may still store into its shared memory
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(sh.tmem_base), "n"(512) : "memory");
  }
}

static size_t smem_bytes() {
  return 1024 + 2 * kKeptBytes + kStages * kStageBytes + 2 * kOneHotBytes + static_cast<size_t>(kXDepth) * kSlots * kTok * sizeof(float);
}

static bool plan(const MergeParams& m, Params& p) {
  if (m.metric != m.x || m.metric_dim != m.dim) return false;          // one pass: similarity and sums on the same tensor
  if (m.dim % kCols != 0 || (m.dim / kCols != 1 && m.dim / kCols != 2 && m.dim / kCols != 4)) return false;
  if (m.n_kept < 1 || m.n_kept > kSlots) return false;
  if (m.row_len != m.cls_offset + m.n_tokens) return false;            // rows past the last token must be the copy's zero fill
  if ((reinterpret_cast<uintptr_t>(m.x) & 15u) != 0 || (reinterpret_cast<uintptr_t>(m.merged) & 15u) != 0) return false;
  p.m = m;
  p.c = m.dim / kCols;
  p.tiles = (m.n_tokens + kTok - 1) / kTok;
  if (p.tiles < kXDepth) return false;                                  // the buffer rotation argument needs a few tiles per instance
  if (1ll * m.instances * p.tiles > 0x3fffffffLL) return false;
  return true;
}

}  // namespace cl

bool merge_cluster_supported(int dtype, const MergeParams& m) {
  cl::Params p;
  return dtype == VSCAN_BF16 && cl::plan(m, p) && tc::encode_fn() != nullptr;
}

vscan_status launch_merge_cluster(const MergeParams& m, cudaStream_t stream) {
  using namespace cl;
  Params p;
  if (!plan(m, p)) return VSCAN_ERR_UNSUPPORTED;
  tc::EncodeTiledFn encode = tc::encode_fn();
  if (!encode) return VSCAN_ERR_UNSUPPORTED;
  CUtensorMap map_x, map_rows;
  const cuuint32_t elem[3] = {1, 1, 1};
  {
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(m.dim), static_cast<cuuint64_t>(m.row_len), static_cast<cuuint64_t>(m.instances)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(m.dim) * 2, static_cast<cuuint64_t>(m.row_len) * m.dim * 2};
    const cuuint32_t box[3] = {64, kTok, 1};
    if (encode(&map_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(m.x), dims, strides, box, elem,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return VSCAN_ERR_UNSUPPORTED;
    const cuuint64_t dims_r[2] = {static_cast<cuuint64_t>(m.dim), static_cast<cuuint64_t>(m.row_len) * static_cast<cuuint64_t>(m.instances)};
    const cuuint64_t strides_r[1] = {static_cast<cuuint64_t>(m.dim) * 2};
    const cuuint32_t box_r[2] = {64, 1};
    if (encode(&map_rows, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(m.x), dims_r, strides_r, box_r, elem,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return VSCAN_ERR_UNSUPPORTED;
  }
  const size_t smem = smem_bytes();
  void (*kernel)(CUtensorMap, CUtensorMap, Params) =
      p.c == 4 ? merge_cluster_kernel<4> : (p.c == 2 ? merge_cluster_kernel<2> : merge_cluster_kernel<1>);
  VSCAN_CUDA_TRY(allow_smem(kernel, smem));
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = p.c; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // as many clusters as can be resident at once (the kernel is persistent), at most one per instance
  cfg.gridDim = dim3(p.c);
  int max_clusters = 0;
  VSCAN_CUDA_TRY(cudaOccupancyMaxActiveClusters(&max_clusters, kernel, &cfg));
  if (max_clusters < 1) return VSCAN_ERR_UNSUPPORTED;
  p.clusters = m.instances < max_clusters ? m.instances : max_clusters;
  cfg.gridDim = dim3(static_cast<unsigned>(p.clusters) * p.c);
  VSCAN_CUDA_TRY(cudaMemsetAsync(m.status, 0, sizeof(uint32_t), stream));
  VSCAN_LAUNCH("merge_cluster", stream, (void)cudaLaunchKernelEx(&cfg, kernel, map_x, map_rows, p));
  return VSCAN_OK;
}

}  // namespace vscan
