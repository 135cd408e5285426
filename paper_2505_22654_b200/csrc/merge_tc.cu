// Tensor-core path of the merge assignment (Sec. 4.1 "Token Merging"): for a tile of 128 tokens the
// dot products with all kept tokens are one tcgen05 MMA chain, D[128 x Nk] (fp32, tensor memory) =
// A[128 tokens x dim] * B[Nk kept x dim]^T with bf16 operands in shared memory.
//   warp 0      TMA producer: the token tile (3-D tensor map over [instance][row][dim], 128B swizzle) and
//               the kept rows, which are not contiguous, four rows per TMA gather
//   warp 1      allocates tensor memory, issues the MMAs (one elected lane), commits to mbarriers
//   warps 2-5   take the squared norms of the kept rows from the B stages while the MMAs run, then
//               read the accumulator back (tcgen05.ld, one token row per thread), scale by 1/|m_s|
//               and keep the running arg-max (lowest slot on ties); with more than 256 kept tokens
//               two accumulators alternate so this overlaps the next round of MMAs
// The similarity matrix never leaves the SM.  Every mbarrier wait is bounded: on expiry the CTA
// records VSCAN_ERR_TIMEOUT in the status word, lets copies in flight land, frees its tensor memory
// and returns.
#include <cstdlib>

#include "merge.cuh"
#include "tc_common.cuh"

namespace vscan {

namespace tc {

constexpr int kThreads = 192;

struct Params {
  MergeParams m;
  int b_packed;     // kept rows come from the packed copy (one tile load per stage) instead of row gathers
  int n_pad;        // kept columns per n-chunk, multiple of 16, <= 256
  int n_chunks;     // ceil(n_kept / n_pad)
  int k_chunks;     // ceil(metric_dim / 64)
  int stages;
  int tmem_cols;    // power of two >= max(32, n_pad)
  int a_stage_bytes, b_stage_bytes;
};

struct Shared {
  uint64_t full[kMaxStages];    // token tile and kept rows of the stage have landed (transaction bytes)
  uint64_t empty[kMaxStages];   // MMAs that read the stage have completed
  uint64_t tmem_full[2];        // accumulator (ping or pong) of an n-chunk complete
  uint64_t tmem_empty[2];       // epilogue has read that accumulator
  uint32_t tmem_base;
  int abort_flag;
  int best_slot[kTileM];
};

// Copies the kept rows of every instance into a contiguous [instance][slot][dim] buffer (slots past
// n_kept are zero).  One warp per slot.
__global__ void __launch_bounds__(256) pack_kept_kernel(MergeParams m, int rows_packed) {
  const int b = blockIdx.y, s = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (s >= rows_packed) return;
  uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(m.kept_packed) +
                                        (static_cast<size_t>(b) * rows_packed + s) * m.metric_dim);
  const int vecs = m.metric_dim / 8;
  if (s < m.n_kept) {
    const int t = min(max(m.kept[static_cast<size_t>(b) * m.n_kept + s], 0), m.n_tokens - 1);
    const uint4* src = reinterpret_cast<const uint4*>(
        static_cast<const __nv_bfloat16*>(m.metric) + (static_cast<size_t>(b) * m.row_len + m.cls_offset + t) * m.metric_dim);
    for (int v = lane; v < vecs; v += 32) st_16(dst + v, ld_nc_16(src + v));
  } else {
    for (int v = lane; v < vecs; v += 32) st_16(dst + v, make_uint4(0u, 0u, 0u, 0u));
  }
}

// The whole life of one assignment CTA: tile of 128 tokens starting at token t0 of instance b.
// smem_dyn: up to 1023 bytes of alignment slack | stages x [A tile 128x64 bf16 | B tile n_pad x 64 bf16] |
// inv_norm[1 or 2][n_pad] floats (kept in dynamic memory so that three CTAs fit in one SM's 228 KB).
// `done` (optional): counter of the instance, incremented once the assignments of the tile are visible
// device-wide (not incremented when a wait of this CTA ran out).
__device__ __forceinline__ void assign_tile(const CUtensorMap* map_a_ptr, const CUtensorMap* map_b_ptr, const Params& p,
                                            Shared& sh, unsigned char* smem_dyn, int b, int t0, int* done) {
  const CUtensorMap& map_a = *map_a_ptr;
  const CUtensorMap& map_b = *map_b_ptr;
  // the swizzle pattern is a function of the shared-memory address: stage bases sit on 1024 bytes
  unsigned char* tiles = smem_dyn + ((1024u - (static_cast<uint32_t>(__cvta_generic_to_shared(smem_dyn)) & 1023u)) & 1023u);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const MergeParams& m = p.m;
  volatile int* abort_flag = &sh.abort_flag;
  const int stage_bytes = p.a_stage_bytes + p.b_stage_bytes;
  float* inv_norm = reinterpret_cast<float*>(tiles + p.stages * stage_bytes);   // [accumulator][n_pad]
  const int32_t* kept = m.kept + static_cast<size_t>(b) * m.n_kept;

  if (threadIdx.x == 0) {
    // a stage is free again once the MMAs that read it have completed and the four epilogue warps
    // have taken the squared norms of its kept-row slice
    for (int s = 0; s < p.stages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 5); }
    for (int a = 0; a < 2; ++a) { mbar_init(&sh.tmem_full[a], 1); mbar_init(&sh.tmem_empty[a], 4); }
    sh.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)), "r"(p.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (m.clear_status && b == 0 && t0 == 0 && threadIdx.x == 0) *m.status = 0u;   // long before any wait can expire
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = sh.tmem_base;
  grid_dependency_launch();
  grid_dependency_wait();   // the kept list comes from the kernel before this one

  if (warp == 0) {
    // ------------------------------------------------------------ producer: TMA tile + TMA row gathers
    // Lane l issues the gathers of row groups l, l+32, ... (four kept rows each); it keeps their row
    // coordinates in registers for the whole n-chunk.  Padding rows repeat the first kept row (their
    // columns are masked in the epilogue).
    const int groups = p.n_pad / 4;                 // gathers per stage
    const int row_base = b * m.row_len + m.cls_offset;
    const int first = row_base + min(max(kept[0], 0), m.n_tokens - 1);
    int it = 0;
    bool ok = true;
    for (int nc = 0; nc < p.n_chunks; ++nc) {
      int rows[2][4];
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int g = lane + 32 * i;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int s_idx = nc * p.n_pad + g * 4 + j;
          rows[i][j] = (g < groups && s_idx < m.n_kept) ? row_base + min(max(kept[s_idx], 0), m.n_tokens - 1) : first;
        }
      }
      for (int kc = 0; kc < p.k_chunks; ++kc, ++it) {
        const int s = it % p.stages, round = it / p.stages;
        if (ok && round > 0) ok = mbar_wait_warp(&sh.empty[s], (round - 1) & 1, abort_flag);
        if (!ok) continue;
        unsigned char* at = tiles + s * stage_bytes;
        if (lane == 0) {
          mbar_arrive_expect_tx(&sh.full[s], p.a_stage_bytes + p.n_pad * 128);
          tma_load_3d(at, &map_a, &sh.full[s], kc * kChunkK, m.cls_offset + t0, b);
          if (p.b_packed) tma_load_3d(at + p.a_stage_bytes, &map_b, &sh.full[s], kc * kChunkK, nc * p.n_pad, b);
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const int g = lane + 32 * i;
          if (g < groups && !p.b_packed)
            tma_gather4(at + p.a_stage_bytes + g * 512, &map_b, &sh.full[s], kc * kChunkK, rows[i][0], rows[i][1],
                        rows[i][2], rows[i][3]);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = instr_desc_bf16(p.n_pad);
      int it = 0;
      for (int nc = 0; nc < p.n_chunks && !*abort_flag; ++nc) {
        const int acc = nc & 1, use = nc >> 1;
        if (use > 0) {
          if (!mbar_wait(&sh.tmem_empty[acc], (use - 1) & 1, abort_flag)) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        }
        const uint32_t d_addr = tmem_acc + acc * p.n_pad;
        bool ok = true;
        for (int kc = 0; kc < p.k_chunks; ++kc, ++it) {
          const int s = it % p.stages, round = it / p.stages;
          if (!mbar_wait(&sh.full[s], round & 1, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = smem_u32(tiles + s * stage_bytes), b_addr = a_addr + p.a_stage_bytes;
          const uint64_t da = smem_desc_sw128(a_addr), db = smem_desc_sw128(b_addr);
#pragma unroll
          for (int k = 0; k < kChunkK / 16; ++k)   // 16 bf16 = 32 bytes per MMA along K: +2 in 16-byte units
            umma_bf16(d_addr, da + 2u * k, db + 2u * k, idesc, kc > 0 || k > 0);
          umma_commit(&sh.empty[s]);
        }
        if (!ok) break;
        umma_commit(&sh.tmem_full[acc]);
      }
    }
    __syncwarp();   // the other lanes wait here, so the warp reaches the barrier below together
  } else {
    // ------------------------------------------------------------ epilogue: accumulator -> arg-max
    const int ptid = (warp - 2) * 32 + lane;  // 0..127
    const int quarter = warp & 3;             // tensor-memory lanes this warp may read
    const int row = quarter * 32 + lane;      // token row of this thread within the tile
    float best_val = -INFINITY;
    int best_idx = 0;
    int it = 0;
    bool ok = true;
    // Once `ok` drops the loop keeps running with its work skipped, so that the four warps execute
    // the same sequence of named barriers and warp-wide instructions whatever happens.
    for (int nc = 0; nc < p.n_chunks; ++nc) {
      const int n0 = nc * p.n_pad, acc = nc & 1, use = nc >> 1;
      // |m_s|^2 of the kept rows of this n-chunk, accumulated from the B stages as they pass through
      // shared memory (thread ptid owns rows ptid and ptid + 128)
      float ss[2] = {0.f, 0.f};
      for (int kc = 0; kc < p.k_chunks; ++kc, ++it) {
        const int s = it % p.stages, round = it / p.stages;
        if (ok) ok = mbar_wait_warp(&sh.full[s], round & 1, abort_flag);
        if (!ok) continue;
        const unsigned char* bt = tiles + s * stage_bytes + p.a_stage_bytes;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int r = ptid + 128 * u;
          if (r < p.n_pad) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              float f[8];
              Vec16<__nv_bfloat16>::unpack(*reinterpret_cast<const uint4*>(bt + r * 128 + ((j ^ (r & 7)) << 4)), f);
#pragma unroll
              for (int e = 0; e < 8; ++e) ss[u] = fmaf(f[e], f[e], ss[u]);
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.empty[s]);
      }
      // the buffer was last read two chunks ago, before that chunk's arrive on tmem_empty
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int r = ptid + 128 * u;
        if (r < p.n_pad) inv_norm[acc * p.n_pad + r] = (n0 + r < m.n_kept) ? 1.f / fmaxf(sqrtf(ss[u]), 1e-12f) : 0.f;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (ok) ok = mbar_wait_warp(&sh.tmem_full[acc], use & 1, abort_flag);
      if (!ok) continue;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t taddr = tmem_acc + (static_cast<uint32_t>(quarter * 32) << 16) + acc * p.n_pad;
      for (int c0 = 0; c0 < p.n_pad; c0 += 32) {
        uint32_t v[32];
        if (p.n_pad - c0 >= 32) tmem_ld32(taddr + c0, v);
        else {
          tmem_ld16(taddr + c0, v);
#pragma unroll
          for (int j = 16; j < 32; ++j) v[j] = 0u;
        }
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const int s_idx = n0 + c0 + j;
          if (c0 + j < p.n_pad && s_idx < m.n_kept) {
            const float val = __uint_as_float(v[j]) * inv_norm[acc * p.n_pad + c0 + j];
            if (val > best_val) { best_val = val; best_idx = s_idx; }
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.tmem_empty[acc]);
    }
    sh.best_slot[row] = best_idx;
    asm volatile("bar.sync 1, 128;" ::: "memory");
    // a kept token belongs to its own slot
    for (int s_idx = ptid; s_idx < m.n_kept; s_idx += 128) {
      const int t = min(max(kept[s_idx], 0), m.n_tokens - 1);
      if (t >= t0 && t < t0 + kTileM) sh.best_slot[t - t0] = s_idx;
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (ok && t0 + ptid < m.n_tokens) m.assign[static_cast<size_t>(b) * m.n_tokens + t0 + ptid] = sh.best_slot[ptid];
    if (done) {   // publish: the 128 stores above first, then one increment
      __threadfence();
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (ptid == 0 && ok && !*abort_flag) atomicAdd(done, 1);
    }
  }

  // ------------------------------------------------------------ teardown
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (sh.abort_flag) {
    if (threadIdx.x == 0) atomicExch(m.status, static_cast<uint32_t>(VSCAN_ERR_TIMEOUT));
    // give copies that are still in flight time to land before the shared memory is released
    for (int i = 0; i < 64; ++i) __nanosleep(2000);
    __syncthreads();
  }
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(p.tmem_cols) : "memory");
  }
}

__global__ void __launch_bounds__(kThreads) assign_tensor_kernel(const __grid_constant__ CUtensorMap map_a,
                                                                 const __grid_constant__ CUtensorMap map_b, Params p) {
  extern __shared__ unsigned char smem_dyn[];
  __shared__ Shared sh;
  assign_tile(&map_a, &map_b, p, sh, smem_dyn, blockIdx.y, blockIdx.x * kTileM, nullptr);
}

// Assignment and group means in ONE launch, so that the second pass over the features (the sums of
// Eq. 4) reads them from L2 while they are still there.  The CTA that has assigned tile t of instance i
// goes on to sum groups of instance i - lag: the column slices t, t + tiles, ... of it.  The hardware
// hands out blocks in index order, so the tiles of instance i - lag were started lag * tiles blocks
// earlier and have normally finished by then; the CTA still checks the instance's counter of finished
// tiles and spins (bounded; on expiry VSCAN_ERR_TIMEOUT) until it is complete.  lag * tiles extra
// CTAs at the end of the grid take the sums of the last `lag` instances.  Nothing waits on a block
// with a higher index, and no CTA exists only to wait.
struct Interleave {
  int* done;        // [instances] finished assignment tiles, zero at launch
  int tiles;        // assignment CTAs per instance
  int slices;       // slices of kSliceCols feature columns
  int x_boxes;      // tile loads (kBoxRows rows x kSliceCols columns) that cover the tokens of an instance
  int lag;          // instances between an assignment and its sums, 1 <= lag <= instances
};
constexpr uint32_t kDoneSpinLimit = 1u << 22;    // polls of ~100 ns
constexpr int kSliceCols = 64;                   // feature columns of one slice (128 bytes per row)
constexpr int kBoxRows = 192;                    // token rows per tile load of a slice
constexpr int kMaxBoxes = 4;
constexpr int kMaxMeanKept = kThreads;           // kept slots the shared tables hold (one thread per slot in the sort)
constexpr int kWarps = kThreads / 32;

struct MeanShared {
  uint64_t full;                       // the current column slice has landed
  uint32_t tmem_base;
  int ready;                           // assignments of the instance complete (0: the wait ran out)
  int warp_sums[33];
  uint16_t begin[kMaxMeanKept + 2];    // first list position of each slot; begin[n_kept] = listed tokens
};

// Sums of the slices `first`, `first + il.tiles`, ... of instance b (a slice = kSliceCols feature columns).
//   1. wait for the instance's assignments; 2. a stable counting sort of its tokens by slot (every slot's
//   members in ascending token order): a bit mask per (slot, 32-token chunk) filled with shared-memory
//   atomics, prefix sums over chunks and slots, then every mask word writes out its tokens; 3. per slice:
//   the 128-byte column slice of all tokens comes in by a few tile loads, then groups of 8 lanes (16
//   bytes each) walk the member lists, one slot per group at a time, adding in list order in fp32, one
//   rounding.  Same order of additions as group_mean_body, hence the same bits.
// smem_dyn: the slice (n_tokens rounded up to boxes x 128 bytes; the sort's scratch before the first
// slice is fetched) followed by the member list (n_tokens x 2 bytes).
__device__ __forceinline__ void mean_share(const CUtensorMap* map_x, const MergeParams& m, const Interleave& il,
                                           MeanShared& ms, unsigned char* smem_dyn, int b, int first) {
  constexpr int kRowBytes = kSliceCols * 2, kLanesPerRow = kRowBytes / 16;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned char* tiles = smem_dyn + ((128u - (smem_u32(smem_dyn) & 127u)) & 127u);
  const uint32_t slice_bytes = static_cast<uint32_t>(il.x_boxes) * kBoxRows * kRowBytes;
  uint16_t* list = reinterpret_cast<uint16_t*>(tiles + slice_bytes);
  const int chunks = (m.n_tokens + 31) / 32;
  uint32_t* bits = reinterpret_cast<uint32_t*>(tiles);                       // [n_kept][chunks] (scratch)
  uint16_t* offs = reinterpret_cast<uint16_t*>(bits + m.n_kept * chunks);    // [n_kept][chunks] (scratch)
  if (threadIdx.x == 0) {
    mbar_init(&ms.full, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const volatile int* flag = il.done + b;
    uint32_t spins = 0;
    while (*flag < il.tiles && spins < kDoneSpinLimit) { __nanosleep(100); ++spins; }
    ms.ready = *flag >= il.tiles;
    if (!ms.ready) atomicExch(m.status, static_cast<uint32_t>(VSCAN_ERR_TIMEOUT));
    __threadfence();
  }
  for (int i = threadIdx.x; i < m.n_kept * chunks; i += kThreads) bits[i] = 0u;
  __syncthreads();
  if (!ms.ready) return;

  // ---- sort
  const int32_t* ag = m.assign + static_cast<size_t>(b) * m.n_tokens;
  for (int c = warp; c < chunks; c += kWarps) {
    const int t = c * 32 + lane;
    if (t < m.n_tokens) {
      const int v = __ldcg(ag + t);
      if (v >= 0 && v < m.n_kept) atomicOr(&bits[v * chunks + c], 1u << lane);
    }
  }
  __syncthreads();
  int total = 0;
  if (threadIdx.x < m.n_kept) {
    for (int c = 0; c < chunks; ++c) {
      offs[threadIdx.x * chunks + c] = static_cast<uint16_t>(total);
      total += __popc(bits[threadIdx.x * chunks + c]);
    }
  }
  int listed;
  const int start = block_exclusive_scan(total, ms.warp_sums, listed);   // contains the barriers
  if (threadIdx.x < m.n_kept) ms.begin[threadIdx.x] = static_cast<uint16_t>(start);
  if (threadIdx.x == 0) ms.begin[m.n_kept] = static_cast<uint16_t>(listed);
  __syncthreads();
  for (int i = threadIdx.x; i < m.n_kept * chunks; i += kThreads) {
    const int sl = i / chunks, c = i - sl * chunks;
    uint32_t word = bits[i];
    int pos = ms.begin[sl] + offs[i];
    while (word) {
      const int bit = __ffs(word) - 1;
      word &= word - 1;
      list[pos++] = static_cast<uint16_t>(c * 32 + bit);
    }
  }
  __syncthreads();   // the list is complete and the scratch is free

  // ---- slices
  volatile int local_abort = 0;
  const int group = threadIdx.x / kLanesPerRow, piece = threadIdx.x % kLanesPerRow;
  int round = 0;
  for (int slice = first; slice < il.slices; slice += il.tiles, ++round) {
    if (threadIdx.x == 0) {
      mbar_arrive_expect_tx(&ms.full, slice_bytes);
      for (int i = 0; i < il.x_boxes; ++i)
        tma_load_3d(tiles + static_cast<size_t>(i) * kBoxRows * kRowBytes, map_x, &ms.full, slice * kSliceCols,
                    m.cls_offset + i * kBoxRows, b);
    }
    // every thread waits itself: the slice was written by the copy engine
    const bool landed = mbar_wait(&ms.full, round & 1, &local_abort);
    if (!landed) {   // (all threads of the CTA wait on the same phase: they give up together)
      if (threadIdx.x == 0) atomicExch(m.status, static_cast<uint32_t>(VSCAN_ERR_TIMEOUT));
      for (int i = 0; i < 64; ++i) __nanosleep(2000);   // let the copies land before the memory is released
      return;
    }
    const unsigned char* rows = tiles + piece * 16;
    const int col = slice * kSliceCols + piece * 8;
    for (int sl = group; sl < m.n_kept; sl += kThreads / kLanesPerRow) {
      const int k0 = ms.begin[sl], k1 = ms.begin[sl + 1];
      float acc[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] = 0.f;
      for (int k = k0; k < k1; k += 4) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (k + u < k1) v[u] = *reinterpret_cast<const uint4*>(rows + static_cast<uint32_t>(list[k + u]) * kRowBytes);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (k + u < k1) {
            float f[8];
            Vec16<__nv_bfloat16>::unpack(v[u], f);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] += f[e];
          }
        }
      }
      const int count = k1 - k0;
      const float inv = 1.f / static_cast<float>(max(count, 1));
      if (col < m.dim) {
        float f[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) f[e] = acc[e] * inv;
        st_16(static_cast<__nv_bfloat16*>(m.merged) + (static_cast<size_t>(b) * m.n_kept + sl) * m.dim + col,
              Vec16<__nv_bfloat16>::pack(f));
      }
      if (slice == 0 && piece == 0 && m.counts) m.counts[static_cast<size_t>(b) * m.n_kept + sl] = count;
    }
    __syncthreads();   // every thread has read the slice: the next one may overwrite it
  }
}

template <int kMinCtas>
__global__ void __launch_bounds__(kThreads, kMinCtas)
merge_interleaved_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                         const __grid_constant__ CUtensorMap map_x, Params p, Interleave il) {
  extern __shared__ unsigned char smem_dyn[];
  __shared__ Shared sh;
  __shared__ MeanShared ms;
  const int n_assign = p.m.instances * il.tiles, bid = blockIdx.x;
  int mean_b, part;
  if (bid < n_assign) {
    const int b = bid / il.tiles;
    part = bid - b * il.tiles;
    assign_tile(&map_a, &map_b, p, sh, smem_dyn, b, part * kTileM, il.done + b);
    mean_b = b - il.lag;
    if (mean_b < 0) return;
    __syncthreads();   // the tile's teardown is complete: shared memory changes hands
  } else {
    const int r = bid - n_assign;
    mean_b = p.m.instances - il.lag + r / il.tiles;
    part = r - (r / il.tiles) * il.tiles;
    // A CTA of a kernel that uses tensor memory keeps the right to allocate it until it gives that right
    // up, and the SM starts no further CTA of the kernel beside it meanwhile: take the smallest
    // allocation and relinquish at once, as the assignment CTAs do.
    if (threadIdx.x < 32) {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ms.tmem_base)), "r"(32) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    grid_dependency_launch();
    grid_dependency_wait();   // the features may come from the kernel before this one
  }
  mean_share(&map_x, p.m, il, ms, smem_dyn, mean_b, part);
  if (bid >= n_assign) {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x < 32) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(ms.tmem_base), "r"(32) : "memory");
    }
  }
}

// ---------------------------------------------------------------------------- host side
static bool plan(const MergeParams& m, Params& p) {
  p.m = m;
  p.b_packed = (m.n_kept > kMaxN && m.kept_packed != nullptr) ? 1 : 0;
  const int n16 = (m.n_kept + 15) / 16 * 16;
  p.n_pad = n16 <= kMaxN ? n16 : kMaxN;
  p.n_chunks = (m.n_kept + p.n_pad - 1) / p.n_pad;
  p.k_chunks = (m.metric_dim + kChunkK - 1) / kChunkK;
  p.tmem_cols = 32;   // one accumulator, or two (ping-pong) when the kept set needs several rounds
  while (p.tmem_cols < p.n_pad * (p.n_chunks > 1 ? 2 : 1)) p.tmem_cols *= 2;
  p.a_stage_bytes = kTileM * kChunkK * 2;
  p.b_stage_bytes = ((p.n_pad * kChunkK * 2) + 1023) / 1024 * 1024;
  const int stage = p.a_stage_bytes + p.b_stage_bytes;
  // three CTAs per SM with three stages each when that fits (their fixed start-up and epilogue
  // costs overlap), else two with up to four, else one CTA with as many stages as fit
  int stages;
  if ((73 * 1024) / stage >= 3) stages = 3;
  else if ((110 * 1024) / stage >= 3) stages = (110 * 1024) / stage > 4 ? 4 : (110 * 1024) / stage;
  else stages = (215 * 1024) / stage;
  if (stages > kMaxStages) stages = kMaxStages;
  p.stages = stages;
  return stages >= 2;
}

// dynamic shared memory of an assignment CTA: alignment slack, the stage ring, the inverse norms
static size_t smem_bytes(const Params& p) {
  return 1024 + static_cast<size_t>(p.stages) * (p.a_stage_bytes + p.b_stage_bytes) +
         static_cast<size_t>(p.n_chunks > 1 ? 2 : 1) * p.n_pad * sizeof(float);
}

}  // namespace tc

bool assign_tensor_supported(int dtype, const MergeParams& m) {
  if (dtype != VSCAN_BF16 || m.metric_dim % 8 != 0 || m.n_kept < 1) return false;
  if ((reinterpret_cast<uintptr_t>(m.metric) & 15u) != 0) return false;
  tc::Params p;
  return tc::plan(m, p) && tc::encode_fn() != nullptr;
}

// Tensor maps of a launch: the token tiles (3-D [instance][row][dim]) and the kept rows (the same memory
// as a 2-D [all rows][dim] tensor for row gathers, or the packed copy for large kept sets).
static vscan_status encode_maps(const MergeParams& m, const tc::Params& p, CUtensorMap& map, CUtensorMap& map_b) {
  tc::EncodeTiledFn encode = tc::encode_fn();
  if (!encode) return VSCAN_ERR_UNSUPPORTED;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(m.metric_dim), static_cast<cuuint64_t>(m.row_len),
                              static_cast<cuuint64_t>(m.instances)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(m.metric_dim) * 2,
                                 static_cast<cuuint64_t>(m.row_len) * m.metric_dim * 2};
  const cuuint32_t box[3] = {tc::kChunkK, tc::kTileM, 1};
  const cuuint32_t elem[3] = {1, 1, 1};
  CUresult r = encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(m.metric), dims, strides, box,
                      elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return VSCAN_ERR_UNSUPPORTED;
  const cuuint64_t dims_b[2] = {static_cast<cuuint64_t>(m.metric_dim),
                                static_cast<cuuint64_t>(m.row_len) * static_cast<cuuint64_t>(m.instances)};
  const cuuint64_t strides_b[1] = {static_cast<cuuint64_t>(m.metric_dim) * 2};
  const cuuint32_t box_b[2] = {tc::kChunkK, 1};
  if (p.b_packed) {
    // large kept sets: the rows were packed into [instance][slot][dim] beforehand, one tile load per stage
    const cuuint64_t rows_packed = static_cast<cuuint64_t>(p.n_chunks) * p.n_pad;
    const cuuint64_t dims_p[3] = {static_cast<cuuint64_t>(m.metric_dim), rows_packed, static_cast<cuuint64_t>(m.instances)};
    const cuuint64_t strides_p[2] = {static_cast<cuuint64_t>(m.metric_dim) * 2, rows_packed * m.metric_dim * 2};
    const cuuint32_t box_p[3] = {tc::kChunkK, static_cast<cuuint32_t>(p.n_pad), 1};
    r = encode(&map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, m.kept_packed, dims_p, strides_p, box_p, elem,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {
    r = encode(&map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(m.metric), dims_b, strides_b, box_b, elem,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  return r == CUDA_SUCCESS ? VSCAN_OK : VSCAN_ERR_UNSUPPORTED;
}

vscan_status launch_assign_tensor(const MergeParams& m, cudaStream_t stream) {
  tc::Params p;
  if (!tc::plan(m, p)) return VSCAN_ERR_UNSUPPORTED;
  CUtensorMap map, map_b;
  vscan_status st = encode_maps(m, p, map, map_b);
  if (st != VSCAN_OK) return st;
  if (p.b_packed) {
    dim3 pgrid((static_cast<unsigned>(p.n_chunks) * p.n_pad + 7) / 8, m.instances);
    VSCAN_LAUNCH("pack_kept", stream, tc::pack_kept_kernel<<<pgrid, 256, 0, stream>>>(m, p.n_chunks * p.n_pad));
  }
  const size_t smem = tc::smem_bytes(p);
  VSCAN_CUDA_TRY(allow_smem(tc::assign_tensor_kernel, smem));
  dim3 grid((m.n_tokens + tc::kTileM - 1) / tc::kTileM, m.instances);
  VSCAN_LAUNCH("assign_tensor", stream,
               (void)launch_dependent(tc::assign_tensor_kernel, grid, dim3(tc::kThreads), smem, stream, map, map_b, p));
  return VSCAN_OK;
}

// ---- assignment + group means in one launch
static int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) n = v;
    else return 148;
  }
  return n;
}

static bool plan_interleaved(const MergeParams& m, tc::Params& p, tc::Interleave& il, int& ctas_per_sm, size_t& smem) {
  if (!tc::plan(m, p) || p.n_chunks != 1 || p.b_packed) return false;
  const int stage = p.a_stage_bytes + p.b_stage_bytes;
  ctas_per_sm = (73 * 1024) / stage >= 3 ? 3 : ((110 * 1024) / stage >= 3 ? 2 : 1);
  smem = tc::smem_bytes(p);
  // the sums: the column slice of every token (whole tile loads) + the member list
  il.x_boxes = (m.n_tokens + tc::kBoxRows - 1) / tc::kBoxRows;
  if (il.x_boxes > tc::kMaxBoxes || m.n_kept > tc::kMaxMeanKept) return false;
  const size_t slice_bytes = static_cast<size_t>(il.x_boxes) * tc::kBoxRows * tc::kSliceCols * 2;
  if (128 + slice_bytes + static_cast<size_t>(m.n_tokens) * 2 > smem) return false;
  if (static_cast<size_t>(m.n_kept) * ((m.n_tokens + 31) / 32) * 6 > slice_bytes) return false;   // the sort's scratch
  if ((reinterpret_cast<uintptr_t>(m.x) & 15u) != 0 || m.dim % 8 != 0) return false;
  il.done = reinterpret_cast<int*>(m.inv_norm);   // the tensor path takes the norms itself: the region is free
  il.tiles = (m.n_tokens + tc::kTileM - 1) / tc::kTileM;
  il.slices = (m.dim + tc::kSliceCols - 1) / tc::kSliceCols;
  // far enough back that the instance's tiles have finished, near enough that its features are still in L2
  int lag = 16;
  if (const char* e = getenv("VSCAN_MERGE_LAG")) lag = atoi(e) > 0 ? atoi(e) : lag;
  il.lag = lag < m.instances ? lag : m.instances;
  if ((static_cast<long long>(m.instances) + il.lag) * il.tiles > 0x7fffffffLL) return false;
  return true;
}

bool merge_interleaved_supported(int dtype, const MergeParams& m) {
  if (!assign_tensor_supported(dtype, m)) return false;
  tc::Params p; tc::Interleave il; int c; size_t smem;
  return plan_interleaved(m, p, il, c, smem);
}

vscan_status launch_merge_interleaved(const MergeParams& m_in, cudaStream_t stream) {
  MergeParams m = m_in;
  m.clear_status = 0;   // the memset below clears the status word together with the counters
  tc::Params p; tc::Interleave il; int ctas_per_sm; size_t smem;
  if (!plan_interleaved(m, p, il, ctas_per_sm, smem)) return VSCAN_ERR_UNSUPPORTED;
  CUtensorMap map, map_b, map_x;
  vscan_status st = encode_maps(m, p, map, map_b);
  if (st != VSCAN_OK) return st;
  {   // column slices of the features for the sums: [instance][row][dim], box = kSliceCols columns x kBoxRows rows
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(m.dim), static_cast<cuuint64_t>(m.row_len),
                                static_cast<cuuint64_t>(m.instances)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(m.dim) * 2, static_cast<cuuint64_t>(m.row_len) * m.dim * 2};
    const cuuint32_t box[3] = {tc::kSliceCols, tc::kBoxRows, 1};
    const cuuint32_t elem[3] = {1, 1, 1};
    if (tc::encode_fn()(&map_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(m.x), dims, strides, box, elem,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return VSCAN_ERR_UNSUPPORTED;
  }
  // status word (first 256 bytes of the workspace) and the counters right behind it
  if (reinterpret_cast<char*>(il.done) != reinterpret_cast<char*>(m.status) + kStatusBytes) return VSCAN_ERR_WORKSPACE;
  VSCAN_CUDA_TRY(cudaMemsetAsync(m.status, 0, kStatusBytes + static_cast<size_t>(m.instances) * sizeof(int), stream));
  const unsigned blocks = static_cast<unsigned>(m.instances + il.lag) * il.tiles;
  if (ctas_per_sm == 3) {
    VSCAN_CUDA_TRY(allow_smem(tc::merge_interleaved_kernel<3>, smem));
    VSCAN_LAUNCH("merge_interleaved", stream,
                 (void)launch_dependent(tc::merge_interleaved_kernel<3>, dim3(blocks), dim3(tc::kThreads), smem, stream, map, map_b, map_x, p, il));
  } else if (ctas_per_sm == 2) {
    VSCAN_CUDA_TRY(allow_smem(tc::merge_interleaved_kernel<2>, smem));
    VSCAN_LAUNCH("merge_interleaved", stream,
                 (void)launch_dependent(tc::merge_interleaved_kernel<2>, dim3(blocks), dim3(tc::kThreads), smem, stream, map, map_b, map_x, p, il));
  } else {
    VSCAN_CUDA_TRY(allow_smem(tc::merge_interleaved_kernel<1>, smem));
    VSCAN_LAUNCH("merge_interleaved", stream,
                 (void)launch_dependent(tc::merge_interleaved_kernel<1>, dim3(blocks), dim3(tc::kThreads), smem, stream, map, map_b, map_x, p, il));
  }
  return VSCAN_OK;
}

}  // namespace vscan
