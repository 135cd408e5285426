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
#include "merge_mean.cuh"
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
  int norms_given;  // 1 / |m_s| comes from the packing kernel (m.inv_norm) instead of being taken from the B stages
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
    // (with norms from the packing kernel the read-back warps never touch the stages)
    for (int s = 0; s < p.stages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], p.norms_given ? 1 : 5); }
    for (int a = 0; a < 2; ++a) { mbar_init(&sh.tmem_full[a], 1); mbar_init(&sh.tmem_empty[a], 4); }
    sh.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)), "r"(p.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = sh.tmem_base;
  grid_dependency_launch();
  grid_dependency_wait();   // the kept list (and the packed rows and norms) come from the kernel before this one
  // Nothing in global memory is written before the wait above: the kernel before this one may belong to an
  // earlier call on the same workspace and still be running.  The clear is still long before any wait can expire.
  if (m.clear_status && b == 0 && t0 == 0 && threadIdx.x == 0) *m.status = 0u;

  if (warp == 0) {
    // ------------------------------------------------------------ producer: TMA tile + TMA row gathers
    // Lane l issues the gathers of row groups l, l+32, ... (four kept rows each); it keeps their row
    // coordinates in registers for the whole n-chunk.  Padding rows repeat the first kept row (their
    // columns are masked in the epilogue).
    const int groups = p.n_pad / 4;                 // gathers per stage
    const int row_base = b * m.row_len + m.cls_offset;
    const int first = row_base + min(max(kept[0], 0), m.n_tokens - 1);
    int s = 0, it = 0;      // ring position kept as counters: no division per stage
    uint32_t phase = 0;
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
        if (ok && it >= p.stages) ok = mbar_wait_warp(&sh.empty[s], phase ^ 1u, abort_flag);
        if (ok) {
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
        if (++s == p.stages) { s = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = instr_desc_bf16(p.n_pad);
      int s = 0;
      uint32_t phase = 0;
      const uint32_t tiles_addr = smem_u32(tiles);
      for (int nc = 0; nc < p.n_chunks && !*abort_flag; ++nc) {
        const int acc = nc & 1, use = nc >> 1;
        if (use > 0) {
          if (!mbar_wait(&sh.tmem_empty[acc], (use - 1) & 1, abort_flag)) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        }
        const uint32_t d_addr = tmem_acc + acc * p.n_pad;
        bool ok = true;
        for (int kc = 0; kc < p.k_chunks; ++kc) {
          if (!mbar_wait(&sh.full[s], phase, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = tiles_addr + s * stage_bytes, b_addr = a_addr + p.a_stage_bytes;
          const uint64_t da = smem_desc_sw128(a_addr), db = smem_desc_sw128(b_addr);
#pragma unroll
          for (int k = 0; k < kChunkK / 16; ++k)   // 16 bf16 = 32 bytes per MMA along K: +2 in 16-byte units
            umma_bf16(d_addr, da + 2u * k, db + 2u * k, idesc, kc > 0 || k > 0);
          umma_commit(&sh.empty[s]);
          if (++s == p.stages) { s = 0; phase ^= 1u; }
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
    int s = 0;
    uint32_t phase = 0;
    bool ok = true;
    // Once `ok` drops the loop keeps running with its work skipped, so that the four warps execute
    // the same sequence of named barriers and warp-wide instructions whatever happens.
    for (int nc = 0; nc < p.n_chunks; ++nc) {
      const int n0 = nc * p.n_pad, acc = nc & 1, use = nc >> 1;
      // |m_s|^2 of the kept rows of this n-chunk, accumulated from the B stages as they pass through
      // shared memory (thread ptid owns rows ptid and ptid + 128)
      float ss[2] = {0.f, 0.f};
      for (int kc = 0; kc < (p.norms_given ? 0 : p.k_chunks); ++kc) {
        const int cur = s;
        if (ok) ok = mbar_wait_warp(&sh.full[cur], phase, abort_flag);
        if (++s == p.stages) { s = 0; phase ^= 1u; }
        if (!ok) continue;
        const unsigned char* bt = tiles + cur * stage_bytes + p.a_stage_bytes;
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
        if (lane == 0) mbar_arrive(&sh.empty[cur]);
      }
      // the buffer was last read two chunks ago, before that chunk's arrive on tmem_empty
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int r = ptid + 128 * u;
        if (r < p.n_pad) {
          float inv = 0.f;
          if (n0 + r < m.n_kept)
            inv = p.norms_given ? __ldcg(m.inv_norm + static_cast<size_t>(b) * m.n_kept + n0 + r) : 1.f / fmaxf(sqrtf(ss[u]), 1e-12f);
          inv_norm[acc * p.n_pad + r] = inv;
        }
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

// ---------------------------------------------------------------------------------------------
// Kept sets above 128 (packed rows, norms from the packing kernel): the assignment on CTA pairs.  A pair of CTAs
// (a cluster of two, on the two SMs of one TPC) takes 256 tokens; each CTA loads its own 128 token rows and HALF of
// the kept rows of a stage, and one MMA of M = 256 issued by the even CTA runs on both SMs, each tensor core reading
// its own token tile and both halves of the kept rows.  Per 128 tokens and stage an SM takes in 16 KB + n_pad/2 rows
// instead of 16 KB + n_pad rows.
// The kernel is persistent: pair i works through items i, i + pairs, ...; an item is a 256-token tile and one of
// `splits` contiguous shares of the n-chunks (two shares when there are at least four chunks, so that the number of
// items divides well over the pairs).  The stage ring and the two accumulators run on across items.
//   warp 0 (both CTAs)   producer: waits on its own `empty`, loads into its own shared memory, bytes counted on
//                        the leader's `full` (armed by the leader's producer with the bytes of both CTAs)
//   warp 1 (leader)      MMA issuer; after a stage's MMAs one commit per CTA frees the stage in both, after an
//                        n-chunk one commit per CTA publishes the accumulator in both
//   warps 2-5 (both)     read their CTA's 128 accumulator rows, running arg-max; the release of an accumulator is
//                        an arrive on the leader's `tmem_empty` (count 8: four warps of each CTA).  With two shares
//                        each leaves (value, slot) per token in the workspace and takes a ticket of its 128-token
//                        tile; whoever comes last compares the two (equal values: the lower slot) and writes the
//                        assignment.  Nobody waits for the other share.
// Tensor memory is allocated and freed by warp 1 of both CTAs (pair-wide allocation); a cluster barrier before the
// release makes sure neither CTA leaves, or frees anything, while the other may still use it.  Every mbarrier wait
// is bounded as in assign_tile.
struct PairPlan {
  int items, ptiles, splits, chunks_per_split;
  float2* partial;    // [splits][instances][n_tokens] (value, slot as int bits), only with splits > 1
  int* tickets;       // [instances][ceil(n_tokens / 128)], zero at launch
};

constexpr int kPairThreads = kThreads + 32;   // a second producer warp
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads)
assign_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, Params p, PairPlan pl) {
  extern __shared__ unsigned char smem_dyn[];
  __shared__ Shared sh;
  __shared__ int ticket;
  unsigned char* tiles = smem_dyn + ((1024u - (static_cast<uint32_t>(__cvta_generic_to_shared(smem_dyn)) & 1023u)) & 1023u);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const MergeParams& m = p.m;
  const uint32_t rank = pair_rank();
  const bool leader = rank == 0;
  const int pair = blockIdx.x >> 1, pairs = gridDim.x >> 1;
  volatile int* abort_flag = &sh.abort_flag;
  const int half_rows = p.n_pad / 2;                              // kept rows of a stage held by this CTA
  const int stage_bytes = p.a_stage_bytes + p.b_stage_bytes;      // b_stage_bytes: half_rows * 128, rounded to 1024
  float* inv_norm = reinterpret_cast<float*>(tiles + p.stages * stage_bytes);   // [accumulator][n_pad]
  const int per_instance = pl.splits * pl.ptiles;
  // item -> instance, share of the n-chunks [c_lo, c_hi), first token of this CTA's 128 rows
  auto decode = [&](int item, int& b, int& share, int& c_lo, int& c_hi, int& t0) {
    b = item / per_instance;
    const int rem = item - b * per_instance;
    share = rem / pl.ptiles;
    t0 = (rem - share * pl.ptiles) * (2 * kTileM) + static_cast<int>(rank) * kTileM;
    c_lo = share * pl.chunks_per_split;
    c_hi = min(p.n_chunks, c_lo + pl.chunks_per_split);
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&sh.tmem_full[a], 1); mbar_init(&sh.tmem_empty[a], 8); }
    sh.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)), "r"(p.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  pair_sync();   // both CTAs' barriers exist before either sends a load or an arrive to the other
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = sh.tmem_base;
  grid_dependency_launch();
  grid_dependency_wait();   // kept list, packed rows, norms and zeroed tickets come from the kernels before this one; nothing is written before
  if (m.clear_status && blockIdx.x == 0 && threadIdx.x == 0) *m.status = 0u;

  if (warp == 0 || warp == 6) {
    // ------------------------------------------------------------ producers: warp 0 the token tiles, warp 6 the kept rows
    // (two warps, so that the two loads of a stage are issued side by side; the leader's warp 0 arms the barrier)
    const bool loads_a = warp == 0;
    int s = 0, it = 0;
    uint32_t phase = 0;     // parity of the stage's current round
    bool ok = true;
    // The token tile of an item comes from DRAM the first time it is read (the later n-chunks find it in L2), and a
    // stage is complete only when its last byte is there: the tile of the NEXT item is therefore asked into L2 while
    // the first n-chunk of the current one streams through (lane 1; the very first tile up front by all lanes).
    if (loads_a && pair < pl.items) {
      int b, share, c_lo, c_hi, t0;
      decode(pair, b, share, c_lo, c_hi, t0);
      for (int kc = lane; kc < p.k_chunks; kc += 32) tma_prefetch_l2_3d(&map_a, kc * kChunkK, m.cls_offset + t0, b);
    }
    const uint32_t full0 = pair_addr(&sh.full[0], 0);   // the leader's `full` barriers, 8 bytes apart
    for (int item = pair; item < pl.items; item += pairs) {
      int b, share, c_lo, c_hi, t0;
      decode(item, b, share, c_lo, c_hi, t0);
      int nb = 0, nshare, nc_lo, nc_hi, nt0 = 0;
      const bool has_next = loads_a && item + pairs < pl.items;
      if (has_next) decode(item + pairs, nb, nshare, nc_lo, nc_hi, nt0);
      for (int nc = c_lo; nc < c_hi; ++nc) {
        const int b_row = nc * p.n_pad + static_cast<int>(rank) * half_rows;
        for (int kc = 0; kc < p.k_chunks; ++kc, ++it) {
          if (ok && it >= p.stages) ok = mbar_wait_warp(&sh.empty[s], phase ^ 1u, abort_flag);
          if (ok) {
            if (lane == 1 && has_next && nc == c_lo) tma_prefetch_l2_3d(&map_a, kc * kChunkK, m.cls_offset + nt0, nb);
            if (lane == 0) {
              unsigned char* at = tiles + s * stage_bytes;
              const uint32_t bar = full0 + 8u * s;
              if (loads_a) {
                if (leader) mbar_arrive_expect_tx(&sh.full[s], 2u * static_cast<uint32_t>(p.a_stage_bytes + half_rows * 128));
                pair_tma_load_3d(at, &map_a, bar, kc * kChunkK, m.cls_offset + t0, b);
              } else {
                pair_tma_load_3d(at + p.a_stage_bytes, &map_b, bar, kc * kChunkK, b_row, b);
              }
            }
          }
          if (++s == p.stages) { s = 0; phase ^= 1u; }
        }
      }
    }
    // the leader's commits to this CTA's `empty` barriers have all arrived before its shared memory goes
    for (int i = 0; i < min(it, p.stages); ++i) {
      if (s == 0) { s = p.stages; phase ^= 1u; }
      --s;
      if (ok) ok = mbar_wait_warp(&sh.empty[s], phase, abort_flag);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader only)
    if (leader && lane == 0) {
      const uint32_t idesc = pair_instr_desc_bf16(p.n_pad);
      int s = 0, g = 0;      // stage of the ring; n-chunks since the start of the kernel
      uint32_t phase = 0;
      bool ok = true;
      const uint32_t tiles_addr = smem_u32(tiles);
      const uint32_t empty_local = smem_u32(&sh.empty[0]), empty_peer = pair_addr(&sh.empty[0], 1);
      for (int item = pair; item < pl.items && ok; item += pairs) {
        int b, share, c_lo, c_hi, t0;
        decode(item, b, share, c_lo, c_hi, t0);
        for (int nc = c_lo; nc < c_hi && ok && !*abort_flag; ++nc, ++g) {
          const int acc = g & 1, use = g >> 1;
          if (use > 0) {
            if (!mbar_wait(&sh.tmem_empty[acc], (use - 1) & 1, abort_flag)) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          }
          const uint32_t d_addr = tmem_acc + acc * p.n_pad;
          for (int kc = 0; kc < p.k_chunks; ++kc) {
            if (!mbar_wait(&sh.full[s], phase, abort_flag)) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a_addr = tiles_addr + s * stage_bytes, b_addr = a_addr + p.a_stage_bytes;
            const uint64_t da = smem_desc_sw128(a_addr), db = smem_desc_sw128(b_addr);
#pragma unroll
            for (int k = 0; k < kChunkK / 16; ++k)
              pair_umma_bf16(d_addr, da + 2u * k, db + 2u * k, idesc, kc > 0 || k > 0);
            pair_umma_commit(empty_local + 8u * s);
            pair_umma_commit(empty_peer + 8u * s);
            if (++s == p.stages) { s = 0; phase ^= 1u; }
          }
          if (!ok) break;
          pair_umma_commit(smem_u32(&sh.tmem_full[acc]));
          pair_umma_commit(pair_addr(&sh.tmem_full[acc], 1));
        }
        if (*abort_flag) ok = false;
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ epilogue: this CTA's 128 accumulator rows -> arg-max
    const int ptid = (warp - 2) * 32 + lane;
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const int tiles128 = (m.n_tokens + kTileM - 1) / kTileM;
    bool ok = true;
    int g = 0;
    // Once `ok` drops the loops keep running with their work skipped, so that the four warps execute the same
    // sequence of named barriers whatever happens.
    for (int item = pair; item < pl.items; item += pairs) {
      int b, share, c_lo, c_hi, t0;
      decode(item, b, share, c_lo, c_hi, t0);
      const int32_t* kept = m.kept + static_cast<size_t>(b) * m.n_kept;
      float best_val = -INFINITY;
      int best_idx = 0;
      for (int nc = c_lo; nc < c_hi; ++nc, ++g) {
        const int n0 = nc * p.n_pad, acc = g & 1, use = g >> 1;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int r = ptid + 128 * u;
          if (r < p.n_pad)
            inv_norm[acc * p.n_pad + r] = n0 + r < m.n_kept ? __ldcg(m.inv_norm + static_cast<size_t>(b) * m.n_kept + n0 + r) : 0.f;
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
        if (lane == 0) {
          if (leader) mbar_arrive(&sh.tmem_empty[acc]);
          else pair_remote_arrive(pair_addr(&sh.tmem_empty[acc], 0));
        }
      }
      // ---- the item's result for token t0 + row is (best_val, best_idx)
      bool write = ok;
      if (pl.splits > 1) {
        const size_t inst_tokens = static_cast<size_t>(m.instances) * m.n_tokens;
        const size_t tok = static_cast<size_t>(b) * m.n_tokens + t0 + row;
        if (ok && t0 + row < m.n_tokens) pl.partial[share * inst_tokens + tok] = make_float2(best_val, __int_as_float(best_idx));
        __threadfence();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (ptid == 0) ticket = (ok && t0 < m.n_tokens) ? atomicAdd(&pl.tickets[b * tiles128 + t0 / kTileM], 1) : -1;
        asm volatile("bar.sync 1, 128;" ::: "memory");
        write = ticket == pl.splits - 1;          // the last share of this tile to finish combines them
        if (write) {
          __threadfence();
          if (t0 + row < m.n_tokens) {
            for (int h2 = 0; h2 < pl.splits; ++h2) {
              if (h2 == share) continue;
              const float2 o = __ldcg(pl.partial + h2 * inst_tokens + tok);
              const int oi = __float_as_int(o.y);
              if (o.x > best_val || (o.x == best_val && oi < best_idx)) { best_val = o.x; best_idx = oi; }
            }
          }
        }
      }
      sh.best_slot[row] = best_idx;
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (write) {
        for (int s_idx = ptid; s_idx < m.n_kept; s_idx += 128) {   // a kept token belongs to its own slot
          const int t = min(max(kept[s_idx], 0), m.n_tokens - 1);
          if (t >= t0 && t < t0 + kTileM) sh.best_slot[t - t0] = s_idx;
        }
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (write && t0 + ptid < m.n_tokens) m.assign[static_cast<size_t>(b) * m.n_tokens + t0 + ptid] = sh.best_slot[ptid];
      asm volatile("bar.sync 1, 128;" ::: "memory");   // best_slot and ticket are reused by the next item
    }
  }

  // ------------------------------------------------------------ teardown
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (sh.abort_flag) {
    if (threadIdx.x == 0) atomicExch(m.status, static_cast<uint32_t>(VSCAN_ERR_TIMEOUT));
    for (int i = 0; i < 64; ++i) __nanosleep(2000);   // copies still in flight land before the shared memory goes
    __syncthreads();
  }
  pair_sync();   // the other CTA's MMAs, loads and tensor-memory reads are over as well
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(p.tmem_cols) : "memory");
  }
}

// Assignment and group means in ONE persistent launch (one CTA per SM), so that the second pass over the
// features (the sums of Eq. 4) reads them from L2 while they are still there, the start-up cost of a CTA
// is paid once per SM instead of once per tile, and the read-back of one tile overlaps the MMAs of the next.
//   warps 0-5   the assignment roles of assign_tile (producer, MMA issuer, four read-back warps), looping
//               over tiles blockIdx.x, blockIdx.x + gridDim.x, ...; two accumulators alternate between
//               tiles; after a tile's assignments are visible device-wide the instance's counter of
//               finished tiles goes up by one
//   warps 6-13  the mean group: takes jobs (16 kept slots of one instance) off a global counter in
//               order, waits (bounded spin; on expiry VSCAN_ERR_TIMEOUT) until the instance's tiles are
//               all finished, lists the members of its slots and sums them, one warp per slot, exactly as
//               group_mean_body does (same order of additions, same bits)
// The assignment warps never wait for a mean group, and every CTA of the grid is resident at once (the
// grid has at most one CTA per SM), so the waits of the mean groups end.
constexpr int kMeanWarps = 8, kMeanThreads = kMeanWarps * 32;
constexpr int kPersistThreads = kThreads + kMeanThreads;
constexpr int kJobSlots = 16;                      // kept slots per mean job: two per warp
constexpr uint32_t kDoneSpinLimit = 1u << 22;      // polls of ~100 ns

struct Persist {
  int* done;              // [instances] finished assignment tiles, zero at launch
  int* job_head;          // next mean job, zero at launch
  int tiles;              // tiles per instance
  int total_tiles;
  int jobs_per_instance;
  int total_jobs;
};

struct PersistShared {
  Shared a;
  int warp_sums[33];
  int job, ready;
};

__device__ __forceinline__ void mean_group_sync() { asm volatile("bar.sync 2, %0;" ::"n"(kMeanThreads) : "memory"); }

// Copies the kept rows of every instance into a contiguous [instance][slot][dim] buffer (slots past n_kept are
// zero) and, having read them anyway, writes 1 / max(|m_s|, eps) of every
// kept token; the first CTA also zeroes the status word and the counters of the persistent kernel that
// follows.  One warp per slot, the whole row in flight at once.
__global__ void __launch_bounds__(256) pack_kept_norm_kernel(MergeParams m, int rows_packed) {
  grid_dependency_launch();
  // The kernel before this one may be the persistent kernel of an earlier call on the same workspace, which lets
  // its successor start early and goes on reading the counters, the packed rows and the norms: every write of
  // this kernel therefore comes after the wait.  (The kept list also comes from the kernel before this one.)
  grid_dependency_wait();
  if (blockIdx.x == 0 && blockIdx.y == 0) {
    if (threadIdx.x == 0) *m.status = 0u;
    for (int i = threadIdx.x; i <= m.instances; i += 256) m.counters[i] = 0;
    if (m.tickets)
      for (int i = threadIdx.x; i < m.instances * ((m.n_tokens + kTileM - 1) / kTileM); i += 256) m.tickets[i] = 0;
  }
  const int b = blockIdx.y, s = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (s >= rows_packed) return;
  uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(m.kept_packed) +
                                        (static_cast<size_t>(b) * rows_packed + s) * m.metric_dim);
  const int vecs = m.metric_dim / 8;
  if (s >= m.n_kept) {
    for (int v = lane; v < vecs; v += 32) st_16(dst + v, make_uint4(0u, 0u, 0u, 0u));
    return;
  }
  const int t = min(max(m.kept[static_cast<size_t>(b) * m.n_kept + s], 0), m.n_tokens - 1);
  const uint4* src = reinterpret_cast<const uint4*>(
      static_cast<const __nv_bfloat16*>(m.metric) + (static_cast<size_t>(b) * m.row_len + m.cls_offset + t) * m.metric_dim);
  float ss = 0.f;
  for (int v0 = 0; v0 < vecs; v0 += 128) {
    uint4 r[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) { const int v = v0 + lane + 32 * u; if (v < vecs) r[u] = ld_nc_16(src + v); }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int v = v0 + lane + 32 * u;
      if (v < vecs) {
        st_16(dst + v, r[u]);
        float f[8];
        Vec16<__nv_bfloat16>::unpack(r[u], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
      }
    }
  }
  ss = warp_sum(ss);
  if (lane == 0) m.inv_norm[static_cast<size_t>(b) * m.n_kept + s] = 1.f / fmaxf(sqrtf(ss), 1e-12f);
}

// dynamic shared memory: alignment slack | stages x [A tile | B tile] | inv_norm[2][n_pad] | list and staged
// assignments of the mean group (2 * n_tokens words)
__global__ void __launch_bounds__(kPersistThreads, 1)
merge_persistent_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, Params p,
                        Persist ps) {
  extern __shared__ unsigned char smem_dyn[];
  __shared__ PersistShared shp;
  Shared& sh = shp.a;
  unsigned char* tiles = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const MergeParams& m = p.m;
  volatile int* abort_flag = &sh.abort_flag;
  const int stage_bytes = p.a_stage_bytes + p.b_stage_bytes;
  float* inv_norm = reinterpret_cast<float*>(tiles + p.stages * stage_bytes);   // [accumulator][n_pad]
  uint32_t* mean_list = reinterpret_cast<uint32_t*>(inv_norm + 2 * p.n_pad);

  if (threadIdx.x == 0) {
    // a stage is free again once the MMAs that read it have completed (the norms of the kept rows come
    // from the packing kernel, so the read-back warps never touch the stages)
    for (int s = 0; s < p.stages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&sh.tmem_full[a], 1); mbar_init(&sh.tmem_empty[a], 4); }
    sh.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)), "r"(p.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = sh.tmem_base;
  grid_dependency_launch();
  grid_dependency_wait();   // packed kept rows, norms and cleared counters come from the kernel before this one

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    const int groups = p.n_pad / 4;
    int it = 0, cur_b = -1;
    int rows[2][4];
    bool ok = true;
    for (int w = blockIdx.x; w < ps.total_tiles && ok; w += gridDim.x) {
      const int b = w / ps.tiles, t0 = (w - b * ps.tiles) * kTileM;
      if (b != cur_b) {   // row coordinates of the instance's kept tokens; padding repeats the first one
        const int32_t* kept = m.kept + static_cast<size_t>(b) * m.n_kept;
        const int row_base = b * m.row_len + m.cls_offset;
        const int first = row_base + min(max(kept[0], 0), m.n_tokens - 1);
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const int g = lane + 32 * i;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int s_idx = g * 4 + j;
            rows[i][j] = (g < groups && s_idx < m.n_kept) ? row_base + min(max(kept[s_idx], 0), m.n_tokens - 1) : first;
          }
        }
        cur_b = b;
      }
      for (int kc = 0; kc < p.k_chunks && ok; ++kc, ++it) {
        const int s = it % p.stages, round = it / p.stages;
        if (round > 0) ok = mbar_wait_warp(&sh.empty[s], (round - 1) & 1, abort_flag);
        if (!ok) break;
        unsigned char* at = tiles + s * stage_bytes;
        if (lane == 0) {
          mbar_arrive_expect_tx(&sh.full[s], p.a_stage_bytes + p.n_pad * 128);
          tma_load_3d(at, &map_a, &sh.full[s], kc * kChunkK, m.cls_offset + t0, b);
          if (p.b_packed) tma_load_3d(at + p.a_stage_bytes, &map_b, &sh.full[s], kc * kChunkK, 0, b);
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
      int it = 0, i = 0;
      bool ok = true;
      for (int w = blockIdx.x; w < ps.total_tiles && ok && !*abort_flag; w += gridDim.x, ++i) {
        const int acc = i & 1, use = i >> 1;
        if (use > 0) {
          if (!mbar_wait(&sh.tmem_empty[acc], (use - 1) & 1, abort_flag)) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        }
        const uint32_t d_addr = tmem_acc + acc * p.n_pad;
        for (int kc = 0; kc < p.k_chunks; ++kc, ++it) {
          const int s = it % p.stages, round = it / p.stages;
          if (!mbar_wait(&sh.full[s], round & 1, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = smem_u32(tiles + s * stage_bytes), b_addr = a_addr + p.a_stage_bytes;
          const uint64_t da = smem_desc_sw128(a_addr), db = smem_desc_sw128(b_addr);
#pragma unroll
          for (int k = 0; k < kChunkK / 16; ++k) umma_bf16(d_addr, da + 2u * k, db + 2u * k, idesc, kc > 0 || k > 0);
          umma_commit(&sh.empty[s]);
        }
        if (ok) umma_commit(&sh.tmem_full[acc]);
      }
    }
    __syncwarp();
  } else if (warp < kThreads / 32) {
    // ------------------------------------------------------------ read-back: accumulator -> arg-max -> assignments
    const int ptid = (warp - 2) * 32 + lane;  // 0..127
    const int quarter = warp & 3;             // tensor-memory lanes this warp may read
    const int row = quarter * 32 + lane;      // token row of this thread within the tile
    int i = 0;
    bool ok = true;
    // Once `ok` drops the loops keep running with their work skipped, so that the four warps execute
    // the same sequence of named barriers and warp-wide instructions whatever happens.
    for (int w = blockIdx.x; w < ps.total_tiles; w += gridDim.x, ++i) {
      const int b = w / ps.tiles, t0 = (w - b * ps.tiles) * kTileM;
      const int acc = i & 1, use = i >> 1;
      const int32_t* kept = m.kept + static_cast<size_t>(b) * m.n_kept;
      // 1 / |m_s| of the instance's kept tokens -> shared memory; this buffer was last read two tiles ago,
      // before that tile's arrive on tmem_empty
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int r = ptid + 128 * u;
        if (r < p.n_pad) inv_norm[acc * p.n_pad + r] = (r < m.n_kept) ? __ldcg(m.inv_norm + static_cast<size_t>(b) * m.n_kept + r) : 0.f;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (ok) ok = mbar_wait_warp(&sh.tmem_full[acc], use & 1, abort_flag);
      float best_val = -INFINITY;
      int best_idx = 0;
      if (ok) {
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
            if (c0 + j < p.n_pad && c0 + j < m.n_kept) {
              const float val = __uint_as_float(v[j]) * inv_norm[acc * p.n_pad + c0 + j];
              if (val > best_val) { best_val = val; best_idx = c0 + j; }
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
      // publish: the stores above first, then one increment of the instance's counter
      __threadfence();
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (ptid == 0 && ok && !*abort_flag) atomicAdd(ps.done + b, 1);
    }
  } else {
    // ------------------------------------------------------------ mean group
    const int gtid = threadIdx.x - kThreads;
    while (true) {
      if (gtid == 0) {
        const int q = atomicAdd(ps.job_head, 1);
        int ready = 1;
        if (q < ps.total_jobs) {
          const volatile int* flag = ps.done + q / ps.jobs_per_instance;
          uint32_t spins = 0;
          while (*flag < ps.tiles && spins < kDoneSpinLimit && !*abort_flag) { __nanosleep(100); ++spins; }
          ready = *flag >= ps.tiles;
          if (!ready) atomicExch(m.status, static_cast<uint32_t>(VSCAN_ERR_TIMEOUT));
          __threadfence();
        }
        shp.job = q;
        shp.ready = ready;
      }
      mean_group_sync();
      const int q = shp.job, ready = shp.ready;
      mean_group_sync();   // everyone has the job before thread 0 takes the next one
      if (q >= ps.total_jobs || !ready) break;
      // the ordered sums of group_mean_kernel: same additions in the same order, hence the same bits
      group_mean_body<__nv_bfloat16, 4, 4, kJobSlots, kMeanWarps>(m, q / ps.jobs_per_instance, (q % ps.jobs_per_instance) * kJobSlots,
                                                                  mean_list, shp.warp_sums, gtid, NamedSync<2, kMeanThreads>());
    }
  }

  // ------------------------------------------------------------ teardown
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (sh.abort_flag) {
    if (threadIdx.x == 0) atomicExch(m.status, static_cast<uint32_t>(VSCAN_ERR_TIMEOUT));
    for (int i = 0; i < 64; ++i) __nanosleep(2000);   // copies still in flight land before the memory is released
    __syncthreads();
  }
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(p.tmem_cols) : "memory");
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
  // Large kept sets: the packing kernel has read every kept row anyway and leaves 1 / |m_s| behind; reading the
  // B stages a second time for the norms competes with the MMAs for shared-memory bandwidth (498 us against 619 us
  // at 2048 kept tokens).  (Two token tiles per CTA sharing every kept-row stage measured slower: 153 us against
  // 124 us per 128 tokens, the MMAs of a round then wait for the read-back of the one before.)
  p.norms_given = p.b_packed;
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
static vscan_status encode_maps(const MergeParams& m, const tc::Params& p, CUtensorMap& map, CUtensorMap& map_b, int packed_box_rows) {
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
    const cuuint32_t box_p[3] = {tc::kChunkK, static_cast<cuuint32_t>(packed_box_rows), 1};
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

static int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) n = v;
    else return 148;
  }
  return n;
}

vscan_status launch_assign_tensor(const MergeParams& m, cudaStream_t stream) {
  tc::Params p;
  if (!tc::plan(m, p)) return VSCAN_ERR_UNSUPPORTED;
  // packed kept rows: CTA pairs, each CTA holding half of a stage's kept rows
  // kept sets of 129-256 take the same form in one round: with row gathers (48 requests per stage at 192 kept tokens)
  // the single-CTA kernel is bound by the issue rate of its producer
  if (!p.b_packed && m.n_kept > 128 && m.kept_packed != nullptr && m.inv_norm != nullptr) { p.b_packed = 1; p.norms_given = 1; }
  const bool pair = p.b_packed && p.norms_given && p.n_pad % 16 == 0;
  if (pair) {
    while (p.tmem_cols < 2 * p.n_pad) p.tmem_cols *= 2;   // the accumulators alternate between n-chunks of successive items
    p.b_stage_bytes = ((p.n_pad / 2 * tc::kChunkK * 2) + 1023) / 1024 * 1024;
    // (a seventh stage, which just fits, measured slower: 301 us against 294 us at 2048 kept tokens)
    int stages = (215 * 1024) / (p.a_stage_bytes + p.b_stage_bytes);
    p.stages = stages > tc::kMaxStages ? tc::kMaxStages : stages;
  }
  CUtensorMap map, map_b;
  vscan_status st = encode_maps(m, p, map, map_b, pair ? p.n_pad / 2 : p.n_pad);
  if (st != VSCAN_OK) return st;
  if (p.b_packed) {
    dim3 pgrid((static_cast<unsigned>(p.n_chunks) * p.n_pad + 7) / 8, m.instances);
    VSCAN_LAUNCH("pack_kept", stream,
                 (void)launch_dependent(tc::pack_kept_norm_kernel, pgrid, dim3(256), 0, stream, m, p.n_chunks * p.n_pad));
  }
  if (pair) {
    tc::PairPlan pl;
    pl.ptiles = (m.n_tokens + 2 * tc::kTileM - 1) / (2 * tc::kTileM);
    pl.splits = (p.n_chunks >= 4 && m.partial && m.tickets) ? 2 : 1;
    pl.chunks_per_split = (p.n_chunks + pl.splits - 1) / pl.splits;
    pl.partial = m.partial; pl.tickets = m.tickets;
    const long long items = 1ll * m.instances * pl.splits * pl.ptiles;
    if (items > 0x3fffffffLL) return VSCAN_ERR_UNSUPPORTED;
    pl.items = static_cast<int>(items);
    const size_t smem = tc::smem_bytes(p) + (p.n_chunks > 1 ? 0 : static_cast<size_t>(p.n_pad) * sizeof(float));   // two norm buffers
    VSCAN_CUDA_TRY(allow_smem(tc::assign_pair_kernel, smem));
    const int pairs_max = sm_count() / 2;
    const unsigned pairs = static_cast<unsigned>(pl.items < pairs_max ? pl.items : pairs_max);
    VSCAN_LAUNCH("assign_tensor", stream,
                 (void)launch_dependent(tc::assign_pair_kernel, dim3(2 * pairs), dim3(tc::kPairThreads), smem, stream, map, map_b, p, pl));
    return VSCAN_OK;
  }
  const size_t smem = tc::smem_bytes(p);
  VSCAN_CUDA_TRY(allow_smem(tc::assign_tensor_kernel, smem));
  dim3 grid((m.n_tokens + tc::kTileM - 1) / tc::kTileM, m.instances);
  VSCAN_LAUNCH("assign_tensor", stream,
               (void)launch_dependent(tc::assign_tensor_kernel, grid, dim3(tc::kThreads), smem, stream, map, map_b, p));
  return VSCAN_OK;
}

// ---- assignment + group means in one persistent launch
static bool plan_persistent(const MergeParams& m, tc::Params& p, tc::Persist& ps, size_t& smem) {
  if (!tc::plan(m, p) || p.n_chunks != 1 || p.b_packed || m.kept_packed == nullptr) return false;
  p.b_packed = 1;   // one producer warp per SM: a tile load of the packed kept rows per stage instead of n_pad / 4 row gathers
  if (m.counters == nullptr || m.inv_norm == nullptr) return false;
  if ((reinterpret_cast<uintptr_t>(m.x) & 15u) != 0 || m.dim % 8 != 0 || m.n_tokens >= (1 << 24)) return false;
  // one CTA per SM: as many stages as fit beside the inverse norms (two accumulators) and the mean group's lists
  const size_t stage = static_cast<size_t>(p.a_stage_bytes + p.b_stage_bytes);
  const size_t fixed = 1024 + 2 * static_cast<size_t>(p.n_pad) * sizeof(float) + static_cast<size_t>(m.n_tokens) * 8 + 16;
  if (fixed + 3 * stage > 224 * 1024) return false;
  size_t stages = (224 * 1024 - fixed) / stage;
  if (stages > tc::kMaxStages) stages = tc::kMaxStages;
  p.stages = static_cast<int>(stages);
  p.tmem_cols = 32;
  while (p.tmem_cols < 2 * p.n_pad) p.tmem_cols *= 2;
  smem = fixed + stages * stage;
  ps.done = m.counters;
  ps.job_head = ps.done + m.instances;
  ps.tiles = (m.n_tokens + tc::kTileM - 1) / tc::kTileM;
  const long long total_tiles = static_cast<long long>(m.instances) * ps.tiles;
  ps.jobs_per_instance = (m.n_kept + tc::kJobSlots - 1) / tc::kJobSlots;
  const long long total_jobs = static_cast<long long>(m.instances) * ps.jobs_per_instance;
  if (total_tiles > 0x3fffffffLL || total_jobs > 0x3fffffffLL) return false;
  ps.total_tiles = static_cast<int>(total_tiles);
  ps.total_jobs = static_cast<int>(total_jobs);
  return true;
}

bool merge_interleaved_supported(int dtype, const MergeParams& m) {
  if (!assign_tensor_supported(dtype, m)) return false;
  tc::Params p; tc::Persist ps; size_t smem;
  return plan_persistent(m, p, ps, smem);
}

vscan_status launch_merge_interleaved(const MergeParams& m_in, cudaStream_t stream) {
  MergeParams m = m_in;
  m.clear_status = 0;   // the packing kernel clears the status word together with the counters
  tc::Params p; tc::Persist ps; size_t smem;
  if (!plan_persistent(m, p, ps, smem)) return VSCAN_ERR_UNSUPPORTED;
  CUtensorMap map, map_b;
  vscan_status st = encode_maps(m, p, map, map_b, p.n_pad);
  if (st != VSCAN_OK) return st;
  {   // packed kept rows + their inverse norms; also clears the status word and the counters
    dim3 pgrid((static_cast<unsigned>(p.n_pad) + 7) / 8, m.instances);
    VSCAN_LAUNCH("pack_kept", stream,
                 (void)launch_dependent(tc::pack_kept_norm_kernel, pgrid, dim3(256), 0, stream, m, p.n_pad));
  }
  const int sms = sm_count();
  const unsigned blocks = static_cast<unsigned>(ps.total_tiles < sms ? ps.total_tiles : sms);
  VSCAN_CUDA_TRY(allow_smem(tc::merge_persistent_kernel, smem));
  VSCAN_LAUNCH("merge_persistent", stream,
               (void)launch_dependent(tc::merge_persistent_kernel, dim3(blocks), dim3(tc::kPersistThreads), smem, stream, map, map_b, p, ps));
  return VSCAN_OK;
}

}  // namespace vscan
