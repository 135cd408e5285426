// Fused merge (Sec. 4.1 "Token Merging", Eq. 4): kept-token norms, similarity MMAs + arg-max, and the
// group means of one encoder instance in ONE kernel, so that the second pass over the features (the
// sums of Eq. 4) finds them in L2 instead of HBM.
//
// One thread-block cluster per instance (1, 2 or 4 CTAs); fewer instances in flight means the
// features an instance streamed in phase 1 are still cache-resident when phase 2 re-reads them.
//   phase 0  warps 2-11: 1 / max(|m_s|, eps) of every kept token -> shared memory
//   phase 1  warp 0 TMA producer (token tiles + gathered kept rows), warp 1 tcgen05 MMA issuer,
//            warps 2-5 epilogue (tensor memory -> arg-max); two accumulators alternate between tiles.
//            Every CTA of the cluster owns a contiguous range of tokens; the slot of each token is
//            written into the `assign` array of every CTA of the cluster (distributed shared memory).
//   cluster barrier
//   phase 2  all 12 warps: CTA r sums the groups of slots r, r + C, ...; members are listed in
//            ascending token order, rows added in that order in fp32, one rounding on output.
// Waits on mbarriers are bounded; on expiry the cluster still meets at its barrier, records
// VSCAN_ERR_TIMEOUT, frees its tensor memory and returns.
#include <cooperative_groups.h>

#include "merge.cuh"
#include "tc_common.cuh"

namespace cg = cooperative_groups;

namespace vscan {
namespace fused {

using namespace tc;

constexpr int kThreads = 384;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxTokens = 8192;

struct Params {
  MergeParams m;
  int n_pad;          // kept columns of the MMA, multiple of 16, <= 256
  int k_chunks;       // ceil(metric_dim / 64)
  int stages;
  int tmem_cols;      // power of two >= 2 * n_pad
  int a_stage_bytes, b_stage_bytes;
  int cluster;        // CTAs per instance
  int rows_per_rank;  // tokens owned by one CTA
  int tiles_per_rank; // ceil(rows_per_rank / 128)
  int tail_rows;      // rows of the last tile of a rank (box height of the tail tensor map)
  int tiles_bytes;    // bytes of the stage ring
};

struct Shared {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t tmem_full[2];
  uint64_t tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;
  int warp_sums[33];
  float inv_norm[kMaxN];
};

// Sum the rows of one group into fp32 accumulators.  `list` holds (slot << 16 | token) in ascending
// token order; lanes split the row in 16-byte pieces (VPL pieces per lane), R rows in flight.
template <int VPL, int R>
__device__ __forceinline__ void sum_group(const uint32_t* list, int n_list, unsigned slot, const __nv_bfloat16* xb,
                                          int dim, int vecs, int v0, float (&acc)[VPL][8], int& count) {
  const int lane = threadIdx.x & 31;
  count = 0;
  for (int c = 0; c < n_list; c += 32) {
    const uint32_t entry = c + lane < n_list ? list[c + lane] : 0xFFFFFFFFu;
    unsigned mask = __ballot_sync(0xffffffffu, (entry >> 16) == slot);
    count += __popc(mask);
    while (mask) {
      int tok[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        tok[r] = -1;
        if (mask) {
          const int l = __ffs(mask) - 1;
          mask &= mask - 1;
          tok[r] = static_cast<int>(__shfl_sync(0xffffffffu, entry, l) & 0xFFFFu);
        }
      }
      uint4 raw[R][VPL];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const uint4* row = reinterpret_cast<const uint4*>(xb + static_cast<size_t>(tok[r] < 0 ? tok[0] : tok[r]) * dim);
#pragma unroll
        for (int i = 0; i < VPL; ++i) {
          const int v = v0 + lane + 32 * i;
          if (v < vecs && tok[r] >= 0) raw[r][i] = ld_nc_16(row + v);
        }
      }
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if (tok[r] < 0) continue;
#pragma unroll
        for (int i = 0; i < VPL; ++i) {
          const int v = v0 + lane + 32 * i;
          if (v < vecs) {
            float f[8];
            Vec16<__nv_bfloat16>::unpack(raw[r][i], f);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[i][e] += f[e];
          }
        }
      }
    }
  }
}

template <int VPL, int R>
__device__ __forceinline__ void group_means(const Params& p, const uint32_t* list, int n_list, int rank, int b) {
  const MergeParams& m = p.m;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int vecs = m.dim / 8;
  const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(m.x) + (static_cast<size_t>(b) * m.row_len + m.cls_offset) * m.dim;
  for (int s = rank + p.cluster * warp; s < m.n_kept; s += p.cluster * kWarps) {
    __nv_bfloat16* out = static_cast<__nv_bfloat16*>(m.merged) + (static_cast<size_t>(b) * m.n_kept + s) * m.dim;
    for (int v0 = 0; v0 < vecs; v0 += 32 * VPL) {
      float acc[VPL][8];
#pragma unroll
      for (int i = 0; i < VPL; ++i)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[i][e] = 0.f;
      int count;
      sum_group<VPL, R>(list, n_list, static_cast<unsigned>(s), xb, m.dim, vecs, v0, acc, count);
      const float inv = 1.f / static_cast<float>(max(count, 1));
#pragma unroll
      for (int i = 0; i < VPL; ++i) {
        const int v = v0 + lane + 32 * i;
        if (v < vecs) {
          float f[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) f[e] = acc[i][e] * inv;
          st_16(reinterpret_cast<uint4*>(out) + v, Vec16<__nv_bfloat16>::pack(f));
        }
      }
      if (v0 == 0 && lane == 0 && m.counts) m.counts[static_cast<size_t>(b) * m.n_kept + s] = count;
    }
  }
}

// dynamic shared memory: [stage ring, 1024-byte aligned] [assign: n_tokens x uint16]
__global__ void __launch_bounds__(kThreads) merge_fused_kernel(const __grid_constant__ CUtensorMap map_a,
                                                               const __grid_constant__ CUtensorMap map_a_tail,
                                                               const __grid_constant__ CUtensorMap map_b, Params p) {
  extern __shared__ unsigned char smem_dyn[];
  __shared__ Shared sh;
  cg::cluster_group cluster = cg::this_cluster();
  unsigned char* tiles = smem_dyn + ((1024u - (static_cast<uint32_t>(__cvta_generic_to_shared(smem_dyn)) & 1023u)) & 1023u);
  uint16_t* assign_sm = reinterpret_cast<uint16_t*>(tiles + p.tiles_bytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = static_cast<int>(cluster.block_rank());
  const int b = blockIdx.x / p.cluster;
  const MergeParams& m = p.m;
  volatile int* abort_flag = &sh.abort_flag;
  const int stage_bytes = p.a_stage_bytes + p.b_stage_bytes;
  const int32_t* kept = m.kept + static_cast<size_t>(b) * m.n_kept;
  const int tok_begin = rank * p.rows_per_rank;                    // first token this CTA owns
  const int my_rows = max(0, min(p.rows_per_rank, m.n_tokens - tok_begin));
  const int my_tiles = (my_rows + kTileM - 1) / kTileM;

  if (threadIdx.x == 0) {
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
  // every CTA of the cluster must be running before anyone writes into its shared memory
  cluster.sync();

  if (warp == 0) {
    // ------------------------------------------------------------ producer: TMA tiles + row gathers
    const int groups = p.n_pad / 4;
    const int row_base = b * m.row_len + m.cls_offset;
    const int first = row_base + min(max(kept[0], 0), m.n_tokens - 1);
    int rows[2][4];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int g = lane + 32 * i;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int s_idx = g * 4 + j;
        rows[i][j] = (g < groups && s_idx < m.n_kept) ? row_base + min(max(kept[s_idx], 0), m.n_tokens - 1) : first;
      }
    }
    int it = 0;
    bool ok = true;
    for (int tile = 0; tile < my_tiles; ++tile) {
      const bool tail = (tile == p.tiles_per_rank - 1) && p.tail_rows != kTileM;
      const int a_bytes = tail ? p.tail_rows * 128 : p.a_stage_bytes;
      for (int kc = 0; kc < p.k_chunks; ++kc, ++it) {
        const int s = it % p.stages, round = it / p.stages;
        if (ok && round > 0) ok = mbar_wait_warp(&sh.empty[s], (round - 1) & 1, abort_flag);
        if (!ok) continue;
        unsigned char* at = tiles + s * stage_bytes;
        if (lane == 0) {
          mbar_arrive_expect_tx(&sh.full[s], a_bytes + p.n_pad * 128);
          tma_load_3d(at, tail ? &map_a_tail : &map_a, &sh.full[s], kc * kChunkK,
                      m.cls_offset + tok_begin + tile * kTileM, b);
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const int g = lane + 32 * i;
          if (g < groups)
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
      for (int tile = 0; tile < my_tiles && !*abort_flag; ++tile) {
        const int acc = tile & 1, use = tile >> 1;
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
          for (int k = 0; k < kChunkK / 16; ++k) umma_bf16(d_addr, da + 2u * k, db + 2u * k, idesc, kc > 0 || k > 0);
          umma_commit(&sh.empty[s]);
        }
        if (!ok) break;
        umma_commit(&sh.tmem_full[acc]);
      }
    }
    __syncwarp();   // the other lanes wait here, so the warp reaches the barriers below together
  } else {
    // ------------------------------------------------------------ phase 0: norms of the kept tokens
    {
      const int hw = warp - 2;   // 0..9
      const __nv_bfloat16* mb = static_cast<const __nv_bfloat16*>(m.metric) +
                                (static_cast<size_t>(b) * m.row_len + m.cls_offset) * m.metric_dim;
      const int vecs = m.metric_dim / 8;
      for (int s0 = hw * 2; s0 < m.n_kept; s0 += (kWarps - 2) * 2) {   // two rows per warp in flight
        float ss[2] = {0.f, 0.f};
        const uint4* row[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          const int s_idx = min(s0 + r, m.n_kept - 1);
          row[r] = reinterpret_cast<const uint4*>(mb + static_cast<size_t>(min(max(kept[s_idx], 0), m.n_tokens - 1)) * m.metric_dim);
        }
        for (int v = lane; v < vecs; v += 32) {
          uint4 raw[2] = {ld_nc_16(row[0] + v), ld_nc_16(row[1] + v)};
#pragma unroll
          for (int r = 0; r < 2; ++r) {
            float f[8];
            Vec16<__nv_bfloat16>::unpack(raw[r], f);
#pragma unroll
            for (int e = 0; e < 8; ++e) ss[r] = fmaf(f[e], f[e], ss[r]);
          }
        }
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          const float tot = warp_sum(ss[r]);
          if (lane == 0 && s0 + r < m.n_kept) sh.inv_norm[s0 + r] = 1.f / fmaxf(sqrtf(tot), 1e-12f);
        }
      }
      asm volatile("bar.sync 2, 320;" ::: "memory");
    }
    if (warp < 6) {
      // ---------------------------------------------------------- phase 1 epilogue: arg-max per token
      const int quarter = warp & 3;
      const int row = quarter * 32 + lane;
      bool ok = true;
      for (int tile = 0; tile < my_tiles; ++tile) {
        const int acc = tile & 1, use = tile >> 1;
        if (ok) ok = mbar_wait_warp(&sh.tmem_full[acc], use & 1, abort_flag);
        if (!ok) continue;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t taddr = tmem_acc + (static_cast<uint32_t>(quarter * 32) << 16) + acc * p.n_pad;
        float best_val = -INFINITY;
        int best_idx = 0;
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
            if (c0 + j < m.n_kept) {
              const float val = __uint_as_float(v[j]) * sh.inv_norm[c0 + j];
              if (val > best_val) { best_val = val; best_idx = c0 + j; }
            }
          }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.tmem_empty[acc]);
        const int local = tile * kTileM + row;
        if (local < my_rows) {
          const int t = tok_begin + local;
          for (int r = 0; r < p.cluster; ++r) cluster.map_shared_rank(assign_sm, r)[t] = static_cast<uint16_t>(best_idx);
        }
      }
    }
  }

  // ------------------------------------------------------------ every token of the instance has its slot
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  cluster.sync();
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(p.tmem_cols) : "memory");
  }
  const bool failed = sh.abort_flag != 0;
  if (failed && threadIdx.x == 0) atomicExch(m.status, static_cast<uint32_t>(VSCAN_ERR_TIMEOUT));
  if (failed) for (int i = 0; i < 64; ++i) __nanosleep(2000);   // let copies still in flight land

  // a kept token belongs to its own slot
  for (int s = threadIdx.x; s < m.n_kept; s += kThreads) assign_sm[min(max(kept[s], 0), m.n_tokens - 1)] = static_cast<uint16_t>(s);
  __syncthreads();
  if (m.assign && !failed)
    for (int i = threadIdx.x; i < my_rows; i += kThreads)
      m.assign[static_cast<size_t>(b) * m.n_tokens + tok_begin + i] = assign_sm[tok_begin + i];

  // ------------------------------------------------------------ phase 2: group means of slots rank, rank+C, ...
  uint32_t* list = reinterpret_cast<uint32_t*>(tiles);   // the stage ring is free now
  const int per = (m.n_tokens + kThreads - 1) / kThreads;
  const int lo = min(m.n_tokens, static_cast<int>(threadIdx.x) * per), hi = min(m.n_tokens, lo + per);
  int mine = 0;
  for (int i = lo; i < hi; ++i) mine += (assign_sm[i] % p.cluster) == rank;
  int n_list;
  int pos = block_exclusive_scan(mine, sh.warp_sums, n_list);
  for (int i = lo; i < hi; ++i) {
    const unsigned s = assign_sm[i];
    if (static_cast<int>(s % p.cluster) == rank) list[pos++] = (s << 16) | static_cast<unsigned>(i);
  }
  __syncthreads();
  if (!failed) {
    if (m.dim / 8 <= 128) group_means<4, 4>(p, list, n_list, rank, b);
    else group_means<8, 2>(p, list, n_list, rank, b);
  }
  // no CTA may exit while another one of the cluster could still write into its shared memory: all
  // such writes happened before the cluster barrier above, so leaving here is safe
}

static bool plan(const MergeParams& m, Params& p, int cluster_override) {
  p.m = m;
  p.n_pad = (m.n_kept + 15) / 16 * 16;
  if (p.n_pad > kMaxN) return false;
  p.k_chunks = (m.metric_dim + kChunkK - 1) / kChunkK;
  p.tmem_cols = 32;
  while (p.tmem_cols < 2 * p.n_pad) p.tmem_cols *= 2;
  p.a_stage_bytes = kTileM * kChunkK * 2;
  p.b_stage_bytes = ((p.n_pad * kChunkK * 2) + 1023) / 1024 * 1024;
  const int stage = p.a_stage_bytes + p.b_stage_bytes;
  const int assign_bytes = (m.n_tokens * 2 + 15) / 16 * 16;
  int stages = (205 * 1024 - assign_bytes) / stage;
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages < 2) return false;
  p.stages = stages;
  p.tiles_bytes = stages * stage;
  if (static_cast<size_t>(m.n_tokens) * 4 > static_cast<size_t>(p.tiles_bytes)) return false;  // phase-2 list
  // two CTAs per instance once an instance has more than two tiles: halves the instances in flight
  p.cluster = cluster_override > 0 ? cluster_override : (m.n_tokens > 2 * kTileM ? 2 : 1);
  p.rows_per_rank = ((m.n_tokens + p.cluster - 1) / p.cluster + 7) / 8 * 8;
  p.tiles_per_rank = (p.rows_per_rank + kTileM - 1) / kTileM;
  p.tail_rows = p.rows_per_rank - (p.tiles_per_rank - 1) * kTileM;
  return true;
}

}  // namespace fused

bool merge_fused_supported(int dtype, const MergeParams& m) {
  if (dtype != VSCAN_BF16 || m.metric_dim % 8 != 0 || m.dim % 8 != 0 || m.n_kept < 1) return false;
  if (m.n_tokens > fused::kMaxTokens || m.n_kept > tc::kMaxN) return false;
  if ((reinterpret_cast<uintptr_t>(m.metric) & 15u) != 0) return false;
  fused::Params p;
  return fused::plan(m, p, 0) && tc::encode_fn() != nullptr;
}

vscan_status launch_merge_fused(const MergeParams& m, cudaStream_t stream) {
  fused::Params p;
  if (!fused::plan(m, p, 0)) return VSCAN_ERR_UNSUPPORTED;
  tc::EncodeTiledFn encode = tc::encode_fn();
  if (!encode) return VSCAN_ERR_UNSUPPORTED;
  CUtensorMap map_a, map_tail, map_b;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(m.metric_dim), static_cast<cuuint64_t>(m.row_len),
                              static_cast<cuuint64_t>(m.instances)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(m.metric_dim) * 2,
                                 static_cast<cuuint64_t>(m.row_len) * m.metric_dim * 2};
  const cuuint32_t elem[3] = {1, 1, 1};
  const cuuint32_t box[3] = {tc::kChunkK, tc::kTileM, 1};
  const cuuint32_t box_tail[3] = {tc::kChunkK, static_cast<cuuint32_t>(p.tail_rows), 1};
  void* base = const_cast<void*>(m.metric);
  if (encode(&map_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
      encode(&map_tail, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box_tail, elem,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return VSCAN_ERR_UNSUPPORTED;
  const cuuint64_t dims_b[2] = {static_cast<cuuint64_t>(m.metric_dim),
                                static_cast<cuuint64_t>(m.row_len) * static_cast<cuuint64_t>(m.instances)};
  const cuuint64_t strides_b[1] = {static_cast<cuuint64_t>(m.metric_dim) * 2};
  const cuuint32_t box_b[2] = {tc::kChunkK, 1};
  if (encode(&map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims_b, strides_b, box_b, elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return VSCAN_ERR_UNSUPPORTED;

  const size_t smem = static_cast<size_t>(p.tiles_bytes) + 1024 + (static_cast<size_t>(m.n_tokens) * 2 + 15) / 16 * 16;
  VSCAN_CUDA_TRY(allow_smem(fused::merge_fused_kernel, smem));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(m.instances) * p.cluster);
  cfg.blockDim = dim3(fused::kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = p.cluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  VSCAN_LAUNCH("merge_fused", stream, (void)cudaLaunchKernelEx(&cfg, fused::merge_fused_kernel, map_a, map_tail, map_b, p));
  return VSCAN_OK;
}

}  // namespace vscan
