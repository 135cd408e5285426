// Group sums of the merge step (Eq. 4) on the tensor cores.  With P the one-hot assignment matrix
// (P[s][t] = 1 iff token t belongs to kept slot s; a kept token belongs to its own slot), the sums of Eq. 4 are
// the product P . X, so the second pass over the features is a plain stream of TMA tile loads feeding
// tcgen05 MMAs: no member lists, no chains of dependent row loads.
//
// Persistent kernel, one CTA per SM.  A work item is (instance, slice of 128 or 256 feature columns); CTA c takes
// items c, c + grid, ...; its roles run through the items without stopping, so the loads of the next item are in
// flight while the sums of the current one are read back.  Per tile of 64 tokens:
//   warp 0      TMA producer: the tile's [64 tokens x 64 columns] boxes of the slice (128B swizzle)
//   warps 2-3   fill the one-hot tiles (slots x tokens, bf16, K-major, 128B swizzle), each for every other token
//               tile: a lane sets the entries of its two tokens and counts the groups
//   warp 1      MMA issuer: acc[slots x columns] += P_tile . X_tile; P^T... the one-hot tile is the K-major A operand
//               (M = 64 or 128 slots, K = tokens), the token tile the B operand read "MN-major" (its columns,
//               contiguous in shared memory, are the N dimension; the tokens are K): one MMA covers all columns of
//               the slice; fp32 accumulators in tensor memory, two sets that alternate between items
//   warps 4-7   per item: accumulator (one slot per thread) -> x 1/count -> bf16 -> 16-byte stores of merged rows
// Every mbarrier wait is bounded; on expiry the CTA records VSCAN_ERR_TIMEOUT, lets copies in flight land,
// frees its tensor memory and returns.
#include "merge.cuh"
#include "tc_common.cuh"

namespace vscan {
namespace tcsum {

using namespace tc;

constexpr int kThreads = 256;
constexpr int kTileTokens = 64;          // tokens per stage: four MMAs of K = 16
constexpr int kBoxBytes = kTileTokens * 128;   // one [64 tokens x 64 columns] box
constexpr int kMaxStagesSum = 6;
constexpr int kOneHots = 4;              // one-hot tiles in rotation: the builders run up to four token tiles ahead of the MMAs

struct Params {
  MergeParams m;
  int n_pad;        // rows of the accumulator: 64 or 128 (MMA M), >= n_kept
  int tiles;        // token tiles per instance
  int m_tiles;      // 128-column halves of a slice (1 or 2): MMA N = 128 * m_tiles
  int stages;
  int tmem_cols;    // two accumulator sets of 128 * m_tiles columns
  int slices;       // column slices per instance
  int items;        // instances * slices
};

struct Shared {
  uint64_t full[kMaxStagesSum];    // the boxes of the stage have landed
  uint64_t empty[kMaxStagesSum];   // the MMAs that read the stage have completed
  uint64_t p_full[kOneHots];       // one-hot tile written
  uint64_t p_empty[kOneHots];      // the MMAs that read the one-hot tile have completed
  uint64_t acc_full[2];            // all MMAs of an item have completed (accumulator set 0 / 1)
  uint64_t acc_empty[2];           // the read-back warps are done with that set and its counts
  uint32_t tmem_base;
  int abort_flag;
  int counts[2][kMaxN];
  float inv_count[2][kMaxN];
};

// Shared-memory matrix descriptor of an MN-major operand with 128-byte swizzle: 64 elements of M are contiguous
// (one 128-byte row per K index), 8 K indices form a 1024-byte group; `lbo` is the distance between blocks of
// 64 M elements, 1024 bytes the distance between groups of 8 K indices.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t smem_addr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= 1ull << 46;
  d |= 2ull << 61;
  return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, A K-major, B MN-major, M = m, N = n.
__device__ __forceinline__ uint32_t instr_desc_bf16_bmn(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(m >> 4) << 24);
}

// Byte offset of element (slot s, token j) of a one-hot tile: rows of 128 bytes, 16-byte chunks swizzled with
// the row index (the layout the K-major descriptor of tc_common.cuh describes).
__device__ __forceinline__ uint32_t onehot_offset(int s, int j) {
  return static_cast<uint32_t>(s) * 128u + (((static_cast<uint32_t>(j) >> 3) ^ (static_cast<uint32_t>(s) & 7u)) << 4) +
         ((static_cast<uint32_t>(j) & 7u) << 1);
}

__global__ void __launch_bounds__(kThreads, 1) group_sum_tensor_kernel(const __grid_constant__ CUtensorMap map_x, Params p) {
  extern __shared__ unsigned char smem_dyn[];
  __shared__ Shared sh;
  unsigned char* base = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const MergeParams& m = p.m;
  const int stage_bytes = p.m_tiles * 2 * kBoxBytes;
  unsigned char* onehot = base + p.stages * stage_bytes;           // kOneHots tiles of n_pad x 128 bytes
  const int onehot_bytes = p.n_pad * 128;
  const int acc_cols = p.m_tiles * 128;                            // columns of one accumulator set
  volatile int* abort_flag = &sh.abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
    for (int a = 0; a < kOneHots; ++a) { mbar_init(&sh.p_full[a], 1); mbar_init(&sh.p_empty[a], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&sh.acc_full[a], 1); mbar_init(&sh.acc_empty[a], 4); }
    sh.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)), "r"(p.tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // the one-hot tiles and both sets of counts start all zero
  for (int i = threadIdx.x; i < kOneHots * onehot_bytes / 16; i += kThreads) reinterpret_cast<uint4*>(onehot)[i] = make_uint4(0u, 0u, 0u, 0u);
  for (int i = threadIdx.x; i < 2 * kMaxN; i += kThreads) (&sh.counts[0][0])[i] = 0;
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = sh.tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------ producer (the features are an input of the call:
    // their loads need not wait for the kernel before this one)
    // Items run from the LAST instance to the first: the assignment pass before this kernel read the instances in
    // ascending order, so the last ones are the part of the features that is still in L2.
    bool ok = true;
    int s = 0, it = 0;       // ring position as counters: no division per tile
    uint32_t phase = 0;
    for (int w = blockIdx.x; w < p.items && ok; w += gridDim.x) {
      const int b = m.instances - 1 - w / p.slices, col0 = (w - (w / p.slices) * p.slices) * p.m_tiles * 128;
      const int boxes = min(p.m_tiles, (m.dim - col0) / 128) * 2;
      for (int t = 0; t < p.tiles && ok; ++t, ++it) {
        if (it >= p.stages) ok = mbar_wait_warp(&sh.empty[s], phase ^ 1u, abort_flag);
        if (!ok) break;
        unsigned char* st = base + s * stage_bytes;
        if (lane == 0) mbar_arrive_expect_tx(&sh.full[s], boxes * kBoxBytes);
        __syncwarp();
        if (lane < boxes)    // one box per lane, issued by one instruction
          tma_load_3d(st + lane * kBoxBytes, &map_x, &sh.full[s], col0 + lane * 64, m.cls_offset + t * kTileTokens, b);
        if (++s == p.stages) { s = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = true;
      int it = 0, i = 0, s = 0;
      uint32_t phase = 0;
      const uint32_t base_addr = smem_u32(base), onehot_addr = smem_u32(onehot);
      for (int w = blockIdx.x; w < p.items && ok && !*abort_flag; w += gridDim.x, ++i) {
        const int col0 = (w % p.slices) * p.m_tiles * 128;
        const int my_tiles = min(p.m_tiles, (m.dim - col0) / 128);
        const uint32_t idesc = instr_desc_bf16_bmn(p.n_pad, my_tiles * 128);
        const int acc = i & 1, use = i >> 1;
        if (use > 0) {   // the read-back of the item that used this accumulator set before
          if (!mbar_wait(&sh.acc_empty[acc], (use - 1) & 1, abort_flag)) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        }
        for (int t = 0; t < p.tiles; ++t, ++it) {
          const int pb = it % kOneHots;
          if (!mbar_wait(&sh.full[s], phase, abort_flag) || !mbar_wait(&sh.p_full[pb], (it / kOneHots) & 1, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t st_addr = base_addr + s * stage_bytes;
          const uint64_t da = smem_desc_sw128(onehot_addr + pb * onehot_bytes);
#pragma unroll
          for (int k = 0; k < kTileTokens / 16; ++k) {   // 16 tokens = 32 bytes of a one-hot row, two 1024-byte groups of the token tile
            const uint64_t db = smem_desc_mn_sw128(st_addr + k * 2048, kBoxBytes);
            umma_bf16(tmem_acc + acc * acc_cols, da + 2u * k, db, idesc, t > 0 || k > 0);
          }
          umma_commit(&sh.empty[s]);
          umma_commit(&sh.p_empty[pb]);
          if (++s == p.stages) { s = 0; phase ^= 1u; }
        }
        if (ok) umma_commit(&sh.acc_full[acc]);
      }
    }
    __syncwarp();
  } else if (warp < 4) {
    // ------------------------------------------------------------ one-hot builders: warp 2 takes the even token tiles
    // of the CTA's tile sequence, warp 3 the odd ones; tile number `it` goes to one-hot tile it % kOneHots; a lane
    // owns token columns lane and lane + 32.  The assignments of a warp's next tile are loaded before it waits.
    const int par = warp - 2;
    grid_dependency_wait();                      // the assignments come from the kernel before this one
    static_assert(kOneHots == 4, "a builder warp keeps the previous slots of two one-hot tiles in registers");
    int pa0 = -1, pa1 = -1, pb0 = -1, pb1 = -1;  // the slots the lane's two columns hold in each of the warp's two tiles
    bool ok = true;
    // position of the warp's current tile: item w (the i-th of this CTA), token tile t, tile number it
    int w = blockIdx.x, i = 0, t = par, it = par;
    auto normalise = [&]() { while (w < p.items && t >= p.tiles) { t -= p.tiles; w += gridDim.x; ++i; } };
    auto load = [&](int ww, int tt, int& a0, int& a1) {
      a0 = -1; a1 = -1;
      if (ww >= p.items) return;
      const int32_t* ag = m.assign + static_cast<size_t>(m.instances - 1 - ww / p.slices) * m.n_tokens;
      const int tok0 = tt * kTileTokens + lane, tok1 = tok0 + 32;
      if (tok0 < m.n_tokens) a0 = __ldcg(ag + tok0);   // raw values: nothing here waits for the loads
      if (tok1 < m.n_tokens) a1 = __ldcg(ag + tok1);
    };
    normalise();
    int a0, a1;
    load(w, t, a0, a1);
    while (w < p.items) {
      const int cw = w, ci = i, ct = t, cit = it;
      t += 2; it += 2;
      normalise();
      int n0, n1;
      load(w, t, n0, n1);                        // in flight during the waits below
      const int pb = cit % kOneHots, use = cit / kOneHots;
      // first tile of an item that reuses a set of counts: the read-back of the earlier item has taken them
      if (ok && (ci >> 1) > 0 && ct < 2) ok = mbar_wait_warp(&sh.acc_empty[ci & 1], ((ci >> 1) - 1) & 1, abort_flag);
      if (ok && use > 0) ok = mbar_wait_warp(&sh.p_empty[pb], (use - 1) & 1, abort_flag);
      a0 = min(a0, m.n_kept - 1); a1 = min(a1, m.n_kept - 1);   // assignments are the library's own; never index past the tile all the same
      if (ok) {
        unsigned char* tile = onehot + pb * onehot_bytes;
        int* counts = sh.counts[ci & 1];
        int& p0 = (pb >> 1) ? pb0 : pa0;
        int& p1 = (pb >> 1) ? pb1 : pa1;
        if (p0 >= 0) *reinterpret_cast<uint16_t*>(tile + onehot_offset(p0, lane)) = 0u;
        if (p1 >= 0) *reinterpret_cast<uint16_t*>(tile + onehot_offset(p1, lane + 32)) = 0u;
        if (a0 >= 0) { *reinterpret_cast<uint16_t*>(tile + onehot_offset(a0, lane)) = 0x3F80u; atomicAdd(&counts[a0], 1); }   // bf16 1.0
        if (a1 >= 0) { *reinterpret_cast<uint16_t*>(tile + onehot_offset(a1, lane + 32)) = 0x3F80u; atomicAdd(&counts[a1], 1); }
        p0 = a0; p1 = a1;
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0 && ok) mbar_arrive(&sh.p_full[pb]);
      a0 = n0; a1 = n1;
      (void)cw;
    }
  } else {
    // ------------------------------------------------------------ read-back (warps 4-7)
    const int tid4 = threadIdx.x - 128;          // 0..127
    const int quarter = warp & 3;
    bool ok = true;
    int i = 0;
    for (int w = blockIdx.x; w < p.items; w += gridDim.x, ++i) {
      const int b = m.instances - 1 - w / p.slices, slice = w - (w / p.slices) * p.slices, col0 = slice * p.m_tiles * 128;
      const int my_tiles = min(p.m_tiles, (m.dim - col0) / 128);
      const int acc = i & 1;
      if (ok) ok = mbar_wait_warp(&sh.acc_full[acc], (i >> 1) & 1, abort_flag);
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      // all one-hot tiles of the item have been consumed, so the builders' counts are final
      for (int s = tid4; s < p.n_pad; s += 128) {
        const int c = sh.counts[acc][s];
        sh.inv_count[acc][s] = 1.f / static_cast<float>(max(c, 1));
        if (slice == 0 && m.counts && s < m.n_kept && ok) m.counts[static_cast<size_t>(b) * m.n_kept + s] = c;
        sh.counts[acc][s] = 0;
      }
      asm volatile("bar.sync 2, 128;" ::: "memory");
      if (ok) {
        // accumulator rows: with M = 128 row r sits in lane r; with M = 64 row r sits in lane 32 * (r / 16) + r % 16
        const int slot = p.n_pad == 128 ? quarter * 32 + lane : quarter * 16 + lane;
        const bool mine = (p.n_pad == 128 || lane < 16) && slot < m.n_kept;
        const float inv = mine ? sh.inv_count[acc][slot] : 0.f;
        uint4* out = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(m.merged) +
                                              (static_cast<size_t>(b) * m.n_kept + (mine ? slot : 0)) * m.dim + col0);
        const uint32_t taddr = tmem_acc + (static_cast<uint32_t>(quarter * 32) << 16) + acc * acc_cols;
        for (int c0 = 0; c0 < my_tiles * 128; c0 += 32) {
          uint32_t v[32];
          tmem_ld32(taddr + c0, v);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          if (mine) {
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
              float f[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[q4 * 8 + e]) * inv;
              st_16(out + c0 / 8 + q4, Vec16<__nv_bfloat16>::pack(f));
            }
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0 && ok) mbar_arrive(&sh.acc_empty[acc]);
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

// (Kept sets of 129-256 as two halves of 128 slots, 128 columns per item, were measured slower than the CUDA-core
// group means: 96 against 79 us for 256 instances with 192 kept tokens.)
static bool plan(const MergeParams& m, Params& p) {
  if (m.dim % 128 != 0 || m.n_kept < 1 || m.n_kept > 128) return false;
  if (m.row_len != m.cls_offset + m.n_tokens) return false;   // rows past the last token must be the copy's zero fill
  if ((reinterpret_cast<uintptr_t>(m.x) & 15u) != 0 || (reinterpret_cast<uintptr_t>(m.merged) & 15u) != 0) return false;
  p.m = m;
  p.n_pad = m.n_kept <= 64 ? 64 : 128;
  p.tiles = (m.n_tokens + kTileTokens - 1) / kTileTokens;
  p.m_tiles = m.dim % 256 == 0 ? 2 : 1;
  p.stages = 4;
  p.slices = (m.dim + p.m_tiles * 128 - 1) / (p.m_tiles * 128);
  const long long items = 1ll * m.instances * p.slices;
  if (items > 0x3fffffffLL) return false;
  p.items = static_cast<int>(items);
  p.tmem_cols = 2 * p.m_tiles * 128;
  return true;
}

static size_t smem_bytes(const Params& p) {
  return 1024 + static_cast<size_t>(p.stages) * p.m_tiles * 2 * kBoxBytes + kOneHots * static_cast<size_t>(p.n_pad) * 128;
}

}  // namespace tcsum

bool group_sum_tensor_supported(int dtype, const MergeParams& m) {
  tcsum::Params p;
  return dtype == VSCAN_BF16 && tcsum::plan(m, p) && tc::encode_fn() != nullptr;
}

vscan_status launch_group_sum_tensor(const MergeParams& m, cudaStream_t stream) {
  tcsum::Params p;
  if (!tcsum::plan(m, p)) return VSCAN_ERR_UNSUPPORTED;
  tc::EncodeTiledFn encode = tc::encode_fn();
  if (!encode) return VSCAN_ERR_UNSUPPORTED;
  CUtensorMap map;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(m.dim), static_cast<cuuint64_t>(m.row_len), static_cast<cuuint64_t>(m.instances)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(m.dim) * 2, static_cast<cuuint64_t>(m.row_len) * m.dim * 2};
  const cuuint32_t box[3] = {64, tcsum::kTileTokens, 1};
  const cuuint32_t elem[3] = {1, 1, 1};
  if (encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(m.x), dims, strides, box, elem,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return VSCAN_ERR_UNSUPPORTED;
  const size_t smem = tcsum::smem_bytes(p);
  VSCAN_CUDA_TRY(allow_smem(tcsum::group_sum_tensor_kernel, smem));
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
  const unsigned blocks = static_cast<unsigned>(p.items < sms ? p.items : sms);
  VSCAN_LAUNCH("group_mean", stream,
               (void)launch_dependent(tcsum::group_sum_tensor_kernel, dim3(blocks), dim3(tcsum::kThreads), smem, stream, map, p));
  return VSCAN_OK;
}

}  // namespace vscan
