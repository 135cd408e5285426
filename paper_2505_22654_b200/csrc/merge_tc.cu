// Tensor-core path of the merge assignment (Sec. 4.1 "Token Merging"): for a tile of 128 tokens the
// dot products with all kept tokens are one tcgen05 MMA chain, D[128 x Nk] (fp32, tensor memory) =
// A[128 tokens x dim] * B[Nk kept x dim]^T with bf16 operands in shared memory.
//   warp 0      TMA producer of the token tile (3-D tensor map over [instance][row][dim], 128B swizzle)
//   warp 1      allocates tensor memory, issues the MMAs (one elected lane), commits to mbarriers
//   warps 2-5   gather the kept rows into the swizzled B stage (kept rows are not contiguous), then
//               read the accumulator back (tcgen05.ld, one token row per thread), scale by 1/|m_s|
//               and keep the running arg-max (lowest slot on ties)
// The similarity matrix never leaves the SM.  Every mbarrier wait is bounded: on expiry the CTA
// records VSCAN_ERR_TIMEOUT in the status word, lets copies in flight land, frees its tensor memory
// and returns.
#include <cuda.h>

#include <mutex>

#include "merge.cuh"

namespace vscan {

namespace tc {

constexpr int kTileM = 128;        // tokens per CTA (UMMA M)
constexpr int kChunkK = 64;        // bf16 elements per k-chunk = one 128-byte swizzle row
constexpr int kMaxN = 256;         // kept tokens per MMA (UMMA N limit)
constexpr int kThreads = 192;
constexpr int kMaxStages = 8;
constexpr uint32_t kSpinLimit = 1u << 20;   // try_wait polls before a wait gives up (well under a second)

struct Params {
  MergeParams m;
  int n_pad;        // kept columns per n-chunk, multiple of 16, <= 256
  int n_chunks;     // ceil(n_kept / n_pad)
  int k_chunks;     // ceil(metric_dim / 64)
  int stages;
  int tmem_cols;    // power of two >= max(32, n_pad)
  int a_stage_bytes, b_stage_bytes;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the limit ran out or another role of this CTA gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 1023u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

// Same, called by a whole warp: every lane gets the same answer, so the warp stays converged.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  const bool r = mbar_wait(bar, parity, abort_flag);
  return __all_sync(0xffffffffu, r);
}

__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);   // start address, 16-byte units
  d |= 1ull << 16;                                            // leading byte offset (unused for this layout)
  d |= static_cast<uint64_t>(1024 >> 4) << 32;                // stride byte offset between 8-row groups
  d |= 1ull << 46;                                            // descriptor version for this architecture
  d |= 2ull << 61;                                            // 128-byte swizzle
  return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t instr_desc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(kTileM >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(static_cast<uint32_t>(accumulate))
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}

struct Shared {
  uint64_t full[kMaxStages];    // A landed (tx bytes) and B gathered (4 warp arrivals)
  uint64_t empty[kMaxStages];   // MMAs that read the stage have completed
  uint64_t tmem_full;           // accumulator of the current n-chunk complete
  uint64_t tmem_empty;          // epilogue has read the accumulator
  uint32_t tmem_base;
  int abort_flag;
  int best_slot[kTileM];
  float inv_norm[kMaxN];
  int kept_row[kMaxN];
};

// dynamic shared memory (1024-byte aligned): stages x [A tile 128x64 bf16 | B tile n_pad x 64 bf16]
__global__ void __launch_bounds__(kThreads) assign_tensor_kernel(const __grid_constant__ CUtensorMap map_a, Params p) {
  extern __shared__ unsigned char smem_dyn[];
  __shared__ Shared sh;
  // the swizzle pattern is a function of the shared-memory address: stage bases sit on 1024 bytes
  unsigned char* tiles = smem_dyn + ((1024u - (static_cast<uint32_t>(__cvta_generic_to_shared(smem_dyn)) & 1023u)) & 1023u);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.y, t0 = blockIdx.x * kTileM;
  const MergeParams& m = p.m;
  volatile int* abort_flag = &sh.abort_flag;
  const int stage_bytes = p.a_stage_bytes + p.b_stage_bytes;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(&sh.full[s], 5); mbar_init(&sh.empty[s], 1); }
    mbar_init(&sh.tmem_full, 1);
    mbar_init(&sh.tmem_empty, 4);
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

  if (warp == 0) {
    // ------------------------------------------------------------ token tile producer (TMA)
    if (lane == 0) {
      int it = 0;
      for (int nc = 0; nc < p.n_chunks && !*abort_flag; ++nc) {
        for (int kc = 0; kc < p.k_chunks; ++kc, ++it) {
          const int s = it % p.stages, round = it / p.stages;
          if (round > 0 && !mbar_wait(&sh.empty[s], (round - 1) & 1, abort_flag)) break;
          mbar_arrive_expect_tx(&sh.full[s], p.a_stage_bytes);
          tma_load_3d(tiles + s * stage_bytes, &map_a, &sh.full[s], kc * kChunkK, m.cls_offset + t0, b);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = instr_desc_bf16(p.n_pad);
      int it = 0;
      for (int nc = 0; nc < p.n_chunks && !*abort_flag; ++nc) {
        if (nc > 0) {
          if (!mbar_wait(&sh.tmem_empty, (nc - 1) & 1, abort_flag)) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        }
        bool ok = true;
        for (int kc = 0; kc < p.k_chunks; ++kc, ++it) {
          const int s = it % p.stages, round = it / p.stages;
          if (!mbar_wait(&sh.full[s], round & 1, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = smem_u32(tiles + s * stage_bytes), b_addr = a_addr + p.a_stage_bytes;
          const uint64_t da = smem_desc_sw128(a_addr), db = smem_desc_sw128(b_addr);
#pragma unroll
          for (int k = 0; k < kChunkK / 16; ++k)   // 16 bf16 = 32 bytes per MMA along K: +2 in 16-byte units
            umma_bf16(tmem_acc, da + 2u * k, db + 2u * k, idesc, kc > 0 || k > 0);
          umma_commit(&sh.empty[s]);
        }
        if (!ok) break;
        umma_commit(&sh.tmem_full);
      }
    }
  } else {
    // ------------------------------------------------------------ kept-row gather, then epilogue
    const int pw = warp - 2;                  // 0..3
    const int ptid = pw * 32 + lane;          // 0..127
    const int quarter = warp & 3;             // tensor-memory lanes this warp may read
    const int row = quarter * 32 + lane;      // token row of this thread within the tile
    const __nv_bfloat16* mb = static_cast<const __nv_bfloat16*>(m.metric) +
                              (static_cast<size_t>(b) * m.row_len + m.cls_offset) * m.metric_dim;
    const int32_t* kept = m.kept + static_cast<size_t>(b) * m.n_kept;
    float best_val = -INFINITY;
    int best_idx = 0;
    int it = 0;
    bool ok = true;
    // Once `ok` drops the loops keep running with their work skipped, so that the four warps execute
    // the same sequence of named barriers and warp-wide instructions whatever happens.
    for (int nc = 0; nc < p.n_chunks; ++nc) {
      const int n0 = nc * p.n_pad;
      // stage the kept rows and scales of this n-chunk (only these four warps touch them)
      asm volatile("bar.sync 1, 128;" ::: "memory");
      for (int j = ptid; j < p.n_pad; j += 128) {
        const int s_idx = n0 + j;
        sh.kept_row[j] = s_idx < m.n_kept ? min(max(kept[s_idx], 0), m.n_tokens - 1) : -1;
        sh.inv_norm[j] = s_idx < m.n_kept ? m.inv_norm[static_cast<size_t>(b) * m.n_kept + s_idx] : 0.f;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      const int chunks = p.n_pad * 8;          // 16-byte pieces per B stage
      for (int kc = 0; kc < p.k_chunks; ++kc, ++it) {
        const int s = it % p.stages, round = it / p.stages;
        if (ok && round > 0) ok = mbar_wait_warp(&sh.empty[s], (round - 1) & 1, abort_flag);
        if (!ok) continue;
        unsigned char* bt = tiles + s * stage_bytes + p.a_stage_bytes;
        const int col0 = kc * kChunkK;
        for (int c0 = ptid; c0 < chunks; c0 += 128 * 4) {
          uint4 v[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int c = c0 + u * 128;
            v[u] = make_uint4(0u, 0u, 0u, 0u);
            if (c < chunks) {
              const int r = c >> 3, piece = c & 7, tk = sh.kept_row[r], col = col0 + piece * 8;
              if (tk >= 0 && col < m.metric_dim) v[u] = ld_nc_16(mb + static_cast<size_t>(tk) * m.metric_dim + col);
            }
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int c = c0 + u * 128;
            if (c < chunks) {
              const int r = c >> 3, piece = c & 7;
              *reinterpret_cast<uint4*>(bt + r * 128 + ((piece ^ (r & 7)) << 4)) = v[u];
            }
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // make the stores visible to the MMA
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.full[s]);
      }
      // accumulator of this n-chunk -> running arg-max of this thread's token row
      if (ok) ok = mbar_wait_warp(&sh.tmem_full, nc & 1, abort_flag);
      if (!ok) continue;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t taddr = tmem_acc + (static_cast<uint32_t>(quarter * 32) << 16);
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
            const float val = __uint_as_float(v[j]) * sh.inv_norm[c0 + j];
            if (val > best_val) { best_val = val; best_idx = s_idx; }
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.tmem_empty);
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

// ---------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static std::once_flag once;
  static EncodeTiledFn fn = nullptr;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  });
  return fn;
}

static bool plan(const MergeParams& m, Params& p) {
  p.m = m;
  const int n16 = (m.n_kept + 15) / 16 * 16;
  p.n_pad = n16 <= kMaxN ? n16 : kMaxN;
  p.n_chunks = (m.n_kept + p.n_pad - 1) / p.n_pad;
  p.k_chunks = (m.metric_dim + kChunkK - 1) / kChunkK;
  p.tmem_cols = 32;
  while (p.tmem_cols < p.n_pad) p.tmem_cols *= 2;
  p.a_stage_bytes = kTileM * kChunkK * 2;
  p.b_stage_bytes = ((p.n_pad * kChunkK * 2) + 1023) / 1024 * 1024;
  const int stage = p.a_stage_bytes + p.b_stage_bytes;
  // two CTAs per SM when four stages fit in half the shared memory, else as many stages as fit
  int stages = (110 * 1024) / stage;
  if (stages < 3) stages = (215 * 1024) / stage;
  if (stages > kMaxStages) stages = kMaxStages;
  if (stages > 4 && (110 * 1024) / stage >= 4) stages = 4;
  p.stages = stages;
  return stages >= 2;
}

}  // namespace tc

bool assign_tensor_supported(int dtype, const MergeParams& m) {
  if (dtype != VSCAN_BF16 || m.metric_dim % 8 != 0 || m.n_kept < 1) return false;
  if ((reinterpret_cast<uintptr_t>(m.metric) & 15u) != 0) return false;
  tc::Params p;
  return tc::plan(m, p) && tc::encode_fn() != nullptr;
}

vscan_status launch_assign_tensor(const MergeParams& m, cudaStream_t stream) {
  tc::Params p;
  if (!tc::plan(m, p)) return VSCAN_ERR_UNSUPPORTED;
  tc::EncodeTiledFn encode = tc::encode_fn();
  if (!encode) return VSCAN_ERR_UNSUPPORTED;
  CUtensorMap map;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(m.metric_dim), static_cast<cuuint64_t>(m.row_len),
                              static_cast<cuuint64_t>(m.instances)};
  const cuuint64_t strides[2] = {static_cast<cuuint64_t>(m.metric_dim) * 2,
                                 static_cast<cuuint64_t>(m.row_len) * m.metric_dim * 2};
  const cuuint32_t box[3] = {tc::kChunkK, tc::kTileM, 1};
  const cuuint32_t elem[3] = {1, 1, 1};
  CUresult r = encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(m.metric), dims, strides, box,
                      elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                      CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return VSCAN_ERR_UNSUPPORTED;
  const size_t smem = static_cast<size_t>(p.stages) * (p.a_stage_bytes + p.b_stage_bytes) + 1024;
  VSCAN_CUDA_TRY(allow_smem(tc::assign_tensor_kernel, smem));
  dim3 grid((m.n_tokens + tc::kTileM - 1) / tc::kTileM, m.instances);
  VSCAN_LAUNCH("assign_tensor", stream, tc::assign_tensor_kernel<<<grid, tc::kThreads, smem, stream>>>(map, p));
  return VSCAN_OK;
}

}  // namespace vscan
