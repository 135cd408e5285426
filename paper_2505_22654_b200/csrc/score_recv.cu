// Score source for encoders without a [CLS] token (Sec. 4.1, text after Eq. 2): for every head h, the average
// attention each token receives from the other tokens, r_h[j] = (1 / (N - 1)) * sum_{i != j} P_h[i][j] with
// P_h = softmax_rows(scale * Q_h K_h^T), computed from Q and K without ever holding the N x N matrix.
//
// Two passes of one kernel over 128 x 128 blocks of the score matrix, both as tcgen05 MMAs with a 128-row tile
// resident in shared memory (A operand) and 128-row tiles of the other tensor streamed through a TMA ring (B operand),
// fp32 blocks in tensor memory (two, alternating), one thread per block row in the read-back:
//   pass 1  A = 128 queries, B = all key tiles: running row maximum and row sum of exponentials (base 2) ->
//           lse2[i] = max_j t_ij + log2 sum_j 2^(t_ij - max), t = scale * log2(e) * q_i . k_j
//   pass 2  A = 128 keys, B = all query tiles (with their 128 lse2 values, a 512-byte bulk copy into the stage):
//           column sums c_j = sum_{i != j} 2^(t_ij - lse2[i]) accumulate in the thread that owns key j
// The head mean of the rows r_h is then the ROW-mode score kernel (Eq. 2).
// Every mbarrier wait is bounded; on expiry the CTA records VSCAN_ERR_TIMEOUT, lets copies in flight land, frees
// its tensor memory and returns.
#include "score.cuh"
#include "tc_common.cuh"

namespace vscan {
namespace recv {

using namespace tc;

constexpr int kThreads = 320;   // warp 0 TMA, warp 1 MMA, warps 2-9 read-back: two warps per quarter of the block rows, 64 columns each
constexpr int kTile = 128;      // rows of the resident tile (MMA M) and of a streamed tile (MMA N)
constexpr int kChunkBytes = kTile * 128;   // one [128 rows x 64 elements] box

struct Params {
  float* lse2;         // [instances * heads][n_pad]  written by pass 1, read by pass 2
  float* rows;         // [instances * heads][n]      written by pass 2
  uint32_t* status;
  int n, n_pad, k_chunks, stages, tiles, pass;
  float scale_log2e;
};

struct Shared {
  uint64_t a_full;
  uint64_t full[kMaxStages], empty[kMaxStages];
  uint64_t tmem_full[2], tmem_empty[2];
  uint32_t tmem_base;
  int abort_flag;
  float part_a[kTile], part_b[kTile];   // the second column half's (maximum, sum) or column sum of every block row
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// map_a: the tensor whose 128-row tile stays resident (queries in pass 1, keys in pass 2); map_b: the streamed one.
__global__ void __launch_bounds__(kThreads) received_kernel(const __grid_constant__ CUtensorMap map_a,
                                                            const __grid_constant__ CUtensorMap map_b, Params p) {
  extern __shared__ unsigned char smem_dyn[];
  __shared__ Shared sh;
  unsigned char* base = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row0 = blockIdx.x * kTile, bh = blockIdx.y;
  const int tile_bytes = p.k_chunks * kChunkBytes;
  unsigned char* a_tile = base;
  unsigned char* ring = base + tile_bytes;            // the streamed tiles, each on a 1024-byte boundary
  unsigned char* lse_ring = ring + p.stages * tile_bytes;   // per stage: the lse2 values of the tile's 128 rows (pass 2)
  volatile int* abort_flag = &sh.abort_flag;

  if (threadIdx.x == 0) {
    mbar_init(&sh.a_full, 1);
    // a stage is released by the MMAs that read it (pass 1) or by the eight read-back warps, which read its lse2
    // values after those MMAs have completed (pass 2)
    for (int s = 0; s < p.stages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], p.pass == 2 ? 8 : 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&sh.tmem_full[a], 1); mbar_init(&sh.tmem_empty[a], 8); }
    sh.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)), "n"(256) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = sh.tmem_base;
  grid_dependency_wait();   // pass 2 reads what pass 1 wrote

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      mbar_arrive_expect_tx(&sh.a_full, tile_bytes);
      for (int kc = 0; kc < p.k_chunks; ++kc) tma_load_3d(a_tile + kc * kChunkBytes, &map_a, &sh.a_full, kc * 64, row0, bh);
    }
    bool ok = true;
    for (int t = 0; t < p.tiles && ok; ++t) {
      const int s = t % p.stages, round = t / p.stages;
      if (round > 0) ok = mbar_wait_warp(&sh.empty[s], (round - 1) & 1, abort_flag);
      if (!ok) break;
      if (lane == 0) {
        unsigned char* st = ring + s * tile_bytes;
        mbar_arrive_expect_tx(&sh.full[s], tile_bytes + (p.pass == 2 ? 512 : 0));
        for (int kc = 0; kc < p.k_chunks; ++kc) tma_load_3d(st + kc * kChunkBytes, &map_b, &sh.full[s], kc * 64, t * kTile, bh);
        if (p.pass == 2) bulk_load(lse_ring + s * 512, p.lse2 + static_cast<size_t>(bh) * p.n_pad + t * kTile, 512, &sh.full[s]);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer: block[128 x 128] = A_tile . B_tile^T
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(kTile >> 3) << 17) |
                             (static_cast<uint32_t>(kTile >> 4) << 24);
      bool ok = mbar_wait(&sh.a_full, 0, abort_flag);
      for (int t = 0; t < p.tiles && ok && !*abort_flag; ++t) {
        const int s = t % p.stages, round = t / p.stages, acc = t & 1, use = t >> 1;
        if (use > 0 && !mbar_wait(&sh.tmem_empty[acc], (use - 1) & 1, abort_flag)) break;
        if (!mbar_wait(&sh.full[s], round & 1, abort_flag)) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t a_addr = smem_u32(a_tile), b_addr = smem_u32(ring + s * tile_bytes);
        for (int kc = 0; kc < p.k_chunks; ++kc) {
          const uint64_t da = smem_desc_sw128(a_addr + kc * kChunkBytes), db = smem_desc_sw128(b_addr + kc * kChunkBytes);
#pragma unroll
          for (int k = 0; k < 4; ++k) umma_bf16(tmem_acc + acc * kTile, da + 2u * k, db + 2u * k, idesc, kc > 0 || k > 0);
        }
        umma_commit(&sh.tmem_full[acc]);
        if (p.pass == 1) umma_commit(&sh.empty[s]);
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ read-back: one block row and 64 of the block's 128
    // columns per thread (warps w and w + 4 share a quarter of the rows); the two halves keep their own running
    // figures and are put together once at the end
    const int quarter = warp & 3, half = (warp - 2) >> 2;
    const int r_in = quarter * 32 + lane;                 // row of this thread within the block
    const int row = row0 + r_in;                          // query (pass 1) or key (pass 2) of this thread
    float run_max = -INFINITY, run_sum = 0.f, col_sum = 0.f;
    bool ok = true;
    for (int t = 0; t < p.tiles; ++t) {
      const int s = t % p.stages, acc = t & 1, use = t >> 1;
      if (ok) ok = mbar_wait_warp(&sh.tmem_full[acc], use & 1, abort_flag);
      if (!ok) continue;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t taddr = tmem_acc + (static_cast<uint32_t>(quarter * 32) << 16) + acc * kTile + half * 64;
      const int col0 = t * kTile + half * 64;
      if (p.pass == 1) {
        // one sweep: per 32 columns the running maximum is raised first, the sum rescaled, the exponentials added
        for (int c0 = 0; c0 < 64; c0 += 32) {
          uint32_t v[32];
          tmem_ld32(taddr + c0, v);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          float cmax = -INFINITY;
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (col0 + c0 + j < p.n) cmax = fmaxf(cmax, __uint_as_float(v[j]) * p.scale_log2e);
          const float new_max = fmaxf(run_max, cmax);
          if (new_max > -INFINITY) {
            float add0 = 0.f, add1 = 0.f;
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
              if (col0 + c0 + j < p.n) add0 += ex2(fmaf(__uint_as_float(v[j]), p.scale_log2e, -new_max));
              if (col0 + c0 + j + 1 < p.n) add1 += ex2(fmaf(__uint_as_float(v[j + 1]), p.scale_log2e, -new_max));
            }
            run_sum = run_sum * ex2(run_max - new_max) + (add0 + add1);   // (first columns: 0 * 2^(-inf) = 0)
            run_max = new_max;
          }
        }
      } else {
        // the copy of the lse2 values completes on the stage's barrier: observe it before reading them
        if (!mbar_wait_warp(&sh.full[s], (t / p.stages) & 1, abort_flag)) { ok = false; continue; }
        const float* lse = reinterpret_cast<const float*>(lse_ring + s * 512) + half * 64;
        for (int c0 = 0; c0 < 64; c0 += 32) {
          uint32_t v[32];
          tmem_ld32(taddr + c0, v);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          float add0 = 0.f, add1 = 0.f;
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            const int i0 = col0 + c0 + j;                  // the queries of these two columns
            if (i0 < p.n && i0 != row) add0 += ex2(fmaf(__uint_as_float(v[j]), p.scale_log2e, -lse[c0 + j]));
            if (i0 + 1 < p.n && i0 + 1 != row) add1 += ex2(fmaf(__uint_as_float(v[j + 1]), p.scale_log2e, -lse[c0 + j + 1]));
          }
          col_sum += add0 + add1;
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&sh.tmem_empty[acc]);
        if (p.pass == 2) mbar_arrive(&sh.empty[s]);
      }
    }
    // ---- the second column half hands its figures to the first, which writes the row's result
    if (half == 1) { sh.part_a[r_in] = p.pass == 1 ? run_max : col_sum; sh.part_b[r_in] = run_sum; }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (half == 0 && ok && row < p.n) {
      if (p.pass == 1) {
        const float m2 = sh.part_a[r_in], s2 = sh.part_b[r_in];
        const float mx = fmaxf(run_max, m2);
        const float sum = (run_sum > 0.f ? run_sum * ex2(run_max - mx) : 0.f) + (s2 > 0.f ? s2 * ex2(m2 - mx) : 0.f);
        p.lse2[static_cast<size_t>(bh) * p.n_pad + row] = mx + log2f(sum);
      } else {
        p.rows[static_cast<size_t>(bh) * p.n + row] = (col_sum + sh.part_a[r_in]) / static_cast<float>(max(p.n - 1, 1));
      }
    }
  }

  // ------------------------------------------------------------ teardown
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (sh.abort_flag) {
    if (threadIdx.x == 0) atomicExch(p.status, static_cast<uint32_t>(VSCAN_ERR_TIMEOUT));
    for (int i = 0; i < 64; ++i) __nanosleep(2000);   // copies still in flight land before the memory is released
    __syncthreads();
  }
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "n"(256) : "memory");
  }
}

}  // namespace recv

bool received_supported(const vscan_score_desc* d) {
  return d->dtype == VSCAN_BF16 && (d->head_dim == 64 || d->head_dim == 128) && d->q_heads == d->kv_heads;
}

// Workspace of the RECEIVED mode: status word | lse2 [batch * heads][n_pad] | per-head rows [batch * heads][n]
size_t received_workspace_bytes(const vscan_score_desc* d) {
  const size_t bh = static_cast<size_t>(d->batch) * d->q_heads, n_pad = round_up(d->seq_len, recv::kTile);
  return kStatusBytes + round_up(bh * n_pad * sizeof(float), 256) + round_up(bh * d->seq_len * sizeof(float), 256);
}

vscan_status launch_received(const vscan_score_desc* d, void* workspace, float* rows_out, cudaStream_t stream) {
  using namespace recv;
  tc::EncodeTiledFn encode = tc::encode_fn();
  if (!encode) return VSCAN_ERR_UNSUPPORTED;
  const size_t bh = static_cast<size_t>(d->batch) * d->q_heads, n_pad = round_up(d->seq_len, kTile);
  char* ws = static_cast<char*>(workspace);
  Params p;
  p.status = reinterpret_cast<uint32_t*>(ws);
  p.lse2 = reinterpret_cast<float*>(ws + kStatusBytes);
  p.rows = rows_out;
  p.n = d->seq_len; p.n_pad = static_cast<int>(n_pad); p.k_chunks = d->head_dim / 64;
  p.tiles = static_cast<int>(n_pad / kTile);
  // two CTAs per SM (shared memory and the 512 columns of tensor memory allow no more): the exponentials of the
  // read-back, not the loads, bound the kernel (head dim 128: 31 ms with three stages and one CTA per SM, 19 ms with two)
  p.stages = p.k_chunks == 1 ? 4 : 2;
  p.scale_log2e = d->scale * 1.4426950408889634f;
  CUtensorMap maps[2];
  const void* ptrs[2] = {d->q, d->k};
  for (int i = 0; i < 2; ++i) {
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(d->head_dim), static_cast<cuuint64_t>(d->seq_len), static_cast<cuuint64_t>(bh)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(d->head_dim) * 2, static_cast<cuuint64_t>(d->seq_len) * d->head_dim * 2};
    const cuuint32_t box[3] = {64, kTile, 1};
    const cuuint32_t elem[3] = {1, 1, 1};
    if (encode(&maps[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptrs[i]), dims, strides, box, elem,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return VSCAN_ERR_UNSUPPORTED;
  }
  const size_t smem = 1024 + static_cast<size_t>(p.k_chunks) * kChunkBytes * (1 + p.stages) + static_cast<size_t>(p.stages) * 512;
  VSCAN_CUDA_TRY(allow_smem(received_kernel, smem));
  VSCAN_CUDA_TRY(cudaMemsetAsync(p.status, 0, sizeof(uint32_t), stream));
  dim3 grid(p.tiles, static_cast<unsigned>(bh));
  p.pass = 1;
  VSCAN_LAUNCH("received_pass1", stream, (received_kernel<<<grid, kThreads, smem, stream>>>(maps[0], maps[1], p)));
  p.pass = 2;
  VSCAN_LAUNCH("received_pass2", stream, (received_kernel<<<grid, kThreads, smem, stream>>>(maps[1], maps[0], p)));
  return VSCAN_OK;
}

}  // namespace vscan
