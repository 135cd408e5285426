// Group means of the merge step (Eq. 4) on CUDA cores: the one body of the ordered sums, shared by the stand-alone
// group_mean kernel and by the mean warps of the persistent merge kernel, and the bit-mask variant for short instances.
#pragma once

#include "merge.cuh"

namespace vscan {

// How the threads that share a group-mean job meet: the whole CTA, or a subset of its warps on a named barrier.
struct CtaSync {
  __device__ __forceinline__ void operator()() const { __syncthreads(); }
};
template <int kBarrier, int kThreadsOfGroup>
struct NamedSync {
  __device__ __forceinline__ void operator()() const { asm volatile("bar.sync %0, %1;" ::"n"(kBarrier), "n"(kThreadsOfGroup) : "memory"); }
};

// Exclusive prefix sum of one int per thread over the kWarps warps of a group; `total` gets the group sum.
// `warp_sums` is shared scratch of at least 33 ints.
template <int kWarps, typename Sync>
__device__ __forceinline__ int group_exclusive_scan(int v, int* warp_sums, int& total, int gwarp, int lane, Sync sync) {
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  sync();   // protect warp_sums from a previous use
  if (lane == 31) warp_sums[gwarp] = incl;
  sync();
  if (gwarp == 0) {
    const int w = lane < kWarps ? warp_sums[lane] : 0;
    int wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += t;
    }
    if (lane < kWarps) warp_sums[lane] = wi - w;
    if (lane == 31) warp_sums[32] = wi;
  }
  sync();
  total = warp_sums[32];
  return warp_sums[gwarp] + incl - v;
}

// The ordered group sums of Eq. 4 for kSlots consecutive kept slots s0 .. s0 + kSlots - 1 of instance b, by a group
// of kWarps warps (thread `gtid` of the group): the stand-alone group_mean kernel calls it with its whole CTA, the
// persistent merge kernel with its mean warps.  The group first lists, in ascending token order, the tokens
// assigned to its slots; warp w then takes slots w, w + kWarps, ..., walks the list and adds the members' rows in
// that order (fp32), R rows in flight, VPL 16-byte pieces per lane and column pass; one rounding on output.
// `list` is shared memory of 2 * n_tokens words: list[n_tokens] of (local slot << 24 | token), then
// assign[n_tokens]; `warp_sums` is shared scratch of 33 ints.
template <typename T, int VPL, int R, int kSlots, int kWarps, typename Sync>
__device__ __forceinline__ void group_mean_body(const MergeParams& p, int b, int s0, uint32_t* list, int* warp_sums,
                                                int gtid, Sync sync) {
  constexpr int kGroupThreads = kWarps * 32;
  constexpr int E = Vec16<T>::kElems;
  const int gwarp = gtid >> 5, lane = gtid & 31;
  // all assignments of the instance -> shared memory (second half of the buffer) in rounds of
  // independent, coalesced loads; the two ordered passes below then run out of shared memory
  int32_t* assign = reinterpret_cast<int32_t*>(list + p.n_tokens);
  {
    const int32_t* ag = p.assign + static_cast<size_t>(b) * p.n_tokens;
    for (int i0 = gtid; i0 < p.n_tokens; i0 += kGroupThreads * 8) {
      int32_t v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) { const int i = i0 + u * kGroupThreads; v[u] = i < p.n_tokens ? __ldcg(ag + i) : 0; }
#pragma unroll
      for (int u = 0; u < 8; ++u) { const int i = i0 + u * kGroupThreads; if (i < p.n_tokens) assign[i] = v[u]; }
    }
  }
  sync();

  // contiguous run of tokens per thread; an odd run length keeps the threads of a warp on different banks
  const int per = ((p.n_tokens + kGroupThreads - 1) / kGroupThreads) | 1;
  const int lo = min(p.n_tokens, gtid * per), hi = min(p.n_tokens, lo + per);
  int mine = 0;
  for (int i = lo; i < hi; ++i) mine += static_cast<unsigned>(assign[i] - s0) < static_cast<unsigned>(kSlots);
  int n_list;
  int pos = group_exclusive_scan<kWarps>(mine, warp_sums, n_list, gwarp, lane, sync);
  for (int i = lo; i < hi; ++i) {
    const unsigned rel = static_cast<unsigned>(assign[i] - s0);
    if (rel < static_cast<unsigned>(kSlots)) list[pos++] = (rel << 24) | static_cast<unsigned>(i);
  }
  sync();

  const int vecs = p.dim / E;
  const T* xb = static_cast<const T*>(p.x) + (static_cast<size_t>(b) * p.row_len + p.cls_offset) * p.dim;
  for (int sl = gwarp; sl < kSlots; sl += kWarps) {
    const int s = s0 + sl;
    if (s >= p.n_kept) break;
    T* out = static_cast<T*>(p.merged) + (static_cast<size_t>(b) * p.n_kept + s) * p.dim;
    for (int v0 = 0; v0 < vecs; v0 += 32 * VPL) {
      float acc[VPL][E];
#pragma unroll
      for (int i = 0; i < VPL; ++i)
#pragma unroll
        for (int e = 0; e < E; ++e) acc[i][e] = 0.f;
      int count = 0;
      for (int c = 0; c < n_list; c += 32) {
        const uint32_t entry = c + lane < n_list ? list[c + lane] : 0xFFFFFFFFu;
        unsigned mask = __ballot_sync(0xffffffffu, (entry >> 24) == static_cast<unsigned>(sl));
        count += __popc(mask);
        while (mask) {
          int tok[R];
#pragma unroll
          for (int r = 0; r < R; ++r) {
            tok[r] = -1;
            if (mask) {
              const int l = __ffs(mask) - 1;
              mask &= mask - 1;
              tok[r] = static_cast<int>(__shfl_sync(0xffffffffu, entry, l) & 0xFFFFFFu);
            }
          }
          uint4 raw[R][VPL];
#pragma unroll
          for (int r = 0; r < R; ++r) {
            const uint4* row = reinterpret_cast<const uint4*>(xb + static_cast<size_t>(tok[r] < 0 ? tok[0] : tok[r]) * p.dim);
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
                float f[E];
                Vec16<T>::unpack(raw[r][i], f);
#pragma unroll
                for (int e = 0; e < E; ++e) acc[i][e] += f[e];
              }
            }
          }
        }
      }
      const float inv = 1.f / static_cast<float>(max(count, 1));
#pragma unroll
      for (int i = 0; i < VPL; ++i) {
        const int v = v0 + lane + 32 * i;
        if (v < vecs) {
          float f[E];
#pragma unroll
          for (int e = 0; e < E; ++e) f[e] = acc[i][e] * inv;
          st_16(reinterpret_cast<uint4*>(out) + v, Vec16<T>::pack(f));
        }
      }
      if (v0 == 0 && lane == 0 && p.counts) p.counts[static_cast<size_t>(b) * p.n_kept + s] = count;
    }
  }
}


}  // namespace vscan

namespace vscan {

// Short instances: the same sums with a cheaper prologue.  Four slots per CTA, warp w owns slot s0 + w.
// Every thread marks its tokens in a bit mask per (slot, 32-token chunk) with shared-memory atomics (two
// block barriers in all, no scan); warp w then turns the masks of its slot into its own list of members
// (ascending token order: chunk by chunk, bit by bit) with one warp-wide prefix sum, and walks it with R
// rows in flight.  Same order of additions as group_mean_body, hence the same bits.
// dynamic shared memory: bits[4][chunks] words | lists[4][n_tokens] halfwords.  n_tokens < 65536.
template <typename T, int VPL, int R>
__device__ __forceinline__ void group_mean_bits_body(const MergeParams& p, int b, int s0, unsigned char* smem) {
  constexpr int E = Vec16<T>::kElems;
  constexpr int kSlots = 4, kThreadsCta = kSlots * 32;
  const int chunks = (p.n_tokens + 31) / 32;
  uint32_t* bits = reinterpret_cast<uint32_t*>(smem);
  uint16_t* lists = reinterpret_cast<uint16_t*>(bits + kSlots * chunks);
  const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = threadIdx.x; i < kSlots * chunks; i += kThreadsCta) bits[i] = 0u;
  __syncthreads();
  {
    const int32_t* ag = p.assign + static_cast<size_t>(b) * p.n_tokens;
    for (int i0 = threadIdx.x; i0 < p.n_tokens; i0 += kThreadsCta * 8) {
      int32_t v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) { const int i = i0 + u * kThreadsCta; v[u] = i < p.n_tokens ? __ldcg(ag + i) : -1; }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int i = i0 + u * kThreadsCta;
        const unsigned rel = static_cast<unsigned>(v[u] - s0);
        if (i < p.n_tokens && rel < static_cast<unsigned>(kSlots)) atomicOr(&bits[rel * chunks + (i >> 5)], 1u << (i & 31));
      }
    }
  }
  __syncthreads();
  const int s = s0 + w;
  if (s >= p.n_kept) return;
  // the members of slot s: lane l expands the mask words l, l + 32, ... in order
  uint16_t* list = lists + static_cast<size_t>(w) * p.n_tokens;
  int count = 0;
  for (int c0 = 0; c0 < chunks; c0 += 32) {
    const int c = c0 + lane;
    uint32_t word = c < chunks ? bits[w * chunks + c] : 0u;
    const int mine = __popc(word);
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    int pos = count + incl - mine;
    while (word) {
      const int bit = __ffs(word) - 1;
      word &= word - 1;
      list[pos++] = static_cast<uint16_t>(c * 32 + bit);
    }
    count += __shfl_sync(0xffffffffu, incl, 31);
  }
  __syncwarp();

  const int vecs = p.dim / E;
  const T* xb = static_cast<const T*>(p.x) + (static_cast<size_t>(b) * p.row_len + p.cls_offset) * p.dim;
  T* out = static_cast<T*>(p.merged) + (static_cast<size_t>(b) * p.n_kept + s) * p.dim;
  for (int v0 = 0; v0 < vecs; v0 += 32 * VPL) {
    float acc[VPL][E];
#pragma unroll
    for (int i = 0; i < VPL; ++i)
#pragma unroll
      for (int e = 0; e < E; ++e) acc[i][e] = 0.f;
    for (int k = 0; k < count; k += R) {
      uint4 raw[R][VPL];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if (k + r < count) {
          const uint4* row = reinterpret_cast<const uint4*>(xb + static_cast<size_t>(list[k + r]) * p.dim);
#pragma unroll
          for (int i = 0; i < VPL; ++i) {
            const int v = v0 + lane + 32 * i;
            if (v < vecs) raw[r][i] = ld_nc_16(row + v);
          }
        }
      }
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if (k + r < count) {
#pragma unroll
          for (int i = 0; i < VPL; ++i) {
            const int v = v0 + lane + 32 * i;
            if (v < vecs) {
              float f[E];
              Vec16<T>::unpack(raw[r][i], f);
#pragma unroll
              for (int e = 0; e < E; ++e) acc[i][e] += f[e];
            }
          }
        }
      }
    }
    const float inv = 1.f / static_cast<float>(max(count, 1));
#pragma unroll
    for (int i = 0; i < VPL; ++i) {
      const int v = v0 + lane + 32 * i;
      if (v < vecs) {
        float f[E];
#pragma unroll
        for (int e = 0; e < E; ++e) f[e] = acc[i][e] * inv;
        st_16(reinterpret_cast<uint4*>(out) + v, Vec16<T>::pack(f));
      }
    }
    if (v0 == 0 && lane == 0 && p.counts) p.counts[static_cast<size_t>(b) * p.n_kept + s] = count;
  }
}

}  // namespace vscan
