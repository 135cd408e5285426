// Exact top-k selection on order-preserving uint32 keys held in shared memory.
//
// "k largest, equal keys to the lowest index" is found in two steps: a radix select yields the
// threshold T (the k-th largest key among the candidates) and `need`, the number of candidates
// equal to T that still belong to the set; every key above T is taken, and of the keys equal to
// T the first `need` in index order.  No sort, no float atomics, exactly k survivors.
#pragma once

#include "common.cuh"

namespace vscan {

struct SelectScratch {
  int hist[256];
  int warp_sums[33];
  uint32_t threshold;
  int need;
};

// One pass of the radix select, first half: every candidate whose bits above the current digit equal
// `prefix` adds one to hist[digit].  hist must be zero; the caller synchronises before reading it.
__device__ __forceinline__ void radix_hist_add(const uint32_t* keys, const uint8_t* excluded, int n, int shift,
                                               uint32_t prefix, uint32_t mask, int* hist) {
  // Scores of one instance share their exponent, so in the first pass nearly every key falls into
  // the same bin: there lanes with equal digits are counted with one shared-memory atomic per warp.
  // Later passes see spread-out digits and add directly.
  if (shift == 24) {
    for (int base = 0; base < n; base += blockDim.x) {
      const int i = base + threadIdx.x;
      const bool valid = i < n && !(excluded && excluded[i]);
      const uint32_t digit = valid ? (keys[i] >> 24) : 0u;
      // the lanes that share the digit of the warp's first candidate are counted with one atomic, the
      // others (few) add one by one
      const unsigned lane = threadIdx.x & 31;
      const unsigned vmask = __ballot_sync(0xffffffffu, valid);
      if (vmask) {
        const int lead = __ffs(vmask) - 1;
        const uint32_t d0 = __shfl_sync(0xffffffffu, digit, lead);
        const unsigned same = __ballot_sync(0xffffffffu, valid && digit == d0);
        if (lane == static_cast<unsigned>(lead)) atomicAdd(&hist[d0], __popc(same));
        if (valid && digit != d0) atomicAdd(&hist[digit], 1);
      }
    }
  } else {
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
      if (excluded && excluded[i]) continue;
      const uint32_t key = keys[i];
      if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
    }
  }
}

// Second half, one warp: lane l holds the counts of bins [8l, 8l+8) in local[]; the bin that holds the
// k_rem-th largest candidate extends the prefix, and the candidates above it inside the bin are taken off
// k_rem.  The owning lane writes sc.threshold / sc.need.
__device__ __forceinline__ void radix_pick(const int (&local)[8], int lane, int k_rem, uint32_t prefix, int shift,
                                           SelectScratch& sc) {
  int sum = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) sum += local[j];
  // above = candidates in bins owned by higher lanes
  int incl = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_down_sync(0xffffffffu, incl, o);
    if (lane + o < 32) incl += t;
  }
  int above = incl - sum;
  // the k_rem-th largest lies in this lane's bins iff above < k_rem <= above + sum
  if (above < k_rem && k_rem <= above + sum) {
    int acc = above;
#pragma unroll
    for (int j = 7; j >= 0; --j) {
      if (acc < k_rem && k_rem <= acc + local[j]) {
        sc.threshold = prefix | (static_cast<uint32_t>(lane * 8 + j) << shift);
        sc.need = k_rem - acc;
      }
      acc += local[j];
    }
  }
}

// Block-wide radix select, 4 passes of 8 bits.  Candidates are the i in [0, n) with
// excluded == nullptr || !excluded[i].  Requires 1 <= k <= #candidates.  All threads of the
// block must call; on return every thread reads the same (threshold, need).
__device__ __forceinline__ void block_radix_select(const uint32_t* keys, const uint8_t* excluded, int n,
                                                   int k, SelectScratch& sc, uint32_t& threshold,
                                                   int& need) {
  uint32_t prefix = 0, mask = 0;
  int k_rem = k;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = threadIdx.x; i < 256; i += blockDim.x) sc.hist[i] = 0;
    __syncthreads();
    radix_hist_add(keys, excluded, n, shift, prefix, mask, sc.hist);
    __syncthreads();
    if (threadIdx.x < 32) {
      // lane l owns bins [8l, 8l+8); walk from the top bin down
      const int lane = threadIdx.x;
      int local[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) local[j] = sc.hist[lane * 8 + j];
      radix_pick(local, lane, k_rem, prefix, shift, sc);
    }
    __syncthreads();
    prefix = sc.threshold;
    k_rem = sc.need;
    mask |= 0xFFu << shift;
    __syncthreads();
  }
  threshold = prefix;
  need = k_rem;
}

// Block-wide: the k largest of keys[0..n) (equal keys to the lowest index) written in ascending index
// order to out[0..k).  n <= 64 * blockDim.x.  All threads must call; 1 <= k <= n.
__device__ __forceinline__ void block_topk_emit(const uint32_t* keys, int n, int k, SelectScratch& sc, int32_t* out) {
  uint32_t thr;
  int need;
  block_radix_select(keys, nullptr, n, k, sc, thr, need);
  const int per = (n + blockDim.x - 1) / blockDim.x;
  const int lo = min(n, static_cast<int>(threadIdx.x) * per), hi = min(n, lo + per);
  int eq_local = 0;
  for (int i = lo; i < hi; ++i) eq_local += (keys[i] == thr);
  int total;
  int eq_before = block_exclusive_scan(eq_local, sc.warp_sums, total);
  int kept_local = 0;
  unsigned long long flags = 0;
  for (int i = lo; i < hi; ++i) {
    const uint32_t key = keys[i];
    bool keep = key > thr;
    if (key == thr) { keep = eq_before < need; ++eq_before; }
    if (keep) { flags |= 1ull << (i - lo); ++kept_local; }
  }
  int pos = block_exclusive_scan(kept_local, sc.warp_sums, total);
  for (int i = lo; i < hi; ++i)
    if ((flags >> (i - lo)) & 1ull) { if (pos < k) out[pos] = i; ++pos; }
}

// Warp-wide bitwise select over m candidates enumerated by `token_of(p)`, p in [0, m), ascending
// in p.  Marks the k winners in `selected` (shared memory, one byte per token).  0 <= k <= m.
template <typename TokenOf>
__device__ __forceinline__ void warp_select_mark(const uint32_t* keys, int m, int k, TokenOf token_of,
                                                 uint8_t* selected) {
  if (k <= 0) return;
  const int lane = threadIdx.x & 31;
  uint32_t prefix = 0;
  int k_rem = k;
  for (int bit = 31; bit >= 0; --bit) {
    const uint32_t hi_mask = ~((2u << bit) - 1u);  // bits above `bit`; 0 when bit == 31
    int cnt = 0;
    for (int p0 = 0; p0 < m; p0 += 32) {
      int p = p0 + lane;
      bool hit = false;
      if (p < m) {
        uint32_t key = keys[token_of(p)];
        hit = ((key & hi_mask) == prefix) && ((key >> bit) & 1u);
      }
      cnt += __popc(__ballot_sync(0xffffffffu, hit));
    }
    if (cnt >= k_rem) prefix |= (1u << bit); else k_rem -= cnt;
  }
  // prefix is the k-th largest key; k_rem of the keys equal to it belong to the set
  int taken_eq = 0;
  for (int p0 = 0; p0 < m; p0 += 32) {
    int p = p0 + lane;
    bool gt = false, eq = false;
    int t = 0;
    if (p < m) {
      t = token_of(p);
      uint32_t key = keys[t];
      gt = key > prefix;
      eq = key == prefix;
    }
    unsigned eq_mask = __ballot_sync(0xffffffffu, eq);
    int rank = taken_eq + __popc(eq_mask & ((1u << lane) - 1u));
    if (gt || (eq && rank < k_rem)) selected[t] = 1;
    taken_eq += __popc(eq_mask);
  }
}

// Warp-wide exact top-k for small candidate sets (m <= 64) by rank counting: candidate p is kept
// iff fewer than k candidates beat it (larger key, or equal key and smaller p).  Two candidates per
// lane live in registers; the keys are passed around with shuffles, no shared-memory traffic.
template <typename TokenOf>
__device__ __forceinline__ void warp_rank_mark(const uint32_t* keys, int m, int k, TokenOf token_of,
                                               uint8_t* selected) {
  if (k <= 0) return;
  const int lane = threadIdx.x & 31;
  const int p0 = lane, p1 = lane + 32;
  const int t0 = p0 < m ? token_of(p0) : 0, t1 = p1 < m ? token_of(p1) : 0;
  const uint32_t k0 = p0 < m ? keys[t0] : 0u, k1 = p1 < m ? keys[t1] : 0u;
  int r0 = 0, r1 = 0;
  const int m0 = min(m, 32);
  for (int j = 0; j < m0; ++j) {
    const uint32_t kj = __shfl_sync(0xffffffffu, k0, j);
    r0 += (kj > k0) || (kj == k0 && j < p0);
    r1 += (kj >= k1);                       // every j < 32 precedes p1
  }
  for (int j = 32; j < m; ++j) {
    const uint32_t kj = __shfl_sync(0xffffffffu, k1, j - 32);
    r0 += (kj > k0);                        // every j >= 32 follows p0
    r1 += (kj > k1) || (kj == k1 && j < p1);
  }
  if (p0 < m && r0 < k) selected[t0] = 1;
  if (p1 < m && r1 < k) selected[t1] = 1;
}

}  // namespace vscan
