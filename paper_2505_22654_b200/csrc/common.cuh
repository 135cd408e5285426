// Shared host/device helpers of the VScan library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "vscan.h"

namespace vscan {

// ------------------------------------------------------------------ host-side bookkeeping
extern std::atomic<uint64_t> g_launches;
extern thread_local int g_last_cuda_error;

inline vscan_status cuda_fail(cudaError_t e) {
  g_last_cuda_error = static_cast<int>(e);
  return VSCAN_ERR_CUDA;
}

#define VSCAN_CUDA_TRY(expr)                                   \
  do {                                                         \
    cudaError_t e__ = (expr);                                  \
    if (e__ != cudaSuccess) return ::vscan::cuda_fail(e__);    \
  } while (0)

// Call after every <<<>>>: records launch-time errors and counts the launch.
#define VSCAN_AFTER_LAUNCH()                                   \
  do {                                                         \
    ::vscan::g_launches.fetch_add(1, std::memory_order_relaxed); \
    cudaError_t e__ = cudaGetLastError();                      \
    if (e__ != cudaSuccess) return ::vscan::cuda_fail(e__);    \
  } while (0)

// Optional per-kernel timing (vscan_profile_begin / vscan_profile_end): when enabled, every launch
// is bracketed by a pair of CUDA events on its stream.
void prof_before(const char* name, cudaStream_t stream);
void prof_after(cudaStream_t stream);

// Launch wrapper: VSCAN_LAUNCH("name", stream, kernel<<<grid, block, smem, stream>>>(args));
#define VSCAN_LAUNCH(name, stream, ...)        \
  do {                                         \
    ::vscan::prof_before(name, stream);        \
    __VA_ARGS__;                               \
    ::vscan::prof_after(stream);               \
    VSCAN_AFTER_LAUNCH();                      \
  } while (0)

// Launch with programmatic stream serialisation: the kernel may start while the previous kernel of
// the stream is still draining; it must execute grid_dependency_wait() before it touches anything
// that kernel produced.  Without a preceding kernel (or with an event in between) this is an
// ordinary launch.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                    Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline size_t dtype_bytes(int dtype) { return dtype == VSCAN_F32 ? 4 : 2; }

// [a, a+na) and [b, b+nb) intersect?
inline bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
  if (!a || !b || na == 0 || nb == 0) return false;
  uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
  return a0 < b0 + nb && b0 < a0 + na;
}

// The first 256 bytes of every workspace hold the device status word.
constexpr size_t kStatusBytes = 256;

// Opt a kernel into more than 48 KB of dynamic shared memory (cached per kernel per device).
template <typename K>
inline cudaError_t allow_smem(K kernel, size_t bytes) {
  if (bytes <= 48 * 1024) return cudaSuccess;
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes));
}

constexpr size_t kMaxDynamicSmem = 227 * 1024;

// ------------------------------------------------------------------ device helpers
// Blocks until the preceding kernel of the stream has completed and its writes are visible (no-op
// for a kernel launched the ordinary way).
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel of the stream be scheduled as soon as every CTA of this grid has got here.
__device__ __forceinline__ void grid_dependency_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename T>
__device__ __forceinline__ float to_float(T v);
template <>
__device__ __forceinline__ float to_float<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// Order-preserving map float -> uint32 (larger float <=> larger key); -0.0 is folded onto +0.0 so
// that equal floats have equal keys.
__device__ __forceinline__ uint32_t float_to_key(float f) {
  uint32_t u = __float_as_uint(f);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// 16-byte vector of elements widened to float.  bf16: 8 values, f32: 4 values.
template <typename T>
struct Vec16;
template <>
struct Vec16<float> {
  static constexpr int kElems = 4;
  __device__ __forceinline__ static void unpack(const uint4& r, float* out) {
    out[0] = __uint_as_float(r.x); out[1] = __uint_as_float(r.y);
    out[2] = __uint_as_float(r.z); out[3] = __uint_as_float(r.w);
  }
  __device__ __forceinline__ static uint4 pack(const float* in) {
    return make_uint4(__float_as_uint(in[0]), __float_as_uint(in[1]), __float_as_uint(in[2]),
                      __float_as_uint(in[3]));
  }
};
template <>
struct Vec16<__nv_bfloat16> {
  static constexpr int kElems = 8;
  __device__ __forceinline__ static void unpack(const uint4& r, float* out) {
    // a bf16 is the high half of the float with the same value
    out[0] = __uint_as_float(r.x << 16); out[1] = __uint_as_float(r.x & 0xFFFF0000u);
    out[2] = __uint_as_float(r.y << 16); out[3] = __uint_as_float(r.y & 0xFFFF0000u);
    out[4] = __uint_as_float(r.z << 16); out[5] = __uint_as_float(r.z & 0xFFFF0000u);
    out[6] = __uint_as_float(r.w << 16); out[7] = __uint_as_float(r.w & 0xFFFF0000u);
  }
  __device__ __forceinline__ static uint4 pack(const float* in) {
    __nv_bfloat162 a = __floats2bfloat162_rn(in[0], in[1]);
    __nv_bfloat162 b = __floats2bfloat162_rn(in[2], in[3]);
    __nv_bfloat162 c = __floats2bfloat162_rn(in[4], in[5]);
    __nv_bfloat162 d = __floats2bfloat162_rn(in[6], in[7]);
    return make_uint4(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b),
                      *reinterpret_cast<uint32_t*>(&c), *reinterpret_cast<uint32_t*>(&d));
  }
};

__device__ __forceinline__ uint4 ld_nc_16(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}
__device__ __forceinline__ void st_16(void* p, const uint4& r) {
  asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(r.x), "r"(r.y), "r"(r.z), "r"(r.w)
               : "memory");
}

// Bounded spin on a flag that another CTA sets (polls about 100 ns apart).  Returns true once *flag >= target,
// false when `limit` polls have gone by; the caller then records VSCAN_ERR_TIMEOUT and leaves.
__device__ __forceinline__ bool wait_flag_bounded(const volatile int* flag, int target, unsigned limit) {
  unsigned spins = 0;
  while (*flag < target && spins < limit) { __nanosleep(100); ++spins; }
  return *flag >= target;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Exclusive prefix sum of one int per thread over the whole block; `total` gets the block sum.
// `warp_sums` is shared scratch of at least 33 ints.  Contains __syncthreads().
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  __syncthreads();  // protect warp_sums from a previous use
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = lane < nwarps ? warp_sums[lane] : 0;
    int wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int t = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += t;
    }
    if (lane < nwarps) warp_sums[lane] = wi - w;
    if (lane == 31) warp_sums[32] = wi;
  }
  __syncthreads();
  total = warp_sums[32];
  return warp_sums[warp] + incl - v;
}

}  // namespace vscan
