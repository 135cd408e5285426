// Housekeeping entry points and process-wide bookkeeping.
#include "common.cuh"

#include <mutex>
#include <string.h>
#include <vector>

namespace vscan {
std::atomic<uint64_t> g_launches{0};
thread_local int g_last_cuda_error = 0;

// ---- per-kernel timing records (off unless vscan_profile_begin was called)
struct ProfRecord { const char* name; cudaEvent_t start, stop; };
static std::mutex g_prof_mutex;
static std::atomic<bool> g_prof_on{false};
static std::vector<ProfRecord> g_prof;   // preallocated pool
static size_t g_prof_used = 0;

void prof_before(const char* name, cudaStream_t stream) {
  if (!g_prof_on.load(std::memory_order_relaxed)) return;
  std::lock_guard<std::mutex> lock(g_prof_mutex);
  if (g_prof_used >= g_prof.size()) return;
  g_prof[g_prof_used].name = name;
  cudaEventRecord(g_prof[g_prof_used].start, stream);
}

void prof_after(cudaStream_t stream) {
  if (!g_prof_on.load(std::memory_order_relaxed)) return;
  std::lock_guard<std::mutex> lock(g_prof_mutex);
  if (g_prof_used >= g_prof.size()) return;
  cudaEventRecord(g_prof[g_prof_used].stop, stream);
  ++g_prof_used;
}
}  // namespace vscan

namespace vscan {
// Eight independent chains of dependent fused multiply-adds per thread: what the fp32 pipes sustain, measured.
__global__ void __launch_bounds__(256) fma_rate_kernel(float* out, int iters) {
  float a[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) a[k] = static_cast<float>(threadIdx.x + k) * 1e-3f;
  const float b = 1.0000001f, c = 1e-7f;
  for (int i = 0; i < iters; ++i) {
#pragma unroll
    for (int k = 0; k < 8; ++k) a[k] = fmaf(a[k], b, c);
  }
  float sum = 0.f;
#pragma unroll
  for (int k = 0; k < 8; ++k) sum += a[k];
  out[blockIdx.x * blockDim.x + threadIdx.x] = sum;
}
}  // namespace vscan

using namespace vscan;

extern "C" vscan_status vscan_selftest_fma_rate(float* scratch, size_t scratch_floats, int32_t blocks, int32_t iters,
                                                double* flops, void* stream) {
  if (!scratch || !flops || blocks <= 0 || iters <= 0 || scratch_floats < static_cast<size_t>(blocks) * 256) return VSCAN_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  VSCAN_LAUNCH("fma_rate", st, (fma_rate_kernel<<<blocks, 256, 0, st>>>(scratch, iters)));
  *flops = 2.0 * 8.0 * 256.0 * static_cast<double>(blocks) * static_cast<double>(iters);
  return VSCAN_OK;
}

extern "C" int32_t vscan_version(void) { return VSCAN_VERSION; }

extern "C" const char* vscan_status_string(vscan_status s) {
  switch (s) {
    case VSCAN_OK: return "ok";
    case VSCAN_ERR_INVALID_ARG: return "invalid argument";
    case VSCAN_ERR_UNSUPPORTED: return "unsupported shape, dtype or path";
    case VSCAN_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case VSCAN_ERR_CUDA: return "CUDA runtime error";
    case VSCAN_ERR_TIMEOUT: return "bounded device wait expired";
  }
  return "unknown status";
}

extern "C" vscan_status vscan_check(const void* workspace, void* stream) {
  if (!workspace) return VSCAN_ERR_INVALID_ARG;
  uint32_t word = 0;
  VSCAN_CUDA_TRY(cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost,
                                 static_cast<cudaStream_t>(stream)));
  VSCAN_CUDA_TRY(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  return word == 0 ? VSCAN_OK : VSCAN_ERR_TIMEOUT;
}

extern "C" int32_t vscan_last_cuda_error(void) { return g_last_cuda_error; }
extern "C" uint64_t vscan_kernel_launches(void) { return g_launches.load(); }

extern "C" vscan_status vscan_profile_begin(int32_t capacity) {
  if (capacity <= 0 || capacity > (1 << 20)) return VSCAN_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_prof_mutex);
  if (g_prof_on.load()) return VSCAN_ERR_INVALID_ARG;
  g_prof.assign(capacity, ProfRecord{nullptr, nullptr, nullptr});
  for (auto& r : g_prof) {
    VSCAN_CUDA_TRY(cudaEventCreate(&r.start));
    VSCAN_CUDA_TRY(cudaEventCreate(&r.stop));
  }
  g_prof_used = 0;
  g_prof_on.store(true);
  return VSCAN_OK;
}

extern "C" int32_t vscan_profile_end(char* names, float* millis, int32_t capacity) {
  std::lock_guard<std::mutex> lock(g_prof_mutex);
  if (!g_prof_on.load()) return -1;
  g_prof_on.store(false);
  int32_t n = 0;
  for (size_t i = 0; i < g_prof_used; ++i) {
    float ms = 0.f;
    if (cudaEventSynchronize(g_prof[i].stop) != cudaSuccess ||
        cudaEventElapsedTime(&ms, g_prof[i].start, g_prof[i].stop) != cudaSuccess)
      ms = -1.f;
    if (names && millis && n < capacity) {
      strncpy(names + static_cast<size_t>(n) * 32, g_prof[i].name ? g_prof[i].name : "", 31);
      names[static_cast<size_t>(n) * 32 + 31] = 0;
      millis[n] = ms;
      ++n;
    }
  }
  for (auto& r : g_prof) {
    if (r.start) cudaEventDestroy(r.start);
    if (r.stop) cudaEventDestroy(r.stop);
  }
  g_prof.clear();
  g_prof_used = 0;
  return n;
}
