// Housekeeping entry points and process-wide bookkeeping.
#include "common.cuh"

namespace vscan {
std::atomic<uint64_t> g_launches{0};
thread_local int g_last_cuda_error = 0;
}  // namespace vscan

using namespace vscan;

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
