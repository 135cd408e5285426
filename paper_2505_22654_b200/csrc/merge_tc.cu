// Tensor-core path of the merge assignment (tcgen05 MMA, accumulators in tensor memory).
#include "merge.cuh"

namespace vscan {

bool assign_tensor_supported(int /*dtype*/, const MergeParams& /*p*/) { return false; }

vscan_status launch_assign_tensor(const MergeParams& /*p*/, cudaStream_t /*stream*/) {
  return VSCAN_ERR_UNSUPPORTED;
}

}  // namespace vscan
