// Tensor-core chain kernel (placeholder until the tcgen05 path lands).
#include "mdn_common.cuh"

namespace mdn {

bool tensor_path_supported(const mdn_params&) { return false; }

cudaError_t launch_intra_tensor(const Plan&, const void*, const void*, int*) { return cudaErrorNotSupported; }

cudaError_t launch_chain_tensor(const Plan&, const void*, const void*, const void*, const float*, const float*,
                                void*, float*, float*, int*) {
  return cudaErrorNotSupported;
}

}  // namespace mdn
