// Stage 2, prefill, tensor-core path for sm_100a (placeholder until the tcgen05 kernel lands).
#include "common.cuh"

namespace dash {

bool prefill_sm100_supported(const Dims&) { return false; }

cudaError_t launch_attend_prefill_sm100(const Dims&, const void*, const void*, const void*, const uint32_t*,
                                        const float*, void*, StatusBlock*, cudaStream_t) {
  return cudaErrorNotSupported;
}

}  // namespace dash
