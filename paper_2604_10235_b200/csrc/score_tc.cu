// placeholder until the tensor-core kernel lands
#include "cc_internal.cuh"
namespace cc {
size_t score_tc_ws_bytes(const BatchTable&, const Geometry&, int) { return 256; }
cudaError_t launch_score_tc(const Launch&, const BatchTable&, const Geometry&, const void*,
                            const void*, float*, float*, void*, void*, int64_t, int*) {
  return cudaErrorNotSupported;
}
}  // namespace cc
