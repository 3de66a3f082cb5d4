// tcgen05 tensor-core versions of the two chunk primitives (placeholder until they land).
#include "common.cuh"

namespace gsa {
bool tc_supported(int, int, int) { return false; }
int tc_value_side_slices(int D) { return D / 64; }
cudaError_t launch_value_side_tc(const ValueSideArgs&, int, int, cudaStream_t, int32_t*) {
    return cudaErrorNotSupported;
}
cudaError_t launch_key_side_tc(const KeySideArgs&, int, int, cudaStream_t, int32_t*) {
    return cudaErrorNotSupported;
}
}  // namespace gsa
