// tcgen05 tensor-core path (placeholder until the kernel lands).
#include "mqa_common.cuh"
namespace mqa {
bool tc_supported(int, int) { return false; }
cudaError_t launch_tc(const Params&, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace mqa
