// bf16 tensor-core path of the linear-attention block (placeholder until the
// mma kernels land: reports "not supported" so the generic kernels run).
#include "common.cuh"
namespace jv {
bool linear_fast_supported(const LinArgs&) { return false; }
cudaError_t launch_linear_fast(const LinArgs&, const LinPlan&, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace jv
