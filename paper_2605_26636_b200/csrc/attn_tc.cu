// tcgen05 / TMEM path of full and window attention (placeholder until the
// kernel lands: reports "not supported" so the generic kernel runs).
#include "common.cuh"
namespace jv {
bool attn_tc_supported(const AttnArgs&, bool) { return false; }
cudaError_t launch_attn_tc(const AttnArgs&, bool, int*, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace jv
