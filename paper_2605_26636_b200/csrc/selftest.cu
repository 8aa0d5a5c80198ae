// jv_selftest_wait_timeout: drives the bounded-wait machinery of the tensor-core kernels to
// its limit without hanging or faulting anything.  One CTA of one warp initialises an
// mbarrier that expects one arrival, nobody ever arrives, and the warp waits on it through
// the same mbar_wait the mixers use, with a short limit.  The wait gives up, sets the sticky
// device status word and the kernel returns normally; the context stays usable.
#include "tc_common.cuh"

namespace jv {
namespace {

__global__ void __launch_bounds__(32)
selftest_wait_kernel(int* status, unsigned long long limit_ns, int* gave_up) {
  __shared__ uint64_t bar;
  __shared__ volatile uint32_t abort_flag;
  if (threadIdx.x == 0) {
    tc::mbar_init(&bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  const bool ok = tc::warp_wait_limit(&bar, 0, &abort_flag, status, limit_ns);
  if (threadIdx.x == 0 && gave_up) *gave_up = ok ? 0 : 1;
}

}  // namespace
}  // namespace jv

extern "C" jv_status jv_selftest_wait_timeout(uint32_t limit_us, int32_t* gave_up, void* cuda_stream) {
  if (limit_us == 0 || limit_us > 1000000u) return JV_ERR_INVALID_ARG;   // at most one second
  int dev = jv::current_device();
  if (dev < 0) return JV_ERR_CUDA;
  int* status = jv::device_status_ptr();
  if (!status) return JV_ERR_CUDA;
  jv::selftest_wait_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(status, (unsigned long long)limit_us * 1000ull,
                                                                     (int*)gave_up);
  jv::count_launch();
  return cudaGetLastError() == cudaSuccess ? JV_OK : JV_ERR_CUDA;
}
