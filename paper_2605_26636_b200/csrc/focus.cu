// Focused feature map (Eq. 3; Table 1 "+ DWC on V + Focusing Factor"): per token and head,
//   phi_p(x) = (||r|| / ||r^p||) r^p,   r = ReLU(x),  r^p element-wise over the D features.
// The linear-attention block with this kernel function is the ReLU block applied to phi_p(Q) and
// phi_p(K) (phi_p is non-negative), so the map runs as one streaming pass over Q and K (one warp
// per token row, fp32 arithmetic, the result stored in the tensors' type) ahead of the block's own
// kernels.  That is two more tensors read and written than the ReLU block needs -- the overhead
// Table 1 reports for this variant, and the reason the paper keeps ReLU.
#include "common.cuh"

namespace jv {
namespace {

template <typename T>
__global__ void __launch_bounds__(256)
focus_map_kernel(const T* __restrict__ q, const T* __restrict__ k, T* __restrict__ qf, T* __restrict__ kf, size_t rows,
                 int D, float p) {
  const size_t row = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int lane = threadIdx.x & 31;
  const T* src = (blockIdx.y == 0 ? q : k) + row * D;
  T* dst = (blockIdx.y == 0 ? qf : kf) + row * D;
  float rp[4];                                    // D <= 128: up to 4 features per lane
  float n1 = 0.f, np = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int e = lane + 32 * i;
    const float r = e < D ? fmaxf(to_f32(src[e]), 0.f) : 0.f;
    float x;
    if (p == 1.f) x = r;
    else if (p == 2.f) x = r * r;
    else if (p == 3.f) x = r * r * r;
    else x = r > 0.f ? exp2f(p * log2f(r)) : 0.f;
    rp[i] = x;
    n1 = fmaf(r, r, n1);
    np = fmaf(x, x, np);
  }
  n1 = warp_sum(n1);
  np = warp_sum(np);
  const float scale = np > 0.f ? sqrtf(n1 / np) : 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int e = lane + 32 * i;
    if (e < D) from_f32(&dst[e], rp[i] * scale);
  }
}

}  // namespace

cudaError_t launch_focus_map(const void* q, const void* k, void* qf, void* kf, const jv_shape& s, float p, cudaStream_t st) {
  const size_t rows = (size_t)s.B * s.H * shape_tokens(s);
  dim3 grid((unsigned)((rows + 7) / 8), 2);
  if (s.dtype == JV_F32)
    focus_map_kernel<float><<<grid, 256, 0, st>>>((const float*)q, (const float*)k, (float*)qf, (float*)kf, rows, s.D, p);
  else
    focus_map_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (__nv_bfloat16*)qf,
                                                          (__nv_bfloat16*)kf, rows, s.D, p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace jv
