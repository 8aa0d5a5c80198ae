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

// four consecutive features of a row as fp32, from / to either element type (8 or 16 bytes at once)
__device__ __forceinline__ float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
  const uint2 u = *reinterpret_cast<const uint2*>(p);
  return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16),
                     __uint_as_float(u.y & 0xffff0000u));
}
__device__ __forceinline__ void store4(float* p, float4 x) { *reinterpret_cast<float4*>(p) = x; }
__device__ __forceinline__ void store4(__nv_bfloat16* p, float4 x) {
  __nv_bfloat162 a = __floats2bfloat162_rn(x.x, x.y), b = __floats2bfloat162_rn(x.z, x.w);
  *reinterpret_cast<uint2*>(p) = make_uint2(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b));
}
__device__ __forceinline__ float powp(float r, float p) {
  if (p == 1.f) return r;
  if (p == 2.f) return r * r;
  if (p == 3.f) return r * r * r;
  return r > 0.f ? exp2f(p * log2f(r)) : 0.f;
}

// A row is D / 4 consecutive lanes (kLanes: 8, 16 or 32), a thread owns four consecutive features; the
// two norms are reduced inside the lane group.  A thread walks kIter rows, all loads first.
template <typename T, int kLanes>
__global__ void __launch_bounds__(256)
focus_map_kernel(const T* __restrict__ q, const T* __restrict__ k, T* __restrict__ qf, T* __restrict__ kf, size_t rows, float p) {
  constexpr int kIter = 4, kRowsPerPass = 256 / kLanes, D = 4 * kLanes;
  const T* src = blockIdx.y == 0 ? q : k;
  T* dst = blockIdx.y == 0 ? qf : kf;
  const int sub = threadIdx.x % kLanes;
  const size_t row0 = (size_t)blockIdx.x * (kRowsPerPass * kIter) + threadIdx.x / kLanes;
  float4 x[kIter];
#pragma unroll
  for (int it = 0; it < kIter; ++it) {
    const size_t row = row0 + (size_t)it * kRowsPerPass;
    x[it] = row < rows ? load4(src + row * D + 4 * sub) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
#pragma unroll
  for (int it = 0; it < kIter; ++it) {
    const size_t row = row0 + (size_t)it * kRowsPerPass;
    float4 r = make_float4(fmaxf(x[it].x, 0.f), fmaxf(x[it].y, 0.f), fmaxf(x[it].z, 0.f), fmaxf(x[it].w, 0.f));
    float4 y = make_float4(powp(r.x, p), powp(r.y, p), powp(r.z, p), powp(r.w, p));
    float n1 = fmaf(r.x, r.x, fmaf(r.y, r.y, fmaf(r.z, r.z, r.w * r.w)));
    float np = fmaf(y.x, y.x, fmaf(y.y, y.y, fmaf(y.z, y.z, y.w * y.w)));
#pragma unroll
    for (int o = kLanes / 2; o > 0; o >>= 1) {
      n1 += __shfl_xor_sync(0xffffffffu, n1, o);
      np += __shfl_xor_sync(0xffffffffu, np, o);
    }
    const float scale = np > 0.f ? sqrtf(n1 / np) : 0.f;
    if (row < rows) store4(dst + row * D + 4 * sub, make_float4(y.x * scale, y.y * scale, y.z * scale, y.w * scale));
  }
}

// any other D (a multiple of 8 elements at most 128): one warp per row
template <typename T>
__global__ void __launch_bounds__(256)
focus_map_any_kernel(const T* __restrict__ q, const T* __restrict__ k, T* __restrict__ qf, T* __restrict__ kf, size_t rows,
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
    rp[i] = powp(r, p);
    n1 = fmaf(r, r, n1);
    np = fmaf(rp[i], rp[i], np);
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

template <typename T>
void launch_t(const void* q, const void* k, void* qf, void* kf, size_t rows, int D, float p, cudaStream_t st) {
  const T *tq = (const T*)q, *tk = (const T*)k;
  T *oq = (T*)qf, *ok = (T*)kf;
  if (D == 32 || D == 64 || D == 128) {
    const int lanes = D / 4, rows_per_block = (256 / lanes) * 4;
    dim3 grid((unsigned)((rows + rows_per_block - 1) / rows_per_block), 2);
    if (lanes == 8) focus_map_kernel<T, 8><<<grid, 256, 0, st>>>(tq, tk, oq, ok, rows, p);
    else if (lanes == 16) focus_map_kernel<T, 16><<<grid, 256, 0, st>>>(tq, tk, oq, ok, rows, p);
    else focus_map_kernel<T, 32><<<grid, 256, 0, st>>>(tq, tk, oq, ok, rows, p);
  } else {
    dim3 grid((unsigned)((rows + 7) / 8), 2);
    focus_map_any_kernel<T><<<grid, 256, 0, st>>>(tq, tk, oq, ok, rows, D, p);
  }
}

}  // namespace

cudaError_t launch_focus_map(const void* q, const void* k, void* qf, void* kf, const jv_shape& s, float p, cudaStream_t st) {
  const size_t rows = (size_t)s.B * s.H * shape_tokens(s);
  if (s.dtype == JV_F32) launch_t<float>(q, k, qf, kf, rows, s.D, p, st);
  else launch_t<__nv_bfloat16>(q, k, qf, kf, rows, s.D, p, st);
  count_launch();
  return cudaGetLastError();
}

}  // namespace jv
