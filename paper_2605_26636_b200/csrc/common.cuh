// Shared host/device helpers of libjetvit (internal; not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "jetvit.h"

namespace jv {

// ---- device status word ---------------------------------------------------
// One int per device lives in api.cu; kernels receive its device address and OR
// error bits into it.  Bit 0: a bounded wait ran out.
constexpr int kStatusTimeout = 1;

int* device_status_ptr();        // device address of the status word (nullptr on failure)
void count_launch(int n = 1);    // launch counter behind jv_launch_count()

// ---- per-device facts --------------------------------------------------------
// The library may be used on several GPUs from one process (one device current per
// call), so whatever CUDA keeps per device is cached per device here.
constexpr int kMaxDevices = 64;
constexpr int kDefaultSmCount = 148;   // B200; used for planning when no device can be asked
int current_device();            // index of the current device, -1 if it cannot be read
int device_sm_count();           // SM count of the current device (kDefaultSmCount without one)

// Runs `f` (which returns a cudaError_t) once per device, with that device current:
// the opt-in to more than 48 KB of dynamic shared memory is a per-device function
// attribute.  Two host threads may both run f; it is idempotent.
class OncePerDevice {
 public:
  template <typename F>
  cudaError_t run(F f) {
    const int d = current_device();
    if (d < 0 || d >= kMaxDevices) return f();
    if (done_[d].load(std::memory_order_acquire)) return cudaSuccess;
    const cudaError_t e = f();
    if (e == cudaSuccess) done_[d].store(1, std::memory_order_release);
    return e;
  }

 private:
  std::atomic<int> done_[kMaxDevices] = {};
};

// ---- element access -------------------------------------------------------
__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_f32(float* p, float x) { *p = x; }
__device__ __forceinline__ void from_f32(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
// tokens per (batch, head): prefix tokens, then the grid
static inline int shape_tokens(const jv_shape& s) { return s.P + s.Hg * s.Wg; }
static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Element strides of the inputs q, k, v over (token, head, batch); o is always [B, H, N, D] contiguous.
struct InStrides {
  int64_t tok, head, batch;
};
static inline InStrides in_strides(const jv_shape& s) {
  const int64_t n = shape_tokens(s);
  if (s.in_layout == JV_LAYOUT_BNHD) {
    const int64_t ts = s.in_tok_stride ? s.in_tok_stride : (int64_t)s.H * s.D;
    return InStrides{ts, (int64_t)s.D, n * ts};
  }
  return InStrides{(int64_t)s.D, n * s.D, (int64_t)s.H * n * s.D};
}
static inline bool in_strided(const jv_shape& s) { return s.in_layout != JV_LAYOUT_BHND; }

// ---- plan of the linear-attention workspace --------------------------------
// State per (batch, head): (D+1) x (D+1) fp32, S[a][e] = sum_j pk[j][a] * pv[j][e]
// with pk = [relu(k) | 1], pv = [v | 1]:  S[a<D][e<D] = KV, S[a][D] = z (k-sum),
// S[D][e] = v-sum, S[D][D] = N.
struct LinPlan {
  int D1;            // D + 1
  int state_elems;   // D1 * D1 rounded up to a multiple of 4
  int chunk_tokens;  // tokens per phase-1 chunk
  int nchunk;        // chunks per (batch, head)
  size_t off_partial, off_state, off_hidden, off_kernel, total;  // byte offsets into ws
  // token-wise dynamic convolution on the tensor-core path: bf16 copies of W1, W2, the hidden layer
  // [B, ntok, R] and the kernels of all tokens as planes [B, C*k*k/64, ntok, 64] (bf16)
  size_t off_tok_w1, off_tok_w2, off_tok_hidden, off_tok_kernel;
};
LinPlan lin_plan(const jv_shape& s, const jv_dwc* dwc);

// ---- kernels' host launchers (each returns a cudaError_t from the launch) ---
struct AttnArgs {
  const void *q, *k, *v;
  void* o;
  int BH, Hg, Wg, D;
  int H;           // heads: (batch, head) index bh = b * H + h
  InStrides in;    // element strides of q, k, v (the tensor-core paths honour them; the others need the default)
  bool strided;    // in differs from the contiguous [B, H, N, D] strides
  int P;       // prefix tokens in front of the Hg x Wg grid tokens (full attention: folded into the "grid")
  int wh, ww;  // window size (wh >= Hg and ww >= Wg: one window = full attention)
  float scale;
  int dtype;
};
cudaError_t launch_attn_generic(const AttnArgs& a, cudaStream_t st, bool prefix_rows_only = false);
// tcgen05 path: bf16, D == 64.  full = true: F over all N tokens; else W with (wh, ww)
// windows whose width ww is a power of two <= 128 (a tile is a box of ww x 128/ww tokens).
bool attn_tc_supported(const AttnArgs& a, bool full);
cudaError_t launch_attn_tc(const AttnArgs& a, bool full, int* status, cudaStream_t st);
// tcgen05 path for windows of one or two 128-token tiles (bf16, D == 64, at most 16 prefix tokens): two windows per CTA
bool attn_w4_supported(const AttnArgs& a);
cudaError_t launch_attn_w4(const AttnArgs& a, int* status, cudaStream_t st);
// tcgen05 path at head_dim 128 (bf16, N >= 128, no prefix tokens in W): two query tiles per CTA.
// full = true: F over all N tokens; else W with windows whose width is a power of two <= 128
bool attn_d128_supported(const AttnArgs& a, bool full);
cudaError_t launch_attn_d128(const AttnArgs& a, bool full, int* status, cudaStream_t st);
// tcgen05 path for full attention over long sequences (bf16, D == 64, N >= 1024): four query tiles per CTA
bool attn_f4_supported(const AttnArgs& a);
cudaError_t launch_attn_f4(const AttnArgs& a, int* status, cudaStream_t st);

struct LinArgs {
  const void *q, *k, *v;
  void* o;
  jv_shape s;
  float eps;
  const jv_dwc* dwc;  // host struct holding device pointers, or nullptr
  void* ws;
};
cudaError_t launch_linear_generic(const LinArgs& a, const LinPlan& p, cudaStream_t st);
bool linear_fast_supported(const LinArgs& a);
cudaError_t launch_linear_fast(const LinArgs& a, const LinPlan& p, cudaStream_t st);
// bf16, D == 64, 3 x 3 kernels: the apply pass with the convolution fused in
bool linear_conv_supported(const LinArgs& a);
cudaError_t launch_linear_apply_conv(const LinArgs& a, const LinPlan& p, const float* partial, const float* w,
                                     int* status, bool programmatic, cudaStream_t st);
// shared by both linear paths: hidden = SiLU(W1 s + b1), w = W2 hidden + b2, with
// s = vsum / N read from vsum[bh * bh_stride + e]
cudaError_t launch_dwc_generator(const LinArgs& a, const LinPlan& p, const float* vsum, int bh_stride,
                                 cudaStream_t st);
cudaError_t launch_lin_reduce(const float* partial, float* state, int nchunk, int state_elems, size_t total,
                              cudaStream_t st);

// Focused feature map of Eq. 3 over every token row of q and k -> qf, kf (same shape and type)
cudaError_t launch_focus_map(const void* q, const void* k, void* qf, void* kf, const jv_shape& s, float p, cudaStream_t st);

// Token-wise dynamic convolution (Table 1): o (which holds the attention output) += the convolution
// of V with every grid token's own kernels.  Generic: everything per token on the fly, any type.
cudaError_t launch_dwc_tokenwise_generic(const LinArgs& a, cudaStream_t st);
// bf16, head_dim 64, 3 x 3, R a multiple of 64: generator as two tensor-core GEMMs, then the convolution
bool dwc_tokenwise_fast_supported(const LinArgs& a);
cudaError_t launch_dwc_tokenwise_fast(const LinArgs& a, const LinPlan& p, int* status, cudaStream_t st);
// the projection GEMM kernel on its own terms: D = act(A W^T + bias), bf16, fp32 accumulation.
//   planes_in:  A is [B, a_planes, N, 64] (K block kb = plane kb % a_planes), else A is [B, N, 64 * kblocks]
//   planes_out: D is [B, F / 64, N, 64] (feature block fb = plane fb), else D is [B, N, F]
//   W: [F, 64 * kblocks], bias fp32 [F] or null, silu: apply x / (1 + exp(-x)) to the result;
//   f16_in: A and W hold fp16 instead of bf16; f16_out: D is stored as fp16 instead of bf16
cudaError_t launch_proj_gemm(bool planes_in, bool planes_out, const void* A, const void* W, const float* bias, void* D, int B,
                             int N, int kblocks, int a_planes, int F, bool silu, bool f16_in, bool f16_out, int* status,
                             cudaStream_t st);

// Projections either side of a mixer (bf16, D == 64): qkv = true computes q, k, v (d0, d1, d2)
// from x [B, N, C]; qkv = false computes y (d0) [B, N, C] from x = o [B, H, N, 64].
bool proj_tc_available();
cudaError_t launch_proj_tc(bool qkv, const void* x, const void* w, const float* bias, void* d0, void* d1, void* d2,
                           const jv_shape& s, int* status, cudaStream_t st);

}  // namespace jv
