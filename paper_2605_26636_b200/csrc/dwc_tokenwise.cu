// Token-wise dynamic depth-wise convolution (Sec. 3.2.1; Table 1 "+ Token-wise Dynamic DWC"):
// the kernel generator (two-layer MLP with SiLU) is fed with every grid token's own value vector and
// gives that token its own k x k kernel per channel,
//   w_i = W2 SiLU(W1 v_i + b1) + b2,    o_i[c] += sum_{dy,dx} w_i[c][dy][dx] V[(y+dy-p, x+dx-p)][c],
// added to the attention output that o already holds.  The paper measures this variant at a 40 %
// lower throughput than a static convolution and replaces it by the pooled (squeeze) generator;
// it is here so that Table 1's rows can be timed side by side.
//
// Two paths.  Generic (any type, any k, any R): one block per (sample, grid token) forms the
// token's hidden layer in shared memory and each thread generates and applies the kernels of one
// channel on the fly.  Tensor-core path (bf16, head_dim 64, 3 x 3, R a multiple of 64): the
// generator is two GEMMs on the projection kernel -- hidden = SiLU(V_tok W1^T + b1) reading V in the
// mixers' [B, H, N, 64] layout, kernels = hidden W2^T + b2 written as planes [B, C*9/64, N, 64] (the
// nine planes 9 h .. 9 h + 8 hold the 576 kernel values of head h's 64 channels) -- and a
// streaming pass (one warp per token and head) applies them.  What makes the variant slow is plain
// here: the kernels of all tokens are 2 * B * N * C * 9 bytes that have to be written and read back.
// Precision: the kernels are of the size of the output itself, so their intermediates are kept
// to 11 significant bits, not 8: W1 enters the first GEMM as a bf16 pair (hi + lo, K doubled; V is
// bf16 anyway), the hidden layer, W2 and the kernels are fp16 (the second GEMM runs on fp16 operands).
#include <cuda_fp16.h>

#include "common.cuh"

namespace jv {
namespace {

constexpr int kD = 64;

// ---- generic: block per (sample, grid token) -------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
dwc_tok_generic_kernel(const T* __restrict__ v, T* __restrict__ o, const float* __restrict__ W1, const float* __restrict__ b1,
                       const float* __restrict__ W2, const float* __restrict__ b2, int H, int D, int P, int Hg, int Wg, int R,
                       int ksz) {
  extern __shared__ float sm[];
  const int C = H * D, ntok = P + Hg * Wg, kk = ksz * ksz, pad = (ksz - 1) / 2;
  float* vi = sm;            // [C] the token's value vector over all heads
  float* hid = sm + C;       // [R]
  const int b = blockIdx.y, i = blockIdx.x, y = i / Wg, x = i % Wg;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int c = threadIdx.x; c < C; c += 256) vi[c] = to_f32(v[(((size_t)b * H + c / D) * ntok + P + i) * D + c % D]);
  __syncthreads();
  for (int r = warp; r < R; r += 8) {
    float s = 0.f;
    for (int c = lane; c < C; c += 32) s = fmaf(__ldg(&W1[(size_t)r * C + c]), vi[c], s);
    s = warp_sum(s);
    if (lane == 0) {
      const float z = s + (b1 ? b1[r] : 0.f);
      hid[r] = z / (1.f + expf(-z));
    }
  }
  __syncthreads();
  for (int c = threadIdx.x; c < C; c += 256) {
    const size_t head = ((size_t)b * H + c / D) * ntok + P;
    float acc = 0.f;
    for (int dy = 0; dy < ksz; ++dy)
      for (int dx = 0; dx < ksz; ++dx) {
        const int yy = y + dy - pad, xx = x + dx - pad;
        if (yy < 0 || yy >= Hg || xx < 0 || xx >= Wg) continue;
        const size_t t = (size_t)c * kk + dy * ksz + dx;
        float w = b2 ? b2[t] : 0.f;
        for (int r = 0; r < R; ++r) w = fmaf(__ldg(&W2[t * R + r]), hid[r], w);
        acc = fmaf(w, to_f32(v[(head + yy * Wg + xx) * D + c % D]), acc);
      }
    T* dst = o + (head + i) * D + c % D;
    from_f32(dst, to_f32(*dst) + acc);
  }
}

// ---- tensor-core path --------------------------------------------------------------------------
// W1 [R, C] fp32 -> [R, 2C] bf16: row r = (hi of row r | lo of row r), lo = w - hi;  W2 [F, R] fp32 -> fp16
__global__ void convert_weights_kernel(const float* __restrict__ W1, __nv_bfloat16* __restrict__ w1, size_t n1, int C,
                                       const float* __restrict__ W2, __half* __restrict__ w2, size_t n2) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n1) {
    const size_t r = i / C, c = i % C;
    const float x = W1[i];
    const __nv_bfloat16 hi = __float2bfloat16_rn(x);
    w1[r * 2 * C + c] = hi;
    w1[r * 2 * C + C + c] = __float2bfloat16_rn(x - __bfloat162float(hi));
  } else if (i < n1 + n2) {
    w2[i - n1] = __float2half_rn(W2[i - n1]);
  }
}

// One warp per (batch*head, grid token), a block walks 8 consecutive tokens of one head.  The 576
// kernel values of the head's channels for this token are nine 128-byte rows (planes 9 h + j); they
// go through shared memory so that lane l ends up with the 18 values of its channels 2 l, 2 l + 1.
__global__ void __launch_bounds__(256)
dwc_tok_apply_kernel(const __nv_bfloat16* __restrict__ v, __nv_bfloat16* __restrict__ o, const __half* __restrict__ wk,
                     int H, int P, int Hg, int Wg) {
  __shared__ uint32_t wsm[8][9 * 32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ntok = P + Hg * Wg, N = Hg * Wg;
  const int bh = blockIdx.y, b = bh / H, h = bh - b * H;
  const int i = blockIdx.x * 8 + warp;
  if (i >= N) return;
  const int y = i / Wg, x = i - y * Wg;
  const size_t planes = (size_t)H * 9;                 // C * 9 / 64 planes per sample
#pragma unroll
  for (int j = 0; j < 9; ++j)
    wsm[warp][32 * j + lane] =
        reinterpret_cast<const uint32_t*>(wk + (((size_t)b * planes + 9 * h + j) * ntok + P + i) * kD)[lane];
  __syncwarp();
  uint32_t wv[9];                                      // kernel values 18 l .. 18 l + 17: channel 2 l taps 0..8, channel 2 l + 1 taps 0..8
#pragma unroll
  for (int j = 0; j < 9; ++j) wv[j] = wsm[warp][9 * lane + j];
  auto wval = [&](int idx) -> float {                  // value idx (0..17) of this lane (fp16)
    const uint32_t u = wv[idx >> 1];
    return __half2float(__ushort_as_half((unsigned short)((idx & 1) ? (u >> 16) : (u & 0xffffu))));
  };
  const __nv_bfloat16* vh = v + ((size_t)bh * ntok + P) * kD + 2 * lane;
  float a0 = 0.f, a1 = 0.f;
#pragma unroll
  for (int dy = 0; dy < 3; ++dy)
#pragma unroll
    for (int dx = 0; dx < 3; ++dx) {
      const int yy = y + dy - 1, xx = x + dx - 1;
      if (yy < 0 || yy >= Hg || xx < 0 || xx >= Wg) continue;
      const uint32_t u = *reinterpret_cast<const uint32_t*>(vh + (size_t)(yy * Wg + xx) * kD);
      a0 = fmaf(wval(3 * dy + dx), __uint_as_float(u << 16), a0);
      a1 = fmaf(wval(9 + 3 * dy + dx), __uint_as_float(u & 0xffff0000u), a1);
    }
  uint32_t* dst = reinterpret_cast<uint32_t*>(o + ((size_t)bh * ntok + P + i) * kD + 2 * lane);
  const uint32_t cur = *dst;
  __nv_bfloat162 r = __floats2bfloat162_rn(__uint_as_float(cur << 16) + a0, __uint_as_float(cur & 0xffff0000u) + a1);
  *dst = *reinterpret_cast<uint32_t*>(&r);
}

}  // namespace

cudaError_t launch_dwc_tokenwise_generic(const LinArgs& a, cudaStream_t st) {
  const jv_shape& s = a.s;
  const jv_dwc& d = *a.dwc;
  const size_t smem = (size_t)(s.H * s.D + d.R) * sizeof(float);
  dim3 grid(s.Hg * s.Wg, s.B);
  if (s.dtype == JV_F32)
    dwc_tok_generic_kernel<float><<<grid, 256, smem, st>>>((const float*)a.v, (float*)a.o, d.W1, d.b1, d.W2, d.b2, s.H, s.D, s.P,
                                                           s.Hg, s.Wg, d.R, d.k);
  else
    dwc_tok_generic_kernel<__nv_bfloat16><<<grid, 256, smem, st>>>((const __nv_bfloat16*)a.v, (__nv_bfloat16*)a.o, d.W1, d.b1,
                                                                   d.W2, d.b2, s.H, s.D, s.P, s.Hg, s.Wg, d.R, d.k);
  count_launch();
  return cudaGetLastError();
}

bool dwc_tokenwise_fast_supported(const LinArgs& a) {
  return a.dwc && a.dwc->token_wise && a.s.dtype == JV_BF16 && a.s.D == kD && a.dwc->k == 3 && a.dwc->R % 64 == 0 &&
         proj_tc_available();
}

cudaError_t launch_dwc_tokenwise_fast(const LinArgs& a, const LinPlan& p, int* status, cudaStream_t st) {
  const jv_shape& s = a.s;
  const jv_dwc& d = *a.dwc;
  const int ntok = shape_tokens(s), C = s.H * kD, F = C * 9;
  char* ws = (char*)a.ws;
  __nv_bfloat16* w1 = (__nv_bfloat16*)(ws + p.off_tok_w1);     // [R, 2C]: hi | lo
  __half* w2 = (__half*)(ws + p.off_tok_w2);
  __half* hidden = (__half*)(ws + p.off_tok_hidden);
  __half* wk = (__half*)(ws + p.off_tok_kernel);
  const size_t n1 = (size_t)d.R * C, n2 = (size_t)F * d.R;
  convert_weights_kernel<<<(unsigned)((n1 + n2 + 255) / 256), 256, 0, st>>>(d.W1, w1, n1, C, d.W2, w2, n2);
  count_launch();
  // hidden[b, n, r] = SiLU(sum_c v[b, c / 64, n, c % 64] (W1hi + W1lo)[r, c] + b1[r]): 2 H K blocks over the H planes of V
  cudaError_t e = launch_proj_gemm(true, false, a.v, w1, d.b1, hidden, s.B, ntok, 2 * s.H, s.H, d.R, true, false, true, status, st);
  if (e != cudaSuccess) return e;
  // kernels[b, t / 64, n, t % 64] = sum_r hidden[b, n, r] W2[t, r] + b2[t], fp16 operands
  e = launch_proj_gemm(false, true, hidden, w2, d.b2, wk, s.B, ntok, d.R / 64, 0, F, false, true, true, status, st);
  if (e != cudaSuccess) return e;
  dim3 grid(ceil_div(s.Hg * s.Wg, 8), s.B * s.H);
  dwc_tok_apply_kernel<<<grid, 256, 0, st>>>((const __nv_bfloat16*)a.v, (__nv_bfloat16*)a.o, wk, s.H, s.P, s.Hg, s.Wg);
  count_launch();
  return cudaGetLastError();
}

}  // namespace jv
