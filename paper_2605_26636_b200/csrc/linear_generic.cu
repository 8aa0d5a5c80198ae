// Linear-attention block (Sec. 3.2.1, Eqs. 2 and 4): workspace plan, the
// shape-generic fp32 kernels, and the squeeze-dynamic-convolution kernel
// generator that both the generic and the bf16 tensor-core paths use.
//
// Three steps, all deterministic (no floating-point atomics):
//   1. per (batch, head, token chunk): partial state  S = [relu(K)|1]^T [V|1]
//   2. fixed-order sum of the chunk partials          -> state per (batch, head)
//   3. streaming apply: o_i = relu(q_i) KV / (relu(q_i).z + eps) [+ DWC(V)_i]
#include "common.cuh"

namespace jv {

LinPlan lin_plan(const jv_shape& s, const jv_dwc* dwc) {
  LinPlan p{};
  const int N = shape_tokens(s), BH = s.B * s.H;
  p.D1 = s.D + 1;
  p.state_elems = (p.D1 * p.D1 + 3) / 4 * 4;
  // Chunks: as many as fit one wave of two CTAs per SM over all (batch, head) pairs, each a
  // multiple of 128 tokens and at least 512 tokens long so that the partials stay small next
  // to K and V.  One wave means no tail, and chunks of equal length finish together.
  int want = (2 * device_sm_count()) / BH;
  if (want < 1) want = 1;
  int chunk = ceil_div(ceil_div(N, want), 128) * 128;
  if (chunk < 512) chunk = 512;
  p.chunk_tokens = chunk;
  p.nchunk = ceil_div(N, chunk);
  size_t off = 0;
  p.off_partial = off; off += align_up((size_t)BH * p.nchunk * p.state_elems * sizeof(float), 256);
  p.off_state = off;   off += align_up((size_t)BH * p.state_elems * sizeof(float), 256);
  p.off_hidden = off;
  p.off_kernel = off;
  p.off_tok_w1 = p.off_tok_w2 = p.off_tok_hidden = p.off_tok_kernel = off;
  if (dwc && dwc->token_wise) {
    const size_t C = (size_t)s.H * s.D, F = C * dwc->k * dwc->k;
    p.off_tok_w1 = off;     off += align_up((size_t)dwc->R * C * 2 * 2, 256);   // bf16 pair (hi | lo) per value
    p.off_tok_w2 = off;     off += align_up(F * dwc->R * 2, 256);
    p.off_tok_hidden = off; off += align_up((size_t)s.B * N * dwc->R * 2, 256);
    p.off_tok_kernel = off; off += align_up((size_t)s.B * N * F * 2, 256);
  } else if (dwc) {
    off += align_up((size_t)s.B * dwc->R * sizeof(float), 256);
    p.off_kernel = off;
    off += align_up((size_t)s.B * s.H * s.D * dwc->k * dwc->k * sizeof(float), 256);
  }
  p.total = off;
  return p;
}

namespace {

// ---- step 1 (generic): partial state of one token chunk ---------------------
template <typename T, int DMAX>
__global__ void __launch_bounds__(256)
lin_state_generic_kernel(const T* __restrict__ k, const T* __restrict__ v, float* __restrict__ partial,
                         int N, int D, int chunk_tokens, int state_elems) {
  constexpr int kTok = 32;
  constexpr int kPerThread = ((DMAX + 1) * (DMAX + 1) + 255) / 256;
  extern __shared__ float smem[];
  const int D1 = D + 1;
  float* ks = smem;              // [kTok][D1]  relu(k), last column 1
  float* vs = ks + kTok * D1;    // [kTok][D1]  v, last column 1
  const int bh = blockIdx.y, chunk = blockIdx.x;
  const int t_begin = chunk * chunk_tokens, t_end = min(N, t_begin + chunk_tokens);
  const size_t base = (size_t)bh * N * D;
  const int total = D1 * D1;

  float acc[kPerThread];
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) acc[i] = 0.f;

  for (int t0 = t_begin; t0 < t_end; t0 += kTok) {
    __syncthreads();
    for (int idx = threadIdx.x; idx < kTok * D1; idx += 256) {
      const int j = idx / D1, e = idx % D1, t = t0 + j;
      float kk = 0.f, vv = 0.f;
      if (t < t_end) {
        kk = e < D ? fmaxf(to_f32(k[base + (size_t)t * D + e]), 0.f) : 1.f;
        vv = e < D ? to_f32(v[base + (size_t)t * D + e]) : 1.f;
      }
      ks[idx] = kk;
      vs[idx] = vv;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kPerThread; ++i) {
      const int idx = threadIdx.x + 256 * i;
      if (idx < total) {
        const int a = idx / D1, e = idx % D1;
        float s = acc[i];
        for (int j = 0; j < kTok; ++j) s = fmaf(ks[j * D1 + a], vs[j * D1 + e], s);
        acc[i] = s;
      }
    }
  }
  float* out = partial + ((size_t)bh * gridDim.x + chunk) * state_elems;
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) {
    const int idx = threadIdx.x + 256 * i;
    if (idx < total) out[idx] = acc[i];
  }
}

// ---- step 2: deterministic second pass --------------------------------------
__global__ void lin_reduce_kernel(const float* __restrict__ partial, float* __restrict__ state,
                                  int nchunk, int state_elems, size_t total) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const size_t bh = i / state_elems, idx = i % state_elems;
  const float* p = partial + bh * nchunk * state_elems + idx;
  float s = 0.f;
  for (int c = 0; c < nchunk; ++c) s += p[(size_t)c * state_elems];   // fixed order
  state[i] = s;
}

// ---- step 3 (generic): apply, one warp per token -----------------------------
template <typename T>
__global__ void __launch_bounds__(256)
lin_apply_generic_kernel(const T* __restrict__ q, const T* __restrict__ v, T* __restrict__ o,
                         const float* __restrict__ state, const float* __restrict__ dwc_w,
                         int H, int P, int Hg, int Wg, int D, int state_elems, float eps, int ksz) {
  extern __shared__ float smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int N = P + Hg * Wg, D1 = D + 1;                    // P prefix tokens, then the grid
  const int bh = blockIdx.y;
  const int tok = blockIdx.x * 8 + warp;
  float* qs = smem + warp * D;
  const size_t base = (size_t)bh * N * D;
  if (tok >= N) return;
  for (int e = lane; e < D; e += 32) qs[e] = fmaxf(to_f32(q[base + (size_t)tok * D + e]), 0.f);
  __syncwarp();
  const float* S = state + (size_t)bh * state_elems;
  float den = eps;
  for (int a = 0; a < D; ++a) den = fmaf(qs[a], __ldg(&S[a * D1 + D]), den);
  const int y = (tok - P) / Wg, x = (tok - P) % Wg, pad = (ksz - 1) / 2;   // (grid tokens only)
  for (int e = lane; e < D; e += 32) {
    float num = 0.f;
    for (int a = 0; a < D; ++a) num = fmaf(qs[a], __ldg(&S[a * D1 + e]), num);
    float r = num / den;
    if (dwc_w && tok >= P) {      // the convolution sees the feature map only
      const int b = bh / H, h = bh % H;
      const float* w = dwc_w + ((size_t)b * H * D + (size_t)h * D + e) * ksz * ksz;
      float c = 0.f;
      for (int dy = 0; dy < ksz; ++dy)
        for (int dx = 0; dx < ksz; ++dx) {
          const int yy = y + dy - pad, xx = x + dx - pad;
          if (yy >= 0 && yy < Hg && xx >= 0 && xx < Wg)
            c = fmaf(__ldg(&w[dy * ksz + dx]), to_f32(v[base + (size_t)(P + yy * Wg + xx) * D + e]), c);
        }
      r += c;
    }
    from_f32(&o[base + (size_t)tok * D + e], r);
  }
}

// ---- kernel generator of the squeeze dynamic convolution ---------------------
// hidden[b][r] = SiLU(b1[r] + sum_c W1[r][c] * mean_v[b][c]); one warp per (b, r).
// vsum points at the v-sum of (batch 0, head 0); consecutive (batch, head) pairs are
// bh_stride floats apart.  The v-sums run over all tokens; the pooling is over the grid
// tokens, so the P prefix rows of V (v: [B*H][ntok][D]) are taken out again.
template <typename T>
__global__ void dwc_hidden_kernel(const float* __restrict__ vsum, const T* __restrict__ v, const float* __restrict__ W1,
                                  const float* __restrict__ b1, float* __restrict__ hidden,
                                  int H, int D, int R, int bh_stride, int P, int ntok, float inv_n) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.y;
  if (warp >= R) return;
  const int C = H * D;
  float s = 0.f;
  for (int c = lane; c < C; c += 32) {
    const int h = c / D, e = c % D;
    float sum = vsum[((size_t)b * H + h) * bh_stride + e];
    for (int t = 0; t < P; ++t) sum -= to_f32(v[(((size_t)b * H + h) * ntok + t) * D + e]);
    const float mean = sum * inv_n;
    s = fmaf(__ldg(&W1[(size_t)warp * C + c]), mean, s);
  }
  s = warp_sum(s);
  if (lane == 0) {
    const float x = s + (b1 ? b1[warp] : 0.f);
    hidden[(size_t)b * R + warp] = x / (1.f + expf(-x));
  }
}

// w[b][t] = b2[t] + sum_r W2[t][r] * hidden[b][r]; one warp per t, all samples.
__global__ void dwc_out_kernel(const float* __restrict__ hidden, const float* __restrict__ W2,
                               const float* __restrict__ b2, float* __restrict__ w, int B, int T, int R) {
  const int t = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (t >= T) return;
  for (int b = 0; b < B; ++b) {
    float s = 0.f;
    for (int r = lane; r < R; r += 32) s = fmaf(__ldg(&W2[(size_t)t * R + r]), hidden[(size_t)b * R + r], s);
    s = warp_sum(s);
    if (lane == 0) w[(size_t)b * T + t] = s + (b2 ? b2[t] : 0.f);
  }
}

template <typename T>
cudaError_t launch_generic_t(const LinArgs& a, const LinPlan& p, cudaStream_t st) {
  const jv_shape& s = a.s;
  const int N = shape_tokens(s), BH = s.B * s.H;
  char* ws = (char*)a.ws;
  float* partial = (float*)(ws + p.off_partial);
  float* state = (float*)(ws + p.off_state);
  const size_t smem1 = (size_t)2 * 32 * p.D1 * sizeof(float);
  dim3 g1(p.nchunk, BH);
  if (s.D <= 64)
    lin_state_generic_kernel<T, 64><<<g1, 256, smem1, st>>>((const T*)a.k, (const T*)a.v, partial, N, s.D,
                                                            p.chunk_tokens, p.state_elems);
  else
    lin_state_generic_kernel<T, 128><<<g1, 256, smem1, st>>>((const T*)a.k, (const T*)a.v, partial, N, s.D,
                                                             p.chunk_tokens, p.state_elems);
  count_launch();
  const size_t total = (size_t)BH * p.state_elems;
  lin_reduce_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(partial, state, p.nchunk, p.state_elems, total);
  count_launch();
  const float* dw = nullptr;
  const bool token_wise = a.dwc && a.dwc->token_wise;
  if (a.dwc && !token_wise) {
    cudaError_t e = launch_dwc_generator(a, p, state + s.D * p.D1, p.state_elems, st);
    if (e != cudaSuccess) return e;
    dw = (const float*)(ws + p.off_kernel);
  }
  dim3 g3(ceil_div(N, 8), BH);
  lin_apply_generic_kernel<T><<<g3, 256, 8 * s.D * sizeof(float), st>>>(
      (const T*)a.q, (const T*)a.v, (T*)a.o, state, dw, s.H, s.P, s.Hg, s.Wg, s.D, p.state_elems, a.eps,
      a.dwc ? a.dwc->k : 0);
  count_launch();
  if (token_wise) return launch_dwc_tokenwise_generic(a, st);   // o += per-token kernels applied to V
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_lin_reduce(const float* partial, float* state, int nchunk, int state_elems, size_t total,
                              cudaStream_t st) {
  lin_reduce_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(partial, state, nchunk, state_elems, total);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_dwc_generator(const LinArgs& a, const LinPlan& p, const float* vsum, int bh_stride,
                                 cudaStream_t st) {
  const jv_shape& s = a.s;
  const jv_dwc& d = *a.dwc;
  char* ws = (char*)a.ws;
  float* hidden = (float*)(ws + p.off_hidden);
  float* w = (float*)(ws + p.off_kernel);
  const int N = s.Hg * s.Wg, ntok = shape_tokens(s);   // pooling: the mean over the grid tokens
  if (d.R > 0) {   // R == 0: static kernels, the output layer just broadcasts b2
    dim3 g1(ceil_div(d.R * 32, 256), s.B);
    if (s.dtype == JV_F32)
      dwc_hidden_kernel<float><<<g1, 256, 0, st>>>(vsum, (const float*)a.v, d.W1, d.b1, hidden, s.H, s.D, d.R, bh_stride,
                                                   s.P, ntok, 1.f / (float)N);
    else
      dwc_hidden_kernel<__nv_bfloat16><<<g1, 256, 0, st>>>(vsum, (const __nv_bfloat16*)a.v, d.W1, d.b1, hidden, s.H, s.D, d.R,
                                                           bh_stride, s.P, ntok, 1.f / (float)N);
    count_launch();
  }
  const int T = s.H * s.D * d.k * d.k;
  dwc_out_kernel<<<ceil_div(T * 32, 256), 256, 0, st>>>(hidden, d.W2, d.b2, w, s.B, T, d.R);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_linear_generic(const LinArgs& a, const LinPlan& p, cudaStream_t st) {
  return a.s.dtype == JV_F32 ? launch_generic_t<float>(a, p, st) : launch_generic_t<__nv_bfloat16>(a, p, st);
}

}  // namespace jv
