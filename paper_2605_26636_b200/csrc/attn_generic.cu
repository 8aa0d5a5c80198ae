// Shape-generic softmax attention (full and windowed) in fp32 arithmetic.
//
// One kernel serves Eq. 1 over all tokens (F) and over non-overlapping windows
// (W, Sec. 3.2.2): a window covering the grid *is* full attention.  It is the
// fp32 path (no tf32, no tensor cores) and the fallback for shapes the tcgen05
// kernels do not take.  Flash-style: keys stream through shared memory in tiles
// of 32, the softmax is kept online in fp32, nothing of size N x N is stored.
//
// Work split: blockIdx.z = (batch, head), blockIdx.y = window, blockIdx.x = group
// of kRows query rows of that window; one warp owns one query row.
//
// Prefix tokens (P of them in front of the grid tokens of every (batch, head)): the keys
// of a window are the P prefix tokens followed by the window's own tokens, and one more
// "window" (blockIdx.y == number of windows) holds the P prefix queries, whose keys are
// all P + N tokens.
#include "common.cuh"

namespace jv {
namespace {

constexpr int kRows = 8;    // query rows (= warps) per block
constexpr int kTile = 32;   // keys per shared-memory tile (= one per lane)
constexpr int kMaxD = 128;

template <typename T>
__global__ void __launch_bounds__(kRows * 32)
attn_generic_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                    T* __restrict__ o, int Hg, int Wg, int D, int P, int wh, int ww, int nwx, int nwin, int win0, float scale) {
  extern __shared__ float smem[];
  const int DP = D + 1;                       // padded row: conflict-free column reads
  float* ks = smem;                           // [kTile][DP]
  float* vs = ks + kTile * DP;                // [kTile][DP]
  float* qs = vs + kTile * DP;                // [kRows][D]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int N = P + Hg * Wg;                                 // tokens per (batch, head)
  const int win = blockIdx.y + win0;                         // (win0: a launch may cover the prefix queries only)
  const bool prefix_rows = win == nwin;                      // the block row of the P prefix queries
  const int wy = win / nwx, wx = win % nwx;
  const int y0 = prefix_rows ? 0 : wy * wh, x0 = prefix_rows ? 0 : wx * ww;
  const int vh = min(wh, Hg - y0), vw = min(ww, Wg - x0);   // valid extent of this window
  const int nq = prefix_rows ? P : vh * vw;                  // query rows of this block row
  const int cnt = prefix_rows ? N : P + vh * vw;             // keys: prefix tokens first, then the window's tokens
  if (blockIdx.x * kRows >= nq) return;                      // whole block beyond a small edge window
  const size_t base = (size_t)blockIdx.z * N * D;
  // token index of key (or prefix query) c of this block row
  auto key_token = [&](int c) -> size_t {
    if (prefix_rows || c < P) return (size_t)c;
    const int g = c - P;
    return (size_t)(P + (y0 + g / vw) * Wg + x0 + g % vw);
  };

  const int row = blockIdx.x * kRows + warp;                 // local query index
  const bool row_ok = row < nq;
  const int qtok = row_ok ? (int)key_token(prefix_rows ? row : P + row) : 0;
  for (int e = lane; e < D; e += 32) qs[warp * D + e] = row_ok ? to_f32(q[base + (size_t)qtok * D + e]) : 0.f;

  float m = -INFINITY, l = 0.f;
  float acc[kMaxD / 32];
#pragma unroll
  for (int i = 0; i < kMaxD / 32; ++i) acc[i] = 0.f;

  for (int t0 = 0; t0 < cnt; t0 += kTile) {
    __syncthreads();   // previous tile fully consumed (and qs written, first time round)
    for (int idx = threadIdx.x; idx < kTile * D; idx += blockDim.x) {
      const int j = idx / D, e = idx % D;
      const int c = t0 + j;
      float kv = 0.f, vv = 0.f;
      if (c < cnt) {
        const size_t tok = key_token(c);
        kv = to_f32(k[base + tok * D + e]);
        vv = to_f32(v[base + tok * D + e]);
      }
      ks[j * DP + e] = kv;
      vs[j * DP + e] = vv;
    }
    __syncthreads();

    float s = 0.f;
    for (int e = 0; e < D; ++e) s = fmaf(qs[warp * D + e], ks[lane * DP + e], s);
    s = (t0 + lane < cnt) ? s * scale : -INFINITY;
    const float m_new = fmaxf(m, warp_max(s));     // finite: every tile holds >= 1 valid key
    const float alpha = expf(m - m_new);           // exp(-inf) = 0 on the first tile
    const float p = expf(s - m_new);
    l = l * alpha + warp_sum(p);
    m = m_new;
#pragma unroll
    for (int i = 0; i < kMaxD / 32; ++i) acc[i] *= alpha;
    for (int j = 0; j < kTile; ++j) {
      const float pj = __shfl_sync(0xffffffffu, p, j);
#pragma unroll
      for (int i = 0; i < kMaxD / 32; ++i) {
        const int e = lane + 32 * i;
        if (e < D) acc[i] = fmaf(pj, vs[j * DP + e], acc[i]);
      }
    }
  }
  if (row_ok) {
    const float inv = 1.f / l;
#pragma unroll
    for (int i = 0; i < kMaxD / 32; ++i) {
      const int e = lane + 32 * i;
      if (e < D) from_f32(&o[base + (size_t)qtok * D + e], acc[i] * inv);
    }
  }
}

}  // namespace

// prefix_rows_only: just the P prefix queries (the windows themselves are served by another kernel,
// the one enqueued right before this call: the launch is programmatic, so that the two may overlap;
// neither reads what the other writes).
cudaError_t launch_attn_generic(const AttnArgs& a, cudaStream_t st, bool prefix_rows_only) {
  const int wh = a.wh < a.Hg ? a.wh : a.Hg, ww = a.ww < a.Wg ? a.ww : a.Wg;
  const int nwy = ceil_div(a.Hg, wh), nwx = ceil_div(a.Wg, ww);
  const int rows_max = (prefix_rows_only || a.P > wh * ww) ? a.P : wh * ww;
  const int win0 = prefix_rows_only ? nwy * nwx : 0;
  dim3 grid(ceil_div(rows_max, kRows), prefix_rows_only ? 1 : nwy * nwx + (a.P > 0 ? 1 : 0), a.BH);
  const size_t smem = (size_t)(2 * kTile * (a.D + 1) + kRows * a.D) * sizeof(float);
  if (prefix_rows_only) {
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kRows * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e;
    if (a.dtype == JV_F32)
      e = cudaLaunchKernelEx(&cfg, attn_generic_kernel<float>, (const float*)a.q, (const float*)a.k, (const float*)a.v, (float*)a.o,
                             a.Hg, a.Wg, a.D, a.P, wh, ww, nwx, nwy * nwx, win0, a.scale);
    else
      e = cudaLaunchKernelEx(&cfg, attn_generic_kernel<__nv_bfloat16>, (const __nv_bfloat16*)a.q, (const __nv_bfloat16*)a.k,
                             (const __nv_bfloat16*)a.v, (__nv_bfloat16*)a.o, a.Hg, a.Wg, a.D, a.P, wh, ww, nwx, nwy * nwx, win0,
                             a.scale);
    count_launch();
    return e;
  }
  if (a.dtype == JV_F32)
    attn_generic_kernel<float><<<grid, kRows * 32, smem, st>>>(
        (const float*)a.q, (const float*)a.k, (const float*)a.v, (float*)a.o, a.Hg, a.Wg, a.D, a.P, wh, ww, nwx, nwy * nwx, win0, a.scale);
  else
    attn_generic_kernel<__nv_bfloat16><<<grid, kRows * 32, smem, st>>>(
        (const __nv_bfloat16*)a.q, (const __nv_bfloat16*)a.k, (const __nv_bfloat16*)a.v,
        (__nv_bfloat16*)a.o, a.Hg, a.Wg, a.D, a.P, wh, ww, nwx, nwy * nwx, win0, a.scale);
  count_launch();
  return cudaGetLastError();
}

}  // namespace jv
