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
#include <cooperative_groups.h>

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

// ---- the P prefix queries of W on their own (they attend all P + N tokens); bf16, head_dim 64 ----
// A handful of query rows against thousands of keys: the keys are what has to be spread, and the
// products are a job for the (legacy, warp-level) tensor-core path: mma.sync m16n8k16 with the
// query rows of a group (up to 16) as the M dimension.  A cluster of kPreSplit blocks serves one
// (batch, head) and group of rows; the 8 warps of each block take the 32-key tiles round-robin over
// the whole cluster.  Per tile a warp stages K and V (32 keys x 128 bytes each) in its own shared
// memory with coalesced loads, forms S = Q K^T (16 x 32) from fragments, updates the online softmax
// of its two rows per thread, and adds P V with P taken straight from the score fragments.  The
// partial results (maximum, sum, weighted V per row) are merged in two steps: the warps of a block
// through its shared memory, the blocks of the cluster through distributed shared memory, read by
// the cluster's first block.  No scratch in global memory, no atomics: bit-reproducible.
constexpr int kPreRows = 16;
constexpr int kPreSplit = 2;
constexpr int kPreD = 64;
constexpr int kPreStride = 144;                       // bytes per staged row: 128 + 16, fragment reads conflict-free

__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

__global__ void __launch_bounds__(256)
attn_prefix_rows_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                        const __nv_bfloat16* __restrict__ v, __nv_bfloat16* __restrict__ o, int N, int P, float scale_log2) {
  namespace cg = cooperative_groups;
  extern __shared__ __align__(16) unsigned char smem_pre[];
  unsigned char* qs = smem_pre;                                  // [16 rows][144 B]: the group's query rows (zeros past P)
  unsigned char* ks = qs + 16 * kPreStride;                      // [8 warps][32 keys][144 B]
  unsigned char* vs = ks + 8 * 32 * kPreStride;                  // [8 warps][32 keys][144 B]
  float* part = reinterpret_cast<float*>(vs + 8 * 32 * kPreStride);   // [8 warps][16 rows][2 + 64], then [16][2 + 64] merged
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  cg::cluster_group cluster = cg::this_cluster();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, tq = lane & 3;
  const int split = blockIdx.x % kPreSplit;                      // this block's rank in its cluster
  const int r0 = blockIdx.y * kPreRows, nr = min(kPreRows, P - r0);
  const size_t base = (size_t)(blockIdx.x / kPreSplit) * N * kPreD;

  for (int i = threadIdx.x; i < 16 * 8; i += 256) {              // 16 rows x 8 chunks of 16 bytes
    const int r = i >> 3, c = i & 7;
    const uint4 x = r < nr ? *reinterpret_cast<const uint4*>(q + base + (size_t)(r0 + r) * kPreD + 8 * c) : make_uint4(0u, 0u, 0u, 0u);
    *reinterpret_cast<uint4*>(qs + r * kPreStride + 16 * c) = x;
  }
  __syncthreads();
  uint32_t qa[4][4];                                             // A fragments of Q: [k step][reg]
#pragma unroll
  for (int ks4 = 0; ks4 < 4; ++ks4) {
    qa[ks4][0] = *reinterpret_cast<const uint32_t*>(qs + g * kPreStride + (16 * ks4 + 2 * tq) * 2);
    qa[ks4][1] = *reinterpret_cast<const uint32_t*>(qs + (g + 8) * kPreStride + (16 * ks4 + 2 * tq) * 2);
    qa[ks4][2] = *reinterpret_cast<const uint32_t*>(qs + g * kPreStride + (16 * ks4 + 8 + 2 * tq) * 2);
    qa[ks4][3] = *reinterpret_cast<const uint32_t*>(qs + (g + 8) * kPreStride + (16 * ks4 + 8 + 2 * tq) * 2);
  }
  unsigned char* kw = ks + warp * 32 * kPreStride;
  unsigned char* vw = vs + warp * 32 * kPreStride;
  float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};        // rows g and g + 8
  float oacc[8][4];                                              // [n tile of 8 channels][c0..c3]
#pragma unroll
  for (int j = 0; j < 8; ++j)
#pragma unroll
    for (int c = 0; c < 4; ++c) oacc[j][c] = 0.f;

  for (int t0 = (split * 8 + warp) * 32; t0 < N; t0 += kPreSplit * 8 * 32) {
    // stage the tile: 32 keys x 8 chunks of K and of V, zeros past the last key
    __syncwarp();
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int idx = lane + 32 * i, key = idx >> 3, c = idx & 7;
      const bool in = t0 + key < N;
      const size_t off = base + (size_t)(t0 + key) * kPreD + 8 * c;
      *reinterpret_cast<uint4*>(kw + key * kPreStride + 16 * c) = in ? *reinterpret_cast<const uint4*>(k + off) : make_uint4(0u, 0u, 0u, 0u);
      *reinterpret_cast<uint4*>(vw + key * kPreStride + 16 * c) = in ? *reinterpret_cast<const uint4*>(v + off) : make_uint4(0u, 0u, 0u, 0u);
    }
    __syncwarp();
    // S = Q K^T: 4 n tiles of 8 keys
    float sc[4][4];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
#pragma unroll
      for (int c = 0; c < 4; ++c) sc[nt][c] = 0.f;
#pragma unroll
      for (int ks4 = 0; ks4 < 4; ++ks4) {
        const unsigned char* kr = kw + (8 * nt + g) * kPreStride + (16 * ks4 + 2 * tq) * 2;
        mma16816(sc[nt], qa[ks4], *reinterpret_cast<const uint32_t*>(kr), *reinterpret_cast<const uint32_t*>(kr + 16));
      }
    }
    // online softmax of rows g (c0, c1) and g + 8 (c2, c3); key of element c: t0 + 8 nt + 2 tq + (c & 1)
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const bool in = t0 + 8 * nt + 2 * tq + (c & 1) < N;
        sc[nt][c] = in ? sc[nt][c] * scale_log2 : -INFINITY;
        mx[c >> 1] = fmaxf(mx[c >> 1], sc[nt][c]);
      }
    float alpha[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
      const float m_new = fmaxf(m[h], mx[h]);                    // finite: the tile holds at least one key
      alpha[h] = exp2f(m[h] - m_new);
      m[h] = m_new;
    }
    float ls[2] = {0.f, 0.f};
    uint32_t pa[2][4];                                           // A fragments of P: [k step of 16 keys][reg]
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      const float p0 = exp2f(sc[nt][0] - m[0]), p1 = exp2f(sc[nt][1] - m[0]);
      const float p2 = exp2f(sc[nt][2] - m[1]), p3 = exp2f(sc[nt][3] - m[1]);
      ls[0] += p0 + p1;
      ls[1] += p2 + p3;
      pa[nt >> 1][(nt & 1) * 2] = pack_bf16x2(p0, p1);           // row g, keys 8 nt + 2 tq ..
      pa[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16x2(p2, p3);       // row g + 8
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      ls[h] += __shfl_xor_sync(0xffffffffu, ls[h], 1);
      ls[h] += __shfl_xor_sync(0xffffffffu, ls[h], 2);
      l[h] = l[h] * alpha[h] + ls[h];
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      oacc[j][0] *= alpha[0]; oacc[j][1] *= alpha[0];
      oacc[j][2] *= alpha[1]; oacc[j][3] *= alpha[1];
    }
    // O += P V: B[k = key][n = channel] gathered from the staged V rows
#pragma unroll
    for (int kk = 0; kk < 2; ++kk)
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const unsigned char* vr = vw + (16 * kk + 2 * tq) * kPreStride + (8 * j + g) * 2;
        const uint32_t b0 = (uint32_t)*reinterpret_cast<const unsigned short*>(vr) |
                            ((uint32_t)*reinterpret_cast<const unsigned short*>(vr + kPreStride) << 16);
        const uint32_t b1 = (uint32_t)*reinterpret_cast<const unsigned short*>(vr + 8 * kPreStride) |
                            ((uint32_t)*reinterpret_cast<const unsigned short*>(vr + 9 * kPreStride) << 16);
        mma16816(oacc[j], pa[kk], b0, b1);
      }
  }
  // merge, step 1: the eight warps of this block -> one partial per row in this block's shared memory
  constexpr int stride = 2 + kPreD;
  __syncthreads();
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    float* dst = part + (warp * kPreRows + g + 8 * h) * stride;
    if (tq == 0) { dst[0] = m[h]; dst[1] = l[h]; }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      dst[2 + 8 * j + 2 * tq] = oacc[j][2 * h];
      dst[2 + 8 * j + 2 * tq + 1] = oacc[j][2 * h + 1];
    }
  }
  __syncthreads();
  float* mine = part + 8 * kPreRows * stride;          // [kPreRows][2 + 64]: this block's merged partial
  for (int r = warp; r < kPreRows; r += 8) {           // a warp merges rows warp and warp + 8; a lane owns two channels
    float M = -INFINITY;
    for (int w = 0; w < 8; ++w) M = fmaxf(M, part[(w * kPreRows + r) * stride]);
    float L = 0.f, out0 = 0.f, out1 = 0.f;
    for (int w = 0; w < 8; ++w) {
      const float* src = part + (w * kPreRows + r) * stride;
      const float f = src[0] == -INFINITY ? 0.f : exp2f(src[0] - M);   // a warp that saw no key
      L = fmaf(src[1], f, L);
      out0 = fmaf(src[2 + lane], f, out0);
      out1 = fmaf(src[2 + 32 + lane], f, out1);
    }
    if (lane == 0) { mine[r * stride] = M; mine[r * stride + 1] = L; }
    mine[r * stride + 2 + lane] = out0;
    mine[r * stride + 2 + 32 + lane] = out1;
  }
  // step 2: the blocks of the cluster, read by its first block through distributed shared memory
  cluster.sync();
  if (split == 0) {
    for (int r = warp; r < nr; r += 8) {
      float M = -INFINITY;
      for (int c = 0; c < kPreSplit; ++c) M = fmaxf(M, cluster.map_shared_rank(mine, c)[r * stride]);
      float L = 0.f, out0 = 0.f, out1 = 0.f;
      for (int c = 0; c < kPreSplit; ++c) {
        const float* src = cluster.map_shared_rank(mine, c) + r * stride;
        const float mc = src[0];
        const float f = mc == -INFINITY ? 0.f : exp2f(mc - M);         // a block that saw no key
        L = fmaf(src[1], f, L);
        out0 = fmaf(src[2 + lane], f, out0);
        out1 = fmaf(src[2 + 32 + lane], f, out1);
      }
      const float inv = 1.f / L;
      __nv_bfloat16* dst = o + base + (size_t)(r0 + r) * kPreD;
      dst[lane] = __float2bfloat16_rn(out0 * inv);
      dst[32 + lane] = __float2bfloat16_rn(out1 * inv);
    }
  }
  cluster.sync();                                      // no block leaves while its shared memory may still be read
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
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = kPreSplit;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.BH * kPreSplit, ceil_div(a.P, kPreRows));
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = (size_t)(16 + 2 * 8 * 32) * kPreStride + (size_t)9 * kPreRows * (2 + kPreD) * sizeof(float);
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (a.dtype != JV_BF16 || a.D != kPreD) return cudaErrorNotSupported;   // (the caller is the bf16 tensor-core path)
    static OncePerDevice smem_opt_in;
    cudaError_t e = smem_opt_in.run([&] {
      return cudaFuncSetAttribute(attn_prefix_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cfg.dynamicSmemBytes);
    });
    if (e != cudaSuccess) return e;
    e = cudaLaunchKernelEx(&cfg, attn_prefix_rows_kernel, (const __nv_bfloat16*)a.q, (const __nv_bfloat16*)a.k,
                           (const __nv_bfloat16*)a.v, (__nv_bfloat16*)a.o, a.P + a.Hg * a.Wg, a.P, a.scale * 1.4426950408889634f);
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
