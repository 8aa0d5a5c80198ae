// bf16 tensor-core path of the linear-attention block (Sec. 3.2.1, Eq. 2
// reordered, Eq. 4), head_dim 64.
//
// The block is bound by HBM traffic (read K, V, Q once, write O once), but only
// if the two 64x64 contractions per token run on tensor cores: at ~32 flop per
// byte they would otherwise exceed the fp32 ALU rate.  Both passes therefore
// stream 64-token tiles through a cp.async ring into XOR-swizzled shared memory
// and feed mma.sync m16n8k16 (bf16 in, fp32 accumulate) via ldmatrix.
//
//   pass 1  lin_state_kernel   per (head, token chunk):  KV = relu(K)^T V, z = relu(K)^T 1,
//                              (v-sum when the dynamic convolution is on) -> fp32 partials
//   pass 2  launch_lin_reduce  fixed-order sum of the chunk partials (bit-reproducible)
//   pass 3  lin_apply_kernel   o = relu(q) KV / (relu(q).z + eps): KV as bf16 MMA operand,
//                              the denominator exactly in fp32 from the A fragments
//   pass 4  dwc_add_kernel     (only with the dynamic convolution) o += DWC_w(V)
//
// Fast-path partial / state layout per (batch, head), in floats:
//   [0, 4096) KV[a][e], [4096, 4160) z[a], [4160, 4224) vsum[e]
#include "common.cuh"

namespace jv {
namespace {

constexpr int kD = 64;
constexpr int kTileTok = 64;                  // tokens per shared-memory tile
constexpr int kTileBytes = kTileTok * kD * 2; // 8 KB
constexpr int kStateFloats = kD * kD + 2 * kD;
constexpr int kOffZ = kD * kD, kOffVsum = kD * kD + kD;
constexpr int kThreads = 128;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;   // size 0: the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t relu_bf16x2(uint32_t x) {
  __nv_bfloat162 v = *reinterpret_cast<__nv_bfloat162*>(&x);
  v = __hmax2(v, __float2bfloat162_rn(0.f));
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float2 bf16x2_to_f2(uint32_t x) {
  return __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&x));
}

// Byte offset of 16-byte chunk `ch` (0..7) of row `row` in a [rows][64 bf16] tile whose
// chunks are XOR-swizzled by the row index, so that ldmatrix reads hit 8 distinct banks groups.
__device__ __forceinline__ uint32_t tile_off(int row, int ch) { return (uint32_t)(row * 128 + ((ch ^ (row & 7)) << 4)); }

// One 64-token tile of a [.., 64] bf16 tensor -> shared memory; rows >= rows_valid are zero-filled.
__device__ __forceinline__ void load_tile(uint32_t dst, const __nv_bfloat16* src, int rows_valid) {
#pragma unroll
  for (int i = 0; i < (kTileTok * 8) / kThreads; ++i) {
    const int c = threadIdx.x + kThreads * i, row = c >> 3, ch = c & 7;
    const bool ok = row < rows_valid;
    cp_async16(dst + tile_off(row, ch), src + (ok ? (size_t)row * kD + ch * 8 : 0), ok);
  }
}

// ---- pass 1: partial state of one token chunk ------------------------------------
template <bool kVsum>
__global__ void __launch_bounds__(kThreads)
lin_state_kernel(const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v,
                 float* __restrict__ partial, int N, int chunk_tokens, int state_elems) {
  constexpr int kStages = 3;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const uint32_t smem = smem_u32(smem_raw);     // stage s: K tile at s*16K, V tile at s*16K + 8K
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.y, chunk = blockIdx.x;
  const int t_begin = chunk * chunk_tokens, t_end = min(N, t_begin + chunk_tokens);
  const int ntiles = (t_end - t_begin + kTileTok - 1) / kTileTok;
  const __nv_bfloat16* kb = k + ((size_t)bh * N + t_begin) * kD;
  const __nv_bfloat16* vb = v + ((size_t)bh * N + t_begin) * kD;

  auto issue = [&](int tile) {
    if (tile < ntiles) {
      const uint32_t st = smem + (tile % kStages) * 2 * kTileBytes;
      const int valid = min(kTileTok, t_end - t_begin - tile * kTileTok);
      load_tile(st, kb + (size_t)tile * kTileTok * kD, valid);
      load_tile(st + kTileBytes, vb + (size_t)tile * kTileTok * kD, valid);
    }
    cp_async_commit();
  };

  float acc[9][4];
#pragma unroll
  for (int j = 0; j < 9; ++j)
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[j][i] = 0.f;
  float vs0 = 0.f, vs1 = 0.f;
  // B fragment of the "ones" column: B[k][n] = 1 for n == 0 -> held by lanes 0..3
  const uint32_t ones = (lane < 4) ? 0x3F803F80u : 0u;

#pragma unroll
  for (int s = 0; s < kStages - 1; ++s) issue(s);

  for (int it = 0; it < ntiles; ++it) {
    cp_async_wait<kStages - 2>();
    __syncthreads();
    issue(it + kStages - 1);
    const uint32_t ks = smem + (it % kStages) * 2 * kTileBytes, vsm = ks + kTileBytes;
#pragma unroll
    for (int kk = 0; kk < kTileTok / 16; ++kk) {
      uint32_t a[4];
      {  // A = relu(K)^T: rows a = 16*warp.., cols = tokens; K is stored [token][a] -> .trans
        const int t = kk * 16 + (lane & 7) + ((lane >> 4) & 1) * 8;
        ldmatrix_x4_trans(a, ks + tile_off(t, 2 * warp + ((lane >> 3) & 1)));
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = relu_bf16x2(a[i]);
      }
      const int tb = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
      for (int jp = 0; jp < 4; ++jp) {
        uint32_t b[4];   // V stored [token][e]: B[k = token][n = e] -> .trans; two n-tiles per load
        ldmatrix_x4_trans(b, vsm + tile_off(tb, 2 * jp + (lane >> 4)));
        mma_bf16(acc[2 * jp], a, b[0], b[1]);
        mma_bf16(acc[2 * jp + 1], a, b[2], b[3]);
        if (kVsum && jp == warp) {   // this warp sums columns 16*warp .. 16*warp+15 of V
          const float2 x0 = bf16x2_to_f2(b[0]), x1 = bf16x2_to_f2(b[1]);
          const float2 y0 = bf16x2_to_f2(b[2]), y1 = bf16x2_to_f2(b[3]);
          vs0 += (x0.x + x0.y) + (x1.x + x1.y);
          vs1 += (y0.x + y0.y) + (y1.x + y1.y);
        }
      }
      mma_bf16(acc[8], a, ones, ones);
    }
  }
  cp_async_wait<0>();

  float* out = partial + ((size_t)bh * gridDim.x + chunk) * state_elems;
  const int g = lane >> 2, tq = lane & 3;
  const int a0 = 16 * warp + g;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    *reinterpret_cast<float2*>(out + a0 * kD + 8 * j + 2 * tq) = make_float2(acc[j][0], acc[j][1]);
    *reinterpret_cast<float2*>(out + (a0 + 8) * kD + 8 * j + 2 * tq) = make_float2(acc[j][2], acc[j][3]);
  }
  if (tq == 0) {
    out[kOffZ + a0] = acc[8][0];
    out[kOffZ + a0 + 8] = acc[8][2];
  }
  if (kVsum) {
    vs0 += __shfl_xor_sync(0xffffffffu, vs0, 1);
    vs0 += __shfl_xor_sync(0xffffffffu, vs0, 2);
    vs1 += __shfl_xor_sync(0xffffffffu, vs1, 1);
    vs1 += __shfl_xor_sync(0xffffffffu, vs1, 2);
    if (tq == 0) {
      out[kOffVsum + 16 * warp + g] = vs0;
      out[kOffVsum + 16 * warp + 8 + g] = vs1;
    }
  } else if (threadIdx.x < kD) {
    out[kOffVsum + threadIdx.x] = 0.f;
  }
}

// ---- pass 3: streaming apply -----------------------------------------------------
__global__ void __launch_bounds__(kThreads)
lin_apply_kernel(const __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ o,
                 const float* __restrict__ state, int N, int cta_tokens, int state_elems, float eps) {
  constexpr int kStages = 3;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const uint32_t smem = smem_u32(smem_raw);
  const uint32_t kv_sm = smem + kStages * kTileBytes;            // bf16 KV[a][e], swizzled, 8 KB
  float* z_sm = reinterpret_cast<float*>(smem_raw + (kStages + 1) * kTileBytes);   // 64 floats
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.y;
  const int t_begin = blockIdx.x * cta_tokens, t_end = min(N, t_begin + cta_tokens);
  const int ntiles = (t_end - t_begin + kTileTok - 1) / kTileTok;
  const __nv_bfloat16* qb = q + ((size_t)bh * N + t_begin) * kD;
  __nv_bfloat16* ob = o + ((size_t)bh * N + t_begin) * kD;

  auto issue = [&](int tile) {
    if (tile < ntiles)
      load_tile(smem + (tile % kStages) * kTileBytes, qb + (size_t)tile * kTileTok * kD,
                min(kTileTok, t_end - t_begin - tile * kTileTok));
    cp_async_commit();
  };
#pragma unroll
  for (int s = 0; s < kStages - 1; ++s) issue(s);

  {  // state -> shared memory: KV rounded to bf16 (MMA operand), z kept in fp32
    const float* S = state + (size_t)bh * state_elems;
#pragma unroll
    for (int i = 0; i < (kD * 8) / kThreads; ++i) {
      const int c = threadIdx.x + kThreads * i, row = c >> 3, ch = c & 7;
      const float4 x = *reinterpret_cast<const float4*>(S + row * kD + ch * 8);
      const float4 y = *reinterpret_cast<const float4*>(S + row * kD + ch * 8 + 4);
      __nv_bfloat162 p0 = __floats2bfloat162_rn(x.x, x.y), p1 = __floats2bfloat162_rn(x.z, x.w);
      __nv_bfloat162 p2 = __floats2bfloat162_rn(y.x, y.y), p3 = __floats2bfloat162_rn(y.z, y.w);
      uint4 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&p0);
      pk.y = *reinterpret_cast<uint32_t*>(&p1);
      pk.z = *reinterpret_cast<uint32_t*>(&p2);
      pk.w = *reinterpret_cast<uint32_t*>(&p3);
      *reinterpret_cast<uint4*>(smem_raw + kStages * kTileBytes + tile_off(row, ch)) = pk;
    }
    if (threadIdx.x < kD) z_sm[threadIdx.x] = S[kOffZ + threadIdx.x];
  }
  __syncthreads();

  const int g = lane >> 2, tq = lane & 3;
  float zr[16];   // z at the 16 k-indices this thread's A fragments cover
#pragma unroll
  for (int kk = 0; kk < 4; ++kk) {
    zr[4 * kk + 0] = z_sm[16 * kk + 2 * tq];
    zr[4 * kk + 1] = z_sm[16 * kk + 2 * tq + 1];
    zr[4 * kk + 2] = z_sm[16 * kk + 8 + 2 * tq];
    zr[4 * kk + 3] = z_sm[16 * kk + 8 + 2 * tq + 1];
  }

  for (int it = 0; it < ntiles; ++it) {
    cp_async_wait<kStages - 2>();
    __syncthreads();
    issue(it + kStages - 1);
    const uint32_t qs = smem + (it % kStages) * kTileBytes;
    unsigned char* qs_ptr = smem_raw + (it % kStages) * kTileBytes;

    float acc[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[j][i] = 0.f;
    float den_lo = 0.f, den_hi = 0.f;
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      uint32_t a[4];   // A = relu(Q): rows = tokens 16*warp.., cols = a
      ldmatrix_x4(a, qs + tile_off(16 * warp + (lane & 7) + ((lane >> 3) & 1) * 8, 2 * kk + (lane >> 4)));
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = relu_bf16x2(a[i]);
      {  // denominator relu(q).z in fp32, from the same fragments
        const float2 f0 = bf16x2_to_f2(a[0]), f1 = bf16x2_to_f2(a[1]);
        const float2 f2 = bf16x2_to_f2(a[2]), f3 = bf16x2_to_f2(a[3]);
        den_lo = fmaf(f0.x, zr[4 * kk], fmaf(f0.y, zr[4 * kk + 1], den_lo));
        den_lo = fmaf(f2.x, zr[4 * kk + 2], fmaf(f2.y, zr[4 * kk + 3], den_lo));
        den_hi = fmaf(f1.x, zr[4 * kk], fmaf(f1.y, zr[4 * kk + 1], den_hi));
        den_hi = fmaf(f3.x, zr[4 * kk + 2], fmaf(f3.y, zr[4 * kk + 3], den_hi));
      }
      const int ab = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
      for (int jp = 0; jp < 4; ++jp) {
        uint32_t b[4];   // KV stored [a][e]: B[k = a][n = e] -> .trans
        ldmatrix_x4_trans(b, kv_sm + tile_off(ab, 2 * jp + (lane >> 4)));
        mma_bf16(acc[2 * jp], a, b[0], b[1]);
        mma_bf16(acc[2 * jp + 1], a, b[2], b[3]);
      }
    }
    den_lo += __shfl_xor_sync(0xffffffffu, den_lo, 1);
    den_lo += __shfl_xor_sync(0xffffffffu, den_lo, 2);
    den_hi += __shfl_xor_sync(0xffffffffu, den_hi, 1);
    den_hi += __shfl_xor_sync(0xffffffffu, den_hi, 2);
    const float inv_lo = 1.f / (den_lo + eps), inv_hi = 1.f / (den_hi + eps);

    // Stage the warp's 16 output rows over its own (now consumed) Q rows, then store 16 B per lane.
    __syncwarp();
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(acc[j][0] * inv_lo, acc[j][1] * inv_lo);
      __nv_bfloat162 hi = __floats2bfloat162_rn(acc[j][2] * inv_hi, acc[j][3] * inv_hi);
      *reinterpret_cast<__nv_bfloat162*>(qs_ptr + tile_off(16 * warp + g, j) + 4 * tq) = lo;
      *reinterpret_cast<__nv_bfloat162*>(qs_ptr + tile_off(16 * warp + g + 8, j) + 4 * tq) = hi;
    }
    __syncwarp();
    const int rows_valid = t_end - t_begin - it * kTileTok;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int c = lane + 32 * i, row = 16 * warp + (c >> 3), ch = c & 7;
      if (row < rows_valid)
        *reinterpret_cast<uint4*>(ob + ((size_t)it * kTileTok + row) * kD + ch * 8) =
            *reinterpret_cast<const uint4*>(qs_ptr + tile_off(row, ch));
    }
  }
  cp_async_wait<0>();
}

// ---- pass 4: o += depth-wise k x k convolution of V with the sample's kernels ------
// One warp walks a run of consecutive tokens of one head; lane owns channels 2*lane, 2*lane+1.
template <int K>
__global__ void __launch_bounds__(256)
dwc_add_kernel(const __nv_bfloat16* __restrict__ v, __nv_bfloat16* __restrict__ o, const float* __restrict__ w,
               int H, int Hg, int Wg, int run) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int N = Hg * Wg, bh = blockIdx.y, b = bh / H, h = bh % H;
  const int t0 = (blockIdx.x * 8 + warp) * run;
  if (t0 >= N) return;
  const int t1 = min(N, t0 + run);
  constexpr int P = (K - 1) / 2;
  float w0[K * K], w1[K * K];
  const float* wp = w + ((size_t)b * H * kD + (size_t)h * kD + 2 * lane) * K * K;
#pragma unroll
  for (int i = 0; i < K * K; ++i) { w0[i] = wp[i]; w1[i] = wp[K * K + i]; }
  const __nv_bfloat16* vb = v + (size_t)bh * N * kD + 2 * lane;
  __nv_bfloat16* ob = o + (size_t)bh * N * kD + 2 * lane;
  for (int t = t0; t < t1; ++t) {
    const int y = t / Wg, x = t % Wg;
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int dy = 0; dy < K; ++dy) {
      const int yy = y + dy - P;
      if (yy < 0 || yy >= Hg) continue;
#pragma unroll
      for (int dx = 0; dx < K; ++dx) {
        const int xx = x + dx - P;
        if (xx < 0 || xx >= Wg) continue;
        const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(vb + (size_t)(yy * Wg + xx) * kD));
        s0 = fmaf(w0[dy * K + dx], f.x, s0);
        s1 = fmaf(w1[dy * K + dx], f.y, s1);
      }
    }
    __nv_bfloat162* op = reinterpret_cast<__nv_bfloat162*>(ob + (size_t)t * kD);
    const float2 cur = __bfloat1622float2(*op);
    *op = __floats2bfloat162_rn(cur.x + s0, cur.y + s1);
  }
}

}  // namespace

bool linear_fast_supported(const LinArgs& a) {
  return a.s.dtype == JV_BF16 && a.s.D == kD;
}

cudaError_t launch_linear_fast(const LinArgs& a, const LinPlan& p, cudaStream_t st) {
  const jv_shape& s = a.s;
  const int N = s.Hg * s.Wg, BH = s.B * s.H;
  char* ws = (char*)a.ws;
  float* partial = (float*)(ws + p.off_partial);
  float* state = (float*)(ws + p.off_state);
  const __nv_bfloat16* q = (const __nv_bfloat16*)a.q;
  const __nv_bfloat16* k = (const __nv_bfloat16*)a.k;
  const __nv_bfloat16* v = (const __nv_bfloat16*)a.v;
  __nv_bfloat16* o = (__nv_bfloat16*)a.o;

  static bool attr_done = false;   // > 48 KB of dynamic shared memory needs the opt-in, once per process
  const size_t smem1 = 3 * 2 * kTileBytes, smem3 = 4 * kTileBytes + kD * sizeof(float);
  if (!attr_done) {
    cudaFuncSetAttribute(lin_state_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1);
    cudaFuncSetAttribute(lin_state_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1);
    attr_done = true;
  }
  dim3 g1(p.nchunk, BH);
  if (a.dwc)
    lin_state_kernel<true><<<g1, kThreads, smem1, st>>>(k, v, partial, N, p.chunk_tokens, p.state_elems);
  else
    lin_state_kernel<false><<<g1, kThreads, smem1, st>>>(k, v, partial, N, p.chunk_tokens, p.state_elems);
  count_launch();
  cudaError_t e = launch_lin_reduce(partial, state, p.nchunk, p.state_elems, (size_t)BH * p.state_elems, st);
  if (e != cudaSuccess) return e;
  const int cta_tokens = 512;
  dim3 g3(ceil_div(N, cta_tokens), BH);
  lin_apply_kernel<<<g3, kThreads, smem3, st>>>(q, o, state, N, cta_tokens, p.state_elems, a.eps);
  count_launch();
  if (a.dwc) {
    e = launch_dwc_generator(a, p, state + kOffVsum, p.state_elems, st);
    if (e != cudaSuccess) return e;
    const float* w = (const float*)(ws + p.off_kernel);
    const int run = 32;
    dim3 g4(ceil_div(ceil_div(N, run), 8), BH);
    if (a.dwc->k == 3)
      dwc_add_kernel<3><<<g4, 256, 0, st>>>(v, o, w, s.H, s.Hg, s.Wg, run);
    else
      dwc_add_kernel<5><<<g4, 256, 0, st>>>(v, o, w, s.H, s.Hg, s.Wg, run);
    count_launch();
  }
  return cudaGetLastError();
}

}  // namespace jv
