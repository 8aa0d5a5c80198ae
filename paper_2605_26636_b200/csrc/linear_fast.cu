// bf16 tensor-core path of the linear-attention block (Sec. 3.2.1, Eq. 2
// reordered, Eq. 4), head_dim 64.
//
// The block is bound by HBM traffic (read K, V, Q once, write O once; V a second
// time, mostly from L2, when the squeeze dynamic convolution is on), but only if the
// two 64x64 contractions per token run on tensor cores: at ~32 flop per byte they
// would otherwise exceed the fp32 ALU rate.  Two kernels, each a one-wave grid of
// CTAs that stream token tiles through a TMA + mbarrier ring (one producer warp, four
// worker warps; 128-byte-swizzled tiles feed ldmatrix / the tensor core without bank conflicts):
//
//   lin_state_kernel   per (head, token chunk):  KV = relu(K)^T V, z = relu(K)^T 1,
//                      (v-sum when the convolution is on) -> fp32 chunk partials
//   lin_apply_kernel   sums the chunk partials of its head in a fixed order (the
//                      deterministic second pass: no floating-point atomics), then
//                      o = relu(q) KV / (relu(q).z + eps) per 128-token tile: ReLU in
//                      place in shared memory, relu(Q) KV as tcgen05.mma with the
//                      accumulator in tensor memory (KV as bf16 operand), the
//                      denominator exactly in fp32, output written back by TMA stores.
//
// The apply kernel is launched with programmatic stream serialisation: its set-up and
// its first Q loads overlap the tail of the state kernel, and it waits for that grid
// (griddepcontrol.wait) only before touching the partials.
//
// With the convolution on, the generator's two layers (tiny kernels laid out for latency) run
// between the state pass and the apply pass.  3 x 3 kernels: the apply pass is the fused
// apply + convolution kernel of linear_conv.cu.  5 x 5 kernels: the apply pass above, the output
// layer beside it, and a read-modify-write convolution pass over o behind both.
//
// Partial layout per (batch, head, chunk), in floats:
//   [0, 4096) KV[a][e], [4096, 4160) z[a], [4160, 4224) vsum[e]

#include "lin_common.cuh"

namespace jv {
namespace {

using namespace tc;
using namespace lin;

constexpr int kTileTok = 64;                  // tokens per shared-memory tile
constexpr int kTileBytes = kTileTok * kD * 2; // 8 KB
constexpr int kConsumers = 128;               // 4 MMA warps
constexpr int kThreads = kConsumers + 32;     // + 1 producer warp

// A box of tokens x 64 channels of an input tensor (channel, token, head, batch) -> shared memory
// (128-byte swizzle); tokens past N arrive as zeros.
__device__ __forceinline__ void tma_load_tile(uint32_t dst, const CUtensorMap* map, uint64_t* bar, int tok, int h, int b) {
  tma_load_4d(dst, map, bar, 0, tok, h, b);
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
struct __align__(8) Ring {
  uint64_t full[8], empty[8];
  volatile uint32_t abort_flag;
};

// ---- pass 1: partial state of one token chunk ------------------------------------
constexpr int kStateStages = 6;               // 6 x (K tile + V tile) = 96 KB per CTA, two CTAs per SM
constexpr size_t kStateSmem = (size_t)kStateStages * 2 * kTileBytes + 1024 + sizeof(Ring);

template <bool kVsum>
__global__ void __launch_bounds__(kThreads)
lin_state_kernel(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
                 float* __restrict__ partial, int* status, int N, int chunk_tokens, int state_elems, int H) {
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment by an offset from the array itself, so that accesses stay shared-space loads and stores
  unsigned char* smem_al = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t smem = smem_u32(smem_al);      // stage s: K tile at s * 16 KB, V tile at s * 16 KB + 8 KB
  Ring* ring = reinterpret_cast<Ring*>(smem_al + (size_t)kStateStages * 2 * kTileBytes);
  const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;
  const int bh = blockIdx.y, chunk = blockIdx.x;
  const int in_b = bh / H, in_h = bh - in_b * H;      // coordinates of the input tensor maps
  const int t_begin = chunk * chunk_tokens, t_end = min(N, t_begin + chunk_tokens);
  const int ntiles = (t_end - t_begin + kTileTok - 1) / kTileTok;

  // let the grid that depends on this one (the apply pass) start its set-up as SMs free up
  griddep_launch_dependents();

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStateStages; ++s) {
      mbar_init(&ring->full[s], 1);
      mbar_init(&ring->empty[s], 4);          // one arrival per MMA warp
    }
    ring->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  if (*reinterpret_cast<volatile int*>(status) != 0) return;   // an earlier kernel gave up: leave at once

  if (warp == 4) {
    // ================= TMA producer =================
    // K is read exactly once in the whole call: it makes room in L2 first.  With the convolution
    // on, V is read again by the apply pass: L2 is asked to keep it.
    const uint64_t pol_k = l2_policy_evict_first(), pol_v = l2_policy_evict_last();
    int s = 0;
    uint32_t par = 1;
    int issued = 0;
    bool ok = true;
    for (int it = 0; it < ntiles; ++it) {
      ok = warp_wait(&ring->empty[s], par, &ring->abort_flag, status);
      if (!ok) break;
      if (elect_one()) {
        mbar_expect_tx(&ring->full[s], 2 * kTileBytes);
        const int tok = t_begin + it * kTileTok;     // a chunk's last tile may run past t_end: only by whole
        tma_load_4d_hint(smem + s * 2 * kTileBytes, &mapK, &ring->full[s], 0, tok, in_h, in_b, pol_k);   // zero rows past N
        if (kVsum) tma_load_4d_hint(smem + s * 2 * kTileBytes + kTileBytes, &mapV, &ring->full[s], 0, tok, in_h, in_b, pol_v);
        else tma_load_tile(smem + s * 2 * kTileBytes + kTileBytes, &mapV, &ring->full[s], tok, in_h, in_b);
      }
      __syncwarp();
      ++issued;
      if (++s == kStateStages) { s = 0; par ^= 1; }
    }
    if (!ok && lane == 0) {   // let the copies in flight land before the CTA leaves
      const unsigned long long t0 = globaltimer();
      for (int g = max(0, issued - kStateStages); g < issued; ++g)
        while (!mbar_try(&ring->full[g % kStateStages], (g / kStateStages) & 1) && globaltimer() - t0 < kWaitLimitNs) {}
    }
    return;
  }

  // ================= MMA warps: warp w owns rows 16 w .. 16 w + 15 of KV =================
  float acc[9][4];
#pragma unroll
  for (int j = 0; j < 9; ++j)
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[j][i] = 0.f;
  float vs0 = 0.f, vs1 = 0.f;
  // B fragment of the "ones" column: B[k][n] = 1 for n == 0 -> held by lanes 0..3
  const uint32_t ones = (lane < 4) ? 0x3F803F80u : 0u;

  int s = 0;
  uint32_t par = 0;
  bool ok = true;
  for (int it = 0; it < ntiles; ++it) {
    ok = warp_wait(&ring->full[s], par, &ring->abort_flag, status);
    if (!ok) break;
    const uint32_t ks = smem + s * 2 * kTileBytes, vsm = ks + kTileBytes;
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
    __syncwarp();
    if (lane == 0) mbar_arrive(&ring->empty[s]);
    if (++s == kStateStages) { s = 0; par ^= 1; }
  }
  if (!ok) return;

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
  }
}

// ---- pass 2: deterministic sum of the chunk partials, then the streaming apply ----------
// 128-token tiles.  Per tile: TMA brings Q in; the four worker warps apply ReLU in place (one
// thread per token row, which also gives that row's denominator relu(q).z exactly in fp32);
// one elected thread issues O_tile = relu(Q) KV as four tcgen05.mma (M128 N64 K16, A = Q tile
// K-major, B = bf16 KV MN-major, accumulator in tensor memory); the same thread-per-row
// mapping reads the accumulator back, divides, rounds to bf16 and stages its row; each warp
// writes its 32 rows with one TMA store.  Accumulators and staging are double-buffered so the
// MMA of tile i + 1 runs under the epilogue of tile i.
constexpr int kApplyTok = 128;                          // tokens per apply tile
constexpr int kApplyTileBytes = kApplyTok * kD * 2;     // 16 KB
constexpr int kApplyStages = 4;                         // Q ring
constexpr uint32_t kApplyTmemCols = 128;                // two 64-column fp32 accumulators
struct __align__(8) ApplyBars {
  uint64_t full[kApplyStages], empty[kApplyStages];
  uint64_t d_full[2];                         // accumulator of tile i ready (tcgen05.commit)
  uint64_t workers;                           // the 128 worker threads among themselves (once, after the state is in place)
  uint64_t relu_done[kApplyStages];           // 128 arrivals: the Q tile in this ring slot is rectified, its denominators stored
  uint64_t d_empty[2];                        // 128 arrivals: the epilogue has read this accumulator buffer
  uint32_t tmem_base;
  volatile uint32_t abort_flag;
};
constexpr int kApplyThreads = 288;                      // 4 rectifier warps, 1 producer / issuer warp, 4 epilogue warps
constexpr int kDenRing = 8;                             // denominators of the tiles between ReLU and epilogue
// shared memory: Q ring | output staging 2 x 16 KB | KV (bf16, swizzled) | z (fp32) | denominators | barriers
constexpr size_t kApplySmem = (size_t)(kApplyStages + 2) * kApplyTileBytes + kTileBytes + 1024 + kD * sizeof(float) +
                              (size_t)kDenRing * kApplyTok * sizeof(float) + sizeof(ApplyBars);

// Instruction descriptor, kind::f16: D fp32, A and B bf16, B MN-major, M = 128, N = 64.
constexpr uint32_t kIdescApply = idesc(128, 64, 1);
__global__ void __launch_bounds__(kApplyThreads, 2)
lin_apply_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapO,
                 const float* __restrict__ partial, int* status, int N, int span_tokens, int nchunk, int state_elems,
                 float eps, int H) {
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment by an offset from the array itself, so that accesses stay shared-space loads and stores
  unsigned char* smem_al = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t smem = smem_u32(smem_al);                                       // Q ring
  unsigned char* out_ptr = smem_al + (size_t)kApplyStages * kApplyTileBytes;     // 2 staging tiles
  const uint32_t out_sm = smem + kApplyStages * kApplyTileBytes;
  unsigned char* kv_ptr = out_ptr + 2 * kApplyTileBytes;                         // bf16 KV[a][e], swizzled
  const uint32_t kv_sm = out_sm + 2 * kApplyTileBytes;
  float* z_sm = reinterpret_cast<float*>(kv_ptr + kTileBytes);
  float* den_sm = z_sm + kD;                                                     // [kDenRing][128]
  ApplyBars* bars = reinterpret_cast<ApplyBars*>(den_sm + kDenRing * kApplyTok);
  const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;
  const int bh = blockIdx.y;
  const int t_begin = blockIdx.x * span_tokens, t_end = min(N, t_begin + span_tokens);
  const int ntiles = (t_end - t_begin + kApplyTok - 1) / kApplyTok;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kApplyStages; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1);          // released by the commit that follows the tile's MMAs
    }
    mbar_init(&bars->d_full[0], 1);
    mbar_init(&bars->d_full[1], 1);
    mbar_init(&bars->workers, kConsumers);
    for (int s = 0; s < kApplyStages; ++s) mbar_init(&bars->relu_done[s], kConsumers);
    mbar_init(&bars->d_empty[0], kConsumers);
    mbar_init(&bars->d_empty[1], kConsumers);
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)),
                 "r"(kApplyTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = __shfl_sync(0xffffffffu, bars->tmem_base, 0);

  // A grid launched behind this one with programmatic serialisation (the output layer of the
  // convolution's generator) may start once this grid lets its dependents go.  It reads what the
  // grids before this one wrote, so no warp here does that before it knows that those grids are
  // complete: the rectifier warps after their griddepcontrol.wait, the other warps after the first
  // barrier that the rectifier warps have arrived on.

  if (warp == 4) {
    // ================= TMA producer and MMA issuer (one elected lane) =================
    // Q does not depend on the state pass: the first loads start at once.  Per tile: refill the
    // ring slot freed by the previous tile's MMAs, wait until the workers have rectified the tile
    // (and are done with the accumulator buffer it will overwrite), issue its four MMAs.
    bool ok = true;
    int issued = 0;
    auto load_tile = [&](int it) {
      if (elect_one()) {
        const int s = it % kApplyStages;
        mbar_expect_tx(&bars->full[s], kApplyTileBytes);
        tma_load_tile(smem + s * kApplyTileBytes, &mapQ, &bars->full[s], t_begin + it * kApplyTok, bh % H, bh / H);
      }
      __syncwarp();
      ++issued;
    };
    for (int it = 0; it < kApplyStages - 1 && it < ntiles; ++it) load_tile(it);
    for (int it = 0; it < ntiles; ++it) {
      const int nx = it + kApplyStages - 1;            // goes into the slot of tile it - 1
      if (nx < ntiles) {
        if (it > 0) {
          ok = warp_wait(&bars->empty[nx % kApplyStages], ((it - 1) / kApplyStages) & 1, &bars->abort_flag, status);
          if (!ok) break;
        }
        load_tile(nx);
      }
      const int s = it % kApplyStages, b = it & 1;
      ok = warp_wait(&bars->relu_done[s], (it / kApplyStages) & 1, &bars->abort_flag, status);
      if (it == 0) griddep_launch_dependents();
      if (ok && it >= 2) ok = warp_wait(&bars->d_empty[b], ((it >> 1) - 1) & 1, &bars->abort_flag, status);
      if (!ok) break;
      tc_fence_after();
      const uint32_t qa = smem + s * kApplyTileBytes;
#pragma unroll
      for (int ks = 0; ks < kD / 16; ++ks) {
        if (elect_one())
          asm volatile(
              "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
              "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
              ::"r"(tmem + b * kD), "l"(smem_desc(qa + ks * 32)), "l"(smem_desc(kv_sm + ks * 2048)), "r"(kIdescApply),
                "r"(ks > 0 ? 1u : 0u) : "memory");
      }
      if (elect_one()) {
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&bars->d_full[b])) : "memory");
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&bars->empty[s])) : "memory");
      }
      __syncwarp();
    }
    if (!ok && lane == 0) {
      const unsigned long long t0 = globaltimer();
      for (int g = max(0, issued - kApplyStages); g < issued; ++g)
        while (!mbar_try(&bars->full[g % kApplyStages], (g / kApplyStages) & 1) && globaltimer() - t0 < kWaitLimitNs) {}
    }
  } else if (warp < 4) {
    // ================= rectifier warps: thread r = 32 warp + lane owns token row r of every tile =================
    griddep_wait();                                    // the grids before this one (state pass, generator's hidden layer) are complete
    griddep_launch_dependents();
    bool ok = *reinterpret_cast<volatile int*>(status) == 0;
    if (!ok) bars->abort_flag = 1;                     // an earlier kernel gave up: every role of this CTA falls through at once
    {  // second pass of the reduction: chunk partials summed in a fixed order; KV -> bf16 MMA operand, z in fp32
      const float* P = partial + (size_t)bh * nchunk * state_elems;
#pragma unroll
      for (int i = 0; i < (kD * 8) / kConsumers; ++i) {
        const int c = threadIdx.x + kConsumers * i, row = c >> 3, ch = c & 7;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f), y = x;
        for (int k0 = 0; k0 < nchunk; k0 += 4) {       // four chunks' loads in flight, summed in chunk order
          float4 xa[4], ya[4];
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const bool in = k0 + k < nchunk;
            const float* src = P + (size_t)(in ? k0 + k : 0) * state_elems + row * kD + ch * 8;
            xa[k] = in ? *reinterpret_cast<const float4*>(src) : make_float4(0.f, 0.f, 0.f, 0.f);
            ya[k] = in ? *reinterpret_cast<const float4*>(src + 4) : make_float4(0.f, 0.f, 0.f, 0.f);
          }
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            x.x += xa[k].x; x.y += xa[k].y; x.z += xa[k].z; x.w += xa[k].w;
            y.x += ya[k].x; y.y += ya[k].y; y.z += ya[k].z; y.w += ya[k].w;
          }
        }
        __nv_bfloat162 p0 = __floats2bfloat162_rn(x.x, x.y), p1 = __floats2bfloat162_rn(x.z, x.w);
        __nv_bfloat162 p2 = __floats2bfloat162_rn(y.x, y.y), p3 = __floats2bfloat162_rn(y.z, y.w);
        uint4 pk;
        pk.x = *reinterpret_cast<uint32_t*>(&p0);
        pk.y = *reinterpret_cast<uint32_t*>(&p1);
        pk.z = *reinterpret_cast<uint32_t*>(&p2);
        pk.w = *reinterpret_cast<uint32_t*>(&p3);
        *reinterpret_cast<uint4*>(kv_ptr + tile_off(row, ch)) = pk;
      }
      if (threadIdx.x < kD) {
        float zs = 0.f;
        for (int k = 0; k < nchunk; ++k) zs += P[(size_t)k * state_elems + kOffZ + threadIdx.x];
        z_sm[threadIdx.x] = zs;
      }
    }
    uint32_t wpar = 0;
    // all 128 worker threads; makes their shared-memory writes visible to the tensor core / TMA
    auto workers_sync = [&]() -> bool {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      tc_fence_before();
      mbar_arrive(&bars->workers);
      const bool w_ok = warp_wait(&bars->workers, wpar, &bars->abort_flag, status);
      wpar ^= 1;
      tc_fence_after();
      return w_ok;
    };
    const int row = threadIdx.x;                       // 0..127: token row of the tile

    // ReLU of this thread's row of the Q tile in stage s, in place; returns relu(q).z.
    // All loads come before the stores (the compiler cannot tell that they do not alias).
    auto relu_row = [&](int s) -> float {
      unsigned char* q = smem_al + (size_t)s * kApplyTileBytes + row * 128;
      uint4 v[8];
#pragma unroll
      for (int c = 0; c < 8; ++c) v[c] = *reinterpret_cast<const uint4*>(q + ((c ^ (row & 7)) << 4));
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        v[c].x = relu_bf16x2(v[c].x); v[c].y = relu_bf16x2(v[c].y); v[c].z = relu_bf16x2(v[c].z); v[c].w = relu_bf16x2(v[c].w);
        const float4 za = *reinterpret_cast<const float4*>(z_sm + 8 * c), zb = *reinterpret_cast<const float4*>(z_sm + 8 * c + 4);
        const float2 f0 = bf16x2_to_f2(v[c].x), f1 = bf16x2_to_f2(v[c].y), f2 = bf16x2_to_f2(v[c].z), f3 = bf16x2_to_f2(v[c].w);
        acc[0] = fmaf(f0.x, za.x, fmaf(f0.y, za.y, acc[0]));
        acc[1] = fmaf(f1.x, za.z, fmaf(f1.y, za.w, acc[1]));
        acc[2] = fmaf(f2.x, zb.x, fmaf(f2.y, zb.y, acc[2]));
        acc[3] = fmaf(f3.x, zb.z, fmaf(f3.y, zb.w, acc[3]));
      }
#pragma unroll
      for (int c = 0; c < 8; ++c) *reinterpret_cast<uint4*>(q + ((c ^ (row & 7)) << 4)) = v[c];
      return (acc[0] + acc[1]) + (acc[2] + acc[3]);
    };
    // this thread's row of the tile in ring slot s is rectified and its denominator stored
    auto publish_relu = [&](int s) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(&bars->relu_done[s]);
    };

    ok = workers_sync() && ok;                         // KV and z written by all
    int s = 0;
    uint32_t par = 0;
    for (int it = 0; it < ntiles && ok; ++it) {
      ok = warp_wait(&bars->full[s], par, &bars->abort_flag, status);
      if (!ok) break;
      den_sm[(it & (kDenRing - 1)) * kApplyTok + row] = relu_row(s);
      publish_relu(s);
      if (++s == kApplyStages) { s = 0; par ^= 1; }
    }
  } else {
    // ================= epilogue warps: thread (quadrant q = warp % 4, lane) owns row 32 q + lane =================
    const int q4 = warp & 3, row = 32 * q4 + lane;
    const uint32_t lane_base = (uint32_t)(q4 << 5) << 16;
    bool ok = true;
    for (int it = 0; it < ntiles && ok; ++it) {
      const int b = it & 1;
      // The tile's MMAs were issued after all 128 rectifier threads had published its rows and
      // denominators, so the accumulator being complete means the denominators are in place.
      ok = warp_wait(&bars->d_full[b], (it >> 1) & 1, &bars->abort_flag, status);
      if (it == 0) griddep_launch_dependents();
      if (!ok) break;
      tc_fence_after();
      const float inv = 1.f / (den_sm[(it & (kDenRing - 1)) * kApplyTok + row] + eps);
      uint32_t v0[32], v1[32];
      tmem_ld32(tmem + lane_base + b * kD, v0);
      tmem_ld32(tmem + lane_base + b * kD + 32, v1);
      tmem_wait_ld(v0);
      tmem_wait_ld(v1);
      tc_fence_before();
      mbar_arrive(&bars->d_empty[b]);                  // the accumulator buffer may be overwritten
      // this warp's staging region (32 rows, 4 KB) of buffer b: its last store must have been read
      if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
      __syncwarp();
      unsigned char* st = out_ptr + b * kApplyTileBytes + row * 128;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint32_t* v = c < 4 ? v0 + 8 * c : v1 + 8 * (c - 4);
        uint4 w;
        __nv_bfloat162 h0 = __floats2bfloat162_rn(__uint_as_float(v[0]) * inv, __uint_as_float(v[1]) * inv);
        __nv_bfloat162 h1 = __floats2bfloat162_rn(__uint_as_float(v[2]) * inv, __uint_as_float(v[3]) * inv);
        __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(v[4]) * inv, __uint_as_float(v[5]) * inv);
        __nv_bfloat162 h3 = __floats2bfloat162_rn(__uint_as_float(v[6]) * inv, __uint_as_float(v[7]) * inv);
        w.x = *reinterpret_cast<uint32_t*>(&h0);
        w.y = *reinterpret_cast<uint32_t*>(&h1);
        w.z = *reinterpret_cast<uint32_t*>(&h2);
        w.w = *reinterpret_cast<uint32_t*>(&h3);
        *reinterpret_cast<uint4*>(st + ((c ^ (row & 7)) << 4)) = w;
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) {
        const int tok = t_begin + it * kApplyTok + 32 * q4;
        if (tok < N)        // rows past N inside the box are clipped by the store itself
          asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
                       ::"l"(&mapO), "r"(out_sm + b * kApplyTileBytes + q4 * 4096), "r"(0), "r"(tok), "r"(bh) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      }
    }
    // the staging tiles must outlive the reads of the last stores
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    // every MMA issued has been waited for (d_full) unless a wait gave up; in that case give the
    // tensor core a bounded time before tensor memory is released
    if (!ok && lane == 0) {
      const unsigned long long t0 = globaltimer();
      while (globaltimer() - t0 < 1000000ull) {}
    }
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kApplyTmemCols) : "memory");
}

// ---- o += depth-wise k x k convolution of V with the sample's kernels ------------------
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

// ---- kernel generator of the squeeze dynamic convolution (Sec. 3.2.1), tuned for latency ------
// Both layers sit on the critical path between the state pass and the apply pass, so each is laid
// out as ONE round trip of independent loads followed by arithmetic.
//
// hidden[b][r] = SiLU(b1[r] + sum_c W1[r][c] * mean_v[b][c]).  A block serves 8 values of r for one
// sample: per tile of 1024 channels it forms the means (the chunk partials' v-sums, summed in chunk
// order) in shared memory while the rows of W1 are already on their way, then warp w takes row r0 + w.
constexpr int kGenTile = 1024;
__global__ void __launch_bounds__(256)
gen_hidden_kernel(const float* __restrict__ partial, const float* __restrict__ W1, const float* __restrict__ b1,
                  float* __restrict__ hidden, int H, int R, int nchunk, int state_elems, float inv_n, int early_trigger,
                  const __nv_bfloat16* __restrict__ v, int P, int ntok) {
  __shared__ __align__(16) float s_sm[kGenTile];
  // early_trigger: the grids behind this one each wait for their predecessor before they read its
  // output, so they may be resident (set up, prefetching inputs of the call) while this one waits.
  if (early_trigger) griddep_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = blockIdx.x * 8 + warp, b = blockIdx.y, C = H * kD;
  const bool r_ok = r < R;
  const float* wrow = W1 + (size_t)(r_ok ? r : 0) * C;
  float dot = 0.f;
  bool waited = false;
  for (int c0 = 0; c0 < C; c0 += kGenTile) {           // C is a multiple of 64
    float4 wv[kGenTile / 128];                         // this lane's part of the row: W1 is an input of the call
#pragma unroll
    for (int i = 0; i < kGenTile / 128; ++i) {
      const int c = c0 + 4 * lane + 128 * i;
      wv[i] = (r_ok && c < C) ? __ldg(reinterpret_cast<const float4*>(wrow + c)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (!waited) {
      griddep_wait();                                  // the state pass is complete
      if (!early_trigger) griddep_launch_dependents(); // the apply grid may set up and load Q meanwhile
      waited = true;
    }
    __syncthreads();                                   // the previous tile's means have been consumed
#pragma unroll
    for (int i = 0; i < kGenTile / 256; ++i) {
      const int c = c0 + threadIdx.x + 256 * i;
      float m = 0.f;
      if (c < C) {
        const float* pv = partial + (size_t)(b * H + c / kD) * nchunk * state_elems + kOffVsum + c % kD;
        for (int k = 0; k < nchunk; ++k) m += __ldcg(pv + (size_t)k * state_elems);
        // the v-sums run over all tokens; the pooling is over the grid: take the prefix rows out again
        for (int t = 0; t < P; ++t) m -= __bfloat162float(v[((size_t)(b * H + c / kD) * ntok + t) * kD + c % kD]);
      }
      s_sm[threadIdx.x + 256 * i] = m * inv_n;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kGenTile / 128; ++i) {
      const float4 sv = *reinterpret_cast<const float4*>(s_sm + 4 * lane + 128 * i);
      dot = fmaf(wv[i].x, sv.x, fmaf(wv[i].y, sv.y, fmaf(wv[i].z, sv.z, fmaf(wv[i].w, sv.w, dot))));
    }
  }
  dot = warp_sum(dot);
  if (lane == 0 && r_ok) {
    const float x = dot + (b1 ? b1[r] : 0.f);
    hidden[(size_t)b * R + r] = x / (1.f + expf(-x));
  }
}
// w[b][t] = b2[t] + sum_r W2[t][r] * hidden[b][r]; 8 lanes per output t, 32 outputs per block, all
// samples (8 at a time, their hidden vectors in shared memory).  kVec (R a multiple of 4): a lane's
// part of the W2 row is fetched as float4, the whole row in flight at once.
template <bool kVec>
__global__ void __launch_bounds__(256)
gen_out_kernel(const float* __restrict__ hidden, const float* __restrict__ W2, const float* __restrict__ b2,
               float* __restrict__ w, int B, int T, int R, int wait_first) {
  extern __shared__ __align__(16) float h_sm[];        // [min(B, 8)][R]: small, so that the grid can be resident early
  // wait_first = 0: launched behind the apply grid, which lets its dependents go only after it has
  // seen the hidden layer's grid complete: hidden is final here and this grid runs beside the apply
  // pass; it waits at its end (below).  wait_first = 1: launched directly behind the hidden layer
  // (or the state pass, with static kernels), ahead of the fused apply + convolution grid: it waits
  // for its predecessor before it reads hidden.
  griddep_launch_dependents();                         // the grid behind this one may set up and prefetch
  const int t = blockIdx.x * 32 + (threadIdx.x >> 3), part = threadIdx.x & 7;
  const bool t_ok = t < T;
  const float* wrow = W2 + (size_t)(t_ok ? t : 0) * R;
  constexpr int kPer = kVec ? 4 : 16;                  // loads per lane and 128 values of r
  bool waited = wait_first == 0;
  for (int b0 = 0; b0 < B; b0 += 8) {
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    const int nb = min(8, B - b0);
    for (int r0 = 0; r0 < R; r0 += 128) {
      float wv[16];                                    // W2 is an input of the call: on its way before the wait
      if (kVec) {
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
          const int r = r0 + 4 * part + 32 * i;
          const float4 x = r < R ? __ldg(reinterpret_cast<const float4*>(wrow + r)) : make_float4(0.f, 0.f, 0.f, 0.f);
          wv[4 * i] = x.x; wv[4 * i + 1] = x.y; wv[4 * i + 2] = x.z; wv[4 * i + 3] = x.w;
        }
      } else {
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
          const int r = r0 + part + 8 * i;
          wv[i] = r < R ? __ldg(wrow + r) : 0.f;
        }
      }
      if (r0 == 0) {                                   // this group of samples' hidden vectors -> shared memory
        if (!waited) { griddep_wait(); waited = true; }
        __syncthreads();
        for (int i = threadIdx.x; i < nb * R; i += 256) h_sm[i] = __ldcg(hidden + (size_t)b0 * R + i);
        __syncthreads();
      }
#pragma unroll
      for (int bb = 0; bb < 8; ++bb) {
        if (bb < nb) {
          const float* hp = h_sm + bb * R + r0;
          if (kVec) {
#pragma unroll
            for (int i = 0; i < kPer; ++i) {
              const int r = 4 * part + 32 * i;
              if (r0 + r < R) {
                const float4 hv = *reinterpret_cast<const float4*>(hp + r);
                acc[bb] = fmaf(wv[4 * i], hv.x, fmaf(wv[4 * i + 1], hv.y, fmaf(wv[4 * i + 2], hv.z, fmaf(wv[4 * i + 3], hv.w, acc[bb]))));
              }
            }
          } else {
#pragma unroll
            for (int i = 0; i < kPer; ++i) {
              const int r = part + 8 * i;
              if (r0 + r < R) acc[bb] = fmaf(wv[i], hp[r], acc[bb]);
            }
          }
        }
      }
    }
    if (R == 0 && !waited) { griddep_wait(); waited = true; }   // static kernels: nothing to read, but completion must chain
#pragma unroll
    for (int bb = 0; bb < 8; ++bb) {
      float sres = acc[bb];
      sres += __shfl_xor_sync(0xffffffffu, sres, 1);
      sres += __shfl_xor_sync(0xffffffffu, sres, 2);
      sres += __shfl_xor_sync(0xffffffffu, sres, 4);
      if (t_ok && part == 0 && bb < nb) w[(size_t)(b0 + bb) * T + t] = sres + (b2 ? b2[t] : 0.f);
    }
  }
  // wait_first = 0: the convolution pass is launched behind this grid and adds into what the apply
  // pass writes: this grid must not retire before the apply grid has.
  if (!wait_first) griddep_wait();
}

}  // namespace

bool linear_fast_supported(const LinArgs& a) {
  if (a.dwc && a.dwc->token_wise && !dwc_tokenwise_fast_supported(a)) return false;
  if (a.dwc && a.s.P > 0 && a.dwc->k != 3) return false;   // prefix tokens + 5 x 5 kernels: the generic kernels
  // inputs with the caller's strides: only what reads them through tensor maps (the passes of the
  // attention proper and the fused 3 x 3 convolution; the pooling's prefix correction reads V directly)
  if (in_strided(a.s) && a.dwc && (a.dwc->token_wise || a.dwc->k != 3 || a.s.P > 0)) return false;
  return a.s.dtype == JV_BF16 && a.s.D == kD && encode_fn() != nullptr;
}

cudaError_t launch_linear_fast(const LinArgs& a, const LinPlan& p, cudaStream_t st) {
  const jv_shape& s = a.s;
  const int N = shape_tokens(s), BH = s.B * s.H;       // the state and the attention proper run over all tokens
  char* ws = (char*)a.ws;
  float* partial = (float*)(ws + p.off_partial);
  int* status = device_status_ptr();
  if (!status) return cudaErrorUnknown;
  if (a.dwc && a.dwc->token_wise) {
    // token-wise dynamic convolution: the attention proper as without a convolution, then o += the
    // convolution of V with every token's own kernels (generator as two tensor-core GEMMs)
    LinArgs plain = a;
    plain.dwc = nullptr;
    const cudaError_t e0 = launch_linear_fast(plain, p, st);
    if (e0 != cudaSuccess) return e0;
    return launch_dwc_tokenwise_fast(a, p, status, st);
  }

  CUtensorMap mq, mk, mv, mo;
  const InStrides in = in_strides(s);
  if (!make_map_tokens_in(&mq, a.q, s.B, s.H, N, kApplyTok, in) || !make_map_tokens_in(&mk, a.k, s.B, s.H, N, kTileTok, in) ||
      !make_map_tokens_in(&mv, a.v, s.B, s.H, N, kTileTok, in) || !make_map_tokens(&mo, a.o, BH, N, 32, N))
    return cudaErrorInvalidValue;

  static OncePerDevice smem_opt_in;   // > 48 KB of dynamic shared memory: a per-device function attribute
  cudaError_t e = smem_opt_in.run([] {
    cudaError_t r;
    if ((r = cudaFuncSetAttribute(lin_state_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStateSmem)) != cudaSuccess) return r;
    if ((r = cudaFuncSetAttribute(lin_state_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStateSmem)) != cudaSuccess) return r;
    return cudaFuncSetAttribute(lin_apply_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kApplySmem);
  });
  if (e != cudaSuccess) return e;
  const int num_sms = device_sm_count();
  dim3 g1(p.nchunk, BH);
  if (a.dwc)
    lin_state_kernel<true><<<g1, kThreads, kStateSmem, st>>>(mk, mv, partial, status, N, p.chunk_tokens, p.state_elems, (int)s.H);
  else
    lin_state_kernel<false><<<g1, kThreads, kStateSmem, st>>>(mk, mv, partial, status, N, p.chunk_tokens, p.state_elems, (int)s.H);
  count_launch();
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;

  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;

  // With the convolution on, the generator's hidden layer (tiny; it needs the state pass only) goes
  // between the state pass and the apply pass, and its output layer behind the apply pass, beside
  // which it runs.  Every launch from here to the output layer uses programmatic serialisation;
  // each grid waits for its predecessor (griddepcontrol.wait) before it reads what that one wrote,
  // the output layer at its very end, so that stream order still means "apply pass complete" for
  // the convolution pass that follows it.
  // apply pass over the first ntokens tokens of every (batch, head): one wave of two CTAs per SM, spans
  // of whole 128-token tiles; launched so that its set-up overlaps the tail of the grid before it
  auto enqueue_apply = [&](const CUtensorMap& map_q, const CUtensorMap& map_o, int ntokens) -> cudaError_t {
    int nspan = (2 * num_sms) / BH;
    if (nspan < 1) nspan = 1;
    int span = ceil_div(ceil_div(ntokens, nspan), kApplyTok) * kApplyTok;
    if (span < 4 * kApplyTok) span = 4 * kApplyTok;
    nspan = ceil_div(ntokens, span);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(nspan, BH);
    cfg.blockDim = dim3(kApplyThreads);
    cfg.dynamicSmemBytes = kApplySmem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, lin_apply_kernel, map_q, map_o, (const float*)partial, status, ntokens,
                                               span, p.nchunk, p.state_elems, a.eps, (int)s.H);
    count_launch();
    return err;
  };

  float* hidden = (float*)(ws + p.off_hidden);
  const bool fused_conv = a.dwc && linear_conv_supported(a);
  if (fused_conv && s.P > 0) {
    // Prefix tokens: the convolution does not see them, their output is the attention output alone.
    // The plain apply pass over the first P tokens of every (batch, head), right behind the state pass
    // (which it waits for; the grids behind it wait for it in turn).
    CUtensorMap mqp, mop;
    if (!make_map_tokens_in(&mqp, a.q, s.B, s.H, s.P, kApplyTok, in) || !make_map_tokens(&mop, a.o, BH, s.P, 32, N))
      return cudaErrorInvalidValue;
    e = enqueue_apply(mqp, mop, s.P);
    if (e != cudaSuccess) return e;
  }
  if (a.dwc && a.dwc->R > 0) {      // R == 0: static kernels, the output layer just broadcasts b2
    const jv_dwc& d = *a.dwc;
    cudaLaunchConfig_t hcfg = {};
    hcfg.stream = st;
    hcfg.attrs = attr;
    hcfg.numAttrs = 1;
    hcfg.gridDim = dim3(ceil_div(d.R, 8), s.B);
    hcfg.blockDim = dim3(256);
    e = cudaLaunchKernelEx(&hcfg, gen_hidden_kernel, (const float*)partial, d.W1, d.b1, hidden, (int)s.H, (int)d.R,
                           p.nchunk, p.state_elems, 1.f / (float)(s.Hg * s.Wg), fused_conv ? 1 : 0, (const __nv_bfloat16*)a.v,
                           (int)s.P, N);
    count_launch();
    if (e != cudaSuccess) return e;
  }

  if (fused_conv) {
    // 3 x 3 kernels: state -> [hidden layer] -> output layer -> apply pass with the convolution fused in.
    // Every grid behind the state pass is launched with programmatic serialisation and waits for its
    // predecessor before it reads that one's output, so completion is transitive along the chain.
    const jv_dwc& d = *a.dwc;
    float* wk = (float*)(ws + p.off_kernel);
    const int T = s.H * kD * d.k * d.k;
    cudaLaunchConfig_t gcfg = {};
    gcfg.stream = st;
    gcfg.attrs = attr;
    gcfg.numAttrs = 1;
    gcfg.gridDim = dim3(ceil_div(T, 32));
    gcfg.blockDim = dim3(256);
    gcfg.dynamicSmemBytes = (size_t)(s.B < 8 ? s.B : 8) * d.R * sizeof(float);
    e = cudaLaunchKernelEx(&gcfg, (d.R % 4 == 0) ? gen_out_kernel<true> : gen_out_kernel<false>, (const float*)hidden, d.W2,
                           d.b2, wk, (int)s.B, T, (int)d.R, 1);
    count_launch();
    if (e != cudaSuccess) return e;
    return launch_linear_apply_conv(a, p, partial, wk, status, true, st);
  }

  e = enqueue_apply(mq, mo, N);
  if (e != cudaSuccess) return e;

  if (a.dwc) {
    const __nv_bfloat16* v = (const __nv_bfloat16*)a.v;
    __nv_bfloat16* o = (__nv_bfloat16*)a.o;
    const jv_dwc& d = *a.dwc;
    float* wk = (float*)(ws + p.off_kernel);
    const int T = s.H * kD * d.k * d.k;
    cudaLaunchConfig_t gcfg = {};
    gcfg.stream = st;
    gcfg.attrs = attr;
    gcfg.numAttrs = 1;
    gcfg.gridDim = dim3(ceil_div(T, 32));
    gcfg.blockDim = dim3(256);
    gcfg.dynamicSmemBytes = (size_t)(s.B < 8 ? s.B : 8) * d.R * sizeof(float);
    e = cudaLaunchKernelEx(&gcfg, (d.R % 4 == 0) ? gen_out_kernel<true> : gen_out_kernel<false>, (const float*)hidden, d.W2,
                           d.b2, wk, (int)s.B, T, (int)d.R, 0);
    count_launch();
    if (e != cudaSuccess) return e;
    const float* w = (const float*)(ws + p.off_kernel);
    const int run = 32;
    dim3 g4(ceil_div(ceil_div(N, run), 8), BH);
    // 5 x 5 kernels (3 x 3 ones took the fused path above): a read-modify-write pass over o
    if (a.dwc->k == 3) dwc_add_kernel<3><<<g4, 256, 0, st>>>(v, o, w, s.H, s.Hg, s.Wg, run);
    else
      dwc_add_kernel<5><<<g4, 256, 0, st>>>(v, o, w, s.H, s.Hg, s.Wg, run);
    count_launch();
  }
  return cudaGetLastError();
}

}  // namespace jv
