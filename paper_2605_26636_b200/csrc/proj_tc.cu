// The linear projections either side of a token mixer (the inherited W_Q, W_K, W_V and W_O
// of every block, Sec. 3.2.4) as tcgen05 GEMMs that read and write the mixers' [B, H, N, 64]
// layout directly, so that no transpose pass runs between the projection and the mixer.
//
//   qkv:  x [B, N, C] (C = H * 64)  times  w [3C, C]^T  ->  q, k, v [B, H, N, 64]
//         output feature f = which * C + h * 64 + e  (which: 0 = q, 1 = k, 2 = v)
//   out:  o [B, H, N, 64]  times  w [C, C]^T  ->  y [B, N, C]
//         input feature h * 64 + e: one K block of 64 is one head of o
//
// One persistent CTA per SM loops over output tiles of 128 tokens x 256 features (feature
// tile fastest, so the CTAs that run together share their token tile in L2 and the weights
// stay L2-resident).  Warp roles:
//   warp 0      TMA producer: A (128 tokens x 64) and B (256 features x 64) through a 4-stage ring
//   warp 1      MMA issuer: 4 x tcgen05.mma M128 N256 K16 per stage into one of two
//               accumulators in tensor memory (2 x 256 columns)
//   warps 4-7   epilogue of the other accumulator: tensor memory -> registers, + bias, bf16,
//               swizzled staging in shared memory, one TMA store per warp and 64-feature block
// Token tiles never cross a batch element: rows past N are zero-filled on load and clipped on
// store by TMA; feature blocks past the last one are skipped.
//
// Every mbarrier wait is bounded; a wait that runs out sets the device status word and the
// CTA's abort flag, and every role falls through to the teardown that frees tensor memory.
#include "tc_common.cuh"

namespace jv {
namespace {

using namespace tc;

constexpr int kD = 64;                       // head_dim = K block = feature block
constexpr int kBM = 128;                     // tokens per tile
constexpr int kBN = 256;                     // features per tile
constexpr int kABytes = kBM * kD * 2;        // 16 KB
constexpr int kBBytes = kBN * kD * 2;        // 32 KB
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kStages = 4;
constexpr int kThreads = 256;
constexpr uint32_t kTmemCols = 512;
constexpr int kStagingBytes = 32 * kD * 2;   // one warp's 32 tokens x 64 features

struct __align__(8) Barriers {
  uint64_t full[kStages], empty[kStages];
  uint64_t acc_full[2], acc_empty[2];
  uint64_t drain;
  uint32_t tmem_base;
  volatile uint32_t abort_flag;
};
constexpr size_t kSmemTiles = (size_t)kStages * kStageBytes + 4 * 2 * kStagingBytes;
constexpr size_t kSmemBytes = kSmemTiles + sizeof(Barriers) + 1024;

struct ProjParams {
  const float* bias;       // [features] or nullptr
  int* status;
  int tiles_m_per_batch;   // ceil(N / 128)
  int tiles_n;             // ceil(features / 256)
  int total_tiles;         // B * tiles_m_per_batch * tiles_n
  int kblocks;             // C / 64
  int H;                   // heads
  int fblocks;             // features / 64
  int N;                   // tokens per batch element
  int silu;                // 1: x / (1 + exp(-x)) on the result (the kernel generator's hidden layer)
  int out_f16;             // 1: the result is stored as fp16 instead of bf16 (same size; the generator's intermediates)
  uint32_t idesc;          // instruction descriptor: M128 N256, both operands K-major, bf16 or fp16 operands
};

// Instruction descriptor: M128 N256, both operands K-major; bf16 operands, or fp16 ones (format 0 in both fields)
constexpr uint32_t kIdesc = idesc(kBM, kBN, 0);
constexpr uint32_t kIdescF16 = kIdesc & ~((1u << 7) | (1u << 10));
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

struct Tile {
  int b, tok0, f0;   // batch element, first token, first feature
};
__device__ __forceinline__ Tile decode_tile(const ProjParams& p, int i) {
  const int tn = i % p.tiles_n, r = i / p.tiles_n;
  const int tm = r % p.tiles_m_per_batch, b = r / p.tiles_m_per_batch;
  return Tile{b, tm * kBM, tn * kBN};
}

// kQKV: A = x as (C, N, B), outputs q, k, v as (64, N, B*H); else A = o as (64, N, B*H),
// output y as (C, N, B).  B (the weights) is (C, features) in both.
template <bool kQKV>
__global__ void __launch_bounds__(kThreads, 1)
proj_tc_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
               const __grid_constant__ CUtensorMap mapD0, const __grid_constant__ CUtensorMap mapD1,
               const __grid_constant__ CUtensorMap mapD2, const ProjParams p) {
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment by an offset from the array itself, so that accesses stay shared-space loads and stores
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  Barriers* bar = reinterpret_cast<Barriers*>(smem + kSmemTiles);
  const uint32_t sRing = smem_u32(smem), sStage = sRing + kStages * kStageBytes;

  const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;

  // a timeout flagged earlier (by any CTA or launch) makes the rest leave at once
  if (threadIdx.x == 0) bar->tmem_base = *reinterpret_cast<volatile int*>(p.status);
  __syncthreads();
  if (bar->tmem_base != 0) return;
  __syncthreads();

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bar->full[s], 1);
      mbar_init(&bar->empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&bar->acc_full[a], 1);
      mbar_init(&bar->acc_empty[a], 4);      // lane 0 of each epilogue warp
    }
    mbar_init(&bar->drain, 1);
    bar->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bar->tmem_base)),
                 "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = __shfl_sync(0xffffffffu, bar->tmem_base, 0);

  const int tile0 = blockIdx.x, tile_step = gridDim.x;

  if (warp == 0) {
    // ================= TMA producer =================
    bool ok = true;
    int s = 0, issued = 0;
    uint32_t par = 1;
    for (int i = tile0; i < p.total_tiles && ok; i += tile_step) {
      const Tile t = decode_tile(p, i);
      for (int kb = 0; kb < p.kblocks; ++kb) {
        ok = warp_wait(&bar->empty[s], par, &bar->abort_flag, p.status);
        if (!ok) break;
        if (elect_one()) {
          const uint32_t dst = sRing + s * kStageBytes;
          mbar_expect_tx(&bar->full[s], kStageBytes);
          if (kQKV) tma_load_3d(dst, &mapA, &bar->full[s], kb * kD, t.tok0, t.b);
          else tma_load_3d(dst, &mapA, &bar->full[s], 0, t.tok0, t.b * p.H + kb % p.H);   // (more K blocks than planes: A repeats)
          tma_load_2d(dst + kABytes, &mapB, &bar->full[s], kb * kD, t.f0);
        }
        __syncwarp();
        ++issued;
        if (++s == kStages) { s = 0; par ^= 1; }
      }
    }
    if (!ok && lane == 0) {
      // let the copies still in flight land before the CTA leaves (bounded by the same limit)
      const unsigned long long t0 = globaltimer();
      for (int g = max(0, issued - kStages); g < issued; ++g)
        while (!mbar_try(&bar->full[g % kStages], (g / kStages) & 1) && globaltimer() - t0 < kWaitLimitNs) {}
    }
  } else if (warp == 1) {
    // ================= MMA issuer =================
    bool ok = true;
    int s = 0, n = 0;
    uint32_t ph = 0;
    for (int i = tile0; i < p.total_tiles && ok; i += tile_step, ++n) {
      const int a = n & 1;
      ok = warp_wait(&bar->acc_empty[a], ((n >> 1) & 1) ^ 1, &bar->abort_flag, p.status);   // epilogue has read tile n - 2
      if (!ok) break;
      tc_fence_after();
      const uint32_t d = tmem + a * kBN;
      for (int kb = 0; kb < p.kblocks; ++kb) {
        ok = warp_wait(&bar->full[s], ph, &bar->abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = sRing + s * kStageBytes, sb = sa + kABytes;
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks)
          mma_ss(d, smem_desc(sa + ks * 32), smem_desc(sb + ks * 32), p.idesc, (kb > 0 || ks > 0) ? 1u : 0u);
        tc_commit(&bar->empty[s]);
        if (++s == kStages) { s = 0; ph ^= 1; }
      }
      if (ok) tc_commit(&bar->acc_full[a]);
    }
    // every MMA issued so far must have retired before tensor memory is released
    tc_commit(&bar->drain);
    if (lane == 0) {
      const unsigned long long t0 = globaltimer();
      while (!mbar_try(&bar->drain, 0) && globaltimer() - t0 < kWaitLimitNs) {}
    }
    __syncwarp();
  } else if (warp >= 4) {
    // ================= epilogue: one thread per token row =================
    const int q4 = warp & 3;
    const uint32_t lane_base = (uint32_t)(q4 << 5) << 16;
    unsigned char* stage_ptr = smem + kStages * kStageBytes + q4 * 2 * kStagingBytes;
    const uint32_t stage_u32 = sStage + q4 * 2 * kStagingBytes;
    bool ok = true;
    int n = 0, nstore = 0;
    for (int i = tile0; i < p.total_tiles && ok; i += tile_step, ++n) {
      const Tile t = decode_tile(p, i);
      const int a = n & 1;
      ok = warp_wait(&bar->acc_full[a], (n >> 1) & 1, &bar->abort_flag, p.status);
      if (!ok) break;
      tc_fence_after();
      const int tok = t.tok0 + 32 * q4;
#pragma unroll 1
      for (int j = 0; j < kBN / kD; ++j) {
        const int fb = t.f0 / kD + j;
        if (fb >= p.fblocks || tok >= p.N) break;   // no such features / none of this warp's rows exists
        uint32_t ob[32];
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          uint32_t v[32];
          tmem_ld32(tmem + lane_base + a * kBN + j * kD + c * 32, v);
          tmem_wait_ld(v);
          if (p.silu) {
#pragma unroll
            for (int i2 = 0; i2 < 32; ++i2) {
              const float z = __uint_as_float(v[i2]) + (p.bias ? __ldg(p.bias + fb * kD + c * 32 + i2) : 0.f);
              v[i2] = __float_as_uint(z / (1.f + __expf(-z)));
            }
#pragma unroll
            for (int i2 = 0; i2 < 16; ++i2)
              ob[16 * c + i2] = p.out_f16 ? pack_f16(__uint_as_float(v[2 * i2]), __uint_as_float(v[2 * i2 + 1]))
                                          : pack_bf16(__uint_as_float(v[2 * i2]), __uint_as_float(v[2 * i2 + 1]));
          } else if (p.out_f16) {
#pragma unroll
            for (int i2 = 0; i2 < 16; ++i2) {
              const float b0 = p.bias ? __ldg(p.bias + fb * kD + c * 32 + 2 * i2) : 0.f;
              const float b1 = p.bias ? __ldg(p.bias + fb * kD + c * 32 + 2 * i2 + 1) : 0.f;
              ob[16 * c + i2] = pack_f16(__uint_as_float(v[2 * i2]) + b0, __uint_as_float(v[2 * i2 + 1]) + b1);
            }
          } else if (p.bias) {
            const float4* b4 = reinterpret_cast<const float4*>(p.bias + fb * kD + c * 32);
#pragma unroll
            for (int i4 = 0; i4 < 8; ++i4) {
              const float4 bb = __ldg(b4 + i4);
              ob[16 * c + 2 * i4] = pack_bf16(__uint_as_float(v[4 * i4]) + bb.x, __uint_as_float(v[4 * i4 + 1]) + bb.y);
              ob[16 * c + 2 * i4 + 1] = pack_bf16(__uint_as_float(v[4 * i4 + 2]) + bb.z, __uint_as_float(v[4 * i4 + 3]) + bb.w);
            }
          } else {
#pragma unroll
            for (int i2 = 0; i2 < 16; ++i2)
              ob[16 * c + i2] = pack_bf16(__uint_as_float(v[2 * i2]), __uint_as_float(v[2 * i2 + 1]));
          }
        }
        // the store issued two blocks ago must have finished reading this staging buffer
        const int sbuf = nstore & 1;
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        __syncwarp();
#pragma unroll
        for (int c = 0; c < 8; ++c)     // 16-byte chunk c of this row, at its 128-byte-swizzle position
          *reinterpret_cast<uint4*>(stage_ptr + sbuf * kStagingBytes + lane * 128 + ((c ^ (lane & 7)) << 4)) =
              make_uint4(ob[4 * c], ob[4 * c + 1], ob[4 * c + 2], ob[4 * c + 3]);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          const uint32_t src = stage_u32 + sbuf * kStagingBytes;
          if (kQKV) {
            const int which = fb / p.H, h = fb - which * p.H;
            const CUtensorMap* m = which == 0 ? &mapD0 : which == 1 ? &mapD1 : &mapD2;
            tma_store_3d(m, src, 0, tok, t.b * p.H + h);
          } else {
            tma_store_3d(&mapD0, src, fb * kD, tok, t.b);
          }
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
        ++nstore;
      }
      // this accumulator may be overwritten once all four warps have read it
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bar->acc_empty[a]);
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  // ================= common teardown =================
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

// ---- host side ----------------------------------------------------------------------
// bf16 tensor (inner, rows, outer), contiguous, with a box of (64, box_rows, 1)
bool map3(CUtensorMap* m, const void* ptr, uint64_t inner, uint64_t rows, uint64_t outer, uint32_t box_rows) {
  const cuuint64_t dims[3] = {inner, rows, outer};
  const cuuint64_t strides[2] = {inner * 2, inner * rows * 2};
  const cuuint32_t box[3] = {(cuuint32_t)kD, box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return encode_fn()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// bf16 matrix (inner, rows), contiguous, with a box of (64, box_rows)
bool map2(CUtensorMap* m, const void* ptr, uint64_t inner, uint64_t rows, uint32_t box_rows) {
  const cuuint64_t dims[2] = {inner, rows};
  const cuuint64_t strides[1] = {inner * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kD, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return encode_fn()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool proj_tc_available() { return encode_fn() != nullptr; }

static cudaError_t proj_opt_in() {   // > 48 KB of dynamic shared memory: a per-device function attribute
  static OncePerDevice once;
  return once.run([] {
    cudaError_t r = cudaFuncSetAttribute(proj_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (r == cudaSuccess)
      r = cudaFuncSetAttribute(proj_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    return r;
  });
}

// The kernel on its own terms (see common.cuh).  kQKV of the kernel means "A is [B, N, K]" for the loads
// and "D is planes" for the stores, which go together in the two projections; the other two
// combinations are reached through the plane count: with one K block per "head" ... the generator's
// GEMMs need A planes -> D rows (the out form, as it is) and A rows -> D planes (the qkv form with
// every feature block a plane of its own: H := F / 64, so that "which" is always 0).
cudaError_t launch_proj_gemm(bool planes_in, bool planes_out, const void* A, const void* W, const float* bias, void* D, int B,
                             int N, int kblocks, int a_planes, int F, bool silu, bool f16_in, bool f16_out, int* status,
                             cudaStream_t st) {
  if (!encode_fn() || planes_in == planes_out || F % kD != 0) return cudaErrorNotSupported;
  const uint64_t K = (uint64_t)kblocks * kD;
  CUtensorMap ma, mb, md;
  bool ok = map2(&mb, W, K, (uint64_t)F, kBN);
  if (planes_in) ok = ok && map3(&ma, A, kD, (uint64_t)N, (uint64_t)B * a_planes, kBM) && map3(&md, D, (uint64_t)F, (uint64_t)N, (uint64_t)B, 32);
  else ok = ok && map3(&ma, A, K, (uint64_t)N, (uint64_t)B, kBM) && map3(&md, D, kD, (uint64_t)N, (uint64_t)B * (F / kD), 32);
  if (!ok) return cudaErrorInvalidValue;
  cudaError_t e = proj_opt_in();
  if (e != cudaSuccess) return e;
  const int num_sms = device_sm_count();
  ProjParams p;
  p.bias = bias;
  p.status = status;
  p.tiles_m_per_batch = ceil_div(N, kBM);
  p.tiles_n = ceil_div(F, kBN);
  const int64_t total = (int64_t)B * p.tiles_m_per_batch * p.tiles_n;
  if (total > 0x7fffffffll) return cudaErrorInvalidValue;
  p.total_tiles = (int)total;
  p.kblocks = kblocks;
  p.H = planes_in ? a_planes : F / kD;
  p.fblocks = F / kD;
  p.N = N;
  p.silu = silu ? 1 : 0;
  p.out_f16 = f16_out ? 1 : 0;
  p.idesc = f16_in ? kIdescF16 : kIdesc;
  const int grid = p.total_tiles < num_sms ? p.total_tiles : num_sms;
  if (planes_in) proj_tc_kernel<false><<<grid, kThreads, kSmemBytes, st>>>(ma, mb, md, md, md, p);
  else proj_tc_kernel<true><<<grid, kThreads, kSmemBytes, st>>>(ma, mb, md, md, md, p);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_proj_tc(bool qkv, const void* x, const void* w, const float* bias, void* d0, void* d1, void* d2,
                           const jv_shape& s, int* status, cudaStream_t st) {
  if (!encode_fn()) return cudaErrorNotSupported;
  const uint64_t N = (uint64_t)shape_tokens(s), C = (uint64_t)s.H * kD, BH = (uint64_t)s.B * s.H;   // prefix and grid tokens alike
  const uint64_t features = qkv ? 3 * C : C;
  CUtensorMap ma, mb, md0, md1, md2;
  bool ok = map2(&mb, w, C, features, kBN);
  if (qkv) {
    ok = ok && map3(&ma, x, C, N, s.B, kBM) && map3(&md0, d0, kD, N, BH, 32) && map3(&md1, d1, kD, N, BH, 32) &&
         map3(&md2, d2, kD, N, BH, 32);
  } else {
    ok = ok && map3(&ma, x, kD, N, BH, kBM) && map3(&md0, d0, C, N, s.B, 32);
    md1 = md0;
    md2 = md0;
  }
  if (!ok) return cudaErrorInvalidValue;

  cudaError_t e = proj_opt_in();
  if (e != cudaSuccess) return e;
  const int num_sms = device_sm_count();
  ProjParams p;
  p.bias = bias;
  p.status = status;
  p.tiles_m_per_batch = ceil_div((int)N, kBM);
  p.tiles_n = ceil_div((int)features, kBN);
  const int64_t total = (int64_t)s.B * p.tiles_m_per_batch * p.tiles_n;
  if (total > 0x7fffffffll) return cudaErrorInvalidValue;
  p.total_tiles = (int)total;
  p.kblocks = s.H;
  p.H = s.H;
  p.fblocks = (int)(features / kD);
  p.N = (int)N;
  p.silu = 0;
  p.out_f16 = 0;
  p.idesc = kIdesc;
  const int grid = p.total_tiles < num_sms ? p.total_tiles : num_sms;
  if (qkv) proj_tc_kernel<true><<<grid, kThreads, kSmemBytes, st>>>(ma, mb, md0, md1, md2, p);
  else proj_tc_kernel<false><<<grid, kThreads, kSmemBytes, st>>>(ma, mb, md0, md1, md2, p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace jv
