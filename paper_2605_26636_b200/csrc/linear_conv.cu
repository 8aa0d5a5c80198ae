// Apply pass of the linear-attention block with the 3 x 3 depth-wise convolution on V fused in
// (Sec. 3.2.1, Eq. 4: O = LA + DWC(V) is one sum): bf16 tensors, head_dim 64.
//
//   o_i = relu(q_i) KV / (relu(q_i) . z + eps) + sum_{dy, dx} w[c][dy][dx] V[(y + dy - 1, x + dx - 1)][c]
//
// One persistent CTA per SM walks a contiguous range of tiles; a tile is a patch of 8 x 16 tokens of
// one (batch, head), so that the convolution's halo is a 10 x 18 box of V that TMA fetches with the
// zero padding for free (positions outside the grid arrive as zeros) and a ragged grid costs nothing
// special: rows and columns of a patch that do not exist are loaded as zeros and never stored.
// Each token of Q, V and O crosses HBM once; the halo overlap between neighbouring patches is served by L2.
//
// Warp roles (19 warps):
//   warps 0-3    rectifiers: per head, the deterministic second pass of the state reduction (chunk
//                partials summed in a fixed order -> KV as bf16 MMA operand, z in fp32); per tile,
//                ReLU of the Q tile in place (one thread per token) and that token's denominator
//   warp 4       TMA producer: Q patches into a ring of kNQ slots, V halos into a ring of kNV slots
//   warps 5-8    epilogue: accumulator (tensor memory) x 1/denominator -> bf16, written over the Q
//                tile it came from (the slot doubles as the output staging tile)
//   warps 9-16   convolution: warp j owns two patch rows x 8 columns; a lane owns 4 channels and 4
//                tokens of both rows, slides the 3 x 3 window over four input rows of the halo
//                (bf16 x bf16 products summed in fp32), adds the result to the attention
//                output waiting in the slot and rounds to bf16
//   warp 17      MMA issuer: relu(Q) KV as tcgen05.mma M128 N64 K64, accumulators double-buffered
//   warp 18      store warp: one TMA store per finished tile (clipped at the grid edge), then the
//                slot goes back to the producer
//
// Every mbarrier wait is bounded; a wait that runs out sets the device status word and the CTA-wide
// abort flag, every role falls through, tensor memory is released.
#include "lin_common.cuh"

namespace jv {
namespace {

using namespace tc;
using namespace lin;

constexpr int kPatchH = 8, kPatchW = 16;              // tokens of a tile: 8 grid rows x 16 grid columns
constexpr int kTileBytes = kPatchH * kPatchW * kD * 2;   // 16 KB
constexpr int kKvBytes = kD * kD * 2;                 // bf16 KV[a][e], 128-byte swizzle
constexpr int kHaloBytes = (kPatchH + 2) * (kPatchW + 2) * kD * 2;   // 23040
constexpr int kHaloSlot = 23552;                      // padded to a multiple of 512
constexpr int kNQ = 5;                                // Q / output ring
constexpr int kNV = 3;                                // V halo ring
constexpr int kDenRing = 8;                           // denominators of the tiles between ReLU and epilogue (> kNQ)
constexpr int kWarps = 19, kThreadsConv = kWarps * 32;
constexpr int kWarpProducer = 4, kWarpEpi0 = 5, kWarpConv0 = 9, kWarpMma = 17, kWarpStore = 18;
constexpr uint32_t kTmemCols = 128;                   // two 64-column fp32 accumulators
constexpr uint32_t kIdesc = idesc(128, 64, 1);        // D fp32, A and B bf16, B MN-major, M = 128, N = 64

struct __align__(8) ConvBars {
  uint64_t q_full[kNQ], q_free[kNQ];                  // TMA landed / the tile's store has read the slot
  uint64_t conv_done[kNQ];                            // 8 arrivals: the convolution warps have finished the tile in this slot
  uint64_t relu_done[kNQ];                            // 128 arrivals: tile rectified, denominators stored
  uint64_t la_done[kNQ];                              // 128 arrivals: attention output (bf16) written into the slot
  uint64_t v_full[kNV], v_free[kNV];                  // TMA landed / the 8 convolution warps are done with the halo
  uint64_t d_full[2], d_empty[2];                     // accumulator complete (tcgen05.commit) / read by the epilogue (128)
  uint64_t kv_free[2];                                // the MMAs that read this KV buffer are complete (tcgen05.commit)
  uint64_t workers;                                   // the 128 rectifier threads among themselves
  uint32_t tmem_base;
  volatile uint32_t abort_flag;
};
// shared memory: Q ring | KV x 2 | V halo ring | z x 2 | denominators | barriers
constexpr size_t kOffKv = (size_t)kNQ * kTileBytes;
constexpr size_t kOffHalo = kOffKv + 2 * kKvBytes;
constexpr size_t kOffZsm = kOffHalo + (size_t)kNV * kHaloSlot;
constexpr size_t kOffDen = kOffZsm + 2 * kD * sizeof(float);
constexpr size_t kOffBars = kOffDen + (size_t)kDenRing * 128 * sizeof(float);
constexpr size_t kConvSmem = kOffBars + sizeof(ConvBars) + 1024;   // + alignment slack

struct ConvParams {
  const float* partial;     // chunk partials of the state pass
  const float* w;           // convolution kernels [B][C][3][3] fp32 (generated, or broadcast static ones)
  int* status;
  int H, BH, Hg, Wg, nchunk, state_elems;
  int ncb, nrb;             // patches per grid row / per grid column
  int total_tiles;          // B*H * ncb * nrb
  float eps;
};

// Mixed-precision arithmetic of sm_100: the product of two bf16 values (exact in fp32) added into
// an fp32 sum, and a bf16 value added to an fp32 one, both with one rounding.  a and b hold two
// bf16 values each; lane-wise: lo += a.lo * b.lo, hi += a.hi * b.hi.
__device__ __forceinline__ void fma_bf16x2(float& lo, float& hi, uint32_t a, uint32_t b) {
  asm("{\n.reg .b16 al, ah, bl, bh;\n"
      "mov.b32 {al, ah}, %2;\nmov.b32 {bl, bh}, %3;\n"
      "fma.rn.f32.bf16 %0, al, bl, %0;\nfma.rn.f32.bf16 %1, ah, bh, %1;\n}\n"
      : "+f"(lo), "+f"(hi) : "r"(a), "r"(b));
}
__device__ __forceinline__ void add_bf16x2(float& lo, float& hi, uint32_t a) {
  asm("{\n.reg .b16 al, ah;\n"
      "mov.b32 {al, ah}, %2;\n"
      "add.rn.f32.bf16 %0, al, %0;\nadd.rn.f32.bf16 %1, ah, %1;\n}\n"
      : "+f"(lo), "+f"(hi) : "r"(a));
}

// Walks the tiles of a CTA's range in order: (batch*head, patch row, patch column).
struct TileIter {
  int bh, py, px;
  __device__ __forceinline__ void init(int tile, int ncb, int nrb) {
    const int np = ncb * nrb;
    bh = tile / np;
    const int pt = tile - bh * np;
    py = pt / ncb;
    px = pt - py * ncb;
  }
  // advances; true when the next tile belongs to another (batch, head)
  __device__ __forceinline__ bool next(int ncb, int nrb) {
    if (++px == ncb) {
      px = 0;
      if (++py == nrb) { py = 0; ++bh; return true; }
    }
    return false;
  }
};

__global__ void __launch_bounds__(kThreadsConv, 1)
lin_apply_conv_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapV,
                      const __grid_constant__ CUtensorMap mapO, const ConvParams p) {
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment by an offset from the array itself, so that accesses stay shared-space loads and stores
  unsigned char* smem_al = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t smem = smem_u32(smem_al);
  float* z_sm = reinterpret_cast<float*>(smem_al + kOffZsm);          // [2][64]
  float* den_sm = reinterpret_cast<float*>(smem_al + kOffDen);        // [kDenRing][128]
  ConvBars* bars = reinterpret_cast<ConvBars*>(smem_al + kOffBars);
  const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;

  // this CTA's contiguous range of tiles
  const int t_begin = (int)((long long)blockIdx.x * p.total_tiles / gridDim.x);
  const int t_end = (int)((long long)(blockIdx.x + 1) * p.total_tiles / gridDim.x);
  const int ntiles = t_end - t_begin;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kNQ; ++s) {
      mbar_init(&bars->q_full[s], 1);
      mbar_init(&bars->q_free[s], 1);
      mbar_init(&bars->conv_done[s], 8);
      mbar_init(&bars->relu_done[s], 128);
      mbar_init(&bars->la_done[s], 128);
    }
    for (int s = 0; s < kNV; ++s) {
      mbar_init(&bars->v_full[s], 1);
      mbar_init(&bars->v_free[s], 8);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&bars->d_full[b], 1);
      mbar_init(&bars->d_empty[b], 128);
      mbar_init(&bars->kv_free[b], 1);
    }
    mbar_init(&bars->workers, 128);
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)),
                 "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = __shfl_sync(0xffffffffu, bars->tmem_base, 0);

  if (warp == kWarpProducer) {
    // ================= TMA producer =================
    // Q and V are inputs of the call: the loads start at once, before the grids ahead of this one
    // in the stream (state pass, kernel generator) are complete.  Q is read once (evict first);
    // V was read by the state pass moments ago (which asked L2 to keep it) and every halo line is
    // wanted again by the neighbouring patches: no hint.
    const uint64_t pol_first = l2_policy_evict_first();
    TileIter ti;
    ti.init(t_begin, p.ncb, p.nrb);
    bool ok = true;
    int issued_q = 0, issued_v = 0;
    for (int it = 0; it < ntiles; ++it) {
      const int sq = it % kNQ, sv = it % kNV;
      if (it >= kNQ) {
        ok = warp_wait(&bars->q_free[sq], ((it / kNQ) - 1) & 1, &bars->abort_flag, p.status);
        if (!ok) break;
      }
      if (elect_one()) {
        mbar_expect_tx(&bars->q_full[sq], kTileBytes);
        const int in_b = ti.bh / p.H;              // the inputs are addressed by (head, batch)
        tma_load_5d_hint(smem + sq * kTileBytes, &mapQ, &bars->q_full[sq], 0, ti.px * kPatchW, ti.py * kPatchH,
                         ti.bh - in_b * p.H, in_b, pol_first);
      }
      __syncwarp();
      ++issued_q;
      if (it >= kNV) {
        ok = warp_wait(&bars->v_free[sv], ((it / kNV) - 1) & 1, &bars->abort_flag, p.status);
        if (!ok) break;
      }
      if (elect_one()) {
        mbar_expect_tx(&bars->v_full[sv], kHaloBytes);
        const int in_b = ti.bh / p.H;
        tma_load_5d(smem + (uint32_t)kOffHalo + sv * kHaloSlot, &mapV, &bars->v_full[sv], 0, ti.px * kPatchW - 1,
                    ti.py * kPatchH - 1, ti.bh - in_b * p.H, in_b);
      }
      __syncwarp();
      ++issued_v;
      ti.next(p.ncb, p.nrb);
    }
    if (!ok && lane == 0) {   // let the copies in flight land before the CTA leaves
      const unsigned long long t0 = globaltimer();
      for (int g = max(0, issued_q - kNQ); g < issued_q; ++g)
        while (!mbar_try(&bars->q_full[g % kNQ], (g / kNQ) & 1) && globaltimer() - t0 < kWaitLimitNs) {}
      for (int g = max(0, issued_v - kNV); g < issued_v; ++g)
        while (!mbar_try(&bars->v_full[g % kNV], (g / kNV) & 1) && globaltimer() - t0 < kWaitLimitNs) {}
    }
  } else if (warp == kWarpMma) {
    // ================= MMA issuer =================
    TileIter ti;
    ti.init(t_begin, p.ncb, p.nrb);
    bool ok = true;
    int nh = 0;                                        // heads seen so far by this CTA: KV buffer nh & 1
    for (int it = 0; it < ntiles; ++it) {
      const int sq = it % kNQ, b = it & 1, hb = nh & 1;
      ok = warp_wait(&bars->relu_done[sq], (it / kNQ) & 1, &bars->abort_flag, p.status);
      if (ok && it >= 2) ok = warp_wait(&bars->d_empty[b], ((it >> 1) - 1) & 1, &bars->abort_flag, p.status);
      if (!ok) break;
      tc_fence_after();
      const uint32_t qa = smem + sq * kTileBytes, kv = smem + (uint32_t)kOffKv + hb * kKvBytes;
#pragma unroll
      for (int ks = 0; ks < kD / 16; ++ks)
        mma_ss(tmem + b * kD, smem_desc(qa + ks * 32), smem_desc(kv + ks * 2048), kIdesc, ks > 0 ? 1u : 0u);
      tc_commit(&bars->d_full[b]);
      const bool head_ends = ti.next(p.ncb, p.nrb);
      if (head_ends) {                                 // the KV buffer may be rebuilt once these MMAs are complete
        tc_commit(&bars->kv_free[hb]);
        ++nh;
      }
    }
  } else if (warp < 4) {
    // ================= rectifier warps: thread r = 32 warp + lane owns token row r of every tile =================
    griddep_wait();                                    // the grids before this one (state pass, kernel generator) are complete
    bool ok = *reinterpret_cast<volatile int*>(p.status) == 0;
    if (!ok) bars->abort_flag = 1;                     // an earlier kernel gave up: every role of this CTA falls through at once
    const int row = threadIdx.x;
    uint32_t wpar = 0;
    // Second pass of the state reduction for (batch, head) bh into KV / z buffer hb: the chunk
    // partials are summed in chunk order (no atomics: bit-reproducible); KV goes to shared memory as
    // the bf16 MMA operand (128-byte swizzle), z stays fp32.  All loads of a chunk are in flight together.
    auto build_state = [&](int bh, int hb) {
      unsigned char* kv_ptr = smem_al + kOffKv + (size_t)hb * kKvBytes;
      const float* P = p.partial + (size_t)bh * p.nchunk * p.state_elems;
      float4 acc[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
      float zs = 0.f;
      for (int k = 0; k < p.nchunk; ++k) {
        const float* Pk = P + (size_t)k * p.state_elems;
        float4 t[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {                  // 16-byte chunk pairs tid, tid + 128, ... of the 64 x 64 matrix
          const float* src = Pk + (threadIdx.x + 128 * i) * 8;
          t[2 * i] = __ldcg(reinterpret_cast<const float4*>(src));
          t[2 * i + 1] = __ldcg(reinterpret_cast<const float4*>(src + 4));
        }
        const float zk = threadIdx.x < kD ? __ldcg(Pk + kOffZ + threadIdx.x) : 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) { acc[j].x += t[j].x; acc[j].y += t[j].y; acc[j].z += t[j].z; acc[j].w += t[j].w; }
        zs += zk;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int c = threadIdx.x + 128 * i;
        uint4 pk;
        pk.x = pack_bf16(acc[2 * i].x, acc[2 * i].y);
        pk.y = pack_bf16(acc[2 * i].z, acc[2 * i].w);
        pk.z = pack_bf16(acc[2 * i + 1].x, acc[2 * i + 1].y);
        pk.w = pack_bf16(acc[2 * i + 1].z, acc[2 * i + 1].w);
        *reinterpret_cast<uint4*>(kv_ptr + tile_off(c >> 3, c & 7)) = pk;
      }
      if (threadIdx.x < kD) z_sm[hb * kD + threadIdx.x] = zs;
    };
    // all 128 rectifier threads: what they wrote is complete and visible to the tensor core
    auto workers_sync = [&]() -> bool {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(&bars->workers);
      const bool w_ok = warp_wait(&bars->workers, wpar, &bars->abort_flag, p.status);
      wpar ^= 1;
      return w_ok;
    };
    TileIter ti;
    ti.init(t_begin, p.ncb, p.nrb);
    const int bh_last = (t_end - 1) / (p.ncb * p.nrb);  // (batch, head) of this CTA's last tile
    int nh = 0;                                        // heads seen so far: buffer nh & 1
    int built = 0;                                     // heads whose state has been built so far
    int head_tile = 0;                                 // tiles of the current head rectified so far
    for (int it = 0; it < ntiles && ok; ++it) {
      const int sq = it % kNQ, hb = nh & 1;
      if (built == nh) {                               // this head's state is not there yet (the CTA's first head)
        if (nh >= 2) {                                 // (or a head that follows one of a single tile)
          ok = warp_wait(&bars->kv_free[hb], ((nh >> 1) - 1) & 1, &bars->abort_flag, p.status);
          if (!ok) break;
        }
        build_state(ti.bh, hb);
        ++built;
        ok = workers_sync();
        if (!ok) break;
      } else if (head_tile == 1 && built == nh + 1 && ti.bh < bh_last) {
        // The next head's state is built ahead, into the other buffer, while the stages behind this
        // one still have tiles of the current head queued: no bubble at the head boundary.  The buffer
        // is free once the MMAs of the head before the current one are complete.
        if (nh >= 1) {
          ok = warp_wait(&bars->kv_free[hb ^ 1], ((nh - 1) >> 1) & 1, &bars->abort_flag, p.status);
          if (!ok) break;
        }
        build_state(ti.bh + 1, hb ^ 1);
        ++built;
        ok = workers_sync();
        if (!ok) break;
      }
      ok = warp_wait(&bars->q_full[sq], (it / kNQ) & 1, &bars->abort_flag, p.status);
      if (!ok) break;
      {  // ReLU of this thread's row in place; its denominator relu(q).z exactly in fp32
        unsigned char* q = smem_al + (size_t)sq * kTileBytes + row * 128;
        const float* z = z_sm + hb * kD;
        uint4 v[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) v[c] = *reinterpret_cast<const uint4*>(q + ((c ^ (row & 7)) << 4));
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          v[c].x = relu_bf16x2(v[c].x); v[c].y = relu_bf16x2(v[c].y); v[c].z = relu_bf16x2(v[c].z); v[c].w = relu_bf16x2(v[c].w);
          const float4 za = *reinterpret_cast<const float4*>(z + 8 * c), zb = *reinterpret_cast<const float4*>(z + 8 * c + 4);
          const float2 f0 = bf16x2_to_f2(v[c].x), f1 = bf16x2_to_f2(v[c].y), f2 = bf16x2_to_f2(v[c].z), f3 = bf16x2_to_f2(v[c].w);
          acc[0] = fmaf(f0.x, za.x, fmaf(f0.y, za.y, acc[0]));
          acc[1] = fmaf(f1.x, za.z, fmaf(f1.y, za.w, acc[1]));
          acc[2] = fmaf(f2.x, zb.x, fmaf(f2.y, zb.y, acc[2]));
          acc[3] = fmaf(f3.x, zb.z, fmaf(f3.y, zb.w, acc[3]));
        }
#pragma unroll
        for (int c = 0; c < 8; ++c) *reinterpret_cast<uint4*>(q + ((c ^ (row & 7)) << 4)) = v[c];
        den_sm[(it & (kDenRing - 1)) * 128 + row] = (acc[0] + acc[1]) + (acc[2] + acc[3]);
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(&bars->relu_done[sq]);
      ++head_tile;
      if (ti.next(p.ncb, p.nrb)) { ++nh; head_tile = 0; }
    }
  } else if (warp >= kWarpEpi0 && warp < kWarpConv0) {
    // ================= epilogue warps: thread (quadrant q4 = warp % 4, lane) owns row 32 q4 + lane =================
    const int q4 = warp & 3, row = 32 * q4 + lane;
    const uint32_t lane_base = (uint32_t)(q4 << 5) << 16;
    bool ok = true;
    for (int it = 0; it < ntiles && ok; ++it) {
      const int sq = it % kNQ, b = it & 1;
      // The tile's MMAs were issued after all 128 rectifier threads had published its rows and
      // denominators, so the accumulator being complete means the denominators are in place; it
      // also means that the tensor core is done reading the Q tile, which is overwritten below.
      ok = warp_wait(&bars->d_full[b], (it >> 1) & 1, &bars->abort_flag, p.status);
      if (!ok) break;
      tc_fence_after();
      const float inv = 1.f / (den_sm[(it & (kDenRing - 1)) * 128 + row] + p.eps);
      uint32_t v0[32], v1[32];
      tmem_ld32(tmem + lane_base + b * kD, v0);
      tmem_ld32(tmem + lane_base + b * kD + 32, v1);
      tmem_wait_ld(v0);
      tmem_wait_ld(v1);
      tc_fence_before();
      mbar_arrive(&bars->d_empty[b]);                  // the accumulator buffer may be overwritten
      unsigned char* st = smem_al + (size_t)sq * kTileBytes + row * 128;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint32_t* v = c < 4 ? v0 + 8 * c : v1 + 8 * (c - 4);
        uint4 w;
        w.x = pack_bf16(__uint_as_float(v[0]) * inv, __uint_as_float(v[1]) * inv);
        w.y = pack_bf16(__uint_as_float(v[2]) * inv, __uint_as_float(v[3]) * inv);
        w.z = pack_bf16(__uint_as_float(v[4]) * inv, __uint_as_float(v[5]) * inv);
        w.w = pack_bf16(__uint_as_float(v[6]) * inv, __uint_as_float(v[7]) * inv);
        *reinterpret_cast<uint4*>(st + ((c ^ (row & 7)) << 4)) = w;
      }
      mbar_arrive(&bars->la_done[sq]);
    }
  } else if (warp >= kWarpConv0 && warp < kWarpMma) {
    // ================= convolution warps: warp j owns patch rows 2 (j / 2), 2 (j / 2) + 1 and the 8
    // columns 8 (j % 2) .. of them; a lane owns channels 4 c4 .. 4 c4 + 3 and 4 consecutive tokens of
    // both rows.  Four input rows of the halo serve the two output rows.  The multiply-adds are the
    // mixed-precision fma.rn.f32.bf16 (bf16 x bf16 product, exact, added into an fp32 sum): V stays
    // packed as loaded and the kernels are held as bf16, the precision the tensor-core products of
    // this block have as well. =================
    const int cw = warp - kWarpConv0;
    const int rp = cw >> 1, c4 = lane & 15;
    const int xt = 8 * (cw & 1) + 4 * (lane >> 4);    // first of this lane's 4 token columns inside the patch
    griddep_wait();                                    // the kernels w come from the grid before this one
    bool ok = true;
    uint32_t wq[2][9];                                 // kernels of this lane's channels as bf16 pairs, [channel pair][tap]
    TileIter ti;
    ti.init(t_begin, p.ncb, p.nrb);
    bool new_head = true;
    for (int it = 0; it < ntiles && ok; ++it) {
      const int sq = it % kNQ, sv = it % kNV;
      if (new_head) {
        const int b = ti.bh / p.H, h = ti.bh - b * p.H;
        const float4* wp = reinterpret_cast<const float4*>(p.w + ((size_t)b * p.H * kD + (size_t)h * kD + 4 * c4) * 9);
        float wf[36];                                  // [channel][tap] as stored
#pragma unroll
        for (int k = 0; k < 9; ++k) {
          const float4 t4 = __ldcg(wp + k);   // written by the grid before this one: read through L2
          wf[4 * k] = t4.x; wf[4 * k + 1] = t4.y; wf[4 * k + 2] = t4.z; wf[4 * k + 3] = t4.w;
        }
#pragma unroll
        for (int pr = 0; pr < 2; ++pr)
#pragma unroll
          for (int tap = 0; tap < 9; ++tap) wq[pr][tap] = pack_bf16(wf[9 * (2 * pr) + tap], wf[9 * (2 * pr + 1) + tap]);
        if (ti.bh + 1 < p.BH) {   // the kernels of the (batch, head) after this one: into L2 ahead of the switch
          const float* wn = reinterpret_cast<const float*>(wp) + kD * 9;
          asm volatile("prefetch.global.L2 [%0];" ::"l"(wn));
          asm volatile("prefetch.global.L2 [%0];" ::"l"(wn + 32));
        }
      }
      ok = warp_wait(&bars->v_full[sv], (it / kNV) & 1, &bars->abort_flag, p.status);
      if (ok) ok = warp_wait(&bars->la_done[sq], (it / kNQ) & 1, &bars->abort_flag, p.status);
      if (!ok) break;
      const int y0 = ti.py * kPatchH + 2 * rp;         // grid row of this warp's first output row
      const int x0 = ti.px * kPatchW + 8 * (cw & 1);   // grid column of this warp's first token
      const bool any = y0 < p.Hg && x0 < p.Wg;         // else none of this warp's tokens exists
      if (any) {
        const unsigned char* vs = smem_al + kOffHalo + (size_t)sv * kHaloSlot + c4 * 8;   // halo: [10][18][128 B]
        unsigned char* os = smem_al + (size_t)sq * kTileBytes;
        float acc[2][4][4];                              // [output row][token][channel]
#pragma unroll
        for (int o = 0; o < 2; ++o)
#pragma unroll
          for (int k = 0; k < 4; ++k)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[o][k][c] = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {                    // input rows 2 rp - 1 + j of the patch = halo rows 2 rp + j
          uint2 u[6];                                    // six tokens of this input row, 4 channels each, as loaded
#pragma unroll
          for (int k = 0; k < 6; ++k)
            u[k] = *reinterpret_cast<const uint2*>(vs + ((2 * rp + j) * (kPatchW + 2) + xt + k) * 128);
#pragma unroll
          for (int o = 0; o < 2; ++o) {
            const int dy = j - o;                        // tap row with which this input row meets output row o
            if (dy < 0 || dy > 2) continue;
#pragma unroll
            for (int k = 0; k < 4; ++k)
#pragma unroll
              for (int dx = 0; dx < 3; ++dx) {
                fma_bf16x2(acc[o][k][0], acc[o][k][1], wq[0][3 * dy + dx], u[k + dx].x);
                fma_bf16x2(acc[o][k][2], acc[o][k][3], wq[1][3 * dy + dx], u[k + dx].y);
              }
          }
        }
#pragma unroll
        for (int o = 0; o < 2; ++o)
#pragma unroll
          for (int k = 0; k < 4; ++k) {                  // add to the attention output waiting in the slot, round once more
            const int r = (2 * rp + o) * kPatchW + xt + k;
            uint2* dst = reinterpret_cast<uint2*>(os + r * 128 + (((c4 >> 1) ^ (r & 7)) << 4) + (c4 & 1) * 8);
            const uint2 la = *dst;
            add_bf16x2(acc[o][k][0], acc[o][k][1], la.x);
            add_bf16x2(acc[o][k][2], acc[o][k][3], la.y);
            uint2 out;
            out.x = pack_bf16(acc[o][k][0], acc[o][k][1]);
            out.y = pack_bf16(acc[o][k][2], acc[o][k][3]);
            *dst = out;
          }
      }
      // the halo slot is free once all lanes have read it; the finished tile goes to the store warp
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&bars->v_free[sv]);
        mbar_arrive(&bars->conv_done[sq]);
      }
      new_head = ti.next(p.ncb, p.nrb);
    }
  } else if (warp == kWarpStore) {
    // ================= store warp: one TMA store per finished tile (the whole 8 x 16 patch; rows and
    // columns past the grid edge are clipped by the store itself) =================
    TileIter ti;
    ti.init(t_begin, p.ncb, p.nrb);
    bool ok = true;
    for (int it = 0; it < ntiles; ++it) {
      const int sq = it % kNQ;
      ok = warp_wait(&bars->conv_done[sq], (it / kNQ) & 1, &bars->abort_flag, p.status);
      if (!ok) break;
      if (lane == 0) {
        asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                     ::"l"(&mapO), "r"(smem + sq * kTileBytes), "r"(0), "r"(ti.px * kPatchW), "r"(ti.py * kPatchH), "r"(ti.bh)
                     : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the slot has been read: the producer may refill it
        mbar_arrive(&bars->q_free[sq]);
      }
      __syncwarp();
      ti.next(p.ncb, p.nrb);
    }
    // wait for the writes of the last stores as well
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  // ================= common teardown =================
  // Every MMA issued has been waited for (d_full) unless a wait gave up; in that case give the
  // tensor core a bounded time before tensor memory is released.
  if (bars->abort_flag && warp == kWarpMma && lane == 0) {
    const unsigned long long t0 = globaltimer();
    while (globaltimer() - t0 < 1000000ull) {}
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

}  // namespace

bool linear_conv_supported(const LinArgs& a) {
  if (!(a.s.dtype == JV_BF16 && a.s.D == kD && a.dwc && a.dwc->k == 3 && encode_fn() != nullptr)) return false;
  const long long tiles = (long long)a.s.B * a.s.H * ceil_div(a.s.Wg, kPatchW) * ceil_div(a.s.Hg, kPatchH);
  return tiles <= 0x7fffffffll;
}

// Enqueues the fused apply + convolution pass over the grid tokens (prefix tokens, which the
// convolution does not see, are left to the plain apply pass).  `partial` holds the chunk partials of the state
// pass, `w` the kernels [B][C][3][3]; both are written by grids ahead of this one in the stream,
// which this grid waits for (griddepcontrol.wait) before it reads them.
cudaError_t launch_linear_apply_conv(const LinArgs& a, const LinPlan& p, const float* partial, const float* w,
                                     int* status, bool programmatic, cudaStream_t st) {
  const jv_shape& s = a.s;
  const int BH = s.B * s.H;
  CUtensorMap mq, mv, mo;
  const InStrides in = in_strides(s);
  if (!make_map_grid_in(&mq, a.q, s.B, s.H, s.P, s.Hg, s.Wg, kPatchW, kPatchH, true, in) ||
      !make_map_grid_in(&mv, a.v, s.B, s.H, s.P, s.Hg, s.Wg, kPatchW + 2, kPatchH + 2, false, in) ||
      !make_map_grid(&mo, a.o, BH, s.P, s.Hg, s.Wg, kPatchW, kPatchH, true))
    return cudaErrorInvalidValue;
  static OncePerDevice smem_opt_in;
  cudaError_t e = smem_opt_in.run([] {
    return cudaFuncSetAttribute(lin_apply_conv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kConvSmem);
  });
  if (e != cudaSuccess) return e;
  ConvParams cp;
  cp.partial = partial;
  cp.w = w;
  cp.status = status;
  cp.H = s.H;
  cp.BH = BH;
  cp.Hg = s.Hg;
  cp.Wg = s.Wg;
  cp.nchunk = p.nchunk;
  cp.state_elems = p.state_elems;
  cp.ncb = ceil_div(s.Wg, kPatchW);
  cp.nrb = ceil_div(s.Hg, kPatchH);
  cp.total_tiles = BH * cp.ncb * cp.nrb;
  cp.eps = a.eps;
  const int num_sms = device_sm_count();
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(cp.total_tiles < num_sms ? cp.total_tiles : num_sms);
  cfg.blockDim = dim3(kThreadsConv);
  cfg.dynamicSmemBytes = kConvSmem;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = programmatic ? 1 : 0;
  e = cudaLaunchKernelEx(&cfg, lin_apply_conv_kernel, mq, mv, mo, cp);
  count_launch();
  return e;
}

}  // namespace jv
