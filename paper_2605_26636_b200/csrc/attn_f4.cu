// Full softmax attention (Eq. 1) for long sequences on the 5th-generation tensor cores:
// four 128-row query tiles per CTA, so that every SM sub-core holds four softmax warps.
// bf16 tensors, head_dim 64.
//
// The softmax of attention at head_dim 64 is bound by the SM's ordinary pipes (exponentials on
// MUFU and the FMA pipe, maxima and conversions on the ALU), not by the tensor pipe, and with one
// thread per query row a CTA of two query tiles gives each sub-core only two warps to overlap those
// pipes and their latencies.  This kernel trades the double-buffered scores of the two-tile kernel
// (attn_tc.cu) for twice the rows: per query tile one 64-column score buffer and one accumulator
// in tensor memory (4 x (64 + 64) = 512 columns), the probabilities written over the scores they
// came from.  A tile's chain  scores -> softmax -> P V, next scores  is strictly serial; the
// other three tiles fill the sub-core meanwhile.
//
// Persistent CTAs (one per SM) loop over work items; an item is four consecutive query tiles of one
// (batch, head) against all key tiles.  Warp roles (19 warps):
//   warp 0        TMA producer: four Q tiles per item, K and V tiles through 3-stage rings
//   warps 1, 2    MMA issuers (warp 1: query tiles 0 and 1, warp 2: tiles 2 and 3), in steps of 64 keys:
//                 O_t += P_t V (A = P from tensor memory, M128 N64 K64) of the previous step, then
//                 S_t = Q_t K^T (M128 N64 K64) of this one
//   warps 3-18    softmax, one thread per query row (warp w: tile (w - 3) / 4, rows 32 (w % 4) ..):
//                 exact two-pass softmax per step (maximum, then exponentials against a running
//                 reference that is raised only when a step exceeds it by 2^8), P as bf16 back into
//                 tensor memory, final 1/l scaling and the store.
//
// Every mbarrier wait is bounded: a wait that runs out sets the device status word, raises a
// CTA-wide abort flag, and every role falls through to the common teardown (tensor memory is
// always released).
#include "tc_common.cuh"

namespace jv {
namespace {

using namespace tc;

#ifndef JV_ATTN_SUSPEND_NS
#define JV_ATTN_SUSPEND_NS 4000
#endif
constexpr uint32_t kSuspendNs = JV_ATTN_SUSPEND_NS;   // suspend-time hint of this kernel's barrier waits (tc_common.cuh)
constexpr int kD = 64;
constexpr int kTile = 128;                  // tokens per tile (MMA M and key-tile rows)
constexpr int kTileBytes = kTile * kD * 2;  // 16 KB
constexpr int kQT = 4;                      // query tiles per work item
constexpr int kStages = 3;                  // K and V ring depth
constexpr int kWarps = 19;
constexpr int kThreads = kWarps * 32;
constexpr int kFirstSoftmaxWarp = 3;
constexpr uint32_t kTmemCols = 512;
constexpr int kSub = 64;                    // keys per step
#ifndef JV_POLY_OF_8
#define JV_POLY_OF_8 2
#endif
constexpr int kPolyOf8 = JV_POLY_OF_8;                 // of every 8 score pairs, this many take the polynomial exponential
// Tensor-memory columns: S_t (and P_t over its first 32 columns) at 64 t, O_t at 256 + 64 t
constexpr uint32_t kColS = 0, kColO = 256;

struct F4Params {
  int* status;
  int N;                 // tokens per (batch, head)
  int ntiles;            // key (and query) tiles per head: ceil(N / 128)
  int qgroups;           // groups of four query tiles per head
  int n_full;            // items [0, n_full) are whole groups, (batch*head, group) with the group fastest;
  int total_items;       // items [n_full, total_items) are half groups (two query tiles), see launch_attn_f4
  FastDiv div_qgroups;
  int H;                 // heads per batch element: the inputs are addressed by (head, batch)
  FastDiv div_H;
  float scale_log2;      // softmax scale * log2(e)
};

struct __align__(8) Barriers {
  uint64_t q_full[kQT], q_empty[kQT];
  uint64_t k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
  uint64_t s_full[kQT], p_full[kQT], o_full[kQT];
  uint64_t drain;
  uint32_t tmem_base;
  volatile uint32_t abort_flag;
};
constexpr size_t kSmemTiles = (2 * kQT + 2 * kStages) * (size_t)kTileBytes;   // Q[4] K[3] V[3] O[4]
constexpr size_t kSmemBytes = kSmemTiles + sizeof(Barriers) + 1024;            // + alignment slack

constexpr uint32_t kIdescQK = idesc(kTile, kSub, 0);
constexpr uint32_t kIdescPV = idesc(kTile, kD, 1);

struct Item {
  int bh, qt0, nt;  // (batch, head), the first of the item's query tiles, and how many it has (4 or 2)
};
// kHalves: the launch has half groups (n_full < total_items); without them the decode is one division.
template <bool kHalves>
__device__ __forceinline__ Item decode_item(const F4Params& p, int i) {
  Item it;
  if (kHalves) {
    const int half = i - p.n_full;                 // >= 0: a half group
    const int g = half < 0 ? i : p.n_full + (half >> 1);
    it.bh = fdiv(g, p.div_qgroups);
    it.qt0 = kQT * (g - it.bh * p.qgroups) + (half < 0 ? 0 : 2 * (half & 1));
    it.nt = half < 0 ? kQT : 2;
  } else {
    it.bh = fdiv(i, p.div_qgroups);
    it.qt0 = kQT * (i - it.bh * p.qgroups);
    it.nt = kQT;
  }
  return it;
}
// query tile t of the item exists: inside the item and inside the head
template <bool kHalves>
__device__ __forceinline__ bool tile_exists(const Item& it, int t, int ntiles) {
  return (!kHalves || t < it.nt) && it.qt0 + t < ntiles;
}

// ---- the kernel ------------------------------------------------------------------
// CTA c works on items c, c + gridDim.x, ...  Every role walks the same item sequence on its own;
// ring stages and barrier parities follow running counters.  A query tile past the last one of
// the head (the last item of a head whose tile count is not a multiple of four), or past the item's
// own two tiles (a half group), is skipped by its softmax warps; its issuer still takes part in the
// ring protocol so that arrival counts hold.  A half group without any tile is skipped by every role.
template <bool kHalves>
__global__ void __launch_bounds__(kThreads, 1)
attn_f4_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
               const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapO,
               const F4Params p) {
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment by an offset from the array itself, so that accesses stay shared-space loads and stores
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  Barriers* bar = reinterpret_cast<Barriers*>(smem + kSmemTiles);
  const uint32_t sQ = smem_u32(smem), sK = sQ + kQT * kTileBytes, sV = sK + kStages * kTileBytes;
  const uint32_t sO = sV + kStages * kTileBytes;      // output staging, one tile per query tile

  const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;

  // a timeout flagged earlier (by any CTA or launch) makes the rest leave at once
  if (threadIdx.x == 0) bar->tmem_base = *reinterpret_cast<volatile int*>(p.status);
  __syncthreads();
  if (bar->tmem_base != 0) return;
  __syncthreads();

  if (threadIdx.x == 0) {
    for (int t = 0; t < kQT; ++t) {
      mbar_init(&bar->q_full[t], 1);
      mbar_init(&bar->q_empty[t], 1);
      mbar_init(&bar->s_full[t], 1);
      mbar_init(&bar->p_full[t], 128);
      mbar_init(&bar->o_full[t], 1);
    }
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bar->k_full[s], 1);
      mbar_init(&bar->k_empty[s], 2);     // one commit from each MMA issuer warp
      mbar_init(&bar->v_full[s], 1);
      mbar_init(&bar->v_empty[s], 2);
    }
    mbar_init(&bar->drain, 2);
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

  const int item0 = blockIdx.x, item_step = gridDim.x;
  const int ntiles = p.ntiles, nsteps = 2 * p.ntiles;

  if (warp == 0) {
    // ================= TMA producer =================
    bool ok = true;
    int n = 0;                 // items seen
    int s = 0;                 // ring stage of the next key tile
    uint32_t par = 1;          // parity of the "empty" phase this pass over the ring waits for
    int issued_v = 0;          // for the abort path: V copies issued so far
    for (int i = item0; i < p.total_items && ok; i += item_step) {
      const Item it = decode_item<kHalves>(p, i);
      if (kHalves && !tile_exists<kHalves>(it, 0, ntiles)) continue;
      const int b = fdiv(it.bh, p.div_H), h = it.bh - b * p.H;   // coordinates of the input tensor maps
      for (int t = 0; t < kQT && ok; ++t) {
        ok = warp_wait<kSuspendNs>(&bar->q_empty[t], (n & 1) ^ 1, &bar->abort_flag, p.status);
        if (!ok) break;
        if (tile_exists<kHalves>(it, t, ntiles) && elect_one()) {
          mbar_expect_tx(&bar->q_full[t], kTileBytes);
          tma_load_4d(sQ + t * kTileBytes, &mapQ, &bar->q_full[t], 0, (it.qt0 + t) * kTile, h, b);
        }
        __syncwarp();
      }
      for (int j = 0; j < ntiles && ok; ++j) {
        ok = warp_wait<kSuspendNs>(&bar->k_empty[s], par, &bar->abort_flag, p.status);
        if (!ok) break;
        if (elect_one()) {
          mbar_expect_tx(&bar->k_full[s], kTileBytes);
          tma_load_4d(sK + s * kTileBytes, &mapK, &bar->k_full[s], 0, j * kTile, h, b);
        }
        __syncwarp();
        ok = warp_wait<kSuspendNs>(&bar->v_empty[s], par, &bar->abort_flag, p.status);
        if (!ok) break;
        if (elect_one()) {
          mbar_expect_tx(&bar->v_full[s], kTileBytes);
          tma_load_4d(sV + s * kTileBytes, &mapV, &bar->v_full[s], 0, j * kTile, h, b);
        }
        __syncwarp();
        ++issued_v;
        if (++s == kStages) { s = 0; par ^= 1; }
      }
      ++n;
    }
    if (!ok && lane == 0) {
      // let the copies still in flight land before the CTA leaves (bounded by the same limit)
      const unsigned long long t0 = globaltimer();
      for (int g = max(0, issued_v - kStages); g < issued_v; ++g)
        while (!mbar_try(&bar->v_full[g % kStages], (g / kStages) & 1) && globaltimer() - t0 < kWaitLimitNs) {}
    }
  } else if (warp == 1 || warp == 2) {
    // ================= MMA issuers: warp 1 serves query tiles 0 and 1, warp 2 tiles 2 and 3 =================
    // Per item and query tile t the work is a chain over 64-key steps u (key tile u / 2, half u % 2):
    //   S_t(u) = Q_t K(u)^T          4 MMAs, M128 N64 K16, operands in shared memory
    //   O_t   += P_t(u) V(u)         4 MMAs, M128 N64 K16, A = P in tensor memory
    // P_t(u) lies over S_t(u), so S_t(u + 1) is issued behind P_t(u) V(u): the tensor pipe executes one
    // thread's MMAs in issue order.  The commit that publishes S_t(u + 1) therefore also tells the
    // softmax warps that P_t(u) V(u) has retired and O_t is quiescent.
    const int tb = 2 * (warp - 1);
    bool ok = true;
    int sk = 0, sv = 0;                     // ring stages of the score key tile and of the P V key tile
    uint32_t phk = 0, phv = 0;              // and their "full" parities
    uint32_t pcnt[2] = {0, 0};              // steps published so far per tile: parity of p_full
    uint32_t qcnt[2] = {0, 0};              // items in which the tile existed: parity of q_full
    for (int i = item0; i < p.total_items && ok; i += item_step) {
      const Item it = decode_item<kHalves>(p, i);
      if (kHalves && !tile_exists<kHalves>(it, 0, ntiles)) continue;
      const bool ex[2] = {tile_exists<kHalves>(it, tb, ntiles), tile_exists<kHalves>(it, tb + 1, ntiles)};
      for (int u = 0; u <= nsteps && ok; ++u) {
        const bool has_qk = u < nsteps, has_pv = u > 0;
        if (has_qk && (u & 1) == 0) {       // first half of a key tile: its K must have landed
          ok = warp_wait<kSuspendNs>(&bar->k_full[sk], phk, &bar->abort_flag, p.status);
          if (!ok) break;
        }
        if (has_pv && ((u - 1) & 1) == 0) { // P V of a first half: its V must have landed
          ok = warp_wait<kSuspendNs>(&bar->v_full[sv], phv, &bar->abort_flag, p.status);
          if (!ok) break;
        }
        const uint32_t kb = sK + sk * kTileBytes + (u & 1) * (kSub * kD * 2);
        const uint32_t vb = sV + sv * kTileBytes + ((u - 1) & 1) * (kSub * kD * 2);
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          if (!ex[x]) continue;
          const int t = tb + x;
          if (u == 0) {
            ok = warp_wait<kSuspendNs>(&bar->q_full[t], qcnt[x] & 1, &bar->abort_flag, p.status);
            ++qcnt[x];
          } else {
            ok = warp_wait<kSuspendNs>(&bar->p_full[t], pcnt[x] & 1, &bar->abort_flag, p.status);
            ++pcnt[x];
          }
          if (!ok) break;
          tc_fence_after();
          if (elect_one()) {                 // one lane issues the step's MMAs back to back
            if (has_pv) {
              const uint64_t dv = smem_desc(vb);
#pragma unroll
              for (int ks = 0; ks < kSub / 16; ++ks)
                mma_ts_1(tmem + kColO + t * kD, tmem + kColS + t * kSub + ks * 8, desc_advance(dv, ks * 2048), kIdescPV,
                         (u > 1 || ks > 0) ? 1u : 0u);
            }
            if (has_qk) {
              const uint64_t dq = smem_desc(sQ + t * kTileBytes), dk = smem_desc(kb);
#pragma unroll
              for (int ks = 0; ks < kD / 16; ++ks)
                mma_ss_1(tmem + kColS + t * kSub, desc_advance(dq, ks * 32), desc_advance(dk, ks * 32), kIdescQK, ks > 0);
            }
          }
          __syncwarp();
          if (has_qk) tc_commit(&bar->s_full[t]);
          else tc_commit(&bar->o_full[t]);
        }
        if (!ok) break;
        if (has_pv && ((u - 1) & 1) == 1) { // both halves of the V tile are in flight or done
          tc_commit(&bar->v_empty[sv]);
          if (++sv == kStages) { sv = 0; phv ^= 1; }
        }
        if (has_qk && (u & 1) == 1) {
          tc_commit(&bar->k_empty[sk]);
          if (u == nsteps - 1) {            // the item's last scores: its query tiles may be replaced
            tc_commit(&bar->q_empty[tb]);
            tc_commit(&bar->q_empty[tb + 1]);
          }
          if (++sk == kStages) { sk = 0; phk ^= 1; }
        }
      }
    }
    // Teardown: every MMA issued so far must have retired before tensor memory is released.
    tc_commit(&bar->drain);
    if (lane == 0) {
      const unsigned long long t0 = globaltimer();
      while (!mbar_try(&bar->drain, 0) && globaltimer() - t0 < kWaitLimitNs) {}
    }
    __syncwarp();
  }
  else if (warp >= kFirstSoftmaxWarp) {
    // ================= softmax + epilogue: one thread per query row =================
    const int t = (warp - kFirstSoftmaxWarp) >> 2;  // query tile of this warp
    const int q4 = warp & 3;                        // tensor-memory quadrant a warp may touch: warp % 4
    const uint32_t lane_base = (uint32_t)(q4 << 5) << 16;
    const uint32_t tS = tmem + lane_base + kColS + t * kSub;   // scores; probabilities over their first 32 columns
    const uint32_t tO = tmem + lane_base + kColO + t * kD;
    const float sl2 = p.scale_log2;
    const float kLazy = 8.f / sl2;                 // the reference maximum moves only when it grew by > 2^8
    const uint64_t sl2x2 = pack2(sl2, sl2);
    const uint32_t sOt = sO + t * kTileBytes + q4 * 4096;      // this warp's quarter of the staging tile
    unsigned char* sOt_ptr = smem + (size_t)(kQT + 2 * kStages + t) * kTileBytes + q4 * 4096;
    const int last_valid = p.N - (ntiles - 1) * kTile;         // keys that exist in the last key tile
    bool ok = true;
    uint32_t scnt = 0;                // steps seen by this tile: parity of s_full
    uint32_t ocnt = 0;                // items seen by this tile: parity of o_full

    for (int i = item0; i < p.total_items && ok; i += item_step) {
      const Item it = decode_item<kHalves>(p, i);
      if (!tile_exists<kHalves>(it, t, ntiles)) continue;   // this query tile does not exist
      float m = -INFINITY, l = 0.f;
      for (int u = 0; u < nsteps; ++u) {
        ok = warp_wait<kSuspendNs>(&bar->s_full[t], scnt & 1, &bar->abort_flag, p.status);
        if (!ok) break;
        ++scnt;
        tc_fence_after();
        uint32_t va[32];
        if ((u >> 1) == ntiles - 1 && last_valid < kTile) {
          // Last key tile of a sequence that is not a multiple of 128: overwrite the scores of keys
          // that do not exist with -inf in tensor memory, then treat the step like any other.
#pragma unroll 1
          for (int c = 0; c < 2; ++c) {
            const int nv = last_valid - (64 * (u & 1) + 32 * c);      // valid keys among these 32
            if (nv < 32) {                                             // warp-uniform
              tmem_ld32(tS + 32 * c, va);
              tmem_wait_ld(va);
#pragma unroll
              for (int x = 0; x < 32; ++x)
                if (x >= nv) va[x] = kNegInf;     // exp2(-inf) = 0 and -inf never wins the maximum
              tmem_st32(tS + 32 * c, va);
            }
          }
          tmem_wait_st();
        }
        // ---- pass 1: the step's maximum (second half first, so that the first half is the one
        // left in registers for pass 2)
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        tmem_ld32(tS + 32, va);
        tmem_wait_ld(va);
        max32(va, mx4);
        tmem_ld32(tS, va);
        tmem_wait_ld(va);
        max32(va, mx4);
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        float o_scale = 1.f;
        if (mx > m + kLazy) {          // always true on the first step (m = -inf, mx finite)
          o_scale = ex2((m - mx) * sl2);            // first step: exp2(-inf) = 0
          l *= o_scale;
          m = mx;
        }
        if (u > 0 && __any_sync(0xffffffffu, o_scale != 1.f)) {
          // Rare: the reference moved.  O_t may be touched: the scores just waited for were committed
          // behind the previous step's P V, and the next P V waits for this step's P.
#pragma unroll 1
          for (int c = 0; c < 2; ++c) {
            uint32_t v[32];
            tmem_ld32(tO + 32 * c, v);
            tmem_wait_ld(v);
#pragma unroll
            for (int x = 0; x < 32; ++x) v[x] = __float_as_uint(__uint_as_float(v[x]) * o_scale);
            tmem_st32(tO + 32 * c, v);
          }
          // pass 2 needs the first half of the scores again
          tmem_wait_st();
          tmem_ld32(tS, va);
          tmem_wait_ld(va);
        }
        // ---- pass 2: exponentials against the reference, P over the scores just consumed
        const float mneg = -m * sl2;
        const uint64_t mnegx2 = pack2(mneg, mneg);
        uint64_t lsum[4] = {0ull, 0ull, 0ull, 0ull};
        uint32_t pk[16];
        exp32<false, kPolyOf8>(va, sl2x2, mnegx2, lsum, pk, mx4);
        tmem_st16(tS, pk);
        tmem_ld32(tS + 32, va);
        tmem_wait_ld(va);
        exp32<false, kPolyOf8>(va, sl2x2, mnegx2, lsum, pk, mx4);
        tmem_st16(tS + 16, pk);
        float a0, a1, b0, b1;
        unpack2(add2(lsum[0], lsum[1]), a0, a1);
        unpack2(add2(lsum[2], lsum[3]), b0, b1);
        l += (a0 + a1) + (b0 + b1);
        // publish P
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bar->p_full[t]);
      }
      if (!ok) break;
      // ---- epilogue: O / l -> bf16 -> this warp's quarter of the staging tile -> one TMA store
      ok = warp_wait<kSuspendNs>(&bar->o_full[t], ocnt & 1, &bar->abort_flag, p.status);
      if (!ok) break;
      ++ocnt;
      tc_fence_after();
      const float inv = 1.f / l;
      const int tok = (it.qt0 + t) * kTile + 32 * q4;          // first token of this warp's 32 rows
      const bool store = tok < p.N;                            // rows past N inside the box are clipped by the store
      if (store) {
        // this warp's previous store must have finished reading its staging quarter
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncwarp();
      }
#pragma unroll 1
      for (int c = 0; c < 2; ++c) {
        uint32_t v[32];
        tmem_ld32(tO + 32 * c, v);
        tmem_wait_ld(v);
        if (store) {
#pragma unroll
          for (int x = 0; x < 4; ++x) {     // 16-byte chunk 4 c + x of this row, at its 128-byte-swizzle position
            const uint4 w = make_uint4(pack_bf16(__uint_as_float(v[8 * x]) * inv, __uint_as_float(v[8 * x + 1]) * inv),
                                       pack_bf16(__uint_as_float(v[8 * x + 2]) * inv, __uint_as_float(v[8 * x + 3]) * inv),
                                       pack_bf16(__uint_as_float(v[8 * x + 4]) * inv, __uint_as_float(v[8 * x + 5]) * inv),
                                       pack_bf16(__uint_as_float(v[8 * x + 6]) * inv, __uint_as_float(v[8 * x + 7]) * inv));
            *reinterpret_cast<uint4*>(sOt_ptr + lane * 128 + (((4 * c + x) ^ (lane & 7)) << 4)) = w;
          }
        }
      }
      tc_fence_before();
      if (store) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          tma_store_3d(&mapO, sOt, 0, tok, it.bh);
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      }
    }
    // the staging tile must outlive the last store's reads; wait for the writes as well
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
}  // namespace

// Long sequences only: with fewer than eight key tiles the two-tile kernel's deeper pipeline wins.
bool attn_f4_supported(const AttnArgs& a) {
  if (a.dtype != JV_BF16 || a.D != kD) return false;
  const int64_t N = (int64_t)a.Hg * a.Wg;
  if (N < 8 * kTile) return false;
  const int64_t ntiles = (N + kTile - 1) / kTile;
  if ((ntiles + kQT - 1) / kQT * a.BH > 0x7fffffffll) return false;
  return encode_fn() != nullptr;
}

cudaError_t launch_attn_f4(const AttnArgs& a, int* status, cudaStream_t st) {
  EncodeFn enc = encode_fn();
  if (!enc) return cudaErrorNotSupported;
  const int N = a.Hg * a.Wg;
  CUtensorMap maps[4];
  const void* ptrs[4] = {a.q, a.k, a.v, a.o};
  const cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)N, (cuuint64_t)a.BH};
  const cuuint64_t strides[2] = {(cuuint64_t)kD * 2, (cuuint64_t)N * kD * 2};
  const cuuint32_t qbox[3] = {(cuuint32_t)kD, 32, 1};          // the output is stored per warp: 32 tokens
  const cuuint32_t estr[3] = {1, 1, 1};
  // the inputs as (d, token, head, batch) with the caller's strides; the output as (d, token, batch*head)
  const cuuint64_t idims[4] = {(cuuint64_t)kD, (cuuint64_t)N, (cuuint64_t)a.H, (cuuint64_t)(a.BH / a.H)};
  const cuuint64_t istrides[3] = {(cuuint64_t)a.in.tok * 2, (cuuint64_t)a.in.head * 2, (cuuint64_t)a.in.batch * 2};
  const cuuint32_t ibox[4] = {(cuuint32_t)kD, (cuuint32_t)kTile, 1, 1};
  const cuuint32_t iestr[4] = {1, 1, 1, 1};
  for (int i = 0; i < 4; ++i) {
    CUresult r = i < 3 ? enc(&maps[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptrs[i]), idims, istrides, ibox,
                             iestr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE)
                       : enc(&maps[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptrs[i]), dims, strides, qbox,
                             estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }
  static OncePerDevice smem_opt_in;   // > 48 KB of dynamic shared memory: a per-device function attribute
  cudaError_t e = smem_opt_in.run([] {
    cudaError_t r = cudaFuncSetAttribute(attn_f4_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (r == cudaSuccess)
      r = cudaFuncSetAttribute(attn_f4_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    return r;
  });
  if (e != cudaSuccess) return e;
  const int num_sms = device_sm_count();
  F4Params p;
  p.status = status;
  p.N = N;
  p.ntiles = ceil_div(N, kTile);
  p.qgroups = ceil_div(p.ntiles, kQT);
  // Items are dealt out round-robin, so the last round is as long as a full one however few CTAs it
  // keeps busy.  When it would keep at most half of them busy, its groups are split into half groups
  // of two query tiles (a serial per-tile chain makes those finish in a little over half the time).
  const int groups = p.qgroups * a.BH;
  const int rem = groups % num_sms;
  const int split = (rem > 0 && rem <= num_sms / 2) ? rem : 0;
  p.n_full = groups - split;
  p.total_items = groups + split;
  p.div_qgroups = make_fastdiv((uint32_t)p.qgroups);
  p.H = a.H;
  p.div_H = make_fastdiv((uint32_t)a.H);
  p.scale_log2 = a.scale * 1.4426950408889634f;
  const int grid = p.total_items < num_sms ? p.total_items : num_sms;
  if (split) attn_f4_kernel<true><<<grid, kThreads, kSmemBytes, st>>>(maps[0], maps[1], maps[2], maps[3], p);
  else attn_f4_kernel<false><<<grid, kThreads, kSmemBytes, st>>>(maps[0], maps[1], maps[2], maps[3], p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace jv
