// Full softmax attention (Eq. 1) and 2-D window attention (Sec. 3.2.2) at head_dim 128 on the
// 5th-generation tensor cores: two 128-row query tiles per CTA.  bf16 tensors, no prefix tokens in W.
//
// The four-tile kernel of head_dim 64 (attn_f4.cu) does not carry over: a 128-column fp32 accumulator
// per query tile leaves tensor memory (512 columns) room for two tiles: per tile two 64-column score
// buffers (the bf16 probabilities written over the scores they came from) and one 128-column
// accumulator.  With two buffers the scores of the next step are computed while the softmax works on
// this one, so a tile's chain is  softmax -> P V  only; at this head_dim there are twice the
// tensor-core flops per exponential, and the tensor pipe and MUFU are about equally loaded.
//
// A tile of 128 tokens x 128 channels lies in shared memory as two 128-byte-swizzled halves of 64
// channels (16 KB each, one TMA box each): Q K^T runs over both halves (8 MMAs of K = 16), P V
// writes the two 64-column halves of the accumulator from the two halves of V (2 x 4 MMAs).
//
// The token grid is a 5-D TMA tensor (d, x, y, head, batch); a tile is a box of 128 tokens (F: 128
// consecutive tokens of the sequence seen as an N x 1 grid; W: ww x 128 / ww tokens of a window).
// Persistent CTAs (one per SM) loop over work items; an item is two consecutive query tiles of one
// window of one (batch, head) against all key tiles of that window.  Keys outside the grid or the
// window arrive as zeros or as a neighbour's tokens and are overwritten with -inf in tensor memory
// before the softmax; query rows outside are not written.  Warp roles (10 warps):
//   warp 0        TMA producer: two Q tiles per item, K tiles through a ring of three, V tiles through a ring of two
//   warp 1        MMA issuer, in steps of 64 keys, both tiles: O_t += P_t V of step u, then S_t = Q_t K^T of step u + 2
//                 into the score buffer that P V has just read
//   warps 2-9     softmax, one thread per query row (warp w: tile (w - 2) / 4, tensor-memory quadrant w % 4):
//                 exact two-pass softmax per step against a lazily raised reference, P as bf16 back into
//                 tensor memory, final 1/l scaling, rows written straight to global memory (256 contiguous
//                 bytes per row and thread)
//
// Every mbarrier wait is bounded: a wait that runs out sets the device status word, raises a
// CTA-wide abort flag, and every role falls through to the common teardown (tensor memory is
// always released).
#include "tc_common.cuh"

namespace jv {
namespace {

using namespace tc;

constexpr uint32_t kSuspendNs = 4000;       // suspend-time hint of this kernel's barrier waits (tc_common.cuh)
constexpr int kD = 128;
constexpr int kHalfD = 64;                  // channels per swizzled half tile
constexpr int kTile = 128;                  // tokens per tile (MMA M and key-tile rows)
constexpr int kHalfBytes = kTile * kHalfD * 2;   // 16 KB
constexpr int kTileBytes = 2 * kHalfBytes;       // 32 KB
constexpr int kQT = 2;                      // query tiles per work item
constexpr int kKS = 3, kVS = 2;             // K and V ring depths
constexpr int kWarps = 10;
constexpr int kThreads = kWarps * 32;
constexpr int kFirstSoftmaxWarp = 2;
constexpr uint32_t kTmemCols = 512;
constexpr int kSub = 64;                    // keys per step
#ifndef JV_D128_POLY
#define JV_D128_POLY 1
#endif
constexpr int kPolyOf8 = JV_D128_POLY;      // of every 8 score pairs, this many take the polynomial exponential
// Tensor-memory columns: score buffer h of tile t (and its P over the first 32 columns) at 128 t + 64 h,
// O_t at 256 + 128 t
constexpr uint32_t kColS = 0, kColO = 256;

struct D128Params {
  __nv_bfloat16* o;      // [B*H, N, 128]
  int* status;
  int N;                 // tokens per (batch, head)
  int gridW, gridH;      // token grid as TMA sees it (F: N x 1)
  int win_w, win_h;      // window extent in (x, y) (F: N x 1)
  int box_w, box_h;      // tile box: box_w * box_h == 128
  int lg_box_w;
  int step_x, step_y;    // origin step from one tile of a window to the next
  int nwx, nwin;         // windows per grid row, per (batch, head)
  int qpairs;            // pairs of query tiles per window (by the full window extent)
  int total_items;       // (batch*head, window, pair), pair fastest
  FastDiv div_qpairs, div_nwin, div_nwx;
  int H;                 // heads per batch element: the inputs are addressed by (head, batch)
  FastDiv div_H;
  float scale_log2;      // softmax scale * log2(e)
};

// One work item: two query tiles of one window of one (batch, head).  F is one window per head: the
// token sequence as an N x 1 grid with boxes of 128 x 1 tokens.
struct Item {
  int bh, x0, y0, x_end, y_end;   // window origin and valid end (exclusive) in the token grid
  int ntiles;                     // tiles of the window: query tiles, and key tiles
  int qt0;                        // first of the item's two query tiles (an item with qt0 >= ntiles is empty)
};
__device__ __forceinline__ Item decode_item(const D128Params& p, int i) {
  Item it;
  const int r = fdiv(i, p.div_qpairs), qp = i - r * p.qpairs;
  it.bh = fdiv(r, p.div_nwin);
  const int win = r - it.bh * p.nwin;
  const int wy = fdiv(win, p.div_nwx), wx = win - wy * p.nwx;
  it.x0 = wx * p.win_w;
  it.y0 = wy * p.win_h;
  it.x_end = min(it.x0 + p.win_w, p.gridW);
  it.y_end = min(it.y0 + p.win_h, p.gridH);
  it.ntiles = p.step_x ? (it.x_end - it.x0 + kTile - 1) / kTile : (it.y_end - it.y0 + p.box_h - 1) / p.box_h;
  it.qt0 = kQT * qp;
  return it;
}

struct __align__(8) Barriers {
  uint64_t q_full[kQT], q_empty[kQT];
  uint64_t k_full[kKS], k_empty[kKS], v_full[kVS], v_empty[kVS];
  uint64_t s_full[kQT][2], p_full[kQT][2];   // per query tile and score buffer
  uint64_t pv_done[kQT];                     // one phase per step: its P V has retired
  uint64_t drain;
  uint32_t tmem_base;
  volatile uint32_t abort_flag;
};
constexpr size_t kSmemTiles = (kQT + kKS + kVS) * (size_t)kTileBytes;          // Q[2] K[3] V[2] = 224 KB
constexpr size_t kSmemBytes = kSmemTiles + sizeof(Barriers) + 1024;            // + alignment slack

constexpr uint32_t kIdescQK = idesc(kTile, kSub, 0);       // S = Q K^T: M128 N64, both operands K-major
constexpr uint32_t kIdescPV = idesc(kTile, kHalfD, 1);     // O half = P V half: M128 N64, V MN-major

// ---- the kernel ------------------------------------------------------------------
// CTA c works on items c, c + gridDim.x, ...  Every role walks the same item sequence on its own;
// ring stages and barrier parities follow running counters.  The second query tile of a head's last
// item does not exist when the head has an odd number of tiles: its softmax warps skip the item, the
// issuer still frees its Q buffer so that arrival counts hold.
__global__ void __launch_bounds__(kThreads, 1)
attn_d128_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                 const __grid_constant__ CUtensorMap mapV, const D128Params p) {
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment by an offset from the array itself, so that accesses stay shared-space loads and stores
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  Barriers* bar = reinterpret_cast<Barriers*>(smem + kSmemTiles);
  const uint32_t sQ = smem_u32(smem), sK = sQ + kQT * kTileBytes, sV = sK + kKS * kTileBytes;

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
      for (int h = 0; h < 2; ++h) {
        mbar_init(&bar->s_full[t][h], 1);
        mbar_init(&bar->p_full[t][h], 128);
      }
      mbar_init(&bar->pv_done[t], 1);
    }
    for (int s = 0; s < kKS; ++s) {
      mbar_init(&bar->k_full[s], 1);
      mbar_init(&bar->k_empty[s], 1);
    }
    for (int s = 0; s < kVS; ++s) {
      mbar_init(&bar->v_full[s], 1);
      mbar_init(&bar->v_empty[s], 1);
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

  const int item0 = blockIdx.x, item_step = gridDim.x;

  if (warp == 0) {
    // ================= TMA producer =================
    // a tile = two boxes of 64 channels x 128 tokens, one per swizzled half
    auto load_tile = [&](uint32_t dst, const CUtensorMap* map, uint64_t* full, int x, int y, int h, int b) {
      mbar_expect_tx(full, kTileBytes);
      tma_load_5d(dst, map, full, 0, x, y, h, b);
      tma_load_5d(dst + kHalfBytes, map, full, kHalfD, x, y, h, b);
    };
    bool ok = true;
    int n = 0;                 // items seen
    int ks = 0, vs = 0;        // ring stages of the next K and V tile
    uint32_t kpar = 1, vpar = 1;   // parity of the "empty" phase this pass over each ring waits for
    int issued_v = 0;          // for the abort path: V copies issued so far
    for (int i = item0; i < p.total_items && ok; i += item_step) {
      const Item it = decode_item(p, i);
      if (it.qt0 >= it.ntiles) continue;
      const int ntiles = it.ntiles, qt0 = it.qt0;
      const int b = fdiv(it.bh, p.div_H), h = it.bh - b * p.H;   // coordinates of the input tensor maps
      for (int t = 0; t < kQT && ok; ++t) {
        ok = warp_wait<kSuspendNs>(&bar->q_empty[t], (n & 1) ^ 1, &bar->abort_flag, p.status);
        if (!ok) break;
        if (qt0 + t < ntiles && elect_one())
          load_tile(sQ + t * kTileBytes, &mapQ, &bar->q_full[t], it.x0 + (qt0 + t) * p.step_x, it.y0 + (qt0 + t) * p.step_y, h, b);
        __syncwarp();
      }
      for (int j = 0; j < ntiles && ok; ++j) {
        ok = warp_wait<kSuspendNs>(&bar->k_empty[ks], kpar, &bar->abort_flag, p.status);
        if (!ok) break;
        if (elect_one()) load_tile(sK + ks * kTileBytes, &mapK, &bar->k_full[ks], it.x0 + j * p.step_x, it.y0 + j * p.step_y, h, b);
        __syncwarp();
        if (++ks == kKS) { ks = 0; kpar ^= 1; }
        ok = warp_wait<kSuspendNs>(&bar->v_empty[vs], vpar, &bar->abort_flag, p.status);
        if (!ok) break;
        if (elect_one()) load_tile(sV + vs * kTileBytes, &mapV, &bar->v_full[vs], it.x0 + j * p.step_x, it.y0 + j * p.step_y, h, b);
        __syncwarp();
        ++issued_v;
        if (++vs == kVS) { vs = 0; vpar ^= 1; }
      }
      ++n;
    }
    if (!ok && lane == 0) {
      // let the copies still in flight land before the CTA leaves (bounded by the same limit)
      const unsigned long long t0 = globaltimer();
      for (int g = max(0, issued_v - kVS); g < issued_v; ++g)
        while (!mbar_try(&bar->v_full[g % kVS], (g / kVS) & 1) && globaltimer() - t0 < kWaitLimitNs) {}
    }
  } else if (warp == 1) {
    // ================= MMA issuer, both query tiles =================
    // Per item and query tile t the work is a chain over 64-key steps u (key tile u / 2, half u % 2):
    //   S_t(u) = Q_t K(u)^T          8 MMAs, M128 N64 K16, operands in shared memory (two channel halves)
    //   O_t   += P_t(u) V(u)         2 x 4 MMAs, M128 N64 K16, A = P in tensor memory, one per channel half of V
    // Two score buffers per tile: the scores of steps u and u + 1 are in flight or done while the softmax
    // works on step u, so it never waits for Q K^T in steady state.  P_t(u) lies over S_t(u) in buffer u % 2,
    // and S_t(u + 2) is issued into that buffer behind P_t(u) V(u): the tensor pipe executes one thread's
    // MMAs in issue order.  pv_done tells the softmax warps that a step's P V has retired (O_t quiescent).
    bool ok = true;
    int sk = 0, sv = 0;                     // ring stages of the score key tile and of the P V key tile
    uint32_t phk = 0, phv = 0;              // and their "full" parities
    uint32_t pcnt[2][2] = {{0, 0}, {0, 0}}; // publications seen so far per tile and buffer: parity of p_full
    uint32_t qcnt[2] = {0, 0};              // items in which the tile existed: parity of q_full
    for (int i = item0; i < p.total_items && ok; i += item_step) {
      const Item it = decode_item(p, i);
      if (it.qt0 >= it.ntiles) continue;
      const int nsteps = 2 * it.ntiles;
      const bool ex[2] = {true, it.qt0 + 1 < it.ntiles};
      // Scores of step u: scores_begin waits for the key tile, scores_tile issues tile x's MMAs into buffer
      // u % 2 (the caller has made sure that the buffer is free: its previous P V has been issued, and one
      // thread's MMAs execute in issue order), scores_end hands the key tile and the query tiles back.
      auto scores_begin = [&](int u) -> bool {
        if ((u & 1) == 0 && !warp_wait<kSuspendNs>(&bar->k_full[sk], phk, &bar->abort_flag, p.status)) return false;
        tc_fence_after();
        return true;
      };
      auto scores_tile = [&](int u, int x) {
        const uint32_t kb = sK + sk * kTileBytes + (u & 1) * (kSub * kHalfD * 2);   // 64 keys = 8 KB into each half tile
        if (elect_one()) {
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const uint64_t dq = smem_desc(sQ + x * kTileBytes + half * kHalfBytes), dk = smem_desc(kb + half * kHalfBytes);
#pragma unroll
            for (int c = 0; c < kHalfD / 16; ++c)
              mma_ss_1(tmem + kColS + x * 128 + (u & 1) * kSub, desc_advance(dq, c * 32), desc_advance(dk, c * 32), kIdescQK,
                       (half > 0 || c > 0) ? 1u : 0u);
          }
        }
        __syncwarp();
        tc_commit(&bar->s_full[x][u & 1]);
      };
      auto scores_end = [&](int u) {
        if ((u & 1) == 1) {
          tc_commit(&bar->k_empty[sk]);
          if (++sk == kKS) { sk = 0; phk ^= 1; }
        }
        if (u == nsteps - 1) {              // the item's last scores: its query tiles may be replaced
          tc_commit(&bar->q_empty[0]);
          tc_commit(&bar->q_empty[1]);
        }
      };
      for (int x = 0; x < 2 && ok; ++x) {
        if (!ex[x]) continue;
        ok = warp_wait<kSuspendNs>(&bar->q_full[x], qcnt[x] & 1, &bar->abort_flag, p.status);
        ++qcnt[x];
      }
      for (int u = 0; u < 2 && ok; ++u) {   // (a key tile is two steps: nsteps >= 2)
        ok = scores_begin(u);
        if (!ok) break;
        for (int x = 0; x < 2; ++x)
          if (ex[x]) scores_tile(u, x);
        scores_end(u);
      }
      for (int u = 0; u < nsteps && ok; ++u) {
        const int hb = u & 1;
        const bool more = u + 2 < nsteps;   // the buffer of step u is free behind its P V: the scores of step u + 2 go there
        if (hb == 0) {                      // P V of a first half: its V must have landed
          ok = warp_wait<kSuspendNs>(&bar->v_full[sv], phv, &bar->abort_flag, p.status);
          if (!ok) break;
        }
        if (more) {
          ok = scores_begin(u + 2);
          if (!ok) break;
        }
        const uint32_t vb = sV + sv * kTileBytes + hb * (kSub * kHalfD * 2);
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          if (!ex[x]) continue;
          ok = warp_wait<kSuspendNs>(&bar->p_full[x][hb], pcnt[x][hb] & 1, &bar->abort_flag, p.status);
          ++pcnt[x][hb];
          if (!ok) break;
          tc_fence_after();
          if (elect_one()) {                 // one lane issues the step's MMAs back to back
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const uint64_t dv = smem_desc(vb + half * kHalfBytes);
#pragma unroll
              for (int c = 0; c < kSub / 16; ++c)
                mma_ts_1(tmem + kColO + x * kD + half * kHalfD, tmem + kColS + x * 128 + hb * kSub + c * 8, desc_advance(dv, c * 2048),
                         kIdescPV, (u > 0 || c > 0) ? 1u : 0u);
            }
          }
          __syncwarp();
          tc_commit(&bar->pv_done[x]);
          if (more) scores_tile(u + 2, x);
        }
        if (!ok) break;
        if (hb == 1) {                      // both halves of the V tile are in flight or done
          tc_commit(&bar->v_empty[sv]);
          if (++sv == kVS) { sv = 0; phv ^= 1; }
        }
        if (more) scores_end(u + 2);
      }
    }
    // Teardown: every MMA issued so far must have retired before tensor memory is released.
    tc_commit(&bar->drain);
    if (lane == 0) {
      const unsigned long long t0 = globaltimer();
      while (!mbar_try(&bar->drain, 0) && globaltimer() - t0 < kWaitLimitNs) {}
    }
    __syncwarp();
  } else {
    // ================= softmax + epilogue: one thread per query row =================
    const int t = (warp - kFirstSoftmaxWarp) >> 2;  // query tile of this warp
    const int q4 = warp & 3;                        // tensor-memory quadrant a warp may touch: warp % 4
    const uint32_t lane_base = (uint32_t)(q4 << 5) << 16;
    const uint32_t tS0 = tmem + lane_base + kColS + t * 128;   // score buffer 0 (buffer 1: + 64); probabilities over a buffer's first 32 columns
    const uint32_t tO = tmem + lane_base + kColO + t * kD;
    const float sl2 = p.scale_log2;
    const float kLazy = 8.f / sl2;                 // the reference maximum moves only when it grew by > 2^8
    const uint64_t sl2x2 = pack2(sl2, sl2);
    bool ok = true;
    uint32_t scnt[2] = {0, 0};        // steps seen by this tile per score buffer: parity of s_full
    uint32_t g = 0;                   // steps seen by this tile in all: phase of pv_done

    for (int i = item0; i < p.total_items && ok; i += item_step) {
      const Item it = decode_item(p, i);
      if (it.qt0 >= it.ntiles) continue;            // an empty item (a short edge window)
      if (it.qt0 + t >= it.ntiles) continue;        // this query tile does not exist
      const int nsteps = 2 * it.ntiles;
      float m = -INFINITY, l = 0.f;
      for (int u = 0; u < nsteps; ++u) {
        const uint32_t tS = tS0 + (u & 1) * kSub;
        ok = warp_wait<kSuspendNs>(&bar->s_full[t][u & 1], scnt[u & 1] & 1, &bar->abort_flag, p.status);
        if (!ok) break;
        ++scnt[u & 1];
        tc_fence_after();
        uint32_t va[32], vb2[32];
        // valid extent of this key tile's box along x and y: a key outside the grid or the window does not exist
        const int vx = it.x_end - (it.x0 + (u >> 1) * p.step_x), vy = it.y_end - (it.y0 + (u >> 1) * p.step_y);
        if (vx < p.box_w || vy < p.box_h) {
          // Edge tile: overwrite the scores of keys that do not exist with -inf in tensor memory, then
          // treat the step like any other.
#pragma unroll 1
          for (int c = 0; c < 2; ++c) {
            const int k0 = 64 * (u & 1) + 32 * c;      // first of the 32 keys, as an index into the box
            uint32_t bits = 0;
            if (p.box_w >= 32) {                       // the 32 keys lie in one box row
              const int ly = k0 >> p.lg_box_w, lx0 = k0 & (p.box_w - 1);
              const int nv = min(32, vx - lx0);
              if (ly < vy && nv > 0) bits = nv >= 32 ? 0xffffffffu : ((1u << nv) - 1u);
            } else {                                   // 32 / box_w whole box rows
              const uint32_t rowbits = (1u << min(vx, p.box_w)) - 1u;
              const int ly0 = k0 >> p.lg_box_w;
              for (int rr = 0; rr < (32 >> p.lg_box_w); ++rr)
                if (ly0 + rr < vy) bits |= rowbits << (rr << p.lg_box_w);
            }
            if (bits != 0xffffffffu) {                 // warp-uniform: the mask depends on the tile only
              tmem_ld32(tS + 32 * c, va);
              tmem_wait_ld(va);
#pragma unroll
              for (int x = 0; x < 32; ++x)
                if (!((bits >> x) & 1u)) va[x] = kNegInf;   // exp2(-inf) = 0 and -inf never wins the maximum
              tmem_st32(tS + 32 * c, va);
            }
          }
          tmem_wait_st();
        }
        // ---- pass 1: the step's maximum; both halves of the scores stay in registers for pass 2
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        tmem_ld32(tS, va);
        tmem_ld32(tS + 32, vb2);
        tmem_wait_ld(va);
        tmem_wait_ld(vb2);
        max32(va, mx4);
        max32(vb2, mx4);
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        bool pv_seen = u == 0;         // every step looks at the phase of the previous step's P V exactly once
        float o_scale = 1.f;
        if (mx > m + kLazy) {          // always true on the first step (m = -inf, mx finite)
          o_scale = ex2((m - mx) * sl2);            // first step: exp2(-inf) = 0
          l *= o_scale;
          m = mx;
        }
        if (u > 0 && __any_sync(0xffffffffu, o_scale != 1.f)) {
          // Rare: the reference moved.  O_t may be touched once the previous step's P V has retired
          // (phase g - 1 of pv_done); the next P V waits for this step's P.
          ok = warp_wait<kSuspendNs>(&bar->pv_done[t], (g - 1) & 1, &bar->abort_flag, p.status);
          if (!ok) break;
          pv_seen = true;
          tc_fence_after();
#pragma unroll 1
          for (int c = 0; c < kD / 32; ++c) {
            uint32_t v[32];
            tmem_ld32(tO + 32 * c, v);
            tmem_wait_ld(v);
#pragma unroll
            for (int x = 0; x < 32; ++x) v[x] = __float_as_uint(__uint_as_float(v[x]) * o_scale);
            tmem_st32(tO + 32 * c, v);
          }
          tmem_wait_st();
        }
        // ---- pass 2: exponentials against the reference, P over the scores just consumed
        const float mneg = -m * sl2;
        const uint64_t mnegx2 = pack2(mneg, mneg);
        uint64_t lsum[4] = {0ull, 0ull, 0ull, 0ull};
        uint32_t pk[16];
        exp32<false, kPolyOf8>(va, sl2x2, mnegx2, lsum, pk, mx4);
        tmem_st16(tS, pk);
        exp32<false, kPolyOf8>(vb2, sl2x2, mnegx2, lsum, pk, mx4);
        tmem_st16(tS + 16, pk);
        float a0, a1, b0, b1;
        unpack2(add2(lsum[0], lsum[1]), a0, a1);
        unpack2(add2(lsum[2], lsum[3]), b0, b1);
        l += (a0 + a1) + (b0 + b1);
        // A parity wait must not skip a phase: the previous step's P V is waited for here at the latest
        // (it retired long ago), before this step's P can set the next one going.
        if (!pv_seen) {
          ok = warp_wait<kSuspendNs>(&bar->pv_done[t], (g - 1) & 1, &bar->abort_flag, p.status);
          if (!ok) break;
        }
        // publish P
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bar->p_full[t][u & 1]);
        ++g;
      }
      if (!ok) break;
      // ---- epilogue: O / l -> bf16 -> this thread's row, 256 contiguous bytes of global memory
      ok = warp_wait<kSuspendNs>(&bar->pv_done[t], (g - 1) & 1, &bar->abort_flag, p.status);   // the item's last P V
      if (!ok) break;
      tc_fence_after();
      const float inv = 1.f / l;
      // this thread's token: row r of the tile's box
      const int r = 32 * q4 + lane;
      const int qx = it.x0 + (it.qt0 + t) * p.step_x + (r & (p.box_w - 1)), qy = it.y0 + (it.qt0 + t) * p.step_y + (r >> p.lg_box_w);
      const bool row_ok = qx < it.x_end && qy < it.y_end;
      __nv_bfloat16* dst = p.o + ((size_t)it.bh * p.N + (size_t)qy * p.gridW + qx) * kD;
#pragma unroll 1
      for (int c = 0; c < kD / 32; ++c) {
        uint32_t v[32];
        tmem_ld32(tO + 32 * c, v);
        tmem_wait_ld(v);
        if (row_ok) {
#pragma unroll
          for (int x = 0; x < 4; ++x)
            *reinterpret_cast<uint4*>(dst + 32 * c + 8 * x) =
                make_uint4(pack_bf16(__uint_as_float(v[8 * x]) * inv, __uint_as_float(v[8 * x + 1]) * inv),
                           pack_bf16(__uint_as_float(v[8 * x + 2]) * inv, __uint_as_float(v[8 * x + 3]) * inv),
                           pack_bf16(__uint_as_float(v[8 * x + 4]) * inv, __uint_as_float(v[8 * x + 5]) * inv),
                           pack_bf16(__uint_as_float(v[8 * x + 6]) * inv, __uint_as_float(v[8 * x + 7]) * inv));
        }
      }
      tc_fence_before();
    }
  }

  // ================= common teardown =================
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

}  // namespace

// F (full = true or one window covering the grid): any N >= 128.  W: windows whose width ww is a power of
// two <= 128 (a tile is a box of ww x 128 / ww tokens), no prefix tokens.
namespace {
struct Geometry {
  int gridW, gridH, win_w, win_h, box_w, box_h, step_x, step_y, nwx, nwy, tiles_per_window;
};
bool geometry(const AttnArgs& a, bool full, Geometry* g) {
  const int N = a.Hg * a.Wg;
  if (full || (a.wh >= a.Hg && a.ww >= a.Wg)) {
    *g = Geometry{N, 1, N, 1, kTile, 1, kTile, 0, 1, 1, ceil_div(N, kTile)};
    return true;
  }
  const int ww = a.ww;
  if (ww < 1 || ww > kTile || (ww & (ww - 1)) != 0) return false;   // box width must divide 128
  const int bh = kTile / ww;
  const int wh = a.wh < a.Hg ? a.wh : a.Hg;
  *g = Geometry{a.Wg, a.Hg, ww, wh, ww, bh, 0, bh, ceil_div(a.Wg, ww), ceil_div(a.Hg, wh), ceil_div(wh, bh)};
  return true;
}
}  // namespace

bool attn_d128_supported(const AttnArgs& a, bool full) {
  if (a.dtype != JV_BF16 || a.D != kD || a.P != 0) return false;
  Geometry g;
  if (!geometry(a, full, &g)) return false;
  if ((int64_t)a.Hg * a.Wg < kTile) return false;           // tiny problems: the generic kernel
  if ((int64_t)g.nwx * g.nwy * ceil_div(g.tiles_per_window, kQT) * a.BH > 0x7fffffffll) return false;
  return encode_fn() != nullptr;
}

cudaError_t launch_attn_d128(const AttnArgs& a, bool full, int* status, cudaStream_t st) {
  Geometry g;
  if (!geometry(a, full, &g)) return cudaErrorInvalidValue;
  EncodeFn enc = encode_fn();
  if (!enc) return cudaErrorNotSupported;
  const int N = a.Hg * a.Wg;
  CUtensorMap maps[3];
  const void* ptrs[3] = {a.q, a.k, a.v};
  // the inputs as (d, x, y, head, batch) with the caller's strides; a box is one 64-channel half of a tile
  const cuuint64_t idims[5] = {(cuuint64_t)kD, (cuuint64_t)g.gridW, (cuuint64_t)g.gridH, (cuuint64_t)a.H, (cuuint64_t)(a.BH / a.H)};
  const cuuint64_t istrides[4] = {(cuuint64_t)a.in.tok * 2, (cuuint64_t)g.gridW * a.in.tok * 2, (cuuint64_t)a.in.head * 2,
                                  (cuuint64_t)a.in.batch * 2};
  const cuuint32_t ibox[5] = {(cuuint32_t)kHalfD, (cuuint32_t)g.box_w, (cuuint32_t)g.box_h, 1, 1};
  const cuuint32_t iestr[5] = {1, 1, 1, 1, 1};
  for (int i = 0; i < 3; ++i) {
    CUresult r = enc(&maps[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(ptrs[i]), idims, istrides, ibox, iestr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }
  static OncePerDevice smem_opt_in;   // > 48 KB of dynamic shared memory: a per-device function attribute
  cudaError_t e = smem_opt_in.run([] {
    return cudaFuncSetAttribute(attn_d128_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  });
  if (e != cudaSuccess) return e;
  D128Params p;
  p.o = (__nv_bfloat16*)a.o;
  p.status = status;
  p.N = N;
  p.gridW = g.gridW;
  p.gridH = g.gridH;
  p.win_w = g.win_w;
  p.win_h = g.win_h;
  p.box_w = g.box_w;
  p.box_h = g.box_h;
  p.lg_box_w = 0;
  while ((1 << p.lg_box_w) < g.box_w) ++p.lg_box_w;
  p.step_x = g.step_x;
  p.step_y = g.step_y;
  p.nwx = g.nwx;
  p.nwin = g.nwx * g.nwy;
  p.qpairs = ceil_div(g.tiles_per_window, kQT);
  p.total_items = p.qpairs * p.nwin * a.BH;
  p.div_qpairs = make_fastdiv((uint32_t)p.qpairs);
  p.div_nwin = make_fastdiv((uint32_t)p.nwin);
  p.div_nwx = make_fastdiv((uint32_t)p.nwx);
  p.H = a.H;
  p.div_H = make_fastdiv((uint32_t)a.H);
  p.scale_log2 = a.scale * 1.4426950408889634f;
  const int num_sms = device_sm_count();
  const int grid = p.total_items < num_sms ? p.total_items : num_sms;
  attn_d128_kernel<<<grid, kThreads, kSmemBytes, st>>>(maps[0], maps[1], maps[2], p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace jv
