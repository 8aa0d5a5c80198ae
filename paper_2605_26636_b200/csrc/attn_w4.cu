// 2-D window attention (Sec. 3.2.2) for windows of one or two 128-token tiles (16 x 16 and the
// like) on the 5th-generation tensor cores: two windows side by side per CTA, four 128-row query
// tiles, so that every SM sub-core holds four softmax warps.  bf16 tensors, head_dim 64, at most 16 prefix tokens.
//
// The softmax of attention at head_dim 64 is bound by the SM's ordinary pipes and their latencies, and a
// window is short work (four 64-key steps per query tile): with two query tiles per CTA (attn_tc.cu) a
// sub-core has two warps to overlap a step's chain  scores -> softmax -> P V  with.  Here a CTA is
// two independent halves ("slots"); each slot walks its own sequence of windows with its own producer
// warp, issuer warp, eight softmax warps and rings of K and V tiles, and shares nothing with the other
// but the SM.  The two slots drift out of phase, so one slot's epilogue and pipeline fill overlap the
// other's steady state.
//
// Warp roles (20 warps):
//   warps 0, 1    TMA producers of slot 0 / 1: per window two Q tiles, K tiles through a ring of two,
//                 V tiles through a ring of three
//   warps 2, 3    MMA issuers of slot 0 / 1, in steps of 64 keys, both query tiles of the window:
//                 O_t += P_t V (A = P from tensor memory) of the previous step, then S_t = Q_t K^T
//   warps 4-19    softmax, one thread per query row (warp w: tile (w - 4) / 4, tensor-memory quadrant w % 4):
//                 exact two-pass softmax per step against a lazily raised reference, P as bf16 over
//                 the scores it came from, final 1/l scaling, store
// Tensor memory: per tile a 64-column score buffer and a 64-column accumulator (4 x 128 = 512 columns).
// Shared memory: Q 4 tiles, K 2 x 2, V 2 x 3 (224 KB).  The output tile of query tile x is staged over
// the V tile x of its own window once both tiles' last P V have retired; the producer may refill that
// stage when the four warps that staged into it have seen their stores read it (v_empty counts them),
// which they check one step into their next window, off the critical path.
// With prefix tokens (template parameter): one more step per window against the prefix rows of K and V,
// which take the shared memory of the third V stage; the rows then go straight to global memory.
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
constexpr int kSlots = 2;                   // windows in flight per CTA
constexpr int kQT = 2 * kSlots;             // query tiles per CTA
constexpr int kKS = 2;                      // K ring depth per slot
constexpr int kVSMax = 3;                   // V ring depth per slot: 3 without prefix tokens (a stage doubles as the
                                            // output's staging tile), 2 with them (rows go straight to global memory)
constexpr int kPreRows = 16;                // prefix keys are one 16-key MMA: P <= 16
constexpr int kPreBytes = kPreRows * kD * 2;   // 2 KB: the prefix rows of K, or of V
constexpr int kWarps = 20;
constexpr int kThreads = kWarps * 32;
constexpr int kFirstSoftmaxWarp = 4;
constexpr uint32_t kTmemCols = 512;
constexpr int kSub = 64;                    // keys per step
constexpr int kPolyOf8 = 2;                 // of every 8 score pairs, this many take the polynomial exponential
// Tensor-memory columns: S_t (and P_t over its first 32 columns) at 64 t, O_t at 256 + 64 t
constexpr uint32_t kColS = 0, kColO = 256;

struct W4Params {
  __nv_bfloat16* o;      // first grid token of (batch, head) 0 (the prefix variant writes rows itself)
  int tokens_per_head;   // P + Hg * Wg
  int P;                 // prefix keys behind every window's own keys (0: none)
  int* status;
  int gridW, gridH;      // token grid
  int win_w, win_h;      // window extent
  int box_w, box_h;      // tile box: box_w * box_h == 128, box_w == win_w
  int lg_box_w;
  int nwx, nwin;         // windows per grid row, per (batch, head)
  int total;             // windows of the whole call: (batch*head, window), window fastest
  FastDiv div_nwin, div_nwx;
  int H;                 // heads per batch element: the inputs are addressed by (head, batch)
  FastDiv div_H;
  float scale_log2;      // softmax scale * log2(e)
};

// One window of one (batch, head)
struct Item {
  int bh, x0, y0, x_end, y_end;   // window origin and valid end (exclusive) in the token grid
  int ntiles;                     // tiles of the window (1 or 2): query tiles, and key tiles
};
__device__ __forceinline__ Item decode_item(const W4Params& p, int r) {
  Item it;
  it.bh = fdiv(r, p.div_nwin);
  const int win = r - it.bh * p.nwin;
  const int wy = fdiv(win, p.div_nwx), wx = win - wy * p.nwx;
  it.x0 = wx * p.win_w;
  it.y0 = wy * p.win_h;
  it.x_end = min(it.x0 + p.win_w, p.gridW);
  it.y_end = min(it.y0 + p.win_h, p.gridH);
  it.ntiles = it.y_end - it.y0 > p.box_h ? 2 : 1;
  return it;
}

struct __align__(8) Barriers {
  uint64_t q_full[kQT], q_empty[kQT];
  uint64_t k_full[kSlots][kKS], k_empty[kSlots][kKS], v_full[kSlots][kVSMax], v_empty[kSlots][kVSMax];
  uint64_t pre_full[kSlots], pre_empty[kSlots];       // the slot's prefix rows of K and V
  uint64_t s_full[kQT], p_full[kQT], o_full[kQT];
  uint64_t drain;
  uint32_t tmem_base;
  volatile uint32_t abort_flag;
};
// shared memory: Q[4] | K[2][2] | V[2][kVS] | (prefix variant: per slot the prefix rows of K, then of V) | barriers
template <bool kPrefix>
struct Layout {
  static constexpr int kVS = kPrefix ? 2 : 3;
  static constexpr size_t kTiles = (kQT + kSlots * (kKS + kVS)) * (size_t)kTileBytes;
  static constexpr size_t kPre = kPrefix ? (size_t)kSlots * 2 * kPreBytes : 0;
  static constexpr size_t kBytes = kTiles + kPre + sizeof(Barriers) + 1024;          // + alignment slack
};

constexpr uint32_t kIdescQK = idesc(kTile, kSub, 0);
constexpr uint32_t kIdescPV = idesc(kTile, kD, 1);
constexpr uint32_t kIdescQKpre = idesc(kTile, kPreRows, 0);   // scores against the 16 prefix rows

__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

// ---- the kernel ------------------------------------------------------------------
// Slot s of CTA c works on windows 2 c + s, 2 c + s + 2 gridDim.x, ...  Every role of a slot walks that
// sequence on its own; ring stages and barrier parities follow running counters.  The second query
// tile of a window that has one tile only (a bottom edge window) is skipped by its softmax warps;
// the issuer still frees its Q buffer so that arrival counts hold.
// kPrefix: every window's queries also attend the P <= 16 prefix tokens of their (batch, head): one more
// step per window with a 16-key score MMA against the prefix rows of K (kept in shared memory per slot,
// reloaded per window from L2) and a 16-key P V.  The prefix QUERIES are not this kernel's work.
template <bool kPrefix>
__global__ void __launch_bounds__(kThreads, 1)
attn_w4_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
               const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapO,
               const __grid_constant__ CUtensorMap mapKp, const __grid_constant__ CUtensorMap mapVp, const W4Params p) {
  constexpr int kVS = Layout<kPrefix>::kVS;
  constexpr size_t kSmemTiles = Layout<kPrefix>::kTiles;
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment by an offset from the array itself, so that accesses stay shared-space loads and stores
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  Barriers* bar = reinterpret_cast<Barriers*>(smem + kSmemTiles + Layout<kPrefix>::kPre);
  const uint32_t sQ = smem_u32(smem), sK = sQ + kQT * kTileBytes, sV = sK + kSlots * kKS * kTileBytes;
  const uint32_t sPre = sQ + (uint32_t)kSmemTiles;   // slot s: prefix rows of K at s * 4 KB, of V 2 KB behind them

  // a grid launched behind this one with programmatic serialisation (the prefix queries of W, which
  // depend on nothing here) may run beside it
  if (kPrefix) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

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
    for (int s = 0; s < kSlots; ++s) {
      for (int g = 0; g < kKS; ++g) {
        mbar_init(&bar->k_full[s][g], 1);
        mbar_init(&bar->k_empty[s][g], 1);
      }
      for (int g = 0; g < kVS; ++g) {
        mbar_init(&bar->v_full[s][g], 1);
        // handed back by the four softmax warps that staged their output into it, or (prefix variant) by the issuer
        mbar_init(&bar->v_empty[s][g], kPrefix ? 1 : 4);
      }
      mbar_init(&bar->pre_full[s], 1);
      mbar_init(&bar->pre_empty[s], 1);
    }
    mbar_init(&bar->drain, kSlots);
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

  const int item_step = kSlots * gridDim.x;

  if (warp < kSlots) {
    // ================= TMA producer of slot `warp` =================
    const int s = warp;
    bool ok = true;
    int n = 0;                       // windows seen
    int ks = 0, vs = 0;              // ring stages of the next K and V tile
    uint32_t kpar = 1, vpar = 1;     // parity of the "empty" phase this pass over each ring waits for
    int issued_v = 0;                // for the abort path: V copies issued so far
    for (int r = kSlots * blockIdx.x + s; r < p.total && ok; r += item_step) {
      const Item it = decode_item(p, r);
      const int b = fdiv(it.bh, p.div_H), h = it.bh - b * p.H;   // coordinates of the input tensor maps
      for (int x = 0; x < 2 && ok; ++x) {
        const int t = 2 * s + x;
        ok = warp_wait<kSuspendNs>(&bar->q_empty[t], (n & 1) ^ 1, &bar->abort_flag, p.status);
        if (!ok) break;
        if (x < it.ntiles && elect_one()) {
          mbar_expect_tx(&bar->q_full[t], kTileBytes);
          tma_load_5d(sQ + t * kTileBytes, &mapQ, &bar->q_full[t], 0, it.x0, it.y0 + x * p.box_h, h, b);
        }
        __syncwarp();
      }
      for (int j = 0; j < it.ntiles && ok; ++j) {      // in the order the issuer needs them: K0, V0, K1, V1
        ok = warp_wait<kSuspendNs>(&bar->k_empty[s][ks], kpar, &bar->abort_flag, p.status);
        if (!ok) break;
        if (elect_one()) {
          mbar_expect_tx(&bar->k_full[s][ks], kTileBytes);
          tma_load_5d(sK + (s * kKS + ks) * kTileBytes, &mapK, &bar->k_full[s][ks], 0, it.x0, it.y0 + j * p.box_h, h, b);
        }
        __syncwarp();
        if (++ks == kKS) { ks = 0; kpar ^= 1; }
        ok = warp_wait<kSuspendNs>(&bar->v_empty[s][vs], vpar, &bar->abort_flag, p.status);
        if (!ok) break;
        if (elect_one()) {
          mbar_expect_tx(&bar->v_full[s][vs], kTileBytes);
          tma_load_5d(sV + (s * kVS + vs) * kTileBytes, &mapV, &bar->v_full[s][vs], 0, it.x0, it.y0 + j * p.box_h, h, b);
        }
        __syncwarp();
        ++issued_v;
        if (++vs == kVS) { vs = 0; vpar ^= 1; }
      }
      if (kPrefix && ok) {            // the prefix rows of K and V of this (batch, head): rows past P arrive as zeros
        ok = warp_wait<kSuspendNs>(&bar->pre_empty[s], (n & 1) ^ 1, &bar->abort_flag, p.status);
        if (!ok) break;
        if (elect_one()) {
          mbar_expect_tx(&bar->pre_full[s], 2 * kPreBytes);
          tma_load_4d(sPre + s * 2 * kPreBytes, &mapKp, &bar->pre_full[s], 0, 0, h, b);
          tma_load_4d(sPre + s * 2 * kPreBytes + kPreBytes, &mapVp, &bar->pre_full[s], 0, 0, h, b);
        }
        __syncwarp();
      }
      ++n;
    }
    if (!ok && lane == 0) {
      // let the copies still in flight land before the CTA leaves (bounded by the same limit)
      const unsigned long long t0 = globaltimer();
      for (int g = max(0, issued_v - kVS); g < issued_v; ++g)
        while (!mbar_try(&bar->v_full[s][g % kVS], (g / kVS) & 1) && globaltimer() - t0 < kWaitLimitNs) {}
    }
  } else if (warp < 2 * kSlots) {
    // ================= MMA issuer of slot `warp - 2`: both query tiles of the slot's window =================
    // Per window and query tile t the work is a chain over 64-key steps u (key tile u / 2, half u % 2):
    //   S_t(u) = Q_t K(u)^T          4 MMAs, M128 N64 K16, operands in shared memory
    //   O_t   += P_t(u) V(u)         4 MMAs, M128 N64 K16, A = P in tensor memory
    // P_t(u) lies over S_t(u), so S_t(u + 1) is issued behind P_t(u) V(u): the tensor pipe executes one
    // thread's MMAs in issue order.  The commit that publishes S_t(u + 1) therefore also tells the
    // softmax warps that P_t(u) V(u) has retired and O_t is quiescent.
    const int s = warp - kSlots, tb = 2 * s;
    bool ok = true;
    int sk = 0, sv = 0;                     // ring stages of the score key tile and of the P V key tile
    uint32_t phk = 0, phv = 0;              // and their "full" parities
    uint32_t pcnt[2] = {0, 0};              // steps published so far per tile: parity of p_full
    uint32_t qcnt[2] = {0, 0};              // windows in which the tile existed: parity of q_full
    uint32_t pre_cnt = 0;                   // windows seen: parity of pre_full
    for (int r = kSlots * blockIdx.x + s; r < p.total && ok; r += item_step) {
      const Item it = decode_item(p, r);
      const int nsteps = 2 * it.ntiles;               // steps against the window's own keys
      const int ns = nsteps + (kPrefix ? 1 : 0);      // and, behind them, one against the prefix rows
      for (int u = 0; u <= ns && ok; ++u) {
        const bool has_qk = u < nsteps, has_pre_qk = kPrefix && u == nsteps;          // scores of step u
        const bool has_pv = u > 0 && u <= nsteps, has_pre_pv = kPrefix && u == ns;    // P V of step u - 1
        if (has_qk && (u & 1) == 0) {       // first half of a key tile: its K must have landed
          ok = warp_wait<kSuspendNs>(&bar->k_full[s][sk], phk, &bar->abort_flag, p.status);
          if (!ok) break;
        }
        if (has_pv && ((u - 1) & 1) == 0) { // P V of a first half: its V must have landed
          ok = warp_wait<kSuspendNs>(&bar->v_full[s][sv], phv, &bar->abort_flag, p.status);
          if (!ok) break;
        }
        if (has_pre_qk) {                   // the prefix rows of K and V must have landed
          ok = warp_wait<kSuspendNs>(&bar->pre_full[s], pre_cnt & 1, &bar->abort_flag, p.status);
          ++pre_cnt;
          if (!ok) break;
        }
        const uint32_t kb = sK + (s * kKS + sk) * kTileBytes + (u & 1) * (kSub * kD * 2);
        const uint32_t vb = sV + (s * kVS + sv) * kTileBytes + ((u - 1) & 1) * (kSub * kD * 2);
        const uint32_t kpb = sPre + s * 2 * kPreBytes, vpb = kpb + kPreBytes;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          if (x >= it.ntiles) continue;
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
              for (int c = 0; c < kSub / 16; ++c)
                mma_ts_1(tmem + kColO + t * kD, tmem + kColS + t * kSub + c * 8, desc_advance(dv, c * 2048), kIdescPV,
                         (u > 1 || c > 0) ? 1u : 0u);
            }
            if (has_pre_pv)                  // 16 prefix keys: one MMA of K = 16
              mma_ts_1(tmem + kColO + t * kD, tmem + kColS + t * kSub, smem_desc(vpb), kIdescPV, 1u);
            if (has_qk) {
              const uint64_t dq = smem_desc(sQ + t * kTileBytes), dk = smem_desc(kb);
#pragma unroll
              for (int c = 0; c < kD / 16; ++c)
                mma_ss_1(tmem + kColS + t * kSub, desc_advance(dq, c * 32), desc_advance(dk, c * 32), kIdescQK, c > 0);
            }
            if (has_pre_qk) {                // scores against the prefix rows: 16 columns
              const uint64_t dq = smem_desc(sQ + t * kTileBytes), dk = smem_desc(kpb);
#pragma unroll
              for (int c = 0; c < kD / 16; ++c)
                mma_ss_1(tmem + kColS + t * kSub, desc_advance(dq, c * 32), desc_advance(dk, c * 32), kIdescQKpre, c > 0);
            }
          }
          __syncwarp();
          if (u < ns) tc_commit(&bar->s_full[t]);
          else tc_commit(&bar->o_full[t]);
        }
        if (!ok) break;
        if (has_pv && ((u - 1) & 1) == 1) { // both halves of the V tile are in flight or done
          // without prefix tokens the stage is handed back by the softmax warps that stage their output over it
          if (kPrefix) tc_commit(&bar->v_empty[s][sv]);
          if (++sv == kVS) { sv = 0; phv ^= 1; }
        }
        if (has_qk && (u & 1) == 1) {
          tc_commit(&bar->k_empty[s][sk]);
          if (++sk == kKS) { sk = 0; phk ^= 1; }
        }
        if (u == ns - 1) {                  // the window's last scores: its query tiles may be replaced
          tc_commit(&bar->q_empty[tb]);
          tc_commit(&bar->q_empty[tb + 1]);
        }
        if (has_pre_pv) tc_commit(&bar->pre_empty[s]);
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
    const int s = t >> 1, x = t & 1;                // its slot, and which of the window's two tiles
    const int q4 = warp & 3;                        // tensor-memory quadrant a warp may touch: warp % 4
    const uint32_t lane_base = (uint32_t)(q4 << 5) << 16;
    const uint32_t tS = tmem + lane_base + kColS + t * kSub;   // scores; probabilities over their first 32 columns
    const uint32_t tO = tmem + lane_base + kColO + t * kD;
    const float sl2 = p.scale_log2;
    const float kLazy = 8.f / sl2;                 // the reference maximum moves only when it grew by > 2^8
    const uint64_t sl2x2 = pack2(sl2, sl2);
    const int sub_y = q4 * (p.box_h >> 2);          // this warp's 32 rows are box_h / 4 whole box rows
    bool ok = true;
    uint32_t scnt = 0;                // steps seen by this tile: parity of s_full
    uint32_t n_all = 0, n_two = 0;    // windows seen, and those of them with two tiles: parities of o_full
    int vrun = 0;                     // ring stage of the window's first V tile
    int held = -1;                    // V stage this warp staged its last output into and has not handed back yet

    // hand back the stage once this warp's store has read it (nothing to wait for if the warp stored nothing)
    auto release = [&]() {
      if (held >= 0) {
        if (lane == 0) {
          asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          mbar_arrive(&bar->v_empty[s][held]);
        }
        __syncwarp();
        held = -1;
      }
    };

    for (int r = kSlots * blockIdx.x + s; r < p.total && ok; r += item_step) {
      const Item it = decode_item(p, r);
      const int stage = (vrun + x) % kVS;
      vrun = (vrun + it.ntiles) % kVS;
      const uint32_t par_own = (x == 0 ? n_all : n_two) & 1, par_other = (x == 0 ? n_two : n_all) & 1;
      ++n_all;
      if (it.ntiles == 2) ++n_two;
      if (x >= it.ntiles) {           // this query tile does not exist
        if (!kPrefix) release();
        continue;
      }
      const int nsteps = 2 * it.ntiles;               // steps against the window's own keys
      const int ns = nsteps + (kPrefix ? 1 : 0);      // and, behind them, one against the prefix rows
      const int vx = it.x_end - it.x0;                   // valid columns of every box of this window
      float m = -INFINITY, l = 0.f;
      for (int u = 0; u < ns; ++u) {
        const bool pre = kPrefix && u == nsteps;      // the step of the prefix keys: 16 score columns, P of them keys
        ok = warp_wait<kSuspendNs>(&bar->s_full[t], scnt & 1, &bar->abort_flag, p.status);
        if (!ok) break;
        ++scnt;
        tc_fence_after();
        uint32_t va[32];
        const int vy = it.y_end - (it.y0 + (u >> 1) * p.box_h);    // valid rows of this key tile's box
        if (pre) {
          // Columns 0 .. P - 1 hold the scores against the prefix keys; up to column 31 everything else
          // (scores against the zero rows behind them, the previous step's leftovers) becomes -inf.
          tmem_ld32(tS, va);
          tmem_wait_ld(va);
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (i >= p.P) va[i] = kNegInf;
          tmem_st32(tS, va);
          tmem_wait_st();
        } else if (vx < p.box_w || vy < p.box_h) {
          // Edge tile: overwrite the scores of keys outside the grid with -inf in tensor memory, then
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
              for (int i = 0; i < 32; ++i)
                if (!((bits >> i) & 1u)) va[i] = kNegInf;   // exp2(-inf) = 0 and -inf never wins the maximum
              tmem_st32(tS + 32 * c, va);
            }
          }
          tmem_wait_st();
        }
        // ---- pass 1: the step's maximum (second half first, so that the first half is the one
        // left in registers for pass 2)
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        if (!pre) {
          tmem_ld32(tS + 32, va);
          tmem_wait_ld(va);
          max32(va, mx4);
        }
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
            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * o_scale);
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
        if (!pre) {
          tmem_ld32(tS + 32, va);
          tmem_wait_ld(va);
          exp32<false, kPolyOf8>(va, sl2x2, mnegx2, lsum, pk, mx4);
          tmem_st16(tS + 16, pk);
        }
        float a0, a1, b0, b1;
        unpack2(add2(lsum[0], lsum[1]), a0, a1);
        unpack2(add2(lsum[2], lsum[3]), b0, b1);
        l += (a0 + a1) + (b0 + b1);
        // publish P
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bar->p_full[t]);
        if (!kPrefix && u == 0) release();   // the previous window's store has long read its staging quarter
      }
      if (!ok) break;
      if (kPrefix) {
        // ---- epilogue with prefix tokens: O / l -> bf16 -> this thread's row, 128 contiguous bytes of global memory
        ok = warp_wait<kSuspendNs>(&bar->o_full[t], par_own, &bar->abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        const float inv = 1.f / l;
        const int rr = 32 * q4 + lane;                                     // row of the tile's box
        const int qx = it.x0 + (rr & (p.box_w - 1)), qy = it.y0 + x * p.box_h + (rr >> p.lg_box_w);
        const bool row_ok = qx < it.x_end && qy < it.y_end;
        __nv_bfloat16* dst = p.o + ((size_t)it.bh * p.tokens_per_head + (size_t)qy * p.gridW + qx) * kD;
#pragma unroll 1
        for (int c = 0; c < 2; ++c) {
          uint32_t v[32];
          tmem_ld32(tO + 32 * c, v);
          tmem_wait_ld(v);
          if (row_ok) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
              *reinterpret_cast<uint4*>(dst + 32 * c + 8 * i) =
                  make_uint4(pack_bf16(__uint_as_float(v[8 * i]) * inv, __uint_as_float(v[8 * i + 1]) * inv),
                             pack_bf16(__uint_as_float(v[8 * i + 2]) * inv, __uint_as_float(v[8 * i + 3]) * inv),
                             pack_bf16(__uint_as_float(v[8 * i + 4]) * inv, __uint_as_float(v[8 * i + 5]) * inv),
                             pack_bf16(__uint_as_float(v[8 * i + 6]) * inv, __uint_as_float(v[8 * i + 7]) * inv));
          }
        }
        tc_fence_before();
        continue;
      }
      // ---- epilogue: O / l -> bf16 -> this warp's quarter of the V tile x of this window -> one TMA store.
      // Both query tiles' last P V read that V tile: both must have retired.
      ok = warp_wait<kSuspendNs>(&bar->o_full[t], par_own, &bar->abort_flag, p.status);
      if (ok && it.ntiles == 2) ok = warp_wait<kSuspendNs>(&bar->o_full[t ^ 1], par_other, &bar->abort_flag, p.status);
      if (!ok) break;
      tc_fence_after();
      const float inv = 1.f / l;
      const int wx0 = it.x0, wy0 = it.y0 + x * p.box_h + sub_y;           // origin of this warp's sub-box
      const bool store = wx0 < it.x_end && wy0 < it.y_end;                // else none of its rows exists
      unsigned char* stg = smem + (size_t)(kQT + kSlots * kKS + s * kVS + stage) * kTileBytes + q4 * 4096;
#pragma unroll 1
      for (int c = 0; c < 2; ++c) {
        uint32_t v[32];
        tmem_ld32(tO + 32 * c, v);
        tmem_wait_ld(v);
        if (store) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {     // 16-byte chunk 4 c + i of this row, at its 128-byte-swizzle position
            const uint4 w = make_uint4(pack_bf16(__uint_as_float(v[8 * i]) * inv, __uint_as_float(v[8 * i + 1]) * inv),
                                       pack_bf16(__uint_as_float(v[8 * i + 2]) * inv, __uint_as_float(v[8 * i + 3]) * inv),
                                       pack_bf16(__uint_as_float(v[8 * i + 4]) * inv, __uint_as_float(v[8 * i + 5]) * inv),
                                       pack_bf16(__uint_as_float(v[8 * i + 6]) * inv, __uint_as_float(v[8 * i + 7]) * inv));
            *reinterpret_cast<uint4*>(stg + lane * 128 + (((4 * c + i) ^ (lane & 7)) << 4)) = w;
          }
        }
      }
      tc_fence_before();
      if (store) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          tma_store_4d(&mapO, smem_u32(stg), 0, wx0, wy0, it.bh);   // rows past the grid edge are clipped
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      }
      held = stage;
    }
    if (!kPrefix && ok) release();
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

}  // namespace

// Windows of exactly one or two tile boxes (box = window width x 128 / width rows); at most 16 prefix tokens
// (contiguous inputs only: the prefix rows are found behind a.k and a.v).
bool attn_w4_supported(const AttnArgs& a) {
  if (a.dtype != JV_BF16 || a.D != kD) return false;
  if (a.P > kPreRows || (a.P > 0 && a.strided)) return false;
  if (a.wh >= a.Hg && a.ww >= a.Wg) return false;         // one window: full attention's kernels
  const int ww = a.ww;
  if (ww < 1 || ww > 32 || (ww & (ww - 1)) != 0) return false;   // a warp's 32 rows are whole box rows
  const int bh = kTile / ww;
  if (a.wh != bh && a.wh != 2 * bh) return false;
  const int64_t nwin = (int64_t)ceil_div(a.Wg, ww) * ceil_div(a.Hg, a.wh);
  if (nwin * a.BH > 0x7fffffffll) return false;
  return encode_fn() != nullptr;
}

cudaError_t launch_attn_w4(const AttnArgs& a, int* status, cudaStream_t st) {
  EncodeFn enc = encode_fn();
  if (!enc) return cudaErrorNotSupported;
  const int N = a.P + a.Hg * a.Wg;                     // tokens per (batch, head): prefix tokens, then the grid
  const int box_w = a.ww, box_h = kTile / a.ww;
  CUtensorMap maps[6];
  // the grid tokens start behind the prefix rows
  const size_t grid0 = (size_t)a.P * kD * 2, igrid0 = (size_t)a.P * (size_t)a.in.tok * 2;
  const void* ptrs[4] = {(const char*)a.q + igrid0, (const char*)a.k + igrid0, (const char*)a.v + igrid0, (char*)a.o + grid0};
  const cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)a.Wg, (cuuint64_t)a.Hg, (cuuint64_t)a.BH};
  const cuuint64_t strides[3] = {(cuuint64_t)kD * 2, (cuuint64_t)a.Wg * kD * 2, (cuuint64_t)N * kD * 2};
  // the output is stored per warp: a quarter of the tile's box (32 tokens)
  const cuuint32_t qbox[4] = {(cuuint32_t)kD, (cuuint32_t)box_w, (cuuint32_t)(box_h / 4), 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  // the inputs as (d, x, y, head, batch) with the caller's strides; the output as (d, x, y, batch*head)
  const cuuint64_t idims[5] = {(cuuint64_t)kD, (cuuint64_t)a.Wg, (cuuint64_t)a.Hg, (cuuint64_t)a.H, (cuuint64_t)(a.BH / a.H)};
  const cuuint64_t istrides[4] = {(cuuint64_t)a.in.tok * 2, (cuuint64_t)a.Wg * a.in.tok * 2, (cuuint64_t)a.in.head * 2,
                                  (cuuint64_t)a.in.batch * 2};
  const cuuint32_t ibox[5] = {(cuuint32_t)kD, (cuuint32_t)box_w, (cuuint32_t)box_h, 1, 1};
  const cuuint32_t iestr[5] = {1, 1, 1, 1, 1};
  for (int i = 0; i < 4; ++i) {
    CUresult r = i < 3 ? enc(&maps[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(ptrs[i]), idims, istrides, ibox,
                             iestr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE)
                       : enc(&maps[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptrs[i]), dims, strides, qbox,
                             estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }
  // the P prefix rows of K and V as (d, row, head, batch), a box of 16 rows: rows past P arrive as zeros
  maps[4] = maps[1];
  maps[5] = maps[2];
  if (a.P > 0) {
    const cuuint64_t pdims[4] = {(cuuint64_t)kD, (cuuint64_t)a.P, (cuuint64_t)a.H, (cuuint64_t)(a.BH / a.H)};
    const cuuint64_t pstrides[3] = {(cuuint64_t)a.in.tok * 2, (cuuint64_t)a.in.head * 2, (cuuint64_t)a.in.batch * 2};
    const cuuint32_t pbox[4] = {(cuuint32_t)kD, (cuuint32_t)kPreRows, 1, 1};
    const void* pptrs[2] = {a.k, a.v};
    for (int i = 0; i < 2; ++i) {
      CUresult r = enc(&maps[4 + i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(pptrs[i]), pdims, pstrides, pbox,
                       estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
  }
  static OncePerDevice smem_opt_in;   // > 48 KB of dynamic shared memory: a per-device function attribute
  cudaError_t e = smem_opt_in.run([] {
    cudaError_t r = cudaFuncSetAttribute(attn_w4_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)Layout<false>::kBytes);
    if (r == cudaSuccess)
      r = cudaFuncSetAttribute(attn_w4_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Layout<true>::kBytes);
    return r;
  });
  if (e != cudaSuccess) return e;
  W4Params p;
  p.o = (__nv_bfloat16*)a.o + (size_t)a.P * kD;        // first grid token of (batch, head) 0
  p.tokens_per_head = N;
  p.P = a.P;
  p.status = status;
  p.gridW = a.Wg;
  p.gridH = a.Hg;
  p.win_w = a.ww;
  p.win_h = a.wh;
  p.box_w = box_w;
  p.box_h = box_h;
  p.lg_box_w = 0;
  while ((1 << p.lg_box_w) < box_w) ++p.lg_box_w;
  p.nwx = ceil_div(a.Wg, a.ww);
  p.nwin = p.nwx * ceil_div(a.Hg, a.wh);
  p.total = p.nwin * a.BH;
  p.div_nwin = make_fastdiv((uint32_t)p.nwin);
  p.div_nwx = make_fastdiv((uint32_t)p.nwx);
  p.H = a.H;
  p.div_H = make_fastdiv((uint32_t)a.H);
  p.scale_log2 = a.scale * 1.4426950408889634f;
  const int num_sms = device_sm_count();
  const int want = ceil_div(p.total, kSlots);
  const int grid = want < num_sms ? want : num_sms;
  if (a.P > 0) {
    attn_w4_kernel<true><<<grid, kThreads, Layout<true>::kBytes, st>>>(maps[0], maps[1], maps[2], maps[3], maps[4], maps[5], p);
  } else {
    attn_w4_kernel<false><<<grid, kThreads, Layout<false>::kBytes, st>>>(maps[0], maps[1], maps[2], maps[3], maps[4], maps[5], p);
  }
  count_launch();
  return cudaGetLastError();
}

}  // namespace jv
