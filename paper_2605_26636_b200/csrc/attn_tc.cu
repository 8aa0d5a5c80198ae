// Full (Eq. 1) and window (Sec. 3.2.2) softmax attention on the 5th-generation
// tensor cores: tcgen05.mma with accumulators in tensor memory, operands staged by
// TMA.  bf16 tensors, head_dim 64.
//
// One kernel serves both mixers.  The token grid is described to TMA as a 4-D tensor
// (d, x, y, batch*head); a "tile" is a box of 128 tokens: 128 consecutive tokens for
// F (x = token index, y = 0), ww x (128/ww) tokens of a window for W.  Keys outside
// the grid arrive as zeros from TMA's out-of-bounds fill and are masked to -inf before
// the softmax; query rows outside the grid / window are never stored.
//
// Persistent CTAs (one per SM) loop over work items; an item is two 128-row query tiles
// against all key tiles of their window.  Warp roles:
//   warp 0        TMA producer: Q tiles (two buffers), K and V tiles through 4-stage rings
//   warps 1, 2    MMA issuers (one elected lane each; warp 1 + t serves query tile t), in steps of 64 keys:
//                 S_t = Q_t K^T (operands in smem, M128 N64 K64),
//                 O_t += P_t V (A = P from tensor memory, B = V MN-major, M128 N64 K64)
//   warps 4-7     softmax of query tile 0   } one thread per query row: fp32 online
//   warps 8-11    softmax of query tile 1   } softmax (exp2 domain, lazy rescale),
//                 P as bf16 back into tensor memory, final 1/l scaling and the store.
// Scores and probabilities are double-buffered per query tile, so the score MMA of step
// u + 2 is issued as soon as the probabilities of step u are published and the softmax
// warps never wait for the tensor pipe in steady state.
//
// Tensor memory (512 columns): scores S(t, b) 4 x 64 in [0, 256), accumulators O(t) 2 x 64
// in [256, 384), probabilities P(t, b) 4 x 32 in [384, 512).
//
// Prefix tokens (P of them in front of the grid tokens; W only): every window's queries also
// attend the P prefix keys.  They come in as one more key tile behind the window's own (a box of
// a second pair of tensor maps that view the prefix rows in the box's shape), with the keys past P
// masked like keys outside the grid.  The P prefix queries themselves (which attend everything)
// are not served here.
//
// Every mbarrier wait is bounded: a wait that runs out sets the device status word,
// raises a CTA-wide abort flag, and every role falls through to the common teardown
// (tensor memory is always released).
#include <type_traits>

#include "tc_common.cuh"

namespace jv {
namespace {

using namespace tc;

#ifndef JV_ATTN_SUSPEND_NS
#define JV_ATTN_SUSPEND_NS 4000
#endif
constexpr uint32_t kSuspendNs = JV_ATTN_SUSPEND_NS;   // suspend-time hint of this kernel's barrier waits (tc_common.cuh)
constexpr int kD = 64;
constexpr int kTile = 128;                 // tokens per tile (MMA M and key-tile N)
constexpr int kTileBytes = kTile * kD * 2; // 16 KB
constexpr int kStages = 4;                 // K and V ring depth
constexpr int kThreads = 384;
constexpr uint32_t kTmemCols = 512;
constexpr int kSub = 64;                    // keys per softmax / MMA step: half a key tile
#ifndef JV_POLY_OF_8
#define JV_POLY_OF_8 1
#endif
constexpr int kPolyOf8 = JV_POLY_OF_8;                 // of every 8 score pairs, this many take the polynomial exponential
// Tensor-memory columns: S(t, b) at kColS + (2 t + b) * 64, O(t) at kColO + 64 t, P(t, b) at kColP + (2 t + b) * 32
constexpr uint32_t kColS = 0, kColO = 256, kColP = 384;

struct TcParams {
  __nv_bfloat16* o;
  int* status;
  int gridW, gridH;      // token grid as TMA sees it (F: N x 1)
  int tokens_per_head;   // N
  int win_w, win_h;      // window extent in (x, y) (F: N x 1)
  int box_w, box_h;      // tile box: box_w * box_h == 128
  int step_x, step_y;    // origin step from one tile of a window to the next
  int nwx;               // windows per grid row
  int nwin;              // windows per (batch, head)
  int qpairs;            // pairs of query tiles per window (by the full window height)
  int total_items;       // work items: (batch*head, window, query-tile pair), pair index fastest
  int lg_box_h;          // log2(box_h)
  int P;                 // prefix keys behind every window's own key tiles (0: none)
  FastDiv div_qpairs, div_nwin, div_nwx;
  int H;                 // heads per batch element: the inputs are addressed by (head, batch)
  FastDiv div_H;
  float scale_log2;      // softmax scale * log2(e)
};

// One work item of the persistent loop: two query tiles of one window of one (batch, head).
struct Item {
  int bh, x0, y0, x_end, y_end;   // window origin and valid end (exclusive) in the token grid
  int ntiles;                     // tiles of the window (query tiles, and key tiles of its own tokens)
  int nkt;                        // key tiles: the window's own, then one of prefix tokens if there are any
  int qt0;                        // first of the two query tiles
};
__device__ __forceinline__ Item decode_item(const TcParams& p, int i) {
  Item it;
  const int r = fdiv(i, p.div_qpairs), qp = i - r * p.qpairs;
  it.bh = fdiv(r, p.div_nwin);
  const int win = r - it.bh * p.nwin;
  const int wy = fdiv(win, p.div_nwx), wx = win - wy * p.nwx;
  it.x0 = wx * p.win_w;
  it.y0 = wy * p.win_h;
  it.x_end = min(it.x0 + p.win_w, p.gridW);
  it.y_end = min(it.y0 + p.win_h, p.gridH);
  it.ntiles = p.step_x ? (it.x_end - it.x0 + kTile - 1) / kTile : (it.y_end - it.y0 + p.box_h - 1) >> p.lg_box_h;
  it.nkt = it.ntiles + (p.P > 0 ? 1 : 0);
  it.qt0 = 2 * qp;                // an item with qt0 >= ntiles (short edge window) is empty: every role skips it
  return it;
}

// ---- shared-memory layout -------------------------------------------------------
struct __align__(8) Barriers {
  uint64_t q_full[2], q_empty[2];                     // the two query buffers (items alternate)
  uint64_t k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
  uint64_t s_full[2][2], p_full[2][2], pv_done[2], o_full[2];
  uint64_t drain;
  uint32_t tmem_base;
  volatile uint32_t abort_flag;
};
constexpr size_t kSmemTiles = (6 + 2 * kStages) * (size_t)kTileBytes;          // Q[2][2] K[kStages] V[kStages] O[2]
constexpr size_t kSmemBytes = kSmemTiles + sizeof(Barriers) + 1024;            // + alignment slack

constexpr uint32_t kIdescQK = idesc(kTile, kSub, 0);
constexpr uint32_t kIdescPV = idesc(kTile, kD, 1);

// ---- the kernel ------------------------------------------------------------------
// Persistent: CTA c works on items c, c + gridDim.x, ...  Every role walks the same item
// sequence on its own; ring stages and barrier parities follow running counters (key tiles
// and items seen so far), so the pipeline runs straight through item boundaries: the next
// item's Q, K and V are already in flight, and its first scores already issued, while the
// current item is being finished and stored.
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
               const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapO,
               const __grid_constant__ CUtensorMap mapKp, const __grid_constant__ CUtensorMap mapVp, const TcParams p) {
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment by an offset from the array itself, so that accesses stay shared-space loads and stores
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  Barriers* bar = reinterpret_cast<Barriers*>(smem + kSmemTiles);
  // Q buffer b holds the two query tiles of an item at sQ + b * 2 tiles
  const uint32_t sQ = smem_u32(smem), sK = sQ + 4 * kTileBytes, sV = sK + kStages * kTileBytes;
  const uint32_t sO = sV + kStages * kTileBytes;      // output staging, one tile per query tile

  // broadcast from lane 0: lets the compiler keep everything derived from the warp index uniform
  const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;

  // a grid launched behind this one with programmatic serialisation (the prefix queries of W, which
  // depend on nothing here) may run beside it
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // Once any CTA has flagged a timeout the rest of the grid (and later launches, until the
  // host reads the status) leave at once instead of each running into the same limit.
  if (threadIdx.x == 0) bar->tmem_base = *reinterpret_cast<volatile int*>(p.status);
  __syncthreads();
  if (bar->tmem_base != 0) return;
  __syncthreads();

  if (threadIdx.x == 0) {
    for (int b = 0; b < 2; ++b) {
      mbar_init(&bar->q_full[b], 1);
      mbar_init(&bar->q_empty[b], 2);     // one commit from each MMA issuer warp
    }
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bar->k_full[s], 1);
      mbar_init(&bar->k_empty[s], 2);
      mbar_init(&bar->v_full[s], 1);
      mbar_init(&bar->v_empty[s], 2);
    }
    for (int t = 0; t < 2; ++t) {
      for (int b = 0; b < 2; ++b) {
        mbar_init(&bar->s_full[t][b], 1);
        mbar_init(&bar->p_full[t][b], 128);
      }
      mbar_init(&bar->pv_done[t], 1);
      mbar_init(&bar->o_full[t], 1);
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

  // Warps 0, 1 and 2 run their loops with all 32 lanes (waits included) so that counters,
  // addresses and descriptors stay warp-uniform; only the TMA / tcgen05 instructions themselves
  // are issued by one elected lane (always the same one: the election is deterministic for a
  // full warp, and tcgen05.commit has to come from the thread that issued the MMAs).
  if (warp == 0) {
    // ================= TMA producer =================
    bool ok = true;
    int n = 0;                 // items seen (non-empty ones): Q buffer n & 1
    int s = 0;                 // ring stage of the next key tile
    uint32_t par = 1;          // parity of the "empty" phase this pass over the ring waits for
    int issued_v = 0;          // for the abort path: V copies issued so far
    for (int i = item0; i < p.total_items && ok; i += item_step) {
      const Item it = decode_item(p, i);
      if (it.qt0 >= it.ntiles) continue;
      const int qb = n & 1;
      const int b = fdiv(it.bh, p.div_H), h = it.bh - b * p.H;   // coordinates of the input tensor maps
      ok = warp_wait<kSuspendNs>(&bar->q_empty[qb], ((n >> 1) & 1) ^ 1, &bar->abort_flag, p.status);
      if (!ok) break;
      if (elect_one()) {
        mbar_expect_tx(&bar->q_full[qb], 2 * kTileBytes);
        for (int t = 0; t < 2; ++t)
          tma_load_5d(sQ + (2 * qb + t) * kTileBytes, &mapQ, &bar->q_full[qb], 0, it.x0 + (it.qt0 + t) * p.step_x,
                      it.y0 + (it.qt0 + t) * p.step_y, h, b);
      }
      __syncwarp();
      for (int j = 0; j < it.nkt; ++j) {
        const bool pre = j == it.ntiles;               // the tile of prefix keys
        ok = warp_wait<kSuspendNs>(&bar->k_empty[s], par, &bar->abort_flag, p.status);
        if (!ok) break;
        if (elect_one()) {
          mbar_expect_tx(&bar->k_full[s], kTileBytes);
          if (pre) tma_load_4d(sK + s * kTileBytes, &mapKp, &bar->k_full[s], 0, 0, 0, it.bh);
          else tma_load_5d(sK + s * kTileBytes, &mapK, &bar->k_full[s], 0, it.x0 + j * p.step_x, it.y0 + j * p.step_y, h, b);
        }
        __syncwarp();
        ok = warp_wait<kSuspendNs>(&bar->v_empty[s], par, &bar->abort_flag, p.status);
        if (!ok) break;
        if (elect_one()) {
          mbar_expect_tx(&bar->v_full[s], kTileBytes);
          if (pre) tma_load_4d(sV + s * kTileBytes, &mapVp, &bar->v_full[s], 0, 0, 0, it.bh);
          else tma_load_5d(sV + s * kTileBytes, &mapV, &bar->v_full[s], 0, it.x0 + j * p.step_x, it.y0 + j * p.step_y, h, b);
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
    // ================= MMA issuers: warp 1 serves query tile 0, warp 2 query tile 1 =================
    // Per query tile t the work is a stream of 64-key steps (key tile G of the CTA's whole run,
    // half h), running on through item boundaries:
    //   S(t, G, h) = Q_t K^T  into score buffer h     (4 MMAs, M128 N64 K16, operands in smem)
    //   O_t      += P(t, G, h) V                       (4 MMAs, M128 N64 K16, A = P in tensor memory)
    // With two score buffers per query tile, the scores of tile G + 1 (half h) are issued as soon
    // as P(t, G, h) has been published (its buffer is free then), so the softmax of the step in
    // between never waits for the tensor pipe.  Each stream is a chain of wait -> issue ->
    // commit latencies, so the two streams run in warps of their own.
    // The commit that publishes scores follows the issue of the preceding P V: seeing the
    // scores of step u + 2 tells the softmax warps that P V (u) has read its probabilities, and
    // seeing those of step u + 1 that P V (u - 1) has retired and O is quiescent (pv_done does
    // that at the very end of the run, where no further scores are issued).
    const int t = warp - 1;
    auto next_item = [&](int i) {           // next non-empty item after index i, or -1
      for (i += item_step; i < p.total_items; i += item_step) {
        const Item it = decode_item(p, i);
        if (it.qt0 < it.ntiles) return i;
      }
      return -1;
    };
    int cur = item0 - item_step;
    cur = next_item(cur);
    bool ok = cur >= 0;
    int n = 0;                              // items seen: Q buffer n & 1, parity (n >> 1) & 1
    int s = 0, s1 = 0;                      // ring stage of the P V key tile and of the score key tile
    uint32_t ph = 0, ph1 = 0;               // and their "full" parities
    uint32_t g_par = 0;                     // parity of the global key-tile index of the P V tile

    // scores of half h of local tile jq of the item in Q buffer qb (n_q-th item), key ring stage s1
    auto issue_qk = [&](int h, int jq, int ntiles_q, int n_q) -> bool {
      const int qb = n_q & 1;
      if (h == 0) {
        if (jq == 0 && !warp_wait<kSuspendNs>(&bar->q_full[qb], (n_q >> 1) & 1, &bar->abort_flag, p.status)) return false;
        if (!warp_wait<kSuspendNs>(&bar->k_full[s1], ph1, &bar->abort_flag, p.status)) return false;
        tc_fence_after();
      }
      const uint32_t kb = sK + s1 * kTileBytes + h * (kSub * kD * 2), qa = sQ + (2 * qb + t) * kTileBytes;
      if (elect_one()) {                     // one lane issues the four MMAs back to back
        const uint64_t dq = smem_desc(qa), dk = smem_desc(kb);
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks)
          mma_ss_1(tmem + kColS + (2 * t + h) * kSub, desc_advance(dq, ks * 32), desc_advance(dk, ks * 32), kIdescQK, ks > 0);
      }
      __syncwarp();
      tc_commit(&bar->s_full[t][h]);
      if (h == 1) {
        tc_commit(&bar->k_empty[s1]);
        if (jq == ntiles_q - 1) tc_commit(&bar->q_empty[qb]);
        if (++s1 == kStages) { s1 = 0; ph1 ^= 1; }
      }
      return true;
    };

    Item it{};
    if (ok) {
      it = decode_item(p, cur);
      ok = issue_qk(0, 0, it.nkt, 0) && issue_qk(1, 0, it.nkt, 0);
    }
    while (ok) {
      const int nxt = next_item(cur);
      Item itn{};
      if (nxt >= 0) itn = decode_item(p, nxt);
      for (int j = 0; j < it.nkt && ok; ++j) {
        ok = warp_wait<kSuspendNs>(&bar->v_full[s], ph, &bar->abort_flag, p.status);
        const bool last = j + 1 == it.nkt;
        for (int h = 0; h < 2 && ok; ++h) {
          ok = warp_wait<kSuspendNs>(&bar->p_full[t][h], g_par, &bar->abort_flag, p.status);
          if (!ok) break;
          tc_fence_after();
          const uint32_t vb = sV + s * kTileBytes + h * (kSub * kD * 2);
          if (elect_one()) {                 // one lane issues the four MMAs back to back
            const uint64_t dv = smem_desc(vb);
#pragma unroll
            for (int ks = 0; ks < kSub / 16; ++ks)
              mma_ts_1(tmem + kColO + t * kD, tmem + kColP + (2 * t + h) * (kSub / 2) + ks * 8, desc_advance(dv, ks * 2048),
                       kIdescPV, (j > 0 || h > 0 || ks > 0) ? 1u : 0u);
          }
          __syncwarp();
          if (last && h == 1) tc_commit(&bar->o_full[t]);
          if (!last) ok = issue_qk(h, j + 1, it.nkt, n);                 // its commit also covers the P V just issued
          else if (nxt >= 0) ok = issue_qk(h, 0, itn.nkt, n + 1);        // first key tile of the next item
          else tc_commit(&bar->pv_done[t]);
        }
        if (ok) tc_commit(&bar->v_empty[s]);
        if (++s == kStages) { s = 0; ph ^= 1; }
        g_par ^= 1;
      }
      if (nxt < 0) break;
      cur = nxt;
      it = itn;
      ++n;
    }
    // Teardown: every MMA issued so far must have retired before tensor memory is released.
    tc_commit(&bar->drain);
    if (lane == 0) {
      const unsigned long long t0 = globaltimer();
      while (!mbar_try(&bar->drain, 0) && globaltimer() - t0 < kWaitLimitNs) {}
    }
    __syncwarp();
  } else if (warp >= 4) {
    // ================= softmax + epilogue: one thread per query row =================
    const int t = (warp - 4) >> 2;                 // query tile of this warpgroup
    const int row = ((warp & 3) << 5) + lane;      // row of the tile == tensor-memory lane
    const uint32_t lane_base = (uint32_t)((warp & 3) << 5) << 16;
    const uint32_t tS = tmem + lane_base + kColS + 2 * t * kSub;          // + h * kSub
    const uint32_t tO = tmem + lane_base + kColO + t * kD;
    const uint32_t tP = tmem + lane_base + kColP + 2 * t * (kSub / 2);    // + h * kSub / 2
    const float sl2 = p.scale_log2;
    const float kLazy = 8.f / sl2;                 // the reference maximum moves only when it grew by > 2^8
    float m = -INFINITY, l = 0.f;
    bool ok = true;

    const uint64_t sl2x2 = pack2(sl2, sl2);
    const int lg_bw = 31 - __clz(p.box_w);          // box_w is a power of two

    // o_scale: factor the accumulator O has to be multiplied by before this step's P V is added.
    float o_scale = 1.f;
    unsigned rescale_vote = 0;        // warp-uniform: some lane has o_scale != 1

    // One 64-key step in two passes over this thread's row: maximum first, then exponentials.
    auto two_pass = [&](uint32_t tSb, uint32_t tPb) {
      uint32_t va[32], vb[32];
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      tmem_ld32(tSb, va);
      tmem_wait_ld(va);
      tmem_ld32(tSb + 32, vb);
      max32(va, mx4);
      tmem_wait_ld(vb);
      max32(vb, mx4);
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      if (mx > m + kLazy) {          // always true on the first step (m = -inf, mx finite)
        const float alpha = ex2((m - mx) * sl2);   // first step: exp2(-inf) = 0
        l *= alpha;
        o_scale *= alpha;
        m = mx;
      }
      const float mneg = -m * sl2;
      const uint64_t mnegx2 = pack2(mneg, mneg);
      uint64_t lsum[4] = {0ull, 0ull, 0ull, 0ull};
      uint32_t pk[16];
      exp32<false, kPolyOf8>(va, sl2x2, mnegx2, lsum, pk, mx4);
      tmem_st16(tPb, pk);
      exp32<false, kPolyOf8>(vb, sl2x2, mnegx2, lsum, pk, mx4);
      tmem_st16(tPb + 16, pk);
      float a0, a1, b0, b1;
      unpack2(add2(lsum[0], lsum[1]), a0, a1);
      unpack2(add2(lsum[2], lsum[3]), b0, b1);
      l += (a0 + a1) + (b0 + b1);
    };

    // Later steps, one pass: the exponentials are taken against the maximum known so far while
    // the step's own maximum is tracked on the side.  Any reference value gives the same
    // softmax as long as nothing overflows, so a larger maximum only matters for the steps
    // that follow: it becomes the reference of the next step, which rescales l and O.
    // A step whose scores exceed the reference by more than 2^kSpecLimit is redone with the
    // two-pass routine (P has not been published yet).
    constexpr float kSpecLimit = 64.f;
    float pend_alpha = 1.f, pend_m = 0.f;
    bool pending = false;
    bool next_ready = false;          // answer of the early test of the next step's score barrier
    auto one_pass = [&](uint32_t tSb, uint32_t tPb, uint64_t* next_bar, uint32_t next_parity) -> bool {
      uint32_t va[32], vb[32];
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      const float mneg = -m * sl2;
      const uint64_t mnegx2 = pack2(mneg, mneg);
      uint64_t lsum[4] = {0ull, 0ull, 0ull, 0ull};
      uint32_t pk[16];
      tmem_ld32(tSb, va);
      tmem_wait_ld(va);
      tmem_ld32(tSb + 32, vb);
      exp32<true, kPolyOf8>(va, sl2x2, mnegx2, lsum, pk, mx4);
      tmem_st16(tPb, pk);
      next_ready = mbar_test(next_bar, next_parity);   // round trip hidden behind the second half
      tmem_wait_ld(vb);
      exp32<true, kPolyOf8>(vb, sl2x2, mnegx2, lsum, pk, mx4);
      tmem_st16(tPb + 16, pk);
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      float a0, a1, b0, b1;
      unpack2(add2(lsum[0], lsum[1]), a0, a1);
      unpack2(add2(lsum[2], lsum[3]), b0, b1);
      const float grow = (mx - m) * sl2;              // log2 of the largest p of this step
      // one vote for both rare cases: bit 1 = redo this step, bit 0 = some O needs rescaling
      const unsigned flags = __reduce_or_sync(0xffffffffu, (grow > kSpecLimit ? 2u : 0u) | (o_scale != 1.f ? 1u : 0u));
      if (flags & 2u) return false;                    // redo (whole warp); l untouched
      l += (a0 + a1) + (b0 + b1);
      if (grow > 8.f) {                                // new reference from the next step on
        pending = true;
        pend_alpha = ex2(-grow);
        pend_m = mx;
      }
      rescale_vote = flags & 1u;
      return true;
    };

    int n = 0;                        // items seen: parity of o_full
    uint32_t g_par = 0;               // parity of the global key-tile index (phase of s_full / p_full)
    auto next_item = [&](int i) {     // next non-empty item after index i, or -1
      for (i += item_step; i < p.total_items; i += item_step) {
        const Item itx = decode_item(p, i);
        if (itx.qt0 < itx.ntiles) return i;
      }
      return -1;
    };

    // ---- epilogue of an item, in two parts around the publication of the next item's first P ----
    // Part 1 reads O (which the next item's first P V will overwrite) and scales it by 1 / l;
    // part 2 writes the bf16 tile to global memory: through a swizzled staging tile and one TMA
    // store when the tile's box, clipped to the grid, lies inside the window (the store clips at
    // the grid edge by itself), row by row otherwise.
    struct Done {
      bool have, store;
      int bh, qx0, qy0, x_end, y_end, par;
      float inv;
    } done{};
    done.have = false;
    const uint32_t sOt = sO + t * kTileBytes;
    unsigned char* sOt_ptr = smem + (size_t)(4 + 2 * kStages + t) * kTileBytes;
    auto epi_load = [&](uint32_t (&ob)[32]) -> bool {
      if (!__all_sync(0xffffffffu, mbar_wait<kSuspendNs>(&bar->o_full[t], done.par, &bar->abort_flag, p.status))) return false;
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t v[32];
        tmem_ld32(tO + 32 * c, v);
        tmem_wait_ld(v);
#pragma unroll
        for (int i = 0; i < 16; ++i)
          ob[16 * c + i] = pack_bf16(__uint_as_float(v[2 * i]) * done.inv, __uint_as_float(v[2 * i + 1]) * done.inv);
      }
      return true;
    };
    // Each warp writes its own quarter of the tile (32 rows = a sub-box of the tile's box): no
    // synchronisation beyond the warp.  One TMA store when the sub-box, clipped to the grid, holds
    // tokens of this window only (the store clips at the grid edge by itself); row by row otherwise.
    const int q4 = warp & 3;
    int sub_x, sub_y;                                   // origin of this warp's sub-box inside the tile's box
    if (p.box_h >= 4) { sub_x = 0; sub_y = q4 * (p.box_h >> 2); }
    else { sub_x = (32 * q4) & (p.box_w - 1); sub_y = (32 * q4) >> lg_bw; }
    const int sub_w = p.box_h >= 4 ? p.box_w : 32, sub_h = p.box_h >= 4 ? (p.box_h >> 2) : 1;
    auto epi_store = [&](const uint32_t (&ob)[32]) -> bool {
      if (!done.store) return true;
      const int wx0 = done.qx0 + sub_x, wy0 = done.qy0 + sub_y;
      if (wx0 >= done.x_end || wy0 >= done.y_end) return true;       // none of this warp's rows exists
      const bool tma = p.step_x != 0 || ((wx0 + sub_w <= done.x_end || done.x_end == p.gridW) &&
                                         (wy0 + sub_h <= done.y_end || done.y_end == p.gridH));
      if (tma) {
        // this warp's previous store must have finished reading its staging quarter
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncwarp();
#pragma unroll
        for (int c = 0; c < 8; ++c)     // 16-byte chunk c of this row, at its 128-byte-swizzle position
          *reinterpret_cast<uint4*>(sOt_ptr + row * 128 + ((c ^ (row & 7)) << 4)) =
              make_uint4(ob[4 * c], ob[4 * c + 1], ob[4 * c + 2], ob[4 * c + 3]);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                       ::"l"(&mapO), "r"(sOt + q4 * 4096), "r"(0), "r"(wx0), "r"(wy0), "r"(done.bh) : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      } else {
        const int qx = done.qx0 + row % p.box_w, qy = done.qy0 + row / p.box_w;
        if (qx < done.x_end && qy < done.y_end) {
          __nv_bfloat16* dst = p.o + ((size_t)done.bh * p.tokens_per_head + (size_t)qy * p.gridW + qx) * kD;
#pragma unroll
          for (int c = 0; c < 8; ++c)
            *reinterpret_cast<uint4*>(dst + 8 * c) = make_uint4(ob[4 * c], ob[4 * c + 1], ob[4 * c + 2], ob[4 * c + 3]);
        }
      }
      return true;
    };

    int cur = next_item(item0 - item_step);
    if (cur >= 0) next_ready = mbar_test(&bar->s_full[t][0], 0);
    while (cur >= 0 && ok) {
      const Item it = decode_item(p, cur);
      const int nxt = next_item(cur);
      const int ntiles = it.ntiles, nsteps = 2 * it.nkt;
      const int x0 = it.x0, y0 = it.y0, x_end = it.x_end, y_end = it.y_end;
      // Which key tiles have keys that do not exist?  A window narrower than the box makes every
      // tile an edge tile; otherwise only the last tile of the window / sequence can be one.
      const bool edge_all = (x_end - x0) < p.box_w && p.step_x == 0;
      const int last_vx = x_end - (x0 + (ntiles - 1) * p.step_x), last_vy = y_end - (y0 + (ntiles - 1) * p.step_y);
      const bool edge_last = last_vx < p.box_w || last_vy < p.box_h;
      m = -INFINITY;
      l = 0.f;
      pending = false;
      // one 64-key step up to (not including) the publication of its P; first_tag: first step of the item
      auto compute_step = [&](auto first_tag, int u) -> bool {
        constexpr bool kFirst = decltype(first_tag)::value;
        const int j = u >> 1, h = u & 1;
        // warp-uniform outcome: the tensor-memory accesses below are warp-collective
        if (!__all_sync(0xffffffffu, next_ready)) {
          ok = __all_sync(0xffffffffu, mbar_wait<kSuspendNs>(&bar->s_full[t][h], g_par, &bar->abort_flag, p.status));
          if (!ok) return false;
        }
        tc_fence_after();
        const uint32_t tSb = tS + h * kSub, tPb = tP + h * (kSub / 2);
        o_scale = 1.f;
        if (pending) {                 // the previous step raised the maximum: new reference from here on
          l *= pend_alpha;
          o_scale = pend_alpha;
          m = pend_m;
          pending = false;
        }
        const bool pre = j == ntiles;                  // (only with prefix tokens: nsteps covers one more tile)
        if (pre || edge_all || (edge_last && j == ntiles - 1)) {
          // Edge tile: overwrite the scores of keys that do not exist (outside the grid or the
          // window; in the tile of prefix keys, past the P-th) with -inf in tensor memory, then
          // treat the step like any other.
          // vx, vy: valid extent of the key tile's box along x and y
          const int vx = x_end - (x0 + j * p.step_x), vy = y_end - (y0 + j * p.step_y);
#pragma unroll 1
          for (int c = 0; c < 2; ++c) {
            const int k0 = 64 * h + 32 * c;            // first of the 32 keys, as an index into the box
            uint32_t bits = 0;
            if (pre) {                                 // box position r holds prefix token r
              const int nv = p.P - k0;
              if (nv > 0) bits = nv >= 32 ? 0xffffffffu : ((1u << nv) - 1u);
            } else if (p.box_w >= 32) {                // the 32 keys lie in one box row
              const int ly = k0 >> lg_bw, lx0 = k0 & (p.box_w - 1);
              const int nv = min(32, vx - lx0);
              if (ly < vy && nv > 0) bits = nv >= 32 ? 0xffffffffu : ((1u << nv) - 1u);
            } else {                                   // 32 / box_w whole box rows
              const uint32_t rowbits = (1u << min(vx, p.box_w)) - 1u;
              const int ly0 = k0 >> lg_bw;
              for (int r = 0; r < (32 >> lg_bw); ++r)
                if (ly0 + r < vy) bits |= rowbits << (r << lg_bw);
            }
            if (bits != 0xffffffffu) {                 // warp-uniform: the mask depends on the tile only
              uint32_t v[32];
              tmem_ld32(tSb + 32 * c, v);
              tmem_wait_ld(v);
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (!((bits >> i) & 1u)) v[i] = kNegInf;   // exp2(-inf) = 0 and -inf never wins the maximum
              tmem_st32(tSb + 32 * c, v);
            }
          }
          tmem_wait_st();
        }
        // the step after this one (possibly the first of the next item): its score barrier
        const bool has_next = u + 1 < nsteps || nxt >= 0;
        uint64_t* next_bar = &bar->s_full[t][h ^ 1];
        const uint32_t next_parity = g_par ^ (uint32_t)h;      // same key tile after h = 0, the next one after h = 1
        if (kFirst || !one_pass(tSb, tPb, next_bar, next_parity)) {
          two_pass(tSb, tPb);
          next_ready = false;
          rescale_vote = __any_sync(0xffffffffu, o_scale != 1.f);
        }
        if (!has_next) next_ready = false;
        if (!kFirst && rescale_vote) {
          // O may be touched once P V of step u - 1 has retired; the next P V waits for our P.
          // The issuer commits the scores of step u + 1 after issuing P V (u - 1), so that barrier
          // tells us; after the last step of the run there are no further scores, and pv_done
          // (committed after each P V of the run's last key tile) does.
          if (has_next)
            ok = __all_sync(0xffffffffu, mbar_wait<kSuspendNs>(next_bar, next_parity, &bar->abort_flag, p.status));
          else
            ok = __all_sync(0xffffffffu, mbar_wait<kSuspendNs>(&bar->pv_done[t], 0, &bar->abort_flag, p.status));
          if (!ok) return false;
          tc_fence_after();
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            uint32_t v[32];
            tmem_ld32(tO + 32 * c, v);
            tmem_wait_ld(v);
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * o_scale);
            tmem_st32(tO + 32 * c, v);
          }
        }
        return true;
      };
      auto publish = [&](int h) {
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bar->p_full[t][h]);
        g_par ^= (uint32_t)h;
      };
      // First step.  The previous item's O has to be read before this item's first P is published
      // (its P V overwrites O); by now that item's last P V has long retired.
      ok = compute_step(std::true_type{}, 0);
      if (!ok) break;
      if (done.have) {
        uint32_t ob[32];
        ok = epi_load(ob);
        if (!ok) break;
        publish(0);
        ok = epi_store(ob);
        done.have = false;
      } else {
        publish(0);
      }
      for (int u = 1; u < nsteps && ok; ++u) {
        ok = compute_step(std::false_type{}, u);
        if (ok) publish(u & 1);
      }
      if (!ok) break;
      // what the deferred epilogue of this item needs
      done.have = true;
      done.store = it.qt0 + t < ntiles;
      done.bh = it.bh;
      done.qx0 = x0 + (it.qt0 + t) * p.step_x;
      done.qy0 = y0 + (it.qt0 + t) * p.step_y;
      done.x_end = x_end;
      done.y_end = y_end;
      done.par = n & 1;
      done.inv = 1.f / l;
      cur = nxt;
      ++n;
    }
    if (ok && done.have) {            // the run's last item
      uint32_t ob[32];
      if (epi_load(ob)) ok = epi_store(ob);
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
  if (ww > kTile || (ww & (ww - 1)) != 0) return false;   // box width must divide 128
  const int bh = kTile / ww;
  const int wh = a.wh < a.Hg ? a.wh : a.Hg;
  *g = Geometry{a.Wg, a.Hg, ww, wh, ww, bh, 0, bh, ceil_div(a.Wg, ww), ceil_div(a.Hg, wh), ceil_div(wh, bh)};
  return true;
}

}  // namespace

bool attn_tc_supported(const AttnArgs& a, bool full) {
  if (a.dtype != JV_BF16 || a.D != kD) return false;
  Geometry g;
  if (!geometry(a, full, &g)) return false;
  if (a.P > kTile) return false;                        // the prefix keys are one key tile
  if ((int64_t)g.nwx * g.nwy * ceil_div(g.tiles_per_window, 2) * a.BH > 0x7fffffffll) return false;
  // 128-byte rows keep every TMA stride a multiple of 16 bytes; the base must be 16-byte aligned (checked by the ABI)
  return encode_fn() != nullptr;
}

cudaError_t launch_attn_tc(const AttnArgs& a, bool full, int* status, cudaStream_t st) {
  Geometry g;
  if (!geometry(a, full, &g)) return cudaErrorInvalidValue;
  EncodeFn enc = encode_fn();
  if (!enc) return cudaErrorNotSupported;
  const int N = a.P + a.Hg * a.Wg;                     // tokens per (batch, head): prefix tokens, then the grid
  CUtensorMap maps[6];
  // the grid tokens start behind the prefix rows
  const size_t grid0 = (size_t)a.P * kD * 2, igrid0 = (size_t)a.P * (size_t)a.in.tok * 2;
  const void* ptrs[4] = {(const char*)a.q + igrid0, (const char*)a.k + igrid0, (const char*)a.v + igrid0, (char*)a.o + grid0};
  const cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)g.gridW, (cuuint64_t)g.gridH, (cuuint64_t)a.BH};
  const cuuint64_t strides[3] = {(cuuint64_t)kD * 2, (cuuint64_t)g.gridW * kD * 2, (cuuint64_t)N * kD * 2};
  const cuuint32_t box[4] = {(cuuint32_t)kD, (cuuint32_t)g.box_w, (cuuint32_t)g.box_h, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  // the output is stored per warp: a quarter of the tile's box (32 tokens)
  const cuuint32_t qbox[4] = {(cuuint32_t)kD, (cuuint32_t)(g.box_h >= 4 ? g.box_w : 32),
                              (cuuint32_t)(g.box_h >= 4 ? g.box_h / 4 : 1), 1};
  // the inputs as (d, x, y, head, batch) with the caller's strides; the output as (d, x, y, batch*head)
  const cuuint64_t idims[5] = {(cuuint64_t)kD, (cuuint64_t)g.gridW, (cuuint64_t)g.gridH, (cuuint64_t)a.H, (cuuint64_t)(a.BH / a.H)};
  const cuuint64_t istrides[4] = {(cuuint64_t)a.in.tok * 2, (cuuint64_t)g.gridW * a.in.tok * 2, (cuuint64_t)a.in.head * 2,
                                  (cuuint64_t)a.in.batch * 2};
  const cuuint32_t ibox[5] = {(cuuint32_t)kD, (cuuint32_t)g.box_w, (cuuint32_t)g.box_h, 1, 1};
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
  // The prefix rows of K and V in the shape of a key box: prefix token r at box position
  // (r % box_w, r / box_w).  Positions past P inside the last box row read grid tokens (they exist:
  // a grid holds at least one box row of tokens) and are masked by the softmax; rows past that are
  // outside the map and arrive as zeros.
  // (prefix tokens come with contiguous inputs only: the caller has checked)
  maps[4] = maps[1];
  maps[5] = maps[2];
  if (a.P > 0) {
    const cuuint64_t pdims[4] = {(cuuint64_t)kD, (cuuint64_t)g.box_w, (cuuint64_t)ceil_div(a.P, g.box_w), (cuuint64_t)a.BH};
    const cuuint64_t pstrides[3] = {(cuuint64_t)kD * 2, (cuuint64_t)g.box_w * kD * 2, (cuuint64_t)N * kD * 2};
    const void* pptrs[2] = {a.k, a.v};
    for (int i = 0; i < 2; ++i) {
      CUresult r = enc(&maps[4 + i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(pptrs[i]), pdims, pstrides, box,
                       estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
  }
  static OncePerDevice smem_opt_in;   // > 48 KB of dynamic shared memory: a per-device function attribute
  cudaError_t e = smem_opt_in.run([] {
    return cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  });
  if (e != cudaSuccess) return e;
  TcParams p;
  p.o = (__nv_bfloat16*)a.o + (size_t)a.P * kD;        // first grid token of (batch, head) 0
  p.status = status;
  p.gridW = g.gridW;
  p.gridH = g.gridH;
  p.tokens_per_head = N;
  p.win_w = g.win_w;
  p.win_h = g.win_h;
  p.box_w = g.box_w;
  p.box_h = g.box_h;
  p.step_x = g.step_x;
  p.step_y = g.step_y;
  p.nwx = g.nwx;
  p.nwin = g.nwx * g.nwy;
  p.qpairs = ceil_div(g.tiles_per_window, 2);
  p.total_items = p.qpairs * p.nwin * a.BH;
  p.P = a.P;
  p.lg_box_h = 0;
  while ((1 << p.lg_box_h) < g.box_h) ++p.lg_box_h;
  p.div_qpairs = make_fastdiv((uint32_t)p.qpairs);
  p.div_nwin = make_fastdiv((uint32_t)p.nwin);
  p.div_nwx = make_fastdiv((uint32_t)p.nwx);
  p.H = a.H;
  p.div_H = make_fastdiv((uint32_t)a.H);
  p.scale_log2 = a.scale * 1.4426950408889634f;
  // persistent: one CTA per SM (shared memory and the 512 tensor-memory columns allow no more)
  const int num_sms = device_sm_count();
  const int grid = p.total_items < num_sms ? p.total_items : num_sms;
  attn_tc_kernel<<<grid, kThreads, kSmemBytes, st>>>(maps[0], maps[1], maps[2], maps[3], maps[4], maps[5], p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace jv
