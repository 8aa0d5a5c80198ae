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
#include <cuda.h>

#include "common.cuh"

namespace jv {
namespace {

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
// Tensor-memory columns: S_t (and P_t over its first 32 columns) at 64 t, O_t at 256 + 64 t
constexpr uint32_t kColS = 0, kColO = 256;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s

// Division by a run-time constant without a divide: q = (umulhi(n, mul) + n) >> shr, exact for
// 0 <= n < 2^31 (mul = floor(2^32 (2^shr - d) / d) + 1, shr = ceil(log2 d)).
struct FastDiv {
  uint32_t mul, shr, d;
};
inline FastDiv make_fastdiv(uint32_t d) {
  uint32_t l = 0;
  while ((1ull << l) < d) ++l;
  return FastDiv{(uint32_t)(((1ull << 32) * ((1ull << l) - d)) / d + 1), l, d};
}
__device__ __forceinline__ int fdiv(int n, const FastDiv& f) { return (int)((__umulhi((uint32_t)n, f.mul) + (uint32_t)n) >> f.shr); }

struct F4Params {
  int* status;
  int N;                 // tokens per (batch, head)
  int ntiles;            // key (and query) tiles per head: ceil(N / 128)
  int qgroups;           // groups of four query tiles per head
  int n_full;            // items [0, n_full) are whole groups, (batch*head, group) with the group fastest;
  int total_items;       // items [n_full, total_items) are half groups (two query tiles), see launch_attn_f4
  FastDiv div_qgroups;
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

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long globaltimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (after flagging the status word and the CTA abort flag)
// if the phase did not complete in time or another role already aborted.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, Barriers* b, int* status) {
  if (mbar_try(bar, parity)) return true;
  unsigned long long t0 = 0;
  for (uint32_t spin = 0;; ++spin) {
    if (mbar_try(bar, parity)) return true;
    if ((spin & 63u) == 63u) {
      if (b->abort_flag) return false;
      const unsigned long long now = globaltimer();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) {
        b->abort_flag = 1;
        atomicOr(status, kStatusTimeout);
        return false;
      }
    }
  }
}

// The same for a whole converged warp, with a warp-uniform outcome.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, Barriers* b, int* status) {
  return __all_sync(0xffffffffu, mbar_wait(bar, parity, b, status));
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

// ---- tcgen05 wrappers -------------------------------------------------------------
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// One lane of a converged warp (the same one every time for a full warp).
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n.reg .pred p;\nelect.sync _|p, 0xffffffff;\nselp.u32 %0, 1, 0, p;\n}\n" : "=r"(pred));
  return pred != 0;
}
// The tcgen05 issue wrappers below are called by a whole converged warp; one elected lane issues.
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  if (elect_one())
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  if (elect_one())
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  if (elect_one())
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// Waits for this thread's outstanding tensor-memory loads.  The registers of the load are
// threaded through the statement so that no use of them can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_wait_ld(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                 "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
                 "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :: "memory");
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// Two fp32 values in one 64-bit register: the packed fp32x2 arithmetic of sm_100.
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// ---- softmax building blocks: 32 scores of one query row at a time -------------------
constexpr uint32_t kNegInf = 0xff800000u;
__device__ __forceinline__ void max32(const uint32_t (&v)[32], float (&mx)[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int u = 0; u < 4; ++u)
      mx[u] = max3(mx[u], __uint_as_float(v[8 * i + 2 * u]), __uint_as_float(v[8 * i + 2 * u + 1]));
}
// exp2 on the FMA pipe, for part of the scores (the MUFU unit, 16 results per clock and SM,
// is the tightest resource of softmax attention at head_dim 64).  x = n + f with n = round(x),
// f in [-0.5, 0.5]; 2^f by a degree-3 minimax polynomial (relative error 7.5e-5, well below
// the bf16 rounding of P); n goes straight into the exponent field.  Valid for x in [-126, 126].
constexpr float kPolyC0 = 0.9999280571937561f, kPolyC1 = 0.6932609677314758f;
constexpr float kPolyC2 = 0.2426111251115799f, kPolyC3 = 0.0551716685295105f;
constexpr float kRoundMagic = 12582912.f;   // 1.5 * 2^23: adding it leaves round(x) in the low mantissa bits
__device__ __forceinline__ void exp2_poly2(uint64_t x, float& p0, float& p1) {
  float x0, x1;
  unpack2(x, x0, x1);
  x = pack2(fmaxf(x0, -126.f), fmaxf(x1, -126.f));
  const uint64_t t = add2(x, pack2(kRoundMagic, kRoundMagic));
  const uint64_t n = add2(t, pack2(-kRoundMagic, -kRoundMagic));
  const uint64_t f = fma2(n, pack2(-1.f, -1.f), x);
  uint64_t q = fma2(f, pack2(kPolyC3, kPolyC3), pack2(kPolyC2, kPolyC2));
  q = fma2(q, f, pack2(kPolyC1, kPolyC1));
  q = fma2(q, f, pack2(kPolyC0, kPolyC0));
  float q0, q1, t0, t1;
  unpack2(q, q0, q1);
  unpack2(t, t0, t1);
  p0 = __uint_as_float(__float_as_uint(q0) + (__float_as_uint(t0) << 23));
  p1 = __uint_as_float(__float_as_uint(q1) + (__float_as_uint(t1) << 23));
}

#ifndef JV_F4_POLY_PAIRS_OF_8
#define JV_F4_POLY_PAIRS_OF_8 1   // of every 8 score pairs, this many take the polynomial path
#endif
// p = exp2(s * sl2 + mneg) for 32 scores; adds them into four packed partial sums and packs
// them to bf16 pairs (even key in the low half).  kTrack also folds the scores into mx.
template <bool kTrack>
__device__ __forceinline__ void exp32(const uint32_t (&v)[32], uint64_t sl2x2, uint64_t mnegx2, uint64_t (&lsum)[4],
                                      uint32_t (&pk)[16], float (&mx)[4]) {
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const float s0 = __uint_as_float(v[2 * i]), s1 = __uint_as_float(v[2 * i + 1]);
    if (kTrack) mx[i & 3] = max3(mx[i & 3], s0, s1);
    const uint64_t x = fma2(pack2(s0, s1), sl2x2, mnegx2);
    float p0, p1;
    if ((i & 7) < JV_F4_POLY_PAIRS_OF_8) {
      exp2_poly2(x, p0, p1);
    } else {
      float x0, x1;
      unpack2(x, x0, x1);
      p0 = ex2(x0);
      p1 = ex2(x1);
    }
    lsum[i & 3] = add2(lsum[i & 3], pack2(p0, p1));
    pk[i] = pack_bf16(p0, p1);
  }
}

// Shared-memory matrix descriptors (128-byte swizzle; 8-row groups 1024 bytes apart).
//   K-major operand  ([rows][64 bf16], used for Q and K): advance 32 bytes per K step of 16.
//   MN-major operand ([keys][64 bf16] used as B = V):      advance 2048 bytes per K step of 16 keys.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | (1ull << 16) /* LBO (unused) */ | (64ull << 32) /* SBO = 1024 B */ |
         (1ull << 46) /* descriptor version */ | (2ull << 61) /* SWIZZLE_128B */;
}
// Instruction descriptor, kind::f16: D fp32, A and B bf16.
constexpr uint32_t idesc(uint32_t M, uint32_t N, uint32_t b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major << 16) | ((N >> 3) << 17) | ((M >> 4) << 24);
}
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
  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
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
      for (int t = 0; t < kQT && ok; ++t) {
        ok = warp_wait(&bar->q_empty[t], (n & 1) ^ 1, bar, p.status);
        if (!ok) break;
        if (tile_exists<kHalves>(it, t, ntiles) && elect_one()) {
          mbar_expect_tx(&bar->q_full[t], kTileBytes);
          tma_load_3d(sQ + t * kTileBytes, &mapQ, &bar->q_full[t], 0, (it.qt0 + t) * kTile, it.bh);
        }
        __syncwarp();
      }
      for (int j = 0; j < ntiles && ok; ++j) {
        ok = warp_wait(&bar->k_empty[s], par, bar, p.status);
        if (!ok) break;
        if (elect_one()) {
          mbar_expect_tx(&bar->k_full[s], kTileBytes);
          tma_load_3d(sK + s * kTileBytes, &mapK, &bar->k_full[s], 0, j * kTile, it.bh);
        }
        __syncwarp();
        ok = warp_wait(&bar->v_empty[s], par, bar, p.status);
        if (!ok) break;
        if (elect_one()) {
          mbar_expect_tx(&bar->v_full[s], kTileBytes);
          tma_load_3d(sV + s * kTileBytes, &mapV, &bar->v_full[s], 0, j * kTile, it.bh);
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
          ok = warp_wait(&bar->k_full[sk], phk, bar, p.status);
          if (!ok) break;
        }
        if (has_pv && ((u - 1) & 1) == 0) { // P V of a first half: its V must have landed
          ok = warp_wait(&bar->v_full[sv], phv, bar, p.status);
          if (!ok) break;
        }
        const uint32_t kb = sK + sk * kTileBytes + (u & 1) * (kSub * kD * 2);
        const uint32_t vb = sV + sv * kTileBytes + ((u - 1) & 1) * (kSub * kD * 2);
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          if (!ex[x]) continue;
          const int t = tb + x;
          if (u == 0) {
            ok = warp_wait(&bar->q_full[t], qcnt[x] & 1, bar, p.status);
            ++qcnt[x];
          } else {
            ok = warp_wait(&bar->p_full[t], pcnt[x] & 1, bar, p.status);
            ++pcnt[x];
          }
          if (!ok) break;
          tc_fence_after();
          if (has_pv) {
#pragma unroll
            for (int ks = 0; ks < kSub / 16; ++ks)
              mma_ts(tmem + kColO + t * kD, tmem + kColS + t * kSub + ks * 8, smem_desc(vb + ks * 2048), kIdescPV,
                     (u > 1 || ks > 0) ? 1u : 0u);
          }
          if (has_qk) {
            const uint32_t qa = sQ + t * kTileBytes;
#pragma unroll
            for (int ks = 0; ks < kD / 16; ++ks)
              mma_ss(tmem + kColS + t * kSub, smem_desc(qa + ks * 32), smem_desc(kb + ks * 32), kIdescQK, ks > 0);
            tc_commit(&bar->s_full[t]);
          } else {
            tc_commit(&bar->o_full[t]);
          }
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
        ok = warp_wait(&bar->s_full[t], scnt & 1, bar, p.status);
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
        exp32<false>(va, sl2x2, mnegx2, lsum, pk, mx4);
        tmem_st16(tS, pk);
        tmem_ld32(tS + 32, va);
        tmem_wait_ld(va);
        exp32<false>(va, sl2x2, mnegx2, lsum, pk, mx4);
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
      ok = warp_wait(&bar->o_full[t], ocnt & 1, bar, p.status);
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
          asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
                       ::"l"(&mapO), "r"(sOt), "r"(0), "r"(tok), "r"(it.bh) : "memory");
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
typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn() {
  static EncodeFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = (EncodeFn)ptr;
  }
  return fn;
}

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
  const cuuint32_t box[3] = {(cuuint32_t)kD, (cuuint32_t)kTile, 1};
  const cuuint32_t qbox[3] = {(cuuint32_t)kD, 32, 1};          // the output is stored per warp: 32 tokens
  const cuuint32_t estr[3] = {1, 1, 1};
  for (int i = 0; i < 4; ++i) {
    CUresult r = enc(&maps[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptrs[i]), dims, strides,
                     i == 3 ? qbox : box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(attn_f4_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(attn_f4_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  static int num_sms = 0;
  if (num_sms == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || num_sms <= 0) {
      num_sms = 0;
      cudaGetLastError();
      return cudaErrorUnknown;
    }
  }
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
  p.scale_log2 = a.scale * 1.4426950408889634f;
  const int grid = p.total_items < num_sms ? p.total_items : num_sms;
  if (split) attn_f4_kernel<true><<<grid, kThreads, kSmemBytes, st>>>(maps[0], maps[1], maps[2], maps[3], p);
  else attn_f4_kernel<false><<<grid, kThreads, kSmemBytes, st>>>(maps[0], maps[1], maps[2], maps[3], p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace jv
