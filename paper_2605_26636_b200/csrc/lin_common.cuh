// Pieces shared by the bf16 kernels of the linear-attention block (linear_fast.cu,
// linear_conv.cu): layout constants of the state, small bf16 helpers, the 128-byte-swizzle
// address function, programmatic-launch controls and the tensor-map builders.
// Internal; every function is inline.
#pragma once

#include "tc_common.cuh"

namespace jv {
namespace lin {

constexpr int kD = 64;
// Partial state per (batch, head, chunk), in floats: [0, 4096) KV[a][e], [4096, 4160) z[a],
// [4160, 4224) vsum[e]
constexpr int kOffZ = kD * kD, kOffVsum = kD * kD + kD;

__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ uint32_t relu_bf16x2(uint32_t x) {
  __nv_bfloat162 v = *reinterpret_cast<__nv_bfloat162*>(&x);
  v = __hmax2(v, __float2bfloat162_rn(0.f));
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float2 bf16x2_to_f2(uint32_t x) {
  return make_float2(__uint_as_float(x << 16), __uint_as_float(x & 0xffff0000u));
}

// Byte offset of 16-byte chunk `ch` (0..7) of row `row` in a [rows][64 bf16] tile in the
// 128-byte-swizzle layout (what TMA writes): chunks are XORed with the row index mod 8, so
// ldmatrix reads of 8 rows hit 8 distinct bank groups.
__device__ __forceinline__ uint32_t tile_off(int row, int ch) { return (uint32_t)(row * 128 + ((ch ^ (row & 7)) << 4)); }

// L2 eviction-priority hints for TMA loads: a tensor that a later kernel of the same call
// reads again is kept (evict_last), one that is read exactly once makes room first (evict_first).
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_load_3d_hint(uint32_t dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1,
                                                 int c2, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], [%2], %6;"
      ::"r"(dst), "l"(map), "r"(tc::smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_load_4d_hint(uint32_t dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1,
                                                 int c2, int c3, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
      ::"r"(dst), "l"(map), "r"(tc::smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy) : "memory");
}

__device__ __forceinline__ void tma_load_5d_hint(uint32_t dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1,
                                                 int c2, int c3, int c4, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6, %7}], [%2], %8;"
      ::"r"(dst), "l"(map), "r"(tc::smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "l"(policy) : "memory");
}

// ---- host side: tensor maps ---------------------------------------------------------------
// The first N tokens of every (batch, head) of a [BH, ntok, 64] bf16 tensor as (channel, token,
// batch*head); boxes of box_tok tokens, 128-byte swizzle; tokens past N arrive as zeros.
inline bool make_map_tokens(CUtensorMap* m, const void* ptr, int BH, int N, int box_tok, int ntok) {
  tc::EncodeFn enc = tc::encode_fn();
  if (!enc) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)N, (cuuint64_t)BH};
  const cuuint64_t strides[2] = {(cuuint64_t)kD * 2, (cuuint64_t)ntok * kD * 2};
  const cuuint32_t box[3] = {(cuuint32_t)kD, (cuuint32_t)box_tok, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// An input tensor (q, k or v) with the caller's strides: the first N tokens of every (batch, head)
// as (channel, token, head, batch); boxes of box_tok tokens, 128-byte swizzle; tokens past N arrive as zeros.
inline bool make_map_tokens_in(CUtensorMap* m, const void* ptr, int B, int H, int N, int box_tok, const InStrides& in) {
  tc::EncodeFn enc = tc::encode_fn();
  if (!enc) return false;
  const cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)N, (cuuint64_t)H, (cuuint64_t)B};
  const cuuint64_t strides[3] = {(cuuint64_t)in.tok * 2, (cuuint64_t)in.head * 2, (cuuint64_t)in.batch * 2};
  const cuuint32_t box[4] = {(cuuint32_t)kD, (cuuint32_t)box_tok, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The Hg x Wg grid tokens (behind P prefix tokens) of an input tensor with the caller's strides as a 5-D
// tensor (channel, x, y, head, batch); boxes of box_x x box_y tokens; positions outside the grid arrive as zeros.
inline bool make_map_grid_in(CUtensorMap* m, const void* ptr, int B, int H, int P, int Hg, int Wg, int box_x, int box_y,
                             bool swizzle128, const InStrides& in) {
  tc::EncodeFn enc = tc::encode_fn();
  if (!enc) return false;
  ptr = (const char*)ptr + (size_t)P * (size_t)in.tok * 2;   // token strides are multiples of 16 bytes
  const cuuint64_t dims[5] = {(cuuint64_t)kD, (cuuint64_t)Wg, (cuuint64_t)Hg, (cuuint64_t)H, (cuuint64_t)B};
  const cuuint64_t strides[4] = {(cuuint64_t)in.tok * 2, (cuuint64_t)Wg * in.tok * 2, (cuuint64_t)in.head * 2,
                                 (cuuint64_t)in.batch * 2};
  const cuuint32_t box[5] = {(cuuint32_t)kD, (cuuint32_t)box_x, (cuuint32_t)box_y, 1, 1};
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(ptr), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The Hg x Wg grid tokens of a [BH, P + Hg*Wg, 64] bf16 tensor (P prefix tokens in front of the
// grid of every (batch, head)) as a 4-D tensor (channel, x, y, batch*head); boxes of box_x x box_y
// tokens; positions outside the grid arrive as zeros on a load and are dropped by a store.
inline bool make_map_grid(CUtensorMap* m, const void* ptr, int BH, int P, int Hg, int Wg, int box_x, int box_y, bool swizzle128) {
  tc::EncodeFn enc = tc::encode_fn();
  if (!enc) return false;
  ptr = (const char*)ptr + (size_t)P * kD * 2;       // rows are 128 bytes: the base stays 16-byte aligned
  const cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)Wg, (cuuint64_t)Hg, (cuuint64_t)BH};
  const cuuint64_t strides[3] = {(cuuint64_t)kD * 2, (cuuint64_t)Wg * kD * 2, (cuuint64_t)(P + Hg * Wg) * kD * 2};
  const cuuint32_t box[4] = {(cuuint32_t)kD, (cuuint32_t)box_x, (cuuint32_t)box_y, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace lin
}  // namespace jv
