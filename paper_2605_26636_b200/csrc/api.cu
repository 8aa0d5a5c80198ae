// C ABI of libjetvit: argument validation, dispatch, device status.
// Every argument error is reported before anything is launched.
#include <atomic>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "common.cuh"

namespace jv {
namespace {

__device__ int g_status_word = 0;          // sticky error bits written by kernels
std::atomic<uint64_t> g_launches{0};
std::atomic<int32_t> g_force_generic{0};

bool aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

// [a, a + na) and [b, b + nb) share at least one byte
bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
  const uintptr_t x = (uintptr_t)a, y = (uintptr_t)b;
  return x < y + nb && y < x + na;
}

size_t tensor_bytes(const jv_shape* s) {
  return (size_t)s->B * s->H * shape_tokens(*s) * s->D * (s->dtype == JV_F32 ? 4 : 2);
}

jv_status check_shape(const jv_shape* s) {
  if (!s) return JV_ERR_INVALID_ARG;
  if (s->B <= 0 || s->H <= 0 || s->Hg <= 0 || s->Wg <= 0 || s->D <= 0 || s->P < 0) return JV_ERR_INVALID_ARG;
  if (s->dtype != JV_F32 && s->dtype != JV_BF16) return JV_ERR_INVALID_ARG;
  if ((int64_t)s->Hg * s->Wg + s->P > (1 << 24)) return JV_ERR_UNSUPPORTED;
  if ((int64_t)s->B * s->H > 65535) return JV_ERR_UNSUPPORTED;
  if (s->D > 128) return JV_ERR_UNSUPPORTED;
  // rows must keep 16-byte alignment for the vector loads
  const int esz = s->dtype == JV_F32 ? 4 : 2;
  if ((s->D * esz) % 16 != 0) return JV_ERR_UNSUPPORTED;
  if (s->in_layout != JV_LAYOUT_BHND && s->in_layout != JV_LAYOUT_BNHD) return JV_ERR_INVALID_ARG;
  if (s->in_layout == JV_LAYOUT_BNHD) {
    const int64_t row = (int64_t)s->H * s->D;
    if (s->in_tok_stride != 0 && s->in_tok_stride < row) return JV_ERR_INVALID_ARG;   // token rows would overlap
    if ((s->in_tok_stride * esz) % 16 != 0) return JV_ERR_INVALID_ARG;
    if (s->in_tok_stride > ((int64_t)1 << 31)) return JV_ERR_UNSUPPORTED;
  } else if (s->in_tok_stride != 0) {
    return JV_ERR_INVALID_ARG;
  }
  return JV_OK;
}

// bytes from the first to one past the last element of an input tensor (q, k or v)
size_t input_bytes(const jv_shape* s) {
  if (!in_strided(*s)) return tensor_bytes(s);
  const InStrides in = in_strides(*s);
  const size_t esz = s->dtype == JV_F32 ? 4 : 2;
  return (size_t)((int64_t)(s->B - 1) * in.batch + (int64_t)(shape_tokens(*s) - 1) * in.tok + (int64_t)s->H * s->D) * esz;
}

jv_status check_tensors(const void* q, const void* k, const void* v, const void* o, const jv_shape* s) {
  if (!q || !k || !v || !o) return JV_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(o, 16)) return JV_ERR_INVALID_ARG;
  const size_t n = tensor_bytes(s), ni = input_bytes(s);      // o may not share a byte with an input
  if (overlaps(o, n, q, ni) || overlaps(o, n, k, ni) || overlaps(o, n, v, ni)) return JV_ERR_INVALID_ARG;
  return JV_OK;
}

jv_status check_dwc(const jv_dwc* d) {
  if (!d) return JV_OK;
  if (d->k != 3 && d->k != 5) return JV_ERR_INVALID_ARG;
  if (d->R < 0 || d->R > 1024) return JV_ERR_INVALID_ARG;
  if (d->token_wise != 0 && d->token_wise != 1) return JV_ERR_INVALID_ARG;
  if (d->token_wise && d->R == 0) return JV_ERR_INVALID_ARG;  // per-token kernels need the generator
  if (d->R == 0) return d->b2 ? JV_OK : JV_ERR_INVALID_ARG;   // static kernels live in b2
  if (!d->W1 || !d->W2) return JV_ERR_INVALID_ARG;
  return JV_OK;
}

jv_status check_ws(const void* ws, size_t ws_bytes, size_t need) {
  if (need == 0) return JV_OK;
  if (!ws || !aligned(ws, 256) || ws_bytes < need) return JV_ERR_WORKSPACE;
  return JV_OK;
}

jv_status check_window(const jv_shape* s, int wh, int ww) {
  if (wh <= 0 || ww <= 0) return JV_ERR_INVALID_ARG;
  const int64_t nwin = (int64_t)ceil_div(s->Hg, wh < s->Hg ? wh : s->Hg) * ceil_div(s->Wg, ww < s->Wg ? ww : s->Wg);
  if (nwin > 65535) return JV_ERR_UNSUPPORTED;
  return JV_OK;
}

jv_status check_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return JV_ERR_CUDA; }
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
    cudaGetLastError();
    return JV_ERR_CUDA;
  }
  return major == 10 ? JV_OK : JV_ERR_UNSUPPORTED;
}

// ptrs[0 .. nin) are inputs, ptrs[nin .. nptr) outputs; bytes[i] is the extent of ptrs[i]
jv_status check_proj(const jv_shape* s, const void* const* ptrs, const size_t* bytes, int nptr, int nin) {
  jv_status st = check_shape(s);
  if (st != JV_OK) return st;
  for (int i = 0; i < nptr; ++i)
    if (!ptrs[i] || !aligned(ptrs[i], 16)) return JV_ERR_INVALID_ARG;
  if (s->dtype != JV_BF16 || s->D != 64) return JV_ERR_UNSUPPORTED;   // (the extents below assume both)
  if (in_strided(*s)) return JV_ERR_UNSUPPORTED;                        // the projections have layouts of their own
  for (int i = nin; i < nptr; ++i)           // outputs overlap neither an input nor each other
    for (int j = 0; j < i; ++j)
      if (overlaps(ptrs[i], bytes[i], ptrs[j], bytes[j])) return JV_ERR_INVALID_ARG;
  return JV_OK;
}

jv_status from_cuda(cudaError_t e) {
  if (e == cudaSuccess) return JV_OK;
  if (getenv("JETVIT_DEBUG")) fprintf(stderr, "libjetvit: CUDA error %d (%s)\n", (int)e, cudaGetErrorString(e));
  return JV_ERR_CUDA;
}

float pick_scale(float scale, int D) { return scale > 0.f ? scale : 1.f / sqrtf((float)D); }

// ---- enqueue helpers (arguments already validated) ---------------------------
jv_status run_attn(const void* q, const void* k, const void* v, void* o, const jv_shape* s, int wh, int ww,
                   float scale, bool full, cudaStream_t st) {
  AttnArgs a{q, k, v, o, s->B * s->H, s->Hg, s->Wg, s->D, s->H, in_strides(*s), in_strided(*s),
             s->P, wh, ww, pick_scale(scale, s->D), s->dtype};
  const bool one_window = full || (wh >= s->Hg && ww >= s->Wg);
  if (one_window) {      // every token attends all P + N tokens: where a token sits does not matter
    a.Hg = 1;
    a.Wg = shape_tokens(*s);
    a.P = 0;
    a.wh = a.Hg;
    a.ww = a.Wg;
  }
  if (!g_force_generic.load() && one_window && attn_f4_supported(a)) {
    int* status = device_status_ptr();
    if (!status) return JV_ERR_CUDA;
    return from_cuda(launch_attn_f4(a, status, st));
  }
  if (!g_force_generic.load() && attn_d128_supported(a, full)) {
    int* status = device_status_ptr();
    if (!status) return JV_ERR_CUDA;
    return from_cuda(launch_attn_d128(a, full, status, st));
  }
  if (!g_force_generic.load() && !one_window && attn_w4_supported(a)) {
    int* status = device_status_ptr();
    if (!status) return JV_ERR_CUDA;
    const jv_status r = from_cuda(launch_attn_w4(a, status, st));
    if (r != JV_OK || a.P == 0) return r;
    return from_cuda(launch_attn_generic(a, st, true));   // the P prefix queries, which attend everything
  }
  if (!g_force_generic.load() && attn_tc_supported(a, full)) {
    int* status = device_status_ptr();
    if (!status) return JV_ERR_CUDA;
    if (a.strided && a.P > 0) return JV_ERR_UNSUPPORTED;  // the prefix queries' kernel reads contiguous tensors
    const jv_status r = from_cuda(launch_attn_tc(a, full, status, st));
    if (r != JV_OK || a.P == 0) return r;
    return from_cuda(launch_attn_generic(a, st, true));   // the P prefix queries, which attend everything
  }
  if (a.strided) return JV_ERR_UNSUPPORTED;               // the generic kernels read contiguous tensors
  return from_cuda(launch_attn_generic(a, st));
}

jv_status run_linear(const void* q, const void* k, const void* v, void* o, const jv_shape* s, float eps,
                     const jv_dwc* dwc, void* ws, cudaStream_t st) {
  LinArgs a{q, k, v, o, *s, eps, dwc, ws};
  if (!dwc && s->P > 0) {   // without the convolution the block is global: where a token sits does not matter
    a.s.Hg = 1;
    a.s.Wg = shape_tokens(*s);
    a.s.P = 0;
  }
  const LinPlan p = lin_plan(*s, dwc);
  if (!g_force_generic.load() && linear_fast_supported(a)) return from_cuda(launch_linear_fast(a, p, st));
  if (in_strided(*s)) return JV_ERR_UNSUPPORTED;          // the generic kernels read contiguous tensors
  return from_cuda(launch_linear_generic(a, p, st));
}

}  // namespace

int* device_status_ptr() {
  // One address per device; looked up once per device and cached.
  static int* cache[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (!cache[dev]) {
    int* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_status_word) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    cache[dev] = p;
  }
  return cache[dev];
}

void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return -1; }
  return dev;
}

int device_sm_count() {
  static std::atomic<int> cache[kMaxDevices] = {};
  const int dev = current_device();
  if (dev < 0 || dev >= kMaxDevices) return kDefaultSmCount;
  int n = cache[dev].load(std::memory_order_relaxed);
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
    cudaGetLastError();
    return kDefaultSmCount;
  }
  cache[dev].store(n, std::memory_order_relaxed);
  return n;
}

}  // namespace jv

using namespace jv;

extern "C" {

size_t jv_workspace_bytes(char mixer, const jv_shape* shape, const jv_dwc* dwc) {
  if (check_shape(shape) != JV_OK || check_dwc(dwc) != JV_OK) return 0;
  switch (mixer) {
    case 'L':
    case 'S':
      return lin_plan(*shape, dwc).total;   // W and F need no scratch
    case 'f':   // the linear block with the focused feature map: two tensors for phi(q), phi(k) behind the block's own scratch
      return align_up(lin_plan(*shape, dwc).total, 256) + 2 * align_up(tensor_bytes(shape), 256);
    case 'W':
    case 'F':
      return 0;
    default:
      return 0;
  }
}

jv_status jv_linear_attn(const void* q, const void* k, const void* v, void* o, const jv_shape* shape, float eps,
                         const jv_dwc* dwc, void* ws, size_t ws_bytes, void* cuda_stream) {
  jv_status st = check_shape(shape);
  if (st != JV_OK) return st;
  if ((st = check_tensors(q, k, v, o, shape)) != JV_OK) return st;
  if (!(eps >= 0.f)) return JV_ERR_INVALID_ARG;
  if ((st = check_dwc(dwc)) != JV_OK) return st;
  if ((st = check_ws(ws, ws_bytes, lin_plan(*shape, dwc).total)) != JV_OK) return st;
  if ((st = check_device()) != JV_OK) return st;
  return run_linear(q, k, v, o, shape, eps, dwc, ws, (cudaStream_t)cuda_stream);
}

jv_status jv_linear_attn_focused(const void* q, const void* k, const void* v, void* o, const jv_shape* shape, float eps,
                                 float focus_p, const jv_dwc* dwc, void* ws, size_t ws_bytes, void* cuda_stream) {
  jv_status st = check_shape(shape);
  if (st != JV_OK) return st;
  if ((st = check_tensors(q, k, v, o, shape)) != JV_OK) return st;
  if (!(eps >= 0.f) || !(focus_p > 0.f) || !(focus_p <= 16.f)) return JV_ERR_INVALID_ARG;
  if ((st = check_dwc(dwc)) != JV_OK) return st;
  if (in_strided(*shape)) return JV_ERR_UNSUPPORTED;      // the feature-map pass reads contiguous q and k
  const size_t lin = align_up(lin_plan(*shape, dwc).total, 256), tb = align_up(tensor_bytes(shape), 256);
  if ((st = check_ws(ws, ws_bytes, lin + 2 * tb)) != JV_OK) return st;
  if ((st = check_device()) != JV_OK) return st;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  void* qf = (char*)ws + lin;
  void* kf = (char*)ws + lin + tb;
  if ((st = from_cuda(launch_focus_map(q, k, qf, kf, *shape, focus_p, stream))) != JV_OK) return st;
  return run_linear(qf, kf, v, o, shape, eps, dwc, ws, stream);
}

jv_status jv_window_attn(const void* q, const void* k, const void* v, void* o, const jv_shape* shape,
                         int32_t win_h, int32_t win_w, float scale, void* ws, size_t ws_bytes,
                         void* cuda_stream) {
  (void)ws; (void)ws_bytes;
  jv_status st = check_shape(shape);
  if (st != JV_OK) return st;
  if ((st = check_tensors(q, k, v, o, shape)) != JV_OK) return st;
  if ((st = check_window(shape, win_h, win_w)) != JV_OK) return st;
  if ((st = check_device()) != JV_OK) return st;
  return run_attn(q, k, v, o, shape, win_h, win_w, scale, false, (cudaStream_t)cuda_stream);
}

jv_status jv_full_attn(const void* q, const void* k, const void* v, void* o, const jv_shape* shape, float scale,
                       void* ws, size_t ws_bytes, void* cuda_stream) {
  (void)ws; (void)ws_bytes;
  jv_status st = check_shape(shape);
  if (st != JV_OK) return st;
  if ((st = check_tensors(q, k, v, o, shape)) != JV_OK) return st;
  if ((st = check_device()) != JV_OK) return st;
  return run_attn(q, k, v, o, shape, shape->Hg, shape->Wg, scale, true, (cudaStream_t)cuda_stream);
}

jv_status jv_hybrid_mixers(int32_t n_layers, const char* schedule, const void* const* q, const void* const* k,
                           const void* const* v, void* const* o, const jv_shape* shape, int32_t win_h,
                           int32_t win_w, float scale, float eps, const jv_dwc* const* dwc, void* ws,
                           size_t ws_bytes, void* cuda_stream) {
  if (n_layers <= 0 || !schedule || !q || !k || !v || !o) return JV_ERR_INVALID_ARG;
  jv_status st = check_shape(shape);
  if (st != JV_OK) return st;
  if (!(eps >= 0.f)) return JV_ERR_INVALID_ARG;
  size_t need = 0;
  bool any_w = false;
  for (int l = 0; l < n_layers; ++l) {
    const char m = schedule[l];
    if (m != 'L' && m != 'W' && m != 'F') return JV_ERR_INVALID_ARG;   // also catches an early '\0'
    if ((st = check_tensors(q[l], k[l], v[l], o[l], shape)) != JV_OK) return st;
    if (m == 'W') any_w = true;
    if (m == 'L') {
      const jv_dwc* d = dwc ? dwc[l] : nullptr;
      if ((st = check_dwc(d)) != JV_OK) return st;
      const size_t n = lin_plan(*shape, d).total;
      if (n > need) need = n;
    }
  }
  if (any_w && (st = check_window(shape, win_h, win_w)) != JV_OK) return st;
  if ((st = check_ws(ws, ws_bytes, need)) != JV_OK) return st;
  if ((st = check_device()) != JV_OK) return st;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  for (int l = 0; l < n_layers; ++l) {
    switch (schedule[l]) {
      case 'L': st = run_linear(q[l], k[l], v[l], o[l], shape, eps, dwc ? dwc[l] : nullptr, ws, stream); break;
      case 'W': st = run_attn(q[l], k[l], v[l], o[l], shape, win_h, win_w, scale, false, stream); break;
      default:  st = run_attn(q[l], k[l], v[l], o[l], shape, shape->Hg, shape->Wg, scale, true, stream); break;
    }
    if (st != JV_OK) return st;
  }
  return JV_OK;
}

jv_status jv_qkv_proj(const void* x, const void* w, const float* bias, void* q, void* k, void* v,
                      const jv_shape* shape, void* cuda_stream) {
  if (!shape) return JV_ERR_INVALID_ARG;
  const void* ptrs[5] = {x, w, q, k, v};
  const size_t C = (size_t)shape->H * shape->D, nt = (size_t)shape->B * shape_tokens(*shape) * C * 2;
  const size_t bytes[5] = {nt, 3 * C * C * 2, nt, nt, nt};
  jv_status st = check_proj(shape, ptrs, bytes, 5, 2);
  if (st != JV_OK) return st;
  if (bias && !aligned(bias, 16)) return JV_ERR_INVALID_ARG;
  if ((st = check_device()) != JV_OK) return st;
  if (!proj_tc_available()) return JV_ERR_CUDA;
  int* status = device_status_ptr();
  if (!status) return JV_ERR_CUDA;
  return from_cuda(launch_proj_tc(true, x, w, bias, q, k, v, *shape, status, (cudaStream_t)cuda_stream));
}

jv_status jv_out_proj(const void* o, const void* w, const float* bias, void* y, const jv_shape* shape,
                      void* cuda_stream) {
  if (!shape) return JV_ERR_INVALID_ARG;
  const void* ptrs[3] = {o, w, y};
  const size_t C = (size_t)shape->H * shape->D, nt = (size_t)shape->B * shape_tokens(*shape) * C * 2;
  const size_t bytes[3] = {nt, C * C * 2, nt};
  jv_status st = check_proj(shape, ptrs, bytes, 3, 2);
  if (st != JV_OK) return st;
  if (bias && !aligned(bias, 16)) return JV_ERR_INVALID_ARG;
  if ((st = check_device()) != JV_OK) return st;
  if (!proj_tc_available()) return JV_ERR_CUDA;
  int* status = device_status_ptr();
  if (!status) return JV_ERR_CUDA;
  return from_cuda(launch_proj_tc(false, o, w, bias, y, nullptr, nullptr, *shape, status, (cudaStream_t)cuda_stream));
}

jv_status jv_device_status(void* cuda_stream) {
  if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) { cudaGetLastError(); return JV_ERR_CUDA; }
  int word = 0;
  if (cudaMemcpyFromSymbol(&word, g_status_word, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return JV_ERR_CUDA; }
  if (word != 0) {
    const int zero = 0;
    cudaMemcpyToSymbol(g_status_word, &zero, sizeof(int));
    return JV_ERR_TIMEOUT;
  }
  return JV_OK;
}

int32_t jv_set_force_generic(int32_t on) { return g_force_generic.exchange(on ? 1 : 0); }

uint64_t jv_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* jv_status_string(jv_status s) {
  switch (s) {
    case JV_OK: return "ok";
    case JV_ERR_INVALID_ARG: return "invalid argument";
    case JV_ERR_UNSUPPORTED: return "unsupported shape, dtype or device";
    case JV_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case JV_ERR_CUDA: return "CUDA call failed";
    case JV_ERR_TIMEOUT: return "a kernel gave up on a bounded wait";
    default: return "unknown status";
  }
}

const char* jv_version(void) { return "jetvit-b200 0.1.0 (sm_100a)"; }

}  // extern "C"
