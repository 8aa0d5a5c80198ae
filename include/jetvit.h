/*
 * jetvit.h -- C ABI of libjetvit: the token mixers of a JetViT hybrid Vision
 * Transformer as CUDA kernels for NVIDIA B200 (sm_100a).
 *
 * Three mixers and a schedule driver (JetViT, Sec. 3.2):
 *   L  linear-attention block: ReLU-kernel linear attention (Eq. 2) with the row
 *      normalisation, plus the optional squeeze dynamic depth-wise convolution
 *      on V (Sec. 3.2.1, Eq. 4);
 *   W  2D window attention over non-overlapping windows (Sec. 3.2.2);
 *   F  full softmax attention (Eq. 1);
 *   S  a per-layer L/W/F schedule over a stack of independent layers
 *      (Sec. 3.2.3, Fig. 1b).
 *
 * Conventions shared by every call
 *   Tensors   q, k, v, o are DEVICE pointers to [B, H, N, D] contiguous arrays,
 *             D fastest, N = P + Hg * Wg: P prefix tokens (jv_shape.P, usually 0), then
 *             grid token t at grid position (t / Wg, t % Wg).
 *             All four have the element type jv_shape.dtype; o must not share a
 *             byte with an input.  Pointers must be 16-byte aligned.
 *   Ownership The caller owns every buffer and the stream.  The library never
 *             allocates or frees device memory; scratch comes from the caller
 *             through (ws, ws_bytes), sized by jv_workspace_bytes(), 256-byte
 *             aligned.  ws may be NULL when jv_workspace_bytes() returns 0.
 *   Stream    cuda_stream is a cudaStream_t passed as void* (NULL = default
 *             stream).  Calls only enqueue work and return; results are valid
 *             once the caller has synchronised the stream.  Calls that share a
 *             workspace must be ordered on one stream.
 *   Errors    Return codes only.  Every argument error is found on the host
 *             before anything is launched.  There is no CPU fallback: without a
 *             usable sm_100 device the calls return JV_ERR_CUDA/JV_ERR_UNSUPPORTED.
 *             Kernels bound every wait (2 s); one that gives up sets a sticky
 *             per-device status word and returns, and jv_device_status()
 *             reports JV_ERR_TIMEOUT.  While the word is set, the tensor-core
 *             kernels (bf16, D = 64) that are launched leave at once WITHOUT
 *             writing their output: calls keep returning JV_OK (they only
 *             enqueue) and o keeps its old contents until jv_device_status()
 *             has been called, which reads and clears the word.  A caller that
 *             must know that its results are valid calls jv_device_status()
 *             after the work it cares about.  With the environment variable
 *             JETVIT_DEBUG set, a call that returns JV_ERR_CUDA also prints
 *             the CUDA error string to stderr.
 *   Precision bf16 tensors: bf16 tensor-core products with fp32 accumulation,
 *             fp32 softmax / state, round-to-nearest-even output.  f32 tensors:
 *             fp32 arithmetic throughout (no tf32).
 */
#ifndef JETVIT_H_
#define JETVIT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  JV_OK = 0,
  JV_ERR_INVALID_ARG = 1,  /* null / misaligned pointer, non-positive size, bad schedule character */
  JV_ERR_UNSUPPORTED = 2,  /* shape or dtype outside what the kernels cover (e.g. D > 128) */
  JV_ERR_WORKSPACE = 3,    /* ws is NULL, misaligned or smaller than jv_workspace_bytes() */
  JV_ERR_CUDA = 4,         /* a CUDA runtime / driver call failed */
  JV_ERR_TIMEOUT = 5       /* a kernel gave up on a bounded wait */
} jv_status;

typedef enum { JV_F32 = 0, JV_BF16 = 1 } jv_dtype;

/*
 * Problem shape.  A (batch, head) holds P prefix tokens followed by the Hg * Wg grid tokens:
 * N = P + Hg * Wg rows of D elements.  P = 0 is the plain feature map.
 *
 * Prefix tokens are the class / register tokens that the base models of the paper (Sec. 4.1)
 * carry in front of their patch tokens.  The paper defines its window partition (Sec. 3.2.2) and
 * the convolution on V (Sec. 3.2.1, Eq. 4) on the feature map and does not mention them; the
 * rule implemented here: F (Eq. 1) and the linear attention proper (Eq. 2) are global over all N
 * tokens; in W a grid token attends its window and the P prefix tokens, a prefix token attends
 * all N tokens; the convolution and the pooling that feeds its kernel generator see the grid only
 * (a prefix token's L output is its linear-attention output alone).
 *
 * in_layout describes q, k and v only (o is always [B, H, N, D] contiguous).  With JV_LAYOUT_BNHD
 * they are [B, N, H, D] arrays whose token rows (H * D elements each, heads side by side) are
 * in_tok_stride elements apart: H * D for a contiguous array (0 selects that), 3 * H * D for the
 * three slices of a fused [B, N, 3, H, D] activation, the form in which a model's QKV projection
 * leaves them (the blocks take their inputs from the inherited projections, Sec. 3.2.4).  Batch
 * element b starts N * in_tok_stride elements after b - 1.  The layout is served by the tensor-core
 * paths only: bf16, D = 64, P = 0 where a convolution is asked for, 3 x 3 pooled or static kernels;
 * everything else returns JV_ERR_UNSUPPORTED.  in_tok_stride * element size must be a multiple of 16.
 */
typedef enum { JV_LAYOUT_BHND = 0, JV_LAYOUT_BNHD = 1 } jv_layout;

typedef struct {
  int32_t B, H, Hg, Wg, D;
  int32_t dtype;         /* jv_dtype */
  int32_t P;             /* prefix tokens in front of the grid tokens, >= 0 */
  int32_t in_layout;     /* jv_layout of q, k, v; 0 = [B, H, N, D] contiguous like o */
  int64_t in_tok_stride; /* JV_LAYOUT_BNHD: elements between token rows; 0 = H * D */
} jv_shape;

/*
 * Kernel generator of the squeeze dynamic depth-wise convolution (Sec. 3.2.1):
 * a two-layer MLP with SiLU fed by the average-pooled V.  All pointers are
 * DEVICE pointers to fp32, row-major; C = H * D, channel c = h * D + e.
 *
 * R = 0 selects the static depth-wise convolution the paper compares against
 * (Sec. 3.2.1, Table 1 "DWC"): no generator, b2 holds the kernels themselves
 * ([C, k, k], shared by every sample and required); W1, b1 and W2 are ignored
 * and may be NULL.
 *
 * token_wise = 1 selects the token-wise dynamic convolution the paper tries first and sets
 * aside for its cost (Sec. 3.2.1, Table 1 "+ Token-wise Dynamic DWC"): the same generator
 * (R > 0) is fed with every grid token's own value vector instead of the pooled one and
 * gives that token its own kernels, which are applied to the token's neighbourhood:
 *   w_i = W2 SiLU(W1 v_i + b1) + b2,   o_i += sum_taps w_i[c][dy][dx] V[(y+dy-p, x+dx-p)][c].
 * The kernels of all tokens pass through the caller's scratch: jv_workspace_bytes() grows by
 * about 2 * B * N * C * k * k bytes.
 */
typedef struct {
  int32_t k;       /* odd kernel edge: 3 or 5 */
  int32_t R;       /* hidden width of the generator, 1..1024; 0 = static kernels in b2 */
  const float* W1; /* [R, C] */
  const float* b1; /* [R] or NULL */
  const float* W2; /* [C*k*k, R] */
  const float* b2; /* [C*k*k] or NULL */
  int32_t token_wise; /* 0: one set of kernels per sample from the pooled V; 1: one set per token */
} jv_dwc;

/*
 * Bytes of scratch the given mixer needs for this shape.  mixer is 'L', 'W', 'F',
 * 'S' (the maximum over the three, for jv_hybrid_mixers) or 'f' (jv_linear_attn_focused).  dwc may be NULL;
 * pass the descriptor that the L call will get, since it enlarges the scratch.
 * Returns 0 on invalid arguments as well as when no scratch is needed.
 */
size_t jv_workspace_bytes(char mixer, const jv_shape* shape, const jv_dwc* dwc);

/*
 * L -- JetViT linear-attention block (Sec. 3.2.1; Eq. 2 reordered, Eq. 4).
 *   KV = sum_j relu(k_j)^T v_j,  z = sum_j relu(k_j)          per (batch, head)
 *   o_i = relu(q_i) KV / (relu(q_i) . z + eps)
 *   and, when dwc != NULL:  s = mean_j v_j (per sample and channel),
 *   w = W2 SiLU(W1 s + b1) + b2 viewed as [C, k, k],
 *   o_i += depth-wise k x k convolution of V (as an Hg x Wg image, zero padding
 *   (k-1)/2, stride 1) with the sample's kernels w.
 * eps is added to the denominator only (1e-6 in the paper's setting; must be >= 0).
 * Phase 1 reduces the state over token chunks into ws; a second pass sums the
 * chunk partials in a fixed order (no floating-point atomics: results are
 * bit-reproducible); phase 2 streams q -> o.
 */
jv_status jv_linear_attn(const void* q, const void* k, const void* v, void* o, const jv_shape* shape,
                         float eps, const jv_dwc* dwc, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * L with the focused feature map in place of ReLU (Eq. 3; the variant "+ DWC on V + Focusing
 * Factor" of Table 1, which the paper measures and sets aside for its cost):
 *   phi_p(x) = (||r|| / ||r^p||) r^p,  r = relu(x),  r^p element-wise over the D features of a token,
 * (the denominator read as in the work Eq. 3 cites: the norm of the element-wise power), then
 * exactly jv_linear_attn with phi_p(q), phi_p(k) in place of relu(q), relu(k).  focus_p in (0, 16];
 * focus_p = 1 is jv_linear_attn.  phi_p(q) and phi_p(k) are formed by one extra streaming pass
 * and kept in the caller's scratch: ws must cover jv_workspace_bytes('f', shape, dwc).
 */
jv_status jv_linear_attn_focused(const void* q, const void* k, const void* v, void* o, const jv_shape* shape,
                                 float eps, float focus_p, const jv_dwc* dwc, void* ws, size_t ws_bytes,
                                 void* cuda_stream);

/*
 * L without caller scratch.  (The paper has no counterpart: this entry point exists for
 * integration, not for the method.)
 *
 * Some callers cannot allocate device memory at the point where they run a mixer: a
 * serving engine whose own pool already owns the whole GPU, a real-time loop that must
 * not hit the device-wide synchronisation of cudaMalloc / cudaFree, a plug-in interface
 * that offers a stream and nothing else.  jv_linear_attn_static computes exactly what
 * jv_linear_attn computes (same kernels, bit-identical output) but takes its scratch from
 * a fixed array of JV_STATIC_SCRATCH_BYTES that is part of the library image; the caller
 * passes only inputs and outputs.  The call allocates nothing and frees nothing.
 *
 *   Limit     jv_workspace_bytes('L', shape, dwc) must not exceed JV_STATIC_SCRATCH_BYTES
 *             (16 MiB).  The scratch grows with B * H (one or more 16.5 KiB partial
 *             states per (batch, head): about 6 MiB for B=8, H=16 on a 64x64 grid, 5 MiB
 *             for B=1, H=16 on a 128x128 grid), not with the token count, plus
 *             B * H * D * k * k * 4 bytes of kernels with the convolution; roughly
 *             B * H <= 480 fits.  Larger problems are refused with JV_ERR_WORKSPACE
 *             before anything is launched; use jv_linear_attn with your own buffer
 *             for those.
 *   Cost      every GPU on which the library is loaded carries the 16 MiB array until the
 *             process exits, whether or not this function is ever called.
 *   Set-up    the first call on each device looks up the array's device address (that
 *             device must be current, as for every call).  Make that first call during
 *             initialisation, before any stream capture begins.
 *   Sharing   there is one array per device and every call uses it.  It keeps whatever
 *             the previous call left; nothing in it needs clearing, because every value
 *             a call consumes is written earlier in that same call.  Two calls that may overlap on the
 *             GPU (different streams, no ordering between them) race on the array and
 *             corrupt each other: order them on one stream or with events.
 * Other arguments and return codes are those of jv_linear_attn.
 */
#define JV_STATIC_SCRATCH_BYTES (16u << 20)
jv_status jv_linear_attn_static(const void* q, const void* k, const void* v, void* o, const jv_shape* shape,
                                float eps, const jv_dwc* dwc, void* cuda_stream);

/*
 * W -- window attention (Sec. 3.2.2): the grid is cut into non-overlapping
 * win_h x win_w windows anchored at (0, 0); softmax attention (Eq. 1) runs
 * inside each window.  When the grid is not a multiple of the window the
 * right / bottom windows hold only the tokens that exist (their missing keys are
 * masked out, their missing query rows are never written).  A window at least as
 * large as the grid is full attention.  scale <= 0 selects 1/sqrt(D).
 */
jv_status jv_window_attn(const void* q, const void* k, const void* v, void* o, const jv_shape* shape,
                         int32_t win_h, int32_t win_w, float scale, void* ws, size_t ws_bytes,
                         void* cuda_stream);

/*
 * F -- full softmax attention (Eq. 1): o = softmax(q k^T * scale) v over all N
 * tokens of each (batch, head), non-causal, computed flash-style with an fp32
 * online softmax.  scale <= 0 selects 1/sqrt(D).
 */
jv_status jv_full_attn(const void* q, const void* k, const void* v, void* o, const jv_shape* shape,
                       float scale, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * S -- hybrid stack (Sec. 3.2.3): for l in [0, n_layers) run mixer schedule[l]
 * ('L', 'W' or 'F') on layer l's tensors.  q, k, v, o are HOST arrays of n_layers
 * DEVICE pointers; all layers share one shape.  dwc is NULL or a HOST array of
 * n_layers entries (each NULL or a host pointer to a jv_dwc) used by the L layers.
 * Layers are independent; they are enqueued in order on one stream with no host
 * synchronisation in between.  ws must cover jv_workspace_bytes('S', ...).
 * The schedule is validated completely before the first launch.
 */
jv_status jv_hybrid_mixers(int32_t n_layers, const char* schedule, const void* const* q,
                           const void* const* k, const void* const* v, void* const* o,
                           const jv_shape* shape, int32_t win_h, int32_t win_w, float scale, float eps,
                           const jv_dwc* const* dwc, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * The projections either side of a mixer (the W_Q, W_K, W_V and W_O that a searched model
 * inherits from its base model for every block, Sec. 3.2.4), as tensor-core GEMMs that write
 * and read the mixers' [B, H, N, D] layout directly: no transpose pass between projection
 * and mixer.  bf16 only, D = 64 only (JV_ERR_UNSUPPORTED otherwise); C = H * D.
 *
 * (N = P + Hg * Wg tokens; a projection does not care which of them are prefix tokens.)
 * jv_qkv_proj:  x [B, N, C] (token-major activations), w [3C, C] row-major (output feature
 *   by input feature, the rows ordered q | k | v and, inside each, head-major: row
 *   which*C + h*D + e), bias fp32 [3C] or NULL.
 *     q[b, h, n, e] = sum_c x[b, n, c] * w[0*C + h*D + e, c] + bias[0*C + h*D + e]
 *   and likewise k (which = 1) and v (which = 2).
 * jv_out_proj:  o [B, H, N, D] (a mixer's output), w [C, C] row-major, bias fp32 [C] or NULL.
 *     y[b, n, f] = sum_{h, e} o[b, h, n, e] * w[f, h*D + e] + bias[f]          y: [B, N, C]
 *
 * Products in bf16 on the tensor cores with fp32 accumulation; the bias is added in fp32
 * and the result rounded to bf16 once (round to nearest even).  All pointers are DEVICE
 * pointers, 16-byte aligned; outputs must not alias inputs.  No scratch.  Errors as for the
 * mixers: argument errors are found on the host before anything is launched.
 */
jv_status jv_qkv_proj(const void* x, const void* w, const float* bias, void* q, void* k, void* v,
                      const jv_shape* shape, void* cuda_stream);
jv_status jv_out_proj(const void* o, const void* w, const float* bias, void* y, const jv_shape* shape,
                      void* cuda_stream);

/*
 * Synchronises the stream, then returns and clears the sticky device status:
 * JV_OK, JV_ERR_TIMEOUT if a kernel abandoned a bounded wait since the last
 * call, or JV_ERR_CUDA if the stream reports a CUDA error.
 */
jv_status jv_device_status(void* cuda_stream);

/*
 * Self-test of the bounded waits (for test suites; the paper has no counterpart).  Enqueues a
 * one-warp kernel that waits, through the same bounded wait the mixers use, on a barrier
 * that nothing ever completes; after limit_us microseconds (1 .. 1000000) the wait gives up,
 * sets the sticky status word exactly as a mixer kernel would, and the kernel returns.
 * Nothing faults or hangs and the context stays usable.  gave_up is NULL or a DEVICE pointer
 * to an int that receives 1 if the wait ran out.  Afterwards jv_device_status() returns
 * JV_ERR_TIMEOUT once, then JV_OK.
 */
jv_status jv_selftest_wait_timeout(uint32_t limit_us, int32_t* gave_up, void* cuda_stream);

/*
 * Tuning / dispatch switch, mainly for tests: 0 (default) lets every call pick
 * its fastest kernel for the shape; 1 forces the shape-generic fp32-arithmetic
 * kernels for every call.  Returns the previous value.  Process-wide.
 */
int32_t jv_set_force_generic(int32_t on);

/*
 * Number of kernel launches the library has enqueued since it was loaded
 * (process-wide counter; used to report launches per benchmark step).
 */
uint64_t jv_launch_count(void);

const char* jv_status_string(jv_status s);
const char* jv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* JETVIT_H_ */
