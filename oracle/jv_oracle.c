/*
 * jv_oracle.c -- float64 CPU oracle for the three JetViT token mixers.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * mixers compute; the parity tests, the smoke check and the CPU-baseline leg of
 * the benchmark are its only callers.  It shares no code, header, table or
 * helper with the CUDA library and the CUDA library never calls it.
 *
 * Everything is double precision, every loop is the definition written out:
 * no tiling, no fusion, no reordering beyond the one the paper itself states
 * (Eq. 2: phi(Q) (phi(K)^T V) instead of (phi(Q) phi(K)^T) V).
 * OpenMP only spreads independent (batch, head) units over the host cores.
 *
 * Layout of q, k, v, o: [B*H][N][D] contiguous, D fastest; token t of an
 * Hg x Wg grid is (y, x) = (t / Wg, t % Wg).
 *
 * Pins (tests/test_oracle_pins.py): brute-force N x N forms, closed forms,
 * library routines (float64 SDPA, float64 depth-wise conv2d), hand-computed
 * fixtures under tests/golden/.  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int jvo_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/*
 * Full softmax attention, Eq. 1 with the row normalisation of softmax:
 *   s_ij = (q_i . k_j) * scale,  m_i = max_j s_ij,  p_ij = exp(s_ij - m_i),
 *   O_i  = sum_j p_ij v_j / sum_j p_ij.
 * Non-causal.  Nq query rows attend Nk key rows (Nq == Nk for self-attention;
 * Nq < Nk lets a test evaluate a sample of the query rows of a large problem,
 * rows being independent of one another).
 * q: [BH][Nq][D], k, v: [BH][Nk][D], o: [BH][Nq][D].
 */
void jvo_full_attn(const double* q, const double* k, const double* v, double* o,
                   int64_t BH, int64_t Nq, int64_t Nk, int64_t D, double scale) {
#pragma omp parallel
  {
    double* s = (double*)malloc(sizeof(double) * (size_t)Nk);
#pragma omp for collapse(2) schedule(dynamic, 16)
    for (int64_t g = 0; g < BH; ++g) {
      for (int64_t i = 0; i < Nq; ++i) {
        const double* qi = q + (g * Nq + i) * D;
        const double* kg = k + g * Nk * D;
        const double* vg = v + g * Nk * D;
        double* oi = o + (g * Nq + i) * D;
        double m = -INFINITY;
        for (int64_t j = 0; j < Nk; ++j) {
          double dot = 0.0;
          for (int64_t e = 0; e < D; ++e) dot += qi[e] * kg[j * D + e];
          s[j] = dot * scale;
          if (s[j] > m) m = s[j];
        }
        double denom = 0.0;
        for (int64_t e = 0; e < D; ++e) oi[e] = 0.0;
        for (int64_t j = 0; j < Nk; ++j) {
          double p = exp(s[j] - m);
          denom += p;
          for (int64_t e = 0; e < D; ++e) oi[e] += p * vg[j * D + e];
        }
        for (int64_t e = 0; e < D; ++e) oi[e] /= denom;
      }
    }
    free(s);
  }
}

/*
 * Window attention (Sec. 3.2.2): the Hg x Wg token grid is cut into
 * non-overlapping wh x ww windows anchored at the grid origin; softmax
 * attention (Eq. 1) runs independently inside each window.  When the grid is
 * not a multiple of the window, the right / bottom windows are simply smaller:
 * they hold the tokens that exist.  Token (y, x) belongs to window
 * (y / wh, x / ww); it attends exactly the tokens with the same window id.
 */
void jvo_window_attn(const double* q, const double* k, const double* v, double* o,
                     int64_t BH, int64_t Hg, int64_t Wg, int64_t D,
                     int64_t wh, int64_t ww, double scale) {
  const int64_t N = Hg * Wg;
#pragma omp parallel
  {
    double* s = (double*)malloc(sizeof(double) * (size_t)(wh * ww));
#pragma omp for collapse(2) schedule(dynamic, 16)
    for (int64_t g = 0; g < BH; ++g) {
      for (int64_t i = 0; i < N; ++i) {
        const int64_t y = i / Wg, x = i % Wg;
        const int64_t y0 = (y / wh) * wh, x0 = (x / ww) * ww;
        const int64_t y1 = (y0 + wh < Hg) ? y0 + wh : Hg;
        const int64_t x1 = (x0 + ww < Wg) ? x0 + ww : Wg;
        const double* qi = q + (g * N + i) * D;
        double* oi = o + (g * N + i) * D;
        double m = -INFINITY;
        int64_t c = 0;
        for (int64_t yy = y0; yy < y1; ++yy)
          for (int64_t xx = x0; xx < x1; ++xx) {
            const double* kj = k + (g * N + yy * Wg + xx) * D;
            double dot = 0.0;
            for (int64_t e = 0; e < D; ++e) dot += qi[e] * kj[e];
            s[c] = dot * scale;
            if (s[c] > m) m = s[c];
            ++c;
          }
        double denom = 0.0;
        for (int64_t e = 0; e < D; ++e) oi[e] = 0.0;
        c = 0;
        for (int64_t yy = y0; yy < y1; ++yy)
          for (int64_t xx = x0; xx < x1; ++xx) {
            const double* vj = v + (g * N + yy * Wg + xx) * D;
            double p = exp(s[c] - m);
            denom += p;
            for (int64_t e = 0; e < D; ++e) oi[e] += p * vj[e];
            ++c;
          }
        for (int64_t e = 0; e < D; ++e) oi[e] /= denom;
      }
    }
    free(s);
  }
}

static double silu(double x) { return x / (1.0 + exp(-x)); }

/*
 * Kernel generator of the squeeze dynamic convolution (Sec. 3.2.1): average
 * pooling of V over the grid, then a two-layer MLP with SiLU.
 *   s[b][c] = (1/N) sum_j V[b][c][j],  hid = SiLU(W1 s + b1),  w[b] = W2 hid + b2.
 * v: [B*H][N][D]; w: [B][C*k*k] with C = H*D, channel c = h*D + e.
 */
void jvo_dwc_generate(const double* v, double* w, int64_t B, int64_t H, int64_t N, int64_t D,
                      int64_t dwc_k, int64_t R, const double* W1, const double* b1,
                      const double* W2, const double* b2) {
  const int64_t C = H * D, kk = dwc_k * dwc_k;
  for (int64_t b = 0; b < B; ++b) {
    double* s = (double*)calloc((size_t)C, sizeof(double));
    double* hid = (double*)calloc((size_t)R, sizeof(double));
    for (int64_t h = 0; h < H; ++h)
      for (int64_t e = 0; e < D; ++e) {
        const double* vg = v + (b * H + h) * N * D;
        double acc = 0.0;
        for (int64_t j = 0; j < N; ++j) acc += vg[j * D + e];
        s[h * D + e] = acc / (double)N;
      }
    for (int64_t r = 0; r < R; ++r) {
      double acc = b1 ? b1[r] : 0.0;
      for (int64_t c = 0; c < C; ++c) acc += W1[r * C + c] * s[c];
      hid[r] = silu(acc);
    }
    for (int64_t t = 0; t < C * kk; ++t) {
      double acc = b2 ? b2[t] : 0.0;
      for (int64_t r = 0; r < R; ++r) acc += W2[t * R + r] * hid[r];
      w[b * C * kk + t] = acc;
    }
    free(s);
    free(hid);
  }
}

/*
 * JetViT linear-attention block (Sec. 3.2.1, Eqs. 2 and 4).
 *
 * Core, per (batch, head), phi = ReLU:
 *   KV = sum_j phi(k_j)^T v_j   (D x D),     z = sum_j phi(k_j)   (D),
 *   LA_i = (phi(q_i) KV) / (phi(q_i) . z + eps).
 * The paper's Eq. 4 prints no denominator; the row normalisation with eps in
 * the denominator only is the reading this build was given.
 *
 * Squeeze dynamic depth-wise convolution on V (used when dwc_k > 0): with
 * C = H*D value channels, channel c = h*D + e,
 *   s[b][c]  = mean over the N grid tokens of V[b][c]          (average pooling)
 *   hid      = SiLU(W1 s + b1)                                 (W1: [R][C])
 *   w[b]     = W2 hid + b2, viewed as [C][k][k]                (W2: [C*k*k][R])
 *   DW_i[c]  = sum_{dy,dx in [0,k)} w[b][c][dy][dx] * V[b][c][(y+dy-p, x+dx-p)]
 *              with p = (k-1)/2 and taps outside the grid contributing zero,
 *   O_i = LA_i + DW_i                                          (Eq. 4)
 * b1 / b2 may be NULL (no bias).  One kernel set per batch sample, shared by
 * all of its tokens.
 */
void jvo_linear_attn(const double* q, const double* k, const double* v, double* o,
                     int64_t B, int64_t H, int64_t Hg, int64_t Wg, int64_t D, double eps,
                     int64_t dwc_k, int64_t R, const double* W1, const double* b1,
                     const double* W2, const double* b2) {
  const int64_t N = Hg * Wg, C = H * D;

#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t g = 0; g < B * H; ++g) {
    const double* qg = q + g * N * D;
    const double* kg = k + g * N * D;
    const double* vg = v + g * N * D;
    double* og = o + g * N * D;
    double* KV = (double*)calloc((size_t)(D * D), sizeof(double));
    double* z = (double*)calloc((size_t)D, sizeof(double));
    for (int64_t j = 0; j < N; ++j)
      for (int64_t a = 0; a < D; ++a) {
        double pk = kg[j * D + a] > 0.0 ? kg[j * D + a] : 0.0;
        z[a] += pk;
        for (int64_t e = 0; e < D; ++e) KV[a * D + e] += pk * vg[j * D + e];
      }
    for (int64_t i = 0; i < N; ++i) {
      double denom = eps;
      for (int64_t e = 0; e < D; ++e) og[i * D + e] = 0.0;
      for (int64_t a = 0; a < D; ++a) {
        double pq = qg[i * D + a] > 0.0 ? qg[i * D + a] : 0.0;
        denom += pq * z[a];
        for (int64_t e = 0; e < D; ++e) og[i * D + e] += pq * KV[a * D + e];
      }
      for (int64_t e = 0; e < D; ++e) og[i * D + e] /= denom;
    }
    free(KV);
    free(z);
  }

  if (dwc_k <= 0) return;

  const int64_t kk = dwc_k * dwc_k, p = (dwc_k - 1) / 2;
  double* wall = (double*)calloc((size_t)(B * C * kk), sizeof(double));
  jvo_dwc_generate(v, wall, B, H, N, D, dwc_k, R, W1, b1, W2, b2);
  for (int64_t b = 0; b < B; ++b) {
    const double* w = wall + b * C * kk;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t h = 0; h < H; ++h)
      for (int64_t y = 0; y < Hg; ++y) {
        const double* vg = v + (b * H + h) * N * D;
        double* og = o + (b * H + h) * N * D;
        for (int64_t x = 0; x < Wg; ++x)
          for (int64_t e = 0; e < D; ++e) {
            const double* wc = w + (h * D + e) * kk;
            double acc = 0.0;
            for (int64_t dy = 0; dy < dwc_k; ++dy)
              for (int64_t dx = 0; dx < dwc_k; ++dx) {
                int64_t yy = y + dy - p, xx = x + dx - p;
                if (yy < 0 || yy >= Hg || xx < 0 || xx >= Wg) continue;
                acc += wc[dy * dwc_k + dx] * vg[(yy * Wg + xx) * D + e];
              }
            og[(y * Wg + x) * D + e] += acc;
          }
      }
  }
  free(wall);
}

/* ------------------------------------------------------------------------------------------
 * Prefix tokens beside the grid.
 *
 * The backbones the method converts (Sec. 4.1: DINOv3, DepthAnythingV2) carry a class token
 * and register tokens in front of the patch tokens.  The paper defines its window partition
 * (Sec. 3.2.2) and the convolution on V (Sec. 3.2.1, Eq. 4) on the feature map only and is
 * silent about these tokens; the reading taken here:
 *   - a sequence is P prefix tokens followed by the N = Hg*Wg grid tokens (row-major grid);
 *   - F (Eq. 1) and the linear attention proper (Eq. 2) are global: all P + N tokens are
 *     queries and keys (both are indifferent to where a token sits);
 *   - W (Sec. 3.2.2): a grid token attends the tokens of its window and the P prefix tokens;
 *     a prefix token attends all P + N tokens;
 *   - the depth-wise convolution and the average pooling that feeds its kernel generator see
 *     the feature map only: prefix rows of V are neither pooled nor convolved, and a prefix
 *     token's output is its linear-attention output alone.
 * With P = 0 each function below performs exactly the operations of its counterpart above,
 * in the same order.
 * ------------------------------------------------------------------------------------------ */

/* q, k, v, o: [BH][P + Hg*Wg][D]. */
void jvo_window_attn_prefix(const double* q, const double* k, const double* v, double* o,
                            int64_t BH, int64_t P, int64_t Hg, int64_t Wg, int64_t D,
                            int64_t wh, int64_t ww, double scale) {
  const int64_t N = Hg * Wg, T = P + N;
#pragma omp parallel
  {
    double* s = (double*)malloc(sizeof(double) * (size_t)T);
    int64_t* idx = (int64_t*)malloc(sizeof(int64_t) * (size_t)T);
#pragma omp for collapse(2) schedule(dynamic, 16)
    for (int64_t g = 0; g < BH; ++g) {
      for (int64_t i = 0; i < T; ++i) {
        /* the keys token i attends, as token indices */
        int64_t nk = 0;
        if (i < P) {
          for (int64_t j = 0; j < T; ++j) idx[nk++] = j;
        } else {
          const int64_t y = (i - P) / Wg, x = (i - P) % Wg;
          const int64_t y0 = (y / wh) * wh, x0 = (x / ww) * ww;
          const int64_t y1 = (y0 + wh < Hg) ? y0 + wh : Hg;
          const int64_t x1 = (x0 + ww < Wg) ? x0 + ww : Wg;
          for (int64_t j = 0; j < P; ++j) idx[nk++] = j;
          for (int64_t yy = y0; yy < y1; ++yy)
            for (int64_t xx = x0; xx < x1; ++xx) idx[nk++] = P + yy * Wg + xx;
        }
        const double* qi = q + (g * T + i) * D;
        double* oi = o + (g * T + i) * D;
        double m = -INFINITY;
        for (int64_t c = 0; c < nk; ++c) {
          const double* kj = k + (g * T + idx[c]) * D;
          double dot = 0.0;
          for (int64_t e = 0; e < D; ++e) dot += qi[e] * kj[e];
          s[c] = dot * scale;
          if (s[c] > m) m = s[c];
        }
        double denom = 0.0;
        for (int64_t e = 0; e < D; ++e) oi[e] = 0.0;
        for (int64_t c = 0; c < nk; ++c) {
          const double* vj = v + (g * T + idx[c]) * D;
          double p = exp(s[c] - m);
          denom += p;
          for (int64_t e = 0; e < D; ++e) oi[e] += p * vj[e];
        }
        for (int64_t e = 0; e < D; ++e) oi[e] /= denom;
      }
    }
    free(s);
    free(idx);
  }
}

/* Kernel generator with prefix tokens: the average pooling runs over the N grid tokens only.
 * v: [B*H][P + N][D]; w: [B][C*k*k]. */
void jvo_dwc_generate_prefix(const double* v, double* w, int64_t B, int64_t H, int64_t P, int64_t N,
                             int64_t D, int64_t dwc_k, int64_t R, const double* W1, const double* b1,
                             const double* W2, const double* b2) {
  const int64_t C = H * D, kk = dwc_k * dwc_k, T = P + N;
  for (int64_t b = 0; b < B; ++b) {
    double* s = (double*)calloc((size_t)C, sizeof(double));
    double* hid = (double*)calloc((size_t)(R > 0 ? R : 1), sizeof(double));
    for (int64_t h = 0; h < H; ++h)
      for (int64_t e = 0; e < D; ++e) {
        const double* vg = v + ((b * H + h) * T + P) * D;   /* first grid token */
        double acc = 0.0;
        for (int64_t j = 0; j < N; ++j) acc += vg[j * D + e];
        s[h * D + e] = acc / (double)N;
      }
    for (int64_t r = 0; r < R; ++r) {
      double acc = b1 ? b1[r] : 0.0;
      for (int64_t c = 0; c < C; ++c) acc += W1[r * C + c] * s[c];
      hid[r] = silu(acc);
    }
    for (int64_t t = 0; t < C * kk; ++t) {
      double acc = b2 ? b2[t] : 0.0;
      for (int64_t r = 0; r < R; ++r) acc += W2[t * R + r] * hid[r];
      w[b * C * kk + t] = acc;
    }
    free(s);
    free(hid);
  }
}

/* q, k, v, o: [B*H][P + Hg*Wg][D]. */
void jvo_linear_attn_prefix(const double* q, const double* k, const double* v, double* o,
                            int64_t B, int64_t H, int64_t P, int64_t Hg, int64_t Wg, int64_t D, double eps,
                            int64_t dwc_k, int64_t R, const double* W1, const double* b1,
                            const double* W2, const double* b2) {
  const int64_t N = Hg * Wg, T = P + N, C = H * D;

#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t g = 0; g < B * H; ++g) {
    const double* qg = q + g * T * D;
    const double* kg = k + g * T * D;
    const double* vg = v + g * T * D;
    double* og = o + g * T * D;
    double* KV = (double*)calloc((size_t)(D * D), sizeof(double));
    double* z = (double*)calloc((size_t)D, sizeof(double));
    for (int64_t j = 0; j < T; ++j)          /* prefix and grid tokens alike */
      for (int64_t a = 0; a < D; ++a) {
        double pk = kg[j * D + a] > 0.0 ? kg[j * D + a] : 0.0;
        z[a] += pk;
        for (int64_t e = 0; e < D; ++e) KV[a * D + e] += pk * vg[j * D + e];
      }
    for (int64_t i = 0; i < T; ++i) {
      double denom = eps;
      for (int64_t e = 0; e < D; ++e) og[i * D + e] = 0.0;
      for (int64_t a = 0; a < D; ++a) {
        double pq = qg[i * D + a] > 0.0 ? qg[i * D + a] : 0.0;
        denom += pq * z[a];
        for (int64_t e = 0; e < D; ++e) og[i * D + e] += pq * KV[a * D + e];
      }
      for (int64_t e = 0; e < D; ++e) og[i * D + e] /= denom;
    }
    free(KV);
    free(z);
  }

  if (dwc_k <= 0) return;

  const int64_t kk = dwc_k * dwc_k, p = (dwc_k - 1) / 2;
  double* wall = (double*)calloc((size_t)(B * C * kk), sizeof(double));
  jvo_dwc_generate_prefix(v, wall, B, H, P, N, D, dwc_k, R, W1, b1, W2, b2);
  for (int64_t b = 0; b < B; ++b) {
    const double* w = wall + b * C * kk;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t h = 0; h < H; ++h)
      for (int64_t y = 0; y < Hg; ++y) {
        const double* vg = v + ((b * H + h) * T + P) * D;   /* the grid part of V */
        double* og = o + ((b * H + h) * T + P) * D;
        for (int64_t x = 0; x < Wg; ++x)
          for (int64_t e = 0; e < D; ++e) {
            const double* wc = w + (h * D + e) * kk;
            double acc = 0.0;
            for (int64_t dy = 0; dy < dwc_k; ++dy)
              for (int64_t dx = 0; dx < dwc_k; ++dx) {
                int64_t yy = y + dy - p, xx = x + dx - p;
                if (yy < 0 || yy >= Hg || xx < 0 || xx >= Wg) continue;
                acc += wc[dy * dwc_k + dx] * vg[(yy * Wg + xx) * D + e];
              }
            og[(y * Wg + x) * D + e] += acc;
          }
      }
  }
  free(wall);
}

/*
 * Focused feature map (Eq. 3; the kernel function of the cited focused linear attention):
 *   phi_p(x) = (||r|| / ||r^p||) r^p,   r = ReLU(x),  r^p element-wise,
 * per token and head over the D features: a sharper direction with the norm of ReLU(x) kept.
 * The paper prints the denominator as ||x||^p; the reading taken is the cited work's ||x^p||
 * (with it the map is positively homogeneous, phi(a x) = a phi(x), and p = 1 is plain ReLU).
 * A row whose ReLU is the zero vector maps to zero.  x, out: [rows][D].
 */
void jvo_focus_map(const double* x, double* out, int64_t rows, int64_t D, double p) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < rows; ++i) {
    const double* xi = x + i * D;
    double* oi = out + i * D;
    double n1 = 0.0, np = 0.0;
    for (int64_t e = 0; e < D; ++e) {
      const double r = xi[e] > 0.0 ? xi[e] : 0.0;
      const double rp = r > 0.0 ? pow(r, p) : 0.0;
      oi[e] = rp;
      n1 += r * r;
      np += rp * rp;
    }
    const double scale = np > 0.0 ? sqrt(n1) / sqrt(np) : 0.0;
    for (int64_t e = 0; e < D; ++e) oi[e] *= scale;
  }
}

/*
 * Token-wise dynamic depth-wise convolution (Sec. 3.2.1 "JetViT Linear Attention Block", the
 * variant the paper tries first and drops for its cost; Table 1 "+ Token-wise Dynamic DWC"):
 * the kernel generator, the same two-layer MLP with SiLU, is fed with each token's own value
 * vector instead of the pooled one and emits one set of kernels per token:
 *   for grid token i of sample b, with v_i in R^C its value vector over all heads (c = h*D + e):
 *     hid_i = SiLU(W1 v_i + b1),   w_i = W2 hid_i + b2  viewed as [C][k][k],
 *     DW_i[c] = sum_{dy,dx} w_i[c][dy][dx] * V[b][c][(y + dy - p, x + dx - p)]   (zero outside the grid)
 *   O_i = LA_i + DW_i.
 * The paper gives no formula; this is the reading: the kernels of the OUTPUT position are
 * applied to that position's neighbourhood, everything else as in the squeeze dynamic variant
 * (prefix tokens: attention only).  q, k, v, o: [B*H][P + Hg*Wg][D].
 */
void jvo_linear_attn_tokenwise(const double* q, const double* k, const double* v, double* o,
                               int64_t B, int64_t H, int64_t P, int64_t Hg, int64_t Wg, int64_t D, double eps,
                               int64_t dwc_k, int64_t R, const double* W1, const double* b1,
                               const double* W2, const double* b2) {
  const int64_t N = Hg * Wg, T = P + N, C = H * D, kk = dwc_k * dwc_k, pad = (dwc_k - 1) / 2;
  jvo_linear_attn_prefix(q, k, v, o, B, H, P, Hg, Wg, D, eps, 0, 0, 0, 0, 0, 0);   /* LA_i for every token */
#pragma omp parallel
  {
    double* vi = (double*)malloc(sizeof(double) * (size_t)C);
    double* hid = (double*)malloc(sizeof(double) * (size_t)(R > 0 ? R : 1));
#pragma omp for collapse(2) schedule(dynamic, 4)
    for (int64_t b = 0; b < B; ++b)
      for (int64_t i = 0; i < N; ++i) {
        const int64_t y = i / Wg, x = i % Wg;
        for (int64_t c = 0; c < C; ++c) vi[c] = v[((b * H + c / D) * T + P + i) * D + c % D];
        for (int64_t r = 0; r < R; ++r) {
          double acc = b1 ? b1[r] : 0.0;
          for (int64_t c = 0; c < C; ++c) acc += W1[r * C + c] * vi[c];
          hid[r] = silu(acc);
        }
        for (int64_t c = 0; c < C; ++c) {
          const double* vg = v + ((b * H + c / D) * T + P) * D + c % D;   /* channel c of the grid, stride D */
          double dw = 0.0;
          for (int64_t dy = 0; dy < dwc_k; ++dy)
            for (int64_t dx = 0; dx < dwc_k; ++dx) {
              const int64_t yy = y + dy - pad, xx = x + dx - pad;
              if (yy < 0 || yy >= Hg || xx < 0 || xx >= Wg) continue;
              const int64_t t = c * kk + dy * dwc_k + dx;
              double w = b2 ? b2[t] : 0.0;
              for (int64_t r = 0; r < R; ++r) w += W2[t * R + r] * hid[r];
              dw += w * vg[(yy * Wg + xx) * D];
            }
          o[((b * H + c / D) * T + P + i) * D + c % D] += dw;
        }
      }
    free(vi);
    free(hid);
  }
}
