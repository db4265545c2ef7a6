/*
 * CPU oracle for the multi-scale ReLU linear attention module (EfficientViT,
 * arXiv 2205.14756, Section 3.1).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64 statement of
 * what the module computes.  It is used by the tests, by the smoke check and
 * by the benchmark's CPU-baseline leg; no product code path may call it.  It
 * shares no code, header, table or helper with the CUDA implementation.
 *
 * Every function is the definition written out as loops: no blocking, no
 * fusion, no reordering beyond what the cited passage states.  OpenMP is used
 * on outermost independent loops only (it does not change any sum's order).
 *
 * Pins (see tests/test_oracle_pins.py): explicit N x N attention of Eq. 1 with
 * the similarity of Eq. 2, invariants of Eq. 3, closed forms of the
 * convolutions, a hand-worked example.  The whole-module function has no
 * end-to-end golden value anywhere in the paper; it is pinned through its
 * parts and through special weight choices that reduce it to them.
 *
 * All tensors are dense, row-major, double precision, caller-owned.
 */
#include <stddef.h>
#include <stdlib.h>
#include <string.h>

#if defined(_OPENMP)
#include <omp.h>
#endif

int oracle_num_threads(void) {
#if defined(_OPENMP)
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void oracle_set_num_threads(int n) {
#if defined(_OPENMP)
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

/*
 * 1x1 convolution = per-token linear projection (Section 3.1: Q = x W_Q,
 * K = x W_K, V = x W_V; and the final linear projection after the head
 * concat).  x [B, Cin, N], w [Cout, Cin], bias [Cout] or NULL, y [B, Cout, N].
 *   y[b,o,n] = sum_c w[o,c] * x[b,c,n] (+ bias[o])
 */
void oracle_conv1x1(const double* x, const double* w, const double* bias, double* y,
                    int B, int Cin, int Cout, long N) {
#pragma omp parallel for collapse(2) schedule(static)
  for (int b = 0; b < B; ++b) {
    for (int o = 0; o < Cout; ++o) {
      double* yrow = y + ((size_t)b * Cout + o) * N;
      for (long n = 0; n < N; ++n) yrow[n] = bias ? bias[o] : 0.0;
      for (int c = 0; c < Cin; ++c) {
        const double wv = w[(size_t)o * Cin + c];
        const double* xrow = x + ((size_t)b * Cin + c) * N;
        for (long n = 0; n < N; ++n) yrow[n] += wv * xrow[n];
      }
    }
  }
}

/*
 * Depthwise k x k convolution used for token aggregation (last paragraph of
 * Section 3.1: a depthwise convolution with a small kernel followed by a grouped
 * 1x1 convolution; Section 4.1 fixes 5x5).
 * Cross-correlation, stride 1, zero padding k/2, output size = input size.
 * x [B, Ch, H, W], w [Ch, k, k] with taps indexed [dy][dx], y [B, Ch, H, W].
 *   y[b,o,r,s] = sum_{dy,dx} w[o,dy,dx] * x[b,o,r+dy-k/2,s+dx-k/2]   (0 outside)
 */
void oracle_dwconv(const double* x, const double* w, double* y,
                   int B, int Ch, int H, int W, int k) {
  const int p = k / 2;
#pragma omp parallel for collapse(2) schedule(static)
  for (int b = 0; b < B; ++b) {
    for (int o = 0; o < Ch; ++o) {
      const double* xp = x + ((size_t)b * Ch + o) * H * W;
      double* yp = y + ((size_t)b * Ch + o) * H * W;
      const double* wk = w + (size_t)o * k * k;
      for (int r = 0; r < H; ++r) {
        for (int s = 0; s < W; ++s) {
          double acc = 0.0;
          for (int dy = 0; dy < k; ++dy) {
            const int rr = r + dy - p;
            if (rr < 0 || rr >= H) continue;
            for (int dx = 0; dx < k; ++dx) {
              const int ss = s + dx - p;
              if (ss < 0 || ss >= W) continue;
              acc += wk[dy * k + dx] * xp[(size_t)rr * W + ss];
            }
          }
          yp[(size_t)r * W + s] = acc;
        }
      }
    }
  }
}

/*
 * Grouped 1x1 convolution (Section 3.1: all 1x1 convs of the aggregation are
 * combined into one group convolution with 3 x #heads groups of d channels).
 * x [B, Ch, N], w [Ch, d], y [B, Ch, N]; Ch must be a multiple of d.
 *   y[b,o,n] = sum_{i<d} w[o,i] * x[b, (o/d)*d + i, n]
 */
void oracle_group1x1(const double* x, const double* w, double* y,
                     int B, int Ch, int d, long N) {
#pragma omp parallel for collapse(2) schedule(static)
  for (int b = 0; b < B; ++b) {
    for (int o = 0; o < Ch; ++o) {
      double* yrow = y + ((size_t)b * Ch + o) * N;
      const int g0 = (o / d) * d;
      for (long n = 0; n < N; ++n) yrow[n] = 0.0;
      for (int i = 0; i < d; ++i) {
        const double wv = w[(size_t)o * d + i];
        const double* xrow = x + ((size_t)b * Ch + g0 + i) * N;
        for (long n = 0; n < N; ++n) yrow[n] += wv * xrow[n];
      }
    }
  }
}

static double relu(double a) { return a > 0.0 ? a : 0.0; }

/*
 * ReLU linear attention, Eq. 3: for each (batch, head)
 *   KV[a,c]  = sum_j relu(K[j,a]) * V[j,c]          (d x d)
 *   ks[a]    = sum_j relu(K[j,a])                   (d x 1)
 *   O[i,c]   = sum_a relu(Q[i,a]) * KV[a,c] / (sum_a relu(Q[i,a]) * ks[a] + eps)
 * q, k, v, out: [B, heads, N, d], d innermost.  eps is added once to the
 * denominator (the paper's Eq. 3 has no eps; with eps the 0/0 case of an
 * all-non-positive query row gives exactly 0).
 */
void oracle_linattn_relu(const double* q, const double* k, const double* v, double* out,
                         int B, int heads, long N, int d, double eps) {
  const long BH = (long)B * heads;
#pragma omp parallel for schedule(dynamic, 1)
  for (long bh = 0; bh < BH; ++bh) {
    const double* qh = q + (size_t)bh * N * d;
    const double* kh = k + (size_t)bh * N * d;
    const double* vh = v + (size_t)bh * N * d;
    double* oh = out + (size_t)bh * N * d;
    double* KV = (double*)calloc((size_t)d * d, sizeof(double));
    double* ks = (double*)calloc((size_t)d, sizeof(double));
    for (long j = 0; j < N; ++j) {
      for (int a = 0; a < d; ++a) {
        const double ka = relu(kh[j * d + a]);
        ks[a] += ka;
        for (int c = 0; c < d; ++c) KV[a * d + c] += ka * vh[j * d + c];
      }
    }
    for (long i = 0; i < N; ++i) {
      double den = 0.0;
      for (int a = 0; a < d; ++a) den += relu(qh[i * d + a]) * ks[a];
      for (int c = 0; c < d; ++c) {
        double num = 0.0;
        for (int a = 0; a < d; ++a) num += relu(qh[i * d + a]) * KV[a * d + c];
        oh[i * d + c] = num / (den + eps);
      }
    }
    free(KV);
    free(ks);
  }
}

/*
 * Whole module (Section 3.1, Figure 2 right), NCHW:
 *   1. qkv  = conv1x1(x, w_qkv)                              [B, 3C', H, W]
 *   2. agg  = group1x1(dwconv_kxk(qkv, w_dw), w_pw)          [B, 3C', H, W]
 *   3. multi-scale tokens = channel concat (qkv, agg): 2*heads heads of 3d
 *      channels each, [q | k | v] inside a head; token n = r*W + s
 *   4. ReLU linear attention per (batch, head) over all N = H*W tokens
 *   5. head outputs concatenated along channels (scale 0 heads first), then
 *      out = conv1x1(att, w_proj, b_proj)                    [B, C_out, H, W]
 * C' = heads * d.  Returns 0, or -1 if a scratch allocation fails.
 */
int oracle_msla_forward(const double* x, const double* w_qkv, const double* w_dw,
                        const double* w_pw, const double* w_proj, const double* b_proj,
                        double* out, int B, int C, int H, int W, int heads, int d,
                        int k, int C_out, double eps) {
  const long N = (long)H * W;
  const int Cp = heads * d;
  const int C3 = 3 * Cp;
  const int Ht = 2 * heads;
  const size_t plane = (size_t)B * C3 * N;
  double* qkv = (double*)malloc(plane * sizeof(double));
  double* dw = (double*)malloc(plane * sizeof(double));
  double* agg = (double*)malloc(plane * sizeof(double));
  const size_t hsz = (size_t)B * Ht * N * d;
  double* qh = (double*)malloc(hsz * sizeof(double));
  double* kh = (double*)malloc(hsz * sizeof(double));
  double* vh = (double*)malloc(hsz * sizeof(double));
  double* oh = (double*)malloc(hsz * sizeof(double));
  double* att = (double*)malloc((size_t)B * 2 * Cp * N * sizeof(double));
  int rc = -1;
  if (qkv && dw && agg && qh && kh && vh && oh && att) {
    oracle_conv1x1(x, w_qkv, NULL, qkv, B, C, C3, N);
    oracle_dwconv(qkv, w_dw, dw, B, C3, H, W, k);
    oracle_group1x1(dw, w_pw, agg, B, C3, d, N);
    /* step 3: gather [B, Ht, N, d] per-head token matrices */
    for (int b = 0; b < B; ++b)
      for (int hh = 0; hh < Ht; ++hh) {
        const double* src = (hh < heads ? qkv : agg) + (size_t)b * C3 * N;
        const int hs = hh < heads ? hh : hh - heads; /* head index inside its scale */
        for (long n = 0; n < N; ++n)
          for (int i = 0; i < d; ++i) {
            const size_t dst = (((size_t)b * Ht + hh) * N + n) * d + i;
            qh[dst] = src[((size_t)hs * 3 * d + 0 * d + i) * N + n];
            kh[dst] = src[((size_t)hs * 3 * d + 1 * d + i) * N + n];
            vh[dst] = src[((size_t)hs * 3 * d + 2 * d + i) * N + n];
          }
      }
    oracle_linattn_relu(qh, kh, vh, oh, B, Ht, N, d, eps);
    /* step 5: head concat along channels, channel = head*d + c */
    for (int b = 0; b < B; ++b)
      for (int hh = 0; hh < Ht; ++hh)
        for (long n = 0; n < N; ++n)
          for (int c = 0; c < d; ++c)
            att[((size_t)b * 2 * Cp + (size_t)hh * d + c) * N + n] =
                oh[(((size_t)b * Ht + hh) * N + n) * d + c];
    oracle_conv1x1(att, w_proj, b_proj, out, B, 2 * Cp, C_out, N);
    rc = 0;
  }
  free(qkv); free(dw); free(agg); free(qh); free(kh); free(vh); free(oh); free(att);
  return rc;
}

/* ------------------------------------------------------------------------
 * The other half of the EfficientViT building block (Section 3.1, second
 * paragraph after Eq. 3, and Fig. 2 left): a feed-forward network with a
 * depthwise convolution inserted into it (FFN+DWConv), which supplies the
 * local information that ReLU linear attention lacks.  The paper names
 * neither the expansion ratio, the activation, the kernel of the depthwise
 * convolution nor the normalisation; all are arguments here.
 *
 * Activation applied after the first linear layer and after the depthwise
 * convolution: 0 identity, 1 ReLU max(a, 0), 2 hard-swish a * min(max(a + 3, 0), 6) / 6
 * (Howard et al., "Searching for MobileNetV3", Eq. for h-swish).
 */
static double ffn_act(double a, int kind) {
  if (kind == 1) return a > 0.0 ? a : 0.0;
  if (kind == 2) {
    double r = a + 3.0;
    if (r < 0.0) r = 0.0;
    if (r > 6.0) r = 6.0;
    return a * r / 6.0;
  }
  return a;
}

/* y[b,c,n] = act(y[b,c,n] + bias[c]), in place; bias [Ch] or NULL. */
void oracle_bias_act(double* y, const double* bias, int B, int Ch, long N, int act) {
#pragma omp parallel for collapse(2) schedule(static)
  for (int b = 0; b < B; ++b)
    for (int c = 0; c < Ch; ++c) {
      double* row = y + ((size_t)b * Ch + c) * N;
      const double bv = bias ? bias[c] : 0.0;
      for (long n = 0; n < N; ++n) row[n] = ffn_act(row[n] + bv, act);
    }
}

/*
 * FFN+DWConv on an NCHW feature map:
 *   h   = act(conv1x1(x, w1) + b1)                 C  -> Ch   (the FFN's first linear layer)
 *   g   = act(dwconv(h, w_dw) + b_dw)              k x k depthwise, zero padding k/2 (the inserted convolution)
 *   out = conv1x1(g, w2) + b2 (+ x if residual)    Ch -> C_out (the FFN's second linear layer)
 * x [B, C, H, W], w1 [Ch, C], w_dw [Ch, k, k], w2 [C_out, Ch], biases [.] or NULL (an inference-time folded
 * normalisation is a bias), out [B, C_out, H, W].  residual != 0 needs C_out == C.
 * Returns 0, -1 if a scratch allocation fails, -2 on residual with C_out != C.
 */
int oracle_ffn_dwconv(const double* x, const double* w1, const double* b1, const double* w_dw,
                      const double* b_dw, const double* w2, const double* b2, double* out, int B,
                      int C, int Ch, int H, int W, int k, int C_out, int act, int residual) {
  if (residual && C_out != C) return -2;
  const long N = (long)H * W;
  const size_t hid = (size_t)B * Ch * N;
  double* h = (double*)malloc(hid * sizeof(double));
  double* g = (double*)malloc(hid * sizeof(double));
  int rc = -1;
  if (h && g) {
    oracle_conv1x1(x, w1, b1, h, B, C, Ch, N);
    oracle_bias_act(h, NULL, B, Ch, N, act);
    oracle_dwconv(h, w_dw, g, B, Ch, H, W, k);
    oracle_bias_act(g, b_dw, B, Ch, N, act);
    oracle_conv1x1(g, w2, b2, out, B, Ch, C_out, N);
    if (residual) {
      const size_t total = (size_t)B * C * N;
      for (size_t i = 0; i < total; ++i) out[i] += x[i];
    }
    rc = 0;
  }
  free(h); free(g);
  return rc;
}

/* ------------------------------------------------------------------------
 * The module with THREE branches (Section 3.1 builds multi-scale tokens by
 * aggregating nearby tokens with several small kernels; Section 4.1 then
 * settles on two branches, which is oracle_msla_forward above): the projected
 * tokens, and two aggregated copies of them, each through its own depthwise
 * k x k convolution and grouped 1x1 convolution.  Heads: all heads of branch
 * 0, then branch 1, then branch 2; w_proj is [C_out, 3C'].  Written out in
 * full rather than folded into the two-branch function so that each can be
 * read against the text on its own.  Returns 0, or -1 if an allocation fails.
 */
int oracle_msla_forward3(const double* x, const double* w_qkv, const double* w_dw1,
                         const double* w_pw1, const double* w_dw2, const double* w_pw2,
                         const double* w_proj, const double* b_proj, double* out, int B, int C,
                         int H, int W, int heads, int d, int k1, int k2, int C_out, double eps) {
  const long N = (long)H * W;
  const int Cp = heads * d;
  const int C3 = 3 * Cp;
  const int Ht = 3 * heads;
  const size_t plane = (size_t)B * C3 * N;
  double* qkv = (double*)malloc(plane * sizeof(double));
  double* dw = (double*)malloc(plane * sizeof(double));
  double* agg1 = (double*)malloc(plane * sizeof(double));
  double* agg2 = (double*)malloc(plane * sizeof(double));
  const size_t hsz = (size_t)B * Ht * N * d;
  double* qh = (double*)malloc(hsz * sizeof(double));
  double* kh = (double*)malloc(hsz * sizeof(double));
  double* vh = (double*)malloc(hsz * sizeof(double));
  double* oh = (double*)malloc(hsz * sizeof(double));
  double* att = (double*)malloc((size_t)B * 3 * Cp * N * sizeof(double));
  int rc = -1;
  if (qkv && dw && agg1 && agg2 && qh && kh && vh && oh && att) {
    oracle_conv1x1(x, w_qkv, NULL, qkv, B, C, C3, N);
    oracle_dwconv(qkv, w_dw1, dw, B, C3, H, W, k1);
    oracle_group1x1(dw, w_pw1, agg1, B, C3, d, N);
    oracle_dwconv(qkv, w_dw2, dw, B, C3, H, W, k2);
    oracle_group1x1(dw, w_pw2, agg2, B, C3, d, N);
    for (int b = 0; b < B; ++b)
      for (int hh = 0; hh < Ht; ++hh) {
        const int branch = hh / heads, hs = hh % heads; /* head index inside its branch */
        const double* src = (branch == 0 ? qkv : branch == 1 ? agg1 : agg2) + (size_t)b * C3 * N;
        for (long n = 0; n < N; ++n)
          for (int i = 0; i < d; ++i) {
            const size_t dst = (((size_t)b * Ht + hh) * N + n) * d + i;
            qh[dst] = src[((size_t)hs * 3 * d + 0 * d + i) * N + n];
            kh[dst] = src[((size_t)hs * 3 * d + 1 * d + i) * N + n];
            vh[dst] = src[((size_t)hs * 3 * d + 2 * d + i) * N + n];
          }
      }
    oracle_linattn_relu(qh, kh, vh, oh, B, Ht, N, d, eps);
    for (int b = 0; b < B; ++b)
      for (int hh = 0; hh < Ht; ++hh)
        for (long n = 0; n < N; ++n)
          for (int c = 0; c < d; ++c)
            att[((size_t)b * 3 * Cp + (size_t)hh * d + c) * N + n] =
                oh[(((size_t)b * Ht + hh) * N + n) * d + c];
    oracle_conv1x1(att, w_proj, b_proj, out, B, 3 * Cp, C_out, N);
    rc = 0;
  }
  free(qkv); free(dw); free(agg1); free(agg2); free(qh); free(kh); free(vh); free(oh); free(att);
  return rc;
}
