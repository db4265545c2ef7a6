// Plain SIMT kernels for every stage of the module, templated on the storage
// type.  They are the fp32 path (a TF32 tensor-core product would not meet the
// fp32 accuracy bound) and the fallback for bf16 shapes the tuned kernels do
// not cover.  All accumulate in fp32 and are deterministic.
#pragma once

#include "msla_common.cuh"

namespace msla {
namespace generic {

// ---------------------------------------------------------------------------
// Strided GEMM for the two 1x1 projections (Section 3.1: Q = xW_Q, K = xW_K,
// V = xW_V; final linear projection):
//   D(m, n) = sum_k A(m, k) * W[n, k] (+ bias[n]),   m = token, n = out channel
// A(m, k) = A[b*sAb + m*sAm + k*sAk];
// D(m, n) = D[b*sDb + (n / group)*sDg + m*sDm + (n % group)*sDn]: out channels
// may be split into groups of `group` that live in separate planes.
// ---------------------------------------------------------------------------
struct GemmArgs {
  long long sAb, sAm, sAk;
  long long sDb, sDm, sDn, sDg;
  int M, Nc, K;  // tokens, out channels, in channels
  int group;     // out channels per plane (>= Nc: one plane)
  int act;       // applied to the sum + bias: 0 none, 1 ReLU, 2 hard-swish
  const void* residual;  // nullptr, or a tensor laid out like D, added after the activation
};

__device__ __forceinline__ float act_f32(float v, int act) {
  if (act == 1) return fmaxf(v, 0.f);
  if (act == 2) return v * fminf(fmaxf(v + 3.f, 0.f), 6.f) / 6.f;
  return v;
}

template <typename T>
__global__ void __launch_bounds__(256)
gemm_kernel(const T* __restrict__ A, const T* __restrict__ Wt, const T* __restrict__ bias,
            T* __restrict__ D, GemmArgs g) {
  constexpr int BM = 64, BN = 64, BK = 16;
  __shared__ float As[BK][BM + 4];
  __shared__ float Ws[BK][BN + 4];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const long long m0 = (long long)blockIdx.x * BM;
  const int n0 = blockIdx.y * BN;
  const int b = blockIdx.z;
  const bool a_m_contig = (g.sAm == 1);
  const bool d_m_contig = (g.sDm == 1);
  const int mi = (d_m_contig ? tx : ty) * 4;
  const int ni = (d_m_contig ? ty : tx) * 4;
  const T* Ab = A + (long long)b * g.sAb;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < g.K; k0 += BK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int e = tid + i * 256;
      int m, k;
      if (a_m_contig) { m = e & (BM - 1); k = e >> 6; } else { k = e & (BK - 1); m = e >> 4; }
      float v = 0.f;
      if (m0 + m < g.M && k0 + k < g.K) v = to_f32(Ab[(m0 + m) * g.sAm + (long long)(k0 + k) * g.sAk]);
      As[k][m] = v;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int e = tid + i * 256;
      const int k = e & (BK - 1), n = e >> 4;
      float v = 0.f;
      if (n0 + n < g.Nc && k0 + k < g.K) v = to_f32(Wt[(long long)(n0 + n) * g.K + k0 + k]);
      Ws[k][n] = v;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[k][mi + i]; w[i] = Ws[k][ni + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
  T* Db = D + (long long)b * g.sDb;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const long long m = m0 + mi + i;
    if (m >= g.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + ni + j;
      if (n >= g.Nc) continue;
      float r = act_f32(acc[i][j] + (bias ? to_f32(bias[n]) : 0.f), g.act);
      const long long at = (long long)(n / g.group) * g.sDg + m * g.sDm + (long long)(n % g.group) * g.sDn;
      if (g.residual) r += to_f32(static_cast<const T*>(g.residual)[(long long)b * g.sDb + at]);
      Db[at] = from_f32<T>(r);
    }
  }
}

// ---------------------------------------------------------------------------
// The depthwise 3x3 convolution inside the FFN (Section 3.1, Fig. 2 left) with its bias and activation, on NCHW:
//   g[b,c,y,x] = act(sum_{dy,dx} w[c,dy,dx] * h[b,c,y+dy-1,x+dx-1] + bias[c]), zero padding 1.  One thread per output.
// ---------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
ffn_dw3x3_nchw_kernel(const T* __restrict__ h, const T* __restrict__ w, const T* __restrict__ bias, T* __restrict__ g,
                      int Ch, int H, int W, int act, long long total) {
  const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
  if (idx >= total) return;
  const int x = (int)(idx % W), y = (int)((idx / W) % H);
  const long long bc = idx / ((long long)W * H);
  const int c = (int)(bc % Ch);
  const T* hp = h + bc * H * W;
  float acc = bias ? to_f32(bias[c]) : 0.f;
  for (int dy = 0; dy < 3; ++dy) {
    const int yy = y + dy - 1;
    if (yy < 0 || yy >= H) continue;
    for (int dx = 0; dx < 3; ++dx) {
      const int xx = x + dx - 1;
      if (xx < 0 || xx >= W) continue;
      acc = fmaf(to_f32(w[(long long)c * 9 + dy * 3 + dx]), to_f32(hp[(long long)yy * W + xx]), acc);
    }
  }
  g[idx] = from_f32<T>(act_f32(acc, act));
}

// 3x3 depthwise taps embedded in a 5x5 filter with a ring of zeros: w5[c][r][s] = w3[c][r-1][s-1] inside, 0 outside.
template <typename T>
__global__ void __launch_bounds__(256)
embed_taps_kernel(const T* __restrict__ w3, T* __restrict__ w5, long long total) {
  const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
  if (idx >= total) return;
  const long long c = idx / 25;
  const int r = (int)(idx % 25) / 5, s = (int)(idx % 5);
  const bool inside = r >= 1 && r <= 3 && s >= 1 && s <= 3;
  w5[idx] = inside ? w3[c * 9 + (r - 1) * 3 + (s - 1)] : from_f32<T>(0.f);
}

// ---------------------------------------------------------------------------
// Multi-scale token aggregation (Section 3.1): 5x5 depthwise convolution
// (cross-correlation, zero padding 2) followed by the grouped 1x1 convolution,
// on planar activations [B, groups, H*W, d].  One CTA = one 8x8 pixel tile of
// one group of d channels.  src(b, g, n, i) = src[b*src_sb + (g*H*W + n)*d + i];
// dst likewise with dst_sb.
// ---------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
aggregate_kernel(const T* __restrict__ src, const T* __restrict__ w_dw, const T* __restrict__ w_pw,
                 T* __restrict__ dst, int H, int W, int d, long long src_sb, long long dst_sb) {
  constexpr int TS = 8, HALO = TS + 4, DMAX = 32;
  __shared__ float tile[HALO * HALO][DMAX + 1];
  __shared__ float dwo[TS * TS][DMAX + 1];
  __shared__ float wdw[DMAX][25];
  __shared__ float wpw[DMAX][DMAX + 1];
  const int tid = threadIdx.x;
  const int tiles_x = (W + TS - 1) / TS;
  const int x0 = (blockIdx.x % tiles_x) * TS, y0 = (blockIdx.x / tiles_x) * TS;
  const int ch0 = blockIdx.y * d;
  const int b = blockIdx.z;
  const T* sb = src + (long long)b * src_sb + (long long)blockIdx.y * H * W * d;
  for (int e = tid; e < d * 25; e += 256) wdw[e / 25][e % 25] = to_f32(w_dw[(long long)ch0 * 25 + e]);
  for (int e = tid; e < d * d; e += 256) wpw[e / d][e % d] = to_f32(w_pw[(long long)ch0 * d + e]);
  for (int e = tid; e < HALO * HALO * d; e += 256) {
    const int c = e % d, p = e / d;
    const int yy = y0 + p / HALO - 2, xx = x0 + p % HALO - 2;
    float v = 0.f;
    if (yy >= 0 && yy < H && xx >= 0 && xx < W) v = to_f32(sb[((long long)yy * W + xx) * d + c]);
    tile[p][c] = v;
  }
  __syncthreads();
  for (int e = tid; e < TS * TS * d; e += 256) {
    const int c = e % d, p = e / d;
    const int py = p / TS, px = p % TS;
    float acc = 0.f;
#pragma unroll
    for (int dy = 0; dy < 5; ++dy)
#pragma unroll
      for (int dx = 0; dx < 5; ++dx)
        acc = fmaf(wdw[c][dy * 5 + dx], tile[(py + dy) * HALO + px + dx][c], acc);
    dwo[p][c] = acc;
  }
  __syncthreads();
  T* db = dst + (long long)b * dst_sb + (long long)blockIdx.y * H * W * d;
  for (int e = tid; e < TS * TS * d; e += 256) {
    const int o = e % d, p = e / d;
    const int yy = y0 + p / TS, xx = x0 + p % TS;
    if (yy >= H || xx >= W) continue;
    float acc = 0.f;
    for (int i = 0; i < d; ++i) acc = fmaf(wpw[o][i], dwo[p][i], acc);
    db[((long long)yy * W + xx) * d + o] = from_f32<T>(acc);
  }
}

// ---------------------------------------------------------------------------
// KV-state reduction, first level (Eq. 3): for one (batch, head) and one chunk
// of tokens,  part[a][c] = sum_j relu(k[j,a]) * v[j,c]  for c < d and
// part[a][d] = sum_j relu(k[j,a]).   Partials: [BH][S][d*(d+1)] fp32.
// ---------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
kv_partial_kernel(const T* __restrict__ k, const T* __restrict__ v, float* __restrict__ partial,
                  HeadView kv, int heads, int N, int d, int S, int chunk) {
  constexpr int TT = 32, DMAX = 32, EPT = 5;  // 256*5 >= 32*33
  __shared__ float ks[TT][DMAX + 1];
  __shared__ float vs[TT][DMAX + 1];
  const int tid = threadIdx.x;
  const int bh = blockIdx.x, s = blockIdx.y;
  const int b = bh / heads, h = bh % heads;
  const long long base = (long long)b * kv.batch + (long long)h * kv.head;
  const int n_begin = s * chunk;
  const int n_end = min(N, n_begin + chunk);
  const int d1 = d + 1, ne = d * d1;
  int ea[EPT], ec[EPT];
  float acc[EPT];
#pragma unroll
  for (int i = 0; i < EPT; ++i) {
    const int e = tid + i * 256;
    ea[i] = e < ne ? e / d1 : 0;
    ec[i] = e < ne ? e % d1 : 0;
    acc[i] = 0.f;
  }
  for (int n0 = n_begin; n0 < n_end; n0 += TT) {
    for (int e = tid; e < TT * d; e += 256) {
      const int i = e % d, t = e / d;
      float kk = 0.f, vv = 0.f;
      if (n0 + t < n_end) {
        const long long off = base + (long long)(n0 + t) * kv.ld + i;
        kk = fmaxf(to_f32(k[off]), 0.f);
        vv = to_f32(v[off]);
      }
      ks[t][i] = kk;
      vs[t][i] = vv;
    }
    for (int t = tid; t < TT; t += 256) vs[t][d] = 1.f;  // the ones column gives sum relu(k)
    __syncthreads();
#pragma unroll
    for (int i = 0; i < EPT; ++i)
      for (int t = 0; t < TT; ++t) acc[i] = fmaf(ks[t][ea[i]], vs[t][ec[i]], acc[i]);
    __syncthreads();
  }
  float* out = partial + ((long long)bh * S + s) * ne;
#pragma unroll
  for (int i = 0; i < EPT; ++i) {
    const int e = tid + i * 256;
    if (e < ne) out[e] = acc[i];
  }
}

// Second level: state[bh][e] = partial[bh][0][e] + partial[bh][1][e] + ... in
// index order, so the result does not depend on scheduling.
__global__ void __launch_bounds__(256)
kv_combine_kernel(const float* __restrict__ partial, float* __restrict__ state, int S, int ne,
                  long long total) {
  const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
  if (idx >= total) return;
  const long long bh = idx / ne;
  const int e = (int)(idx % ne);
  const float* p = partial + bh * S * ne + e;
  float acc = 0.f;
  for (int s = 0; s < S; ++s) acc += p[(long long)s * ne];
  state[idx] = acc;
}

// Token-sharded forward: state[i] = states[0][i] + states[1][i] + ... over the R bands of the image in band
// order (Eq. 3's sums over tokens, cut into bands), the same order on every rank.
__global__ void __launch_bounds__(256)
band_state_sum_kernel(const float* __restrict__ states, float* __restrict__ state, int R, long long total) {
  const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
  if (idx >= total) return;
  float acc = 0.f;
  for (int r = 0; r < R; ++r) acc += states[(long long)r * total + idx];
  state[idx] = acc;
}

// ---------------------------------------------------------------------------
// Apply step (Eq. 3): out[i,c] = relu(q[i]) . KV[:,c] / (relu(q[i]) . ks + eps),
// written at channel offset head*d of the output view (head concat).
// One thread per token; state [BH][d*(d+1)] fp32 staged in shared memory.
// ---------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(128)
apply_kernel(const T* __restrict__ q, const float* __restrict__ state, T* __restrict__ out,
             HeadView qv, HeadView ov, int heads, int N, int d, float eps) {
  constexpr int DMAX = 32;
  __shared__ float st[DMAX * (DMAX + 1)];
  const int bh = blockIdx.y;
  const int b = bh / heads, h = bh % heads;
  const int d1 = d + 1;
  for (int e = threadIdx.x; e < d * d1; e += 128) st[e] = state[(long long)bh * d * d1 + e];
  __syncthreads();
  const int n = blockIdx.x * 128 + threadIdx.x;
  if (n >= N) return;
  const T* qp = q + (long long)b * qv.batch + (long long)h * qv.head + (long long)n * qv.ld;
  T* op = out + (long long)b * ov.batch + (long long)h * ov.head + (long long)n * ov.ld;
  float qr[DMAX];
#pragma unroll
  for (int a = 0; a < DMAX; ++a) qr[a] = a < d ? fmaxf(to_f32(qp[a]), 0.f) : 0.f;
  float den = 0.f;
#pragma unroll
  for (int a = 0; a < DMAX; ++a)
    if (a < d) den = fmaf(qr[a], st[a * d1 + d], den);
  const float inv = 1.f / (den + eps);
  for (int c = 0; c < d; ++c) {
    float num = 0.f;
#pragma unroll
    for (int a = 0; a < DMAX; ++a)
      if (a < d) num = fmaf(qr[a], st[a * d1 + c], num);
    op[c] = from_f32<T>(num * inv);
  }
}

}  // namespace generic
}  // namespace msla
