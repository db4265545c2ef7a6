// Tuned bf16 attention core (Eq. 3): KV-state reduction and apply step on
// warp-level tensor-core MMAs with fp32 accumulation.
//
// Both steps are HBM-bound only if their small contractions (d x (d+1) per
// token) stay off the plain fp32 pipes, so each warp feeds mma.sync.m16n8k16
// directly from registers filled by vectorised global loads.  The freedom that
// makes this work without any shared-memory transpose: the contraction index
// of an MMA may be assigned to tokens (reduction) or channels (apply) in any
// order, as long as both operands use the same assignment.
#include "msla_common.cuh"
#include "msla_host.h"

// Launch shapes (overridable at build time for tuning sweeps).
#ifndef MSLA_KV_WARPS
#define MSLA_KV_WARPS 8
#endif
#ifndef MSLA_KV_U
#define MSLA_KV_U 4
#endif
#ifndef MSLA_AP_WARPS
#define MSLA_AP_WARPS 4
#endif
#ifndef MSLA_AP_U
#define MSLA_AP_U 4
#endif

namespace msla {
namespace {

using bf16 = __nv_bfloat16;

__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t relu2(uint32_t x) {  // packed bf16x2 max(x, 0)
  uint32_t r;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(0u));
  return r;
}

__device__ __forceinline__ uint32_t lo_pair(uint32_t a, uint32_t b) { return __byte_perm(a, b, 0x5410); }
__device__ __forceinline__ uint32_t hi_pair(uint32_t a, uint32_t b) { return __byte_perm(a, b, 0x7632); }

// Streaming loads: every byte is used once, keep it out of L1.
__device__ __forceinline__ void ldg_stream(const void* p, uint32_t (&r)[1]) {
  asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(r[0]) : "l"(p));
}
__device__ __forceinline__ void ldg_stream(const void* p, uint32_t (&r)[2]) {
  asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "l"(p));
}
__device__ __forceinline__ void ldg_stream(const void* p, uint32_t (&r)[4]) {
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "l"(p));
}
__device__ __forceinline__ void stg(void* p, const uint32_t (&r)[2]) {
  asm volatile("st.global.v2.u32 [%0], {%1,%2};" ::"l"(p), "r"(r[0]), "r"(r[1]) : "memory");
}
__device__ __forceinline__ void stg(void* p, const uint32_t (&r)[4]) {
  asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// ---------------------------------------------------------------------------
// KV-state reduction, first level.  One CTA = one (batch, head, token chunk);
// each warp owns 16-token MMA steps, U of them per loop trip.
//
// MMA view: state[a][c] += sum over 16 tokens of relu(k[n][a]) * v[n][c],
// A = relu(K)^T (rows = channel a, contraction = token), B = [V | 1].
// Lane (g = lane/4, t = lane%4) loads, for the four tokens {t, t+4, t+8, t+12}
// of a step, the D/8 consecutive channels starting at g*D/8 of K and of V
// (8 bytes for D = 32).  Those tokens sit in contraction slots {2t, 2t+1,
// 2t+8, 2t+9}: exactly the slots this lane must supply for both operands.
// Word w of a load holds channels (2w, 2w+1) of the lane's group:
//   A tile w   : row g = channel g*D/8 + 2w, row g+8 = channel g*D/8 + 2w + 1
//   B tile 2w+p: column g = channel g*D/8 + 2w + p
// An extra B tile of ones yields sum relu(k).
// ---------------------------------------------------------------------------
template <int D, int NWARPS, int U>
__global__ void __launch_bounds__(NWARPS * 32)
kv_state_mma_kernel(const bf16* __restrict__ k, const bf16* __restrict__ v, float* __restrict__ partial,
                    HeadView kv, int heads, int N, int S, int chunk) {
  constexpr int W = D / 16;   // 32-bit words per lane per token
  constexpr int MT = D / 16;  // A tiles (16 channels each)
  constexpr int NT = D / 8;   // B tiles (8 channels each), + 1 tile of ones
  constexpr int CG = D / 8;   // channels per lane group
  constexpr int NE = D * (D + 1);
  __shared__ float red[NWARPS][NE];

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int bh = blockIdx.x, s = blockIdx.y;
  const int b = bh / heads, h = bh % heads;
  const long long base = (long long)b * kv.batch + (long long)h * kv.head + g * CG;
  const int n_begin = s * chunk;
  const int n_end = min(N, n_begin + chunk);

  float acc[MT][NT + 1][4];
#pragma unroll
  for (int i = 0; i < MT; ++i)
#pragma unroll
    for (int j = 0; j <= NT; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.f;

  for (int n0 = n_begin + warp * (16 * U); n0 < n_end; n0 += NWARPS * 16 * U) {
    uint32_t kr[U][4][W], vr[U][4][W];
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int n = n0 + u * 16 + t + 4 * j;
        if (n < n_end) {
          const long long off = base + (long long)n * kv.ld;
          ldg_stream(k + off, kr[u][j]);
          ldg_stream(v + off, vr[u][j]);
        } else {
#pragma unroll
          for (int w = 0; w < W; ++w) kr[u][j][w] = vr[u][j][w] = 0u;
        }
      }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      uint32_t A[MT][4], Bt[NT][2];
#pragma unroll
      for (int w = 0; w < W; ++w) {
        const uint32_t k0 = relu2(kr[u][0][w]), k1 = relu2(kr[u][1][w]);
        const uint32_t k2 = relu2(kr[u][2][w]), k3 = relu2(kr[u][3][w]);
        A[w][0] = lo_pair(k0, k1); A[w][1] = hi_pair(k0, k1);
        A[w][2] = lo_pair(k2, k3); A[w][3] = hi_pair(k2, k3);
        Bt[2 * w][0] = lo_pair(vr[u][0][w], vr[u][1][w]);
        Bt[2 * w][1] = lo_pair(vr[u][2][w], vr[u][3][w]);
        Bt[2 * w + 1][0] = hi_pair(vr[u][0][w], vr[u][1][w]);
        Bt[2 * w + 1][1] = hi_pair(vr[u][2][w], vr[u][3][w]);
      }
#pragma unroll
      for (int i = 0; i < MT; ++i) {
#pragma unroll
        for (int j = 0; j < NT; ++j) mma_bf16(acc[i][j], A[i], Bt[j][0], Bt[j][1]);
        mma_bf16(acc[i][NT], A[i], 0x3F803F80u, 0x3F803F80u);  // bf16 ones
      }
    }
  }

  // fixed-order combine of the warps' accumulators (level one of two)
#pragma unroll
  for (int i = 0; i < MT; ++i)
#pragma unroll
    for (int j = 0; j <= NT; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int a = g * CG + 2 * i + (e >> 1);
        const int col = 2 * t + (e & 1);
        if (j < NT) red[warp][a * (D + 1) + col * CG + j] = acc[i][j][e];
        else if (col == 0) red[warp][a * (D + 1) + D] = acc[i][j][e];
      }
  __syncthreads();
  float* out = partial + ((long long)bh * S + s) * NE;
  for (int e = threadIdx.x; e < NE; e += NWARPS * 32) {
    float sum = red[0][e];
#pragma unroll
    for (int w = 1; w < NWARPS; ++w) sum += red[w][e];
    out[e] = sum;
  }
}

// Level two: state[bh][e] = partial[bh][0][e] + partial[bh][1][e] + ... in index order.
__global__ void __launch_bounds__(256)
kv_combine_bf16path_kernel(const float* __restrict__ partial, float* __restrict__ state, int S, int ne, long long total) {
  const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
  if (idx >= total) return;
  const long long bh = idx / ne;
  const int e = (int)(idx % ne);
  const float* p = partial + bh * S * ne + e;
  float acc = 0.f;
  for (int s = 0; s < S; ++s) acc += p[(long long)s * ne];
  state[idx] = acc;
}

// ---------------------------------------------------------------------------
// Apply step with the normaliser and the head concat fused.
//
// MMA view: [num | den][n][c] = sum_a relu(q[n][a]) * [KV | ks][a][c],
// A = relu(Q) (rows = 16 tokens, contraction = channel), B = state.
// Lane (g, t) loads D/4 consecutive channels starting at t*D/4 of tokens g and
// g+8 (16 bytes each for D = 32); these fill contraction slots {2t, 2t+1, 2t+8,
// 2t+9} of D/16 MMA steps with no data movement.  Output tile j gives the lane
// columns (2t, 2t+1), mapped to channels t*D/4 + 2j + {0,1}, so a lane ends up
// with the same D/4 consecutive channels of its two tokens and stores 16 bytes.
// The fp32 state is fed as bf16 hi + bf16 lo (two MMAs) to keep ~16 mantissa
// bits; one extra tile whose columns all hold ks gives the denominator.
// ---------------------------------------------------------------------------
template <int D, int NWARPS, int U>
__global__ void __launch_bounds__(NWARPS * 32)
apply_mma_kernel(const bf16* __restrict__ q, const float* __restrict__ state, bf16* __restrict__ out,
                 HeadView qv, HeadView ov, int heads, int N, float eps, int tok_per_cta) {
  constexpr int KS = D / 16;  // MMA steps over the channel contraction
  constexpr int NT = D / 8;   // output tiles, + 1 for the denominator
  constexpr int CPT = D / 4;  // channels per lane per token
  constexpr int WQ = D / 8;   // 32-bit words per lane per token
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int bh = blockIdx.y;
  const int b = bh / heads, h = bh % heads;

  uint32_t bhi[KS][NT + 1][2], blo[KS][NT + 1][2];
  {
    const float* st = state + (long long)bh * D * (D + 1);
#pragma unroll
    for (int ks = 0; ks < KS; ++ks)
#pragma unroll
      for (int j = 0; j <= NT; ++j)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          const int a0 = CPT * t + 4 * ks + 2 * r;
          const int c = j < NT ? (g >> 1) * CPT + 2 * j + (g & 1) : D;
          const float v0 = st[a0 * (D + 1) + c], v1 = st[(a0 + 1) * (D + 1) + c];
          const bf16 h0 = __float2bfloat16_rn(v0), h1 = __float2bfloat16_rn(v1);
          bhi[ks][j][r] = pack_bf16(v0, v1);
          blo[ks][j][r] = pack_bf16(v0 - __bfloat162float(h0), v1 - __bfloat162float(h1));
        }
  }

  const long long qbase = (long long)b * qv.batch + (long long)h * qv.head + t * CPT;
  const long long obase = (long long)b * ov.batch + (long long)h * ov.head + t * CPT;
  const int n_begin = blockIdx.x * tok_per_cta;
  const int n_end = min(N, n_begin + tok_per_cta);

  for (int n0 = n_begin + warp * (16 * U); n0 < n_end; n0 += NWARPS * 16 * U) {
    uint32_t qa[U][WQ], qb[U][WQ];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int na = n0 + u * 16 + g, nb = na + 8;
      if (na < n_end) ldg_stream(q + qbase + (long long)na * qv.ld, qa[u]);
      else {
#pragma unroll
        for (int w = 0; w < WQ; ++w) qa[u][w] = 0u;
      }
      if (nb < n_end) ldg_stream(q + qbase + (long long)nb * qv.ld, qb[u]);
      else {
#pragma unroll
        for (int w = 0; w < WQ; ++w) qb[u][w] = 0u;
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float acc[NT + 1][4];
#pragma unroll
      for (int j = 0; j <= NT; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[j][e] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const uint32_t A[4] = {relu2(qa[u][2 * ks]), relu2(qb[u][2 * ks]), relu2(qa[u][2 * ks + 1]), relu2(qb[u][2 * ks + 1])};
#pragma unroll
        for (int j = 0; j <= NT; ++j) {
          mma_bf16(acc[j], A, bhi[ks][j][0], bhi[ks][j][1]);
          mma_bf16(acc[j], A, blo[ks][j][0], blo[ks][j][1]);
        }
      }
      const float inv_a = 1.f / (acc[NT][0] + eps), inv_b = 1.f / (acc[NT][2] + eps);
      uint32_t oa[WQ], ob[WQ];
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        oa[j] = pack_bf16(acc[j][0] * inv_a, acc[j][1] * inv_a);
        ob[j] = pack_bf16(acc[j][2] * inv_b, acc[j][3] * inv_b);
      }
      const int na = n0 + u * 16 + g, nb = na + 8;
      if (na < n_end) stg(out + obase + (long long)na * ov.ld, oa);
      if (nb < n_end) stg(out + obase + (long long)nb * ov.ld, ob);
    }
  }
}

template <int D>
msla_status_t launch_core(const bf16* q, const bf16* k, const bf16* v, bf16* out, HeadView in, HeadView ov, int B,
                          int heads, int N, float eps, const CorePlan& p, char* ws, cudaStream_t st, cudaEvent_t mid) {
  constexpr int KV_WARPS = MSLA_KV_WARPS, KV_U = MSLA_KV_U, AP_WARPS = MSLA_AP_WARPS, AP_U = MSLA_AP_U;
  const long long BH = (long long)B * heads;
  float* partial = reinterpret_cast<float*>(ws + p.partial_off);
  float* state = reinterpret_cast<float*>(ws + p.state_off);
  kv_state_mma_kernel<D, KV_WARPS, KV_U><<<dim3((unsigned)BH, p.S), KV_WARPS * 32, 0, st>>>(k, v, partial, in, heads, N, p.S, p.chunk);
  const long long total = BH * p.ne;
  kv_combine_bf16path_kernel<<<(unsigned)ceil_div_ll(total, 256), 256, 0, st>>>(partial, state, p.S, p.ne, total);
  if (mid) cudaEventRecord(mid, st);
  const int tok_per_cta = p.apply_tokens;
  apply_mma_kernel<D, AP_WARPS, AP_U><<<dim3((unsigned)ceil_div_ll(N, tok_per_cta), (unsigned)BH), AP_WARPS * 32, 0, st>>>(
      q, state, out, in, ov, heads, N, eps, tok_per_cta);
  count_launches(3);
  return check_launch("attention core kernels (bf16)");
}

}  // namespace

msla_status_t run_core_bf16(const void* q, const void* k, const void* v, void* out, HeadView in, HeadView ov, int B,
                            int heads, int N, int d, float eps, const CorePlan& p, void* ws, cudaStream_t st,
                            cudaEvent_t mid) {
  if (d == 32)
    return launch_core<32>((const bf16*)q, (const bf16*)k, (const bf16*)v, (bf16*)out, in, ov, B, heads, N, eps, p, (char*)ws, st, mid);
  return launch_core<16>((const bf16*)q, (const bf16*)k, (const bf16*)v, (bf16*)out, in, ov, B, heads, N, eps, p, (char*)ws, st, mid);
}

}  // namespace msla
