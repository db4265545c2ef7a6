// Tuned 16-bit (bf16, and fp16) attention core (Eq. 3): KV-state reduction and apply step on
// warp-level tensor-core MMAs with fp32 accumulation.
//
// Both steps are HBM-bound only if their small contractions (d x (d+1) per
// token) stay off the plain fp32 pipes, so each warp feeds mma.sync.m16n8k16
// from data that cp.async streams through per-warp shared-memory rings (bytes
// in flight independent of registers and occupancy).  The freedom used to
// avoid data shuffling: the contraction index of an MMA may be assigned to
// tokens (reduction) or channels (apply) in any order, as long as both
// operands use the same assignment; where a transpose is unavoidable (tokens
// along the contraction, rows of channels in memory) ldmatrix.trans does it.
#include "msla_common.cuh"
#include "msla_host.h"

namespace msla {
namespace {

using bf16 = __nv_bfloat16;

// F16 selects the 16-bit storage type of the operands: IEEE binary16 instead of bfloat16.  Accumulators are fp32 in both.
template <bool F16>
__device__ __forceinline__ void mma16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  if constexpr (F16)
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
  else
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <bool F16>
__device__ __forceinline__ uint32_t relu2(uint32_t x) {  // packed max(x, 0) on two 16-bit values
  uint32_t r;
  if constexpr (F16) asm("max.f16x2 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(0u));
  else asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(x), "r"(0u));
  return r;
}


__device__ __forceinline__ void stg(void* p, const uint32_t (&r)[2]) {
  asm volatile("st.global.v2.u32 [%0], {%1,%2};" ::"l"(p), "r"(r[0]), "r"(r[1]) : "memory");
}
__device__ __forceinline__ void stg(void* p, const uint32_t (&r)[4]) {
  asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}

template <bool F16>
__device__ __forceinline__ uint32_t pack16(float lo, float hi) {
  uint32_t r;
  if constexpr (F16) asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  else asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
// v rounded to the 16-bit type and widened again
template <bool F16>
__device__ __forceinline__ float round16(float v) {
  if constexpr (F16) return __half2float(__float2half_rn(v));
  else return __bfloat162float(__float2bfloat16_rn(v));
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// 16-byte asynchronous global->shared copy; src_bytes = 0 writes zeros instead.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void lds128(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void lds64(uint32_t (&r)[2], uint32_t addr) {
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}

// ---------------------------------------------------------------------------
// KV-state reduction, first level.  One CTA = one (batch, head, token chunk).
//
// MMA view: state[a][c] += sum over 16 tokens of relu(k[n][a]) * v[n][c],
// A = relu(K)^T (rows = channel a, contraction = token), B = [V | 1].
//
// Every warp runs its own STAGES-deep ring of cp.async groups: a stage holds TS
// tokens of K and of V as [token][channel] rows in shared memory (16-byte
// chunks XOR-swizzled by row so that ldmatrix is bank-conflict free).  Both
// operands want the token index along the contraction, i.e. the transpose of
// how the rows lie in memory, which is exactly ldmatrix.trans.  Memory latency
// is covered by the ring (bytes in flight do not depend on registers or
// occupancy); no block-wide barrier is taken inside the loop.  An extra B tile
// of bf16 ones yields sum relu(k).
// ---------------------------------------------------------------------------
template <int D, int NWARPS, int STAGES, bool F16>
__global__ void __launch_bounds__(NWARPS * 32)
kv_state_mma_kernel(const bf16* __restrict__ k, const bf16* __restrict__ v, float* __restrict__ partial,
                    HeadView kv, int heads, int N, int S, int chunk) {
  constexpr int TS = 32;            // tokens per stage
  constexpr int MT = D / 16;        // A tiles (16 channels each)
  constexpr int NT = D / 8;         // B tiles (8 channels each), + 1 tile of ones
  constexpr int CH = D / 8;         // 16-byte chunks per token row
  constexpr int ROWB = D * 2;       // bytes per token row
  constexpr int TILEB = TS * ROWB;  // bytes of one K (or V) tile
  constexpr int SW_SHIFT = CH == 4 ? 1 : 2;
  constexpr int NE = D * (D + 1);
  constexpr int CPL = TS * CH / 32;  // cp.async per lane per tile
  constexpr int RPI = 32 / CH;       // token rows covered by one warp-wide cp.async
  extern __shared__ __align__(128) unsigned char smem[];
  static_assert(NWARPS * STAGES * 2 * TILEB >= NWARPS * NE * 4, "reduction buffer must fit in the stage ring");

  pdl_launch_dependents();
  pdl_wait();  // k and v come from the previous kernel
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int bh = blockIdx.x, s = blockIdx.y;
  const int b = bh / heads, h = bh % heads;
  const long long base = (long long)b * kv.batch + (long long)h * kv.head;
  const int n_begin = s * chunk;
  const int n_end = min(N, n_begin + chunk);
  const int groups = (n_end - n_begin + TS - 1) / TS;           // TS-token groups in this chunk
  const int my_groups = groups > warp ? (groups - warp + NWARPS - 1) / NWARPS : 0;

  const uint32_t ring = smem_u32(smem) + warp * (STAGES * 2 * TILEB);
  // this lane's slot in a warp-wide copy: row r_cp (+ RPI per copy), chunk c_cp
  const int r_cp = lane / CH, c_cp = lane % CH;
  const bf16* ksrc = k + base + c_cp * 8;
  const bf16* vsrc = v + base + c_cp * 8;

  auto issue = [&](int it) {  // it-th group of this warp -> stage it % STAGES
    const uint32_t dstK = ring + (it % STAGES) * (2 * TILEB), dstV = dstK + TILEB;
    const int n0 = n_begin + (warp + it * NWARPS) * TS;
#pragma unroll
    for (int i = 0; i < CPL; ++i) {
      const int r = r_cp + i * RPI;
      const int n = n0 + r;
      const bool ok = n < n_end;
      const long long off = (long long)(ok ? n : n_begin) * kv.ld;
      const uint32_t d = r * ROWB + ((c_cp ^ ((r >> SW_SHIFT) & (CH - 1))) << 4);
      cp_async16(dstK + d, ksrc + off, ok ? 16 : 0);
      cp_async16(dstV + d, vsrc + off, ok ? 16 : 0);
    }
  };

  float acc[MT][NT + 1][4];
#pragma unroll
  for (int i = 0; i < MT; ++i)
#pragma unroll
    for (int j = 0; j <= NT; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.f;

#pragma unroll
  for (int p = 0; p < STAGES - 1; ++p) {
    if (p < my_groups) issue(p);
    cp_async_commit();
  }
  // ldmatrix row address pieces for this lane: matrix m = lane/8, row lane%8
  const int lm = lane >> 3, lr = lane & 7;
  for (int it = 0; it < my_groups; ++it) {
    if (it + STAGES - 1 < my_groups) issue(it + STAGES - 1);
    cp_async_commit();
    cp_async_wait<STAGES - 1>();
    __syncwarp();
    const uint32_t tK = ring + (it % STAGES) * (2 * TILEB), tV = tK + TILEB;
#pragma unroll
    for (int ks = 0; ks < TS / 16; ++ks) {
      uint32_t A[MT][4], Bt[NT][2];
#pragma unroll
      for (int i = 0; i < MT; ++i) {
        // matrices: (tok 0-7, ch chunk 2i) (tok 0-7, chunk 2i+1) (tok 8-15, chunk 2i) (tok 8-15, chunk 2i+1)
        const int r = ks * 16 + lr + ((lm >> 1) << 3);
        const int c = 2 * i + (lm & 1);
        ldsm_x4_trans(A[i], tK + r * ROWB + ((c ^ ((r >> SW_SHIFT) & (CH - 1))) << 4));
#pragma unroll
        for (int e = 0; e < 4; ++e) A[i][e] = relu2<F16>(A[i][e]);
      }
#pragma unroll
      for (int j = 0; j < NT; j += 2) {
        // matrices: (tok 0-7, chunk j) (tok 8-15, chunk j) (tok 0-7, chunk j+1) (tok 8-15, chunk j+1)
        const int r = ks * 16 + lr + ((lm & 1) << 3);
        const int c = j + (lm >> 1);
        uint32_t x[4];
        ldsm_x4_trans(x, tV + r * ROWB + ((c ^ ((r >> SW_SHIFT) & (CH - 1))) << 4));
        Bt[j][0] = x[0]; Bt[j][1] = x[1]; Bt[j + 1][0] = x[2]; Bt[j + 1][1] = x[3];
      }
#pragma unroll
      for (int i = 0; i < MT; ++i) {
#pragma unroll
        for (int j = 0; j < NT; ++j) mma16<F16>(acc[i][j], A[i], Bt[j][0], Bt[j][1]);
        mma16<F16>(acc[i][NT], A[i], F16 ? 0x3C003C00u : 0x3F803F80u, F16 ? 0x3C003C00u : 0x3F803F80u);  // ones
      }
    }
    __syncwarp();  // all lanes done with this stage before a later issue() overwrites it
  }
  cp_async_wait<0>();
  __syncthreads();  // every warp has left its ring: reuse it for the reduction

  // fixed-order combine of the warps' accumulators (level one of two)
  float* red = reinterpret_cast<float*>(smem);
#pragma unroll
  for (int i = 0; i < MT; ++i)
#pragma unroll
    for (int j = 0; j <= NT; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int a = 16 * i + g + 8 * (e >> 1);
        const int col = 2 * t + (e & 1);
        if (j < NT) red[warp * NE + a * (D + 1) + 8 * j + col] = acc[i][j][e];
        else if (col == 0) red[warp * NE + a * (D + 1) + D] = acc[i][j][e];
      }
  __syncthreads();
  float* out = partial + ((long long)bh * S + s) * NE;
  for (int e = threadIdx.x; e < NE; e += NWARPS * 32) {
    float sum = red[e];
#pragma unroll
    for (int w = 1; w < NWARPS; ++w) sum += red[w * NE + e];
    out[e] = sum;
  }
}

// Level two: state[bh][e] = partial[bh][0][e] + partial[bh][1][e] + ... in index order.
__global__ void __launch_bounds__(256)
kv_combine_bf16path_kernel(const float* __restrict__ partial, float* __restrict__ state, int S, int ne, long long total) {
  pdl_launch_dependents();
  pdl_wait();
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
// PAIR: one CTA serves heads 2p (even warps) and 2p+1 (odd warps) of a paired
// output view, so that the two 64-byte halves of each 128-byte output row are
// written at nearly the same time.
// state_scale: the state (numerator and denominator columns alike) and eps are multiplied by it before they are cut
// into 16-bit pieces; the quotient of Eq. 3 does not change.  1 for bf16 (its exponent range is fp32's); for fp16 a
// power of two near 1/N, so that sums over N tokens fit the format.
template <int D, int NWARPS, int STAGES, int U, bool PAIR, bool F16>
__global__ void __launch_bounds__(NWARPS * 32)
apply_mma_kernel(const bf16* __restrict__ q, const float* __restrict__ state, bf16* __restrict__ out,
                 HeadView qv, HeadView ov, int heads, int N, float eps, int tok_per_cta, float state_scale) {
  constexpr int KS = D / 16;   // MMA steps over the channel contraction
  constexpr int NT = D / 8;    // output tiles, + 1 for the denominator
  constexpr int CPT = D / 4;   // channels per lane per token
  constexpr int WQ = D / 8;    // 32-bit words per lane per token
  constexpr int LB = CPT * 2;  // bytes per lane per token (16 or 8)
  constexpr int STAGEB = U * 2 * 32 * LB;
  // Each lane streams its own query bytes through a private FIFO in shared
  // memory (cp.async in, plain load out), so loads run STAGES groups ahead of
  // the MMAs without holding registers and without any cross-lane hand-off.
  __shared__ __align__(16) unsigned char fifo[NWARPS * STAGES * STAGEB];
  pdl_launch_dependents();
  pdl_wait();  // the state comes from the previous kernel
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  constexpr int NW = PAIR ? NWARPS / 2 : NWARPS;  // warps sharing one head's tokens
  const int wslot = PAIR ? warp >> 1 : warp;
  const int bh = PAIR ? 2 * blockIdx.y + (warp & 1) : blockIdx.y;
  const int b = bh / heads, h = bh % heads;
  const long long qbase = (long long)b * qv.batch + (long long)h * qv.head + t * CPT;
  const long long obase = PAIR ? (long long)b * ov.batch + (long long)(h >> 1) * ov.head + (h & 1) * D + t * CPT
                               : (long long)b * ov.batch + (long long)h * ov.head + t * CPT;
  const int n_begin = blockIdx.x * tok_per_cta;
  const int n_end = min(N, n_begin + tok_per_cta);
  constexpr int TS = 16 * U;
  const int groups = (n_end - n_begin + TS - 1) / TS;
  const int my_groups = groups > wslot ? (groups - wslot + NW - 1) / NW : 0;
  const uint32_t ring = smem_u32(fifo) + warp * (STAGES * STAGEB) + lane * LB;

  auto issue = [&](int it) {
    const uint32_t dst = ring + (it % STAGES) * STAGEB;
    const int n0 = n_begin + (wslot + it * NW) * TS + g;
#pragma unroll
    for (int u = 0; u < 2 * U; ++u) {  // u even: token g of tile u/2, odd: token g+8
      const int n = n0 + u * 8;
      const bool ok = n < n_end;
      const bf16* src = q + qbase + (long long)(ok ? n : n_begin) * qv.ld;
      if constexpr (LB == 16)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + u * 32 * LB), "l"(src), "r"(ok ? 16 : 0) : "memory");
      else
        asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst + u * 32 * LB), "l"(src), "r"(ok ? 8 : 0) : "memory");
    }
  };
#pragma unroll
  for (int p = 0; p < STAGES - 1; ++p) {
    if (p < my_groups) issue(p);
    cp_async_commit();
  }

  // state -> B fragments (bf16 hi + lo), overlapping the first copies
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
          const float v0 = st[a0 * (D + 1) + c] * state_scale, v1 = st[(a0 + 1) * (D + 1) + c] * state_scale;
          bhi[ks][j][r] = pack16<F16>(v0, v1);
          blo[ks][j][r] = pack16<F16>(v0 - round16<F16>(v0), v1 - round16<F16>(v1));
        }
  }

  for (int it = 0; it < my_groups; ++it) {
    if (it + STAGES - 1 < my_groups) issue(it + STAGES - 1);
    cp_async_commit();
    cp_async_wait<STAGES - 1>();
    const uint32_t src = ring + (it % STAGES) * STAGEB;
    const int n0 = n_begin + (wslot + it * NW) * TS;
    uint32_t qa[U][WQ], qb[U][WQ];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if constexpr (LB == 16) {
        lds128(qa[u], src + (2 * u) * 32 * LB);
        lds128(qb[u], src + (2 * u + 1) * 32 * LB);
      } else {
        lds64(qa[u], src + (2 * u) * 32 * LB);
        lds64(qb[u], src + (2 * u + 1) * 32 * LB);
      }
    }
    float acc[U][NT + 1][4];
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int j = 0; j <= NT; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[u][j][e] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      uint32_t A[U][4];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        A[u][0] = relu2<F16>(qa[u][2 * ks]); A[u][1] = relu2<F16>(qb[u][2 * ks]);
        A[u][2] = relu2<F16>(qa[u][2 * ks + 1]); A[u][3] = relu2<F16>(qb[u][2 * ks + 1]);
      }
#pragma unroll
      for (int j = 0; j <= NT; ++j)
#pragma unroll
        for (int u = 0; u < U; ++u) mma16<F16>(acc[u][j], A[u], bhi[ks][j][0], bhi[ks][j][1]);
#pragma unroll
      for (int j = 0; j <= NT; ++j)
#pragma unroll
        for (int u = 0; u < U; ++u) mma16<F16>(acc[u][j], A[u], blo[ks][j][0], blo[ks][j][1]);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const float inv_a = 1.f / (acc[u][NT][0] + eps), inv_b = 1.f / (acc[u][NT][2] + eps);
      uint32_t oa[WQ], ob[WQ];
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        oa[j] = pack16<F16>(acc[u][j][0] * inv_a, acc[u][j][1] * inv_a);
        ob[j] = pack16<F16>(acc[u][j][2] * inv_b, acc[u][j][3] * inv_b);
      }
      const int na = n0 + u * 16 + g, nb = na + 8;
      if (na < n_end) stg(out + obase + (long long)na * ov.ld, oa);
      if (nb < n_end) stg(out + obase + (long long)nb * ov.ld, ob);
    }
  }
  cp_async_wait<0>();
}

template <int D, bool F16>
msla_status_t launch_core(const bf16* q, const bf16* k, const bf16* v, bf16* out, HeadView in, HeadView ov, int B,
                          int heads, int N, float eps, const CorePlan& p, char* ws, cudaStream_t st, cudaEvent_t mid, int phases) {
  // 4 warps per CTA and 4-deep rings in both kernels; two 16-token MMA tiles per FIFO stage of the apply step
  constexpr int KV_WARPS = 4, KV_STAGES = 4, AP_WARPS = 4, AP_STAGES = 4, AP_U = 2;
  const long long BH = (long long)B * heads;
  float* partial = reinterpret_cast<float*>(ws + p.partial_off);
  float* state = reinterpret_cast<float*>(ws + p.state_off);
  constexpr int kv_smem = KV_WARPS * KV_STAGES * 2 * 32 * D * 2;
  static std::atomic<unsigned long long> attr_done{0};
  const msla_status_t as = ensure_smem_attr(attr_done, kv_state_mma_kernel<D, KV_WARPS, KV_STAGES, F16>, kv_smem);
  if (as != MSLA_OK) return as;
  int launches = 0;
  if (phases & CORE_STATE) {
    launch_pdl(kv_state_mma_kernel<D, KV_WARPS, KV_STAGES, F16>, dim3((unsigned)BH, p.S), dim3(KV_WARPS * 32), kv_smem, st, k, v, partial, in, heads, N, p.S, p.chunk);
    ++launches;
  }
  if (phases & CORE_COMBINE) {
    const long long total = BH * p.ne;
    launch_pdl(kv_combine_bf16path_kernel, dim3((unsigned)ceil_div_ll(total, 256)), dim3(256), 0, st, partial, state, p.S, p.ne, total);
    ++launches;
  }
  if (mid) cudaEventRecord(mid, st);
  if (phases & CORE_APPLY) {
    // fp16 pieces of the state must fit the format: a sum over N tokens is scaled by the power of two just above 1/N
    float state_scale = 1.f;
    if (F16) for (long long n = 1; n < N; n *= 2) state_scale *= 0.5f;
    eps *= state_scale;
    if (ov.pair) {  // heads is even here, so a pair never straddles two images
      const int tok_per_cta = p.apply_tokens / 2;
      launch_pdl(apply_mma_kernel<D, AP_WARPS, AP_STAGES, AP_U, true, F16>, dim3((unsigned)ceil_div_ll(N, tok_per_cta), (unsigned)(BH / 2)),
                 dim3(AP_WARPS * 32), 0, st, q, state, out, in, ov, heads, N, eps, tok_per_cta, state_scale);
    } else {
      const int tok_per_cta = p.apply_tokens;
      launch_pdl(apply_mma_kernel<D, AP_WARPS, AP_STAGES, AP_U, false, F16>, dim3((unsigned)ceil_div_ll(N, tok_per_cta), (unsigned)BH),
                 dim3(AP_WARPS * 32), 0, st, q, state, out, in, ov, heads, N, eps, tok_per_cta, state_scale);
    }
    ++launches;
  }
  count_launches(launches);
  return check_launch(F16 ? "attention core kernels (fp16)" : "attention core kernels (bf16)");
}

}  // namespace

msla_status_t run_core_bf16(const void* q, const void* k, const void* v, void* out, HeadView in, HeadView ov, int B,
                            int heads, int N, int d, float eps, const CorePlan& p, void* ws, cudaStream_t st,
                            cudaEvent_t mid, int phases, bool f16) {
  // the kernels move 16-bit values untyped; only the MMA, ReLU and conversion instructions depend on the format
  const bf16 *q16 = (const bf16*)q, *k16 = (const bf16*)k, *v16 = (const bf16*)v;
  if (f16) {
    if (d == 32) return launch_core<32, true>(q16, k16, v16, (bf16*)out, in, ov, B, heads, N, eps, p, (char*)ws, st, mid, phases);
    return launch_core<16, true>(q16, k16, v16, (bf16*)out, in, ov, B, heads, N, eps, p, (char*)ws, st, mid, phases);
  }
  if (d == 32) return launch_core<32, false>(q16, k16, v16, (bf16*)out, in, ov, B, heads, N, eps, p, (char*)ws, st, mid, phases);
  return launch_core<16, false>(q16, k16, v16, (bf16*)out, in, ov, B, heads, N, eps, p, (char*)ws, st, mid, phases);
}

}  // namespace msla
