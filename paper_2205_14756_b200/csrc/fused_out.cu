// Steps 4 and 5 of the module (Section 3.1: apply step of Eq. 3, head concat,
// final linear projection) as one tensor-core GEMM per image.
//
// Eq. 3 gives, for head h and token n,  O_h[n][c] = sum_a relu(q_h[n][a]) S_h[a][c] / den_h[n]
// with den_h[n] = sum_a relu(q_h[n][a]) ks_h[a] + eps, and the projection is
// y[m][n] = sum_h sum_c w[m][h*d + c] O_h[n][c] + bias[m].  Re-associating the two sums,
//
//   y[m][n] = sum_h sum_a  M[m][h*d + a] * qt[h*d + a][n]  + bias[m],
//   M[m][h*d + a] = sum_c w[m][h*d + c] S_h[a][c]          (per image, C_out x 2C', tiny)
//   qt[h*d + a][n] = relu(q_h[n][a]) / den_h[n]            (the queries, scaled per head and token)
//
// which is exact in real arithmetic: the d x d contraction of the apply step moves
// from every token into the small matrix M, and what is left per token and head is
// one d-term dot product (the normaliser) and a scaling.  M and qt are rounded to
// bf16 where the unfused path rounds S and O.
//
// state_fold_kernel : sums the partial states in index order (fixed order, so the result
//                     is reproducible bit for bit), writes ks and M (fp32 accumulate, bf16 out).
// fused_out_kernel  : clusters of two CTAs, paired tensor-core MMAs (cta_group::2, M = 256).
//   Each CTA keeps its 128 rows of M (<= 128 KB) in shared memory while the image lasts and
//   owns 128 of the pair's 256 tokens per tile.  The unit handed from role to role is a pair of
//   heads (two slices of d query channels in one ring slot, one set of barriers): the thread that
//   issues the MMAs pays a wait and a commit per unit, and its serial chain is what bounds the kernel.
//     warp 0       TMA: per head one box of 128 tokens x d channels of the head's planar [N][d]
//                  query matrix (one contiguous 8 KB piece for d = 32; swizzle span = the row)
//     warps 2-13   turn q into qt in place (normaliser on the fp32 pipes, one token per lane);
//                  three groups of four warps, each taking every third slice
//     warp 1       (leader CTA only) issues tcgen05.mma 256 x 256 x 16: A = M, B = qt, both
//                  K-major, fp32 accumulators in both CTAs' tensor memory
//     warps 14-17  drain the accumulators: TMEM -> bf16 (+ bias) -> swizzled staging -> TMA
//                  stores of 32-channel x 64-token blocks into the NCHW output
//                  (RES kernels: the same block of a residual tensor, fetched by TMA into a block of its own one
//                  block ahead of its use, is added before the conversion: the residual connection around the module)
//   Two accumulator sets (2 x 256 TMEM columns) let the drain of a tile overlap the next.
// No TMA load is multicast: each CTA loads its own operands; only tcgen05.commit signals
// both CTAs' barriers.  Every mbarrier wait is bounded as in the GEMM.
#include <cuda.h>

#include "msla_common.cuh"
#include "msla_host.h"
#include "tma_host.h"
#include "tcgen05_util.cuh"

namespace msla {
namespace {

using bf16 = __nv_bfloat16;

constexpr int OT = 128;                  // tokens per CTA and tile (256 per pair); 64 where that spreads a small problem over more pairs
constexpr int OM = 128;                  // output channels per CTA (256 per pair)
constexpr int OKS = 64;                  // k-extent of one resident slice of M (one 128-byte swizzle span)
constexpr int O_A_SLICE = OM * OKS * 2;  // 16 KB: 128 rows of M x 64 k
constexpr int O_MAX_KS = 8;              // K = 2C' <= 512
constexpr int O_MIN_STAGES = 2, O_MAX_STAGES = 16;  // query ring: as many slots (of two slices each) as shared memory holds (the host decides)
constexpr int O_XWARPS = 12;             // transform warps: three groups of four, each taking every third slice
constexpr int O_THREADS = 32 * (2 + O_XWARPS + 4);
constexpr int O_STAGING_WARP = 32 * 128;
constexpr int O_STAGING = 4 * O_STAGING_WARP;
constexpr int O_BAR_BYTES = 512;
constexpr int O_SMEM_FIXED = O_STAGING + O_BAR_BYTES + 1024;  // besides the rows of M, the ring and the residual blocks
constexpr int O_SMEM_LIMIT = 226 * 1024;                     // dynamic shared memory of a CTA (1 KB of the 227 left to static data)
static_assert(24 * O_MAX_STAGES + 16 + 16 + 8 + 8 + 8 + 4 * 8 <= O_BAR_BYTES, "barrier block");

__device__ int g_fused_timeout_flag = 0;

struct OutParams {
  const float* ks;   // [B][Ht][d] key sums
  const bf16* bias;  // [Cout] or nullptr
  const bf16* residual;  // RES kernels: [B][Cout][N], added to the output (the residual connection around the module)
  int B, N, Cout, Ht, d;
  int kslices;       // 64-wide k-slices of M: ceil(Ht * d / 64)
  int ot;            // tokens per CTA and tile: 128 or 64
  int stages;        // slots of the query ring (a slot holds the slices of two consecutive heads)
  int tiles_per_image, num_tiles;  // tiles of 2 * ot tokens
  float eps;
};

// ---- cluster helpers
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {  // shared::cta address -> shared::cluster address in CTA `rank`
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred P1;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 P1, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, P1;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait on a barrier that other CTAs of the cluster (or tcgen05.commit) arrive on.
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait_cluster(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait_cluster(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
      *abort_flag = 1;
      return false;
    }
  }
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
// K-major shared-memory matrix descriptor whose swizzle span is the row: rows of 64 bytes (mode 4) or 32 bytes (mode 6);
// sbo16 = distance between groups of 8 rows in 16-byte units.
__device__ __forceinline__ uint64_t make_desc_kmajor(uint32_t addr, uint32_t sbo16, uint64_t mode) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)sbo16 << 32) | (1ull << 46) | (mode << 61);
}
__device__ __forceinline__ void umma2_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives (once the MMAs issued so far have completed) on the barrier at this shared-memory offset in both CTAs of the pair.
__device__ __forceinline__ void umma2_commit_both(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((unsigned short)3) : "memory");
}

// F16 kernels: the 16-bit storage type is IEEE binary16 instead of bfloat16.  The values travel untyped; the conversions,
// the packed maximum and the MMA's operand format differ.
template <bool F16> __device__ __forceinline__ float lo16(uint32_t w) {
  if constexpr (F16) return __low2float(*reinterpret_cast<const __half2*>(&w));
  else return __uint_as_float(w << 16);
}
template <bool F16> __device__ __forceinline__ float hi16(uint32_t w) {
  if constexpr (F16) return __high2float(*reinterpret_cast<const __half2*>(&w));
  else return __uint_as_float(w & 0xffff0000u);
}
template <bool F16> __device__ __forceinline__ uint32_t pack16(float lo, float hi) {
  if constexpr (F16) {
    uint32_t r;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
  } else {
    return pack2(lo, hi);
  }
}

// ---------------------------------------------------------------------------
// Second level of the state reduction (Eq. 3) and the fold of the state into the projection weights.
// Grid (B * Ht, chunks): a CTA takes one head and `da` = d / chunks of its key channels a, i.e. `da` consecutive rows of the
// head's state.  partial: [B*Ht][S][d*(d+1)] fp32, entry [a][c], column d = key sum.
//   ks[bh][a]            = sum_s partial[bh][s][a][d]
//   M[b][m][hh*d + a]    = sum_c w[m][hh*d + c] * (sum_s partial[bh][s][a][c])        (bf16, row stride K), all m < Cout
// Fixed summation order: the S partial states are cut into FOLD_RUNS runs of consecutive indices, each run is summed in
// index order by its own thread, and the run sums are added in run order.  A thread issues all loads of its run
// (<= 8 vectors of 16 bytes) before the first add, so the kernel pays one round trip to memory, not S.
// ---------------------------------------------------------------------------
constexpr int FOLD_THREADS = 1024;
constexpr int FOLD_RUNS = 8;       // S <= 64: at most 8 partial states per run
constexpr int FOLD_RUN_BYTES = FOLD_RUNS * 32 * 33 * 4, FOLD_ST_BYTES = 32 * 33 * 4;
constexpr int FOLD_SMEM = FOLD_RUN_BYTES + FOLD_ST_BYTES + 256 * 32 * 2;  // + the head's [Cout <= 256][d <= 32] weight columns
// F16: M and ks are multiplied by `scale`, a power of two near 1 / N (the output kernel scales eps alike, so Eq. 3's quotient is
// unchanged): sums over N tokens then stay inside binary16's range.
template <bool F16>
__global__ void __launch_bounds__(FOLD_THREADS)
state_fold_kernel(const float* __restrict__ partial, int S, const bf16* __restrict__ w, bf16* __restrict__ M, float* __restrict__ ks,
                  int Ht, int d, int Cout, int K, int da, float scale) {
  extern __shared__ __align__(16) unsigned char fold_smem[];
  float4 (*run_sum)[32 * 33 / 4] = reinterpret_cast<float4 (*)[32 * 33 / 4]>(fold_smem);
  float* st = reinterpret_cast<float*>(fold_smem + FOLD_RUN_BYTES);
  uint4* wtile = reinterpret_cast<uint4*>(fold_smem + FOLD_RUN_BYTES + FOLD_ST_BYTES);  // the head's columns of w: [Cout][d] bf16
  pdl_launch_dependents();
  const int bh = blockIdx.x, b = bh / Ht, hh = bh % Ht;
  // the projection weights do not come from the previous kernel: staged while it drains
  for (int i = threadIdx.x; i < Cout * (d / 8); i += FOLD_THREADS) {
    const int m = i / (d / 8), c8 = i - m * (d / 8);
    wtile[i] = __ldg(reinterpret_cast<const uint4*>(w + (long long)m * K + hh * d) + c8);  // 16-byte aligned: K and d are multiples of 8
  }
  pdl_wait();  // the partial states come from the previous kernel
  const int d1 = d + 1, ne = d * d1;
  const int a0 = blockIdx.y * da;
  const int nq4 = da * d1 / 4;  // this CTA's rows of the state, in 16-byte vectors (da * d1 is a multiple of 4)
  const float4* sp = reinterpret_cast<const float4*>(partial + (long long)bh * S * ne + a0 * d1);
  const int ne4 = ne / 4;
  for (int item = threadIdx.x; item < FOLD_RUNS * nq4; item += FOLD_THREADS) {
    const int j = item / nq4, e = item - j * nq4;
    const int s0 = S * j / FOLD_RUNS, s1 = S * (j + 1) / FOLD_RUNS;
    float4 t[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) t[u] = s0 + u < s1 ? __ldg(sp + (long long)(s0 + u) * ne4 + e) : make_float4(0.f, 0.f, 0.f, 0.f);
    float4 v = t[0];
#pragma unroll
    for (int u = 1; u < 8; ++u) { v.x += t[u].x; v.y += t[u].y; v.z += t[u].z; v.w += t[u].w; }
    run_sum[j][e] = v;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < nq4; e += FOLD_THREADS) {
    float4 v = run_sum[0][e];
#pragma unroll
    for (int j = 1; j < FOLD_RUNS; ++j) { const float4 r = run_sum[j][e]; v.x += r.x; v.y += r.y; v.z += r.z; v.w += r.w; }
    reinterpret_cast<float4*>(st)[e] = v;  // st[al * d1 + c], al = a - a0
  }
  __syncthreads();
  for (int al = threadIdx.x; al < da; al += FOLD_THREADS) ks[(long long)bh * d + a0 + al] = F16 ? st[al * d1 + d] * scale : st[al * d1 + d];
  // M: a thread keeps key channel al = threadIdx.x % da (FOLD_THREADS is a multiple of da), i.e. one row of the state,
  // in registers and walks the output channels m = threadIdx.x / da, + FOLD_THREADS / da, ...
  const int al = threadIdx.x % da;
  float srow[32];
#pragma unroll
  for (int c = 0; c < 32; ++c) srow[c] = c < d ? st[al * d1 + c] : 0.f;
  for (int m = threadIdx.x / da; m < Cout; m += FOLD_THREADS / da) {
    const uint4* wr = wtile + m * (d / 8);
    uint4 wv[4];
#pragma unroll
    for (int c8 = 0; c8 < 4; ++c8) wv[c8] = c8 < d / 8 ? wr[c8] : make_uint4(0u, 0u, 0u, 0u);
    float acc = 0.f;
#pragma unroll
    for (int c8 = 0; c8 < 4; ++c8) {
      const uint32_t word[4] = {wv[c8].x, wv[c8].y, wv[c8].z, wv[c8].w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {  // channels beyond d carry zeros on both sides
        acc = fmaf(lo16<F16>(word[e]), srow[8 * c8 + 2 * e], acc);
        acc = fmaf(hi16<F16>(word[e]), srow[8 * c8 + 2 * e + 1], acc);
      }
    }
    bf16* mp = M + ((long long)b * Cout + m) * K + hh * d + a0 + al;
    if constexpr (F16) *reinterpret_cast<__half*>(mp) = __float2half_rn(acc * scale);
    else *mp = __float2bfloat16_rn(acc);
  }
}

template <int D, bool RES, bool F16>
__global__ void __launch_bounds__(O_THREADS, 1)
fused_out_kernel(const __grid_constant__ CUtensorMap tmM, const __grid_constant__ CUtensorMap tmQ,
                 const __grid_constant__ CUtensorMap tmO, const __grid_constant__ CUtensorMap tmR, OutParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;  // swizzle atoms need 1024-byte alignment
  const uint32_t a_base = smem_base;                                  // resident rows of M: kslices x 16 KB
  constexpr int SLICE = OT * D * 2;                                    // one head's queries of this CTA's (up to) 128 tokens
  constexpr int SLOT = 2 * SLICE;                                      // ring slot: two consecutive heads
  constexpr int ROWB = D * 2;                                          // bytes per token row = the swizzle span
  const uint32_t ring = a_base + (uint32_t)p.kslices * O_A_SLICE;
  const uint32_t staging = ring + (uint32_t)p.stages * SLOT;
  const uint32_t resbuf = staging + O_STAGING;           // RES: one 32-channel x 64-token block of the residual per epilogue warp
  const uint32_t bars = resbuf + (RES ? O_STAGING : 0);
  const uint32_t full_bar = bars;                        // [stage] both heads' boxes landed (own CTA)
  const uint32_t empty_bar = bars + 8 * O_MAX_STAGES;        // [stage] MMAs have read the slice (commit, both CTAs)
  const uint32_t ready_bar = bars + 16 * O_MAX_STAGES;       // [stage] both CTAs' slices transformed (leader only)
  const uint32_t tfull_bar = bars + 24 * O_MAX_STAGES;       // [acc] accumulator complete (commit, both CTAs)
  const uint32_t tempty_bar = tfull_bar + 16;            // [acc] both CTAs' epilogues have drained it (leader only)
  const uint32_t res_bar = tempty_bar + 16;              // rows of M landed (own CTA)
  const uint32_t peer_res_bar = res_bar + 8;             // the peer's rows of M landed (leader only)
  const uint32_t tmem_slot = peer_res_bar + 8;
  const uint32_t resid_bar = tmem_slot + 8;              // [epilogue warp] RES: the warp's residual block landed
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_sh;

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();               // 0 = leader of the pair
  // A pair works on a run of consecutive tiles, so that it changes image (and reloads its rows of M) as seldom as possible.
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int tiles_per_pair = (p.num_tiles + npairs - 1) / npairs;
  const int tile_first = min(pair * tiles_per_pair, p.num_tiles), tile_end = min(tile_first + tiles_per_pair, p.num_tiles);

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(full_bar + 8 * s, 1);
      mbar_init(empty_bar + 8 * s, 1);
      mbar_init(ready_bar + 8 * s, 2 * 2 * 4);  // per head the four warps of one transform group, in both CTAs
    }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar + 8 * a, 1); mbar_init(tempty_bar + 8 * a, 2 * 4); }
    mbar_init(res_bar, 1);
    mbar_init(peer_res_bar, 1);
    if (RES)
      for (int w = 0; w < 4; ++w) mbar_init(resid_bar + 8 * w, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // one warp of each CTA of the pair: all 512 tensor-memory columns in both
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (threadIdx.x == 0) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(tmem_slot));
    tmem_base_sh = v;
  }
  cluster_sync_all();  // both CTAs' barriers exist before anything arrives on them from the other CTA
  const uint32_t tmem_base = tmem_base_sh;
  pdl_wait();  // queries, states and M come from earlier kernels

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (each CTA for itself)
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmM) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmQ) : "memory");
      uint32_t local = 0, s = 0, ph = 0;  // ring slot and the parity of its current use
      int cur_b = -1;
      bool ok = true;
      for (int tile = tile_first; ok && tile < tile_end; ++tile, ++local) {
        const int b = tile / p.tiles_per_image, nt = tile % p.tiles_per_image;
        if (b != cur_b) {
          if (cur_b >= 0) {  // every MMA that reads the previous image's rows of M must be complete
            const uint32_t last = local - 1;
            ok = mbar_wait_cluster(tfull_bar + 8 * (last & 1), (last >> 1) & 1, &abort_flag);
            if (!ok) break;
          }
          cur_b = b;
          mbar_expect_tx(res_bar, (uint32_t)(p.kslices * O_A_SLICE));
          for (int ks = 0; ks < p.kslices; ++ks)
            tma_load_3d(a_base + ks * O_A_SLICE, &tmM, res_bar, ks * OKS, (int)rank * OM, b);
        }
        const int n0 = nt * (2 * p.ot) + (int)rank * p.ot;
        for (int h = 0; ok && h < p.Ht; h += 2) {
          ok = mbar_wait_cluster(empty_bar + 8 * s, ph ^ 1, &abort_flag);
          if (!ok) break;
          const bool two = h + 1 < p.Ht;  // an odd head count leaves the last slot half used
          mbar_expect_tx(full_bar + 8 * s, (uint32_t)((two ? 2 : 1) * p.ot * ROWB));
          tma_load_4d(ring + s * SLOT, &tmQ, full_bar + 8 * s, 0, n0, h, b);  // rows past the last token are filled with zeros
          if (two) tma_load_4d(ring + s * SLOT + SLICE, &tmQ, full_bar + 8 * s, 0, n0, h + 1, b);
          if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader) / M hand-shake (peer)
    if (lane == 0) {
      // instruction descriptor: D = f32, A = B = bf16, both K-major, N = 256, M = 256 (pair)
      const uint32_t idesc = (1u << 4) | (F16 ? 0u : ((1u << 7) | (1u << 10))) | ((uint32_t)((2 * p.ot) >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
      const uint32_t peer_res_remote = map_to_cta(peer_res_bar, 0);
      uint32_t local = 0, res_ph = 0, s = 0, ph = 0;  // s, ph: ring slot and the parity of its current use
      // Matrix descriptors: the high words are constants; the low words carry the start address in 16-byte units
      // (A: the 128B-swizzled rows of M; B: the slice, K-major, the swizzle span being the token row).
      const uint64_t a_hi = make_desc(0, 1, 1024 >> 4), b_hi = make_desc_kmajor(0, (8 * ROWB) >> 4, D == 32 ? 4ull : 6ull);
      const uint32_t a_lo0 = (a_base & 0x3FFFFu) >> 4, b_lo0 = (ring & 0x3FFFFu) >> 4;
      int cur_b = -1;
      bool ok = true;
      for (int tile = tile_first; ok && tile < tile_end; ++tile, ++local) {
        const int b = tile / p.tiles_per_image;
        if (b != cur_b) {
          cur_b = b;
          ok = mbar_wait(res_bar, res_ph, &abort_flag);  // own rows of M
          if (!ok) break;
          if (rank == 0) {
            ok = mbar_wait_cluster(peer_res_bar, res_ph, &abort_flag);  // the peer's rows of M
            if (!ok) break;
          } else {
            mbar_arrive_cluster(peer_res_remote);
          }
          res_ph ^= 1;
        }
        if (rank != 0) continue;
        const uint32_t acc = local & 1, acc_ph = (local >> 1) & 1;
        ok = mbar_wait_cluster(tempty_bar + 8 * acc, acc_ph ^ 1, &abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * 256;
        uint32_t a_lo = a_lo0;  // walks the columns of M: 32 bytes per 16 columns, 64-column slices O_A_SLICE apart
        int col = 0;
        for (int h = 0; ok && h < p.Ht; h += 2) {
          ok = mbar_wait_cluster(ready_bar + 8 * s, ph, &abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t b_lo = b_lo0 + s * (uint32_t)(SLOT >> 4);
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            if (h + j >= p.Ht) break;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
              umma2_bf16(d_tmem, a_hi | a_lo, b_hi | (b_lo + (uint32_t)(j * (SLICE >> 4) + 2 * kk)), idesc, (h > 0 || j > 0 || kk > 0) ? 1u : 0u);
              col += 16;
              a_lo += (col & 63) ? 2u : (uint32_t)((O_A_SLICE - 96) >> 4);
            }
          }
          umma2_commit_both(empty_bar + 8 * s);  // both CTAs may refill the slot once these MMAs have read it
          if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1; }
        }
        if (ok) umma2_commit_both(tfull_bar + 8 * acc);
      }
    }
  } else if (warp < 2 + O_XWARPS) {
    // ------------------------------------------------------------ transform warps: q -> relu(q) / den, in place
    // Group xg of four warps takes every third slice, starting with slice xg; its 128 lanes own one token
    // row each (d channels: 64 or 32 bytes, 16-byte pieces XOR-swizzled with the row as the TMA unit
    // wrote them and as the MMA reads them; eight consecutive rows cover all banks once).
    constexpr int PCS = D / 8;     // 16-byte pieces per token row
    const int xw = warp - 2, xg = xw >> 2, wig = xw & 3;
    const uint32_t ready_remote = map_to_cta(ready_bar, 0);
    const uint32_t row = (uint32_t)(wig * 32 + lane);
    const uint32_t swz = D == 32 ? (row >> 1) & 3u : (row >> 2) & 1u;
    const uint32_t row_off = row * ROWB;
    uint32_t s = 0, ph = 0, turn = 0;  // ring slot, the parity of its current use, and the group whose turn it is
    const int h_end = (p.Ht + 1) & ~1;  // an odd head count: the empty half of the last slot still has to be signed off
    bool ok = true;
    for (int tile = tile_first; ok && tile < tile_end; ++tile) {
      const int b = tile / p.tiles_per_image;
      for (int h = 0; ok && h < h_end; ++h) {
        const uint32_t cs = s, cph = ph;  // this slice's slot; the counters move on to the next slice
        const bool mine = (int)turn == xg;
        if (h & 1) { if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1; } }
        if (++turn == O_XWARPS / 4) turn = 0;
        if (!mine) continue;
        // with 64-token tiles only the first two warps of a group own rows; past the last head there is nothing to do
        const bool has_row = (int)row < p.ot && h < p.Ht;
        // the head's key sums, fetched before the wait so that their latency hides behind it
        float kk[D];
        const float4* ksp = reinterpret_cast<const float4*>(p.ks + ((long long)b * p.Ht + min(h, p.Ht - 1)) * D);
#pragma unroll
        for (int a4 = 0; a4 < D / 4; ++a4) {
          const float4 v = __ldg(ksp + a4);
          kk[4 * a4] = v.x; kk[4 * a4 + 1] = v.y; kk[4 * a4 + 2] = v.z; kk[4 * a4 + 3] = v.w;
        }
        ok = mbar_wait(full_bar + 8 * cs, cph, &abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const uint32_t rbase = ring + cs * SLOT + (uint32_t)(h & 1) * SLICE + row_off;
        if (!has_row) {  // warp-uniform
          if (lane == 0) mbar_arrive_cluster(ready_remote + 8 * cs);
          continue;
        }
        uint32_t q[D / 2];  // word w = channels 2w (low half), 2w+1 (high half)
#pragma unroll
        for (int c = 0; c < PCS; ++c)
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(q[4 * c]), "=r"(q[4 * c + 1]), "=r"(q[4 * c + 2]), "=r"(q[4 * c + 3])
                       : "r"(rbase + (((uint32_t)c ^ swz) << 4)));
        float den[4] = {0.f, 0.f, 0.f, 0.f};  // four chains
#pragma unroll
        for (int w = 0; w < D / 2; ++w) {
          if constexpr (F16) asm("max.f16x2 %0, %1, %2;" : "=r"(q[w]) : "r"(q[w]), "r"(0u));
          else asm("max.bf16x2 %0, %1, %2;" : "=r"(q[w]) : "r"(q[w]), "r"(0u));
          den[2 * (w & 1)] = fmaf(lo16<F16>(q[w]), kk[2 * w], den[2 * (w & 1)]);
          den[2 * (w & 1) + 1] = fmaf(hi16<F16>(q[w]), kk[2 * w + 1], den[2 * (w & 1) + 1]);
        }
        const float inv = __frcp_rn((den[0] + den[1]) + (den[2] + den[3]) + p.eps);
#pragma unroll
        for (int w = 0; w < D / 2; ++w) q[w] = pack16<F16>(lo16<F16>(q[w]) * inv, hi16<F16>(q[w]) * inv);
#pragma unroll
        for (int c = 0; c < PCS; ++c)
          asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(rbase + (((uint32_t)c ^ swz) << 4)), "r"(q[4 * c]), "r"(q[4 * c + 1]),
                       "r"(q[4 * c + 2]), "r"(q[4 * c + 3]) : "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the tensor cores read what was just written
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(ready_remote + 8 * cs);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue
    // Four warps; warp % 4 selects the TMEM lane quarter (a hardware rule).  A lane owns one output
    // channel of this CTA's 128; the accumulator's 256 columns are the pair's 256 tokens.
    const int quarter = warp & 3;
    const uint32_t stage = staging + (uint32_t)(warp - 2 - O_XWARPS) * O_STAGING_WARP;
    const uint32_t my_row = stage + lane * 128, sw = (uint32_t)(lane & 7);
    const int row0 = (int)rank * OM + quarter * 32;
    const float bias = !(p.bias && row0 + lane < p.Cout) ? 0.f : F16 ? __half2float(reinterpret_cast<const __half*>(p.bias)[row0 + lane]) : __bfloat162float(p.bias[row0 + lane]);
    const uint32_t tempty_remote = map_to_cta(tempty_bar, 0);
    // RES: the residual arrives by TMA, one 32-channel x 64-token block per warp and request, a block ahead of its use
    const uint32_t my_resid_bar = resid_bar + 8 * (uint32_t)(warp - 2 - O_XWARPS);
    const uint32_t my_res = resbuf + (uint32_t)(warp - 2 - O_XWARPS) * O_STAGING_WARP, my_res_row = my_res + lane * 128;
    uint32_t res_count = 0;
    auto request_residual = [&](int t2, int j2) {  // one lane
      mbar_expect_tx(my_resid_bar, O_STAGING_WARP);
      tma_load_3d(my_res, &tmR, my_resid_bar, (t2 % p.tiles_per_image) * (2 * p.ot) + j2 * 64, row0, t2 / p.tiles_per_image);
    };
    if (RES && lane == 0 && row0 < p.Cout && tile_first < tile_end) request_residual(tile_first, 0);
    uint32_t local = 0;
    bool ok = true;
    for (int tile = tile_first; ok && tile < tile_end; ++tile, ++local) {
      const int b = tile / p.tiles_per_image, nt = tile % p.tiles_per_image;
      const uint32_t acc = local & 1, acc_ph = (local >> 1) & 1;
      ok = mbar_wait_cluster(tfull_bar + 8 * acc, acc_ph, &abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + acc * 256 + ((uint32_t)(quarter * 32) << 16);
      uint32_t r[2][32];
      tmem_ld32(taddr, r[0]);
      const int chunks = (2 * p.ot) / 32;  // the accumulator's columns are the pair's tokens
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        if (c >= chunks) break;
        tmem_ld_wait();
        if (c + 1 < chunks) tmem_ld32(taddr + (c + 1) * 32, r[(c + 1) & 1]);  // next chunk streams in meanwhile
        const uint32_t(&rc)[32] = r[c & 1];
        const int n0 = nt * (2 * p.ot) + (c >> 1) * 64;  // first token of the 64-token block
        if (n0 >= p.N || row0 >= p.Cout) continue;    // warp-uniform
        if ((c & 1) == 0) {  // the previous block must have been read out of the staging buffer
          if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          __syncwarp();
          if (RES) {           // this block of the residual was requested one block ago
            ok = mbar_wait(my_resid_bar, res_count & 1, &abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            ++res_count;
          }
        }
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const uint32_t pc = (uint32_t)((c & 1) * 4 + v);
          uint4 rv = make_uint4(0u, 0u, 0u, 0u);  // the same 16-byte piece of the lane's row in the residual block (same box, same swizzle)
          if (RES) asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(rv.x), "=r"(rv.y), "=r"(rv.z), "=r"(rv.w) : "r"(my_res_row + ((pc ^ sw) << 4)));
          const uint32_t rw[4] = {rv.x, rv.y, rv.z, rv.w};
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float f0 = __uint_as_float(rc[v * 8 + 2 * e]) + bias, f1 = __uint_as_float(rc[v * 8 + 2 * e + 1]) + bias;
            if (RES) { f0 += lo16<F16>(rw[e]); f1 += hi16<F16>(rw[e]); }
            w[e] = pack16<F16>(f0, f1);
          }
          asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(my_row + ((pc ^ sw) << 4)), "r"(w[0]), "r"(w[1]), "r"(w[2]),
                       "r"(w[3]) : "memory");
        }
        if (c & 1) {
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // also orders the reads of the residual block before its refill
          __syncwarp();
          if (lane == 0) {
            tma_store_3d(&tmO, stage, n0, row0, b);
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            if (RES) {  // request the next block this warp will drain: the next 64 tokens of this tile, else the next tile's first
              int t2 = tile, j2 = (c >> 1) + 1;
              if (j2 * 64 >= 2 * p.ot || (t2 % p.tiles_per_image) * (2 * p.ot) + j2 * 64 >= p.N) { ++t2; j2 = 0; }
              if (t2 < tile_end) request_residual(t2, j2);
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(tempty_remote + 8 * acc);  // this warp's quarter of the accumulator is drained
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // stores done before the CTA retires
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    // give copies and MMAs still in flight time to land before memory is released
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    if (threadIdx.x == 0) atomicExch(&g_fused_timeout_flag, 1);
    __syncthreads();
  }
  cluster_sync_all();  // neither CTA leaves (or frees tensor memory) while the other may still touch its barriers or shared memory
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

}  // namespace

bool fused_out_bf16_supported(int Ht, int d, int Cout, int N) {
  return (d == 16 || d == 32) && Ht >= 1 && Ht * d <= O_MAX_KS * OKS && Cout >= 1 && Cout <= 2 * OM && Cout % 8 == 0 && N >= 8 && N % 8 == 0;
}

// Scratch: M [B][Cout][Ht*d] bf16, then ks [B][Ht][d] fp32 (256-byte aligned).
static size_t fused_out_m_bytes(int B, int Ht, int d, int Cout) { return ((size_t)B * Cout * Ht * d * 2 + 255) / 256 * 256; }
size_t fused_out_scratch_bytes(int B, int Ht, int d, int Cout) { return fused_out_m_bytes(B, Ht, d, Cout) + (size_t)B * Ht * d * sizeof(float); }

// y[b][m][n] = sum_h sum_c w[m][h*d + c] * att[b][h][n][c] + bias[m], att = Eq. 3 applied to query head h with the
// state of (b, h) = sum over s < S of partial[(b * Ht + h) * S + s] ([d][d+1] fp32 each: KV, then the key sum in
// column d).  q: planar bf16 query matrices [N][d], head h of image b at q + b*q_sb + h*q_sh (elements); y: NCHW
// [B, Cout, N].
namespace {
template <int D, bool RES, bool F16>
msla_status_t launch_fused(dim3 grid, int smem, cudaStream_t st, const CUtensorMap& tmM, const CUtensorMap& tmQ, const CUtensorMap& tmO,
                           const CUtensorMap& tmR, const OutParams& p) {
  static std::atomic<unsigned long long> attr_done{0};
  const msla_status_t s = ensure_smem_attr(attr_done, fused_out_kernel<D, RES, F16>, O_SMEM_LIMIT);
  if (s != MSLA_OK) return s;
  launch_pdl_cluster2(fused_out_kernel<D, RES, F16>, grid, dim3(O_THREADS), (size_t)smem, st, tmM, tmQ, tmO, tmR, p);
  return MSLA_OK;
}
template <bool F16>
msla_status_t launch_fused_for(int d, bool res, dim3 grid, int smem, cudaStream_t st, const CUtensorMap& tmM, const CUtensorMap& tmQ,
                               const CUtensorMap& tmO, const CUtensorMap& tmR, const OutParams& p) {
  if (d == 32) return res ? launch_fused<32, true, F16>(grid, smem, st, tmM, tmQ, tmO, tmR, p) : launch_fused<32, false, F16>(grid, smem, st, tmM, tmQ, tmO, tmR, p);
  return res ? launch_fused<16, true, F16>(grid, smem, st, tmM, tmQ, tmO, tmR, p) : launch_fused<16, false, F16>(grid, smem, st, tmM, tmQ, tmO, tmR, p);
}
}  // namespace

// f16: queries, weights, bias, residual and output are IEEE binary16 instead of bfloat16; M, the key sums and eps are
// scaled by the power of two just above 1 / N (N tokens' sums would leave binary16's range otherwise).
msla_status_t run_fused_out_bf16(const void* q, long long q_sb, long long q_sh, const float* partial, int S, void* scratch,
                                 const void* w, const void* bias, const void* residual, void* y, int B, int Ht, int d, int N, int Cout,
                                 float eps, cudaStream_t st, bool f16) {
  if (!fused_out_bf16_supported(Ht, d, Cout, N) || q_sb % 8 != 0 || q_sh % 8 != 0)
    return fail(MSLA_ERR_UNSUPPORTED, "fused apply + projection: %d heads of %d channels, %d output channels, %d tokens", Ht, d, Cout, N);
  if (S < 1 || S > 8 * FOLD_RUNS) return fail(MSLA_ERR_UNSUPPORTED, "fused apply + projection: %d partial states per head (1 .. %d)", S, 8 * FOLD_RUNS);
  const int K = Ht * d;
  // 256-token tiles per pair of CTAs; 128-token tiles for problems so small that half the pairs would have nothing
  // to do (the larger tile is the more efficient one as soon as every pair has work)
  const int sms = device_sm_count();
  const int ot = 2LL * B * ((N + 2 * OT - 1) / (2 * OT)) <= sms / 2 ? OT / 2 : OT;
  bf16* M = (bf16*)scratch;
  float* ks = (float*)((char*)scratch + fused_out_m_bytes(B, Ht, d, Cout));
  CUtensorMap tmM, tmQ, tmO, tmR;
  {
    const cuuint64_t dM[3] = {(cuuint64_t)K, (cuuint64_t)Cout, (cuuint64_t)B};
    const cuuint64_t sM[2] = {(cuuint64_t)K * 2, (cuuint64_t)K * Cout * 2};
    const cuuint32_t bM[3] = {OKS, OM, 1};
    const cuuint64_t dQ[4] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)Ht, (cuuint64_t)B};
    const cuuint64_t sQ[3] = {(cuuint64_t)d * 2, (cuuint64_t)q_sh * 2, (cuuint64_t)q_sb * 2};
    const cuuint32_t bQ[4] = {(cuuint32_t)d, (cuuint32_t)ot, 1, 1};
    const cuuint64_t dO[3] = {(cuuint64_t)N, (cuuint64_t)Cout, (cuuint64_t)B};
    const cuuint64_t sO[2] = {(cuuint64_t)N * 2, (cuuint64_t)Cout * N * 2};
    const cuuint32_t bO[3] = {64, 32, 1};
    if (!tma_make_map_bf16(&tmM, M, 3, dM, sM, bM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !tma_make_map_bf16(&tmQ, q, 4, dQ, sQ, bQ, d == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B) ||
        !tma_make_map_bf16(&tmO, y, 3, dO, sO, bO, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !tma_make_map_bf16(&tmR, residual ? residual : y, 3, dO, sO, bO, CU_TENSOR_MAP_SWIZZLE_128B))
      return fail(MSLA_ERR_CUDA, "cuTensorMapEncodeTiled failed for the fused apply + output projection");
  }
  OutParams p{};
  p.ks = ks; p.bias = (const bf16*)bias; p.residual = (const bf16*)residual;
  float scale = 1.f;
  if (f16)
    for (long long n = 1; n < N; n <<= 1) scale *= 0.5f;
  p.B = B; p.N = N; p.Cout = Cout; p.Ht = Ht; p.d = d; p.eps = eps * scale;
  p.kslices = (K + OKS - 1) / OKS;
  p.ot = ot;
  p.tiles_per_image = (N + 2 * ot - 1) / (2 * ot);
  const long long tiles = (long long)B * p.tiles_per_image;
  if (tiles > 0x7fffffffLL) return fail(MSLA_ERR_UNSUPPORTED, "too many token tiles");
  p.num_tiles = (int)tiles;
  // the query ring takes what shared memory is left beside the rows of M (and the residual blocks)
  const int smem_fixed = p.kslices * O_A_SLICE + O_SMEM_FIXED + (residual ? O_STAGING : 0), slot = 2 * OT * d * 2;
  p.stages = (O_SMEM_LIMIT - smem_fixed) / slot;
  if (p.stages > O_MAX_STAGES) p.stages = O_MAX_STAGES;
  if (p.stages < O_MIN_STAGES) return fail(MSLA_ERR_UNSUPPORTED, "fused apply + projection: no room for the query ring (%d slots)", p.stages);
  const int smem = smem_fixed + p.stages * slot;
  long long pairs = sms / 2;
  if (pairs > tiles) pairs = tiles;
  if (pairs < 1) pairs = 1;
  // about one CTA per SM: few heads -> up to eight CTAs per head, each with a share of the head's key channels
  // (a share's rows of the state, da * (d + 1) floats, must stay a whole number of 16-byte vectors: da >= 4)
  int fold_chunks = sms / (B * Ht);
  fold_chunks = (fold_chunks >= 8 && d == 32) ? 8 : fold_chunks >= 4 ? 4 : (fold_chunks >= 2 ? 2 : 1);
  static std::atomic<unsigned long long> attr_fold{0}, attr_fold16{0};
  msla_status_t s = f16 ? ensure_smem_attr(attr_fold16, state_fold_kernel<true>, FOLD_SMEM) : ensure_smem_attr(attr_fold, state_fold_kernel<false>, FOLD_SMEM);
  if (s != MSLA_OK) return s;
  const dim3 fold_grid((unsigned)(B * Ht), (unsigned)fold_chunks);
  if (f16) launch_pdl(state_fold_kernel<true>, fold_grid, dim3(FOLD_THREADS), FOLD_SMEM, st, partial, S, (const bf16*)w, M, ks, Ht, d, Cout, K, d / fold_chunks, scale);
  else launch_pdl(state_fold_kernel<false>, fold_grid, dim3(FOLD_THREADS), FOLD_SMEM, st, partial, S, (const bf16*)w, M, ks, Ht, d, Cout, K, d / fold_chunks, scale);
  const dim3 grid((unsigned)(2 * pairs));
  s = f16 ? launch_fused_for<true>(d, residual != nullptr, grid, smem, st, tmM, tmQ, tmO, tmR, p)
          : launch_fused_for<false>(d, residual != nullptr, grid, smem, st, tmM, tmQ, tmO, tmR, p);
  if (s != MSLA_OK) return s;
  count_launches(2);
  return check_launch("fused apply + output projection (tcgen05, paired CTAs)");
}

int fused_timeout_flag() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_fused_timeout_flag, sizeof(int)) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  return v;
}

}  // namespace msla
