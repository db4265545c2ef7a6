// Steps 4 and 5 of the module in one kernel (bf16, d = 32): the normalised
// attention output of Eq. 3 is produced tile by tile in shared memory and
// consumed there as the activation operand of the output projection, so the
// head concat never goes to HBM (Section 3.1; the fusion changes no value that
// is defined there: the operand is rounded to bf16 exactly as when it is stored).
//
// One persistent CTA per SM works on tiles of 128 tokens.  Roles:
//   warp 0      TMA producer of w_proj slices (64 k x 128 rows, K-major, 128B swizzle)
//   warp 1      issues tcgen05.mma 128x128x16; owns the tensor-memory allocation
//   warps 2-9   "apply" warps.  In round r warp a serves head 8r + a: it streams that
//               head's query rows through a per-lane cp.async FIFO, multiplies them
//               with the head's state (rounded to bf16, one extra column block for
//               the denominator) on mma.sync, normalises, and writes the
//               128 x 32 result into its half of B slice a/2 (128 tokens x 64
//               channels, the layout a 128B-swizzled TMA load would have produced)
//   warps 10-13 drain the accumulators: TMEM -> bf16 (+ bias) -> swizzled staging ->
//               TMA store of 32-channel x 32-token blocks into the NCHW output
// Four B slices (one round = 8 heads) are live at a time; a slice is rewritten
// once the MMAs that read it have completed (bempty), so rounds and tiles
// pipeline.  Two accumulator sets (2 x 2 x 128 TMEM columns) let the drain of a
// tile overlap the next tile.  Every mbarrier wait is bounded as in the GEMMs.
#include <cuda.h>

#include "msla_common.cuh"
#include "msla_host.h"
#include "tma_host.h"
#include "tcgen05_util.cuh"

namespace msla {
namespace {

using bf16 = __nv_bfloat16;

constexpr int FD = 32;             // channels per head
constexpr int FT = 128;            // tokens per tile (UMMA N)
constexpr int FBM = 128;           // output channels per accumulator (UMMA M)
constexpr int FBK = 64;            // channels per k-slice: one pair of heads
constexpr int F_APPLY_WARPS = 8;
constexpr int F_SLICES = F_APPLY_WARPS / 2;
constexpr int F_ASTAGES = 4;
constexpr int F_QSTAGES = 4;       // depth of the per-lane query FIFO
constexpr int F_U = 2;             // 16-token MMA tiles per FIFO stage
constexpr int F_STEP_TOKENS = 16 * F_U;
constexpr int F_STEPS = FT / F_STEP_TOKENS;  // FIFO stages per (tile, round)
constexpr int F_THREADS = 32 * (2 + F_APPLY_WARPS + 4);
constexpr int F_SLICE_BYTES = FT * FBK * 2;            // 16 KB
constexpr int F_A_BYTES = FBM * FBK * 2;               // 16 KB
constexpr int F_QSTAGE_BYTES = F_U * 2 * 32 * 16;      // 2 KB per warp and stage
constexpr int F_FIFO_BYTES = F_APPLY_WARPS * F_QSTAGES * F_QSTAGE_BYTES;
constexpr int F_STAGING_BYTES = 4 * 2048;
constexpr int F_SMEM_BYTES = F_SLICES * F_SLICE_BYTES + F_ASTAGES * F_A_BYTES + F_FIFO_BYTES + F_STAGING_BYTES + 256 + 1024;

__device__ int g_fused_timeout_flag = 0;

constexpr int F_FRAG_WORDS = (FD / 16) * (FD / 8 + 1) * 2;  // 20 words per lane and head

struct FusedParams {
  const bf16* q;        // query planes, strides in qv
  const uint4* frags;   // [B * heads][10][32 lanes]: the states as mma.sync B fragments (state_fragments_kernel)
  const bf16* bias;     // [Cout] or nullptr
  HeadView qv;
  int heads;            // heads per image over all scales (even); K = 32 * heads
  int B, N, Cout;
  int m_tiles;          // 1 or 2 accumulators of 128 output channels
  int tiles_per_batch, num_tiles;
  float eps;
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void lds128(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ uint32_t relu2(uint32_t v) {
  uint32_t r;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(v), "r"(0u));
  return r;
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void mma_bf16_first(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {  // C = 0
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.f));
}

// Second level of the state reduction, straight into the form the apply warps consume.  Four CTAs per
// head, eight state rows each: every state entry [32][33] (KV | key sum) is the sum of its S partial states in index order (a
// fixed order, so results are reproducible bit for bit), accumulated in fp32 and kept in shared
// memory; the CTA then writes the state as per-lane B fragments of mma.sync.  Word (ks*5 + j)*2 + e
// of lane (g, t) packs rows a0, a0+1 (a0 = 8t + 4ks + 2e) of column c = 8(g/2) + 2j + (g&1), or of the
// key-sum column for j = 4, rounded to bf16 like every other tensor-core operand of the module
// (feeding the remainders as a second set of fragments doubles the kernel's mma.sync work for a
// change of the module's relative L2 error from 0.33 % to 0.30 %).  Laid out so that a lane fetches
// its 20 words with five 16-byte loads, consecutive lanes 16 bytes apart.
constexpr int F_NE = FD * (FD + 1);
constexpr int F_FRAG_ROWS = 8;                       // state rows per CTA: rows 8q .. 8q+7 feed exactly the lanes with t = q
constexpr int F_FRAG_THREADS = F_FRAG_ROWS * (FD + 1);  // one state entry per thread
__global__ void __launch_bounds__(F_FRAG_THREADS) state_fragments_kernel(const float* __restrict__ partial, int S, uint32_t* __restrict__ table) {
  __shared__ float st[F_FRAG_ROWS * (FD + 1)];
  pdl_launch_dependents();
  pdl_wait();  // the partial states come from the previous kernel
  const int head = blockIdx.x, q = blockIdx.y;
  const float* sp = partial + (long long)head * S * F_NE + q * F_FRAG_ROWS * (FD + 1) + threadIdx.x;
  float v = 0.f;
#pragma unroll 8
  for (int s = 0; s < S; ++s) v += sp[(long long)s * F_NE];
  st[threadIdx.x] = v;
  __syncthreads();
  uint32_t* tp = table + (long long)head * (F_FRAG_WORDS * 32);
  for (int i = threadIdx.x; i < F_FRAG_WORDS * 8; i += F_FRAG_THREADS) {  // the 20 words of the 8 lanes (g, t = q)
    const int g = i & 7, w = i >> 3, lane = 4 * g + q;
    const int e = w & 1, j = (w >> 1) % (FD / 8 + 1), ks = (w >> 1) / (FD / 8 + 1);
    const int a0 = 4 * ks + 2 * e;                     // row 8q + a0 of the state, local row a0
    const int c = j < FD / 8 ? (g >> 1) * 8 + 2 * j + (g & 1) : FD;
    tp[((w >> 2) * 32 + lane) * 4 + (w & 3)] = pack2(st[a0 * (FD + 1) + c], st[(a0 + 1) * (FD + 1) + c]);
  }
}

__global__ void __launch_bounds__(F_THREADS, 1)
apply_project_fused_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmO, FusedParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;  // swizzle atoms need 1024-byte alignment
  const uint32_t slices = smem_base;
  const uint32_t aring = slices + F_SLICES * F_SLICE_BYTES;
  const uint32_t fifo = aring + F_ASTAGES * F_A_BYTES;
  const uint32_t staging = fifo + F_FIFO_BYTES;
  const uint32_t bars = staging + F_STAGING_BYTES;
  const uint32_t afull = bars, aempty = bars + 8 * F_ASTAGES;
  const uint32_t bfull = bars + 16 * F_ASTAGES, bempty = bfull + 8 * F_SLICES;
  const uint32_t tfull = bempty + 8 * F_SLICES, tempty = tfull + 16;
  const uint32_t tmem_slot = tempty + 16;
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_sh;

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int P = p.heads >> 1;              // pairs of heads = k-slices
  const int rounds = (p.heads + F_APPLY_WARPS - 1) / F_APPLY_WARPS;
  const int my_tiles = blockIdx.x < p.num_tiles ? (p.num_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < F_ASTAGES; ++s) { mbar_init(afull + 8 * s, 1); mbar_init(aempty + 8 * s, 1); }
    for (int s = 0; s < F_SLICES; ++s) { mbar_init(bfull + 8 * s, 2); mbar_init(bempty + 8 * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull + 8 * a, 1); mbar_init(tempty + 8 * a, 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // whole warp: all 512 tensor-memory columns (one CTA per SM)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (threadIdx.x == 0) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(tmem_slot));
    tmem_base_sh = v;
  }
  __syncthreads();
  const uint32_t tmem_base = tmem_base_sh;
  pdl_wait();  // queries and states come from earlier kernels

  if (warp == 0) {
    // --------------------------------------------------- TMA producer (weights)
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
      uint32_t it = 0;
      bool ok = true;
      for (int ti = 0; ok && ti < my_tiles; ++ti)
        for (int pair = 0; ok && pair < P; ++pair)   // the order in which the MMA warp meets the slices
          for (int mt = 0; ok && mt < p.m_tiles; ++mt, ++it) {
            const uint32_t s = it % F_ASTAGES, ph = (it / F_ASTAGES) & 1;
            ok = mbar_wait(aempty + 8 * s, ph ^ 1, &abort_flag);
            if (!ok) break;
            mbar_expect_tx(afull + 8 * s, F_A_BYTES);
            tma_load_3d(aring + s * F_A_BYTES, &tmA, afull + 8 * s, pair * FBK, mt * FBM, 0);
          }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // instruction descriptor: D = f32, A = B = bf16, both K-major, N = 128, M = 128
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(FT >> 3) << 17) | ((uint32_t)(FBM >> 4) << 24);
      uint32_t it = 0;
      bool ok = true;
      for (int ti = 0; ok && ti < my_tiles; ++ti) {
        const uint32_t acc = ti & 1, acc_ph = (ti >> 1) & 1;
        ok = mbar_wait(tempty + 8 * acc, acc_ph ^ 1, &abort_flag);
        if (!ok) break;
        tc_fence_after();
        for (int pair = 0; ok && pair < P; ++pair) {
          const int s = pair % F_SLICES, r = pair / F_SLICES;
          const int uses_per_tile = (P - s + F_SLICES - 1) / F_SLICES;  // rounds in which slice s is used
          const uint32_t use = (uint32_t)(ti * uses_per_tile + r);
          ok = mbar_wait(bfull + 8 * s, use & 1, &abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sb = slices + s * F_SLICE_BYTES;
          for (int mt = 0; ok && mt < p.m_tiles; ++mt, ++it) {
            const uint32_t sa_i = it % F_ASTAGES, ph = (it / F_ASTAGES) & 1;
            ok = mbar_wait(afull + 8 * sa_i, ph, &abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t sa = aring + sa_i * F_A_BYTES;
            const uint32_t d_tmem = tmem_base + acc * 256 + mt * FT;
#pragma unroll
            for (int kk = 0; kk < FBK / 16; ++kk)
              umma_bf16(d_tmem, make_desc(sa + kk * 32, 1, 1024 >> 4), make_desc(sb + kk * 32, 1, 1024 >> 4), idesc,
                        (pair > 0 || kk > 0) ? 1u : 0u);
            umma_commit(aempty + 8 * sa_i);
          }
          if (ok) umma_commit(bempty + 8 * s);  // the slice may be rewritten once these MMAs have read it
        }
        if (ok) umma_commit(tfull + 8 * acc);
      }
    }
  } else if (warp < 2 + F_APPLY_WARPS) {
    // ------------------------------------------------------------ apply warps
    // A = relu(Q) (rows = 16 tokens), B = state; lane (g, t) holds channels 8t..8t+7 of tokens g and
    // g+8 of each 16-token tile (the fragment layout of the stand-alone apply kernel).
    constexpr int KS = FD / 16, NT = FD / 8;
    const int aw = warp - 2;
    const int g = lane >> 2, t = lane & 3;
    // MMA rows g and g+8 of a 16-token tile are tokens gp and gp+8: the eight lanes of a quarter-warp
    // (g = 2i, 2i+1) then write slice rows i and i+4, whose 16-byte pieces fall into different banks
    const int gp = (g >> 1) | ((g & 1) << 2);
    const int s = aw >> 1;                                 // B slice of this warp's pair
    const int uses_per_tile = P > s ? (P - s + F_SLICES - 1) / F_SLICES : 0;
    const uint32_t ring = fifo + aw * (F_QSTAGES * F_QSTAGE_BYTES) + lane * 16;
    const uint32_t slice = slices + s * F_SLICE_BYTES;
    const int steps_per_tile = rounds * F_STEPS;
    const int total_steps = my_tiles * steps_per_tile;

    // One FIFO stage per step; steps run over (tile, round, 32-token group).  The copies run
    // F_QSTAGES-1 steps ahead of the arithmetic, each with its own cursor (no divisions per step).
    struct Cursor { int ti, r, st, b, nt; };
    auto locate = [&](Cursor& c) {                         // batch and token tile of c.ti
      const int tile = blockIdx.x + c.ti * gridDim.x;
      c.b = tile / p.tiles_per_batch;
      c.nt = tile - c.b * p.tiles_per_batch;
    };
    auto advance = [&](Cursor& c) {
      if (++c.st == F_STEPS) {
        c.st = 0;
        if (++c.r == rounds) { c.r = 0; ++c.ti; locate(c); }
      }
    };
    Cursor ic{0, 0, 0, 0, 0}, cc{0, 0, 0, 0, 0};
    locate(ic);
    locate(cc);
    int issued = 0;
    auto issue = [&]() {                                   // copies of step `issued` (cursor ic)
      const int h = ic.r * F_APPLY_WARPS + aw;
      if (h < p.heads) {                                   // else idle in the last round
        const bf16* qh = p.q + (long long)ic.b * p.qv.batch + (long long)h * p.qv.head + t * 8;
        const uint32_t dst = ring + (issued % F_QSTAGES) * F_QSTAGE_BYTES;
        const int n0 = ic.nt * FT + ic.st * F_STEP_TOKENS + gp;
#pragma unroll
        for (int u = 0; u < 2 * F_U; ++u) {                // u even: token g of tile u/2, odd: token g+8
          const int n = n0 + u * 8;
          const bool in = n < p.N;
          cp_async16(dst + u * 512, qh + (long long)(in ? n : 0) * p.qv.ld, in ? 16u : 0u);  // zero fill past the end
        }
      }
      ++issued;
      advance(ic);
    };
#pragma unroll
    for (int i = 0; i < F_QSTAGES - 1; ++i) {
      if (i < total_steps) issue();
      cp_async_commit();
    }

    uint32_t bf[F_FRAG_WORDS];  // word (ks*(NT+1) + j)*2 + e
    bool ok = true, head_ok = false;
    for (int stp = 0; stp < total_steps; ++stp, advance(cc)) {
      const int ti = cc.ti, r = cc.r, st = cc.st;
      if (issued < total_steps) issue();
      cp_async_commit();
      if (st == 0) {
        const int h = r * F_APPLY_WARPS + aw;
        head_ok = h < p.heads;
        if (head_ok) {
          const uint4* fp = p.frags + ((long long)cc.b * p.heads + h) * (F_FRAG_WORDS / 4 * 32) + lane;
#pragma unroll
          for (int v = 0; v < F_FRAG_WORDS / 4; ++v) {
            const uint4 x = fp[v * 32];
            bf[4 * v] = x.x; bf[4 * v + 1] = x.y; bf[4 * v + 2] = x.z; bf[4 * v + 3] = x.w;
          }
          // the MMAs that read this slice in its previous use must be done
          const uint32_t use = (uint32_t)(ti * uses_per_tile + r);
          ok = mbar_wait(bempty + 8 * s, (use & 1) ^ 1, &abort_flag);
        }
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      cp_async_wait<F_QSTAGES - 1>();
      if (!head_ok) continue;
      const uint32_t src = ring + (stp % F_QSTAGES) * F_QSTAGE_BYTES;
      uint32_t qa[F_U][4], qb[F_U][4];
#pragma unroll
      for (int u = 0; u < F_U; ++u) {
        lds128(qa[u], src + (2 * u) * 512);
        lds128(qb[u], src + (2 * u + 1) * 512);
      }
      float acc[F_U][NT + 1][4];
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        uint32_t A[F_U][4];
#pragma unroll
        for (int u = 0; u < F_U; ++u) {
          A[u][0] = relu2(qa[u][2 * ks]); A[u][1] = relu2(qb[u][2 * ks]);
          A[u][2] = relu2(qa[u][2 * ks + 1]); A[u][3] = relu2(qb[u][2 * ks + 1]);
        }
#pragma unroll
        for (int j = 0; j <= NT; ++j)
#pragma unroll
          for (int u = 0; u < F_U; ++u) {
            const int w = (ks * (NT + 1) + j) * 2;
            if (ks == 0) mma_bf16_first(acc[u][j], A[u], bf[w], bf[w + 1]);
            else mma_bf16(acc[u][j], A[u], bf[w], bf[w + 1]);
          }
      }
      // normalise and store into the slice: row = token of the tile (128 bytes = 64 channels of the pair),
      // this head's half = 16-byte chunks 4*(aw&1) + t, XOR-swizzled with the row as the 128B mode expects
#pragma unroll
      for (int u = 0; u < F_U; ++u) {
        const float inv_a = 1.f / (acc[u][NT][0] + p.eps), inv_b = 1.f / (acc[u][NT][2] + p.eps);
        uint32_t oa[4], ob[4];
#pragma unroll
        for (int j = 0; j < NT; ++j) {
          oa[j] = pack2(acc[u][j][0] * inv_a, acc[u][j][1] * inv_a);
          ob[j] = pack2(acc[u][j][2] * inv_b, acc[u][j][3] * inv_b);
        }
        const uint32_t ra = (uint32_t)(st * F_STEP_TOKENS + u * 16 + gp), rb = ra + 8;
        const uint32_t chunk = (uint32_t)(4 * (aw & 1) + t);
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(slice + ra * 128 + ((chunk ^ (ra & 7)) << 4)),
                     "r"(oa[0]), "r"(oa[1]), "r"(oa[2]), "r"(oa[3]) : "memory");
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(slice + rb * 128 + ((chunk ^ (rb & 7)) << 4)),
                     "r"(ob[0]), "r"(ob[1]), "r"(ob[2]), "r"(ob[3]) : "memory");
      }
      if (st == F_STEPS - 1) {  // this head's half of the slice is complete
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(bfull + 8 * s);
      }
    }
    cp_async_wait<0>();
  } else {
    // -------------------------------------------------------------- epilogue
    // Four warps; warp % 4 selects the TMEM lane quarter (a hardware rule).  A lane owns one output
    // channel; each 32-channel x 32-token block goes through a 64B-swizzled staging buffer and one
    // TMA store, which writes whole lines and clips channels >= Cout and tokens >= N.
    const int quarter = warp & 3;
    const uint32_t stage = staging + (uint32_t)(warp - 2 - F_APPLY_WARPS) * 2048;
    const uint32_t my_row = stage + lane * 64, sw = (uint32_t)((lane >> 1) & 3);
    bool ok = true;
    for (int ti = 0; ok && ti < my_tiles; ++ti) {
      const int tile = blockIdx.x + ti * gridDim.x;
      const int b = tile / p.tiles_per_batch, nt = tile % p.tiles_per_batch;
      const uint32_t acc = ti & 1, acc_ph = (ti >> 1) & 1;
      ok = mbar_wait(tfull + 8 * acc, acc_ph, &abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      for (int mt = 0; mt < p.m_tiles; ++mt) {
        const int row0 = mt * FBM + quarter * 32;
        const int m = row0 + lane;
        const float bias = (p.bias && m < p.Cout) ? __bfloat162float(p.bias[m]) : 0.f;
        const uint32_t taddr = tmem_base + acc * 256 + mt * FT + ((uint32_t)(quarter * 32) << 16);
        uint32_t r[2][32];
        tmem_ld32(taddr, r[0]);
#pragma unroll
        for (int c = 0; c < FT / 32; ++c) {
          tmem_ld_wait();
          if (c + 1 < FT / 32) tmem_ld32(taddr + (c + 1) * 32, r[(c + 1) & 1]);  // next chunk streams in meanwhile
          const uint32_t(&rc)[32] = r[c & 1];
          const int n0 = nt * FT + c * 32;
          if (n0 >= p.N || row0 >= p.Cout) continue;  // warp-uniform
          if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // staging buffer read out
          __syncwarp();
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e)
              w[e] = pack2(__uint_as_float(rc[v * 8 + 2 * e]) + bias, __uint_as_float(rc[v * 8 + 2 * e + 1]) + bias);
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(my_row + (((uint32_t)v ^ sw) << 4)), "r"(w[0]),
                         "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) {
            tma_store_3d(&tmO, stage, n0, row0, b);
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty + 8 * acc);  // this warp's quarter of the accumulators is drained
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
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

}  // namespace

bool apply_project_bf16_supported(int heads, int d, int Cout, int N, HeadView qv) {
  return d == FD && heads >= 2 && heads % 2 == 0 && Cout >= 1 && Cout <= 2 * FBM && N % 8 == 0 && qv.batch % 8 == 0 &&
         qv.head % 8 == 0 && qv.ld % 8 == 0;
}

// y[b][m][n] = sum_h sum_c w[m][32 h + c] * att[b][h][n][c] + bias[m], att = Eq. 3 applied to query head h with
// the state of (b, h) = sum over s < S of partial[(b * heads + h) * S + s] ([32][33] fp32 each: KV, then the
// key sum in column 32); y is NCHW [B, Cout, N].
// scratch: apply_project_scratch_bytes(B, heads) bytes of device memory, 16-byte aligned (the states as fragments).
size_t apply_project_scratch_bytes(int B, int heads) { return (size_t)B * heads * F_FRAG_WORDS * 32 * sizeof(uint32_t); }

msla_status_t run_apply_project_bf16(const void* q, const float* partial, int S, void* scratch, const void* w, const void* bias, void* y,
                                     HeadView qv, int B, int heads, int N, int Cout, float eps, cudaStream_t st) {
  const int K = heads * FD;
  CUtensorMap tmA, tmO;
  {
    const cuuint64_t dA[3] = {(cuuint64_t)K, (cuuint64_t)Cout, 1};
    const cuuint64_t sA[2] = {(cuuint64_t)K * 2, (cuuint64_t)K * Cout * 2};
    const cuuint32_t bA[3] = {(cuuint32_t)FBK, (cuuint32_t)FBM, 1};
    const cuuint64_t dO[3] = {(cuuint64_t)N, (cuuint64_t)Cout, (cuuint64_t)B};
    const cuuint64_t sO[2] = {(cuuint64_t)N * 2, (cuuint64_t)Cout * N * 2};
    const cuuint32_t bO[3] = {32, 32, 1};
    if (!tma_make_map_bf16(&tmA, w, 3, dA, sA, bA, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !tma_make_map_bf16(&tmO, y, 3, dO, sO, bO, CU_TENSOR_MAP_SWIZZLE_64B))
      return fail(MSLA_ERR_CUDA, "cuTensorMapEncodeTiled failed for the fused apply + output projection");
  }
  FusedParams p{};
  p.q = (const bf16*)q; p.frags = (const uint4*)scratch; p.bias = (const bf16*)bias; p.qv = qv;
  p.heads = heads; p.B = B; p.N = N; p.Cout = Cout; p.eps = eps;
  p.m_tiles = (Cout + FBM - 1) / FBM;
  p.tiles_per_batch = (N + FT - 1) / FT;
  const long long tiles = (long long)B * p.tiles_per_batch;
  if (tiles > 0x7fffffffLL) return fail(MSLA_ERR_UNSUPPORTED, "too many token tiles");
  p.num_tiles = (int)tiles;
  static unsigned long long attr_done = 0;  // devices on which the attribute is set (a race only repeats the call)
  const unsigned long long dev_bit = current_device_bit();
  if (!(attr_done & dev_bit)) {
    if (cudaFuncSetAttribute(apply_project_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, F_SMEM_BYTES) != cudaSuccess) {
      cudaGetLastError();
      return fail(MSLA_ERR_CUDA, "cannot reserve %d bytes of shared memory for the fused apply + output projection", F_SMEM_BYTES);
    }
    attr_done |= dev_bit;
  }
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
  const int grid = (int)(tiles < sms ? tiles : sms);
  launch_pdl(state_fragments_kernel, dim3((unsigned)(B * heads), FD / F_FRAG_ROWS), dim3(F_FRAG_THREADS), 0, st, partial, S, (uint32_t*)scratch);
  launch_pdl(apply_project_fused_kernel, dim3(grid), dim3(F_THREADS), F_SMEM_BYTES, st, tmA, tmO, p);
  count_launches(2);
  return check_launch("fused apply + output projection (tcgen05)");
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
