// bf16 GEMM for the module's two 1x1 projections (Section 3.1: Q = xW_Q,
// K = xW_K, V = xW_V, and the final linear projection) on the 5th-generation
// tensor cores: TMA loads into 128B-swizzled shared memory, tcgen05.mma with
// fp32 accumulators in tensor memory, tcgen05.ld epilogue.
//
//   D[m][n] = sum_k A[m][k] * B[n][k] (+ bias),   fp32 accumulate, bf16 out,
//   out[batch * out_batch_stride + m * ld_out + n]                     (group == 0), or
//   out[batch * out_batch_stride + ((n / group) * M + m) * group + n % group]
//   (columns split into planes of `group` channels, each plane [M][group])
//
// Input projection : m = token, n = output channel; A = x taken straight from
//                    NCHW (the token index is contiguous: an "MN-major" operand),
//                    B = w_qkv (K-major).
// Output projection: m = output channel, n = token; A = w_proj (K-major),
//                    B = attention output (K-major): either token-major
//                    [N][2C'] or one [N][64] plane per pair of heads; D rows are NCHW
//                    planes, so a row of the tile is a run of tokens.
//
// One persistent CTA per SM, warp-specialised: warp 0 issues TMA, warp 1
// issues MMAs (and owns the tensor-memory allocation), warps 2-9 drain the
// accumulators.  Two 128x256 fp32 accumulators (all 512 TMEM columns) let the
// epilogue of one tile overlap the MMAs of the next.  The epilogue converts to
// bf16, stages 32x32 blocks in shared memory and writes them with TMA stores
// (whole lines; a lane-per-row store of 16-byte pieces was twice as slow).
// A second kernel keeps the CTA's weight block resident in shared memory and
// streams only activations (used for the input projection).  Every mbarrier wait is
// bounded: on time-out the CTA raises a flag, all roles leave their loops, the
// tensor memory is released and the kernel returns.
#include <cuda.h>

#include "msla_common.cuh"
#include "msla_host.h"
#include "tma_host.h"
#include "tcgen05_util.cuh"

namespace msla {
namespace {

using bf16 = __nv_bfloat16;

constexpr int BM = 128, BN = 256, BK = 64;  // CTA tile; BK = one 128-byte swizzle span of bf16
constexpr int STAGES = 4;
constexpr int A_STAGE_BYTES = BM * BK * 2;  // 16 KB
constexpr int B_STAGE_BYTES = BN * BK * 2;  // 32 KB
constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
constexpr int NUM_THREADS = 320;  // TMA warp, MMA warp, 8 epilogue warps
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 8 * 2048 + 256 + 1024;  // ring + epilogue staging + barriers + alignment slack

// Sticky: set when any wait in any GEMM launch of this process timed out.
__device__ int g_gemm_timeout_flag = 0;

struct GemmParams {
  int M, N, K;            // per batch
  int batches;
  int m_tiles, n_tiles;   // per batch
  long long out_batch_stride;  // elements between consecutive batches of the output
  long long ld_out;       // output row stride (elements) when group == 0
  int group;              // 0, or channels per output plane (16 or 32)
  int bias_per_row;       // 1: bias[m], 0: bias[n] (ignored when bias == nullptr)
  int n_fastest;          // tile order: 1 = consecutive tiles share the A tile, 0 = share the B tile
  const bf16* bias;
  bf16* out;
  int tma_store;          // 1: epilogue stages 32x32 blocks in shared memory and writes them with TMA (tmO)
  int planes_per_batch;   // planar output: plane coordinate of (batch, n) = batch*planes_per_batch + n/32
  int plane_shift;        // log2 of the channels per TMA-stored output plane (5: planes of 32, 6: planes of 64)
  float act_a, act_b;     // EPI 1: act(v) = v * sat(v * act_a + act_b)
  const bf16* residual;   // EPI 2: a tensor laid out like the row-major output, added after the bias
};

__device__ __forceinline__ void tile_coords(const GemmParams& p, int tile, int& b, int& mt, int& nt) {
  const int per_batch = p.m_tiles * p.n_tiles;
  b = tile / per_batch;
  const int r = tile % per_batch;
  if (p.n_fastest) { mt = r / p.n_tiles; nt = r % p.n_tiles; }
  else             { nt = r / p.m_tiles; mt = r % p.m_tiles; }
}

constexpr int STAGING_BYTES = 8 * 2048;  // one 32-row x 64-byte block per epilogue warp

// One epilogue warp's share of a finished 128x256 accumulator: TMEM lanes
// 32*quarter .. +31 (= tile rows), columns col_half*128 .. +127, converted to
// bf16 (+ bias).  A lane owns one row, so storing straight from registers
// scatters 16-byte pieces over 32 rows per instruction; instead each 32x32
// block is laid out in shared memory (64-byte rows, 16-byte chunks XOR-swizzled
// as the TMA unit's 64B mode expects) and written by one TMA store, which
// emits whole lines and clips rows and columns outside the tensor.  Without a
// store map (planes of 16 channels) the lane stores its vectors directly.
// EPI selects what else the epilogue does (compiled out of the plain projections):
//   0  nothing
//   1  column biases read from shared memory (bias_sm: the tile's 256 columns as fp32) and the activation
//      act(v) = v * sat(v * p.act_a + p.act_b), which is the identity for (0, 1), hard-swish for (1/6, 1/2) and ReLU
//      for (1e30, 0); the staging block is double-buffered (NBUF = 2) so that this arithmetic overlaps the previous
//      block's TMA store instead of lengthening the chain tmem load -> convert -> stage -> store
//   2  adds p.residual (laid out like the row-major output) after the bias
// F16: operands and output are IEEE binary16 instead of bfloat16 (16-bit values travel untyped; the MMA's operand
// format bits and the conversions differ).
// (The bf16 loads stay written as `__bfloat162float(p.bias[i])` at their sites: routed through this helper the input
// projection's epilogue came out 10 % slower, 0.109 -> 0.119 ms.)
template <bool F16> __device__ __forceinline__ float ld16(const bf16* p) {
  if constexpr (F16) return __half2float(*reinterpret_cast<const __half*>(p));
  else return __bfloat162float(*p);
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
template <bool F16> __device__ __forceinline__ void unpack16(uint32_t w, float& lo, float& hi) {
  if constexpr (F16) {
    const __half2 h = *reinterpret_cast<const __half2*>(&w);
    lo = __low2float(h); hi = __high2float(h);
  } else {
    lo = __uint_as_float(w << 16); hi = __uint_as_float(w & 0xffff0000u);
  }
}
template <bool F16> __device__ __forceinline__ constexpr uint32_t operand_format_bits() { return F16 ? 0u : ((1u << 7) | (1u << 10)); }

template <int EPI, int NBUF = 1, bool F16 = false>
__device__ __forceinline__ void drain_accumulator(const GemmParams& p, const CUtensorMap* tmO, uint32_t stage, int b,
                                                  int mt, int nt, uint32_t tmem_acc, int quarter, int col_half, int lane,
                                                  const float* bias_sm = nullptr) {
  const int gs = p.group == 32 ? 5 : 4;  // log2(group) when the output is planar
  const int row0 = mt * BM + quarter * 32;
  const int m = row0 + lane;
  const bool row_ok = m < p.M;
  bf16* obase = p.out + (long long)b * p.out_batch_stride;
  const float bias_row = (EPI != 1 && p.bias && p.bias_per_row && row_ok) ? (F16 ? ld16<true>(p.bias + m) : __bfloat162float(p.bias[m])) : 0.f;
  const bool bias_col = EPI != 1 && p.bias && !p.bias_per_row;
  const int ncol0 = nt * BN + col_half * 128;
  const uint32_t taddr = tmem_acc + col_half * 128 + ((uint32_t)(quarter * 32) << 16);
  const uint32_t sw = (uint32_t)((lane >> 1) & 3);
  uint32_t r[2][32];
  tmem_ld32(taddr, r[0]);
  // residual: the lane's row of the output-shaped tensor, 32 tokens (64 bytes) per chunk, fetched one chunk ahead
  const bf16* res_row = (EPI == 2 && p.residual && row_ok) ? p.residual + (long long)b * p.out_batch_stride + (long long)m * p.ld_out : nullptr;
  uint4 rs[2][4];
  auto load_residual = [&](int c) {
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const int n = ncol0 + c * 32 + v * 8;
      rs[c & 1][v] = (res_row && n < p.N) ? __ldg(reinterpret_cast<const uint4*>(res_row + n)) : make_uint4(0u, 0u, 0u, 0u);
    }
  };
  if (EPI == 2) load_residual(0);
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    tmem_ld_wait();
    if (c + 1 < 4) tmem_ld32(taddr + (c + 1) * 32, r[(c + 1) & 1]);  // next chunk streams in while this one is stored
    if (EPI == 2 && c + 1 < 4) load_residual(c + 1);
    const uint32_t(&rc)[32] = r[c & 1];
    const int n0 = ncol0 + c * 32;
    if (n0 >= p.N) continue;  // warp-uniform
    uint32_t w[4][4];
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      float bc[8];
      if (EPI == 1 && bias_sm) {  // same address in every lane: broadcast reads
        const float4 b0 = *reinterpret_cast<const float4*>(bias_sm + col_half * 128 + c * 32 + v * 8);
        const float4 b1 = *reinterpret_cast<const float4*>(bias_sm + col_half * 128 + c * 32 + v * 8 + 4);
        bc[0] = b0.x; bc[1] = b0.y; bc[2] = b0.z; bc[3] = b0.w; bc[4] = b1.x; bc[5] = b1.y; bc[6] = b1.z; bc[7] = b1.w;
      } else if (EPI == 1) {      // no staged copy (the kernel whose CTAs change weight block from tile to tile)
#pragma unroll
        for (int i = 0; i < 8; ++i) bc[i] = (p.bias && n0 + v * 8 < p.N) ? (F16 ? ld16<true>(p.bias + n0 + v * 8 + i) : __bfloat162float(p.bias[n0 + v * 8 + i])) : 0.f;
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float f0 = __uint_as_float(rc[v * 8 + 2 * e]), f1 = __uint_as_float(rc[v * 8 + 2 * e + 1]);
        if (EPI == 1) {
          f0 += bc[2 * e]; f1 += bc[2 * e + 1];
          f0 *= __saturatef(fmaf(f0, p.act_a, p.act_b));
          f1 *= __saturatef(fmaf(f1, p.act_a, p.act_b));
        } else {
          f0 += bias_row; f1 += bias_row;
          if (bias_col && n0 + v * 8 < p.N) {
            if constexpr (F16) { f0 += ld16<true>(p.bias + n0 + v * 8 + 2 * e); f1 += ld16<true>(p.bias + n0 + v * 8 + 2 * e + 1); }
            else { f0 += __bfloat162float(p.bias[n0 + v * 8 + 2 * e]); f1 += __bfloat162float(p.bias[n0 + v * 8 + 2 * e + 1]); }
          }
        }
        if (EPI == 2) {
          const uint32_t rw = e == 0 ? rs[c & 1][v].x : e == 1 ? rs[c & 1][v].y : e == 2 ? rs[c & 1][v].z : rs[c & 1][v].w;
          float r0f, r1f;
          unpack16<F16>(rw, r0f, r1f);
          f0 += r0f; f1 += r1f;
        }
        w[v][e] = pack16<F16>(f0, f1);
      }
    }
    if (p.tma_store) {
      const uint32_t buf = stage + (NBUF == 2 ? (uint32_t)(c & 1) * 2048u : 0u);
      // the block stored from this buffer before must have been read out of it
      if (lane == 0) {
        if (NBUF == 2) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        else           asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
      }
      __syncwarp();
#pragma unroll
      for (int v = 0; v < 4; ++v)
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(buf + lane * 64 + (((uint32_t)v ^ sw) << 4)), "r"(w[v][0]),
                     "r"(w[v][1]), "r"(w[v][2]), "r"(w[v][3]) : "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) {
        if (p.group) tma_store_3d(tmO, buf, n0 & ((1 << p.plane_shift) - 1), row0, b * p.planes_per_batch + (n0 >> p.plane_shift));
        else         tma_store_3d(tmO, buf, n0, row0, b);
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      }
    } else if (row_ok) {
#pragma unroll
      for (int v = 0; v < 4; ++v) {  // 4 x (8 columns = 16 bytes); N is a multiple of 8
        const int n = n0 + v * 8;
        if (n < p.N) {
          bf16* dst = p.group ? obase + (((long long)(n >> gs) * p.M + m) << gs) + (n & (p.group - 1))
                              : obase + (long long)m * p.ld_out + n;
          asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(dst), "r"(w[v][0]), "r"(w[v][1]), "r"(w[v][2]), "r"(w[v][3]) : "memory");
        }
      }
    }
  }
}

// B_PLANAR (output projection with the attention output kept as one [N][64]
// plane per pair of heads): the 64-wide k-slice kb of B is plane kb of the image.
template <bool A_MN_MAJOR, bool B_PLANAR, int EPI, bool F16>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_bf16_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                         const __grid_constant__ CUtensorMap tmO, GemmParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;  // swizzle atoms need 1024-byte alignment
  const uint32_t staging = smem_base + STAGES * STAGE_BYTES;
  const uint32_t bars = staging + STAGING_BYTES;
  const uint32_t full_bar = bars, empty_bar = bars + 8 * STAGES;
  const uint32_t tfull_bar = bars + 16 * STAGES, tempty_bar = tfull_bar + 16;
  const uint32_t tmem_slot = tempty_bar + 16;
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_sh;

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = p.batches * p.m_tiles * p.n_tiles;
  const int k_iters = (p.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar + 8 * s, 1); mbar_init(empty_bar + 8 * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar + 8 * a, 1); mbar_init(tempty_bar + 8 * a, 8); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // whole warp: allocate all 512 tensor-memory columns (one CTA per SM)
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
  pdl_wait();  // barriers and tensor memory are set up; the activations come from the previous kernel

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB) : "memory");
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        int b, mt, nt;
        tile_coords(p, tile, b, mt, nt);
        for (int kb = 0; ok && kb < k_iters; ++kb, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
          ok = mbar_wait(empty_bar + 8 * s, ph ^ 1, &abort_flag);
          if (!ok) break;
          const uint32_t sa = smem_base + s * STAGE_BYTES, sb = sa + A_STAGE_BYTES;
          mbar_expect_tx(full_bar + 8 * s, STAGE_BYTES);
          if (B_PLANAR) {    // 64 k x 128 weight rows, and one plane: 64 channels x 256 tokens
            tma_load_3d(sa, &tmA, full_bar + 8 * s, kb * BK, mt * BM, 0);
            tma_load_3d(sb, &tmB, full_bar + 8 * s, 0, nt * BN, b * p.planes_per_batch + kb);
          } else {
            if (A_MN_MAJOR) {  // two boxes of 64 tokens x 64 k
              tma_load_3d(sa, &tmA, full_bar + 8 * s, mt * BM, kb * BK, b);
              tma_load_3d(sa + A_STAGE_BYTES / 2, &tmA, full_bar + 8 * s, mt * BM + 64, kb * BK, b);
            } else {           // one box of 64 k x 128 rows
              tma_load_3d(sa, &tmA, full_bar + 8 * s, kb * BK, mt * BM, 0);
            }
            tma_load_3d(sb, &tmB, full_bar + 8 * s, kb * BK, nt * BN, A_MN_MAJOR ? 0 : b);
          }
        }
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      // instruction descriptor: D = f32, A = B = bf16, A major, B K-major, N = 256, M = 128
      const uint32_t idesc = (1u << 4) | operand_format_bits<F16>() | ((A_MN_MAJOR ? 1u : 0u) << 15) |
                             ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      uint32_t it = 0, local = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++local) {
        const uint32_t acc = local & 1, acc_ph = (local >> 1) & 1;
        ok = mbar_wait(tempty_bar + 8 * acc, acc_ph ^ 1, &abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; ok && kb < k_iters; ++kb, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
          ok = mbar_wait(full_bar + 8 * s, ph, &abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sa = smem_base + s * STAGE_BYTES, sb = sa + A_STAGE_BYTES;
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk) {
            // MN-major A: 16 k-slices of 128 B further on; K-major: 32 B along the swizzled row
            uint64_t ad, bd;
            ad = A_MN_MAJOR ? make_desc(sa + kk * 2048, (A_STAGE_BYTES / 2) >> 4, 1024 >> 4)
                            : make_desc(sa + kk * 32, 1, 1024 >> 4);
            bd = make_desc(sb + kk * 32, 1, 1024 >> 4);
            umma_bf16(d_tmem, ad, bd, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
          }
          umma_commit(empty_bar + 8 * s);  // stage reusable once these MMAs have read it
        }
        if (ok) umma_commit(tfull_bar + 8 * acc);  // accumulator complete
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    // Eight warps: warp%4 selects the TMEM lane quarter (a hardware rule), the
    // other bit selects which 128 of the tile's 256 columns the warp drains.
    const int quarter = warp & 3;
    const int col_half = (warp - 2) >> 2;
    uint32_t local = 0;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++local) {
      int b, mt, nt;
      tile_coords(p, tile, b, mt, nt);
      const uint32_t acc = local & 1, acc_ph = (local >> 1) & 1;
      ok = mbar_wait(tfull_bar + 8 * acc, acc_ph, &abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      drain_accumulator<EPI, 1, F16>(p, &tmO, staging + (warp - 2) * 2048, b, mt, nt, tmem_base + acc * BN, quarter, col_half, lane);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar + 8 * acc);  // this warp's share of the accumulator is drained
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // TMA stores done before the CTA retires
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    // give copies and MMAs still in flight time to land before memory is released
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    if (threadIdx.x == 0) atomicExch(&g_gemm_timeout_flag, 1);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}


// ---------------------------------------------------------------------------
// Weight-stationary variant.  Every CTA of the streaming kernel above re-reads
// the same weight slices from L2 at the same time, and those few hot lines
// serialise in their L2 slices.  Here a CTA owns one block of output channels
// for its whole life: that block of the weight matrix (<= 128 KB) is loaded
// into shared memory once, and only activation tiles stream through a ring.
// Used for the input projection: B = 256 weight rows resident (K <= 256), A = 128-token x tiles,
// MN-major, 16 KB stages (5 deep).  CTA c serves weight block c % blocks and the activation
// tiles c / blocks, c / blocks + workers, ...  Barriers, TMEM use and epilogue are as above.
// ---------------------------------------------------------------------------
constexpr int RES_BYTES = 128 * 1024;
constexpr int WS_RING_BYTES = 80 * 1024;
constexpr int WS_SMEM_BYTES = RES_BYTES + WS_RING_BYTES + STAGING_BYTES + 256 + 1024;
constexpr int WS_MAX_STAGES = 6;

template <int EPI, bool F16>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_bf16_stationary_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                            const __grid_constant__ CUtensorMap tmO, GemmParams p, int blocks, int workers) {
  constexpr int STREAM_BYTES = A_STAGE_BYTES;             // one k-slice of the streamed operand (the x tile)
  constexpr int NBUF = EPI == 1 ? 2 : 1;                  // staging blocks per epilogue warp
  constexpr int RING_BYTES = WS_RING_BYTES - (NBUF - 1) * STAGING_BYTES;  // the second staging block comes out of the ring
  constexpr int NSTAGE = RING_BYTES / STREAM_BYTES;       // 5 (4 with double-buffered staging)
  constexpr int RES_SLICE = B_STAGE_BYTES;                // one k-slice of the resident operand (256 weight rows)
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t res_base = smem_base, ring_base = smem_base + RES_BYTES;
  const uint32_t staging = ring_base + RING_BYTES;
  const uint32_t bars = staging + NBUF * STAGING_BYTES;
  const uint32_t full_bar = bars, empty_bar = bars + 8 * WS_MAX_STAGES;
  const uint32_t tfull_bar = bars + 16 * WS_MAX_STAGES, tempty_bar = tfull_bar + 16;
  const uint32_t res_bar = tempty_bar + 16, tmem_slot = res_bar + 8;
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_sh;
  __shared__ __align__(16) float bias_sm[EPI == 1 ? BN : 4];  // the CTA's 256 column biases (weights: not the previous kernel's output)

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int k_iters = (p.K + BK - 1) / BK;
  const int blk = blockIdx.x % blocks, worker = blockIdx.x / blocks;
  if (EPI == 1) {
    for (int i = threadIdx.x; i < BN; i += NUM_THREADS) {
      const int n = blk * BN + i;
      bias_sm[i] = (p.bias && !p.bias_per_row && n < p.N) ? (F16 ? ld16<true>(p.bias + n) : __bfloat162float(p.bias[n])) : 0.f;
    }
  }
  const int stream_per_batch = p.m_tiles;
  const int stream_total = p.batches * stream_per_batch;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < NSTAGE; ++s) { mbar_init(full_bar + 8 * s, 1); mbar_init(empty_bar + 8 * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar + 8 * a, 1); mbar_init(tempty_bar + 8 * a, 8); }
    mbar_init(res_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
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

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB) : "memory");
      // the resident weight block: all k-slices on one barrier
      mbar_expect_tx(res_bar, (uint32_t)(k_iters * RES_SLICE));
      for (int kb = 0; kb < k_iters; ++kb) tma_load_3d(res_base + kb * RES_SLICE, &tmB, res_bar, kb * BK, blk * BN, 0);
      pdl_wait();  // the streamed operand may come from the previous kernel; the weights above do not
      uint32_t it = 0;
      bool ok = true;
      for (int si = worker; ok && si < stream_total; si += workers) {
        const int b = si / stream_per_batch, st = si % stream_per_batch;
        for (int kb = 0; ok && kb < k_iters; ++kb, ++it) {
          const uint32_t s = it % NSTAGE, ph = (it / NSTAGE) & 1;
          ok = mbar_wait(empty_bar + 8 * s, ph ^ 1, &abort_flag);
          if (!ok) break;
          const uint32_t dst = ring_base + s * STREAM_BYTES;
          mbar_expect_tx(full_bar + 8 * s, STREAM_BYTES);
          // x tile: two boxes of 64 tokens x 64 k
          tma_load_3d(dst, &tmA, full_bar + 8 * s, st * BM, kb * BK, b);
          tma_load_3d(dst + STREAM_BYTES / 2, &tmA, full_bar + 8 * s, st * BM + 64, kb * BK, b);
        }
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | operand_format_bits<F16>() | (1u << 15) |
                             ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      uint32_t it = 0, local = 0;
      bool ok = mbar_wait(res_bar, 0, &abort_flag);
      for (int si = worker; ok && si < stream_total; si += workers, ++local) {
        const uint32_t acc = local & 1, acc_ph = (local >> 1) & 1;
        ok = mbar_wait(tempty_bar + 8 * acc, acc_ph ^ 1, &abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; ok && kb < k_iters; ++kb, ++it) {
          const uint32_t s = it % NSTAGE, ph = (it / NSTAGE) & 1;
          ok = mbar_wait(full_bar + 8 * s, ph, &abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t stream = ring_base + s * STREAM_BYTES, res = res_base + kb * RES_SLICE;
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk) {
            const uint64_t ad = make_desc(stream + kk * 2048, (A_STAGE_BYTES / 2) >> 4, 1024 >> 4);  // MN-major x tile
            const uint64_t bd = make_desc(res + kk * 32, 1, 1024 >> 4);
            umma_bf16(d_tmem, ad, bd, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
          }
          umma_commit(empty_bar + 8 * s);
        }
        if (ok) umma_commit(tfull_bar + 8 * acc);
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    const int quarter = warp & 3;
    const int col_half = (warp - 2) >> 2;
    uint32_t local = 0;
    bool ok = true;
    pdl_wait();  // no global write before the previous kernel is done with the output buffer
    for (int si = worker; ok && si < stream_total; si += workers, ++local) {
      const int b = si / stream_per_batch, st = si % stream_per_batch;
      const int mt = st, nt = blk;
      const uint32_t acc = local & 1, acc_ph = (local >> 1) & 1;
      ok = mbar_wait(tfull_bar + 8 * acc, acc_ph, &abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      drain_accumulator<EPI, NBUF, F16>(p, &tmO, staging + (warp - 2) * 2048 * NBUF, b, mt, nt, tmem_base + acc * BN, quarter, col_half, lane, bias_sm);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar + 8 * acc);
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    if (threadIdx.x == 0) atomicExch(&g_gemm_timeout_flag, 1);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

// ------------------------------------------------------------------- host side
// 3-D bf16 tensor map, 128-byte swizzle, zero fill outside the tensor.
// dims/box are innermost first; strides (bytes) are for dims 1 and 2.
bool make_map(CUtensorMap* map, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t s1, uint64_t s2,
              uint32_t b0, uint32_t b1) {
  const cuuint64_t dims[3] = {d0, d1, d2};
  const cuuint64_t strides[2] = {s1, s2};
  const cuuint32_t box[3] = {b0, b1, 1};
  return tma_make_map_bf16(map, base, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
}

template <int EPI, bool F16>
msla_status_t launch_stationary(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmO, const GemmParams& p,
                                int blocks, cudaStream_t st) {
  static std::atomic<unsigned long long> attr_done{0};
  const msla_status_t as = ensure_smem_attr(attr_done, gemm_bf16_stationary_kernel<EPI, F16>, WS_SMEM_BYTES);
  if (as != MSLA_OK) return as;
  const long long stream_total = (long long)p.batches * p.m_tiles;
  long long workers = device_sm_count() / blocks;
  if (workers > stream_total) workers = stream_total;
  launch_pdl(gemm_bf16_stationary_kernel<EPI, F16>, dim3((unsigned)(workers * blocks)), dim3(NUM_THREADS), WS_SMEM_BYTES, st, tmA, tmB, tmO, p, blocks, (int)workers);
  count_launches(1);
  return check_launch("projection GEMM (tcgen05, stationary weights)");
}

template <bool A_MN, bool B_PLANAR = false, int EPI = 0, bool F16 = false>
msla_status_t launch(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmO, const GemmParams& p, cudaStream_t st) {
  // weight-stationary kernel when the CTA's weight block fits its 128 KB of shared memory
  const int blocks = A_MN ? p.n_tiles : p.m_tiles;
  const int k_iters = (p.K + BK - 1) / BK;
  if (A_MN && k_iters * B_STAGE_BYTES <= RES_BYTES && blocks <= 16 && blocks <= device_sm_count())
    return launch_stationary<EPI, F16>(tmA, tmB, tmO, p, blocks, st);
  static std::atomic<unsigned long long> attr_done{0};
  const msla_status_t as = ensure_smem_attr(attr_done, gemm_bf16_tcgen05_kernel<A_MN, B_PLANAR, EPI, F16>, SMEM_BYTES);
  if (as != MSLA_OK) return as;
  const long long tiles = (long long)p.batches * p.m_tiles * p.n_tiles;
  const int grid = (int)(tiles < device_sm_count() ? tiles : device_sm_count());
  launch_pdl(gemm_bf16_tcgen05_kernel<A_MN, B_PLANAR, EPI, F16>, dim3(grid), dim3(NUM_THREADS), SMEM_BYTES, st, tmA, tmB, tmO, p);
  count_launches(1);
  return check_launch("projection GEMM (tcgen05)");
}

}  // namespace

bool project_in_bf16_supported(int C, int Cout, int N, int d) {
  return C % 8 == 0 && Cout % 8 == 0 && N % 8 == 0 && (d == 16 || d == 32) && Cout % d == 0;
}

// y[b][o / d][n][o % d] = sum_c w[o][c] * x[b][c][n];  x NCHW [B, C, N], y planar with batch stride y_sb.
msla_status_t run_project_in_bf16(const void* x, const void* w, void* y, int B, int C, int Cout, int N, int d,
                                  long long y_sb, cudaStream_t st, bool f16) {
  CUtensorMap tmA, tmB;
  if (!make_map(&tmA, x, (uint64_t)N, (uint64_t)C, (uint64_t)B, (uint64_t)N * 2, (uint64_t)C * N * 2, 64, BK) ||
      !make_map(&tmB, w, (uint64_t)C, (uint64_t)Cout, 1, (uint64_t)C * 2, (uint64_t)C * Cout * 2, BK, BN))
    return fail(MSLA_ERR_CUDA, "cuTensorMapEncodeTiled failed for the input projection");
  GemmParams p{};
  p.M = N; p.N = Cout; p.K = C; p.batches = B;
  p.m_tiles = (N + BM - 1) / BM; p.n_tiles = (Cout + BN - 1) / BN;
  p.out_batch_stride = y_sb; p.ld_out = 0; p.group = d; p.bias_per_row = 0; p.n_fastest = 1;
  p.bias = nullptr; p.out = (bf16*)y;
  // planes of 32 channels are written as 32-token x 32-channel blocks by TMA
  CUtensorMap tmO = tmA;  // placeholder when the direct-store epilogue is used
  const long long plane_elems = (long long)N * 32;
  if (d == 32 && y_sb % plane_elems == 0) {
    p.tma_store = 1; p.plane_shift = 5;
    p.planes_per_batch = (int)(y_sb / plane_elems);
    const cuuint64_t dims[3] = {32, (cuuint64_t)N, (cuuint64_t)B * p.planes_per_batch};
    const cuuint64_t strides[2] = {64, (cuuint64_t)N * 64};
    const cuuint32_t box[3] = {32, 32, 1};
    if (!tma_make_map_bf16(&tmO, y, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_64B))
      return fail(MSLA_ERR_CUDA, "cuTensorMapEncodeTiled failed for the input projection's output");
  }
  return f16 ? launch<true, false, 0, true>(tmA, tmB, tmO, p, st) : launch<true>(tmA, tmB, tmO, p, st);
}

bool project_out_bf16_supported(int Cin, int Cout, int N) { return Cin % 8 == 0 && N % 8 == 0 && Cout >= 1; }

// y[b][m][n] = sum_j w[m][j] * a[b][n][j] + bias[m];  a token-major [B, N, Cin], y NCHW [B, Cout, N].
msla_status_t run_project_out_bf16(const void* a, const void* w, const void* bias, const void* residual, void* y, int B, int Cin,
                                   int Cout, int N, cudaStream_t st, bool f16) {
  CUtensorMap tmA, tmB;
  if (!make_map(&tmA, w, (uint64_t)Cin, (uint64_t)Cout, 1, (uint64_t)Cin * 2, (uint64_t)Cin * Cout * 2, BK, BM) ||
      !make_map(&tmB, a, (uint64_t)Cin, (uint64_t)N, (uint64_t)B, (uint64_t)Cin * 2, (uint64_t)N * Cin * 2, BK, BN))
    return fail(MSLA_ERR_CUDA, "cuTensorMapEncodeTiled failed for the output projection");
  GemmParams p{};
  p.M = Cout; p.N = N; p.K = Cin; p.batches = B;
  p.m_tiles = (Cout + BM - 1) / BM; p.n_tiles = (N + BN - 1) / BN;
  p.out_batch_stride = (long long)Cout * N; p.ld_out = N; p.group = 0; p.bias_per_row = 1; p.n_fastest = 0;
  p.bias = (const bf16*)bias; p.out = (bf16*)y;
  CUtensorMap tmO;  // NCHW output as [batch][channel][token]; blocks of 32 channels x 32 tokens
  {
    p.tma_store = 1;
    const cuuint64_t dims[3] = {(cuuint64_t)N, (cuuint64_t)Cout, (cuuint64_t)B};
    const cuuint64_t strides[2] = {(cuuint64_t)N * 2, (cuuint64_t)Cout * N * 2};
    const cuuint32_t box[3] = {32, 32, 1};
    if (!tma_make_map_bf16(&tmO, y, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_64B))
      return fail(MSLA_ERR_CUDA, "cuTensorMapEncodeTiled failed for the output projection's output");
  }
  p.residual = (const bf16*)residual;
  if (f16) return residual ? launch<false, false, 2, true>(tmA, tmB, tmO, p, st) : launch<false, false, 0, true>(tmA, tmB, tmO, p, st);
  return residual ? launch<false, false, 2>(tmA, tmB, tmO, p, st) : launch<false>(tmA, tmB, tmO, p, st);
}

bool project_out_planar_bf16_supported(int Cin, int Cout, int N) { return Cin % 64 == 0 && N % 8 == 0 && Cout >= 1; }

// Same product with the attention output kept planar: a[b][j / 64][n][j % 64] (one [N][64] plane per pair of heads).
msla_status_t run_project_out_planar_bf16(const void* a, const void* w, const void* bias, const void* residual, void* y, int B,
                                          int Cin, int Cout, int N, cudaStream_t st, bool f16) {
  CUtensorMap tmA, tmB, tmO;
  const int planes = Cin / 64;
  {
    const cuuint64_t dO[3] = {(cuuint64_t)N, (cuuint64_t)Cout, (cuuint64_t)B};
    const cuuint64_t sO[2] = {(cuuint64_t)N * 2, (cuuint64_t)Cout * N * 2};
    const cuuint32_t bO[3] = {32, 32, 1};
    if (!make_map(&tmA, w, (uint64_t)Cin, (uint64_t)Cout, 1, (uint64_t)Cin * 2, (uint64_t)Cin * Cout * 2, BK, BM) ||
        !make_map(&tmB, a, 64, (uint64_t)N, (uint64_t)B * planes, 128, (uint64_t)N * 128, BK, BN) ||
        !tma_make_map_bf16(&tmO, y, 3, dO, sO, bO, CU_TENSOR_MAP_SWIZZLE_64B))
      return fail(MSLA_ERR_CUDA, "cuTensorMapEncodeTiled failed for the output projection");
  }
  GemmParams p{};
  p.M = Cout; p.N = N; p.K = Cin; p.batches = B;
  p.m_tiles = (Cout + BM - 1) / BM; p.n_tiles = (N + BN - 1) / BN;
  p.out_batch_stride = (long long)Cout * N; p.ld_out = N; p.group = 0; p.bias_per_row = 1; p.n_fastest = 0;
  p.bias = (const bf16*)bias; p.out = (bf16*)y;
  p.tma_store = 1; p.planes_per_batch = planes;
  p.residual = (const bf16*)residual;
  if (f16) return residual ? launch<false, true, 2, true>(tmA, tmB, tmO, p, st) : launch<false, true, 0, true>(tmA, tmB, tmO, p, st);
  return residual ? launch<false, true, 2>(tmA, tmB, tmO, p, st) : launch<false, true>(tmA, tmB, tmO, p, st);
}

// ---- the two linear layers of the FFN with a depthwise convolution (Section 3.1, Fig. 2 left)
bool ffn_bf16_supported(int C, int Ch, int Cout, int N) {
  return C % 8 == 0 && Ch % 64 == 0 && Cout % 8 == 0 && N % 8 == 0;
}

// First layer: h[b][o / 32][n][o % 32] = act(sum_c w1[o][c] * x[b][c][n] + b1[o]); x NCHW, h planes of 32 channels
// (dense 2 KB per 32 tokens for the epilogue's TMA stores: half-line stores into 64-channel planes cost this GEMM 2x).
msla_status_t run_ffn_expand_bf16(const void* x, const void* w1, const void* b1, void* h, int B, int C, int Ch, int N, int act,
                                  cudaStream_t st, bool f16) {
  CUtensorMap tmA, tmB, tmO;
  const cuuint64_t dims[3] = {32, (cuuint64_t)N, (cuuint64_t)B * (Ch / 32)};
  const cuuint64_t strides[2] = {64, (cuuint64_t)N * 64};
  const cuuint32_t box[3] = {32, 32, 1};
  if (!make_map(&tmA, x, (uint64_t)N, (uint64_t)C, (uint64_t)B, (uint64_t)N * 2, (uint64_t)C * N * 2, 64, BK) ||
      !make_map(&tmB, w1, (uint64_t)C, (uint64_t)Ch, 1, (uint64_t)C * 2, (uint64_t)C * Ch * 2, BK, BN) ||
      !tma_make_map_bf16(&tmO, h, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_64B))
    return fail(MSLA_ERR_CUDA, "cuTensorMapEncodeTiled failed for the FFN's first layer");
  GemmParams p{};
  p.M = N; p.N = Ch; p.K = C; p.batches = B;
  p.m_tiles = (N + BM - 1) / BM; p.n_tiles = (Ch + BN - 1) / BN;
  p.out_batch_stride = (long long)Ch * N; p.ld_out = 0; p.group = 32; p.bias_per_row = 0; p.n_fastest = 1;
  p.bias = (const bf16*)b1; p.out = (bf16*)h;
  p.tma_store = 1; p.planes_per_batch = Ch / 32; p.plane_shift = 5;
  p.act_a = act == 2 ? 1.f / 6.f : (act == 1 ? 1e30f : 0.f);  // act(v) = v * sat(v * act_a + act_b)
  p.act_b = act == 2 ? 0.5f : (act == 1 ? 0.f : 1.f);
  p.residual = nullptr;
  return f16 ? launch<true, false, 1, true>(tmA, tmB, tmO, p, st) : launch<true, false, 1>(tmA, tmB, tmO, p, st);
}

// Second layer: y[b][m][n] = sum_j w2[m][j] * g[b][j / 64][n][j % 64] + b2[m] (+ residual[b][m][n]); g planes of 64 channels, y NCHW.
msla_status_t run_ffn_project_bf16(const void* g, const void* w2, const void* b2, const void* residual, void* y, int B, int Ch,
                                   int Cout, int N, cudaStream_t st, bool f16) {
  CUtensorMap tmA, tmB, tmO;
  const int planes = Ch / 64;
  const cuuint64_t dO[3] = {(cuuint64_t)N, (cuuint64_t)Cout, (cuuint64_t)B};
  const cuuint64_t sO[2] = {(cuuint64_t)N * 2, (cuuint64_t)Cout * N * 2};
  const cuuint32_t bO[3] = {32, 32, 1};
  if (!make_map(&tmA, w2, (uint64_t)Ch, (uint64_t)Cout, 1, (uint64_t)Ch * 2, (uint64_t)Ch * Cout * 2, BK, BM) ||
      !make_map(&tmB, g, 64, (uint64_t)N, (uint64_t)B * planes, 128, (uint64_t)N * 128, BK, BN) ||
      !tma_make_map_bf16(&tmO, y, 3, dO, sO, bO, CU_TENSOR_MAP_SWIZZLE_64B))
    return fail(MSLA_ERR_CUDA, "cuTensorMapEncodeTiled failed for the FFN's second layer");
  GemmParams p{};
  p.M = Cout; p.N = N; p.K = Ch; p.batches = B;
  p.m_tiles = (Cout + BM - 1) / BM; p.n_tiles = (N + BN - 1) / BN;
  p.out_batch_stride = (long long)Cout * N; p.ld_out = N; p.group = 0; p.bias_per_row = 1; p.n_fastest = 0;
  p.bias = (const bf16*)b2; p.out = (bf16*)y;
  p.tma_store = 1; p.planes_per_batch = planes;
  p.residual = (const bf16*)residual;
  return f16 ? launch<false, true, 2, true>(tmA, tmB, tmO, p, st) : launch<false, true, 2>(tmA, tmB, tmO, p, st);
}

// Self-test of the bounded wait every kernel of the library relies on: one thread waits, with the given cycle
// limit, on a barrier nothing ever arrives at, and reports how the wait ended.  No product kernel is involved.
namespace {
__global__ void wait_selftest_kernel(long long limit_cycles, int* result) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const bool ok = mbar_wait_limit(smem_u32(&bar), 0, &abort_flag, limit_cycles);
    result[0] = ok ? 0 : 1;     // 1: the wait gave up
    result[1] = abort_flag;     // and raised the flag the other roles of a kernel poll
  }
}
}  // namespace

// 1 if a wait on a barrier nobody arrives at gave up after `limit_cycles` and raised the abort flag (the expected
// outcome), 0 if it claimed success, -1 on a CUDA error.  `scratch` is device memory for two ints.
int run_wait_selftest(long long limit_cycles, int* scratch, cudaStream_t st) {
  wait_selftest_kernel<<<1, 32, 0, st>>>(limit_cycles, scratch);
  int host[2] = {-1, -1};
  if (cudaMemcpyAsync(host, scratch, sizeof(host), cudaMemcpyDeviceToHost, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  return (host[0] == 1 && host[1] == 1) ? 1 : 0;
}

// Non-zero once any projection GEMM of this process hit a wait time-out (synchronises the device).
int gemm_timeout_flag() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_gemm_timeout_flag, sizeof(int)) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  return v;
}

}  // namespace msla
