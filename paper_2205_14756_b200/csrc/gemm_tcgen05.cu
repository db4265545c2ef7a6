// bf16 GEMM for the module's 1x1 projections (Section 3.1: Q = xW_Q, K = xW_K,
// V = xW_V, and the final linear projection) on channel-major activations, on the
// 5th-generation tensor cores: TMA loads into 128B-swizzled shared memory,
// tcgen05.mma with fp32 accumulators in tensor memory, tcgen05.ld epilogue.
//
//   y[b][m][n] = sum_k w[m][k] * x[b][k][n] (+ bias[m]),   fp32 accumulate, bf16 out
//
// x is [B][K][N] and y is [B][M][N] (NCHW with N = H*W), so both the activation
// operand and the result have the token index contiguous.  The MMA takes
//   A = 128 rows of w (K-major: k contiguous),
//   B = a 256-token tile of x as an MN-major operand (n contiguous), four TMA
//       boxes of 64 k x 64 tokens per 64-wide k-slice,
//   D = 128 output channels (tensor-memory lanes) x 256 tokens (columns).
// The weight block of a CTA (<= 128 KB) stays in shared memory for the CTA's
// whole life when it fits (K <= 512): every CTA of a streaming kernel would
// otherwise re-read the same few weight lines from L2 at the same time.  CTA c
// serves weight block c % blocks and the token tiles c / blocks, + workers, ...
//
// One persistent CTA per SM, warp-specialised: warp 0 issues TMA, warp 1 issues
// MMAs (and owns the tensor-memory allocation), warps 2-9 drain the
// accumulators.  Two 128x256 fp32 accumulators (all 512 TMEM columns) let the
// epilogue of one tile overlap the MMAs of the next.  The epilogue converts to
// bf16, stages 32-channel x 64-token blocks in shared memory (128-byte rows,
// 128B swizzle) and writes them with TMA stores, which emit whole lines and
// clip at the tensor's edges.  Every mbarrier wait is bounded: on time-out the
// CTA raises a flag, all roles leave their loops, the tensor memory is released
// and the kernel returns.
#include <cuda.h>

#include "msla_common.cuh"
#include "msla_host.h"
#include "tma_host.h"
#include "tcgen05_util.cuh"

namespace msla {
namespace {

using bf16 = __nv_bfloat16;

constexpr int BM = 128, BN = 256, BK = 64;  // CTA tile; BK = one 128-byte swizzle span of bf16
constexpr int A_SLICE = BM * BK * 2;        // 16 KB: 128 weight rows x 64 k
constexpr int B_BOX = 64 * BK * 2;          // 8 KB: 64 k x 64 tokens
constexpr int B_SLICE = (BN / 64) * B_BOX;  // 32 KB
constexpr int NUM_THREADS = 320;            // TMA warp, MMA warp, 8 epilogue warps
constexpr int STAGING_WARP = 32 * 128;      // one 32-channel x 64-token block per epilogue warp
constexpr int STAGING_BYTES = 8 * STAGING_WARP;
constexpr int MAX_STAGES = 6;
constexpr int BAR_BYTES = 256;
constexpr int SMEM_BUDGET = 226 * 1024;  // 227 KB per CTA less the static shared memory and some slack
constexpr int RES_MAX_BYTES = 128 * 1024;

// Sticky: set when any wait in any GEMM launch of this process timed out.
__device__ int g_gemm_timeout_flag = 0;

struct GemmParams {
  int M, N, K;      // output channels, tokens per image, input channels
  int batches;
  int n_tiles;      // 256-token tiles per image
  int blocks;       // 128-row blocks of w
  int workers;      // CTAs per block
  int a_resident;   // 1: the CTA's weight block stays in shared memory
  int stages;       // ring depth
  const bf16* bias; // [M] or nullptr
};

__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_wx_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
               const __grid_constant__ CUtensorMap tmO, GemmParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;  // swizzle atoms need 1024-byte alignment
  const int k_iters = (p.K + BK - 1) / BK;
  const uint32_t res_base = smem_base;
  const uint32_t ring_base = res_base + (p.a_resident ? (uint32_t)(k_iters * A_SLICE) : 0u);
  const uint32_t stage_bytes = (uint32_t)B_SLICE + (p.a_resident ? 0u : (uint32_t)A_SLICE);
  const uint32_t staging = ring_base + (uint32_t)p.stages * stage_bytes;
  const uint32_t bars = staging + STAGING_BYTES;
  const uint32_t full_bar = bars, empty_bar = bars + 8 * MAX_STAGES;
  const uint32_t tfull_bar = bars + 16 * MAX_STAGES, tempty_bar = tfull_bar + 16;
  const uint32_t res_bar = tempty_bar + 16, tmem_slot = res_bar + 8;
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_sh;

  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int blk = blockIdx.x % p.blocks, worker = blockIdx.x / p.blocks;
  const int stream_total = p.batches * p.n_tiles;
  const uint32_t nstage = (uint32_t)p.stages;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < MAX_STAGES; ++s) { mbar_init(full_bar + 8 * s, 1); mbar_init(empty_bar + 8 * s, 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar + 8 * a, 1); mbar_init(tempty_bar + 8 * a, 8); }
    mbar_init(res_bar, 1);
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

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmX) : "memory");
      if (p.a_resident) {  // the weights are no earlier kernel's output: load them before the dependency wait
        mbar_expect_tx(res_bar, (uint32_t)(k_iters * A_SLICE));
        for (int kb = 0; kb < k_iters; ++kb) tma_load_3d(res_base + kb * A_SLICE, &tmW, res_bar, kb * BK, blk * BM, 0);
      }
      pdl_wait();  // the activations may come from the previous kernel
      uint32_t it = 0;
      bool ok = true;
      for (int si = worker; ok && si < stream_total; si += p.workers) {
        const int b = si / p.n_tiles, nt = si % p.n_tiles;
        for (int kb = 0; ok && kb < k_iters; ++kb, ++it) {
          const uint32_t s = it % nstage, ph = (it / nstage) & 1;
          ok = mbar_wait(empty_bar + 8 * s, ph ^ 1, &abort_flag);
          if (!ok) break;
          const uint32_t dst = ring_base + s * stage_bytes;
          mbar_expect_tx(full_bar + 8 * s, stage_bytes);
#pragma unroll
          for (int j = 0; j < BN / 64; ++j)  // boxes past the last token are filled with zeros
            tma_load_3d(dst + j * B_BOX, &tmX, full_bar + 8 * s, nt * BN + 64 * j, kb * BK, b);
          if (!p.a_resident) tma_load_3d(dst + B_SLICE, &tmW, full_bar + 8 * s, kb * BK, blk * BM, 0);
        }
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      // instruction descriptor: D = f32, A = B = bf16, A K-major, B MN-major, N = 256, M = 128
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      uint32_t it = 0, local = 0;
      bool ok = p.a_resident ? mbar_wait(res_bar, 0, &abort_flag) : true;
      for (int si = worker; ok && si < stream_total; si += p.workers, ++local) {
        const uint32_t acc = local & 1, acc_ph = (local >> 1) & 1;
        ok = mbar_wait(tempty_bar + 8 * acc, acc_ph ^ 1, &abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; ok && kb < k_iters; ++kb, ++it) {
          const uint32_t s = it % nstage, ph = (it / nstage) & 1;
          ok = mbar_wait(full_bar + 8 * s, ph, &abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t sb = ring_base + s * stage_bytes;
          const uint32_t sa = p.a_resident ? res_base + kb * A_SLICE : sb + B_SLICE;
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk) {
            // K-major w: 32 bytes further along the swizzled row; MN-major x: 16 k-rows of 128 bytes
            // further, 64-token blocks 8 KB apart, groups of 8 k-rows 1 KB apart
            const uint64_t ad = make_desc(sa + kk * 32, 1, 1024 >> 4);
            const uint64_t bd = make_desc(sb + kk * 2048, B_BOX >> 4, 1024 >> 4);
            umma_bf16(d_tmem, ad, bd, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
          }
          umma_commit(empty_bar + 8 * s);  // stage reusable once these MMAs have read it
        }
        if (ok) umma_commit(tfull_bar + 8 * acc);  // accumulator complete
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    // Eight warps: warp % 4 selects the TMEM lane quarter (a hardware rule), the other bit which 128
    // of the tile's 256 tokens the warp drains.  A lane owns one output channel; two 32-token chunks
    // fill a 32-channel x 64-token block (128-byte rows, 16-byte pieces XOR-swizzled with the row as
    // the TMA unit's 128B mode expects), written by one TMA store.
    const int quarter = warp & 3;
    const int col_half = (warp - 2) >> 2;
    const uint32_t stage = staging + (uint32_t)(warp - 2) * STAGING_WARP;
    const uint32_t my_row = stage + lane * 128, sw = (uint32_t)(lane & 7);
    const int row0 = blk * BM + quarter * 32;
    const float bias = (p.bias && row0 + lane < p.M) ? __bfloat162float(p.bias[row0 + lane]) : 0.f;
    uint32_t local = 0;
    bool ok = true;
    pdl_wait();  // no global write before the previous kernel is done with the output buffer
    for (int si = worker; ok && si < stream_total; si += p.workers, ++local) {
      const int b = si / p.n_tiles, nt = si % p.n_tiles;
      const uint32_t acc = local & 1, acc_ph = (local >> 1) & 1;
      ok = mbar_wait(tfull_bar + 8 * acc, acc_ph, &abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + acc * BN + col_half * 128 + ((uint32_t)(quarter * 32) << 16);
      const int ncol0 = nt * BN + col_half * 128;
      uint32_t r[2][32];
      tmem_ld32(taddr, r[0]);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        tmem_ld_wait();
        if (c + 1 < 4) tmem_ld32(taddr + (c + 1) * 32, r[(c + 1) & 1]);  // next chunk streams in meanwhile
        const uint32_t(&rc)[32] = r[c & 1];
        const int n0 = ncol0 + (c >> 1) * 64;   // first token of the 64-token block
        if (n0 >= p.N || row0 >= p.M) continue;  // warp-uniform: nothing of this block lies inside the tensor
        if ((c & 1) == 0) {  // the previous block must have been read out of the staging buffer
          if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          __syncwarp();
        }
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e)
            w[e] = pack2(__uint_as_float(rc[v * 8 + 2 * e]) + bias, __uint_as_float(rc[v * 8 + 2 * e + 1]) + bias);
          const uint32_t piece = (uint32_t)((c & 1) * 4 + v);
          asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(my_row + ((piece ^ sw) << 4)), "r"(w[0]), "r"(w[1]),
                       "r"(w[2]), "r"(w[3]) : "memory");
        }
        if (c & 1) {
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

}  // namespace

bool gemm_bf16_supported(int M, int N, int K) { return M >= 1 && N >= 8 && N % 8 == 0 && K >= 8 && K % 8 == 0; }

// y[b][m][n] = sum_k w[m][k] * x[b][k][n] + bias[m];  x: [B][K][N] with batch stride x_sb, y: [B][M][N] with
// batch stride y_sb (elements; multiples of 8), w: [M][K], bias: [M] or nullptr.
msla_status_t run_gemm_bf16(const void* x, const void* w, const void* bias, void* y, int B, int K, int M, int N,
                            long long x_sb, long long y_sb, cudaStream_t st) {
  if (!gemm_bf16_supported(M, N, K) || x_sb % 8 != 0 || y_sb % 8 != 0)
    return fail(MSLA_ERR_UNSUPPORTED, "projection GEMM: M = %d, N = %d, K = %d", M, N, K);
  CUtensorMap tmW, tmX, tmO;
  {
    const cuuint64_t dW[3] = {(cuuint64_t)K, (cuuint64_t)M, 1};
    const cuuint64_t sW[2] = {(cuuint64_t)K * 2, (cuuint64_t)K * M * 2};
    const cuuint32_t bW[3] = {BK, BM, 1};
    const cuuint64_t dX[3] = {(cuuint64_t)N, (cuuint64_t)K, (cuuint64_t)B};
    const cuuint64_t sX[2] = {(cuuint64_t)N * 2, (cuuint64_t)x_sb * 2};
    const cuuint32_t bX[3] = {64, BK, 1};
    const cuuint64_t dO[3] = {(cuuint64_t)N, (cuuint64_t)M, (cuuint64_t)B};
    const cuuint64_t sO[2] = {(cuuint64_t)N * 2, (cuuint64_t)y_sb * 2};
    const cuuint32_t bO[3] = {64, 32, 1};
    if (!tma_make_map_bf16(&tmW, w, 3, dW, sW, bW, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !tma_make_map_bf16(&tmX, x, 3, dX, sX, bX, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !tma_make_map_bf16(&tmO, y, 3, dO, sO, bO, CU_TENSOR_MAP_SWIZZLE_128B))
      return fail(MSLA_ERR_CUDA, "cuTensorMapEncodeTiled failed for the projection GEMM");
  }
  GemmParams p{};
  p.M = M; p.N = N; p.K = K; p.batches = B;
  p.n_tiles = (N + BN - 1) / BN;
  p.blocks = (M + BM - 1) / BM;
  p.bias = (const bf16*)bias;
  const int k_iters = (K + BK - 1) / BK;
  const int sms = device_sm_count();
  const long long stream_total = (long long)B * p.n_tiles;
  if (stream_total > 0x7fffffffLL) return fail(MSLA_ERR_UNSUPPORTED, "too many token tiles");
  p.a_resident = (k_iters * A_SLICE <= RES_MAX_BYTES && p.blocks <= sms) ? 1 : 0;
  const int fixed = STAGING_BYTES + BAR_BYTES + 1024 + (p.a_resident ? k_iters * A_SLICE : 0);
  const int stage_bytes = B_SLICE + (p.a_resident ? 0 : A_SLICE);
  int stages = (SMEM_BUDGET - fixed) / stage_bytes;
  p.stages = stages > MAX_STAGES ? MAX_STAGES : stages;
  const int smem = fixed + p.stages * stage_bytes;
  long long workers = p.a_resident ? sms / p.blocks : 1;
  if (!p.a_resident) {  // streaming: every CTA walks all (block, tile) pairs of its share; keep the block fixed per CTA all the same
    workers = sms / p.blocks;
    if (workers < 1) workers = 1;
  }
  if (workers > stream_total) workers = stream_total;
  p.workers = (int)workers;
  // with more blocks than SMs the grid is larger than one wave; CTAs do not depend on one another
  static std::atomic<unsigned long long> attr_done{0};
  msla_status_t s = ensure_smem_attr(attr_done, gemm_wx_kernel, SMEM_BUDGET);
  if (s != MSLA_OK) return s;
  launch_pdl(gemm_wx_kernel, dim3((unsigned)(p.workers * p.blocks)), dim3(NUM_THREADS), (size_t)smem, st, tmW, tmX, tmO, p);
  count_launches(1);
  return check_launch("projection GEMM (tcgen05)");
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
