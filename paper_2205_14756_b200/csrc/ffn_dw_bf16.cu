// The depthwise convolution inserted into the FFN (Section 3.1: a depthwise convolution in each FFN layer supplies
// the local information ReLU linear attention lacks; Fig. 2 left), with the bias (a folded normalisation) and the
// activation that follow it:
//
//   g[b][c][y][x] = act( sum_{dy,dx} w[c][dy][dx] * h[b][c][y+dy-1][x+dx-1] + bias[c] ),   3x3, zero padding 1
//
// Input: the hidden tensor as planes of 32 channels, h[b][c / 32][y*W + x][c % 32] (what the first linear layer's
// epilogue writes: dense 64-byte token rows); output: planes of 64 channels, g[b][c / 64][y*W + x][c % 64] (what the
// second linear layer's tile loads want: 128-byte token rows).  The change of plane width costs nothing here.
//
// The filter has no contraction over channels, so there is nothing for the tensor cores: at 9 multiply-adds per
// element read and written (2.25 MAC per byte) the step is bound by HBM if enough bytes are in flight and every
// input element is touched few times.  Persistent CTAs, one per SM, each with a contiguous run of 32 x 8 pixel tiles:
//   warp 16     TMA producer: per tile, image row and input plane one 4-D box [32 channels][34 px] (the tile with its
//               halo; rows and columns outside the image are zero-filled by the TMA unit = the zero padding), 64B
//               swizzle, each into a 40-pixel slot so that a pixel's swizzle phase is the same in every row and the
//               consumers' addresses are constants plus a per-thread offset; 4-deep ring
//   warps 0-15  a thread owns 4 channels (8 bytes) of one pixel column and walks the tile's rows with the three
//               filter rows' partial sums in registers: 3 shared-memory loads per output instead of 9; the 36 taps
//               of its channels sit in registers as fp32; bias, activation, bf16, one 8-byte store per output
//               (a warp writes 256 contiguous bytes).  With 8 channels per thread the registers allow 8 warps only,
//               too few to hide the latencies of the dependent load -> multiply-add -> store chain.
// Every mbarrier wait is bounded; on time-out the CTA raises a flag and all roles leave their loops.
#include <cuda.h>

#include "msla_common.cuh"
#include "msla_host.h"
#include "tma_host.h"
#include "tcgen05_util.cuh"

namespace msla {
namespace {

using bf16 = __nv_bfloat16;

constexpr int DW_PX = 32;      // output pixel columns per tile
constexpr int DW_ROWS = 8;     // output rows per tile
constexpr int DW_BOX_PX = DW_PX + 2, DW_BOX_ROWS = DW_ROWS + 2;
constexpr int DW_ROW_BYTES = DW_BOX_PX * 64;                               // one image row of one input plane's box: 2 176
constexpr int DW_ROW_PITCH = 40 * 64;                                      // its slot: a multiple of the 64B-swizzle atom (8 pixels =
                                                                           // 512 bytes), so the swizzle phase of a pixel does not depend on the row
constexpr int DW_HALF_STRIDE = DW_BOX_ROWS * DW_ROW_PITCH;                 // one input plane's rows: 25 600
constexpr int DW_TILE_BYTES = 2 * DW_BOX_ROWS * DW_ROW_BYTES;              // bytes the TMA unit delivers per tile
constexpr int DW_STAGE_BYTES = 2 * DW_HALF_STRIDE;                         // 51 200
constexpr int DW_STAGES = 4;
constexpr int DW_CPT = 4;                                                  // channels per thread
constexpr int DW_CONSUMERS = DW_PX * (64 / DW_CPT);                        // 512 threads: 16 warps to hide the latencies
constexpr int DW_THREADS = DW_CONSUMERS + 32;
constexpr int DW_SMEM = DW_STAGES * DW_STAGE_BYTES + 256 + 1024;

__device__ int g_dw_timeout_flag = 0;


__device__ __forceinline__ void tma_load_tile(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

// F16: the 16-bit storage type is IEEE binary16 instead of bfloat16 (values travel untyped; only the conversions differ).
template <bool F16> __device__ __forceinline__ void unpack16(uint32_t w, float& lo, float& hi) {
  if constexpr (F16) {
    const __half2 h = *reinterpret_cast<const __half2*>(&w);
    lo = __low2float(h); hi = __high2float(h);
  } else {
    lo = __uint_as_float(w << 16); hi = __uint_as_float(w & 0xffff0000u);
  }
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

struct DwParams {
  const bf16* w_dw;  // [Ch][3][3]
  const bf16* b_dw;  // [Ch] or nullptr
  bf16* g;
  int H, W, planes;
  float act_a, act_b;  // act(v) = v * sat(v * act_a + act_b): identity (0, 1), hard-swish (1/6, 1/2), ReLU (1e30, 0)
  int tiles_x, tiles_y;
  long long num_tiles;
};

template <bool F16>
__global__ void __launch_bounds__(DW_THREADS, 1)
ffn_dw3x3_kernel(const __grid_constant__ CUtensorMap tmH, DwParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bars = ring + DW_STAGES * DW_STAGE_BYTES;
  const uint32_t full_bar = bars, empty_bar = bars + 8 * DW_STAGES;
  __shared__ int abort_flag;
  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < DW_STAGES; ++s) { mbar_init(full_bar + 8 * s, 1); mbar_init(empty_bar + 8 * s, DW_CONSUMERS / 32); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // contiguous run of tiles: down a column of tiles first (the two halo rows a tile shares with the one above were
  // loaded a moment ago), then the next column, then the next (image, plane)
  const long long t_first = p.num_tiles * blockIdx.x / gridDim.x, t_end = p.num_tiles * (blockIdx.x + 1) / gridDim.x;
  const int per_z = p.tiles_x * p.tiles_y;
  pdl_wait();  // h is the previous kernel's output; g may still be read by an earlier one

  if (warp == DW_CONSUMERS / 32) {
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmH) : "memory");
      uint32_t it = 0;
      for (long long t = t_first; t < t_end; ++t, ++it) {
        const uint32_t s = it % DW_STAGES, ph = (it / DW_STAGES) & 1;
        if (!mbar_wait(empty_bar + 8 * s, ph ^ 1, &abort_flag)) break;
        const int z = (int)(t / per_z), r = (int)(t % per_z);
        const int tx = r / p.tiles_y, ty = r % p.tiles_y;
        mbar_expect_tx(full_bar + 8 * s, DW_TILE_BYTES);
        for (int row = 0; row < DW_BOX_ROWS; ++row) {  // one box per image row and input plane, each into its own slot
          const uint32_t dst = ring + s * DW_STAGE_BYTES + row * DW_ROW_PITCH;
          tma_load_tile(dst, &tmH, full_bar + 8 * s, 0, tx * DW_PX - 1, ty * DW_ROWS - 1 + row, 2 * z);
          tma_load_tile(dst + DW_HALF_STRIDE, &tmH, full_bar + 8 * s, 0, tx * DW_PX - 1, ty * DW_ROWS - 1 + row, 2 * z + 1);
        }
      }
    }
  } else {
    // lane bits: [2:0] 8-byte piece (4 channels) of the plane's 64-byte row, [3] pixel bit 0, [4] input plane of the
    // pair: sixteen consecutive lanes read 128 contiguous bytes of shared memory, a warp writes 256 contiguous bytes
    const int piece = lane & 7, side = lane >> 4;
    const int ch = side * 32 + piece * 4;       // first of the thread's 4 channels inside the 64-channel output plane
    const int px = warp * 2 + ((lane >> 3) & 1);
    uint32_t pre[3];  // offset of the thread's 8 bytes of pixel px + dx inside a row slot (64B swizzle: 16-byte chunk XOR pixel bits 1-2)
#pragma unroll
    for (int dx = 0; dx < 3; ++dx)
      pre[dx] = (uint32_t)(px + dx) * 64u + ((((uint32_t)piece >> 1) ^ (((uint32_t)(px + dx) >> 1) & 3u)) << 4) + (((uint32_t)piece & 1u) << 3);
    float wt[9][4], bias[4];
    int plane_loaded = -1;
    uint32_t it = 0;
    bool ok = true;
    for (long long t = t_first; ok && t < t_end; ++t, ++it) {
      const uint32_t s = it % DW_STAGES, ph = (it / DW_STAGES) & 1;
      const int z = (int)(t / per_z), r0 = (int)(t % per_z);
      const int tx = r0 / p.tiles_y, ty = r0 % p.tiles_y;
      const int plane = z % p.planes;
      if (plane != plane_loaded) {  // the thread's 4 channels x 9 taps: 72 contiguous bytes of the weight tensor
        const uint2* wp = reinterpret_cast<const uint2*>(p.w_dw + (long long)(plane * 64 + ch) * 9);
        float flat[36];  // element e = channel e / 9, tap e % 9
#pragma unroll
        for (int v = 0; v < 9; ++v) {
          const uint2 q = __ldg(wp + v);
          unpack16<F16>(q.x, flat[4 * v], flat[4 * v + 1]);
          unpack16<F16>(q.y, flat[4 * v + 2], flat[4 * v + 3]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int tp = 0; tp < 9; ++tp) wt[tp][i] = flat[i * 9 + tp];
        if (p.b_dw) {
          const uint2 q = __ldg(reinterpret_cast<const uint2*>(p.b_dw + plane * 64 + ch));
          unpack16<F16>(q.x, bias[0], bias[1]);
          unpack16<F16>(q.y, bias[2], bias[3]);
        } else {
#pragma unroll
          for (int i = 0; i < 4; ++i) bias[i] = 0.f;
        }
        plane_loaded = plane;
      }
      ok = mbar_wait(full_bar + 8 * s, ph, &abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const uint32_t tile = ring + s * DW_STAGE_BYTES + side * DW_HALF_STRIDE;
      const int x = tx * DW_PX + px, y0 = ty * DW_ROWS;
      bf16* gp = p.g + ((long long)z * p.H * p.W) * 64 + ch;
      float acc[3][4];  // acc[o % 3]: output row o under construction
#pragma unroll
      for (int r = 0; r < DW_BOX_ROWS; ++r) {  // box row r = image row y0 - 1 + r: filter row dy of output row r - dy
        float in[3][4];
#pragma unroll
        for (int dx = 0; dx < 3; ++dx) {
          uint2 v;
          asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(tile + r * DW_ROW_PITCH + pre[dx]));
          unpack16<F16>(v.x, in[dx][0], in[dx][1]);
          unpack16<F16>(v.y, in[dx][2], in[dx][3]);
        }
#pragma unroll
        for (int dy = 0; dy < 3; ++dy) {
          const int o = r - dy;
          if (o < 0 || o >= DW_ROWS) continue;
          float (&a)[4] = acc[o % 3];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            float v = dy == 0 ? bias[i] : a[i];  // filter row 0 opens the accumulator
            v = fmaf(wt[dy * 3 + 0][i], in[0][i], v);
            v = fmaf(wt[dy * 3 + 1][i], in[1][i], v);
            v = fmaf(wt[dy * 3 + 2][i], in[2][i], v);
            a[i] = v;
          }
        }
        const int od = r - 2;  // output row completed by this box row
        if (od >= 0 && y0 + od < p.H && x < p.W) {
          const float (&a)[4] = acc[od % 3];
          uint2 out;
          float o4[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) o4[i] = a[i] * __saturatef(fmaf(a[i], p.act_a, p.act_b));
          out.x = pack16<F16>(o4[0], o4[1]);
          out.y = pack16<F16>(o4[2], o4[3]);
          *reinterpret_cast<uint2*>(gp + ((long long)(y0 + od) * p.W + x) * 64) = out;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar + 8 * s);  // the warp has read all it needs of this stage
    }
  }
  __syncthreads();
  if (abort_flag && threadIdx.x == 0) atomicExch(&g_dw_timeout_flag, 1);
}

}  // namespace

// h: [B][Ch / 32][H * W][32], g: [B][Ch / 64][H * W][64] bf16 (f16: binary16); w_dw [Ch][3][3]; b_dw [Ch] or nullptr.
msla_status_t run_ffn_dw3x3_bf16(const void* h, const void* w_dw, const void* b_dw, void* g, int B, int Ch, int H, int W, int act,
                                 cudaStream_t st, bool f16) {
  const long long z = (long long)B * (Ch / 64);
  if (Ch % 64 != 0 || z > 0x7fffffffLL)
    return fail(MSLA_ERR_UNSUPPORTED, "FFN depthwise convolution: %d hidden channels, batch %d", Ch, B);
  CUtensorMap tmH;
  const cuuint64_t dims[4] = {32, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)(2 * z)};
  const cuuint64_t strides[3] = {64, (cuuint64_t)W * 64, (cuuint64_t)H * W * 64};
  const cuuint32_t box[4] = {32, DW_BOX_PX, 1, 1};  // one image row of a tile with its halo columns
  if (!tma_make_map_bf16(&tmH, h, 4, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_64B))
    return fail(MSLA_ERR_CUDA, "cuTensorMapEncodeTiled failed for the FFN's depthwise convolution");
  DwParams p{};
  p.w_dw = (const bf16*)w_dw; p.b_dw = (const bf16*)b_dw; p.g = (bf16*)g;
  p.H = H; p.W = W; p.planes = Ch / 64;
  p.act_a = act == 2 ? 1.f / 6.f : (act == 1 ? 1e30f : 0.f);
  p.act_b = act == 2 ? 0.5f : (act == 1 ? 0.f : 1.f);
  p.tiles_x = (W + DW_PX - 1) / DW_PX; p.tiles_y = (H + DW_ROWS - 1) / DW_ROWS;
  p.num_tiles = z * p.tiles_x * p.tiles_y;
  static std::atomic<unsigned long long> attr_done{0}, attr_done16{0};
  const msla_status_t as = f16 ? ensure_smem_attr(attr_done16, ffn_dw3x3_kernel<true>, DW_SMEM) : ensure_smem_attr(attr_done, ffn_dw3x3_kernel<false>, DW_SMEM);
  if (as != MSLA_OK) return as;
  const long long grid = p.num_tiles < device_sm_count() ? p.num_tiles : device_sm_count();
  if (f16) launch_pdl(ffn_dw3x3_kernel<true>, dim3((unsigned)grid), dim3(DW_THREADS), DW_SMEM, st, tmH, p);
  else launch_pdl(ffn_dw3x3_kernel<false>, dim3((unsigned)grid), dim3(DW_THREADS), DW_SMEM, st, tmH, p);
  count_launches(1);
  return check_launch(f16 ? "FFN depthwise convolution (fp16)" : "FFN depthwise convolution (bf16)");
}

int dw_timeout_flag() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_dw_timeout_flag, sizeof(int)) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  return v;
}

}  // namespace msla
