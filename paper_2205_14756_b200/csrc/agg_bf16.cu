// Fused multi-scale token aggregation for bf16 (Section 3.1): the 5x5 depthwise
// convolution and the grouped 1x1 convolution of one block of 32 channels in
// one kernel, on planar activations.  The library uses it for d = 16 (two
// groups per block, D16 = true); d = 32 runs the kernel of agg_toeplitz.cu.
//
// One CTA = a run of TW x TH pixel tiles of one group.  TMA copies stage the
// (TW+4) x (TH+4) halo tiles in a two-deep ring in shared memory; coordinates
// outside the image are zero-filled by the TMA unit, which is exactly the
// convolution's zero padding.  Each warp owns an 8x8 pixel block: lane
// (g = lane/4, t = lane%4) accumulates, in fp32 registers, the depthwise result
// of the 8 pixels of column g for channels 8t..8t+7.  Four of the five tap
// columns are evaluated on tensor cores (a tap is a multiplication by a
// diagonal matrix, and the lane's 16-byte loads are already the A fragments),
// the fifth with packed fp32 FMAs sliding down the column.  The result is
// rounded once to bf16 and used, in place, as the A operand of
// mma.sync.m16n8k16 against the group's 32x32 pointwise weights: the grouped
// 1x1 is fed from registers, with no shared-memory round trip in between.
#include <cuda.h>

#include "msla_common.cuh"
#include "msla_host.h"
#include "tma_host.h"

#ifndef MSLA_AGG_WX
#define MSLA_AGG_WX 2  // warps along x (8 pixels each)
#endif
#ifndef MSLA_AGG_WY
#define MSLA_AGG_WY 2  // warps along y
#endif

#ifndef MSLA_AGG_TC_COLS
#define MSLA_AGG_TC_COLS 4  // tap columns (dx) of the depthwise filter evaluated on tensor cores: 0, 2 or 4
#endif
#ifndef MSLA_AGG_MIN_BLOCKS
#define MSLA_AGG_MIN_BLOCKS 3
#endif

namespace msla {
namespace {

using bf16 = __nv_bfloat16;
constexpr int D = 32;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000LL;

__device__ int g_agg_timeout_flag = 0;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void fma2(float2& acc, const float2& a, const float2& b) {
  unsigned long long& c = reinterpret_cast<unsigned long long&>(acc);
  asm("fma.rn.f32x2 %0, %1, %2, %0;"
      : "+l"(c)
      : "l"(reinterpret_cast<const unsigned long long&>(a)), "l"(reinterpret_cast<const unsigned long long&>(b)));
}
__device__ __forceinline__ float2 unpack_bf16x2(uint32_t v) {  // exact widening
  return make_float2(__uint_as_float(v << 16), __uint_as_float(v & 0xffff0000u));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

struct AggParams {
  const bf16* w_dw;  // [Ch][5][5]
  const bf16* w_pw;  // [Ch][32]
  bf16* dst;         // planar output
  long long dst_batch_stride;  // elements
  int src_planes_per_batch;    // plane index of (b, group) in the tensor map = b * this + group
  int H, W;
  int tiles_x, tiles_total;    // tiles per plane
  int tiles_per_cta;           // consecutive tiles of one plane handled by one CTA
};

// D16 = false: one group of 32 channels, planes [H*W][32].
// D16 = true : d = 16.  Two neighbouring groups of 16 channels are handled as one block of 32 channels
// (the depthwise part does not care about groups; the 1x1 becomes block-diagonal).  Their two planes
// [H*W][16] are staged as two tiles; the second one is fetched two pixels further left, so that it sits
// 64 bytes further on in shared memory and the two planes' 16-byte chunks fall into different banks.
template <int WX, int WY, bool D16>
__global__ void __launch_bounds__(WX * WY * 32, MSLA_AGG_MIN_BLOCKS)
aggregate_bf16_kernel(const __grid_constant__ CUtensorMap tm_src, AggParams p) {
  constexpr int TW = 8 * WX, TH = 8 * WY, HH = TH + 4;
  constexpr int HW_ = D16 ? TW + 6 : TW + 4;          // pixels per staged row (d = 16: two spare columns)
  constexpr int PIXB = D16 ? 32 : 64;                  // bytes per staged pixel
  constexpr int PLANE_BYTES = HW_ * HH * PIXB;         // one TMA box
  constexpr int TILE_BYTES = D16 ? 2 * PLANE_BYTES : PLANE_BYTES;
  constexpr int TILE_PITCH = (TILE_BYTES + 64 + 127) / 128 * 128;
  constexpr int TC_COLS = MSLA_AGG_TC_COLS;
  extern __shared__ __align__(128) unsigned char tiles[];  // two halo tiles (double buffer), dynamic
  __shared__ __align__(16) float wdw_s[5][5][D];           // [dx][dy][channel]
  // Depthwise taps of the first TC_COLS tap columns as per-lane B fragments of 8x8 diagonal
  // matrices (see below): [dx][dy][channel-pair block jn][lane].
  __shared__ uint32_t bdiag[TC_COLS > 0 ? TC_COLS : 1][5][4][32];
  __shared__ __align__(8) unsigned long long bar_storage[2];
  __shared__ int timed_out;

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int wx = warp % WX, wy = warp / WX;
  const int group = blockIdx.y, b = blockIdx.z;
  const int ch0 = group * D;
  const int tile_first = blockIdx.x * p.tiles_per_cta;
  const int tile_count = min(p.tiles_per_cta, p.tiles_total - tile_first);
  const int plane_idx = b * p.src_planes_per_batch + group;
  const uint32_t bar0 = smem_u32(&bar_storage[0]);
  const uint32_t tiles0 = smem_u32(tiles);

  // One elected thread feeds the two-deep ring.  x and y may start at -2 (and
  // run past W, H): the TMA unit returns zeros there, i.e. the zero padding.
  auto issue = [&](int k) {
    const int tile = tile_first + k;
    const int tx0 = (tile % p.tiles_x) * TW, ty0 = (tile / p.tiles_x) * TH;
    const uint32_t bar = bar0 + 8 * (k & 1);
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(TILE_BYTES) : "memory");
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(tiles0 + (k & 1) * TILE_PITCH), "l"(&tm_src), "r"(bar), "r"(0), "r"(tx0 - 2), "r"(ty0 - 2),
          "r"(D16 ? 2 * plane_idx - b * p.src_planes_per_batch : plane_idx) : "memory");
    if (D16)  // second plane of the pair, two pixels further left (see above)
      asm volatile(
          "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
          ::"r"(tiles0 + (k & 1) * TILE_PITCH + PLANE_BYTES), "l"(&tm_src), "r"(bar), "r"(0), "r"(tx0 - 4), "r"(ty0 - 2),
            "r"(2 * plane_idx - b * p.src_planes_per_batch + 1) : "memory");
  };

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    timed_out = 0;
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar0) : "memory");
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar0 + 8) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    pdl_wait();  // the planes read here come from the previous kernel; the tables below only need the weights
    issue(0);
  }
  // depthwise taps -> fp32 [dx][dy][c] while the first copy is in flight
  for (int e = threadIdx.x; e < 25 * D; e += WX * WY * 32) {
    const int c = e % D, tap = e / D;  // consecutive threads -> consecutive channels: conflict-free stores
    wdw_s[tap % 5][tap / 5][c] = __bfloat162float(p.w_dw[(long long)(ch0 + c) * 25 + tap]);
  }
  // B fragment of diag(w[ch]) over the channel set {8t'+2jn+e}: lane (g, t) holds rows k = 2t, 2t+1 of
  // column n = g, so only lanes with g/2 == t hold a non-zero: the tap of channel 8t+2jn+(g&1), in the
  // low (g even) or high (g odd) half of the register.
  for (int e = threadIdx.x; e < TC_COLS * 5 * 4 * 32; e += WX * WY * 32) {
    const int ln = e & 31, jn = (e >> 5) & 3, dy = (e >> 7) % 5, dx = (e >> 7) / 5;
    const int lg = ln >> 2, lt = ln & 3;
    uint32_t v = 0;
    if ((lg >> 1) == lt) {
      const bf16 wv = p.w_dw[(long long)(ch0 + 8 * lt + 2 * jn + (lg & 1)) * 25 + dy * 5 + dx];
      v = (uint32_t)__bfloat16_as_ushort(wv) << (16 * (lg & 1));
    }
    bdiag[dx][dy][jn][ln] = v;
  }
  // pointwise weights as B fragments: slots (2t,2t+1)+8r <-> in channels 8t+4ks+2r,+1; column g <-> out channel oc(jn)
  uint32_t bw[2][4][2];
#pragma unroll
  for (int ks = 0; ks < 2; ++ks)
#pragma unroll
    for (int jn = 0; jn < 4; ++jn)
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const int oc = 8 * (g >> 1) + 2 * jn + (g & 1);
        const int ic = 8 * t + 4 * ks + 2 * r;  // first in-channel of the pair, inside the block of 32
        if (D16)  // block-diagonal: two 16x16 groups
          bw[ks][jn][r] = (oc >> 4) == (ic >> 4)
                              ? *reinterpret_cast<const uint32_t*>(p.w_pw + (long long)(ch0 + oc) * 16 + (ic & 15)) : 0u;
        else
          bw[ks][jn][r] = *reinterpret_cast<const uint32_t*>(p.w_pw + (long long)(ch0 + oc) * D + ic);
      }
  __syncthreads();  // barriers initialised and taps staged before anyone proceeds
  pdl_wait();

  // output: plane `group` of 32 channels, or for d = 16 the plane (2*group + t/2) of 16 channels
  bf16* plane = D16 ? p.dst + (long long)b * p.dst_batch_stride + (long long)(2 * group + (t >> 1)) * p.H * p.W * 16
                    : p.dst + (long long)b * p.dst_batch_stride + (long long)group * p.H * p.W * D;
#pragma unroll 1
  for (int k = 0; k < tile_count; ++k) {
    // prefetch the next tile into the buffer everyone left at the end of iteration k-1
    if (threadIdx.x == 0 && k + 1 < tile_count) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // order the earlier generic reads before the async write
      issue(k + 1);
    }
    {  // bounded wait for this tile
      const uint32_t bar = bar0 + 8 * (k & 1), parity = (k >> 1) & 1;
      uint32_t ok = 0;
      const long long t_start = clock64();
      while (true) {
        asm volatile(
            "{\n\t.reg .pred P1;\n\tmbarrier.try_wait.parity.shared::cta.b64 P1, [%1], %2;\n\tselp.b32 %0, 1, 0, P1;\n\t}"
            : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) break;
        if (timed_out || clock64() - t_start > WAIT_LIMIT_CYCLES) { timed_out = 1; break; }
      }
    }
    if (__syncthreads_or(timed_out)) {  // leave without touching this tile; the copy had two seconds to land
      if (threadIdx.x == 0) atomicExch(&g_agg_timeout_flag, 1);
      return;
    }
    const int tile = tile_first + k;
    const int x0 = (tile % p.tiles_x) * TW, y0 = (tile / p.tiles_x) * TH;

    // ---- depthwise 5x5: column (wx*8 + g), rows wy*8 .. +7, channels 8t .. 8t+7
    float2 acc[8][4];
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
      for (int q = 0; q < 4; ++q) acc[r][q] = make_float2(0.f, 0.f);
    // this lane's 16 bytes of the pixel at (row 0, column 0) of its column's window
    const uint32_t col_base = tiles0 + (k & 1) * TILE_PITCH +
                              (D16 ? (uint32_t)((t >> 1) * (PLANE_BYTES + 64) + ((wy * 8) * HW_ + wx * 8 + g) * PIXB + (t & 1) * 16)
                                   : (uint32_t)(((wy * 8) * HW_ + wx * 8 + g) * PIXB + t * 16));
    // Tap columns 0 .. TC_COLS-1 on tensor cores, two columns per MMA.  For one tap (dy, dx) and one
    // block jn of 8 channels, out[pixel][ch] += in[pixel + (dy, dx)][ch] * w[ch] is the product of a
    // 16x8 pixel-by-channel matrix with the 8x8 matrix diag(w); m16n8k16 takes the taps (dy, dx) and
    // (dy, dx+1) at once (contraction slots 0-7 and 8-15).  With MMA rows g / g+8 = pixels (x, 2j) /
    // (x, 2j+1) and the channel set {8t'+2jn+e}, the A fragment of lane (g, t) is word jn of the very
    // 16 bytes it loads for the fp32 path (input rows 2j+dy, 2j+dy+1 of columns dx, dx+1), untouched,
    // and the accumulator fragment is acc[2j][jn], acc[2j+1][jn].  Products of bf16 values are exact
    // and accumulation is fp32: the same arithmetic as the FMA path, on a pipe that is idle here.
#pragma unroll 1
    for (int dx = 0; dx < TC_COLS; dx += 2) {
      uint32_t bd0[5][4], bd1[5][4];
#pragma unroll
      for (int dy = 0; dy < 5; ++dy)
#pragma unroll
        for (int jn = 0; jn < 4; ++jn) { bd0[dy][jn] = bdiag[dx][dy][jn][lane]; bd1[dy][jn] = bdiag[dx + 1][dy][jn][lane]; }
      uint32_t A[4][4];  // [jn][a0: row i col dx, a1: row i+1 col dx, a2: row i col dx+1, a3: row i+1 col dx+1]
      {
        uint32_t r0[4], r1[4];
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r0[0]), "=r"(r0[1]), "=r"(r0[2]), "=r"(r0[3])
                     : "r"(col_base + (uint32_t)(dx * PIXB)));
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r1[0]), "=r"(r1[1]), "=r"(r1[2]), "=r"(r1[3])
                     : "r"(col_base + (uint32_t)((dx + 1) * PIXB)));
#pragma unroll
        for (int jn = 0; jn < 4; ++jn) { A[jn][1] = r0[jn]; A[jn][3] = r1[jn]; }
      }
#pragma unroll
      for (int i = 0; i < 11; ++i) {  // input rows i and i+1 feed output rows (i-dy, i-dy+1)
        uint32_t r0[4], r1[4];
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r0[0]), "=r"(r0[1]), "=r"(r0[2]), "=r"(r0[3])
                     : "r"(col_base + (uint32_t)(((i + 1) * HW_ + dx) * PIXB)));
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r1[0]), "=r"(r1[1]), "=r"(r1[2]), "=r"(r1[3])
                     : "r"(col_base + (uint32_t)(((i + 1) * HW_ + dx + 1) * PIXB)));
#pragma unroll
        for (int jn = 0; jn < 4; ++jn) { A[jn][0] = A[jn][1]; A[jn][2] = A[jn][3]; A[jn][1] = r0[jn]; A[jn][3] = r1[jn]; }
#pragma unroll
        for (int dy = 0; dy < 5; ++dy) {
          const int r = i - dy;
          if (r >= 0 && r < 8 && (r & 1) == 0) {
#pragma unroll
            for (int jn = 0; jn < 4; ++jn) {
              float c[4] = {acc[r][jn].x, acc[r][jn].y, acc[r + 1][jn].x, acc[r + 1][jn].y};
              mma_bf16(c, A[jn], bd0[dy][jn], bd1[dy][jn]);
              acc[r][jn] = make_float2(c[0], c[1]); acc[r + 1][jn] = make_float2(c[2], c[3]);
            }
          }
        }
      }
    }
#pragma unroll 1
    for (int dx = TC_COLS; dx < 5; ++dx) {
      float2 w[5][4];
#pragma unroll
      for (int dy = 0; dy < 5; ++dy) {
        const float4 lo = *reinterpret_cast<const float4*>(&wdw_s[dx][dy][8 * t]);
        const float4 hi = *reinterpret_cast<const float4*>(&wdw_s[dx][dy][8 * t + 4]);
        w[dy][0] = make_float2(lo.x, lo.y); w[dy][1] = make_float2(lo.z, lo.w);
        w[dy][2] = make_float2(hi.x, hi.y); w[dy][3] = make_float2(hi.z, hi.w);
      }
#pragma unroll
      for (int i = 0; i < 12; ++i) {  // input row i of the column feeds output rows i-4 .. i
        uint32_t raw[4];
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(raw[0]), "=r"(raw[1]), "=r"(raw[2]), "=r"(raw[3])
                     : "r"(col_base + (uint32_t)((i * HW_ + dx) * PIXB)));
        float2 in[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) in[q] = unpack_bf16x2(raw[q]);
#pragma unroll
        for (int dy = 0; dy < 5; ++dy) {
          const int r = i - dy;
          if (r >= 0 && r < 8) {
#pragma unroll
            for (int q = 0; q < 4; ++q) fma2(acc[r][q], w[dy][q], in[q]);
          }
        }
      }
    }

    // ---- grouped 1x1 on tensor cores, straight from the accumulators
    const int x = x0 + wx * 8 + g;
#pragma unroll
    for (int j = 0; j < 4; ++j) {  // MMA rows g / g+8 = pixels (x, 2j) / (x, 2j+1) of the warp block
      float c[4][4];
#pragma unroll
      for (int jn = 0; jn < 4; ++jn)
#pragma unroll
        for (int e = 0; e < 4; ++e) c[jn][e] = 0.f;
#pragma unroll
      for (int ks = 0; ks < 2; ++ks) {
        const uint32_t A[4] = {pack_bf16(acc[2 * j][2 * ks].x, acc[2 * j][2 * ks].y),
                               pack_bf16(acc[2 * j + 1][2 * ks].x, acc[2 * j + 1][2 * ks].y),
                               pack_bf16(acc[2 * j][2 * ks + 1].x, acc[2 * j][2 * ks + 1].y),
                               pack_bf16(acc[2 * j + 1][2 * ks + 1].x, acc[2 * j + 1][2 * ks + 1].y)};
#pragma unroll
        for (int jn = 0; jn < 4; ++jn) mma_bf16(c[jn], A, bw[ks][jn][0], bw[ks][jn][1]);
      }
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int y = y0 + wy * 8 + 2 * j + half;
        if (x < p.W && y < p.H) {
          bf16* dst = D16 ? plane + ((long long)y * p.W + x) * 16 + 8 * (t & 1) : plane + ((long long)y * p.W + x) * D + 8 * t;
          asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(dst),
                       "r"(pack_bf16(c[0][2 * half], c[0][2 * half + 1])), "r"(pack_bf16(c[1][2 * half], c[1][2 * half + 1])),
                       "r"(pack_bf16(c[2][2 * half], c[2][2 * half + 1])), "r"(pack_bf16(c[3][2 * half], c[3][2 * half + 1]))
                       : "memory");
        }
      }
    }
    __syncthreads();  // every warp is done with buffer k&1 before iteration k+1 refills it (for tile k+2)
  }
}

}  // namespace

bool aggregate_bf16_supported(int H, int W, int Ch, int d) {
  return (d == 32 || d == 16) && Ch % 32 == 0 && H >= 1 && W >= 1;
}

namespace {
template <bool D16>
msla_status_t launch_aggregate(const void* src, long long src_planes_total, int src_ppb, const void* w_dw,
                               const void* w_pw, void* dst, long long dst_sb, int B, int H, int W, int Ch,
                               cudaStream_t st) {
  constexpr int WX = MSLA_AGG_WX, WY = MSLA_AGG_WY, TW = 8 * WX, TH = 8 * WY;
  constexpr int DP = D16 ? 16 : 32;           // channels per plane
  constexpr int BOXW = D16 ? TW + 6 : TW + 4;  // staged pixels per row
  CUtensorMap tm;
  const cuuint64_t dims[4] = {(cuuint64_t)DP, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)src_planes_total};
  const cuuint64_t strides[3] = {(cuuint64_t)DP * 2, (cuuint64_t)W * DP * 2, (cuuint64_t)H * W * DP * 2};
  const cuuint32_t box[4] = {(cuuint32_t)DP, (cuuint32_t)BOXW, (cuuint32_t)(TH + 4), 1};
  if (!tma_make_map_bf16(&tm, src, 4, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE))
    return fail(MSLA_ERR_CUDA, "cuTensorMapEncodeTiled failed for the aggregation input");
  AggParams p;
  p.w_dw = (const bf16*)w_dw; p.w_pw = (const bf16*)w_pw; p.dst = (bf16*)dst;
  p.dst_batch_stride = dst_sb; p.src_planes_per_batch = src_ppb; p.H = H; p.W = W;
  p.tiles_x = (W + TW - 1) / TW;
  const long long tiles = (long long)p.tiles_x * ((H + TH - 1) / TH);
  if (tiles > 0x7fffffffLL) return fail(MSLA_ERR_UNSUPPORTED, "too many aggregation tiles");
  p.tiles_total = (int)tiles;
  // enough CTAs for a few waves over the GPU, otherwise as many tiles per CTA as possible (up to 8)
  const long long units = tiles * (Ch / D) * B;
  p.tiles_per_cta = units >= 8 * 2400 ? 8 : units >= 4 * 2400 ? 4 : units >= 2 * 2400 ? 2 : 1;
  dim3 grid((unsigned)((tiles + p.tiles_per_cta - 1) / p.tiles_per_cta), (unsigned)(Ch / D), (unsigned)B);
  constexpr int one_tile = (D16 ? 2 : 1) * BOXW * (TH + 4) * DP * 2;
  constexpr int tile_bytes = 2 * ((one_tile + 64 + 127) / 128 * 128);  // must match TILE_PITCH in the kernel
  static bool attr_done = false;
  if (!attr_done) {
    cudaFuncSetAttribute(aggregate_bf16_kernel<WX, WY, D16>, cudaFuncAttributeMaxDynamicSharedMemorySize, tile_bytes);
    attr_done = true;
  }
  launch_pdl(aggregate_bf16_kernel<WX, WY, D16>, grid, dim3(WX * WY * 32), tile_bytes, st, tm, p);
  count_launches(1);
  return check_launch("token aggregation (bf16)");
}
}  // namespace

// src, dst: planar bf16 [.., planes, H*W, d], d in {16, 32}; group g of image b is plane b*src_ppb + g of
// src (src_planes_total planes in all) and lives at dst + b*dst_sb + g*H*W*d.  Ch must be a multiple of 32.
// d = 32 goes to the Toeplitz kernel (agg_toeplitz.cu), d = 16 to the kernel above.
msla_status_t run_aggregate_bf16(const void* src, long long src_planes_total, int src_ppb, const void* w_dw,
                                 const void* w_pw, void* dst, long long dst_sb, int B, int H, int W, int Ch, int d,
                                 cudaStream_t st) {
  if (d == 16) return launch_aggregate<true>(src, src_planes_total, src_ppb, w_dw, w_pw, dst, dst_sb, B, H, W, Ch, st);
  const long long plane = (long long)H * W * d;
  if (!aggregate_toeplitz_bf16_supported(H, W, Ch, d) || dst_sb % plane != 0)
    return fail(MSLA_ERR_UNSUPPORTED, "aggregation: d = %d with an output batch stride of %lld elements", d, dst_sb);
  const long long dst_ppb = dst_sb / plane;
  return run_aggregate_toeplitz_bf16(src, src_planes_total, src_ppb, w_dw, w_pw, dst, (B - 1) * dst_ppb + Ch / d, (int)dst_ppb,
                                     B, H, W, Ch, st);
}

int agg_timeout_flag() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_agg_timeout_flag, sizeof(int)) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  return v;
}

}  // namespace msla
