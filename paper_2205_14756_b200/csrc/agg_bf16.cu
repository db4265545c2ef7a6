// Fused multi-scale token aggregation for bf16 (Section 3.1): the 5x5 depthwise
// convolution and the grouped 1x1 convolution of one block of 32 channels in
// one kernel, on planar activations [planes][H*W][d], with the depthwise filter
// evaluated on tensor cores as banded (Toeplitz) matrices.  d = 32: a block is
// one group; d = 16: two neighbouring groups (two planes of 16 channels, staged
// by two TMA copies; the 1x1 weights become block-diagonal).
//
// For one channel and one filter row dy, the horizontal part of the filter is a
// matrix product: out[y][x] += sum_k in[y + dy - 2][x0 - 4 + k] * T[k][x - x0] with
// T[k][n] = w[dy][k - n - 2] (zero outside the five taps).  With 16 image rows as
// the M dimension, a 16-pixel window as K and 8 output pixels as N this is one
// mma.sync.m16n8k16 per (channel, dy, 8 output columns): 5 of 16 products are
// useful, against 2 of 16 when a tap is written as a diagonal matrix over
// channels.  The operand needs, per channel, pixels along the contraction, so
// the kernel first turns the staged tile around in shared memory.
//
// One CTA = a run of 16 x 16 pixel tiles of one group; per tile:
//   P1  TMA box [20 rows][24 pixels][32 channels] (64B swizzle, zero fill outside
//       the image = the convolution's padding) -> ldmatrix.trans -> planar tile
//       [channel][row parity][row / 2][24 pixels].  Splitting rows by parity makes
//       the eight rows y, y+2, .. of an A fragment consecutive in memory.
//   P2  depthwise: warp w owns channels 4w .. 4w+3 (their Toeplitz B fragments stay
//       in registers for the CTA's whole life).  MMA row g is image row 2g, row g+8
//       is image row 2g+1, so the fragment for (dy+1) reuses half of the one for dy:
//       18 ldmatrix matrices feed 10 MMAs per channel.  fp32 accumulators, rounded
//       once to bf16 into a [channel][pixel] tile.
//   P3  grouped 1x1: A = that tile through ldmatrix.trans (pixels x channels),
//       B = the group's 32x32 weights from registers; each warp stages its 8 x 4
//       pixels and writes them with one TMA store, which also clips at the image
//       border (stores issued by the lanes themselves cost the load/store pipe
//       four times the cycles of the staging writes).
// The single TMA buffer is refilled for the next tile as soon as P1 is over.
// The grid is persistent: two CTAs per SM, each with a contiguous run of
// (image, group, tile) units; the weight fragments are reloaded when the group
// changes.
#include <cuda.h>

#include "msla_common.cuh"
#include "msla_host.h"
#include "tma_host.h"

namespace msla {
namespace {

using bf16 = __nv_bfloat16;
constexpr int TD = 32;                       // channels per group
constexpr int TW = 16, TH = 16;              // output pixels per tile
constexpr int BOXW = TW + 8;                 // staged pixels per row: x0-4 .. x0+19
constexpr int BOXH = TH + 4;                 // staged rows: y0-2 .. y0+17
constexpr int BOX_ROW = BOXW * 64;           // bytes per staged row
constexpr int BOX_BYTES = BOXH * BOX_ROW;    // one TMA box
constexpr int PL_ROW = BOXW * 2;             // planar tile: bytes per (channel, row)
constexpr int PL_HALF = (BOXH / 2) * PL_ROW; // rows of one parity
constexpr int PL_CH = 2 * PL_HALF + 16;      // 976 = 16 * 61: channel pitch, odd in 16-byte units
constexpr int PL_BYTES = TD * PL_CH;
constexpr int DWO_CH = TW * TH * 2 + 16;     // 528 = 16 * 33: depthwise output, bytes per channel
constexpr int DWO_BYTES = TD * DWO_CH;
constexpr int T_BAND = 4;                    // tile rows per band of the traversal
constexpr int T_WARPS = 8;
constexpr int T_THREADS = 32 * T_WARPS;
constexpr int OUT_WARP_BYTES = 4 * 8 * 64;   // output staging per warp: 4 rows x 8 pixels x 32 channels
constexpr int OUT_BYTES = T_WARPS * OUT_WARP_BYTES;
constexpr int T_SMEM_BYTES = 1024 + BOX_BYTES + PL_BYTES + DWO_BYTES + OUT_BYTES;
constexpr long long T_WAIT_LIMIT_CYCLES = 4000000000LL;
static_assert(BOXH % 2 == 0 && (PL_CH / 16) % 2 == 1 && (DWO_CH / 16) % 2 == 1 && (PL_ROW / 16) % 2 == 1, "bank-conflict-free pitches");
static_assert(PL_BYTES % 128 == 0 && DWO_BYTES % 128 == 0, "the output staging must stay 128-byte aligned");
static_assert(BOX_ROW % 512 == 0, "the 64B swizzle pattern must restart with every staged row");

__device__ int g_aggt_timeout_flag = 0;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// F16: the 16-bit storage type is IEEE binary16 instead of bfloat16 (activations and weights alike); the kernel moves
// 16-bit values untyped, only the conversions and the MMA operand type differ.  Accumulators are fp32 in both.
template <bool F16>
__device__ __forceinline__ uint32_t pack_x2(float lo, float hi) {
  uint32_t r;
  if constexpr (F16) asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  else asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
template <bool F16>
__device__ __forceinline__ void mma_16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  if constexpr (F16)
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  else
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldsm_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2(uint32_t& r0, uint32_t& r1, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v) { asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory"); }

struct ToeplitzParams {
  const bf16* w_dw;  // [Ch][5][5]
  const bf16* w_pw;  // [Ch][d]
  int src_planes_per_batch;    // plane index of (b, plane) in a tensor map = b * planes_per_batch + plane
  int dst_planes_per_batch;
  int groups;                  // blocks of 32 channels per image: plane `group` (d = 32) or planes 2*group, 2*group+1 (d = 16)
  int tiles_x, tiles_y, tiles_total;  // tiles per plane
  long long units;             // B * groups * tiles_total, tile fastest
  long long units_per_cta;
};

template <bool D16, bool F16>
__global__ void __launch_bounds__(T_THREADS, 2)
aggregate_toeplitz_kernel(const __grid_constant__ CUtensorMap tm_src, const __grid_constant__ CUtensorMap tm_dst, ToeplitzParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t box = (smem_addr(smem_raw) + 1023u) & ~1023u;  // the swizzle pattern is a function of the address
  const uint32_t pl = box + BOX_BYTES, dwo = pl + PL_BYTES, outs = dwo + DWO_BYTES;
  __shared__ __align__(8) unsigned long long bar_storage;
  __shared__ int timed_out;

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const long long unit_first = (long long)blockIdx.x * p.units_per_cta;
  const int unit_count = (int)max(0LL, min(p.units_per_cta, p.units - unit_first));
  const uint32_t bar = smem_addr(&bar_storage);

  // Cursor over (image, group, tile) units, tile fastest, advanced without divisions.  Inside a plane the
  // tiles run down bands of T_BAND tile rows, column by column, so that a tile's lower and right
  // neighbours follow within a few iterations and find the shared halo rows and columns in L2.
  struct Unit { int tile, tx, ty, band_end, group, b; };  // band_end: first tile row below the current band
  auto locate = [&](long long u) {
    const long long bg = u / p.tiles_total;
    Unit r;
    r.tile = (int)(u - bg * p.tiles_total);
    const int band = r.tile / (T_BAND * p.tiles_x), rem = r.tile - band * (T_BAND * p.tiles_x);
    r.band_end = min(band * T_BAND + T_BAND, p.tiles_y);
    const int bh = r.band_end - band * T_BAND;
    r.tx = rem / bh;
    r.ty = band * T_BAND + rem - r.tx * bh;
    r.b = (int)(bg / p.groups);
    r.group = (int)(bg - (long long)r.b * p.groups);
    return r;
  };
  auto advance = [&](Unit& u) {
    ++u.tile;
    if (++u.ty == u.band_end) {
      const int band_start = (u.band_end - 1) / T_BAND * T_BAND;
      if (++u.tx == p.tiles_x) { u.tx = 0; u.ty = u.band_end; u.band_end = min(u.band_end + T_BAND, p.tiles_y); }
      else u.ty = band_start;
    }
    if (u.tile == p.tiles_total) {
      u.tile = 0; u.ty = 0; u.band_end = min(T_BAND, p.tiles_y);
      if (++u.group == p.groups) { u.group = 0; ++u.b; }
    }
  };
  // x and y may start below 0 and run past W, H: the TMA unit returns zeros there.
  auto issue = [&](const Unit& u) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(BOX_BYTES) : "memory");
    const int plane = u.b * p.src_planes_per_batch + (D16 ? 2 * u.group : u.group);
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(box), "l"(&tm_src), "r"(bar), "r"(0), "r"(u.tx * TW - 4), "r"(u.ty * TH - 2), "r"(plane) : "memory");
    if (D16)  // second plane of the pair behind the first
      asm volatile(
          "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
          ::"r"(box + BOX_BYTES / 2), "l"(&tm_src), "r"(bar), "r"(0), "r"(u.tx * TW - 4), "r"(u.ty * TH - 2), "r"(plane + 1) : "memory");
  };
  Unit un = locate(unit_first), nxt = un;  // nxt: the unit whose copy is issued next (thread 0 only)

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    timed_out = 0;
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    pdl_wait();  // the planes read here come from the previous kernel; the fragments below only need the weights
    if (unit_count > 0) issue(nxt);
  }

  uint32_t bt[4][5][2];  // Toeplitz B fragments of this warp's four channels
  uint32_t bw[2][4][2];  // pointwise weights as B fragments
  auto load_weights = [&](int group) {
    const int ch0 = group * TD;
    // lane (g, t) holds rows k = 2t, 2t+1 (b0) and 2t+8, 2t+9 (b1) of column n = g, i.e. taps dx = k - g - 2 of filter row dy
#pragma unroll
    for (int cc = 0; cc < 4; ++cc)
#pragma unroll
      for (int dy = 0; dy < 5; ++dy) {
        const bf16* wrow = p.w_dw + (long long)(ch0 + 4 * warp + cc) * 25 + dy * 5;
        const int i0 = 2 * t - g - 2;
        auto tap = [&](int i) -> uint32_t { return (i >= 0 && i < 5) ? (uint32_t)__bfloat16_as_ushort(wrow[i]) : 0u; };
        bt[cc][dy][0] = tap(i0) | (tap(i0 + 1) << 16);
        bt[cc][dy][1] = tap(i0 + 8) | (tap(i0 + 9) << 16);
      }
    // Contraction slots are the input channels in order; column n = g of block jn is output channel
    // 8(g/2) + 2jn + (g&1), so that a lane ends up with channels 8t .. 8t+7.
#pragma unroll
    for (int ks = 0; ks < 2; ++ks)
#pragma unroll
      for (int jn = 0; jn < 4; ++jn) {
        const int oc = 8 * (g >> 1) + 2 * jn + (g & 1);
        if (D16) {  // two 16 x 16 groups: contraction step ks holds the input channels of group ks
          const bf16* wr = p.w_pw + (long long)(ch0 + oc) * 16 + 2 * t;
          const bool same = (oc >> 4) == ks;
          bw[ks][jn][0] = same ? *reinterpret_cast<const uint32_t*>(wr) : 0u;
          bw[ks][jn][1] = same ? *reinterpret_cast<const uint32_t*>(wr + 8) : 0u;
        } else {
          const bf16* wr = p.w_pw + (long long)(ch0 + oc) * TD + 16 * ks + 2 * t;
          bw[ks][jn][0] = *reinterpret_cast<const uint32_t*>(wr);
          bw[ks][jn][1] = *reinterpret_cast<const uint32_t*>(wr + 8);
        }
      }
  };
  int cur_group = un.group;
  load_weights(cur_group);

  // Per-lane address offsets of the six ldmatrix loads of a channel.  Matrix (r, h) = staged rows
  // 2g'+r (g' = 0..7), 16-byte piece h of the row; lane l supplies row l&7 of matrix l>>3.
  //   load 0 (x4): (0,0) (1,0) (0,1) (1,1)    load 1 (x2): (0,2) (1,2)
  //   load 2 (x4): (2,0) (2,1) (2,2) (3,0)    load 3 (x2): (3,1) (3,2)
  //   load 4 (x4): (4,0) (4,1) (4,2) (5,0)    load 5 (x2): (5,1) (5,2)
  uint32_t aoff[6];
  {
    const int mi = lane >> 3, row = lane & 7;
    auto off = [&](int r, int h) { return (uint32_t)((r & 1) * PL_HALF + (row + (r >> 1)) * PL_ROW + h * 16); };
    aoff[0] = off(mi & 1, mi >> 1);
    aoff[1] = off(mi & 1, 2);
    aoff[2] = mi < 3 ? off(2, mi) : off(3, 0);
    aoff[3] = off(3, 1 + (mi & 1));
    aoff[4] = mi < 3 ? off(4, mi) : off(5, 0);
    aoff[5] = off(5, 1 + (mi & 1));
  }
  __syncthreads();  // barrier initialised before anyone waits on it
  pdl_wait();

  // this warp's 8 x 4 pixels of a tile: columns 8(w/4) .. +7, rows 4(w%4) .. +3
  const uint32_t my_out = outs + (uint32_t)(warp * OUT_WARP_BYTES);
#pragma unroll 1
  for (int k = 0; k < unit_count; ++k, advance(un)) {
    {  // bounded wait for this tile
      const uint32_t parity = k & 1;
      uint32_t ok = 0;
      const long long t_start = clock64();
      while (true) {
        asm volatile(
            "{\n\t.reg .pred P1;\n\tmbarrier.try_wait.parity.shared::cta.b64 P1, [%1], %2;\n\tselp.b32 %0, 1, 0, P1;\n\t}"
            : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) break;
        if (timed_out || clock64() - t_start > T_WAIT_LIMIT_CYCLES) { timed_out = 1; break; }
      }
    }
    const int x0 = un.tx * TW, y0 = un.ty * TH;
    if (un.group != cur_group) {  // uniform over the CTA
      cur_group = un.group;
      load_weights(cur_group);
    }

    // ---- P1: [row][pixel][channel] -> [channel][row parity][row/2][pixel].  One unit = one staged row
    // and 8 pixels: four 8x8 matrices (8 pixels x 8 channels each), transposed by ldmatrix, so that lane
    // (g, t) gets channel 8cb+g, pixels 2t, 2t+1 as one word.
    for (int u = warp; u < BOXH * (BOXW / 8); u += T_WARPS) {
      const int ry = u / (BOXW / 8), pb = u - ry * (BOXW / 8);
      const int pix = pb * 8 + (lane & 7), cb = lane >> 3;
      uint32_t r0, r1, r2, r3;
      // d = 32: pixels of 64 bytes, 64B swizzle; d = 16: plane cb/2, pixels of 32 bytes, 32B swizzle
      const uint32_t src = D16 ? (uint32_t)((cb >> 1) * (BOX_BYTES / 2) + ry * (BOX_ROW / 2) + pix * 32 + (((cb & 1) ^ ((pix >> 2) & 1)) << 4))
                               : (uint32_t)(ry * BOX_ROW + pix * 64 + ((cb ^ ((pix >> 1) & 3)) << 4));
      ldsm_x4_trans(r0, r1, r2, r3, box + src);
      const uint32_t d = pl + (uint32_t)(g * PL_CH + (ry & 1) * PL_HALF + (ry >> 1) * PL_ROW + (pb * 8 + 2 * t) * 2);
      sts32(d, r0);
      sts32(d + 8 * PL_CH, r1);
      sts32(d + 16 * PL_CH, r2);
      sts32(d + 24 * PL_CH, r3);
    }
    if (__syncthreads_or(timed_out)) {  // the copy had two seconds to land: give up, leave the output alone
      if (threadIdx.x == 0) atomicExch(&g_aggt_timeout_flag, 1);
      return;
    }
    if (threadIdx.x == 0 && k + 1 < unit_count) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // order the generic reads above before the async write
      advance(nxt);
      issue(nxt);
    }

    // ---- P2: depthwise 5x5 of channels 4w .. 4w+3
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
      const int c = 4 * warp + cc;
      const uint32_t cb = pl + (uint32_t)(c * PL_CH);
      uint32_t R[6][3];
      ldsm_x4(R[0][0], R[1][0], R[0][1], R[1][1], cb + aoff[0]);
      ldsm_x2(R[0][2], R[1][2], cb + aoff[1]);
      ldsm_x4(R[2][0], R[2][1], R[2][2], R[3][0], cb + aoff[2]);
      ldsm_x2(R[3][1], R[3][2], cb + aoff[3]);
      ldsm_x4(R[4][0], R[4][1], R[4][2], R[5][0], cb + aoff[4]);
      ldsm_x2(R[5][1], R[5][2], cb + aoff[5]);
      float acc[2][4];
#pragma unroll
      for (int nb = 0; nb < 2; ++nb)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[nb][e] = 0.f;
#pragma unroll
      for (int dy = 0; dy < 5; ++dy)
#pragma unroll
        for (int nb = 0; nb < 2; ++nb)
          mma_16<F16>(acc[nb], R[dy][nb], R[dy + 1][nb], R[dy][nb + 1], R[dy + 1][nb + 1], bt[cc][dy][0], bt[cc][dy][1]);
      // pixel pair (row 2g + half, columns 8nb + 2t, +1) goes to word (2nb + half) * 32 + lane of the channel's row
      const uint32_t o = dwo + (uint32_t)(c * DWO_CH + lane * 4);
#pragma unroll
      for (int nb = 0; nb < 2; ++nb)
#pragma unroll
        for (int half = 0; half < 2; ++half)
          sts32(o + (uint32_t)((2 * nb + half) * 128), pack_x2<F16>(acc[nb][2 * half], acc[nb][2 * half + 1]));
    }
    __syncthreads();

    // ---- P3: grouped 1x1 on 32 pixels per warp.  8-pixel block q of the depthwise tile is image row
    // 2(q&7) + ((q>>3)&1), columns 8(q>>4) .. +7; rows 4a .. 4a+3 of column block xb are q = 16xb + 2a,
    // 16xb + 8 + 2a, 16xb + 2a + 1, 16xb + 8 + 2a + 1.
    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // the previous tile's store has read the staging
    __syncwarp();
#pragma unroll
    for (int mb = 0; mb < 2; ++mb) {
      const int qa = 16 * (warp >> 2) + 2 * (warp & 3) + mb;  // MMA rows g: block qa (row 4a + 2mb), rows g+8: block qa + 8 (row 4a + 2mb + 1)
      float c[4][4];
#pragma unroll
      for (int jn = 0; jn < 4; ++jn)
#pragma unroll
        for (int e = 0; e < 4; ++e) c[jn][e] = 0.f;
#pragma unroll
      for (int ks = 0; ks < 2; ++ks) {
        const int mi = lane >> 3;
        uint32_t a0, a1, a2, a3;  // rows = pixels of block qa / qa+8, contraction = channels 16ks .. 16ks+15
        ldsm_x4_trans(a0, a1, a2, a3, dwo + (uint32_t)((16 * ks + 8 * (mi >> 1) + (lane & 7)) * DWO_CH + (qa + 8 * (mi & 1)) * 16));
#pragma unroll
        for (int jn = 0; jn < 4; ++jn) mma_16<F16>(c[jn], a0, a1, a2, a3, bw[ks][jn][0], bw[ks][jn][1]);
      }
#pragma unroll
      for (int half = 0; half < 2; ++half)  // staging: [row 2mb + half][pixel g][channels 8t .. 8t+7]; d = 16: one such block of 16 channels per plane
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(my_out + (D16 ? (uint32_t)((t >> 1) * (OUT_WARP_BYTES / 2) + ((2 * mb + half) * 8 + g) * 32 + (t & 1) * 16)
                                                                                        : (uint32_t)(((2 * mb + half) * 8 + g) * 64 + t * 16))),
                     "r"(pack_x2<F16>(c[0][2 * half], c[0][2 * half + 1])), "r"(pack_x2<F16>(c[1][2 * half], c[1][2 * half + 1])),
                     "r"(pack_x2<F16>(c[2][2 * half], c[2][2 * half + 1])), "r"(pack_x2<F16>(c[3][2 * half], c[3][2 * half + 1]))
                     : "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (lane == 0) {  // pixels outside the image are clipped by the TMA unit
      const int plane = un.b * p.dst_planes_per_batch + (D16 ? 2 * un.group : un.group);
      asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                   ::"l"(&tm_dst), "r"(my_out), "r"(0), "r"(x0 + 8 * (warp >> 2)), "r"(y0 + 4 * (warp & 3)), "r"(plane) : "memory");
      if (D16)
        asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                     ::"l"(&tm_dst), "r"(my_out + OUT_WARP_BYTES / 2), "r"(0), "r"(x0 + 8 * (warp >> 2)), "r"(y0 + 4 * (warp & 3)), "r"(plane + 1) : "memory");
      asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    }
    // No barrier here: the next tile's P1 only writes the planar tile (last read before the barrier
    // above), and its trailing barrier comes before anything overwrites the depthwise tile.
  }
  if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // stores done before the CTA retires
}

}  // namespace

bool aggregate_bf16_supported(int H, int W, int Ch, int d) { return (d == 32 || d == 16) && Ch % TD == 0 && H >= 1 && W >= 1; }

namespace {
template <bool D16, bool F16>
msla_status_t launch_toeplitz(const void* src, long long src_planes_total, int src_ppb, const void* w_dw, const void* w_pw,
                              void* dst, long long dst_planes_total, int dst_ppb, int B, int H, int W, int Ch, cudaStream_t st) {
  constexpr int DP = D16 ? 16 : 32;  // channels per plane
  CUtensorMap tm_src, tm_dst;
  {
    const cuuint64_t dims[4] = {(cuuint64_t)DP, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)src_planes_total};
    const cuuint64_t ddims[4] = {(cuuint64_t)DP, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)dst_planes_total};
    const cuuint64_t strides[3] = {(cuuint64_t)DP * 2, (cuuint64_t)W * DP * 2, (cuuint64_t)H * W * DP * 2};
    const cuuint32_t bx[4] = {(cuuint32_t)DP, (cuuint32_t)BOXW, (cuuint32_t)BOXH, 1};
    const cuuint32_t ob[4] = {(cuuint32_t)DP, 8, 4, 1};
    if (!tma_make_map_bf16(&tm_src, src, 4, dims, strides, bx, D16 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_64B) ||
        !tma_make_map_bf16(&tm_dst, dst, 4, ddims, strides, ob, CU_TENSOR_MAP_SWIZZLE_NONE))
      return fail(MSLA_ERR_CUDA, "cuTensorMapEncodeTiled failed for the aggregation");
  }
  ToeplitzParams p;
  p.w_dw = (const bf16*)w_dw; p.w_pw = (const bf16*)w_pw;
  p.src_planes_per_batch = src_ppb; p.dst_planes_per_batch = dst_ppb; p.groups = Ch / TD;
  p.tiles_x = (W + TW - 1) / TW;
  p.tiles_y = (H + TH - 1) / TH;
  const long long tiles = (long long)p.tiles_x * p.tiles_y;
  if (tiles > 0x7fffffffLL) return fail(MSLA_ERR_UNSUPPORTED, "too many aggregation tiles");
  p.tiles_total = (int)tiles;
  p.units = tiles * p.groups * B;
  const int sms = device_sm_count();
  // two CTAs per SM; small problems get one unit per CTA
  const long long ctas = p.units < 2LL * sms ? p.units : 2LL * sms;
  p.units_per_cta = (p.units + ctas - 1) / ctas;
  if (p.units_per_cta > 0x7fffffffLL) return fail(MSLA_ERR_UNSUPPORTED, "too many aggregation tiles");
  const unsigned grid = (unsigned)((p.units + p.units_per_cta - 1) / p.units_per_cta);
  static std::atomic<unsigned long long> attr_done{0};
  const msla_status_t as = ensure_smem_attr(attr_done, aggregate_toeplitz_kernel<D16, F16>, T_SMEM_BYTES);
  if (as != MSLA_OK) return as;
  launch_pdl(aggregate_toeplitz_kernel<D16, F16>, dim3(grid), dim3(T_THREADS), T_SMEM_BYTES, st, tm_src, tm_dst, p);
  count_launches(1);
  return check_launch(F16 ? "token aggregation (fp16)" : "token aggregation (bf16)");
}
}  // namespace

// src, dst: planar bf16 [.., planes, H*W, d], d in {16, 32}, Ch a multiple of 32; group g of image b is plane
// b*src_ppb + g of src (src_planes_total planes in all) and lives at dst + b*dst_sb + g*H*W*d (dst_sb a multiple of
// the plane size).
msla_status_t run_aggregate_bf16(const void* src, long long src_planes_total, int src_ppb, const void* w_dw,
                                 const void* w_pw, void* dst, long long dst_sb, int B, int H, int W, int Ch, int d,
                                 cudaStream_t st, bool f16) {
  const long long plane = (long long)H * W * d;
  if (!aggregate_bf16_supported(H, W, Ch, d) || dst_sb % plane != 0)
    return fail(MSLA_ERR_UNSUPPORTED, "aggregation: d = %d, %d channels, output batch stride %lld elements", d, Ch, dst_sb);
  const long long dst_ppb = dst_sb / plane, dst_total = (B - 1) * dst_ppb + Ch / d;
  if (f16)
    return d == 16 ? launch_toeplitz<true, true>(src, src_planes_total, src_ppb, w_dw, w_pw, dst, dst_total, (int)dst_ppb, B, H, W, Ch, st)
                   : launch_toeplitz<false, true>(src, src_planes_total, src_ppb, w_dw, w_pw, dst, dst_total, (int)dst_ppb, B, H, W, Ch, st);
  return d == 16 ? launch_toeplitz<true, false>(src, src_planes_total, src_ppb, w_dw, w_pw, dst, dst_total, (int)dst_ppb, B, H, W, Ch, st)
                 : launch_toeplitz<false, false>(src, src_planes_total, src_ppb, w_dw, w_pw, dst, dst_total, (int)dst_ppb, B, H, W, Ch, st);
}

int agg_timeout_flag() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_aggt_timeout_flag, sizeof(int)) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  return v;
}

}  // namespace msla
