// Fused multi-scale token aggregation for bf16 (Section 3.1): the 5x5 depthwise
// convolution and the grouped 1x1 convolution of one block of 32 channels in
// one kernel, on channel-major activations [B, Ch, H, W], with the depthwise
// filter evaluated on tensor cores as banded (Toeplitz) matrices.  d = 32: a
// block is one group; d = 16: two neighbouring groups (the 1x1 weights become
// block-diagonal and the off-diagonal products are skipped).
//
// For one channel and one filter row dy, the horizontal part of the filter is a
// matrix product: out[y][x] += sum_k in[y + dy - 2][x0 - 4 + k] * T[k][x - x0] with
// T[k][n] = w[dy][k - n - 2] (zero outside the five taps).  With 16 image rows as
// the M dimension, a 16-pixel window as K and 8 output pixels as N this is one
// mma.sync.m16n8k16 per (channel, dy, 8 output columns): 5 of 16 products are
// useful.  The A operand wants pixel pairs of one channel in a register, which is
// how a channel-major image lies in memory, so the fragments are read straight
// from the staged tile.
//
// One CTA = a run of 16-row x 24-pixel tiles of one block; per tile:
//   load  two TMA boxes [32 channels][10 rows][40 pixels], one with the even and one
//         with the odd image rows y0-2 .. y0+17 (two tensor maps over the same
//         image, row stride 2W), pixels x0-8 .. x0+31 (a TMA box starts on a 16-byte
//         boundary), zero fill outside the image = the convolution's padding.
//         MMA row g is image row 2g, row g+8 is image row 2g+1, so the fragment for
//         filter row dy+1 reuses half of the one for dy, and with the rows split by
//         parity the eight rows of a fragment are 80 bytes apart: no bank conflicts.
//   P2    depthwise: warp w owns channels 4w .. 4w+3 (their Toeplitz B fragments stay
//         in registers): 24 four-byte loads feed 15 MMAs per channel; fp32
//         accumulators, rounded once to bf16 into a [channel][pixel] tile.
//   P3    grouped 1x1, transposed: D[out channel][pixel] = W[out][in] * dw[in][pixel]
//         with W from registers and dw through ldmatrix.trans, so that the result is
//         channel-major again: warp w fills the [32 channels][24 pixels] slabs of image
//         rows 2w and 2w+1 and writes each with one TMA store (clipped at the border).
// The grid is persistent: two CTAs per SM, each with a contiguous run of
// (image, block, tile) units; the weight fragments are reloaded when the block
// changes.  The wait for a tile's TMA copy is bounded.
#include <cuda.h>

#include "msla_common.cuh"
#include "msla_host.h"
#include "tma_host.h"

namespace msla {
namespace {

using bf16 = __nv_bfloat16;
constexpr int CB = 32;                        // channels per block
constexpr int TH = 16, NB = 3, TW = 8 * NB;   // output rows and pixels per tile
constexpr int BOXW = TW + 16;                 // staged pixels per row: x0-8 .. x0+31
constexpr int BOXR = TH / 2 + 2;              // staged rows per parity
constexpr int ROW_B = BOXW * 2;               // 80 bytes: 16 * 5, odd in 16-byte units
constexpr int CH_B = BOXR * ROW_B;            // 800 bytes per channel and parity
constexpr int HALF_B = CB * CH_B;             // one TMA box
constexpr int BOX_BYTES = 2 * HALF_B;
constexpr int DWO_CH = 2 * NB * 128 + 16;     // depthwise output: bytes per channel, odd in 16-byte units
constexpr int DWO_BYTES = CB * DWO_CH;
constexpr int SLAB_B = CB * TW * 2;           // one image row of the tile, all 32 channels
constexpr int T_WARPS = 8;
constexpr int T_THREADS = 32 * T_WARPS;
constexpr int SLABS_BYTES = T_WARPS * 2 * SLAB_B;
constexpr int T_BAND = 4;                     // tile rows per band of the traversal
constexpr int T_SMEM_BYTES = 1024 + BOX_BYTES + DWO_BYTES + SLABS_BYTES;
constexpr long long T_WAIT_LIMIT_CYCLES = 4000000000LL;
static_assert((ROW_B / 16) % 2 == 1 && (DWO_CH / 16) % 2 == 1 && ((TW * 2) / 16) % 2 == 1, "bank-conflict-free pitches");
static_assert(HALF_B % 128 == 0 && DWO_BYTES % 128 == 0 && SLAB_B % 128 == 0, "TMA buffers must stay 128-byte aligned");

__device__ int g_agg_timeout_flag = 0;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v) { asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory"); }

struct AggParams {
  const bf16* w_dw;  // [Ch][5][5]
  const bf16* w_pw;  // [Ch][d]
  int Ch, d, H, W;
  int blocks;                         // blocks of 32 channels per image
  int tiles_x, tiles_y, tiles_total;  // tiles per channel plane
  long long units;                    // B * blocks * tiles_total, tile fastest
  long long units_per_cta;
};

__global__ void __launch_bounds__(T_THREADS, 2)
aggregate_nchw_kernel(const __grid_constant__ CUtensorMap tm_even, const __grid_constant__ CUtensorMap tm_odd,
                      const __grid_constant__ CUtensorMap tm_dst, AggParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t box = (smem_addr(smem_raw) + 1023u) & ~1023u;
  const uint32_t dwo = box + BOX_BYTES, slabs = dwo + DWO_BYTES;
  __shared__ __align__(8) unsigned long long bar_storage;
  __shared__ int timed_out;

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const long long unit_first = (long long)blockIdx.x * p.units_per_cta;
  const int unit_count = (int)max(0LL, min(p.units_per_cta, p.units - unit_first));
  const uint32_t bar = smem_addr(&bar_storage);

  // Cursor over (image, block, tile) units, tile fastest, advanced without divisions.  Inside a plane the
  // tiles run down bands of T_BAND tile rows, column by column, so that a tile's lower and right
  // neighbours follow within a few iterations and find the shared halo rows and columns in L2.
  struct Unit { int tile, tx, ty, band_end, blk, b; };  // band_end: first tile row below the current band
  auto locate = [&](long long u) {
    const long long bg = u / p.tiles_total;
    Unit r;
    r.tile = (int)(u - bg * p.tiles_total);
    const int band = r.tile / (T_BAND * p.tiles_x), rem = r.tile - band * (T_BAND * p.tiles_x);
    r.band_end = min(band * T_BAND + T_BAND, p.tiles_y);
    const int bh = r.band_end - band * T_BAND;
    r.tx = rem / bh;
    r.ty = band * T_BAND + rem - r.tx * bh;
    r.b = (int)(bg / p.blocks);
    r.blk = (int)(bg - (long long)r.b * p.blocks);
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
      if (++u.blk == p.blocks) { u.blk = 0; ++u.b; }
    }
  };
  // x and the row index may start below 0 and run past the image: the TMA unit returns zeros there.
  auto issue = [&](const Unit& u) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(BOX_BYTES) : "memory");
    const int x = u.tx * TW - 8, r = u.ty * (TH / 2) - 1, c = u.blk * CB;
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(box), "l"(&tm_even), "r"(bar), "r"(x), "r"(r), "r"(c), "r"(u.b) : "memory");
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(box + HALF_B), "l"(&tm_odd), "r"(bar), "r"(x), "r"(r), "r"(c), "r"(u.b) : "memory");
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
  uint32_t aw[2][2][4];  // 1x1 weights as A fragments: [16 output channels][16 input channels] blocks
  const bool d16 = p.d == 16;
  auto load_weights = [&](int blk) {
    const int ch0 = blk * CB;
    // lane (g, t) holds rows k = 2t, 2t+1 (b0) and 2t+8, 2t+9 (b1) of column n = g, i.e. taps dx = k - g - 2 of filter row dy
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
      const int ch = ch0 + 4 * warp + cc;
      const bool in = ch < p.Ch;
#pragma unroll
      for (int dy = 0; dy < 5; ++dy) {
        const bf16* wrow = p.w_dw + (long long)(in ? ch : 0) * 25 + dy * 5;
        const int i0 = 2 * t - g - 2;
        auto tap = [&](int i) -> uint32_t { return (in && i >= 0 && i < 5) ? (uint32_t)__bfloat16_as_ushort(wrow[i]) : 0u; };
        bt[cc][dy][0] = tap(i0) | (tap(i0 + 1) << 16);
        bt[cc][dy][1] = tap(i0 + 8) | (tap(i0 + 9) << 16);
      }
    }
    // A fragment of block (mb, kb): a0 = (row g, k 2t..), a1 = (row g+8, k 2t..), a2 = (row g, k 2t+8..), a3 = (row g+8, k 2t+8..)
#pragma unroll
    for (int mb = 0; mb < 2; ++mb)
#pragma unroll
      for (int kb = 0; kb < 2; ++kb)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int o = ch0 + 16 * mb + g + 8 * (e & 1);   // output channel
          const int k = 16 * kb + 2 * t + 8 * (e >> 1);    // input channel within the block
          uint32_t v = 0u;
          if (o < p.Ch) {
            if (d16) { if (mb == kb) v = *reinterpret_cast<const uint32_t*>(p.w_pw + (long long)o * 16 + (k - 16 * kb)); }
            else v = *reinterpret_cast<const uint32_t*>(p.w_pw + (long long)o * 32 + k);
          }
          aw[mb][kb][e] = v;
        }
  };
  int cur_blk = un.blk;
  load_weights(cur_blk);

  const uint32_t lane_off = (uint32_t)(g * ROW_B + 8 + t * 4);  // row g of a parity, pixels 4 + 2t, +1 of the staged row
  __syncthreads();  // barrier initialised before anyone waits on it
  pdl_wait();

  const uint32_t my_slabs = slabs + (uint32_t)(warp * 2 * SLAB_B);
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
    if (un.blk != cur_blk) {  // uniform over the CTA
      cur_blk = un.blk;
      load_weights(cur_blk);
    }
    const int nbv = min(NB, (p.W - x0 + 7) >> 3);  // 8-pixel column blocks that lie inside the image

    // ---- P2: depthwise 5x5 of channels 4w .. 4w+3
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
      const int c = 4 * warp + cc;
      const uint32_t cb = box + (uint32_t)(c * CH_B) + lane_off;
      uint32_t R[6][NB + 1];  // R[r][h]: staged row 2g + r, pixels 4 + 8h + 2t, +1
#pragma unroll
      for (int r = 0; r < 6; ++r)
#pragma unroll
        for (int h = 0; h <= NB; ++h) R[r][h] = lds32(cb + (uint32_t)((r & 1) * HALF_B + (r >> 1) * ROW_B + h * 16));
      float acc[NB][4];
#pragma unroll
      for (int nb = 0; nb < NB; ++nb)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[nb][e] = 0.f;
#pragma unroll
      for (int dy = 0; dy < 5; ++dy)
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
          if (nb < nbv) mma_bf16(acc[nb], R[dy][nb], R[dy + 1][nb], R[dy][nb + 1], R[dy + 1][nb + 1], bt[cc][dy][0], bt[cc][dy][1]);
      // pixel pair (row 2g + half, columns 8nb + 2t, +1) goes to word (2nb + half) * 32 + lane of the channel's row
      const uint32_t o = dwo + (uint32_t)(c * DWO_CH + lane * 4);
#pragma unroll
      for (int nb = 0; nb < NB; ++nb)
#pragma unroll
        for (int half = 0; half < 2; ++half)
          sts32(o + (uint32_t)((2 * nb + half) * 128), pack_bf16x2(acc[nb][2 * half], acc[nb][2 * half + 1]));
    }
    if (__syncthreads_or(timed_out)) {  // the copy had two seconds to land: give up, leave the output alone
      if (threadIdx.x == 0) atomicExch(&g_agg_timeout_flag, 1);
      break;
    }
    if (threadIdx.x == 0 && k + 1 < unit_count) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // order the generic reads above before the async write
      advance(nxt);
      issue(nxt);
    }

    // ---- P3: grouped 1x1 on the 48 pixels of image rows 2w, 2w+1.  8-pixel block q = (2nb + half) * 8 + w of the
    // depthwise tile is image row 2w + half, columns 8nb .. 8nb+7.
    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // the previous tile's stores have read the slabs
    __syncwarp();
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      if (nb >= nbv) break;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int q = (2 * nb + half) * 8 + warp;
        uint32_t b0, b1, b2, b3;  // B fragments: input channels 0-7, 8-15, 16-23, 24-31 of the block's 8 pixels
        ldsm_x4_trans(b0, b1, b2, b3, dwo + (uint32_t)((8 * (lane >> 3) + (lane & 7)) * DWO_CH + q * 16));
        float c[2][4];
#pragma unroll
        for (int mb = 0; mb < 2; ++mb) {
#pragma unroll
          for (int e = 0; e < 4; ++e) c[mb][e] = 0.f;
          if (!d16 || mb == 0) mma_bf16(c[mb], aw[mb][0][0], aw[mb][0][1], aw[mb][0][2], aw[mb][0][3], b0, b1);
          if (!d16 || mb == 1) mma_bf16(c[mb], aw[mb][1][0], aw[mb][1][1], aw[mb][1][2], aw[mb][1][3], b2, b3);
        }
        // slab of image row 2w + half: [channel][24 pixels]; this lane holds channels 16mb + g, + 8, pixels 8nb + 2t, +1
        const uint32_t sl = my_slabs + (uint32_t)(half * SLAB_B + (8 * nb + 2 * t) * 2);
#pragma unroll
        for (int mb = 0; mb < 2; ++mb) {
          sts32(sl + (uint32_t)((16 * mb + g) * (TW * 2)), pack_bf16x2(c[mb][0], c[mb][1]));
          sts32(sl + (uint32_t)((16 * mb + g + 8) * (TW * 2)), pack_bf16x2(c[mb][2], c[mb][3]));
        }
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (lane == 0) {  // pixels and channels outside the tensor are clipped by the TMA unit
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int y = y0 + 2 * warp + half;
        if (y < p.H)
          asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                       ::"l"(&tm_dst), "r"(my_slabs + (uint32_t)(half * SLAB_B)), "r"(x0), "r"(y), "r"(un.blk * CB), "r"(un.b) : "memory");
      }
      asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    }
    __syncthreads();  // every warp has read the depthwise tile before the next tile's P2 overwrites it
  }
  if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // stores done before the CTA retires
}

}  // namespace

bool aggregate_bf16_supported(int H, int W, int Ch, int d) {
  return (d == 32 || d == 16) && Ch % d == 0 && H >= 2 && W >= 8 && W % 8 == 0;
}

// src, dst: channel-major bf16 [B, Ch, H, W] with batch strides src_sb, dst_sb (elements, multiples of 8); w_dw [Ch][5][5],
// w_pw [Ch][d]; W a multiple of 8 (rows must start on 16-byte boundaries for the TMA unit), H >= 2.
msla_status_t run_aggregate_bf16(const void* src, long long src_sb, const void* w_dw, const void* w_pw, void* dst,
                                 long long dst_sb, int B, int H, int W, int Ch, int d, cudaStream_t st) {
  if (!aggregate_bf16_supported(H, W, Ch, d) || src_sb % 8 != 0 || dst_sb % 8 != 0)
    return fail(MSLA_ERR_UNSUPPORTED, "aggregation: d = %d, %d channels, %d x %d pixels", d, Ch, H, W);
  CUtensorMap tm_even, tm_odd, tm_dst;
  {
    const cuuint64_t de[4] = {(cuuint64_t)W, (cuuint64_t)((H + 1) / 2), (cuuint64_t)Ch, (cuuint64_t)B};
    const cuuint64_t dodd[4] = {(cuuint64_t)W, (cuuint64_t)(H / 2), (cuuint64_t)Ch, (cuuint64_t)B};
    const cuuint64_t sp[3] = {(cuuint64_t)W * 4, (cuuint64_t)H * W * 2, (cuuint64_t)src_sb * 2};
    const cuuint32_t bx[4] = {(cuuint32_t)BOXW, (cuuint32_t)BOXR, (cuuint32_t)CB, 1};
    const cuuint64_t dd[4] = {(cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)Ch, (cuuint64_t)B};
    const cuuint64_t sd[3] = {(cuuint64_t)W * 2, (cuuint64_t)H * W * 2, (cuuint64_t)dst_sb * 2};
    const cuuint32_t ob[4] = {(cuuint32_t)TW, 1, (cuuint32_t)CB, 1};
    if (!tma_make_map_bf16(&tm_even, src, 4, de, sp, bx, CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !tma_make_map_bf16(&tm_odd, (const bf16*)src + W, 4, dodd, sp, bx, CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !tma_make_map_bf16(&tm_dst, dst, 4, dd, sd, ob, CU_TENSOR_MAP_SWIZZLE_NONE))
      return fail(MSLA_ERR_CUDA, "cuTensorMapEncodeTiled failed for the aggregation");
  }
  AggParams p;
  p.w_dw = (const bf16*)w_dw; p.w_pw = (const bf16*)w_pw;
  p.Ch = Ch; p.d = d; p.H = H; p.W = W;
  p.blocks = (Ch + CB - 1) / CB;
  p.tiles_x = (W + TW - 1) / TW;
  p.tiles_y = (H + TH - 1) / TH;
  const long long tiles = (long long)p.tiles_x * p.tiles_y;
  if (tiles > 0x7fffffffLL) return fail(MSLA_ERR_UNSUPPORTED, "too many aggregation tiles");
  p.tiles_total = (int)tiles;
  p.units = tiles * p.blocks * B;
  const int sms = device_sm_count();
  // two CTAs per SM; small problems get one unit per CTA
  const long long ctas = p.units < 2LL * sms ? p.units : 2LL * sms;
  p.units_per_cta = (p.units + ctas - 1) / ctas;
  if (p.units_per_cta > 0x7fffffffLL) return fail(MSLA_ERR_UNSUPPORTED, "too many aggregation tiles");
  const unsigned grid = (unsigned)((p.units + p.units_per_cta - 1) / p.units_per_cta);
  static std::atomic<unsigned long long> attr_done{0};
  msla_status_t s = ensure_smem_attr(attr_done, aggregate_nchw_kernel, T_SMEM_BYTES);
  if (s != MSLA_OK) return s;
  launch_pdl(aggregate_nchw_kernel, dim3(grid), dim3(T_THREADS), T_SMEM_BYTES, st, tm_even, tm_odd, tm_dst, p);
  count_launches(1);
  return check_launch("token aggregation (bf16)");
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
