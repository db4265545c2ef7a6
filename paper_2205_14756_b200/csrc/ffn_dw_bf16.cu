// The depthwise convolution inserted into the FFN (Section 3.1: a depthwise convolution in each FFN layer supplies
// the local information ReLU linear attention lacks; Fig. 2 left), with the bias (a folded normalisation) and the
// activation that follow it:
//
//   g[b][c][y][x] = act( sum_{dy,dx} w[c][dy][dx] * h[b][c][y+dy-1][x+dx-1] + bias[c] ),   3x3, zero padding 1
//
// on the hidden tensor kept as planes of 64 channels, h[b][c / 64][y*W + x][c % 64]: what the first linear layer's
// epilogue writes and what the second one's tile loads want (128-byte token rows).
//
// The filter has no contraction over channels, so there is nothing for the tensor cores: at 9 multiply-adds per
// element read and written (2.25 MAC per byte) the step is bound by HBM as long as the loads stay low.  A thread owns
// 8 channels (16 bytes) of one pixel column and walks R rows with the three filter rows' partial sums in registers:
// every input row is loaded once per column triple (3 vectors per output instead of 9), a warp's loads and stores
// are 512 contiguous bytes, and the 72 filter taps of the thread's channels sit in registers as fp32.
#include "msla_common.cuh"
#include "msla_host.h"
#include "tcgen05_util.cuh"

namespace msla {
namespace {

using bf16 = __nv_bfloat16;

constexpr int DW_PX = 32;      // pixel columns per CTA
constexpr int DW_ROWS = 8;     // output rows per CTA
constexpr int DW_THREADS = DW_PX * 8;

__device__ __forceinline__ float dw_act(float v, int act) {
  if (act == 1) return fmaxf(v, 0.f);
  if (act == 2) return v * __saturatef((v + 3.f) * (1.f / 6.f));  // v * min(max(v + 3, 0), 6) / 6
  return v;
}

__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    f[2 * e] = __uint_as_float(w[e] << 16);
    f[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
  }
}

// grid: (ceil(W / DW_PX), ceil(H / DW_ROWS), B * planes); planes = Ch / 64
__global__ void __launch_bounds__(DW_THREADS)
ffn_dw3x3_kernel(const bf16* __restrict__ h, const bf16* __restrict__ w_dw, const bf16* __restrict__ b_dw, bf16* __restrict__ g,
                 int H, int W, int planes, int act) {
  __shared__ float wsh[9][64];
  __shared__ float bsh[64];
  pdl_launch_dependents();
  const int plane = blockIdx.z % planes;
  for (int i = threadIdx.x; i < 9 * 64; i += DW_THREADS) {  // weights do not come from the previous kernel
    const int c = i / 9, t = i - c * 9;
    wsh[t][c] = __bfloat162float(w_dw[(long long)(plane * 64 + c) * 9 + t]);
  }
  for (int i = threadIdx.x; i < 64; i += DW_THREADS) bsh[i] = b_dw ? __bfloat162float(b_dw[plane * 64 + i]) : 0.f;
  __syncthreads();
  const int c8 = threadIdx.x & 7, x = blockIdx.x * DW_PX + (threadIdx.x >> 3);
  float wt[9][8], bias[8];
#pragma unroll
  for (int t = 0; t < 9; ++t)
#pragma unroll
    for (int i = 0; i < 8; ++i) wt[t][i] = wsh[t][c8 * 8 + i];
#pragma unroll
  for (int i = 0; i < 8; ++i) bias[i] = bsh[c8 * 8 + i];
  pdl_wait();  // h is the previous kernel's output
  if (x >= W) return;
  const long long base = (long long)blockIdx.z * H * W * 64 + c8 * 8;
  const bf16* hp = h + base;
  bf16* gp = g + base;
  const int y0 = blockIdx.y * DW_ROWS;
  const bool has_l = x > 0, has_r = x + 1 < W;
  float acc[3][8];  // acc[o % 3]: output row o under construction
#pragma unroll
  for (int r = 0; r < DW_ROWS + 2; ++r) {  // input row y0 - 1 + r feeds output rows y0 + r - 2 .. y0 + r
    const int yi = y0 - 1 + r;
    const bool row_in = yi >= 0 && yi < H;
    float in[3][8];
    {
      const uint4 z = make_uint4(0u, 0u, 0u, 0u);
      const bf16* rp = hp + ((long long)yi * W + x) * 64;
      const uint4 vl = (row_in && has_l) ? __ldg(reinterpret_cast<const uint4*>(rp - 64)) : z;
      const uint4 vc = row_in ? __ldg(reinterpret_cast<const uint4*>(rp)) : z;
      const uint4 vr = (row_in && has_r) ? __ldg(reinterpret_cast<const uint4*>(rp + 64)) : z;
      unpack8(vl, in[0]); unpack8(vc, in[1]); unpack8(vr, in[2]);
    }
#pragma unroll
    for (int dy = 0; dy < 3; ++dy) {       // this input row is filter row dy of output row o = r - dy (relative to y0)
      const int o = r - dy;
      if (o < 0 || o >= DW_ROWS) continue;
      float (&a)[8] = acc[o % 3];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float v = dy == 0 ? bias[i] : a[i];  // filter row 0 opens the accumulator
        v = fmaf(wt[dy * 3 + 0][i], in[0][i], v);
        v = fmaf(wt[dy * 3 + 1][i], in[1][i], v);
        v = fmaf(wt[dy * 3 + 2][i], in[2][i], v);
        a[i] = v;
      }
    }
    const int od = r - 2;                  // output row completed by this input row
    if (od >= 0 && y0 + od < H) {
      const float (&a)[8] = acc[od % 3];
      uint4 out;
      out.x = pack2(dw_act(a[0], act), dw_act(a[1], act));
      out.y = pack2(dw_act(a[2], act), dw_act(a[3], act));
      out.z = pack2(dw_act(a[4], act), dw_act(a[5], act));
      out.w = pack2(dw_act(a[6], act), dw_act(a[7], act));
      *reinterpret_cast<uint4*>(gp + ((long long)(y0 + od) * W + x) * 64) = out;
    }
  }
}

}  // namespace

// h, g: [B][Ch / 64][H * W][64] bf16; w_dw [Ch][3][3]; b_dw [Ch] or nullptr.
msla_status_t run_ffn_dw3x3_bf16(const void* h, const void* w_dw, const void* b_dw, void* g, int B, int Ch, int H, int W, int act,
                                 cudaStream_t st) {
  const long long z = (long long)B * (Ch / 64);
  if (Ch % 64 != 0 || z > 65535 || (H + DW_ROWS - 1) / DW_ROWS > 65535)
    return fail(MSLA_ERR_UNSUPPORTED, "FFN depthwise convolution: %d hidden channels, batch %d, %d rows", Ch, B, H);
  launch_pdl(ffn_dw3x3_kernel, dim3((unsigned)((W + DW_PX - 1) / DW_PX), (unsigned)((H + DW_ROWS - 1) / DW_ROWS), (unsigned)z),
             dim3(DW_THREADS), 0, st, (const bf16*)h, (const bf16*)w_dw, (const bf16*)b_dw, (bf16*)g, H, W, Ch / 64, act);
  count_launches(1);
  return check_launch("FFN depthwise convolution (bf16)");
}

}  // namespace msla
