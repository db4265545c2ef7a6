// Host-side declarations shared by the translation units of libmsla.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>

#include <atomic>

#include "../../include/msla.h"

namespace msla {

// Carving of the attention core's scratch: fp32 partial states
// [BH][S][d*(d+1)] at partial_off, combined states [BH][d*(d+1)] at state_off.
struct CorePlan {
  int S;       // number of token chunks per (batch, head)
  int chunk;   // tokens per chunk (multiple of 64)
  int ne;      // d*(d+1) state entries
  int apply_tokens;  // tokens per CTA of the tuned apply kernel (multiple of 256)
  size_t partial_off, state_off, bytes;
};

CorePlan make_core_plan(long long BH, int N, int d);

// Records a thread-local message and returns `st`.
msla_status_t fail(msla_status_t st, const char* fmt, ...);
// MSLA_OK, or MSLA_ERR_CUDA if a launch since the last check failed.
msla_status_t check_launch(const char* what);

void count_launches(int n);

// Function attributes (the dynamic shared-memory limit) belong to one device: a launch site keeps an
// atomic mask of the devices on which it has set them.  Bit of the current device; 0 for device numbers
// past 63, which makes the site set the attribute on every call there.
inline unsigned long long current_device_bit() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 0; }
  return (dev >= 0 && dev < 64) ? 1ull << dev : 0ull;
}

// Raises the dynamic shared-memory limit of `kernel` to `bytes` on the current device, once per device
// (two threads racing on the first call both set it, which is harmless).
template <typename Kernel>
inline msla_status_t ensure_smem_attr(std::atomic<unsigned long long>& done, Kernel kernel, int bytes) {
  const unsigned long long bit = current_device_bit();
  if (bit && (done.load(std::memory_order_acquire) & bit)) return MSLA_OK;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) {
    cudaGetLastError();
    return fail(MSLA_ERR_CUDA, "cannot reserve %d bytes of shared memory for a kernel", bytes);
  }
  done.fetch_or(bit, std::memory_order_release);
  return MSLA_OK;
}

// Number of SMs of the current device (looked up once per device).
int device_sm_count();

// Launches `kernel` with programmatic stream serialization allowed: it may become resident before the
// previous kernel of the stream has finished, and orders itself with pdl_wait() (msla_common.cuh).
template <typename... KArgs, typename... Args>
inline void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);  // errors surface in check_launch()
}

// The same for a kernel that runs as clusters of two CTAs (grid.x must be even).
template <typename... KArgs, typename... Args>
inline void launch_pdl_cluster2(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = 2;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);  // errors surface in check_launch()
}

struct HeadView;
// Tuned attention core for 16-bit storage, bf16 or (f16 = true) fp16 (d in {16, 32}); all view strides must be multiples of 8 elements.
// `phases` selects what runs: CORE_STATE the partial states (at ws + p.partial_off, p.S per head), CORE_COMBINE their
// fixed-order sum (at ws + p.state_off), CORE_APPLY the apply step reading that sum; without CORE_APPLY `out` and `ov` are unused.
enum : int { CORE_STATE = 1, CORE_COMBINE = 2, CORE_APPLY = 4, CORE_ALL = 7 };
msla_status_t run_core_bf16(const void* q, const void* k, const void* v, void* out, HeadView in, HeadView ov, int B,
                            int heads, int N, int d, float eps, const CorePlan& p, void* ws, cudaStream_t st,
                            cudaEvent_t mid, int phases, bool f16 = false);

// FFN with a depthwise convolution (gemm_tcgen05.cu, ffn_dw_bf16.cu): bf16; the hidden tensor is planes of 32 channels
// [B][Ch / 32][N][32] after the first layer, planes of 64 channels [B][Ch / 64][N][64] after the depthwise convolution.
// act: 0 none, 1 ReLU, 2 hard-swish.
bool ffn_bf16_supported(int C, int Ch, int Cout, int N);
msla_status_t run_ffn_expand_bf16(const void* x, const void* w1, const void* b1, void* h, int B, int C, int Ch, int N, int act,
                                  cudaStream_t st, bool f16 = false);
msla_status_t run_ffn_dw3x3_bf16(const void* h, const void* w_dw, const void* b_dw, void* g, int B, int Ch, int H, int W, int act,
                                 cudaStream_t st, bool f16 = false);
msla_status_t run_ffn_project_bf16(const void* g, const void* w2, const void* b2, const void* residual, void* y, int B, int Ch,
                                   int Cout, int N, cudaStream_t st, bool f16 = false);

// Apply step and output projection as one GEMM per image (fused_out.cu): bf16, d in {16, 32}, at most 512 attention
// channels and 256 output channels.  q: planar query matrices [N][d], head h of image b at q + b*q_sb + h*q_sh
// (elements).
bool fused_out_bf16_supported(int Ht, int d, int Cout, int N);
size_t fused_out_scratch_bytes(int B, int Ht, int d, int Cout);
msla_status_t run_fused_out_bf16(const void* q, long long q_sb, long long q_sh, const float* partial, int S, void* scratch,
                                 const void* w, const void* bias, const void* residual, void* y, int B, int Ht, int d, int N, int Cout,
                                 float eps, cudaStream_t st, bool f16 = false);
int fused_timeout_flag();
int dw_timeout_flag();

// bf16 projections on tcgen05 tensor cores (gemm_tcgen05.cu).
bool project_in_bf16_supported(int C, int Cout, int N, int d);
msla_status_t run_project_in_bf16(const void* x, const void* w, void* y, int B, int C, int Cout, int N, int d,
                                  long long y_batch_stride, cudaStream_t st, bool f16 = false);
bool project_out_bf16_supported(int Cin, int Cout, int N);
// residual: nullptr, or a tensor shaped like y that is added to it
msla_status_t run_project_out_bf16(const void* a, const void* w, const void* bias, const void* residual, void* y, int B, int Cin,
                                   int Cout, int N, cudaStream_t st, bool f16 = false);
bool project_out_planar_bf16_supported(int Cin, int Cout, int N);
msla_status_t run_project_out_planar_bf16(const void* a, const void* w, const void* bias, const void* residual, void* y, int B,
                                          int Cin, int Cout, int N, cudaStream_t st, bool f16 = false);
int gemm_timeout_flag();
int run_wait_selftest(long long limit_cycles, int* scratch, cudaStream_t st);

// bf16 aggregation (d = 16 or 32, Ch a multiple of 32): TMA halo tiles, depthwise filter as banded matrices on
// tensor cores (agg_bf16.cu).  dst_sb must be a multiple of the plane size H*W*d.
bool aggregate_bf16_supported(int H, int W, int Ch, int d);
msla_status_t run_aggregate_bf16(const void* src, long long src_planes_total, int src_ppb, const void* w_dw,
                                 const void* w_pw, void* dst, long long dst_sb, int B, int H, int W, int Ch, int d,
                                 cudaStream_t st, bool f16 = false);
int agg_timeout_flag();

}  // namespace msla
