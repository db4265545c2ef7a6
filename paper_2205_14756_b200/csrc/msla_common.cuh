// Shared device/host helpers for libmsla kernels (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace msla {

// Strided view of per-head token matrices: element (b, h, n, i) of tensor t is
//   t[b * batch + h * head + n * ld + i].
// Dense [B, heads, N, d] input:        batch = heads*N*d, head = N*d, ld = d.
// Token-major multi-scale buffer
// [B, N, 6C'] with [q|k|v] per head:   batch = N*6C',  head = 3d,  ld = 6C'.
// Paired heads (pair = 1, outputs only): heads 2p and 2p+1 share one [N][2d]
// plane, head 2p+1 in its upper d columns:
//   t[b * batch + (h / 2) * head + (h % 2) * d + n * ld + i],  ld = 2d.
struct HeadView {
  long long batch;
  long long head;
  long long ld;
  int pair;
};

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float to_f32(__half v) { return __half2float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) {
  return __float2bfloat16_rn(v);
}
template <> __device__ __forceinline__ __half from_f32<__half>(float v) { return __float2half_rn(v); }

// Programmatic dependent launch.  The tuned kernels are launched so that a
// kernel may become resident while its predecessor in the stream is still
// running: it sets up what depends on no earlier kernel (barriers, tensor
// memory, tables built from the weights) and then waits here, which returns
// once the predecessor has finished and its writes are visible.  Every global
// read of an earlier kernel's output, and every global write, comes after it.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel of the stream be scheduled as soon as every CTA of this
// one has started (it still waits in pdl_wait for this kernel's completion).
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__host__ __device__ __forceinline__ long long ceil_div_ll(long long a, long long b) {
  return (a + b - 1) / b;
}

}  // namespace msla
