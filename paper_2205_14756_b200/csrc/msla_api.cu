// C ABI of libmsla: host-side validation, workspace carving and kernel dispatch.
#include "../../include/msla.h"

#include <atomic>
#include <cstdarg>
#include <type_traits>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "generic_kernels.cuh"
#include "msla_common.cuh"
#include "msla_host.h"

namespace msla {

static thread_local char g_last_error[512] = "";

msla_status_t fail(msla_status_t st, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_last_error, sizeof(g_last_error), fmt, ap);
  va_end(ap);
  return st;
}

static thread_local unsigned long long g_launches = 0;
void count_launches(int n) { g_launches += (unsigned long long)n; }

msla_status_t check_launch(const char* what) {
  const cudaError_t e = cudaPeekAtLastError();
  if (e != cudaSuccess) {
    cudaGetLastError();
    return fail(MSLA_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
  }
  return MSLA_OK;
}

// The library's kernels are built for sm_100a only, and an architecture-specific image loads on no other
// device: compute capability 10.0 exactly.
static msla_status_t check_arch() {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return fail(MSLA_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  }
  static std::atomic<int> cached_cc[64];  // major * 16 + minor + 1; 0 = unknown
  int cc = (dev >= 0 && dev < 64) ? cached_cc[dev].load(std::memory_order_relaxed) : 0;
  if (cc == 0) {
    int major = 0, minor = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev);
    if (e != cudaSuccess) {
      cudaGetLastError();
      return fail(MSLA_ERR_CUDA, "cudaDeviceGetAttribute: %s", cudaGetErrorString(e));
    }
    cc = major * 16 + minor + 1;
    if (dev >= 0 && dev < 64) cached_cc[dev].store(cc, std::memory_order_relaxed);
  }
  if (cc != 10 * 16 + 0 + 1)
    return fail(MSLA_ERR_ARCH, "device %d has compute capability %d.%d; 10.0 (sm_100a) is required", dev, (cc - 1) / 16, (cc - 1) % 16);
  return MSLA_OK;
}

int device_sm_count() {
  static std::atomic<int> cached[64];  // 0 = unknown
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 148; }
  int n = (dev >= 0 && dev < 64) ? cached[dev].load(std::memory_order_relaxed) : 0;
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) { cudaGetLastError(); n = 148; }
    if (dev >= 0 && dev < 64) cached[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
  const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
  return a0 < b0 + nb && b0 < a0 + na;
}

static size_t elem_size(msla_dtype_t t) { return t == MSLA_F32 ? 4 : 2; }
static bool known_dtype(msla_dtype_t t) { return t == MSLA_F32 || t == MSLA_BF16 || t == MSLA_F16; }
static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ----------------------------------------------------------------- core plan
// The split of the token reduction is a function of the shape only.
CorePlan make_core_plan(long long BH, int N, int d) {
  CorePlan p;
  p.ne = d * (d + 1);
  const long long s_max = ceil_div_ll(N, 256);
  const long long s_want = ceil_div_ll(592, BH);
  long long S = s_max < s_want ? s_max : s_want;
  if (S > 64) S = 64;
  if (S < 1) S = 1;
  long long chunk = ceil_div_ll(N, S);
  chunk = ceil_div_ll(chunk, 64) * 64;
  p.chunk = (int)chunk;
  p.S = (int)ceil_div_ll(N, chunk);
  long long at = ceil_div_ll(ceil_div_ll((long long)N * BH, 1184), 256) * 256;
  p.apply_tokens = (int)(at < 256 ? 256 : (at > 2048 ? 2048 : at));
  p.partial_off = 0;
  p.state_off = align_up((size_t)BH * p.S * p.ne * sizeof(float), 256);
  p.bytes = p.state_off + align_up((size_t)BH * p.ne * sizeof(float), 256);
  return p;
}

static bool core_shape_ok(int B, int heads, int N, int d) {
  return B >= 1 && heads >= 1 && N >= 1 && (d == 16 || d == 32) && (long long)B * heads <= 65535;
}

template <typename T>
static msla_status_t run_core_generic(const T* q, const T* k, const T* v, T* out, HeadView in,
                                      HeadView ov, int B, int heads, int N, int d, float eps,
                                      const CorePlan& p, char* ws, cudaStream_t st, cudaEvent_t mid, int phases) {
  const long long BH = (long long)B * heads;
  float* partial = reinterpret_cast<float*>(ws + p.partial_off);
  float* state = reinterpret_cast<float*>(ws + p.state_off);
  int launches = 0;
  if (phases & CORE_STATE) {
    generic::kv_partial_kernel<T><<<dim3((unsigned)BH, p.S), 256, 0, st>>>(k, v, partial, in, heads, N, d, p.S, p.chunk);
    ++launches;
  }
  if (phases & CORE_COMBINE) {
    const long long total = BH * p.ne;
    generic::kv_combine_kernel<<<(unsigned)ceil_div_ll(total, 256), 256, 0, st>>>(partial, state, p.S, p.ne, total);
    ++launches;
  }
  if (mid) cudaEventRecord(mid, st);
  if (phases & CORE_APPLY) {
    generic::apply_kernel<T><<<dim3((unsigned)ceil_div_ll(N, 128), (unsigned)BH), 128, 0, st>>>(
        q, state, out, in, ov, heads, N, d, eps);
    ++launches;
  }
  count_launches(launches);
  return check_launch("attention core kernels");
}

// q/k/v views share strides; k = q + d and v = q + 2d in the module layout,
// separate tensors in the dense layout, so three pointers are passed.
static msla_status_t run_core(msla_dtype_t dtype, const void* q, const void* k, const void* v,
                              void* out, HeadView in, HeadView ov, int B, int heads, int N, int d,
                              float eps, const CorePlan& p, void* ws, cudaStream_t st,
                              cudaEvent_t mid = nullptr, int phases = CORE_ALL) {
  if (ov.pair && (dtype == MSLA_F32 || (heads & 1)))  // only the tensor-core kernels write paired planes
    return fail(MSLA_ERR_UNSUPPORTED, "paired output planes need 16-bit storage and an even number of heads");
  if (dtype == MSLA_F32)
    return run_core_generic<float>((const float*)q, (const float*)k, (const float*)v, (float*)out,
                                   in, ov, B, heads, N, d, eps, p, (char*)ws, st, mid, phases);
  if (dtype == MSLA_F16) {  // the tensor-core kernels take fp16 too; other strides run on the plain kernels
    const bool ok16 = in.batch % 8 == 0 && in.head % 8 == 0 && in.ld % 8 == 0 && ov.batch % 8 == 0 && ov.head % 8 == 0 && ov.ld % 8 == 0;
    if (ok16) return run_core_bf16(q, k, v, out, in, ov, B, heads, N, d, eps, p, ws, st, mid, phases, true);
    if (ov.pair) return fail(MSLA_ERR_UNSUPPORTED, "paired output planes need strides that are multiples of 8 elements");
    return run_core_generic<__half>((const __half*)q, (const __half*)k, (const __half*)v, (__half*)out,
                                    in, ov, B, heads, N, d, eps, p, (char*)ws, st, mid, phases);
  }
  const bool strides_ok = in.batch % 8 == 0 && in.head % 8 == 0 && in.ld % 8 == 0 && ov.batch % 8 == 0 &&
                          ov.head % 8 == 0 && ov.ld % 8 == 0;
  if (strides_ok) return run_core_bf16(q, k, v, out, in, ov, B, heads, N, d, eps, p, ws, st, mid, phases);
  if (ov.pair) return fail(MSLA_ERR_UNSUPPORTED, "paired output planes need strides that are multiples of 8 elements");
  return run_core_generic<__nv_bfloat16>((const __nv_bfloat16*)q, (const __nv_bfloat16*)k,
                                         (const __nv_bfloat16*)v, (__nv_bfloat16*)out, in, ov, B,
                                         heads, N, d, eps, p, (char*)ws, st, mid, phases);
}

static msla_status_t core_entry(msla_dtype_t dtype, const void* q, const void* k, const void* v,
                                void* out, int B, int heads, int N, int d, float eps, void* ws,
                                size_t ws_bytes, bool own_ws, cudaStream_t st) {
  if (!known_dtype(dtype)) return fail(MSLA_ERR_INVALID_ARG, "unknown dtype %d", (int)dtype);
  if (!q || !k || !v || !out) return fail(MSLA_ERR_INVALID_ARG, "null tensor pointer");
  if (B < 1 || heads < 1 || N < 1 || d < 1) return fail(MSLA_ERR_INVALID_ARG, "B, heads, N, d must be positive (got %d, %d, %d, %d)", B, heads, N, d);
  if (!(eps >= 0.f)) return fail(MSLA_ERR_INVALID_ARG, "eps must be >= 0");
  if (d != 16 && d != 32) return fail(MSLA_ERR_UNSUPPORTED, "d = %d; only 16 and 32 are supported", d);
  if ((long long)B * heads > 65535) return fail(MSLA_ERR_UNSUPPORTED, "B*heads = %lld exceeds 65535", (long long)B * heads);
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return fail(MSLA_ERR_ALIGNMENT, "q, k, v, out must be 16-byte aligned");
  const size_t bytes = (size_t)B * heads * N * d * elem_size(dtype);
  if (overlaps(out, bytes, q, bytes) || overlaps(out, bytes, k, bytes) || overlaps(out, bytes, v, bytes))
    return fail(MSLA_ERR_INVALID_ARG, "out overlaps an input");
  const CorePlan p = make_core_plan((long long)B * heads, N, d);
  if (!own_ws) {
    if (!ws || ws_bytes < p.bytes) return fail(MSLA_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", p.bytes, ws ? ws_bytes : (size_t)0);
    if (!aligned16(ws)) return fail(MSLA_ERR_ALIGNMENT, "workspace must be 16-byte aligned");
    if (overlaps(out, bytes, ws, p.bytes) || overlaps(q, bytes, ws, p.bytes) ||
        overlaps(k, bytes, ws, p.bytes) || overlaps(v, bytes, ws, p.bytes))
      return fail(MSLA_ERR_INVALID_ARG, "workspace overlaps a tensor");
  }
  msla_status_t s = check_arch();
  if (s != MSLA_OK) return s;
  if (own_ws) {
    const cudaError_t e = cudaMallocAsync(&ws, p.bytes, st);
    if (e != cudaSuccess) {
      cudaGetLastError();
      return fail(MSLA_ERR_CUDA, "cudaMallocAsync(%zu): %s", p.bytes, cudaGetErrorString(e));
    }
  }
  const HeadView in{(long long)heads * N * d, (long long)N * d, d};
  s = run_core(dtype, q, k, v, out, in, in, B, heads, N, d, eps, p, ws, st);
  if (own_ws) cudaFreeAsync(ws, st);
  return s;
}

// ------------------------------------------------ allocation-free variant
// Scratch for msla_linattn_relu_noalloc.  In host code this name is only a
// handle for the symbol; the address kernels can use comes from
// cudaGetSymbolAddress, queried once per device with that device current.
static __device__ __align__(256) unsigned char g_noalloc_scratch[MSLA_NOALLOC_SCRATCH_BYTES];

static msla_status_t noalloc_scratch(void** out_ptr) {
  static std::mutex mu;
  static void* per_device[64];  // nullptr = not looked up yet
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return fail(MSLA_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  }
  if (dev < 0 || dev >= 64) return fail(MSLA_ERR_UNSUPPORTED, "device ordinal %d is beyond the 64 this entry point tracks", dev);
  std::lock_guard<std::mutex> lock(mu);
  if (!per_device[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
    if (e != cudaSuccess || !ptr) {
      cudaGetLastError();
      return fail(MSLA_ERR_CUDA, "cudaGetSymbolAddress(scratch): %s", cudaGetErrorString(e));
    }
    per_device[dev] = ptr;
  }
  *out_ptr = per_device[dev];
  return MSLA_OK;
}

static msla_status_t core_entry_noalloc(msla_dtype_t dtype, const void* q, const void* k, const void* v,
                                        void* out, int B, int heads, int N, int d, float eps, cudaStream_t st) {
  if (!known_dtype(dtype)) return fail(MSLA_ERR_INVALID_ARG, "unknown dtype %d", (int)dtype);
  if (!q || !k || !v || !out) return fail(MSLA_ERR_INVALID_ARG, "null tensor pointer");
  if (B < 1 || heads < 1 || N < 1 || d < 1) return fail(MSLA_ERR_INVALID_ARG, "B, heads, N, d must be positive (got %d, %d, %d, %d)", B, heads, N, d);
  if (!(eps >= 0.f)) return fail(MSLA_ERR_INVALID_ARG, "eps must be >= 0");
  if (d != 16 && d != 32) return fail(MSLA_ERR_UNSUPPORTED, "d = %d; only 16 and 32 are supported", d);
  if ((long long)B * heads > 65535) return fail(MSLA_ERR_UNSUPPORTED, "B*heads = %lld exceeds 65535", (long long)B * heads);
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return fail(MSLA_ERR_ALIGNMENT, "q, k, v, out must be 16-byte aligned");
  const size_t bytes = (size_t)B * heads * N * d * elem_size(dtype);
  if (overlaps(out, bytes, q, bytes) || overlaps(out, bytes, k, bytes) || overlaps(out, bytes, v, bytes))
    return fail(MSLA_ERR_INVALID_ARG, "out overlaps an input");
  const CorePlan p = make_core_plan((long long)B * heads, N, d);
  if (p.bytes > (size_t)MSLA_NOALLOC_SCRATCH_BYTES)
    return fail(MSLA_ERR_WORKSPACE, "this shape needs %zu bytes of scratch; the built-in array holds %u (use msla_linattn_relu_ws)",
                p.bytes, (unsigned)MSLA_NOALLOC_SCRATCH_BYTES);
  msla_status_t s = check_arch();
  if (s != MSLA_OK) return s;
  void* ws = nullptr;
  if ((s = noalloc_scratch(&ws)) != MSLA_OK) return s;
  // Every partial and state entry the apply step reads is written earlier in
  // this same call, so nothing left over from a previous call needs clearing.
  const HeadView in{(long long)heads * N * d, (long long)N * d, d};
  return run_core(dtype, q, k, v, out, in, in, B, heads, N, d, eps, p, ws, st);
}

// ------------------------------------------------------------- module plan
struct ForwardPlan {
  size_t ms_off, att_off, core_off, wpad_off, bytes;  // wpad: 3x3 aggregation taps embedded in 5x5 (agg_kernel == 3)
  CorePlan core;
  int Cp, N;
  int S;              // branches: the projected tokens and S - 1 aggregated copies
  size_t wpad2_off;   // embedded taps of the second aggregated branch
};

static msla_status_t validate_desc(const msla_desc* d, ForwardPlan* plan) {
  if (!d) return fail(MSLA_ERR_INVALID_ARG, "null descriptor");
  if (d->struct_size != sizeof(msla_desc)) return fail(MSLA_ERR_INVALID_ARG, "desc.struct_size = %u, expected %zu", d->struct_size, sizeof(msla_desc));
  if (!known_dtype(d->dtype)) return fail(MSLA_ERR_INVALID_ARG, "unknown dtype %d", (int)d->dtype);
  if (d->B < 1 || d->C < 1 || d->H < 1 || d->W < 1 || d->heads < 1 || d->d < 1 || d->C_out < 1)
    return fail(MSLA_ERR_INVALID_ARG, "B, C, H, W, heads, d, C_out must be positive");
  if (!(d->eps >= 0.f)) return fail(MSLA_ERR_INVALID_ARG, "eps must be >= 0");
  if (d->n_scales != 2 && d->n_scales != 3) return fail(MSLA_ERR_UNSUPPORTED, "n_scales = %d; two or three branches are supported", d->n_scales);
  if (d->agg_kernel != 5 && d->agg_kernel != 3)
    return fail(MSLA_ERR_UNSUPPORTED, "agg_kernel = %d; 5x5 and 3x3 aggregation are supported", d->agg_kernel);
  if (d->n_scales == 3 && d->agg_kernel2 != 5 && d->agg_kernel2 != 3)
    return fail(MSLA_ERR_UNSUPPORTED, "agg_kernel2 = %d; 5x5 and 3x3 aggregation are supported", d->agg_kernel2);
  if (d->d != 16 && d->d != 32) return fail(MSLA_ERR_UNSUPPORTED, "d = %d; only 16 and 32 are supported", d->d);
  if ((long long)d->H * d->W > 0x7fffffffLL) return fail(MSLA_ERR_UNSUPPORTED, "H*W exceeds 2^31-1");
  if (d->C % 8 != 0 || d->C_out % 8 != 0) return fail(MSLA_ERR_UNSUPPORTED, "C and C_out must be multiples of 8");
  const int S = d->n_scales;
  if ((long long)d->B * S * d->heads > 65535 || d->B > 65535) return fail(MSLA_ERR_UNSUPPORTED, "B*n_scales*heads exceeds 65535");
  plan->S = S;
  plan->Cp = d->heads * d->d;
  plan->N = d->H * d->W;
  const size_t e = elem_size(d->dtype);
  const size_t tokens = (size_t)d->B * plan->N;
  plan->core = make_core_plan((long long)d->B * S * d->heads, plan->N, d->d);
  plan->ms_off = 0;
  plan->att_off = align_up(tokens * 3 * S * plan->Cp * e, 256);
  // the attention output's region doubles as scratch of the fused apply + projection kernel, which writes no attention output
  size_t att_bytes = tokens * S * plan->Cp * e;
  const size_t fused_scratch = fused_out_bf16_supported(S * d->heads, d->d, d->C_out, plan->N) ? fused_out_scratch_bytes(d->B, S * d->heads, d->d, d->C_out) : 0;
  if (att_bytes < fused_scratch) att_bytes = fused_scratch;
  plan->core_off = plan->att_off + align_up(att_bytes, 256);
  plan->wpad_off = plan->core_off + plan->core.bytes;
  plan->wpad2_off = plan->wpad_off + (d->agg_kernel == 3 ? align_up((size_t)3 * plan->Cp * 25 * e, 256) : 0);
  plan->bytes = plan->wpad2_off + (S == 3 && d->agg_kernel2 == 3 ? align_up((size_t)3 * plan->Cp * 25 * e, 256) : 0);
  return MSLA_OK;
}

template <typename T>
static void launch_gemm(const T* A, const T* W, const T* bias, T* D, generic::GemmArgs g, int B, cudaStream_t st) {
  dim3 grid((unsigned)ceil_div_ll(g.M, 64), (unsigned)ceil_div_ll(g.Nc, 64), (unsigned)B);
  generic::gemm_kernel<T><<<grid, 256, 0, st>>>(A, W, bias, D, g);
  count_launches(1);
}

// y planar: y[b*y_sb + ((o/d)*N + n)*d + o%d]
static msla_status_t run_project_in(msla_dtype_t dt, const void* x, const void* w, void* y, int B,
                                    int C, int Cout, int N, int d, long long y_sb, cudaStream_t st) {
  if (dt != MSLA_F32 && project_in_bf16_supported(C, Cout, N, d)) return run_project_in_bf16(x, w, y, B, C, Cout, N, d, y_sb, st, dt == MSLA_F16);
  generic::GemmArgs g{(long long)C * N, 1, N, y_sb, d, 1, (long long)N * d, N, Cout, C, d};
  if (dt == MSLA_F32) launch_gemm<float>((const float*)x, (const float*)w, nullptr, (float*)y, g, B, st);
  else if (dt == MSLA_F16) launch_gemm<__half>((const __half*)x, (const __half*)w, nullptr, (__half*)y, g, B, st);
  else launch_gemm<__nv_bfloat16>((const __nv_bfloat16*)x, (const __nv_bfloat16*)w, nullptr, (__nv_bfloat16*)y, g, B, st);
  return check_launch("input projection");
}

static msla_status_t run_project_out(msla_dtype_t dt, const void* a, const void* w, const void* bias,
                                     void* y, int B, int Cin, int Cout, int N, cudaStream_t st, const void* residual = nullptr) {
  if (dt != MSLA_F32 && project_out_bf16_supported(Cin, Cout, N))
    return run_project_out_bf16(a, w, bias, residual, y, B, Cin, Cout, N, st, dt == MSLA_F16);
  generic::GemmArgs g{(long long)N * Cin, Cin, 1, (long long)Cout * N, 1, N, 0, N, Cout, Cin, Cout, 0, residual};
  if (dt == MSLA_F32) launch_gemm<float>((const float*)a, (const float*)w, (const float*)bias, (float*)y, g, B, st);
  else if (dt == MSLA_F16) launch_gemm<__half>((const __half*)a, (const __half*)w, (const __half*)bias, (__half*)y, g, B, st);
  else launch_gemm<__nv_bfloat16>((const __nv_bfloat16*)a, (const __nv_bfloat16*)w, (const __nv_bfloat16*)bias, (__nv_bfloat16*)y, g, B, st);
  return check_launch("output projection");
}

// src, dst planar [B, Ch/d, H*W, d] with batch strides src_sb, dst_sb (elements)
static msla_status_t run_aggregate(msla_dtype_t dt, const void* src, const void* w_dw, const void* w_pw,
                                   void* dst, int B, int H, int W, int Ch, int d, long long src_sb,
                                   long long dst_sb, cudaStream_t st) {
  const long long plane = (long long)H * W * d;
  const bool f16 = dt == MSLA_F16;
  if (dt != MSLA_F32 && src_sb % plane == 0 && dst_sb % plane == 0) {
    if (aggregate_bf16_supported(H, W, Ch, d))
      return run_aggregate_bf16(src, (long long)B * (src_sb / plane), (int)(src_sb / plane), w_dw, w_pw, dst, dst_sb, B, H, W, Ch, d, st, f16);
    if (d == 16 && Ch > 16 && aggregate_bf16_supported(H, W, Ch - 16, d)) {
      // odd number of 16-channel groups: the tuned kernel takes them in pairs, the plain one the last group
      msla_status_t s = run_aggregate_bf16(src, (long long)B * (src_sb / plane), (int)(src_sb / plane), w_dw, w_pw, dst, dst_sb, B, H, W, Ch - 16, d, st, f16);
      if (s != MSLA_OK) return s;
      dim3 grid1((unsigned)(ceil_div_ll(W, 8) * ceil_div_ll(H, 8)), 1u, (unsigned)B);
      auto last_group = [&](auto* tag) {
        using T = std::remove_pointer_t<decltype(tag)>;
        generic::aggregate_kernel<T><<<grid1, 256, 0, st>>>((const T*)src + (long long)(Ch / 16 - 1) * plane, (const T*)w_dw + (long long)(Ch - 16) * 25,
                                                            (const T*)w_pw + (long long)(Ch - 16) * 16, (T*)dst + (long long)(Ch / 16 - 1) * plane, H, W, d,
                                                            src_sb, dst_sb);
      };
      if (f16) last_group((__half*)nullptr);
      else last_group((__nv_bfloat16*)nullptr);
      count_launches(1);
      return check_launch("token aggregation (last group)");
    }
  }
  dim3 grid((unsigned)(ceil_div_ll(W, 8) * ceil_div_ll(H, 8)), (unsigned)(Ch / d), (unsigned)B);
  if (dt == MSLA_F32)
    generic::aggregate_kernel<float><<<grid, 256, 0, st>>>((const float*)src, (const float*)w_dw, (const float*)w_pw,
                                                           (float*)dst, H, W, d, src_sb, dst_sb);
  else if (dt == MSLA_F16)
    generic::aggregate_kernel<__half><<<grid, 256, 0, st>>>((const __half*)src, (const __half*)w_dw, (const __half*)w_pw,
                                                            (__half*)dst, H, W, d, src_sb, dst_sb);
  else
    generic::aggregate_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)src, (const __nv_bfloat16*)w_dw,
                                                                   (const __nv_bfloat16*)w_pw, (__nv_bfloat16*)dst, H, W, d,
                                                                   src_sb, dst_sb);
  count_launches(1);
  return check_launch("token aggregation");
}

// The aggregation kernels are 5x5.  A 3x3 depthwise filter (another of Section 3.1's small kernels) is the same
// filter with a ring of zero taps around it: w5[c][dy+1][dx+1] = w3[c][dy][dx].  Returns the taps to use.
static const void* aggregation_taps(const msla_desc* desc, const msla_weights* w, const ForwardPlan& p, int branch, cudaStream_t st) {
  const void* w_dw = branch == 1 ? w->w_dw : w->w_dw2;
  if ((branch == 1 ? desc->agg_kernel : desc->agg_kernel2) == 5) return w_dw;
  void* w5 = (char*)desc->workspace + (branch == 1 ? p.wpad_off : p.wpad2_off);
  const long long total = 3LL * p.Cp * 25;
  if (desc->dtype == MSLA_F32)
    generic::embed_taps_kernel<float><<<(unsigned)ceil_div_ll(total, 256), 256, 0, st>>>((const float*)w_dw, (float*)w5, total);
  else  // 16-bit patterns are copied as they are: bf16 and fp16 alike (zero is all bits clear in both)
    generic::embed_taps_kernel<__nv_bfloat16><<<(unsigned)ceil_div_ll(total, 256), 256, 0, st>>>((const __nv_bfloat16*)w_dw, (__nv_bfloat16*)w5, total);
  count_launches(1);
  return w5;
}

// Step 2 for every aggregated branch: the scale-0 planes through that branch's filters into the branch's planes.
static msla_status_t run_branches(const msla_desc* desc, const msla_weights* w, const ForwardPlan& p, char* ms, long long ms_sb, cudaStream_t st) {
  const size_t branch_bytes = (size_t)3 * p.Cp * p.N * elem_size(desc->dtype);
  for (int br = 1; br < p.S; ++br) {
    const msla_status_t s = run_aggregate(desc->dtype, ms, aggregation_taps(desc, w, p, br, st), br == 1 ? w->w_pw : w->w_pw2, ms + br * branch_bytes,
                                          desc->B, desc->H, desc->W, 3 * p.Cp, desc->d, ms_sb, ms_sb, st);
    if (s != MSLA_OK) return s;
  }
  return MSLA_OK;
}

static msla_status_t record(void* const* events, int i, cudaStream_t st) {
  if (!events) return MSLA_OK;
  const cudaError_t e = cudaEventRecord((cudaEvent_t)events[i], st);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return fail(MSLA_ERR_CUDA, "cudaEventRecord: %s", cudaGetErrorString(e));
  }
  return MSLA_OK;
}

// host_io: x and out are host pointers staged through the tail of the workspace.
// residual: nullptr, or a device tensor shaped like out that the output projection adds (the block's first residual connection).
static msla_status_t forward_impl(const msla_desc* desc, const void* x, const msla_weights* w, void* out,
                                  cudaStream_t st, void* const* events, bool host_io, const void* residual = nullptr) {
  ForwardPlan p;
  msla_status_t s = validate_desc(desc, &p);
  if (s != MSLA_OK) return s;
  if (!x || !out || !w) return fail(MSLA_ERR_INVALID_ARG, "null x, out or weights");
  if (!w->w_qkv || !w->w_dw || !w->w_pw || !w->w_proj) return fail(MSLA_ERR_INVALID_ARG, "null weight pointer");
  if (p.S == 3 && (!w->w_dw2 || !w->w_pw2)) return fail(MSLA_ERR_INVALID_ARG, "three branches need w_dw2 and w_pw2");
  const void* ptrs[] = {host_io ? nullptr : x, host_io ? nullptr : out, w->w_qkv, w->w_dw, w->w_pw, w->w_proj, w->b_proj, desc->workspace,
                        p.S == 3 ? w->w_dw2 : nullptr, p.S == 3 ? w->w_pw2 : nullptr};
  for (const void* ptr : ptrs)
    if (ptr && !aligned16(ptr)) return fail(MSLA_ERR_ALIGNMENT, "all device pointers must be 16-byte aligned");
  const size_t e = elem_size(desc->dtype);
  const size_t xb = (size_t)desc->B * desc->C * p.N * e, ob = (size_t)desc->B * desc->C_out * p.N * e;
  const size_t need = p.bytes + (host_io ? align_up(xb, 256) + align_up(ob, 256) : 0);
  if (!desc->workspace || desc->workspace_bytes < need)
    return fail(MSLA_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, desc->workspace ? desc->workspace_bytes : (size_t)0);
  if (overlaps(out, ob, x, xb)) return fail(MSLA_ERR_INVALID_ARG, "out overlaps x");
  if (!host_io && (overlaps(out, ob, desc->workspace, need) || overlaps(x, xb, desc->workspace, need)))
    return fail(MSLA_ERR_INVALID_ARG, "workspace overlaps x or out");
  s = check_arch();
  if (s != MSLA_OK) return s;

  char* ws = (char*)desc->workspace;
  const void* x_dev = x;
  void* out_dev = out;
  if (host_io) {
    x_dev = ws + p.bytes;
    out_dev = ws + p.bytes + align_up(xb, 256);
    const cudaError_t ce = cudaMemcpyAsync((void*)x_dev, x, xb, cudaMemcpyHostToDevice, st);
    if (ce != cudaSuccess) {
      cudaGetLastError();
      return fail(MSLA_ERR_CUDA, "host-to-device copy of x: %s", cudaGetErrorString(ce));
    }
  }
  const int Cp = p.Cp, N = p.N, d = desc->d, heads = desc->heads;
  const int S = p.S, Ht = S * heads;
  const long long ld_att = (long long)S * Cp;
  const long long ms_sb = 3LL * S * Cp * N;  // elements per image of the multi-scale buffer
  // ms: planar [B][6*heads planes][N][d]; plane (s*heads + h)*3 + t holds q (t=0), k (1) or v (2)
  // of head h at scale s (0: projected tokens, 1: aggregated tokens).
  char* ms = ws + p.ms_off;
  char* att = ws + p.att_off;  // [B, N, 2C'] token-major head concat
  if ((s = record(events, 0, st)) != MSLA_OK) return s;
  // 1. QKV projection into the scale-0 planes
  s = run_project_in(desc->dtype, x_dev, w->w_qkv, ms, desc->B, desc->C, 3 * Cp, N, d, ms_sb, st);
  if (s != MSLA_OK) return s;
  if ((s = record(events, 1, st)) != MSLA_OK) return s;
  // 2. aggregation of every scale-0 plane into the matching scale-1 plane
  if ((s = run_branches(desc, w, p, ms, ms_sb, st)) != MSLA_OK) return s;
  if ((s = record(events, 2, st)) != MSLA_OK) return s;
  // 3+4. attention over 2*heads heads of [q|k|v]; outputs land at channel head*d (concat)
  const HeadView in{ms_sb, 3LL * N * d, d};
  // Attention output: one [N][2d] plane per pair of heads when the tcgen05 output projection can
  // take it (dense 128-byte rows for the apply kernel's stores and the GEMM's tile loads),
  // otherwise token-major [N][2C'].
  const bool f16 = desc->dtype == MSLA_F16;
  const bool att_planar = desc->dtype != MSLA_F32 && d == 32 && Ht % 2 == 0 && project_out_planar_bf16_supported(S * Cp, desc->C_out, N);
  const HeadView ov = att_planar ? HeadView{(long long)N * ld_att, (long long)N * 2 * d, 2 * d, 1}
                                 : HeadView{(long long)N * ld_att, d, ld_att, 0};
  // Steps 4 and 5 run as one kernel when it takes the shape: the head concat then stays in shared memory.
  const bool fused = desc->dtype != MSLA_F32 && fused_out_bf16_supported(Ht, d, desc->C_out, N);
  s = run_core(desc->dtype, ms, ms + (size_t)N * d * e, ms + (size_t)2 * N * d * e, att, in, ov, desc->B, Ht, N, d, desc->eps, p.core,
               ws + p.core_off, st, events ? (cudaEvent_t)events[3] : nullptr, fused ? CORE_STATE : CORE_ALL);
  if (s != MSLA_OK) return s;
  if ((s = record(events, 4, st)) != MSLA_OK) return s;
  // 5. output projection back to NCHW
  if (fused)
    s = run_fused_out_bf16(ms, ms_sb, 3LL * N * d, reinterpret_cast<const float*>(ws + p.core_off + p.core.partial_off), p.core.S, att, w->w_proj,
                           w->b_proj, residual, out_dev, desc->B, Ht, d, N, desc->C_out, desc->eps, st, f16);
  else
    s = att_planar ? run_project_out_planar_bf16(att, w->w_proj, w->b_proj, residual, out_dev, desc->B, S * Cp, desc->C_out, N, st, f16)
                   : run_project_out(desc->dtype, att, w->w_proj, w->b_proj, out_dev, desc->B, S * Cp, desc->C_out, N, st, residual);
  if (s != MSLA_OK) return s;
  if ((s = record(events, 5, st)) != MSLA_OK) return s;
  if (host_io) {
    const cudaError_t ce = cudaMemcpyAsync(out, out_dev, ob, cudaMemcpyDeviceToHost, st);
    if (ce != cudaSuccess) {
      cudaGetLastError();
      return fail(MSLA_ERR_CUDA, "device-to-host copy of out: %s", cudaGetErrorString(ce));
    }
  }
  return MSLA_OK;
}

// ------------------------------------------------------- token-sharded forward
// A band is a run of whole image rows; desc->H counts the band's rows plus halo_top rows above and halo_bottom rows
// below it.  Steps 1 and 2 run on the band with its halo as if it were an image of its own: the 5x5 window of a band
// row then sees true neighbours inside the image and zero padding only where the halo is absent, i.e. at the image
// border.  Steps 3 to 5 read the band's own tokens, which are a contiguous range of every [N][d] plane.
struct BandPlan {
  ForwardPlan f;
  CorePlan core;     // split of the band's tokens
  int Nb;            // tokens of the band
  long long tok_off; // first band token inside a plane
};

static msla_status_t validate_band(const msla_desc* desc, int halo_top, int halo_bottom, BandPlan* b) {
  msla_status_t s = validate_desc(desc, &b->f);
  if (s != MSLA_OK) return s;
  if (halo_top < 0 || halo_bottom < 0 || halo_top + halo_bottom >= desc->H)
    return fail(MSLA_ERR_INVALID_ARG, "halo rows (%d above, %d below) must be >= 0 and leave at least one of the %d rows", halo_top, halo_bottom, desc->H);
  b->Nb = (desc->H - halo_top - halo_bottom) * desc->W;
  b->tok_off = (long long)halo_top * desc->W;
  b->core = make_core_plan((long long)desc->B * b->f.S * desc->heads, b->Nb, desc->d);
  if (b->core.bytes > b->f.core.bytes) return fail(MSLA_ERR_WORKSPACE, "band plan exceeds the forward plan");
  if (!desc->workspace || desc->workspace_bytes < b->f.bytes)
    return fail(MSLA_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", b->f.bytes, desc->workspace ? desc->workspace_bytes : (size_t)0);
  if (!aligned16(desc->workspace)) return fail(MSLA_ERR_ALIGNMENT, "workspace must be 16-byte aligned");
  return MSLA_OK;
}

static msla_status_t band_states_impl(const msla_desc* desc, const void* x, const msla_weights* w, int halo_top,
                                      int halo_bottom, float* state_out, cudaStream_t st) {
  BandPlan b;
  msla_status_t s = validate_band(desc, halo_top, halo_bottom, &b);
  if (s != MSLA_OK) return s;
  if (!x || !w || !state_out) return fail(MSLA_ERR_INVALID_ARG, "null x, weights or state_out");
  if (!w->w_qkv || !w->w_dw || !w->w_pw) return fail(MSLA_ERR_INVALID_ARG, "null weight pointer");
  if (b.f.S == 3 && (!w->w_dw2 || !w->w_pw2)) return fail(MSLA_ERR_INVALID_ARG, "three branches need w_dw2 and w_pw2");
  const void* ptrs[] = {x, w->w_qkv, w->w_dw, w->w_pw, state_out, b.f.S == 3 ? w->w_dw2 : x, b.f.S == 3 ? w->w_pw2 : x};
  for (const void* ptr : ptrs)
    if (!aligned16(ptr)) return fail(MSLA_ERR_ALIGNMENT, "all device pointers must be 16-byte aligned");
  const ForwardPlan& p = b.f;
  const size_t e = elem_size(desc->dtype);
  const size_t xb = (size_t)desc->B * desc->C * p.N * e;
  const size_t sb = (size_t)desc->B * p.S * desc->heads * b.core.ne * sizeof(float);
  if (overlaps(x, xb, desc->workspace, p.bytes) || overlaps(state_out, sb, desc->workspace, p.bytes) || overlaps(state_out, sb, x, xb))
    return fail(MSLA_ERR_INVALID_ARG, "x, state_out and the workspace must not overlap");
  if ((s = check_arch()) != MSLA_OK) return s;
  char* ws = (char*)desc->workspace;
  const int Cp = p.Cp, N = p.N, d = desc->d;
  const long long ms_sb = 3LL * p.S * Cp * N;
  char* ms = ws + p.ms_off;
  s = run_project_in(desc->dtype, x, w->w_qkv, ms, desc->B, desc->C, 3 * Cp, N, d, ms_sb, st);
  if (s != MSLA_OK) return s;
  if ((s = run_branches(desc, w, p, ms, ms_sb, st)) != MSLA_OK) return s;
  const HeadView in{ms_sb, 3LL * N * d, d};
  const char* q = ms + (size_t)b.tok_off * d * e;
  s = run_core(desc->dtype, q, q + (size_t)N * d * e, q + (size_t)2 * N * d * e, nullptr, in, in, desc->B, p.S * desc->heads, b.Nb, d, desc->eps,
               b.core, ws + p.core_off, st, nullptr, CORE_STATE | CORE_COMBINE);
  if (s != MSLA_OK) return s;
  const cudaError_t ce = cudaMemcpyAsync(state_out, ws + p.core_off + b.core.state_off, sb, cudaMemcpyDeviceToDevice, st);
  if (ce != cudaSuccess) {
    cudaGetLastError();
    return fail(MSLA_ERR_CUDA, "copy of the band's state: %s", cudaGetErrorString(ce));
  }
  return MSLA_OK;
}

static msla_status_t band_output_impl(const msla_desc* desc, const msla_weights* w, int halo_top, int halo_bottom,
                                      const float* states, int R, void* out, cudaStream_t st) {
  BandPlan b;
  msla_status_t s = validate_band(desc, halo_top, halo_bottom, &b);
  if (s != MSLA_OK) return s;
  if (!w || !states || !out) return fail(MSLA_ERR_INVALID_ARG, "null weights, states or out");
  if (!w->w_proj) return fail(MSLA_ERR_INVALID_ARG, "null weight pointer");
  if (R < 1 || R > 4096) return fail(MSLA_ERR_INVALID_ARG, "R = %d bands; 1 .. 4096 are accepted", R);
  const void* ptrs[] = {w->w_proj, w->b_proj, states, out};
  for (const void* ptr : ptrs)
    if (ptr && !aligned16(ptr)) return fail(MSLA_ERR_ALIGNMENT, "all device pointers must be 16-byte aligned");
  const ForwardPlan& p = b.f;
  const size_t e = elem_size(desc->dtype);
  const int Cp = p.Cp, N = p.N, Nb = b.Nb, d = desc->d, heads = desc->heads;
  const int Ht = p.S * heads;
  const long long total = (long long)desc->B * Ht * b.core.ne;
  const size_t ob = (size_t)desc->B * desc->C_out * Nb * e, sb = (size_t)R * total * sizeof(float);
  if (overlaps(out, ob, desc->workspace, p.bytes) || overlaps(states, sb, desc->workspace, p.bytes) || overlaps(out, ob, states, sb))
    return fail(MSLA_ERR_INVALID_ARG, "out, states and the workspace must not overlap");
  if ((s = check_arch()) != MSLA_OK) return s;
  char* ws = (char*)desc->workspace;
  const long long ms_sb = 3LL * p.S * Cp * N, ld_att = (long long)p.S * Cp;
  char* ms = ws + p.ms_off;
  char* att = ws + p.att_off;
  float* state = reinterpret_cast<float*>(ws + p.core_off + b.core.state_off);
  generic::band_state_sum_kernel<<<(unsigned)ceil_div_ll(total, 256), 256, 0, st>>>(states, state, R, total);
  count_launches(1);
  if ((s = check_launch("sum of the bands' states")) != MSLA_OK) return s;
  const char* q = ms + (size_t)b.tok_off * d * e;
  if (desc->dtype != MSLA_F32 && fused_out_bf16_supported(Ht, d, desc->C_out, Nb))
    return run_fused_out_bf16(q, ms_sb, 3LL * N * d, state, 1, att, w->w_proj, w->b_proj, nullptr, out, desc->B, Ht, d, Nb, desc->C_out, desc->eps, st,
                              desc->dtype == MSLA_F16);
  const HeadView in{ms_sb, 3LL * N * d, d};
  const bool att_planar = desc->dtype != MSLA_F32 && d == 32 && Ht % 2 == 0 && project_out_planar_bf16_supported(p.S * Cp, desc->C_out, Nb);
  const HeadView ov = att_planar ? HeadView{(long long)Nb * ld_att, (long long)Nb * 2 * d, 2 * d, 1}
                                 : HeadView{(long long)Nb * ld_att, d, ld_att, 0};
  s = run_core(desc->dtype, q, q + (size_t)N * d * e, q + (size_t)2 * N * d * e, att, in, ov, desc->B, Ht, Nb, d, desc->eps, b.core,
               ws + p.core_off, st, nullptr, CORE_APPLY);
  if (s != MSLA_OK) return s;
  return att_planar ? run_project_out_planar_bf16(att, w->w_proj, w->b_proj, nullptr, out, desc->B, p.S * Cp, desc->C_out, Nb, st, desc->dtype == MSLA_F16)
                    : run_project_out(desc->dtype, att, w->w_proj, w->b_proj, out, desc->B, p.S * Cp, desc->C_out, Nb, st);
}

// ---------------------------------------------------------- FFN with a depthwise convolution
struct FfnPlan {
  size_t h_off, g_off, bytes;
  int N;
  bool tuned;  // bf16 / fp16 tensor-core path with the hidden tensor as planes of 64 channels
};

static msla_status_t validate_ffn(const msla_ffn_desc* d, FfnPlan* plan) {
  if (!d) return fail(MSLA_ERR_INVALID_ARG, "null descriptor");
  if (d->struct_size != sizeof(msla_ffn_desc)) return fail(MSLA_ERR_INVALID_ARG, "desc.struct_size = %u, expected %zu", d->struct_size, sizeof(msla_ffn_desc));
  if (!known_dtype(d->dtype)) return fail(MSLA_ERR_INVALID_ARG, "unknown dtype %d", (int)d->dtype);
  if (d->B < 1 || d->C < 1 || d->H < 1 || d->W < 1 || d->C_hidden < 1 || d->C_out < 1)
    return fail(MSLA_ERR_INVALID_ARG, "B, C, H, W, C_hidden, C_out must be positive");
  if (d->act != MSLA_ACT_IDENTITY && d->act != MSLA_ACT_RELU && d->act != MSLA_ACT_HARDSWISH)
    return fail(MSLA_ERR_INVALID_ARG, "unknown activation %d", (int)d->act);
  if (d->dw_kernel != 3) return fail(MSLA_ERR_UNSUPPORTED, "dw_kernel = %d; only the 3x3 depthwise convolution is supported", d->dw_kernel);
  if (d->residual && d->C_out != d->C) return fail(MSLA_ERR_INVALID_ARG, "the residual connection needs C_out == C (%d, %d)", d->C_out, d->C);
  if ((long long)d->H * d->W > 0x7fffffffLL) return fail(MSLA_ERR_UNSUPPORTED, "H*W exceeds 2^31-1");
  if (d->C % 8 != 0 || d->C_hidden % 8 != 0 || d->C_out % 8 != 0) return fail(MSLA_ERR_UNSUPPORTED, "C, C_hidden and C_out must be multiples of 8");
  if (d->B > 65535) return fail(MSLA_ERR_UNSUPPORTED, "B exceeds 65535");
  plan->N = d->H * d->W;
  plan->tuned = d->dtype != MSLA_F32 && ffn_bf16_supported(d->C, d->C_hidden, d->C_out, plan->N) &&
                (long long)d->B * (d->C_hidden / 64) <= 65535;
  const size_t hid = align_up((size_t)d->B * d->C_hidden * plan->N * elem_size(d->dtype), 256);
  plan->h_off = 0;
  plan->g_off = hid;
  plan->bytes = 2 * hid;
  return MSLA_OK;
}

static msla_status_t ffn_impl(const msla_ffn_desc* desc, const void* x, const msla_ffn_weights* w, void* out, bool residual,
                              cudaStream_t st) {
  FfnPlan p;
  msla_status_t s = validate_ffn(desc, &p);
  if (s != MSLA_OK) return s;
  if (!x || !out || !w) return fail(MSLA_ERR_INVALID_ARG, "null x, out or weights");
  if (!w->w1 || !w->w_dw || !w->w2) return fail(MSLA_ERR_INVALID_ARG, "null weight pointer");
  const void* ptrs[] = {x, out, w->w1, w->b1, w->w_dw, w->b_dw, w->w2, w->b2, desc->workspace};
  for (const void* ptr : ptrs)
    if (ptr && !aligned16(ptr)) return fail(MSLA_ERR_ALIGNMENT, "all device pointers must be 16-byte aligned");
  if (!desc->workspace || desc->workspace_bytes < p.bytes)
    return fail(MSLA_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", p.bytes, desc->workspace ? desc->workspace_bytes : (size_t)0);
  const size_t e = elem_size(desc->dtype);
  const int N = p.N, B = desc->B, C = desc->C, Ch = desc->C_hidden, Co = desc->C_out, act = (int)desc->act;
  const size_t xb = (size_t)B * C * N * e, ob = (size_t)B * Co * N * e;
  if (overlaps(out, ob, x, xb) || overlaps(out, ob, desc->workspace, p.bytes) || overlaps(x, xb, desc->workspace, p.bytes))
    return fail(MSLA_ERR_INVALID_ARG, "x, out and the workspace must not overlap");
  if ((s = check_arch()) != MSLA_OK) return s;
  char* ws = (char*)desc->workspace;
  void* h = ws + p.h_off;
  void* g = ws + p.g_off;
  const void* res = residual ? x : nullptr;
  if (p.tuned) {
    const bool f16 = desc->dtype == MSLA_F16;
    if ((s = run_ffn_expand_bf16(x, w->w1, w->b1, h, B, C, Ch, N, act, st, f16)) != MSLA_OK) return s;
    if ((s = run_ffn_dw3x3_bf16(h, w->w_dw, w->b_dw, g, B, Ch, desc->H, desc->W, act, st, f16)) != MSLA_OK) return s;
    return run_ffn_project_bf16(g, w->w2, w->b2, res, out, B, Ch, Co, N, st, f16);
  }
  // plain kernels, hidden tensor NCHW
  generic::GemmArgs g1{(long long)C * N, 1, N, (long long)Ch * N, 1, N, 0, N, Ch, C, Ch, act, nullptr};
  generic::GemmArgs g2{(long long)Ch * N, 1, N, (long long)Co * N, 1, N, 0, N, Co, Ch, Co, 0, res};
  const long long total = (long long)B * Ch * N;
  auto plain = [&](auto* tag) {
    using T = std::remove_pointer_t<decltype(tag)>;
    launch_gemm<T>((const T*)x, (const T*)w->w1, (const T*)w->b1, (T*)h, g1, B, st);
    generic::ffn_dw3x3_nchw_kernel<T><<<(unsigned)ceil_div_ll(total, 256), 256, 0, st>>>((const T*)h, (const T*)w->w_dw, (const T*)w->b_dw, (T*)g, Ch,
                                                                                        desc->H, desc->W, act, total);
    launch_gemm<T>((const T*)g, (const T*)w->w2, (const T*)w->b2, (T*)out, g2, B, st);
  };
  if (desc->dtype == MSLA_F32) plain((float*)nullptr);
  else if (desc->dtype == MSLA_F16) plain((__half*)nullptr);
  else plain((__nv_bfloat16*)nullptr);
  count_launches(1);
  return check_launch("FFN with a depthwise convolution");
}

static msla_status_t block_impl(const msla_desc* attn, const msla_weights* aw, const msla_ffn_desc* ffn, const msla_ffn_weights* fw,
                                const void* x, void* y, void* out, cudaStream_t st) {
  ForwardPlan ap;
  FfnPlan fp;
  msla_status_t s = validate_desc(attn, &ap);
  if (s != MSLA_OK) return s;
  if ((s = validate_ffn(ffn, &fp)) != MSLA_OK) return s;
  if (attn->B != ffn->B || attn->H != ffn->H || attn->W != ffn->W || attn->dtype != ffn->dtype)
    return fail(MSLA_ERR_INVALID_ARG, "the two halves of the block describe different B, H, W or dtype");
  if (attn->C != attn->C_out || ffn->C != attn->C || ffn->C_out != attn->C)
    return fail(MSLA_ERR_INVALID_ARG, "the block's residual connections need one channel count throughout (%d, %d, %d, %d)", attn->C, attn->C_out, ffn->C, ffn->C_out);
  if (!x || !y || !out) return fail(MSLA_ERR_INVALID_ARG, "null x, y or out");
  if (!aligned16(y)) return fail(MSLA_ERR_ALIGNMENT, "all device pointers must be 16-byte aligned");
  const size_t bytes = (size_t)attn->B * attn->C * ap.N * elem_size(attn->dtype);
  if (overlaps(y, bytes, x, bytes) || overlaps(y, bytes, out, bytes) ||
      (attn->workspace && overlaps(y, bytes, attn->workspace, ap.bytes)) || (ffn->workspace && overlaps(y, bytes, ffn->workspace, fp.bytes)))
    return fail(MSLA_ERR_INVALID_ARG, "y overlaps x, out or a workspace");
  // y = MSLA(x) + x: the output projection's epilogue adds the residual
  if ((s = forward_impl(attn, x, aw, y, st, nullptr, false, x)) != MSLA_OK) return s;
  return ffn_impl(ffn, y, fw, out, true, st);
}

}  // namespace msla

using namespace msla;

extern "C" {

msla_status_t msla_linattn_relu(const void* q, const void* k, const void* v, void* out, int B,
                                int heads, int N, int d, float eps, void* stream) {
  return core_entry(MSLA_BF16, q, k, v, out, B, heads, N, d, eps, nullptr, 0, true, (cudaStream_t)stream);
}

msla_status_t msla_linattn_relu_f32(const float* q, const float* k, const float* v, float* out,
                                    int B, int heads, int N, int d, float eps, void* stream) {
  return core_entry(MSLA_F32, q, k, v, out, B, heads, N, d, eps, nullptr, 0, true, (cudaStream_t)stream);
}

size_t msla_linattn_relu_workspace_bytes(int B, int heads, int N, int d) {
  if (!core_shape_ok(B, heads, N, d)) return 0;
  return make_core_plan((long long)B * heads, N, d).bytes;
}

msla_status_t msla_linattn_relu_ws(msla_dtype_t dtype, const void* q, const void* k, const void* v,
                                   void* out, int B, int heads, int N, int d, float eps,
                                   void* workspace, size_t workspace_bytes, void* stream) {
  return core_entry(dtype, q, k, v, out, B, heads, N, d, eps, workspace, workspace_bytes, false, (cudaStream_t)stream);
}

msla_status_t msla_linattn_relu_noalloc(msla_dtype_t dtype, const void* q, const void* k, const void* v,
                                        void* out, int B, int heads, int N, int d, float eps, void* stream) {
  return core_entry_noalloc(dtype, q, k, v, out, B, heads, N, d, eps, (cudaStream_t)stream);
}

size_t msla_forward_workspace_bytes(const msla_desc* desc) {
  ForwardPlan p;
  if (validate_desc(desc, &p) != MSLA_OK) return 0;
  return p.bytes;
}

msla_status_t msla_forward(const msla_desc* desc, const void* x, const msla_weights* w, void* out, void* stream) {
  return forward_impl(desc, x, w, out, (cudaStream_t)stream, nullptr, false);
}

msla_status_t msla_forward_profiled(const msla_desc* desc, const void* x, const msla_weights* w, void* out,
                                    void* stream, void* const* events, int n_events) {
  if (!events || n_events != 6) return fail(MSLA_ERR_INVALID_ARG, "events must hold exactly 6 cudaEvent_t handles");
  for (int i = 0; i < 6; ++i)
    if (!events[i]) return fail(MSLA_ERR_INVALID_ARG, "events[%d] is null", i);
  return forward_impl(desc, x, w, out, (cudaStream_t)stream, events, false);
}

size_t msla_forward_host_workspace_bytes(const msla_desc* desc) {
  ForwardPlan p;
  if (validate_desc(desc, &p) != MSLA_OK) return 0;
  const size_t e = elem_size(desc->dtype);
  return p.bytes + align_up((size_t)desc->B * desc->C * p.N * e, 256) + align_up((size_t)desc->B * desc->C_out * p.N * e, 256);
}

msla_status_t msla_forward_host(const msla_desc* desc, const void* x_host, const msla_weights* w, void* out_host, void* stream) {
  return forward_impl(desc, x_host, w, out_host, (cudaStream_t)stream, nullptr, true);
}

msla_status_t msla_band_states(const msla_desc* desc, const void* x_band, const msla_weights* w, int halo_top, int halo_bottom,
                               float* state_out, void* stream) {
  return band_states_impl(desc, x_band, w, halo_top, halo_bottom, state_out, (cudaStream_t)stream);
}

msla_status_t msla_band_output(const msla_desc* desc, const msla_weights* w, int halo_top, int halo_bottom, const float* states,
                               int n_bands, void* out_band, void* stream) {
  return band_output_impl(desc, w, halo_top, halo_bottom, states, n_bands, out_band, (cudaStream_t)stream);
}

size_t msla_ffn_workspace_bytes(const msla_ffn_desc* desc) {
  FfnPlan p;
  if (validate_ffn(desc, &p) != MSLA_OK) return 0;
  return p.bytes;
}

msla_status_t msla_ffn_dwconv(const msla_ffn_desc* desc, const void* x, const msla_ffn_weights* w, void* out, void* stream) {
  return ffn_impl(desc, x, w, out, desc && desc->residual, (cudaStream_t)stream);
}

msla_status_t msla_evit_block(const msla_desc* attn, const msla_weights* aw, const msla_ffn_desc* ffn, const msla_ffn_weights* fw,
                              const void* x, void* y, void* out, void* stream) {
  return block_impl(attn, aw, ffn, fw, x, y, out, (cudaStream_t)stream);
}

int msla_forward_fuses_apply(const msla_desc* desc) {
  ForwardPlan p;
  if (validate_desc(desc, &p) != MSLA_OK) return -1;
  return desc->dtype == MSLA_BF16 && fused_out_bf16_supported(p.S * desc->heads, desc->d, desc->C_out, p.N) ? 1 : 0;
}

unsigned long long msla_kernel_launches(void) { return g_launches; }

int msla_debug_wait_timeouts(void) {
  const int a = gemm_timeout_flag(), b = agg_timeout_flag(), c = fused_timeout_flag(), e = dw_timeout_flag();
  return (a < 0 || b < 0 || c < 0 || e < 0) ? -1 : (a | b | c | e);
}

int msla_debug_wait_selftest(long long limit_cycles, void* scratch, void* stream) {
  if (limit_cycles < 1 || limit_cycles > 2000000000LL || !scratch) return -1;  // at most about a second
  if (check_arch() != MSLA_OK) return -1;
  return run_wait_selftest(limit_cycles, (int*)scratch, (cudaStream_t)stream);
}

msla_status_t msla_project_in(msla_dtype_t dtype, const void* x, const void* w, void* y, int B, int C, int Cout, int N, int d, void* stream) {
  if (!known_dtype(dtype)) return fail(MSLA_ERR_INVALID_ARG, "unknown dtype");
  if (!x || !w || !y) return fail(MSLA_ERR_INVALID_ARG, "null pointer");
  if (B < 1 || C < 1 || Cout < 1 || N < 1 || B > 65535) return fail(MSLA_ERR_INVALID_ARG, "sizes must be positive (B <= 65535)");
  if (C % 8 || Cout % 8) return fail(MSLA_ERR_UNSUPPORTED, "C and Cout must be multiples of 8");
  if (d != 16 && d != 32) return fail(MSLA_ERR_UNSUPPORTED, "d = %d; only 16 and 32 are supported", d);
  if (Cout % d) return fail(MSLA_ERR_INVALID_ARG, "Cout must be a multiple of d");
  if (!aligned16(x) || !aligned16(w) || !aligned16(y)) return fail(MSLA_ERR_ALIGNMENT, "pointers must be 16-byte aligned");
  msla_status_t s = check_arch();
  if (s != MSLA_OK) return s;
  return run_project_in(dtype, x, w, y, B, C, Cout, N, d, (long long)Cout * N, (cudaStream_t)stream);
}

msla_status_t msla_aggregate(msla_dtype_t dtype, const void* t, const void* w_dw, const void* w_pw, void* y, int B, int H, int W, int Ch, int d, void* stream) {
  if (!known_dtype(dtype)) return fail(MSLA_ERR_INVALID_ARG, "unknown dtype");
  if (!t || !w_dw || !w_pw || !y) return fail(MSLA_ERR_INVALID_ARG, "null pointer");
  if (B < 1 || H < 1 || W < 1 || Ch < 1 || d < 1 || B > 65535) return fail(MSLA_ERR_INVALID_ARG, "sizes must be positive (B <= 65535)");
  if ((long long)H * W > 0x7fffffffLL) return fail(MSLA_ERR_UNSUPPORTED, "H*W exceeds 2^31-1");
  if (d != 16 && d != 32) return fail(MSLA_ERR_UNSUPPORTED, "d = %d; only 16 and 32 are supported", d);
  if (Ch % d) return fail(MSLA_ERR_INVALID_ARG, "Ch must be a multiple of d");
  if (Ch / d > 65535) return fail(MSLA_ERR_UNSUPPORTED, "more than 65535 groups");
  if (!aligned16(t) || !aligned16(w_dw) || !aligned16(w_pw) || !aligned16(y)) return fail(MSLA_ERR_ALIGNMENT, "pointers must be 16-byte aligned");
  const size_t bytes = (size_t)B * H * W * Ch * elem_size(dtype);
  if (overlaps(t, bytes, y, bytes)) return fail(MSLA_ERR_INVALID_ARG, "y overlaps t");
  msla_status_t s = check_arch();
  if (s != MSLA_OK) return s;
  return run_aggregate(dtype, t, w_dw, w_pw, y, B, H, W, Ch, d, (long long)Ch * H * W, (long long)Ch * H * W, (cudaStream_t)stream);
}

msla_status_t msla_project_out(msla_dtype_t dtype, const void* a, const void* w, const void* bias, void* y, int B, int Cin, int Cout, int N, void* stream) {
  if (!known_dtype(dtype)) return fail(MSLA_ERR_INVALID_ARG, "unknown dtype");
  if (!a || !w || !y) return fail(MSLA_ERR_INVALID_ARG, "null pointer");
  if (B < 1 || Cin < 1 || Cout < 1 || N < 1 || B > 65535) return fail(MSLA_ERR_INVALID_ARG, "sizes must be positive (B <= 65535)");
  if (Cin % 8 || Cout % 8) return fail(MSLA_ERR_UNSUPPORTED, "Cin and Cout must be multiples of 8");
  if (!aligned16(a) || !aligned16(w) || !aligned16(y) || (bias && !aligned16(bias))) return fail(MSLA_ERR_ALIGNMENT, "pointers must be 16-byte aligned");
  msla_status_t s = check_arch();
  if (s != MSLA_OK) return s;
  return run_project_out(dtype, a, w, bias, y, B, Cin, Cout, N, (cudaStream_t)stream);
}

const char* msla_status_string(msla_status_t s) {
  switch (s) {
    case MSLA_OK: return "ok";
    case MSLA_ERR_INVALID_ARG: return "invalid argument";
    case MSLA_ERR_UNSUPPORTED: return "unsupported shape or option";
    case MSLA_ERR_ALIGNMENT: return "misaligned pointer";
    case MSLA_ERR_WORKSPACE: return "workspace missing or too small";
    case MSLA_ERR_ARCH: return "device is not sm_100";
    case MSLA_ERR_CUDA: return "CUDA error";
  }
  return "unknown status";
}

const char* msla_last_error(void) { return g_last_error; }

int msla_version(void) { return 100; }

}  // extern "C"
