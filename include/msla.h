/*
 * libmsla -- forward pass of the multi-scale ReLU linear attention module of
 * EfficientViT (arXiv 2205.14756, Section 3.1) for NVIDIA B200 (sm_100a).
 *
 * Conventions shared by every entry point
 *   - Plain C ABI.  Pointers named q, k, v, x, out, weights' members and
 *     workspaces are DEVICE pointers; desc / weights structs are HOST memory and
 *     are read only during the call.  `stream` is a cudaStream_t passed as
 *     void* (NULL = the legacy default stream).
 *   - Calls validate on the host, enqueue kernels on `stream` and return; they
 *     never synchronise, print, throw or abort.  A non-zero status means no
 *     kernel was launched by that call (except MSLA_ERR_CUDA raised by a launch
 *     in the middle of a multi-kernel call).  msla_last_error() gives a
 *     thread-local detail string for the most recent failure on this thread.
 *   - All buffers are caller-owned.  The library keeps no pointer past the
 *     completion of the work it enqueued.  Outputs must not overlap inputs or
 *     the workspace (overlap is reported as MSLA_ERR_INVALID_ARG).
 *   - Device pointers must be 16-byte aligned (MSLA_ERR_ALIGNMENT otherwise).
 *   - Accumulation is always fp32; bf16 conversions round to nearest even.
 *   - Results are bitwise reproducible for a given shape and dtype: no
 *     floating-point atomics, and the split of the token reduction depends on
 *     the shape only.
 *   - There is no CPU fallback: on a device that is not compute capability
 *     10.x every compute call returns MSLA_ERR_ARCH.
 */
#ifndef MSLA_H_
#define MSLA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MSLA_OK = 0,
  MSLA_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, inconsistent descriptor, overlap */
  MSLA_ERR_UNSUPPORTED = 2, /* a shape or option this build has no kernel for */
  MSLA_ERR_ALIGNMENT = 3,   /* a device pointer is not 16-byte aligned */
  MSLA_ERR_WORKSPACE = 4,   /* workspace missing or smaller than the *_workspace_bytes() answer */
  MSLA_ERR_ARCH = 5,        /* current device is not sm_100 */
  MSLA_ERR_CUDA = 6         /* a CUDA runtime call or launch failed; see msla_last_error() */
} msla_status_t;

/* Storage type of activations and weights.  Arithmetic and the attention state are fp32 for all three.  MSLA_F16
 * (the paper's deployment precision, Section 4.1): every tensor-core kernel of the bf16 path (projections, aggregation,
 * attention core, fused apply + output projection, FFN) is instantiated for it; what is stored in 16 bits of the state
 * is scaled by a power of two near 1 / N, which leaves Eq. 3's quotient unchanged.  MSLA_F16 is accepted wherever a dtype is taken (msla_linattn_relu_ws and _noalloc, msla_forward*, the band
 * pair, the stage entry points, msla_ffn_dwconv, msla_evit_block). */
typedef enum { MSLA_F32 = 0, MSLA_BF16 = 1, MSLA_F16 = 2 } msla_dtype_t;

/* ------------------------------------------------------------------------- *
 * Attention core: ReLU linear attention, Eq. 3 of the paper (the linear-time
 * re-association of Eq. 1 under the similarity of Eq. 2), per (batch, head):
 *
 *   KV[a,c] = sum_j relu(k[j,a]) * v[j,c]        ks[a] = sum_j relu(k[j,a])
 *   out[i,c] = sum_a relu(q[i,a]) * KV[a,c] / (sum_a relu(q[i,a]) * ks[a] + eps)
 *
 * q, k, v, out: device, dense [B, heads, N, d] with d innermost; bf16 for
 * msla_linattn_relu, fp32 for msla_linattn_relu_f32.  d must be 16 or 32
 * (MSLA_ERR_UNSUPPORTED otherwise); B, heads, N >= 1.  eps is added once to the
 * denominator, so a query row with no positive entry gives an all-zero output
 * row rather than 0/0.  There is no 1/sqrt(d) scaling (that belongs to the
 * softmax similarity only).
 *
 * The reduction over tokens is split into chunks whose fp32 partial states
 * live in scratch memory.  These two calls take that scratch from the stream's
 * memory pool (cudaMallocAsync / cudaFreeAsync on `stream`); use
 * msla_linattn_relu_ws to supply it yourself.
 * ------------------------------------------------------------------------- */
msla_status_t msla_linattn_relu(const void* q, const void* k, const void* v, void* out,
                                int B, int heads, int N, int d, float eps, void* stream);
msla_status_t msla_linattn_relu_f32(const float* q, const float* k, const float* v, float* out,
                                    int B, int heads, int N, int d, float eps, void* stream);

/* Scratch bytes the core needs for this shape (0 if the shape is invalid). */
size_t msla_linattn_relu_workspace_bytes(int B, int heads, int N, int d);

/* Same operation (Eq. 3) with caller-owned scratch: `workspace` is device
 * memory of at least msla_linattn_relu_workspace_bytes() bytes, 16-byte
 * aligned, contents irrelevant on entry and undefined on exit.  Two calls that
 * may run concurrently must not share a workspace. */
msla_status_t msla_linattn_relu_ws(msla_dtype_t dtype, const void* q, const void* k, const void* v,
                                   void* out, int B, int heads, int N, int d, float eps,
                                   void* workspace, size_t workspace_bytes, void* stream);

/* Attention core for callers that must not allocate.  (The paper has no
 * counterpart to this entry point; it exists for deployment reasons only.)
 *
 * Some hosts of this library cannot call cudaMalloc or its stream-ordered
 * relatives when they need the result: control loops with a hard deadline
 * that forbid allocation after start-up (an allocation may block, synchronise
 * the device or fail), and plug-ins living inside a runtime that owns every
 * byte of device memory and hands none out at call time.  For them the
 * scratch of the token reduction comes from a fixed array that is part of the
 * library image: MSLA_NOALLOC_SCRATCH_BYTES of device memory, reserved on
 * every GPU that loads the library for as long as the process lives.
 *
 * Same arguments and result as msla_linattn_relu_ws without the workspace.
 * Shapes whose scratch need (msla_linattn_relu_workspace_bytes) exceeds
 * MSLA_NOALLOC_SCRATCH_BYTES are refused with MSLA_ERR_WORKSPACE and nothing
 * is launched.  The call never allocates or frees memory, on host or device.
 *
 * The first call on each device looks up the array's device address (a
 * symbol query, not an allocation), and the first call for each (device,
 * dtype, d) loads and configures that variant's kernels, which the driver may
 * back with device memory of its own: make one warm-up call per (device,
 * dtype, d) at start-up, outside any stream capture; from then on a call does
 * no set-up and no allocation.  The looked-up address does not survive
 * cudaDeviceReset.  All calls on a device share the one array, and its contents
 * persist from call to call, so two calls whose kernels may overlap on the GPU
 * (different streams, no ordering between them) race; order them on one stream
 * or with events. */
#define MSLA_NOALLOC_SCRATCH_BYTES (4u << 20)
msla_status_t msla_linattn_relu_noalloc(msla_dtype_t dtype, const void* q, const void* k, const void* v,
                                        void* out, int B, int heads, int N, int d, float eps,
                                        void* stream);

/* ------------------------------------------------------------------------- *
 * Whole module (Section 3.1, Figure 2 right) on an NCHW feature map:
 *
 *   1. qkv = 1x1 conv (x, w_qkv)                    C  -> 3C'   (Q = xW_Q, K = xW_K, V = xW_V)
 *   2. agg = grouped 1x1 (depthwise kxk (qkv))      3C' -> 3C'  multi-scale token aggregation:
 *            one depthwise conv, stride 1, zero padding k/2, cross-correlation,
 *            then one 1x1 group convolution with 3*heads groups of d channels
 *   3. multi-scale tokens = {qkv, agg}: 2*heads heads; in each head the 3d
 *      channels are [q | k | v]; token n = row*W + col
 *   4. ReLU linear attention (Eq. 3) per (batch, head) over all N = H*W tokens
 *   5. head outputs concatenated along channels (all heads of the original
 *      scale first, then the aggregated scale), then
 *      out = 1x1 conv (att, w_proj) (+ b_proj)      2C' -> C_out
 *
 * with C' = heads*d.  Section 4.1 fixes two branches and 5x5 aggregation:
 * n_scales = 2, agg_kernel = 5.  Also accepted, in the sense of Section 3.1's
 * "small kernels" and multi-scale tokens: agg_kernel = 3, and n_scales = 3, a
 * second aggregated branch with its own filters (w_dw2, w_pw2, agg_kernel2);
 * the heads of branch 0 come first in the concat, then branch 1, then branch
 * 2, and w_proj is [C_out, n_scales*C'].  No bias, normalisation or
 * activation sits between the stages; the residual connection around the
 * module is the caller's.
 * ------------------------------------------------------------------------- */
typedef struct {
  uint32_t struct_size;   /* sizeof(msla_desc), for versioning */
  int B, C, H, W;         /* input x is [B, C, H, W] */
  int heads, d;           /* heads per scale and channels per head; d in {16, 32} */
  int n_scales;           /* 2 (Section 4.1), or 3: a second aggregated branch */
  int agg_kernel;         /* 5 (Section 4.1) or 3 */
  int C_out;              /* output channels */
  msla_dtype_t dtype;     /* type of x, out and all weights */
  float eps;              /* added to the attention denominator */
  void* workspace;        /* device scratch, >= msla_forward_workspace_bytes(desc) */
  size_t workspace_bytes;
  int agg_kernel2;        /* n_scales == 3: filter size of the second aggregated branch, 5 or 3; else ignored */
} msla_desc;

typedef struct {
  const void* w_qkv;  /* [3C', C]     row o = output channel (h*3 + t)*d + i, t: 0 q, 1 k, 2 v */
  const void* w_dw;   /* [3C', k, k]  taps [dy][dx]; tap reads pixel (row+dy-k/2, col+dx-k/2) */
  const void* w_pw;   /* [3C', d]     out channel o reads in channels (o/d)*d .. (o/d)*d + d-1 */
  const void* w_proj; /* [C_out, n_scales*C'] column j = att channel head*d + c */
  const void* b_proj; /* [C_out] or NULL */
  const void* w_dw2;  /* n_scales == 3: [3C', k2, k2] and [3C', d] of the second aggregated branch; else ignored */
  const void* w_pw2;
} msla_weights;

/* Scratch bytes msla_forward needs for this descriptor (workspace fields are
 * ignored); 0 if the descriptor is invalid or unsupported. */
size_t msla_forward_workspace_bytes(const msla_desc* desc);

/* x: device [B, C, H, W]; out: device [B, C_out, H, W]; both of desc->dtype.
 * C and C_out must be multiples of 8. */
msla_status_t msla_forward(const msla_desc* desc, const void* x, const msla_weights* weights,
                           void* out, void* stream);

/* msla_forward with CUDA events recorded between the module's five steps, so
 * that each step can be timed inside a real forward pass.  `events` is a host
 * array of n_events = 6 cudaEvent_t handles (as void*): events[0] is recorded
 * on `stream` before step 1 and events[i] after step i (1 projection, 2
 * aggregation, 3 KV-state reduction, 4 apply, 5 output projection; Section
 * 3.1).  When msla_forward_fuses_apply(desc) == 1 steps 4 and 5 are one
 * kernel: events[3] is then recorded after the first level of the state
 * reduction (the per-chunk partial states), events[4] directly after it, so
 * the interval of step 4 is empty and events[4]..events[5] covers the second
 * level of the state reduction (fixed-order sum of the partial states, folded
 * into the projection weights) together with apply + projection.  Everything
 * else is as for msla_forward. */
msla_status_t msla_forward_profiled(const msla_desc* desc, const void* x, const msla_weights* weights,
                                    void* out, void* stream, void* const* events, int n_events);

/* msla_forward for callers whose activations live in HOST memory (the paper's
 * latency protocol, Section 4.1, includes the data transfer).  x_host and
 * out_host are host pointers (pinned memory if the copies are to be
 * asynchronous); weights stay device pointers.  The call enqueues a
 * host-to-device copy of x, the five steps and a device-to-host copy of the
 * result on `stream`.  desc->workspace must hold
 * msla_forward_host_workspace_bytes(desc) bytes: the forward scratch plus
 * device staging for x and out. */
size_t msla_forward_host_workspace_bytes(const msla_desc* desc);
msla_status_t msla_forward_host(const msla_desc* desc, const void* x_host, const msla_weights* weights,
                                void* out_host, void* stream);

/* The module forward cut into bands of image rows, for one image spread over
 * several GPUs (the module is linear in the token count, Section 3.1, so
 * high-resolution inputs are where it is used; Eq. 3's two sums over tokens
 * are the only coupling between the bands besides the 5x5 window of step 2).
 * Rank r of R holds a run of whole rows of the image.  desc->H counts the rows
 * of x_band: the band's own rows plus halo_top rows above and halo_bottom rows
 * below, copies of the neighbouring bands' edge rows of x (2 each, the reach of
 * the 5x5 aggregation; 0 where the band touches the image border, which is
 * where step 2 pads with zeros).  desc->workspace, of
 * msla_forward_workspace_bytes(desc) bytes, carries the band's multi-scale
 * tokens from the first call to the second and must not be touched in between.
 *
 *   msla_band_states: steps 1 and 2 on x_band [B, C, H, W], step 3 on the
 *     band's own tokens.  state_out: device fp32 [B][2*heads][d][d+1], entry
 *     [a][c] = sum over the band's tokens of ReLU(k[a])*v[c], column d = sum of
 *     ReLU(k[a]) (the band's share of Eq. 3's two sums).
 *   -- the caller gathers the R states into states[R][B][2*heads][d][d+1],
 *      band 0 first (an all-gather; every rank must hold the same bytes) --
 *   msla_band_output: adds the R states in band order (a fixed order, so every
 *     rank forms the same sums bit for bit), then steps 4 and 5 on the band's
 *     own tokens.  out_band: device [B, C_out, H - halo_top - halo_bottom, W].
 *
 * Both calls enqueue on `stream` and return; pointers are device pointers,
 * 16-byte aligned, caller-owned, and must not overlap one another or the
 * workspace.  With R = 1 and no halo the pair computes what msla_forward does
 * (the state is then summed in a different, still fixed, order).  Errors as
 * for msla_forward; INVALID_ARG if the halos leave no row. */
msla_status_t msla_band_states(const msla_desc* desc, const void* x_band, const msla_weights* weights,
                               int halo_top, int halo_bottom, float* state_out, void* stream);
msla_status_t msla_band_output(const msla_desc* desc, const msla_weights* weights, int halo_top,
                               int halo_bottom, const float* states, int n_bands, void* out_band,
                               void* stream);

/* ---------------------------------------------------------------------------
 * The other half of the building block (Section 3.1, Fig. 2 left): an FFN with
 * a depthwise convolution inserted into it (FFN+DWConv), which supplies the
 * local information ReLU linear attention lacks, and the block itself.
 *
 *   h   = act(conv1x1(x, w1) + b1)                  C        -> C_hidden
 *   g   = act(dwconv3x3(h, w_dw) + b_dw)            depthwise, stride 1, zero padding 1, cross-correlation
 *   out = conv1x1(g, w2) + b2 (+ x if residual)     C_hidden -> C_out
 *
 * The paper fixes neither the expansion ratio, the activation nor the
 * normalisation: they are fields here (a normalisation folded for inference
 * is a bias).  dw_kernel must be 3.  residual != 0 needs C_out == C.
 * ------------------------------------------------------------------------- */
typedef enum {
  MSLA_ACT_IDENTITY = 0,
  MSLA_ACT_RELU = 1,      /* max(a, 0) */
  MSLA_ACT_HARDSWISH = 2  /* a * min(max(a + 3, 0), 6) / 6 */
} msla_act_t;

typedef struct {
  uint32_t struct_size;   /* sizeof(msla_ffn_desc) */
  int B, C, H, W;         /* input x is [B, C, H, W] */
  int C_hidden;           /* width between the two linear layers */
  int C_out;
  int dw_kernel;          /* 3 */
  msla_act_t act;         /* after the first linear layer and after the depthwise convolution */
  int residual;           /* != 0: out += x */
  msla_dtype_t dtype;     /* type of x, out, weights and biases */
  void* workspace;        /* device scratch, >= msla_ffn_workspace_bytes(desc) */
  size_t workspace_bytes;
} msla_ffn_desc;

typedef struct {
  const void* w1;    /* [C_hidden, C] */
  const void* b1;    /* [C_hidden] or NULL */
  const void* w_dw;  /* [C_hidden, 3, 3] taps [dy][dx]; tap reads pixel (row+dy-1, col+dx-1) */
  const void* b_dw;  /* [C_hidden] or NULL */
  const void* w2;    /* [C_out, C_hidden] */
  const void* b2;    /* [C_out] or NULL */
} msla_ffn_weights;

/* Scratch bytes msla_ffn_dwconv needs (workspace fields ignored); 0 if the
 * descriptor is invalid or unsupported. */
size_t msla_ffn_workspace_bytes(const msla_ffn_desc* desc);

/* x: device [B, C, H, W]; out: device [B, C_out, H, W]; out must not overlap x
 * or the workspace.  C, C_hidden and C_out must be multiples of 8.  Enqueues
 * on `stream` and returns.  Errors as for msla_forward. */
msla_status_t msla_ffn_dwconv(const msla_ffn_desc* desc, const void* x, const msla_ffn_weights* weights,
                              void* out, void* stream);

/* The building block of Fig. 2 left with its two residual connections:
 *   y = x + MSLA(x)  (msla_forward),   out = y + FFN+DWConv(y)  (msla_ffn_dwconv with residual).
 * attn and ffn describe the same B, H, W and dtype with attn->C == attn->C_out
 * == ffn->C == ffn->C_out; each carries its own workspace; `y`, device
 * [B, C, H, W], receives the intermediate (caller-owned, no overlap with x,
 * out or the workspaces).  ffn->residual is taken as 1. */
msla_status_t msla_evit_block(const msla_desc* attn, const msla_weights* attn_weights, const msla_ffn_desc* ffn,
                              const msla_ffn_weights* ffn_weights, const void* x, void* y, void* out, void* stream);

/* 1 if msla_forward runs steps 4 and 5 of Section 3.1 (apply and output
 * projection) as one kernel for this descriptor, so that the head concat never
 * goes to device memory; 0 if they run as two kernels; -1 on an invalid
 * descriptor.  A pure function of the descriptor (workspace fields ignored);
 * host only, launches nothing.  Benchmarks use it to attribute time and bytes. */
int msla_forward_fuses_apply(const msla_desc* desc);

/* Number of kernels this library has launched from the calling thread since it
 * was loaded (a bookkeeping counter for benchmarks; no paper counterpart). */
unsigned long long msla_kernel_launches(void);

/* Diagnostic (no paper counterpart): every wait inside the library's kernels
 * is bounded; a kernel whose wait ran out raises a sticky device flag, releases
 * what it holds and returns, leaving its output undefined.  This call
 * SYNCHRONISES the device and returns 1 if that ever happened in this process,
 * 0 if not, -1 if the flag could not be read. */
int msla_debug_wait_timeouts(void);

/* Diagnostic (no paper counterpart): runs the bounded wait itself on a barrier
 * that nothing ever arrives at, with a limit of `limit_cycles` SM cycles
 * (1 .. 2e9, i.e. at most about a second), in a one-warp kernel of its own on
 * `stream`, and SYNCHRONISES the stream.  `scratch` is device memory for two
 * ints.  Returns 1 if the wait gave up at the limit and raised the kernel's
 * abort flag (what every kernel of the library relies on), 0 if not, -1 on a
 * bad argument or CUDA error.  The context stays usable either way. */
int msla_debug_wait_selftest(long long limit_cycles, void* scratch, void* stream);

/* Stage entry points (the module's steps 1, 2 and 5 of Section 3.1 on their
 * own), exposed so that each kernel can be checked and timed in isolation.
 * Between the steps the library keeps activations "planar": channels are cut
 * into groups of d (one group = the q, k or v of one head, which is also one
 * group of the aggregation's 1x1 group convolution), each group a dense
 * [N][d] matrix: act[b][group][n][i], channel = group*d + i.
 *   msla_project_in : x [B, C, N] (NCHW), w [Cout, C]              -> y [B, Cout/d, N, d]
 *   msla_aggregate  : t [B, Ch/d, H*W, d], w_dw [Ch,5,5], w_pw [Ch,d] -> y [B, Ch/d, H*W, d]
 *   msla_project_out: a [B, N, Cin] (token-major), w [Cout, Cin], bias [Cout]|NULL -> y [B, Cout, N] (NCHW)
 * d must be 16 or 32 and divide Cout / Ch.
 */
msla_status_t msla_project_in(msla_dtype_t dtype, const void* x, const void* w, void* y,
                              int B, int C, int Cout, int N, int d, void* stream);
msla_status_t msla_aggregate(msla_dtype_t dtype, const void* t, const void* w_dw, const void* w_pw,
                             void* y, int B, int H, int W, int Ch, int d, void* stream);
msla_status_t msla_project_out(msla_dtype_t dtype, const void* a, const void* w, const void* bias,
                               void* y, int B, int Cin, int Cout, int N, void* stream);

const char* msla_status_string(msla_status_t status);
const char* msla_last_error(void); /* thread-local; empty string if none */
int msla_version(void);            /* major*10000 + minor*100 + patch */

#ifdef __cplusplus
}
#endif
#endif /* MSLA_H_ */
