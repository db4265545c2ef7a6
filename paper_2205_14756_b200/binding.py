"""ctypes binding of libmsla: argument marshalling only.

Every function has the name and argument order of its C entry point in
``include/msla.h``; tensors are torch CUDA tensors whose ``data_ptr()`` is
passed through.  PyTorch supplies device memory and streams, nothing else.
There is no fallback: if ``libmsla.so`` is missing the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("MSLA_LIBRARY_PATH") or os.path.join(_PKG, "libmsla.so")

MSLA_F32, MSLA_BF16, MSLA_F16 = 0, 1, 2
_DTYPES = {torch.float32: MSLA_F32, torch.bfloat16: MSLA_BF16, torch.float16: MSLA_F16}

c_int, c_float, c_size_t, c_void_p = ctypes.c_int, ctypes.c_float, ctypes.c_size_t, ctypes.c_void_p


class MslaError(RuntimeError):
    def __init__(self, status: int, name: str, detail: str):
        super().__init__(f"libmsla status {status} ({name}): {detail}")
        self.status = status


class msla_desc(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("B", c_int), ("C", c_int), ("H", c_int), ("W", c_int),
                ("heads", c_int), ("d", c_int), ("n_scales", c_int), ("agg_kernel", c_int),
                ("C_out", c_int), ("dtype", c_int), ("eps", c_float), ("workspace", c_void_p),
                ("workspace_bytes", c_size_t), ("agg_kernel2", c_int)]


class msla_weights(ctypes.Structure):
    _fields_ = [("w_qkv", c_void_p), ("w_dw", c_void_p), ("w_pw", c_void_p), ("w_proj", c_void_p),
                ("b_proj", c_void_p), ("w_dw2", c_void_p), ("w_pw2", c_void_p)]


MSLA_ACT_IDENTITY, MSLA_ACT_RELU, MSLA_ACT_HARDSWISH = 0, 1, 2


class msla_ffn_desc(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("B", c_int), ("C", c_int), ("H", c_int), ("W", c_int),
                ("C_hidden", c_int), ("C_out", c_int), ("dw_kernel", c_int), ("act", c_int), ("residual", c_int),
                ("dtype", c_int), ("workspace", c_void_p), ("workspace_bytes", c_size_t)]


class msla_ffn_weights(ctypes.Structure):
    _fields_ = [("w1", c_void_p), ("b1", c_void_p), ("w_dw", c_void_p), ("b_dw", c_void_p), ("w2", c_void_p),
                ("b2", c_void_p)]


EXPORTS = {
    "msla_linattn_relu": (c_int, [c_void_p] * 4 + [c_int] * 4 + [c_float, c_void_p]),
    "msla_linattn_relu_f32": (c_int, [c_void_p] * 4 + [c_int] * 4 + [c_float, c_void_p]),
    "msla_linattn_relu_workspace_bytes": (c_size_t, [c_int] * 4),
    "msla_linattn_relu_ws": (c_int, [c_int] + [c_void_p] * 4 + [c_int] * 4 + [c_float, c_void_p, c_size_t, c_void_p]),
    "msla_linattn_relu_noalloc": (c_int, [c_int] + [c_void_p] * 4 + [c_int] * 4 + [c_float, c_void_p]),
    "msla_forward_workspace_bytes": (c_size_t, [ctypes.POINTER(msla_desc)]),
    "msla_forward": (c_int, [ctypes.POINTER(msla_desc), c_void_p, ctypes.POINTER(msla_weights), c_void_p, c_void_p]),
    "msla_forward_profiled": (c_int, [ctypes.POINTER(msla_desc), c_void_p, ctypes.POINTER(msla_weights), c_void_p, c_void_p,
                                      ctypes.POINTER(c_void_p), c_int]),
    "msla_forward_host_workspace_bytes": (c_size_t, [ctypes.POINTER(msla_desc)]),
    "msla_forward_host": (c_int, [ctypes.POINTER(msla_desc), c_void_p, ctypes.POINTER(msla_weights), c_void_p, c_void_p]),
    "msla_band_states": (c_int, [ctypes.POINTER(msla_desc), c_void_p, ctypes.POINTER(msla_weights), c_int, c_int, c_void_p, c_void_p]),
    "msla_band_output": (c_int, [ctypes.POINTER(msla_desc), ctypes.POINTER(msla_weights), c_int, c_int, c_void_p, c_int, c_void_p,
                                 c_void_p]),
    "msla_ffn_workspace_bytes": (c_size_t, [ctypes.POINTER(msla_ffn_desc)]),
    "msla_ffn_dwconv": (c_int, [ctypes.POINTER(msla_ffn_desc), c_void_p, ctypes.POINTER(msla_ffn_weights), c_void_p, c_void_p]),
    "msla_evit_block": (c_int, [ctypes.POINTER(msla_desc), ctypes.POINTER(msla_weights), ctypes.POINTER(msla_ffn_desc),
                                ctypes.POINTER(msla_ffn_weights), c_void_p, c_void_p, c_void_p, c_void_p]),
    "msla_forward_fuses_apply": (c_int, [ctypes.POINTER(msla_desc)]),
    "msla_kernel_launches": (ctypes.c_ulonglong, []),
    "msla_debug_wait_timeouts": (c_int, []),
    "msla_debug_wait_selftest": (c_int, [ctypes.c_longlong, c_void_p, c_void_p]),
    "msla_project_in": (c_int, [c_int] + [c_void_p] * 3 + [c_int] * 5 + [c_void_p]),
    "msla_aggregate": (c_int, [c_int] + [c_void_p] * 4 + [c_int] * 5 + [c_void_p]),
    "msla_project_out": (c_int, [c_int] + [c_void_p] * 4 + [c_int] * 4 + [c_void_p]),
    "msla_status_string": (ctypes.c_char_p, [c_int]),
    "msla_last_error": (ctypes.c_char_p, []),
    "msla_version": (c_int, []),
}

_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    """The loaded library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} not found: build it with `python -m paper_2205_14756_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def _check(status: int) -> None:
    if status != 0:
        handle = lib()
        raise MslaError(status, handle.msla_status_string(status).decode(), handle.msla_last_error().decode())


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("libmsla takes contiguous CUDA tensors")
    return t.data_ptr()


def msla_version() -> int:
    return lib().msla_version()


def msla_linattn_relu_workspace_bytes(B: int, heads: int, N: int, d: int) -> int:
    return lib().msla_linattn_relu_workspace_bytes(B, heads, N, d)


def msla_linattn_relu(q, k, v, out, B, heads, N, d, eps=1e-15, stream=None) -> None:
    """bf16 attention core on [B, heads, N, d] tensors (scratch from the stream's pool)."""
    _check(lib().msla_linattn_relu(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, heads, N, d, eps, _stream(stream)))


def msla_linattn_relu_f32(q, k, v, out, B, heads, N, d, eps=1e-15, stream=None) -> None:
    _check(lib().msla_linattn_relu_f32(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, heads, N, d, eps, _stream(stream)))


def msla_linattn_relu_ws(dtype, q, k, v, out, B, heads, N, d, eps, workspace, workspace_bytes, stream=None) -> None:
    _check(lib().msla_linattn_relu_ws(dtype, _ptr(q), _ptr(k), _ptr(v), _ptr(out), B, heads, N, d, eps,
                                      _ptr(workspace), workspace_bytes, _stream(stream)))


MSLA_NOALLOC_SCRATCH_BYTES = 4 << 20


def msla_linattn_relu_noalloc(dtype, q, k, v, out, B, heads, N, d, eps=1e-15, stream=None) -> None:
    """Attention core that takes its scratch from the library's built-in device
    array instead of allocating: for callers that may not allocate (deadline
    loops that forbid allocation after start-up, runtimes that own all memory).
    Shapes needing more than MSLA_NOALLOC_SCRATCH_BYTES raise MslaError(4).
    Calls on one device share the array: keep them ordered on the GPU."""
    _check(lib().msla_linattn_relu_noalloc(dtype, _ptr(q), _ptr(k), _ptr(v), _ptr(out), B, heads, N, d, eps,
                                           _stream(stream)))


def make_desc(B, C, H, W, heads, d, C_out, dtype, eps=1e-15, n_scales=2, agg_kernel=5,
              workspace: Optional[torch.Tensor] = None, agg_kernel2=3) -> msla_desc:
    desc = msla_desc()
    desc.struct_size = ctypes.sizeof(msla_desc)
    desc.B, desc.C, desc.H, desc.W = B, C, H, W
    desc.heads, desc.d, desc.n_scales, desc.agg_kernel, desc.C_out = heads, d, n_scales, agg_kernel, C_out
    desc.dtype = dtype
    desc.eps = eps
    desc.agg_kernel2 = agg_kernel2
    desc.workspace = _ptr(workspace) if workspace is not None else None
    desc.workspace_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    return desc


def msla_forward_workspace_bytes(desc: msla_desc) -> int:
    return lib().msla_forward_workspace_bytes(ctypes.byref(desc))


def msla_forward(desc: msla_desc, x, weights: msla_weights, out, stream=None) -> None:
    _check(lib().msla_forward(ctypes.byref(desc), _ptr(x), ctypes.byref(weights), _ptr(out), _stream(stream)))


def msla_forward_profiled(desc: msla_desc, x, weights: msla_weights, out, stream, events) -> None:
    """`events`: six torch.cuda.Event(enable_timing=True) objects (created, i.e. recorded once)."""
    handles = (c_void_p * 6)(*[e.cuda_event for e in events])
    _check(lib().msla_forward_profiled(ctypes.byref(desc), _ptr(x), ctypes.byref(weights), _ptr(out), _stream(stream),
                                       handles, 6))


def msla_forward_host_workspace_bytes(desc: msla_desc) -> int:
    return lib().msla_forward_host_workspace_bytes(ctypes.byref(desc))


def msla_forward_host(desc: msla_desc, x_host, weights: msla_weights, out_host, stream=None) -> None:
    """x_host / out_host: contiguous CPU tensors (pinned for asynchronous copies)."""
    for t in (x_host, out_host):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("msla_forward_host takes contiguous host tensors")
    _check(lib().msla_forward_host(ctypes.byref(desc), x_host.data_ptr(), ctypes.byref(weights), out_host.data_ptr(),
                                   _stream(stream)))


def msla_band_states(desc: msla_desc, x_band, weights: msla_weights, halo_top: int, halo_bottom: int, state_out,
                     stream=None) -> None:
    """Steps 1-3 on a band of image rows (desc.H = band rows + halos); state_out: fp32 [B, 2*heads, d, d+1]."""
    _check(lib().msla_band_states(ctypes.byref(desc), _ptr(x_band), ctypes.byref(weights), halo_top, halo_bottom,
                                  _ptr(state_out), _stream(stream)))


def msla_band_output(desc: msla_desc, weights: msla_weights, halo_top: int, halo_bottom: int, states, n_bands: int,
                     out_band, stream=None) -> None:
    """Steps 4-5 on the band's own tokens from the gathered states [n_bands, B, 2*heads, d, d+1]."""
    _check(lib().msla_band_output(ctypes.byref(desc), ctypes.byref(weights), halo_top, halo_bottom, _ptr(states), n_bands,
                                  _ptr(out_band), _stream(stream)))


def make_ffn_desc(B, C, H, W, C_hidden, C_out, dtype, act=MSLA_ACT_HARDSWISH, residual=False, dw_kernel=3,
                  workspace: Optional[torch.Tensor] = None) -> msla_ffn_desc:
    desc = msla_ffn_desc()
    desc.struct_size = ctypes.sizeof(msla_ffn_desc)
    desc.B, desc.C, desc.H, desc.W, desc.C_hidden, desc.C_out = B, C, H, W, C_hidden, C_out
    desc.dw_kernel, desc.act, desc.residual, desc.dtype = dw_kernel, act, int(residual), dtype
    desc.workspace = _ptr(workspace) if workspace is not None else None
    desc.workspace_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    return desc


def make_ffn_weights(w1, w_dw, w2, b1=None, b_dw=None, b2=None) -> msla_ffn_weights:
    w = msla_ffn_weights()
    w.w1, w.b1, w.w_dw, w.b_dw, w.w2, w.b2 = _ptr(w1), _ptr(b1), _ptr(w_dw), _ptr(b_dw), _ptr(w2), _ptr(b2)
    return w


def msla_ffn_workspace_bytes(desc: msla_ffn_desc) -> int:
    return lib().msla_ffn_workspace_bytes(ctypes.byref(desc))


def msla_ffn_dwconv(desc: msla_ffn_desc, x, weights: msla_ffn_weights, out, stream=None) -> None:
    _check(lib().msla_ffn_dwconv(ctypes.byref(desc), _ptr(x), ctypes.byref(weights), _ptr(out), _stream(stream)))


def msla_evit_block(attn: msla_desc, attn_weights: msla_weights, ffn: msla_ffn_desc, ffn_weights: msla_ffn_weights, x, y, out,
                    stream=None) -> None:
    _check(lib().msla_evit_block(ctypes.byref(attn), ctypes.byref(attn_weights), ctypes.byref(ffn), ctypes.byref(ffn_weights),
                                 _ptr(x), _ptr(y), _ptr(out), _stream(stream)))


def msla_debug_wait_timeouts() -> int:
    return lib().msla_debug_wait_timeouts()


def msla_debug_wait_selftest(limit_cycles: int, scratch, stream=None) -> int:
    """Runs the library's bounded wait on a barrier nobody arrives at; 1 = it gave up at the limit."""
    return lib().msla_debug_wait_selftest(limit_cycles, _ptr(scratch), _stream(stream))


def msla_forward_fuses_apply(desc: msla_desc) -> int:
    return lib().msla_forward_fuses_apply(ctypes.byref(desc))


def msla_kernel_launches() -> int:
    return lib().msla_kernel_launches()


def make_weights(w_qkv, w_dw, w_pw, w_proj, b_proj=None, w_dw2=None, w_pw2=None) -> msla_weights:
    w = msla_weights()
    w.w_qkv, w.w_dw, w.w_pw, w.w_proj, w.b_proj = _ptr(w_qkv), _ptr(w_dw), _ptr(w_pw), _ptr(w_proj), _ptr(b_proj)
    w.w_dw2, w.w_pw2 = _ptr(w_dw2), _ptr(w_pw2)
    return w


def msla_project_in(dtype, x, w, y, B, C, Cout, N, d, stream=None) -> None:
    _check(lib().msla_project_in(dtype, _ptr(x), _ptr(w), _ptr(y), B, C, Cout, N, d, _stream(stream)))


def msla_aggregate(dtype, t, w_dw, w_pw, y, B, H, W, Ch, d, stream=None) -> None:
    _check(lib().msla_aggregate(dtype, _ptr(t), _ptr(w_dw), _ptr(w_pw), _ptr(y), B, H, W, Ch, d, _stream(stream)))


def msla_project_out(dtype, a, w, bias, y, B, Cin, Cout, N, stream=None) -> None:
    _check(lib().msla_project_out(dtype, _ptr(a), _ptr(w), _ptr(bias), _ptr(y), B, Cin, Cout, N, _stream(stream)))


def dtype_code(t: torch.dtype) -> int:
    return _DTYPES[t]
