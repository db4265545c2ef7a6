"""fp64 CPU oracle for the multi-scale ReLU linear attention module.

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  The product (the CUDA library and its binding)
never imports this package, and this package never imports the product.

The arithmetic lives in ``msla_oracle.c`` (plain C loops, fp64); this file only
compiles it with gcc on first use and marshals numpy arrays through ctypes.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "msla_oracle.c")
_LIB = os.path.join(_HERE, "libmsla_oracle.so")
_lib: Optional[ctypes.CDLL] = None

_dp = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile the oracle into a shared object next to its source."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_set_num_threads.argtypes = [ctypes.c_int]
        lib.oracle_conv1x1.argtypes = [_dp, _dp, _dp, _dp, ctypes.c_int, ctypes.c_int,
                                       ctypes.c_int, ctypes.c_long]
        lib.oracle_conv1x1.restype = None
        lib.oracle_dwconv.argtypes = [_dp, _dp, _dp] + [ctypes.c_int] * 5
        lib.oracle_dwconv.restype = None
        lib.oracle_group1x1.argtypes = [_dp, _dp, _dp, ctypes.c_int, ctypes.c_int,
                                        ctypes.c_int, ctypes.c_long]
        lib.oracle_group1x1.restype = None
        lib.oracle_linattn_relu.argtypes = [_dp, _dp, _dp, _dp, ctypes.c_int, ctypes.c_int,
                                            ctypes.c_long, ctypes.c_int, ctypes.c_double]
        lib.oracle_linattn_relu.restype = None
        lib.oracle_msla_forward.argtypes = [_dp] * 7 + [ctypes.c_int] * 8 + [ctypes.c_double]
        lib.oracle_msla_forward.restype = ctypes.c_int
        lib.oracle_msla_forward3.argtypes = [_dp] * 9 + [ctypes.c_int] * 9 + [ctypes.c_double]
        lib.oracle_msla_forward3.restype = ctypes.c_int
        lib.oracle_bias_act.argtypes = [_dp, _dp, ctypes.c_int, ctypes.c_int, ctypes.c_long, ctypes.c_int]
        lib.oracle_bias_act.restype = None
        lib.oracle_ffn_dwconv.argtypes = [_dp] * 8 + [ctypes.c_int] * 9
        lib.oracle_ffn_dwconv.restype = ctypes.c_int
        _lib = lib
    return _lib


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(_dp)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(int(n))


def conv1x1(x, w, bias=None) -> np.ndarray:
    """x [B, Cin, ...spatial], w [Cout, Cin] -> [B, Cout, ...spatial]."""
    x, w = _f64(x), _f64(w)
    B, Cin = x.shape[:2]
    Cout = w.shape[0]
    assert w.shape == (Cout, Cin)
    N = int(np.prod(x.shape[2:]))
    b = None if bias is None else _f64(bias)
    y = np.empty((B, Cout) + x.shape[2:], dtype=np.float64)
    _load().oracle_conv1x1(_p(x), _p(w), _p(b), _p(y), B, Cin, Cout, N)
    return y


def dwconv(x, w) -> np.ndarray:
    """x [B, Ch, H, W], w [Ch, k, k] -> [B, Ch, H, W] (zero pad k//2)."""
    x, w = _f64(x), _f64(w)
    B, Ch, H, W = x.shape
    k = w.shape[-1]
    assert w.shape == (Ch, k, k) and k % 2 == 1
    y = np.empty_like(x)
    _load().oracle_dwconv(_p(x), _p(w), _p(y), B, Ch, H, W, k)
    return y


def group1x1(x, w) -> np.ndarray:
    """x [B, Ch, ...spatial], w [Ch, d] -> [B, Ch, ...spatial]; groups of d."""
    x, w = _f64(x), _f64(w)
    B, Ch = x.shape[:2]
    d = w.shape[1]
    assert w.shape == (Ch, d) and Ch % d == 0
    N = int(np.prod(x.shape[2:]))
    y = np.empty_like(x)
    _load().oracle_group1x1(_p(x), _p(w), _p(y), B, Ch, d, N)
    return y


def linattn_relu(q, k, v, eps: float = 1e-15) -> np.ndarray:
    """Eq. 3 on q, k, v [B, heads, N, d] -> [B, heads, N, d]."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    assert q.shape == k.shape == v.shape and q.ndim == 4
    B, heads, N, d = q.shape
    out = np.empty_like(q)
    _load().oracle_linattn_relu(_p(q), _p(k), _p(v), _p(out), B, heads, N, d, float(eps))
    return out


def msla_forward(x, w_qkv, w_dw, w_pw, w_proj, b_proj=None, *, heads: int, d: int,
                 eps: float = 1e-15) -> np.ndarray:
    """Whole module on NCHW x [B, C, H, W] -> [B, C_out, H, W]."""
    x, w_qkv, w_dw, w_pw, w_proj = map(_f64, (x, w_qkv, w_dw, w_pw, w_proj))
    B, C, H, W = x.shape
    Cp = heads * d
    k = w_dw.shape[-1]
    C_out = w_proj.shape[0]
    assert w_qkv.shape == (3 * Cp, C)
    assert w_dw.shape == (3 * Cp, k, k)
    assert w_pw.shape == (3 * Cp, d)
    assert w_proj.shape == (C_out, 2 * Cp)
    b = None if b_proj is None else _f64(b_proj)
    out = np.empty((B, C_out, H, W), dtype=np.float64)
    rc = _load().oracle_msla_forward(_p(x), _p(w_qkv), _p(w_dw), _p(w_pw), _p(w_proj), _p(b),
                                     _p(out), B, C, H, W, heads, d, k, C_out, float(eps))
    if rc != 0:
        raise MemoryError("oracle_msla_forward: scratch allocation failed")
    return out


def msla_forward3(x, w_qkv, w_dw, w_pw, w_dw2, w_pw2, w_proj, b_proj=None, *, heads: int, d: int, eps: float = 1e-15) -> np.ndarray:
    """The module with three branches (projected tokens and two aggregated copies) on NCHW x -> [B, C_out, H, W]."""
    x, w_qkv, w_dw, w_pw, w_dw2, w_pw2, w_proj = map(_f64, (x, w_qkv, w_dw, w_pw, w_dw2, w_pw2, w_proj))
    B, C, H, W = x.shape
    Cp, k1, k2, C_out = heads * d, w_dw.shape[-1], w_dw2.shape[-1], w_proj.shape[0]
    assert w_qkv.shape == (3 * Cp, C) and w_dw.shape == (3 * Cp, k1, k1) and w_dw2.shape == (3 * Cp, k2, k2)
    assert w_pw.shape == (3 * Cp, d) and w_pw2.shape == (3 * Cp, d) and w_proj.shape == (C_out, 3 * Cp)
    b = None if b_proj is None else _f64(b_proj)
    out = np.empty((B, C_out, H, W), dtype=np.float64)
    rc = _load().oracle_msla_forward3(_p(x), _p(w_qkv), _p(w_dw), _p(w_pw), _p(w_dw2), _p(w_pw2), _p(w_proj), _p(b), _p(out),
                                      B, C, H, W, heads, d, k1, k2, C_out, float(eps))
    if rc != 0:
        raise MemoryError("oracle_msla_forward3: scratch allocation failed")
    return out


ACT = {"identity": 0, "relu": 1, "hardswish": 2}


def bias_act(y, bias=None, act: str = "identity") -> np.ndarray:
    """act(y + bias[c]) on y [B, Ch, ...spatial]; returns a new array."""
    y = _f64(y).copy()
    B, Ch = y.shape[:2]
    b = None if bias is None else _f64(bias)
    _load().oracle_bias_act(_p(y), _p(b), B, Ch, int(np.prod(y.shape[2:])), ACT[act])
    return y


def ffn_dwconv(x, w1, w_dw, w2, b1=None, b_dw=None, b2=None, *, act: str = "hardswish", residual: bool = False) -> np.ndarray:
    """FFN with a depthwise convolution (Section 3.1, Fig. 2 left) on NCHW x [B, C, H, W] -> [B, C_out, H, W]."""
    x, w1, w_dw, w2 = map(_f64, (x, w1, w_dw, w2))
    B, C, H, W = x.shape
    Ch, k, C_out = w1.shape[0], w_dw.shape[-1], w2.shape[0]
    assert w1.shape == (Ch, C) and w_dw.shape == (Ch, k, k) and k % 2 == 1 and w2.shape == (C_out, Ch)
    bs = [None if b is None else _f64(b) for b in (b1, b_dw, b2)]
    out = np.empty((B, C_out, H, W), dtype=np.float64)
    rc = _load().oracle_ffn_dwconv(_p(x), _p(w1), _p(bs[0]), _p(w_dw), _p(bs[1]), _p(w2), _p(bs[2]), _p(out),
                                   B, C, Ch, H, W, k, C_out, ACT[act], int(residual))
    if rc == -2:
        raise ValueError("residual needs C_out == C")
    if rc != 0:
        raise MemoryError("oracle_ffn_dwconv: scratch allocation failed")
    return out


def evit_block(x, msla_w, ffn_w, *, heads: int, d: int, act: str = "hardswish", eps: float = 1e-15) -> np.ndarray:
    """The building block of Fig. 2 left: y = x + MSLA(x), out = y + FFN+DWConv(y).
    msla_w: dict with w_qkv, w_dw, w_pw, w_proj, optional b_proj; ffn_w: dict with w1, w_dw, w2, optional b1, b_dw, b2."""
    y = _f64(x) + msla_forward(x, msla_w["w_qkv"], msla_w["w_dw"], msla_w["w_pw"], msla_w["w_proj"], msla_w.get("b_proj"),
                               heads=heads, d=d, eps=eps)
    return ffn_dwconv(y, ffn_w["w1"], ffn_w["w_dw"], ffn_w["w2"], ffn_w.get("b1"), ffn_w.get("b_dw"), ffn_w.get("b2"),
                      act=act, residual=True)
