"""Seeded synthetic inputs for the multi-scale linear attention (MSLA) module.

This module only *draws numbers and names shapes*.  It holds none of the
method's arithmetic, so both the CPU oracle's tests and the CUDA path may use
it without sharing any computation.

Generator: a counter-based scheme.  Element ``i`` of tensor ``stream`` under
``seed`` is obtained from two 64-bit hashes (the splitmix64 finaliser applied
to a counter built from seed, stream and index), mapped to two uniforms and
then to one standard normal by the Box-Muller transform.  The value of an
element therefore depends only on (seed, stream, i) -- never on tensor shape,
draw order, numpy version or thread count.

The paper evaluates on Cityscapes / ADE20K / FFHQ-sized feature maps with
trained weights; neither is available offline, and the module has no
data-dependent control flow, so N(0,1) activations and N(0, 1/fan_in) weights
of the same shapes stand in for them.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Tuple

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _splitmix64(z: np.ndarray) -> np.ndarray:
    """splitmix64 output function (Steele, Lea, Flood 2014) on uint64 arrays."""
    with np.errstate(over="ignore"):
        z = (z + _GOLDEN).astype(np.uint64)
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


def normal(seed: int, stream: int, count: int, std: float = 1.0) -> np.ndarray:
    """``count`` draws of N(0, std^2) as float64, element i a pure function of
    (seed, stream, i)."""
    out = np.empty(count, dtype=np.float64)
    step = 1 << 22
    with np.errstate(over="ignore"):
        base = _splitmix64(np.array([(seed << 32) ^ stream], dtype=np.uint64))[0]
    for lo in range(0, count, step):
        hi = min(count, lo + step)
        idx = np.arange(lo, hi, dtype=np.uint64)
        with np.errstate(over="ignore"):
            c = base + idx * np.uint64(2)
            h1 = _splitmix64(c)
            h2 = _splitmix64(c + np.uint64(1))
        # 53-bit uniforms; u1 in (0,1], u2 in [0,1)
        u1 = ((h1 >> np.uint64(11)).astype(np.float64) + 1.0) * (1.0 / 9007199254740992.0)
        u2 = (h2 >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)
        out[lo:hi] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    if std != 1.0:
        out *= std
    return out


def round_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float -> bfloat16 bit patterns (uint16), round-to-nearest-even."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> float32, exact."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def quantise(a: np.ndarray, dtype: str) -> np.ndarray:
    """Round ``a`` to the storage type of a config ('f32', 'bf16' or 'f16') and return
    it widened back to float32.  Both implementations consume these values."""
    if dtype == "f32":
        return np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "bf16":
        return bf16_bits_to_f32(round_to_bf16_bits(a)).reshape(a.shape)
    if dtype == "f16":  # IEEE binary16, round to nearest even (numpy's conversion)
        return np.ascontiguousarray(a, dtype=np.float32).astype(np.float16).astype(np.float32)
    raise ValueError(dtype)


@dataclass(frozen=True)
class ModuleShape:
    """One multi-scale linear attention module call on an NCHW feature map."""
    name: str
    dtype: str          # 'f32' | 'bf16' : storage type of activations and weights
    B: int
    C: int
    H: int
    W: int
    heads: int          # heads per scale
    d: int              # channels per head
    seed: int
    n_scales: int = 2   # identity branch + one 5x5-aggregated branch
    agg_kernel: int = 5
    eps: float = 1e-15
    agg_kernel2: int = 3  # filter of the second aggregated branch when n_scales == 3

    @property
    def N(self) -> int:
        return self.H * self.W

    @property
    def Cp(self) -> int:            # C' = heads * d
        return self.heads * self.d

    @property
    def C_out(self) -> int:
        return self.C


@dataclass(frozen=True)
class CoreShape:
    """One attention-core call on [B, heads, N, d] tensors."""
    name: str
    dtype: str
    B: int
    heads: int
    N: int
    d: int
    seed: int
    eps: float = 1e-15


# The five benchmark configurations (shapes only).
CONFIG1 = ModuleShape("cfg1_module_f32_16x16", "f32", 1, 64, 16, 16, 4, 16, seed=0)
CONFIG2 = CoreShape("cfg2_core_bf16_b8_h16_n4096_d32", "bf16", 8, 16, 4096, 32, seed=1)
CONFIG3 = ModuleShape("cfg3_module_bf16_64x128_c192", "bf16", 1, 192, 64, 128, 6, 32, seed=2)
CONFIG4 = ModuleShape("cfg4_module_bf16_b16_64x64_c256", "bf16", 16, 256, 64, 64, 8, 32, seed=3)
CONFIG5 = tuple(
    ModuleShape(f"cfg5_module_bf16_{w}x{w}_c256", "bf16", 1, 256, w, w, 8, 32, seed=4)
    for w in (32, 64, 128, 256, 512)
)


def module_inputs(s: ModuleShape) -> Dict[str, np.ndarray]:
    """Activations ~ N(0,1); weights ~ N(0, 1/fan_in) (second argument is the
    variance).  Values are already rounded to the config's storage type and
    returned as float32 arrays.

    x      [B, C, H, W]
    w_qkv  [3C', C]          fan_in = C
    w_dw   [3C', k, k]       fan_in = k*k
    w_pw   [3C', d]          fan_in = d
    w_proj [C_out, S*C']     fan_in = S*C'
    """
    Cp, k = s.Cp, s.agg_kernel
    shapes = {
        "x": ((s.B, s.C, s.H, s.W), 1.0),
        "w_qkv": ((3 * Cp, s.C), s.C ** -0.5),
        "w_dw": ((3 * Cp, k, k), (k * k) ** -0.5),
        "w_pw": ((3 * Cp, s.d), s.d ** -0.5),
        "w_proj": ((s.C_out, s.n_scales * Cp), (s.n_scales * Cp) ** -0.5),
    }
    out = {}
    for stream, (name, (shape, std)) in enumerate(shapes.items()):
        n = int(np.prod(shape))
        out[name] = quantise(normal(s.seed, stream, n, std).reshape(shape), s.dtype)
    if s.n_scales == 3:  # the second aggregated branch's filters: streams 5 and 6
        k2 = s.agg_kernel2
        out["w_dw2"] = quantise(normal(s.seed, 5, 3 * Cp * k2 * k2, 1.0 / k2).reshape(3 * Cp, k2, k2), s.dtype)
        out["w_pw2"] = quantise(normal(s.seed, 6, 3 * Cp * s.d, s.d ** -0.5).reshape(3 * Cp, s.d), s.dtype)
    return out


def core_inputs(s: CoreShape) -> Dict[str, np.ndarray]:
    """q, k, v ~ N(0,1), each [B, heads, N, d], rounded to the storage type."""
    shape = (s.B, s.heads, s.N, s.d)
    n = int(np.prod(shape))
    return {
        name: quantise(normal(s.seed, stream, n).reshape(shape), s.dtype)
        for stream, name in enumerate(("q", "k", "v"))
    }


@dataclass(frozen=True)
class FfnShape:
    """One FFN with a depthwise convolution on an NCHW feature map (the second half of the building block)."""
    name: str
    dtype: str          # 'f32' | 'bf16'
    B: int
    C: int
    H: int
    W: int
    C_hidden: int
    C_out: int
    seed: int

    @property
    def N(self) -> int:
        return self.H * self.W


def ffn_inputs(s: FfnShape, biases: bool = True) -> Dict[str, np.ndarray]:
    """Activations ~ N(0,1); weights ~ N(0, 1/fan_in); biases ~ N(0, 0.25) (a folded normalisation's shift).

    x [B, C, H, W]; w1 [C_hidden, C] fan_in C; w_dw [C_hidden, 3, 3] fan_in 9; w2 [C_out, C_hidden] fan_in C_hidden;
    b1, b_dw [C_hidden]; b2 [C_out].  Streams 8.. so that a block's two halves draw different numbers under one seed."""
    shapes = {
        "x": ((s.B, s.C, s.H, s.W), 1.0),
        "w1": ((s.C_hidden, s.C), s.C ** -0.5),
        "w_dw": ((s.C_hidden, 3, 3), 1.0 / 3.0),
        "w2": ((s.C_out, s.C_hidden), s.C_hidden ** -0.5),
        "b1": ((s.C_hidden,), 0.5),
        "b_dw": ((s.C_hidden,), 0.5),
        "b2": ((s.C_out,), 0.5),
    }
    out = {}
    for stream, (name, (shape, std)) in enumerate(shapes.items()):
        if not biases and name.startswith("b"):
            continue
        n = int(np.prod(shape))
        out[name] = quantise(normal(s.seed, 8 + stream, n, std).reshape(shape), s.dtype)
    return out
