"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

from paper_2205_14756_b200 import binding, inputs

TORCH_DTYPE = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}
CODE = {"f32": binding.MSLA_F32, "bf16": binding.MSLA_BF16, "f16": binding.MSLA_F16}

# Acceptance bounds: fp32 storage -> max-abs error over max |ref| <= 1e-4;
# bf16 storage with fp32 accumulation -> relative L2 error <= 1e-2.
TOL_F32_MAXABS = 1e-4
TOL_BF16_RELL2 = 1e-2


def dev(a: np.ndarray, dtype: str) -> torch.Tensor:
    """Host values (already representable in `dtype`) -> contiguous CUDA tensor."""
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to("cuda").to(TORCH_DTYPE[dtype]).contiguous()


def host(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


def max_abs_rel(got: np.ndarray, ref: np.ndarray) -> float:
    return float(np.max(np.abs(got - ref)) / max(np.max(np.abs(ref)), 1e-300))


def rel_l2(got: np.ndarray, ref: np.ndarray) -> float:
    return float(np.linalg.norm((got - ref).ravel()) / max(np.linalg.norm(ref.ravel()), 1e-300))


# Beside the whole-tensor bound, bf16 results are checked block by block, because a defect confined to one image
# border, one tile seam or one head moves the norm of a 67 M-element tensor by far less than 1e-2:
#   - relative L2 error <= 1e-2 on every block (module output: 32 channels x 16 x 16 pixels; core output: one
#     (batch, head) x 256 tokens), measured against the block's own norm, or against a tenth of the tensor's RMS
#     level where the block's reference is (nearly) zero;
#   - max |got - ref| <= 3e-2 * max |ref|: an element passes through four or five bf16 roundings (each <= 2^-9
#     relative to values no larger than a few times the output's maximum) and fp32 sums in another order; 3e-2 is
#     about 15 half-ulps of bf16 at the tensor's maximum.
MODULE_BLOCK = (1, 32, 16, 16)
CORE_BLOCK = (1, 1, 256, 0)   # 0 = the whole axis
TOL_BF16_MAXABS = 3e-2
# fp16 storage (fp32 arithmetic, one rounding per stored value): the bf16 bounds scaled by the ratio of the unit
# roundoffs, 2^-11 / 2^-8 = 1/8.
TOL_F16_RELL2 = 1.25e-3
TOL_F16_MAXABS = 3.75e-3


def worst_block(got: np.ndarray, ref: np.ndarray, block) -> tuple:
    """Largest per-block relative L2 error and where it is."""
    assert got.ndim == len(block)
    steps = [b if b > 0 else n for b, n in zip(block, got.shape)]
    floor = 0.1 * float(np.sqrt(np.mean(ref * ref)))
    worst, where = 0.0, None
    for idx in np.ndindex(*[(n + s - 1) // s for n, s in zip(got.shape, steps)]):
        sl = tuple(slice(i * s, min((i + 1) * s, n)) for i, s, n in zip(idx, steps, got.shape))
        r, g = ref[sl], got[sl]
        den = max(float(np.linalg.norm(r.ravel())), floor * np.sqrt(r.size), 1e-300)
        e = float(np.linalg.norm((g - r).ravel())) / den
        if e > worst:
            worst, where = e, idx
    return worst, where


def assert_close(got: np.ndarray, ref: np.ndarray, dtype: str, what: str = "", block=None) -> None:
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.all(np.isfinite(got)), f"{what}: non-finite values in the GPU result"
    if dtype == "f32":
        err = max_abs_rel(got, ref)
        assert err <= TOL_F32_MAXABS, f"{what}: max-abs/max|ref| = {err:.3e} > {TOL_F32_MAXABS}"
    else:
        tol_l2, tol_max = (TOL_F16_RELL2, TOL_F16_MAXABS) if dtype == "f16" else (TOL_BF16_RELL2, TOL_BF16_MAXABS)
        err = rel_l2(got, ref)
        assert err <= tol_l2, f"{what}: rel-L2 = {err:.3e} > {tol_l2}"
        mx = max_abs_rel(got, ref)
        assert mx <= tol_max, f"{what}: max-abs/max|ref| = {mx:.3e} > {tol_max}"
        if block is not None:
            w, where = worst_block(got, ref, block)
            assert w <= tol_l2, f"{what}: block {where} has rel-L2 = {w:.3e} > {tol_l2}"


# Guard regions: every output and workspace handed to the library sits inside a larger allocation whose 4 KB on
# either side hold a byte pattern; a store that lands outside its buffer shows up as a changed guard byte.
GUARD = 4096
GUARD_BYTE = 0xA5


class Guarded:
    """`nbytes` of device memory between two guard regions; `.view(dtype, shape)` gives the tensor to pass on."""

    def __init__(self, nbytes: int):
        self.nbytes = int(nbytes)
        self.pad = (-self.nbytes) % 256
        self.full = torch.full((GUARD + self.nbytes + self.pad + GUARD,), GUARD_BYTE, dtype=torch.uint8, device="cuda")
        self.body = self.full[GUARD:GUARD + self.nbytes]

    def view(self, dtype: torch.dtype, shape, fill=float("nan")) -> torch.Tensor:
        t = self.body.view(dtype).reshape(shape)
        t.fill_(fill)
        return t

    def check(self, what: str = "") -> None:
        lo, hi = self.full[:GUARD], self.full[GUARD + self.nbytes:]
        assert bool((lo == GUARD_BYTE).all()) and bool((hi == GUARD_BYTE).all()), f"{what}: a store landed outside its buffer"


def run_core(t: dict, dtype: str, eps: float = 1e-15, use_ws: bool = True) -> np.ndarray:
    """GPU attention core through the C ABI on host arrays q, k, v [B,heads,N,d]."""
    B, heads, N, d = t["q"].shape
    q, k, v = (dev(t[n], dtype) for n in ("q", "k", "v"))
    esz = 4 if dtype == "f32" else 2
    og = Guarded(q.numel() * esz)
    out = og.view(TORCH_DTYPE[dtype], q.shape)
    if use_ws:
        nbytes = binding.msla_linattn_relu_workspace_bytes(B, heads, N, d)
        wg = Guarded(nbytes)
        ws = wg.view(torch.float32, (nbytes // 4,)) if nbytes % 4 == 0 else wg.body
        binding.msla_linattn_relu_ws(CODE[dtype], q, k, v, out, B, heads, N, d, eps, ws, nbytes)
        torch.cuda.synchronize()
        wg.check("core workspace")
    elif dtype == "bf16":
        binding.msla_linattn_relu(q, k, v, out, B, heads, N, d, eps)
    else:
        binding.msla_linattn_relu_f32(q, k, v, out, B, heads, N, d, eps)
    torch.cuda.synchronize()
    og.check("core output")
    return host(out)


def run_module(s: inputs.ModuleShape, t: dict, bias=None) -> np.ndarray:
    """GPU module forward through the C ABI on host arrays."""
    dt = s.dtype
    x, w_qkv, w_dw, w_pw, w_proj = (dev(t[n], dt) for n in ("x", "w_qkv", "w_dw", "w_pw", "w_proj"))
    b = dev(bias, dt) if bias is not None else None
    c_out = t["w_proj"].shape[0]
    desc = binding.make_desc(s.B, s.C, s.H, s.W, s.heads, s.d, c_out, CODE[dt], s.eps, n_scales=s.n_scales, agg_kernel=s.agg_kernel, agg_kernel2=s.agg_kernel2)
    nbytes = binding.msla_forward_workspace_bytes(desc)
    assert nbytes > 0
    wg = Guarded(nbytes)
    ws = wg.view(torch.float32, (nbytes // 4,))
    desc = binding.make_desc(s.B, s.C, s.H, s.W, s.heads, s.d, c_out, CODE[dt], s.eps, n_scales=s.n_scales, agg_kernel=s.agg_kernel, agg_kernel2=s.agg_kernel2, workspace=ws)
    esz = 4 if dt == "f32" else 2
    og = Guarded(s.B * c_out * s.H * s.W * esz)
    out = og.view(TORCH_DTYPE[dt], (s.B, c_out, s.H, s.W))
    extra = [dev(t[n], dt) for n in ("w_dw2", "w_pw2")] if s.n_scales == 3 else [None, None]
    w = binding.make_weights(w_qkv, w_dw, w_pw, w_proj, b, *extra)
    binding.msla_forward(desc, x, w, out)
    torch.cuda.synchronize()
    wg.check("module workspace")
    og.check("module output")
    return host(out)


ACT_CODE = {"identity": 0, "relu": 1, "hardswish": 2}


def run_ffn(s: inputs.FfnShape, t: dict, act: str, residual: bool) -> np.ndarray:
    """GPU FFN+DWConv through the C ABI on host arrays (guarded output and workspace)."""
    dt = s.dtype
    d = {k: dev(v, dt) for k, v in t.items()}
    desc = binding.make_ffn_desc(s.B, s.C, s.H, s.W, s.C_hidden, s.C_out, CODE[dt], ACT_CODE[act], residual)
    nbytes = binding.msla_ffn_workspace_bytes(desc)
    assert nbytes > 0
    wg = Guarded(nbytes)
    ws = wg.view(torch.float32, (nbytes // 4,))
    desc = binding.make_ffn_desc(s.B, s.C, s.H, s.W, s.C_hidden, s.C_out, CODE[dt], ACT_CODE[act], residual, workspace=ws)
    esz = 4 if dt == "f32" else 2
    og = Guarded(s.B * s.C_out * s.N * esz)
    out = og.view(TORCH_DTYPE[dt], (s.B, s.C_out, s.H, s.W))
    w = binding.make_ffn_weights(d["w1"], d["w_dw"], d["w2"], d.get("b1"), d.get("b_dw"), d.get("b2"))
    binding.msla_ffn_dwconv(desc, d["x"], w, out)
    torch.cuda.synchronize()
    wg.check("FFN workspace")
    og.check("FFN output")
    return host(out)


def run_block(s: inputs.ModuleShape, t: dict, f: dict, c_hidden: int, act: str) -> np.ndarray:
    """GPU building block (attention module + FFN, two residual connections) through the C ABI."""
    dt = s.dtype
    x, w_qkv, w_dw, w_pw, w_proj = (dev(t[n], dt) for n in ("x", "w_qkv", "w_dw", "w_pw", "w_proj"))
    fd = {k: dev(v, dt) for k, v in f.items() if k != "x"}
    a0 = binding.make_desc(s.B, s.C, s.H, s.W, s.heads, s.d, s.C, CODE[dt], s.eps)
    f0 = binding.make_ffn_desc(s.B, s.C, s.H, s.W, c_hidden, s.C, CODE[dt], ACT_CODE[act], True)
    ag, fg = Guarded(binding.msla_forward_workspace_bytes(a0)), Guarded(binding.msla_ffn_workspace_bytes(f0))
    adesc = binding.make_desc(s.B, s.C, s.H, s.W, s.heads, s.d, s.C, CODE[dt], s.eps, workspace=ag.view(torch.uint8, (ag.nbytes,), 0))
    fdesc = binding.make_ffn_desc(s.B, s.C, s.H, s.W, c_hidden, s.C, CODE[dt], ACT_CODE[act], True,
                                  workspace=fg.view(torch.uint8, (fg.nbytes,), 0))
    esz = 4 if dt == "f32" else 2
    yg, og = Guarded(x.numel() * esz), Guarded(x.numel() * esz)
    y, out = yg.view(TORCH_DTYPE[dt], x.shape), og.view(TORCH_DTYPE[dt], x.shape)
    binding.msla_evit_block(adesc, binding.make_weights(w_qkv, w_dw, w_pw, w_proj), fdesc,
                            binding.make_ffn_weights(fd["w1"], fd["w_dw"], fd["w2"], fd.get("b1"), fd.get("b_dw"), fd.get("b2")), x, y, out)
    torch.cuda.synchronize()
    for gd, what in ((ag, "attention workspace"), (fg, "FFN workspace"), (yg, "y"), (og, "block output")):
        gd.check(what)
    return host(out)
