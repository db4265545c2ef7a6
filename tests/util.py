"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

from paper_2205_14756_b200 import binding, inputs

TORCH_DTYPE = {"f32": torch.float32, "bf16": torch.bfloat16}
CODE = {"f32": binding.MSLA_F32, "bf16": binding.MSLA_BF16}

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


def assert_close(got: np.ndarray, ref: np.ndarray, dtype: str, what: str = "") -> None:
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.all(np.isfinite(got)), f"{what}: non-finite values in the GPU result"
    if dtype == "f32":
        err = max_abs_rel(got, ref)
        assert err <= TOL_F32_MAXABS, f"{what}: max-abs/max|ref| = {err:.3e} > {TOL_F32_MAXABS}"
    else:
        err = rel_l2(got, ref)
        assert err <= TOL_BF16_RELL2, f"{what}: rel-L2 = {err:.3e} > {TOL_BF16_RELL2}"


def run_core(t: dict, dtype: str, eps: float = 1e-15, use_ws: bool = True) -> np.ndarray:
    """GPU attention core through the C ABI on host arrays q, k, v [B,heads,N,d]."""
    B, heads, N, d = t["q"].shape
    q, k, v = (dev(t[n], dtype) for n in ("q", "k", "v"))
    out = torch.full_like(q, float("nan"))
    if use_ws:
        nbytes = binding.msla_linattn_relu_workspace_bytes(B, heads, N, d)
        ws = torch.full((nbytes // 4,), float("nan"), dtype=torch.float32, device="cuda")
        binding.msla_linattn_relu_ws(CODE[dtype], q, k, v, out, B, heads, N, d, eps, ws, nbytes)
    elif dtype == "bf16":
        binding.msla_linattn_relu(q, k, v, out, B, heads, N, d, eps)
    else:
        binding.msla_linattn_relu_f32(q, k, v, out, B, heads, N, d, eps)
    torch.cuda.synchronize()
    return host(out)


def run_module(s: inputs.ModuleShape, t: dict, bias=None) -> np.ndarray:
    """GPU module forward through the C ABI on host arrays."""
    dt = s.dtype
    x, w_qkv, w_dw, w_pw, w_proj = (dev(t[n], dt) for n in ("x", "w_qkv", "w_dw", "w_pw", "w_proj"))
    b = dev(bias, dt) if bias is not None else None
    desc = binding.make_desc(s.B, s.C, s.H, s.W, s.heads, s.d, s.C_out, CODE[dt], s.eps)
    nbytes = binding.msla_forward_workspace_bytes(desc)
    assert nbytes > 0
    ws = torch.full((nbytes // 4,), float("nan"), dtype=torch.float32, device="cuda")
    desc = binding.make_desc(s.B, s.C, s.H, s.W, s.heads, s.d, s.C_out, CODE[dt], s.eps, workspace=ws)
    out = torch.full((s.B, s.C_out, s.H, s.W), float("nan"), dtype=TORCH_DTYPE[dt], device="cuda")
    w = binding.make_weights(w_qkv, w_dw, w_pw, w_proj, b)
    binding.msla_forward(desc, x, w, out)
    torch.cuda.synchronize()
    return host(out)
