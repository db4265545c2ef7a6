"""Runs a few launches of the library on synthetic data, for use under a profiler.

    python -m paper_2205_14756_b200.profile_run module B C H W heads d [iters]
    python -m paper_2205_14756_b200.profile_run core   B heads N d     [iters]
    python -m paper_2205_14756_b200.profile_run ffn    B C H W C_hidden [iters]

Inputs are drawn on the device (values do not matter to a profile); the calls
go through the same C ABI as everything else.  Exits non-zero if a kernel
reported a wait time-out.
"""
from __future__ import annotations

import sys

import torch

from . import binding


def run_module(B, C, H, W, heads, d, iters=3):
    Cp = heads * d
    bf = torch.bfloat16
    x = torch.randn(B, C, H, W, device="cuda").to(bf)
    wq = (torch.randn(3 * Cp, C, device="cuda") / C ** 0.5).to(bf)
    wd = (torch.randn(3 * Cp, 5, 5, device="cuda") / 5).to(bf)
    wp = (torch.randn(3 * Cp, d, device="cuda") / d ** 0.5).to(bf)
    wo = (torch.randn(C, 2 * Cp, device="cuda") / (2 * Cp) ** 0.5).to(bf)
    out = torch.empty(B, C, H, W, device="cuda", dtype=bf)
    d0 = binding.make_desc(B, C, H, W, heads, d, C, binding.MSLA_BF16)
    ws = torch.empty(binding.msla_forward_workspace_bytes(d0), dtype=torch.uint8, device="cuda")
    desc = binding.make_desc(B, C, H, W, heads, d, C, binding.MSLA_BF16, workspace=ws)
    w = binding.make_weights(wq, wd, wp, wo)
    for _ in range(iters):
        binding.msla_forward(desc, x, w, out)
    torch.cuda.synchronize()
    return float(out.float().abs().mean())


def run_core(B, heads, N, d, iters=3):
    bf = torch.bfloat16
    q, k, v = (torch.randn(B, heads, N, d, device="cuda").to(bf) for _ in range(3))
    o = torch.empty_like(q)
    nbytes = binding.msla_linattn_relu_workspace_bytes(B, heads, N, d)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    for _ in range(iters):
        binding.msla_linattn_relu_ws(binding.MSLA_BF16, q, k, v, o, B, heads, N, d, 1e-15, ws, nbytes)
    torch.cuda.synchronize()
    return float(o.float().abs().mean())


def run_ffn(B, C, H, W, Ch, iters=3):
    """FFN with a depthwise convolution: hard-swish, all three biases, residual."""
    bf = torch.bfloat16
    x = torch.randn(B, C, H, W, device="cuda").to(bf)
    w1 = (torch.randn(Ch, C, device="cuda") / C ** 0.5).to(bf)
    wd = (torch.randn(Ch, 3, 3, device="cuda") / 3).to(bf)
    w2 = (torch.randn(C, Ch, device="cuda") / Ch ** 0.5).to(bf)
    b1, bd, b2 = (torch.randn(n, device="cuda").to(bf) for n in (Ch, Ch, C))
    out = torch.empty_like(x)
    d0 = binding.make_ffn_desc(B, C, H, W, Ch, C, binding.MSLA_BF16, binding.MSLA_ACT_HARDSWISH, True)
    ws = torch.empty(binding.msla_ffn_workspace_bytes(d0), dtype=torch.uint8, device="cuda")
    desc = binding.make_ffn_desc(B, C, H, W, Ch, C, binding.MSLA_BF16, binding.MSLA_ACT_HARDSWISH, True, workspace=ws)
    w = binding.make_ffn_weights(w1, wd, w2, b1, bd, b2)
    for _ in range(iters):
        binding.msla_ffn_dwconv(desc, x, w, out)
    torch.cuda.synchronize()
    return float(out.float().abs().mean())


def main(argv):
    kind, nums = argv[0], [int(a) for a in argv[1:]]
    if kind == "module":
        val = run_module(*nums[:6], *(nums[6:7] or [3]))
    elif kind == "core":
        val = run_core(*nums[:4], *(nums[4:5] or [3]))
    elif kind == "ffn":
        val = run_ffn(*nums[:5], *(nums[5:6] or [3]))
    else:
        raise SystemExit(__doc__)
    if binding.msla_debug_wait_timeouts() != 0:
        raise SystemExit("a kernel reported a wait time-out")
    print(f"ok mean|out| = {val:.4f}")


if __name__ == "__main__":
    main(sys.argv[1:])
