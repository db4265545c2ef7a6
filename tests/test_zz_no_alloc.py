"""The allocation-free attention-core entry point.

Some users of the library cannot allocate device memory when they call it: a
control loop with a deadline that forbids allocation after start-up (an
allocation may block or fail), a plug-in inside a runtime that owns all device
memory.  msla_linattn_relu_noalloc serves them from a fixed scratch array built
into the library.  Here it must reproduce the workspace-taking entry point on
two calls in a row (the second reuses the array with the first call's leftovers
in it), must agree with the CPU oracle like every other entry point, must leave
the device's free memory untouched once its kernels are warm, and must refuse
shapes whose scratch does not fit.

Collected last on purpose: a failure here cannot hide the other tests from a
run that stops at the first failure."""
import numpy as np
import pytest
import torch

import __graft_entry__  # noqa: F401
import oracle
import util
from paper_2205_14756_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _both(dtype, B, heads, N, d, seed):
    t = inputs.core_inputs(inputs.CoreShape("noalloc", dtype, B, heads, N, d, seed=seed))
    q, k, v = (util.dev(t[n], dtype) for n in ("q", "k", "v"))
    out = torch.full_like(q, float("nan"))
    binding.msla_linattn_relu_noalloc(util.CODE[dtype], q, k, v, out, B, heads, N, d, 1e-15)
    torch.cuda.synchronize()
    return util.host(out), util.run_core(t, dtype, use_ws=True)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_noalloc_matches_workspace_entry_point_twice_in_a_row(dtype):
    # first call: several chunks per head; second call: a different, smaller
    # shape that finds the first call's partial states still in the array
    for B, heads, N, d, seed in [(2, 3, 3000, 32, 21), (1, 2, 333, 16, 22), (2, 3, 3000, 32, 21)]:
        got, ref = _both(dtype, B, heads, N, d, seed)
        assert np.all(np.isfinite(got))
        util.assert_close(got, ref, dtype, f"noalloc {dtype} {B}x{heads}x{N}x{d}")
        assert np.array_equal(got, ref), "same kernels and same split: results should be identical"


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_noalloc_matches_the_oracle_and_allocates_nothing(dtype):
    B, heads, N, d = 2, 3, 3000, 32
    t = inputs.core_inputs(inputs.CoreShape("noalloc_oracle", dtype, B, heads, N, d, seed=24))
    q, k, v = (util.dev(t[n], dtype) for n in ("q", "k", "v"))
    og = util.Guarded(q.numel() * q.element_size())
    out = og.view(q.dtype, q.shape)
    binding.msla_linattn_relu_noalloc(util.CODE[dtype], q, k, v, out, B, heads, N, d, 1e-15)   # warm-up: loads the kernels
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    out.fill_(float("nan"))
    binding.msla_linattn_relu_noalloc(util.CODE[dtype], q, k, v, out, B, heads, N, d, 1e-15)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "a warmed call changed the device's free memory"
    og.check("noalloc output")
    util.assert_close(util.host(out), oracle.linattn_relu(t["q"], t["k"], t["v"], 1e-15), dtype, f"noalloc vs oracle {dtype}",
                      block=util.CORE_BLOCK)


def test_noalloc_full_config2_fits():
    s = inputs.CONFIG2
    assert binding.msla_linattn_relu_workspace_bytes(s.B, s.heads, s.N, s.d) <= binding.MSLA_NOALLOC_SCRATCH_BYTES


def test_noalloc_refuses_oversized_shapes_and_stays_usable():
    B, heads, N, d = 64, 64, 256, 32          # 4096 states need more than the built-in array
    assert binding.msla_linattn_relu_workspace_bytes(B, heads, N, d) > binding.MSLA_NOALLOC_SCRATCH_BYTES
    q = torch.zeros(B, heads, N, d, device="cuda", dtype=torch.bfloat16)
    out = torch.empty_like(q)
    with pytest.raises(binding.MslaError) as e:
        binding.msla_linattn_relu_noalloc(binding.MSLA_BF16, q, q, q, out, B, heads, N, d)
    assert e.value.status == 4 and "scratch" in str(e.value)
    got, ref = _both("bf16", 1, 1, 100, 32, 23)
    assert np.array_equal(got, ref)
