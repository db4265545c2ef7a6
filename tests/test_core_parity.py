"""GPU attention core (through the C ABI) against the fp64 CPU oracle."""
import numpy as np
import pytest
import torch

import __graft_entry__  # noqa: F401
import oracle
import util
from paper_2205_14756_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _case(dtype, B, heads, N, d, seed):
    s = inputs.CoreShape("case", dtype, B, heads, N, d, seed=seed)
    t = inputs.core_inputs(s)
    return t, oracle.linattn_relu(t["q"], t["k"], t["v"], s.eps)


# sizes span one chunk, several chunks, ragged tails and single tokens
SHAPES = [(1, 1, 1, 32), (1, 2, 7, 16), (2, 3, 64, 32), (1, 2, 257, 32), (2, 2, 1000, 16),
          (1, 3, 4099, 32), (1, 1, 20000, 32), (3, 5, 513, 16), (1, 1, 65, 32)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,heads,N,d", SHAPES)
def test_core_matches_oracle(dtype, B, heads, N, d):
    t, ref = _case(dtype, B, heads, N, d, seed=100 + N)
    util.assert_close(util.run_core(t, dtype), ref, dtype, f"core {dtype} {B}x{heads}x{N}x{d}", block=util.CORE_BLOCK)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_core_pool_scratch_variant(dtype):
    t, ref = _case(dtype, 2, 2, 777, 32, seed=7)
    util.assert_close(util.run_core(t, dtype, use_ws=False), ref, dtype, "core (pool scratch)")


def test_core_full_size_config2():
    """Config 2 at full size in the launch configuration the benchmark times."""
    s = inputs.CONFIG2
    t = inputs.core_inputs(s)
    ref = oracle.linattn_relu(t["q"], t["k"], t["v"], s.eps)
    util.assert_close(util.run_core(t, "bf16"), ref, "bf16", "config 2", block=util.CORE_BLOCK)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_core_zero_denominator_rows_are_zero(dtype):
    t, _ = _case(dtype, 1, 2, 300, 32, seed=9)
    t["q"][0, 0, 5] = -1.0               # no positive entry: 0 / (0 + eps)
    t["q"][0, 1, 299] = 0.0
    t["k"][0, 1] = -np.abs(t["k"][0, 1])  # a head whose keys are all non-positive
    got = util.run_core(t, dtype)
    ref = oracle.linattn_relu(t["q"], t["k"], t["v"], 1e-15)
    assert np.all(np.isfinite(got))
    assert np.all(got[0, 0, 5] == 0.0) and np.all(got[0, 1] == 0.0)
    util.assert_close(got, ref, dtype, "zero-denominator case")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_core_is_bitwise_reproducible(dtype):
    t, _ = _case(dtype, 2, 4, 3001, 32, seed=11)
    a = util.run_core(t, dtype)
    for _ in range(2):
        assert np.array_equal(a, util.run_core(t, dtype))


def test_core_constant_v_property_large():
    """A property that holds at any size: constant V gives that constant."""
    B, heads, N, d = 1, 2, 100_000, 32
    g = torch.Generator(device="cuda").manual_seed(3)
    q = torch.randn(B, heads, N, d, device="cuda", generator=g).to(torch.bfloat16)
    k = torch.randn(B, heads, N, d, device="cuda", generator=g).to(torch.bfloat16)
    q[..., 0] = q[..., 0].abs() + 0.5
    v = torch.full_like(q, 1.5)
    out = torch.empty_like(q)
    binding.msla_linattn_relu(q, k, v, out, B, heads, N, d, 1e-15)
    torch.cuda.synchronize()
    assert torch.allclose(out.float(), torch.full_like(out, 1.5).float(), rtol=2e-2)


def test_core_runtime_argument_errors():
    q = torch.zeros(1, 1, 8, 32, device="cuda", dtype=torch.bfloat16)
    out = torch.empty_like(q)
    with pytest.raises(binding.MslaError) as e:
        binding.msla_linattn_relu(q, q, q, q, 1, 1, 8, 32)
    assert e.value.status == 1
    with pytest.raises(binding.MslaError) as e:
        binding.msla_linattn_relu(q, q, q, out, 1, 1, 8, 48)
    assert e.value.status == 2
    ws = torch.empty(4, device="cuda")
    with pytest.raises(binding.MslaError) as e:
        binding.msla_linattn_relu_ws(1, q, q, q, out, 1, 1, 8, 32, 1e-15, ws, 16)
    assert e.value.status == 4
    # the context is still usable afterwards
    binding.msla_linattn_relu(q, q, q, out, 1, 1, 8, 32)
    torch.cuda.synchronize()
