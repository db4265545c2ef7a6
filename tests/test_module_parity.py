"""GPU module forward and its stages (through the C ABI) against the oracle."""
import numpy as np
import pytest
import torch

import __graft_entry__  # noqa: F401
import oracle
import util
from paper_2205_14756_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _ref(s, t, bias=None):
    return oracle.msla_forward(t["x"], t["w_qkv"], t["w_dw"], t["w_pw"], t["w_proj"], bias,
                               heads=s.heads, d=s.d, eps=s.eps)


def test_config1_fp32():
    s = inputs.CONFIG1
    t = inputs.module_inputs(s)
    util.assert_close(util.run_module(s, t), _ref(s, t), "f32", "config 1")


SMALL = [
    # name, dtype, B, C, H, W, heads, d: ragged tiles, images narrower than a tile, H=1
    ("r1", "f32", 2, 32, 5, 7, 2, 16),
    ("r2", "bf16", 1, 64, 9, 33, 2, 32),
    ("r3", "bf16", 2, 32, 1, 40, 1, 32),
    ("r4", "f32", 1, 64, 3, 3, 2, 32),
    ("r5", "bf16", 1, 96, 24, 20, 3, 32),
    ("r6", "bf16", 3, 64, 17, 16, 4, 16),
    ("r7", "f32", 1, 16, 1, 1, 1, 16),
    ("r8", "bf16", 1, 128, 40, 24, 8, 16),
    ("r9", "bf16", 2, 48, 11, 13, 3, 16),
    # 10 heads over both scales: the fused apply + projection kernel runs a second round with two heads only;
    # 240 tokens per image: a ragged last token tile in each of two images
    ("r10", "bf16", 2, 160, 12, 20, 5, 32),
]


@pytest.mark.parametrize("name,dtype,B,C,H,W,heads,d", SMALL)
def test_small_modules(name, dtype, B, C, H, W, heads, d):
    s = inputs.ModuleShape(name, dtype, B, C, H, W, heads, d, seed=40 + H)
    t = inputs.module_inputs(s)
    util.assert_close(util.run_module(s, t), _ref(s, t), dtype, name, block=util.MODULE_BLOCK)


# Output widths and biases that differ from the input's: C_out = 40 (one ragged block of output channels in the fused
# apply + projection), and two shapes with d = 32 and C_out > 256, which the fused kernel does not take: they run the
# tensor-core apply step on paired head planes followed by the planar output-projection GEMM (one with a bias, one
# with a ragged token tile and an odd number of head pairs).
@pytest.mark.parametrize("B,C,H,W,heads,d,c_out,with_bias,fused", [(1, 64, 8, 8, 2, 32, 40, True, 1),
                                                                    (2, 64, 8, 16, 2, 32, 264, True, 0),
                                                                    (1, 64, 12, 20, 3, 32, 320, False, 0),
                                                                    (1, 64, 16, 16, 4, 16, 72, True, 1)])
def test_module_with_bias_and_different_c_out(B, C, H, W, heads, d, c_out, with_bias, fused):
    s = inputs.ModuleShape("cout", "bf16", B, C, H, W, heads, d, seed=77)
    t = inputs.module_inputs(s)
    k = 2 * heads * d
    t["w_proj"] = inputs.quantise(inputs.normal(77, 9, c_out * k, k ** -0.5).reshape(c_out, k), "bf16")
    bias = inputs.quantise(inputs.normal(77, 10, c_out), "bf16") if with_bias else None
    desc = binding.make_desc(B, C, H, W, heads, d, c_out, binding.MSLA_BF16)
    assert binding.msla_forward_fuses_apply(desc) == fused
    got = util.run_module(s, t, bias)
    util.assert_close(got, _ref(s, t, bias), "bf16", f"C_out = {c_out}", block=util.MODULE_BLOCK)
    assert binding.msla_debug_wait_timeouts() == 0


# A 3x3 aggregation filter (another of Section 3.1's small kernels): same kernels, taps embedded in 5x5.
@pytest.mark.parametrize("dtype,B,C,H,W,heads,d", [("f32", 1, 32, 9, 11, 2, 16), ("bf16", 2, 64, 24, 40, 2, 32), ("bf16", 1, 96, 16, 16, 6, 16)])
def test_module_with_3x3_aggregation(dtype, B, C, H, W, heads, d):
    s = inputs.ModuleShape("agg3", dtype, B, C, H, W, heads, d, seed=41, agg_kernel=3)
    t = inputs.module_inputs(s)
    assert t["w_dw"].shape[-2:] == (3, 3)
    util.assert_close(util.run_module(s, t), _ref(s, t), dtype, "3x3 aggregation", block=util.MODULE_BLOCK if dtype == "bf16" else None)


# Three branches (Section 3.1's multi-scale tokens with a second aggregated copy): 5x5 + 3x3 and 3x3 + 5x5 filters;
# fp32 on the plain kernels, bf16 with 3C' <= 512 through the fused output kernel, with 3C' = 768 and with an odd
# number of heads through the apply kernel and a projection GEMM.
@pytest.mark.parametrize("dtype,B,C,H,W,heads,d,k1,k2,fused", [("f32", 1, 32, 7, 9, 2, 16, 5, 3, 0), ("bf16", 2, 64, 24, 40, 2, 32, 5, 3, 1),
                                                              ("bf16", 1, 128, 16, 24, 4, 32, 3, 5, 1), ("bf16", 1, 256, 16, 16, 8, 32, 5, 3, 0),
                                                              ("bf16", 1, 32, 12, 12, 1, 32, 5, 5, 1), ("bf16", 1, 96, 16, 16, 6, 16, 5, 3, 1)])
def test_module_with_three_branches(dtype, B, C, H, W, heads, d, k1, k2, fused):
    s = inputs.ModuleShape("three", dtype, B, C, H, W, heads, d, seed=43, n_scales=3, agg_kernel=k1, agg_kernel2=k2)
    t = inputs.module_inputs(s)
    assert t["w_proj"].shape == (C, 3 * heads * d) and t["w_dw2"].shape[-1] == k2
    desc = binding.make_desc(B, C, H, W, heads, d, C, binding.MSLA_BF16 if dtype == "bf16" else binding.MSLA_F32, n_scales=3,
                             agg_kernel=k1, agg_kernel2=k2)
    assert binding.msla_forward_fuses_apply(desc) == fused
    ref = oracle.msla_forward3(t["x"], t["w_qkv"], t["w_dw"], t["w_pw"], t["w_dw2"], t["w_pw2"], t["w_proj"], heads=heads, d=d)
    util.assert_close(util.run_module(s, t), ref, dtype, "three branches", block=util.MODULE_BLOCK if dtype == "bf16" else None)
    assert binding.msla_debug_wait_timeouts() == 0


def test_config3_bf16():
    s = inputs.CONFIG3
    t = inputs.module_inputs(s)
    util.assert_close(util.run_module(s, t), _ref(s, t), "bf16", "config 3", block=util.MODULE_BLOCK)


def test_config4_bf16():
    s = inputs.CONFIG4
    t = inputs.module_inputs(s)
    util.assert_close(util.run_module(s, t), _ref(s, t), "bf16", "config 4", block=util.MODULE_BLOCK)


@pytest.mark.parametrize("idx", [0, 1, 2, 3, 4])
def test_config5_sweep_bf16(idx):
    """The resolution sweep, element by element against the oracle; idx 4 (512x512,
    262144 tokens) is the shape and launch configuration the benchmark times."""
    s = inputs.CONFIG5[idx]
    t = inputs.module_inputs(s)
    util.assert_close(util.run_module(s, t), _ref(s, t), "bf16", s.name, block=util.MODULE_BLOCK)


def test_module_is_bitwise_reproducible():
    s = inputs.ModuleShape("det", "bf16", 2, 64, 20, 24, 2, 32, seed=8)
    t = inputs.module_inputs(s)
    a = util.run_module(s, t)
    assert np.array_equal(a, util.run_module(s, t))


# ------------------------------------------------------------------ stages
def _tok_major(a):      # [B, C, H, W] -> [B, H*W, C]
    B, C = a.shape[:2]
    return np.ascontiguousarray(a.reshape(B, C, -1).transpose(0, 2, 1))


def _planar(a, d):      # [B, C, H, W] -> [B, C/d, H*W, d]
    B, C = a.shape[:2]
    return np.ascontiguousarray(a.reshape(B, C // d, d, -1).transpose(0, 1, 3, 2))


@pytest.mark.parametrize("dtype,B,C,Cout,N", [("f32", 2, 24, 48, 100), ("bf16", 1, 64, 192, 333), ("bf16", 2, 256, 768, 4096),
                                              ("bf16", 1, 64, 192, 128), ("bf16", 3, 72, 208, 1000), ("bf16", 1, 192, 576, 8192),
                                              ("bf16", 2, 8, 16, 8)])
def test_stage_project_in(dtype, B, C, Cout, N):
    d = 32 if Cout % 32 == 0 else 16 if Cout % 16 == 0 else 8
    x = inputs.quantise(inputs.normal(1, 0, B * C * N).reshape(B, C, N), dtype)
    w = inputs.quantise(inputs.normal(1, 1, Cout * C, C ** -0.5).reshape(Cout, C), dtype)
    y = torch.empty(B, Cout // d, N, d, dtype=util.TORCH_DTYPE[dtype], device="cuda")
    binding.msla_project_in(util.CODE[dtype], util.dev(x, dtype), util.dev(w, dtype), y, B, C, Cout, N, d)
    torch.cuda.synchronize()
    ref = _planar(oracle.conv1x1(x[..., None], w), d)
    util.assert_close(util.host(y), ref, dtype, "project_in")
    assert binding.msla_debug_wait_timeouts() == 0


@pytest.mark.parametrize("dtype,B,Cin,Cout,N", [("f32", 2, 24, 40, 100), ("bf16", 1, 128, 64, 333), ("bf16", 2, 512, 256, 4096),
                                                ("bf16", 1, 128, 64, 256), ("bf16", 3, 136, 200, 1000), ("bf16", 1, 384, 192, 8192),
                                                ("bf16", 2, 8, 8, 8)])
def test_stage_project_out(dtype, B, Cin, Cout, N):
    a = inputs.quantise(inputs.normal(2, 0, B * N * Cin).reshape(B, N, Cin), dtype)
    w = inputs.quantise(inputs.normal(2, 1, Cout * Cin, Cin ** -0.5).reshape(Cout, Cin), dtype)
    bias = inputs.quantise(inputs.normal(2, 2, Cout), dtype)
    y = torch.empty(B, Cout, N, dtype=util.TORCH_DTYPE[dtype], device="cuda")
    binding.msla_project_out(util.CODE[dtype], util.dev(a, dtype), util.dev(w, dtype), util.dev(bias, dtype), y, B, Cin, Cout, N)
    torch.cuda.synchronize()
    ref = oracle.conv1x1(np.ascontiguousarray(a.transpose(0, 2, 1)), w, bias)
    util.assert_close(util.host(y), ref, dtype, "project_out")
    assert binding.msla_debug_wait_timeouts() == 0


@pytest.mark.parametrize("dtype,B,H,W,Ch,d", [("f32", 1, 6, 9, 48, 16), ("bf16", 2, 13, 21, 96, 32), ("bf16", 1, 1, 5, 32, 32),
                                              ("bf16", 1, 64, 64, 192, 32), ("bf16", 1, 3, 70, 64, 16), ("bf16", 2, 16, 16, 32, 32),
                                              ("bf16", 1, 17, 35, 64, 32), ("bf16", 1, 5, 3, 32, 32), ("bf16", 1, 40, 7, 32, 32),
                                              ("bf16", 2, 19, 37, 96, 16), ("bf16", 1, 64, 64, 192, 16), ("bf16", 1, 2, 2, 32, 16),
                                              ("bf16", 1, 9, 9, 48, 16),
                                              # 432 (image, group, tile) units of 9 tiles per plane: the persistent CTAs' runs cross
                                              # tile-band, group and image boundaries
                                              ("bf16", 4, 48, 48, 384, 32)])
def test_stage_aggregate(dtype, B, H, W, Ch, d):
    t = inputs.quantise(inputs.normal(3, 0, B * Ch * H * W).reshape(B, Ch, H, W), dtype)
    w_dw = inputs.quantise(inputs.normal(3, 1, Ch * 25, 0.2).reshape(Ch, 5, 5), dtype)
    w_pw = inputs.quantise(inputs.normal(3, 2, Ch * d, d ** -0.5).reshape(Ch, d), dtype)
    y = torch.empty(B, Ch // d, H * W, d, dtype=util.TORCH_DTYPE[dtype], device="cuda")
    binding.msla_aggregate(util.CODE[dtype], util.dev(_planar(t, d), dtype), util.dev(w_dw, dtype), util.dev(w_pw, dtype), y, B, H, W, Ch, d)
    torch.cuda.synchronize()
    ref = _planar(oracle.group1x1(oracle.dwconv(t, w_dw), w_pw), d)
    util.assert_close(util.host(y), ref, dtype, "aggregate")
    assert binding.msla_debug_wait_timeouts() == 0


# ------------------------------------------------- other entry points of the module
def test_forward_host_and_profiled_match_forward():
    """msla_forward_host (host buffers, copies inside the call) and msla_forward_profiled
    (events between the steps) run the same kernels as msla_forward: bitwise equal output."""
    s = inputs.ModuleShape("entry", "bf16", 2, 64, 24, 40, 2, 32, seed=31)
    t = inputs.module_inputs(s)
    ref = util.run_module(s, t)
    dt = torch.bfloat16
    x, w_qkv, w_dw, w_pw, w_proj = (util.dev(t[n], "bf16") for n in ("x", "w_qkv", "w_dw", "w_pw", "w_proj"))
    weights = binding.make_weights(w_qkv, w_dw, w_pw, w_proj)
    d0 = binding.make_desc(s.B, s.C, s.H, s.W, s.heads, s.d, s.C_out, binding.MSLA_BF16, s.eps)
    nbytes = binding.msla_forward_host_workspace_bytes(d0)
    assert nbytes > binding.msla_forward_workspace_bytes(d0)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    desc = binding.make_desc(s.B, s.C, s.H, s.W, s.heads, s.d, s.C_out, binding.MSLA_BF16, s.eps, workspace=ws)
    # host buffers
    hx = x.cpu().pin_memory()
    ho = torch.empty(s.B, s.C_out, s.H, s.W, dtype=dt).pin_memory()
    binding.msla_forward_host(desc, hx, weights, ho)
    torch.cuda.synchronize()
    assert np.array_equal(util.host(ho), ref)
    # events between the steps
    out = torch.empty(s.B, s.C_out, s.H, s.W, dtype=dt, device="cuda")
    st = torch.cuda.current_stream()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
    for e in evs:
        e.record(st)
    launches = binding.msla_kernel_launches()
    binding.msla_forward_profiled(desc, x, weights, out, st, evs)
    torch.cuda.synchronize()
    # fused steps 4+5: projection, aggregation, partial states, state fragments, apply + projection
    assert binding.msla_kernel_launches() - launches == (5 if binding.msla_forward_fuses_apply(desc) == 1 else 6)
    assert np.array_equal(util.host(out), ref)
    assert all(evs[i].elapsed_time(evs[i + 1]) >= 0.0 for i in range(5))
    # too small a workspace for the host variant is refused before anything runs
    small = binding.make_desc(s.B, s.C, s.H, s.W, s.heads, s.d, s.C_out, binding.MSLA_BF16, s.eps,
                              workspace=ws[:binding.msla_forward_workspace_bytes(d0)])
    with pytest.raises(binding.MslaError) as err:
        binding.msla_forward_host(small, hx, weights, ho)
    assert err.value.status == 4


def test_module_argument_errors_on_device():
    s = inputs.ModuleShape("err", "bf16", 1, 64, 8, 8, 2, 32, seed=1)
    x = torch.zeros(1, 64, 8, 8, dtype=torch.bfloat16, device="cuda")
    w = [torch.zeros(n, dtype=torch.bfloat16, device="cuda") for n in (192 * 64, 192 * 25, 192 * 32, 64 * 128)]
    weights = binding.make_weights(*w)
    d0 = binding.make_desc(1, 64, 8, 8, 2, 32, 64, binding.MSLA_BF16)
    ws = torch.empty(binding.msla_forward_workspace_bytes(d0), dtype=torch.uint8, device="cuda")
    desc = binding.make_desc(1, 64, 8, 8, 2, 32, 64, binding.MSLA_BF16, workspace=ws)
    with pytest.raises(binding.MslaError) as e:      # out aliases x
        binding.msla_forward(desc, x, weights, x)
    assert e.value.status == 1
    out = torch.empty_like(x)
    bad = binding.make_desc(1, 64, 8, 8, 2, 32, 64, binding.MSLA_BF16, workspace=ws[16:])
    bad.workspace_bytes = 8
    with pytest.raises(binding.MslaError) as e:
        binding.msla_forward(bad, x, weights, out)
    assert e.value.status == 4
    binding.msla_forward(desc, x, weights, out)       # the context is still usable; zeros in, zeros out
    torch.cuda.synchronize()
    assert float(out.float().abs().max()) == 0.0


def test_bounded_wait_gives_up_and_leaves_the_context_usable():
    """The wait every kernel relies on, run on a barrier nobody arrives at with a limit of about a millisecond: it
    must give up and say so (no product kernel is made to time out), and the library must work afterwards."""
    scratch = torch.zeros(2, dtype=torch.int32, device="cuda")
    assert binding.msla_debug_wait_selftest(2_000_000, scratch) == 1
    assert scratch.tolist() == [1, 1]
    assert binding.msla_debug_wait_selftest(0, scratch) == -1          # refused: no limit given
    s = inputs.ModuleShape("after", "bf16", 1, 64, 8, 8, 2, 32, seed=3)
    t = inputs.module_inputs(s)
    util.assert_close(util.run_module(s, t), _ref(s, t), "bf16", "forward after the wait self-test")
    assert binding.msla_debug_wait_timeouts() == 0                     # the self-test does not touch the product kernels' flag


def test_no_kernel_wait_timed_out():
    """Every device-side wait in the library is bounded; none of the runs above may have hit its limit."""
    assert binding.msla_debug_wait_timeouts() == 0
