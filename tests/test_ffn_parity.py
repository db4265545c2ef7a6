"""FFN with a depthwise convolution and the whole building block (Section 3.1, Fig. 2 left) on the GPU, through the
C ABI, element by element against the fp64 oracle on the same seeded inputs."""
import numpy as np
import pytest

import oracle
import util
from paper_2205_14756_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _ref(t, act, residual):
    return oracle.ffn_dwconv(t["x"], t["w1"], t["w_dw"], t["w2"], t.get("b1"), t.get("b_dw"), t.get("b2"), act=act, residual=residual)


@pytest.mark.parametrize("act", ["identity", "relu", "hardswish"])
def test_ffn_f32_plain_kernels(act):
    s = inputs.FfnShape("ffn_f32", "f32", 2, 16, 7, 9, 40, 16, seed=31)
    t = inputs.ffn_inputs(s)
    util.assert_close(util.run_ffn(s, t, act, True), _ref(t, act, True), "f32", f"fp32 {act}")


# Tensor-core path (bf16, hidden width a multiple of 64): shapes with ragged token tiles (N not a multiple of 128 or
# 256), several weight blocks (C_hidden > 256), image edges in every position of the depthwise kernel's 32 x 8 tiles,
# C > 256 (first layer streams its weights), C_out not a multiple of 128.
@pytest.mark.parametrize("B,C,H,W,Ch,Cout,act,residual,biases", [
    (1, 64, 16, 16, 256, 64, "hardswish", True, True),
    (2, 64, 13, 20, 128, 64, "relu", True, True),
    (1, 32, 9, 33, 64, 40, "hardswish", False, True),
    (1, 128, 24, 40, 512, 128, "identity", True, False),
    (1, 320, 8, 24, 640, 320, "hardswish", True, True),
    (3, 64, 5, 3, 64, 64, "relu", False, False),
    (1, 64, 8, 12, 128, 64, "hardswish", True, True),       # W not a multiple of 8
    (2, 64, 13, 24, 192, 72, "hardswish", False, True),     # ragged tiles in both directions, C_out not a multiple of 32
    (1, 256, 40, 48, 1024, 256, "relu", True, True),
    (1, 64, 16, 16, 1088, 64, "hardswish", True, False),    # 17 hidden planes of 64 channels
])
def test_ffn_bf16_tensor_core_path(B, C, H, W, Ch, Cout, act, residual, biases):
    s = inputs.FfnShape("ffn_bf16", "bf16", B, C, H, W, Ch, Cout, seed=32)
    t = inputs.ffn_inputs(s, biases)
    got = util.run_ffn(s, t, act, residual)
    util.assert_close(got, _ref(t, act, residual), "bf16", f"{(B, C, H, W, Ch, Cout, act)}", block=util.MODULE_BLOCK)
    assert binding.msla_debug_wait_timeouts() == 0


def test_ffn_bf16_shapes_the_tensor_core_path_does_not_take():
    s = inputs.FfnShape("ffn_bf16_odd", "bf16", 1, 24, 6, 10, 72, 24, seed=33)     # hidden width not a multiple of 64
    t = inputs.ffn_inputs(s)
    util.assert_close(util.run_ffn(s, t, "hardswish", True), _ref(t, "hardswish", True), "bf16", "odd widths")


def test_ffn_at_the_bench_width_256x256():
    """C = 256, expansion 4, 65 536 tokens: the bench workload's channel widths on a quarter of its tokens."""
    s = inputs.FfnShape("ffn_c256_256x256", "bf16", 1, 256, 256, 256, 1024, 256, seed=34)
    t = inputs.ffn_inputs(s)
    util.assert_close(util.run_ffn(s, t, "hardswish", True), _ref(t, "hardswish", True), "bf16", "C=256 256x256", block=util.MODULE_BLOCK)
    assert binding.msla_debug_wait_timeouts() == 0


def test_ffn_at_the_bench_shape_on_sampled_pixels():
    """[1, 256, 512, 512], expansion 4: the shape and launch configuration the benchmark times.  The oracle computes
    sampled output pixels one by one from the 3x3 neighbourhood each depends on (image corners and edges included)."""
    s = inputs.FfnShape("ffn_c256_512x512", "bf16", 1, 256, 512, 512, 1024, 256, seed=36)
    t = inputs.ffn_inputs(s)
    got = util.run_ffn(s, t, "hardswish", True)
    rng = np.random.default_rng(36)
    pts = [(0, 0), (0, 511), (511, 0), (511, 511), (0, 200), (300, 511), (255, 256), (31, 32), (8, 7)]
    pts += [(int(a), int(b)) for a, b in zip(rng.integers(0, 512, 40), rng.integers(0, 512, 40))]
    ref, val = [], []
    for (y, x) in pts:
        y0, y1, x0, x1 = max(y - 1, 0), min(y + 2, 512), max(x - 1, 0), min(x + 2, 512)
        crop = dict(t, x=np.ascontiguousarray(t["x"][:, :, y0:y1, x0:x1]))
        ref.append(_ref(crop, "hardswish", True)[0, :, y - y0, x - x0])
        val.append(got[0, :, y, x])
    ref, val = np.stack(ref), np.stack(val)
    assert np.linalg.norm(val - ref) <= util.TOL_BF16_RELL2 * np.linalg.norm(ref)
    assert np.abs(val - ref).max() <= util.TOL_BF16_MAXABS * np.abs(ref).max()
    assert np.isfinite(got).all()
    assert binding.msla_debug_wait_timeouts() == 0


@pytest.mark.parametrize("dtype,B,C,H,W,heads,d,Ch", [("f32", 1, 32, 8, 8, 2, 16, 64), ("bf16", 2, 64, 16, 24, 2, 32, 256),
                                                      ("bf16", 1, 256, 64, 64, 8, 32, 1024)])
def test_block_matches_the_oracle(dtype, B, C, H, W, heads, d, Ch):
    s = inputs.ModuleShape("block", dtype, B, C, H, W, heads, d, seed=35)
    t = inputs.module_inputs(s)
    f = inputs.ffn_inputs(inputs.FfnShape("block_ffn", dtype, B, C, H, W, Ch, C, seed=35))
    ref = oracle.evit_block(t["x"], t, f, heads=heads, d=d, act="hardswish")
    got = util.run_block(s, t, f, Ch, "hardswish")
    util.assert_close(got, ref, dtype, "block", block=util.MODULE_BLOCK if dtype == "bf16" else None)


def test_ffn_rejects_bad_descriptors():
    import torch
    x = torch.zeros(1, 64, 8, 8, device="cuda", dtype=torch.bfloat16)
    good = dict(B=1, C=64, H=8, W=8, C_hidden=128, C_out=64, dtype=binding.MSLA_BF16)
    assert binding.msla_ffn_workspace_bytes(binding.make_ffn_desc(**good)) > 0
    assert binding.msla_ffn_workspace_bytes(binding.make_ffn_desc(**dict(good, C_out=72), residual=True)) == 0
    assert binding.msla_ffn_workspace_bytes(binding.make_ffn_desc(**good, dw_kernel=5)) == 0
    assert binding.msla_ffn_workspace_bytes(binding.make_ffn_desc(**good, act=7)) == 0
    desc = binding.make_ffn_desc(**good)                                           # no workspace given
    w = [torch.zeros(n, device="cuda", dtype=torch.bfloat16) for n in (128 * 64, 128 * 9, 64 * 128)]
    with pytest.raises(binding.MslaError):
        binding.msla_ffn_dwconv(desc, x, binding.make_ffn_weights(*w), torch.empty_like(x))
