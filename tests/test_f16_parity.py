"""fp16 storage (the paper's deployment precision, Section 4.1's TensorRT fp16 runs) through the C ABI: every entry
point with dtype MSLA_F16, element by element against the fp64 oracle on inputs rounded to fp16.  The projections, the
aggregation, the attention core, the fused apply + output projection and the FFN (both linear layers, the depthwise
convolution, the residual epilogues) run on their tensor-core kernels instantiated for f16; shapes those do not take
run on the plain kernels.  fp32 accumulation and state throughout."""
import numpy as np
import pytest

import oracle
import util
from paper_2205_14756_b200 import binding, inputs

pytestmark = pytest.mark.gpu


# The attention core takes fp16 on its tensor-core kernels (mma.sync f16, fp32 accumulators and state; the state is
# scaled by a power of two near 1/N before it is cut into two fp16 pieces, which leaves Eq. 3's quotient unchanged):
# ragged sizes, config 2's shape, and the benchmark's token count, where unscaled sums (~1e5) would overflow fp16.
@pytest.mark.parametrize("B,heads,N,d", [(2, 3, 300, 32), (1, 4, 4096, 16), (1, 2, 7, 32), (8, 16, 4096, 32), (1, 2, 262144, 32),
                                         (1, 1, 262144, 16)])
def test_core_f16(B, heads, N, d):
    s = inputs.CoreShape("core_f16", "f16", B, heads, N, d, seed=51)
    t = inputs.core_inputs(s)
    got = util.run_core(t, "f16")
    util.assert_close(got, oracle.linattn_relu(t["q"], t["k"], t["v"]), "f16", "core fp16", block=util.CORE_BLOCK)


@pytest.mark.parametrize("B,C,H,W,heads,d,n_scales,k1", [(1, 64, 16, 16, 4, 16, 2, 5), (2, 64, 9, 20, 2, 32, 2, 3), (1, 96, 12, 12, 3, 32, 3, 5),
                                                         (1, 256, 64, 64, 8, 32, 2, 5), (2, 64, 24, 40, 2, 32, 2, 5), (1, 48, 11, 13, 3, 16, 2, 5),
                                                         (1, 192, 64, 128, 6, 32, 2, 5), (1, 320, 16, 24, 10, 32, 2, 5)])
def test_module_f16(B, C, H, W, heads, d, n_scales, k1):
    s = inputs.ModuleShape("module_f16", "f16", B, C, H, W, heads, d, seed=52, n_scales=n_scales, agg_kernel=k1)
    t = inputs.module_inputs(s)
    if n_scales == 3:
        ref = oracle.msla_forward3(t["x"], t["w_qkv"], t["w_dw"], t["w_pw"], t["w_dw2"], t["w_pw2"], t["w_proj"], heads=heads, d=d)
    else:
        ref = oracle.msla_forward(t["x"], t["w_qkv"], t["w_dw"], t["w_pw"], t["w_proj"], heads=heads, d=d)
    util.assert_close(util.run_module(s, t), ref, "f16", "module fp16", block=util.MODULE_BLOCK)


@pytest.mark.parametrize("side", [128, 512])
def test_many_tokens_do_not_overflow_f16(side):
    """The state sums over all tokens (16 384 and, at the benchmark's resolution, 262 144 per head: entries of the
    order of 10^4 and 10^5) and stays in fp32; what is stored in 16 bits is scaled by a power of two near 1 / N (the
    state folded into the projection weights, the key sums and eps alike), which leaves Eq. 3's quotient unchanged."""
    s = inputs.ModuleShape(f"module_f16_{side}x{side}", "f16", 1, 32, side, side, 1, 32, seed=53)
    t = inputs.module_inputs(s)
    ref = oracle.msla_forward(t["x"], t["w_qkv"], t["w_dw"], t["w_pw"], t["w_proj"], heads=1, d=32)
    util.assert_close(util.run_module(s, t), ref, "f16", f"fp16, {side * side} tokens", block=util.MODULE_BLOCK)


def test_ffn_and_block_f16():
    fs = inputs.FfnShape("ffn_f16", "f16", 2, 32, 9, 12, 96, 32, seed=54)
    ft = inputs.ffn_inputs(fs)
    ref = oracle.ffn_dwconv(ft["x"], ft["w1"], ft["w_dw"], ft["w2"], ft["b1"], ft["b_dw"], ft["b2"], act="hardswish", residual=True)
    util.assert_close(util.run_ffn(fs, ft, "hardswish", True), ref, "f16", "FFN fp16", block=util.MODULE_BLOCK)
    s = inputs.ModuleShape("block_f16", "f16", 1, 64, 12, 16, 2, 32, seed=55)
    t = inputs.module_inputs(s)
    f = inputs.ffn_inputs(inputs.FfnShape("block_ffn_f16", "f16", 1, 64, 12, 16, 128, 64, seed=55))
    ref = oracle.evit_block(t["x"], t, f, heads=2, d=32, act="hardswish")
    util.assert_close(util.run_block(s, t, f, 128, "hardswish"), ref, "f16", "block fp16", block=util.MODULE_BLOCK)


def test_f16_never_takes_the_fused_bf16_kernels():
    desc = binding.make_desc(1, 256, 64, 64, 8, 32, 256, binding.MSLA_F16)
    assert binding.msla_forward_workspace_bytes(desc) > 0 and binding.msla_forward_fuses_apply(desc) == 0


# fp16 FFN on the tensor-core kernels (C_hidden a multiple of 64, H*W a multiple of 8): ragged tiles in both
# directions, every activation, with and without the residual connection.
@pytest.mark.parametrize("B,C,H,W,Ch,act,residual", [(1, 64, 20, 36, 128, "hardswish", True), (2, 32, 9, 16, 64, "relu", False),
                                                     (1, 128, 33, 40, 256, "identity", True), (3, 64, 8, 8, 192, "hardswish", False)])
def test_ffn_f16_tensor_core_shapes(B, C, H, W, Ch, act, residual):
    fs = inputs.FfnShape("ffn_f16_tc", "f16", B, C, H, W, Ch, C, seed=56)
    ft = inputs.ffn_inputs(fs)
    ref = oracle.ffn_dwconv(ft["x"], ft["w1"], ft["w_dw"], ft["w2"], ft["b1"], ft["b_dw"], ft["b2"], act=act, residual=residual)
    util.assert_close(util.run_ffn(fs, ft, act, residual), ref, "f16", "FFN fp16 (tensor cores)", block=util.MODULE_BLOCK)
