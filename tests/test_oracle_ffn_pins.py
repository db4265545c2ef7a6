"""Pins of the oracle's FFN+DWConv functions (the second half of the building block, Section 3.1 / Fig. 2 left)
against things other than themselves: hand-worked values, closed forms, an independent composition (numpy einsum +
scipy correlate), locality and independence properties.  CPU only."""
import os

import numpy as np
import pytest
from scipy.signal import correlate2d

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _table(name):
    return np.loadtxt(os.path.join(GOLDEN, name), comments="#", ndmin=2)


def test_hardswish_values_by_hand():
    t = _table("hardswish_values.txt")
    got = oracle.bias_act(t[:, 0].reshape(1, 1, -1), None, "hardswish").ravel()
    assert np.allclose(got, t[:, 1], rtol=0, atol=1e-15)


def test_relu_identity_and_bias_per_channel():
    y = np.array([[[-1.0, 2.0], [3.0, -4.0]]])                       # [1, 2 channels, 2]
    assert np.array_equal(oracle.bias_act(y, None, "identity"), y)
    assert np.array_equal(oracle.bias_act(y, None, "relu"), np.maximum(y, 0))
    got = oracle.bias_act(y, np.array([10.0, -10.0]), "relu")         # the bias belongs to the channel, before the activation
    assert np.array_equal(got, np.array([[[9.0, 12.0], [0.0, 0.0]]]))


def test_ffn_worked_example():
    t = _table("ffn_worked_example.txt")
    x = t[:, 0].reshape(1, 1, 1, 3)
    w1 = np.array([[1.0], [-1.0]])
    b1 = np.array([0.0, 1.0])
    w_dw = np.zeros((2, 3, 3))
    w_dw[0, 1] = [1, 2, 0]
    w_dw[1, 1] = [0, 1, -1]
    w_dw[:, 0] = 7.0                                                  # rows above and below the image: must not matter
    w_dw[:, 2] = -7.0
    b_dw = np.array([0.0, 0.5])
    w2 = np.array([[1.0, 2.0]])
    b2 = np.array([-1.0])
    got = oracle.ffn_dwconv(x, w1, w_dw, w2, b1, b_dw, b2, act="relu")
    assert np.allclose(got.ravel(), t[:, 1], atol=1e-14)
    got = oracle.ffn_dwconv(x, w1, w_dw, w2, b1, b_dw, b2, act="relu", residual=True)
    assert np.allclose(got.ravel(), t[:, 2], atol=1e-14)


def _independent_ffn(x, w1, w_dw, w2, b1, b_dw, b2, act, residual):
    """The same definition from other building blocks: einsum for the linear layers, scipy for the depthwise filter."""
    def a(v):
        if act == "relu":
            return np.maximum(v, 0)
        if act == "hardswish":
            return v * np.clip(v + 3, 0, 6) / 6
        return v
    h = a(np.einsum("oc,bchw->bohw", w1, x) + b1[None, :, None, None])
    g = np.empty_like(h)
    for b in range(h.shape[0]):
        for c in range(h.shape[1]):
            g[b, c] = correlate2d(h[b, c], w_dw[c], mode="same", boundary="fill", fillvalue=0)
    g = a(g + b_dw[None, :, None, None])
    out = np.einsum("oc,bchw->bohw", w2, g) + b2[None, :, None, None]
    return out + x if residual else out


@pytest.mark.parametrize("act", ["identity", "relu", "hardswish"])
@pytest.mark.parametrize("shape", [(2, 3, 8, 5, 4, 3), (1, 4, 12, 1, 6, 4), (1, 2, 4, 3, 3, 5)])
def test_ffn_against_an_independent_composition(act, shape):
    B, C, Ch, H, W, C_out = shape
    rng = np.random.default_rng(hash((act,) + shape) % 2**32)
    x = rng.standard_normal((B, C, H, W)) * 2
    w1, w_dw, w2 = rng.standard_normal((Ch, C)), rng.standard_normal((Ch, 3, 3)), rng.standard_normal((C_out, Ch))
    b1, b_dw, b2 = rng.standard_normal(Ch), rng.standard_normal(Ch), rng.standard_normal(C_out)
    for residual in ([False, True] if C_out == C else [False]):
        ref = _independent_ffn(x, w1, w_dw, w2, b1, b_dw, b2, act, residual)
        got = oracle.ffn_dwconv(x, w1, w_dw, w2, b1, b_dw, b2, act=act, residual=residual)
        assert np.abs(got - ref).max() <= 1e-12 * max(1.0, np.abs(ref).max())


def test_ffn_reduces_to_the_identity():
    """Identity activation, w1 = [I; 0], centre-delta depthwise taps, w2 = [I 0]: FFN(x) = x, and 2x with the residual."""
    rng = np.random.default_rng(5)
    C, Ch = 3, 7
    x = rng.standard_normal((2, C, 4, 6))
    w1 = np.zeros((Ch, C)); w1[:C] = np.eye(C)
    w_dw = np.zeros((Ch, 3, 3)); w_dw[:, 1, 1] = 1.0
    w2 = np.zeros((C, Ch)); w2[:, :C] = np.eye(C)
    assert np.array_equal(oracle.ffn_dwconv(x, w1, w_dw, w2, act="identity"), x)
    assert np.array_equal(oracle.ffn_dwconv(x, w1, w_dw, w2, act="identity", residual=True), 2 * x)
    assert np.array_equal(oracle.ffn_dwconv(x, w1, w_dw, w2, act="relu"), np.maximum(x, 0))     # relu(relu(x)) = relu(x)


def test_zero_weights_leave_the_biases():
    x = np.ones((1, 2, 3, 3))
    z = lambda *s: np.zeros(s)
    b2 = np.array([1.5, -2.5])
    got = oracle.ffn_dwconv(x, z(4, 2), z(4, 3, 3), z(2, 4), b2=b2, act="hardswish")
    assert np.array_equal(got, np.broadcast_to(b2[None, :, None, None], got.shape))
    # a constant hidden bias through all-ones taps counts the taps inside the image: 4 / 6 / 9
    w2 = np.zeros((1, 4)); w2[0, 0] = 1.0
    got = oracle.ffn_dwconv(x, z(4, 2), np.ones((4, 3, 3)), w2, b1=np.array([1.0, 0, 0, 0]), act="identity")
    assert np.array_equal(got[0, 0], np.array([[4, 6, 4], [6, 9, 6], [4, 6, 4]], dtype=float))


def test_one_pixel_reaches_its_3x3_neighbourhood_only():
    rng = np.random.default_rng(9)
    C, Ch, H, W = 2, 6, 7, 8
    x = rng.standard_normal((1, C, H, W))
    w = (rng.standard_normal((Ch, C)), rng.standard_normal((Ch, 3, 3)), rng.standard_normal((C, Ch)))
    base = oracle.ffn_dwconv(x, *w, act="hardswish")
    x2 = x.copy(); x2[0, :, 3, 4] += 1.0
    diff = np.abs(oracle.ffn_dwconv(x2, *w, act="hardswish") - base).max(axis=(0, 1)) > 0
    expect = np.zeros((H, W), bool); expect[2:5, 3:6] = True
    assert np.array_equal(diff, expect)


def test_each_tap_is_the_right_shift():
    """Tap [dy][dx] of the inserted convolution reads pixel (row + dy - 1, col + dx - 1): orientation and sign."""
    x = np.zeros((1, 1, 5, 5)); x[0, 0, 2, 2] = 1.0
    one = np.ones((1, 1))
    for dy in range(3):
        for dx in range(3):
            w_dw = np.zeros((1, 3, 3)); w_dw[0, dy, dx] = 1.0
            got = oracle.ffn_dwconv(x, one, w_dw, one, act="identity")[0, 0]
            expect = np.zeros((5, 5)); expect[2 - (dy - 1), 2 - (dx - 1)] = 1.0
            assert np.array_equal(got, expect)


def test_hidden_channels_do_not_mix_in_the_depthwise_step():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((1, 2, 4, 4))
    w1, w_dw = rng.standard_normal((3, 2)), rng.standard_normal((3, 3, 3))
    w2 = np.eye(3)
    base = oracle.ffn_dwconv(x, w1, w_dw, w2, act="identity")
    w_dw2 = w_dw.copy(); w_dw2[1] *= 2.0
    got = oracle.ffn_dwconv(x, w1, w_dw2, w2, act="identity")
    assert np.array_equal(got[:, [0, 2]], base[:, [0, 2]]) and np.allclose(got[:, 1], 2 * base[:, 1], rtol=1e-15)


def test_residual_needs_equal_widths():
    with pytest.raises(ValueError):
        oracle.ffn_dwconv(np.zeros((1, 2, 2, 2)), np.zeros((4, 2)), np.zeros((4, 3, 3)), np.zeros((3, 4)), residual=True)


def test_block_is_the_two_residual_halves():
    """y = x + MSLA(x); out = y + FFN(y): checked against the pinned parts composed here, and with an FFN that is
    switched off (zero second layer) the block is x + MSLA(x)."""
    from paper_2205_14756_b200 import inputs
    s = inputs.ModuleShape("t", "f32", 1, 16, 5, 6, 1, 16, seed=4)
    t = inputs.module_inputs(s)
    rng = np.random.default_rng(4)
    f = {"w1": rng.standard_normal((32, 16)) / 4, "w_dw": rng.standard_normal((32, 3, 3)) / 3, "w2": rng.standard_normal((16, 32)) / 6,
         "b1": rng.standard_normal(32), "b2": rng.standard_normal(16)}
    m = oracle.msla_forward(t["x"], t["w_qkv"], t["w_dw"], t["w_pw"], t["w_proj"], heads=1, d=16)
    y = t["x"].astype(np.float64) + m
    ref = _independent_ffn(y, f["w1"], f["w_dw"], f["w2"], f["b1"], np.zeros(32), f["b2"], "hardswish", True)
    got = oracle.evit_block(t["x"], t, f, heads=1, d=16, act="hardswish")
    assert np.abs(got - ref).max() <= 1e-12 * np.abs(ref).max()
    off = dict(f, w2=np.zeros((16, 32)), b2=None)
    assert np.array_equal(oracle.evit_block(t["x"], t, off, heads=1, d=16), y)
