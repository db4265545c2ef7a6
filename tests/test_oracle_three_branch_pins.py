"""Pins of the oracle's three-branch module (Section 3.1's multi-scale tokens with two aggregated branches) against
things other than itself: the pinned two-branch function, an independent composition of the pinned parts, and
structural properties.  CPU only."""
import numpy as np
import pytest
from scipy.signal import correlate2d

import oracle


def _weights(rng, C, heads, d, k1, k2, C_out, branches=3):
    Cp = heads * d
    return dict(w_qkv=rng.standard_normal((3 * Cp, C)) / C ** 0.5, w_dw=rng.standard_normal((3 * Cp, k1, k1)) / k1,
                w_pw=rng.standard_normal((3 * Cp, d)) / d ** 0.5, w_dw2=rng.standard_normal((3 * Cp, k2, k2)) / k2,
                w_pw2=rng.standard_normal((3 * Cp, d)) / d ** 0.5, w_proj=rng.standard_normal((C_out, branches * Cp)) / (branches * Cp) ** 0.5)


def _fwd3(x, w, heads, d, b=None):
    return oracle.msla_forward3(x, w["w_qkv"], w["w_dw"], w["w_pw"], w["w_dw2"], w["w_pw2"], w["w_proj"], b, heads=heads, d=d)


def _independent(x, w, heads, d, bias=None, eps=1e-15):
    """einsum for the projections, scipy for the depthwise filters, the explicit N x N form of Eq. 1 with Eq. 2's similarity."""
    B, C, H, W = x.shape
    Cp = heads * d
    qkv = np.einsum("oc,bchw->bohw", w["w_qkv"], x)
    branches = [qkv]
    for wd, wp in ((w["w_dw"], w["w_pw"]), (w["w_dw2"], w["w_pw2"])):
        dw = np.empty_like(qkv)
        for b in range(B):
            for c in range(3 * Cp):
                dw[b, c] = correlate2d(qkv[b, c], wd[c], mode="same", boundary="fill", fillvalue=0)
        g = dw.reshape(B, 3 * heads, d, H, W)
        branches.append(np.einsum("goi,bgihw->bgohw", wp.reshape(3 * heads, d, d), g).reshape(B, 3 * Cp, H, W))
    att = []
    for t in branches:
        t = t.reshape(B, heads, 3, d, H * W)
        q, k, v = np.maximum(t[:, :, 0], 0), np.maximum(t[:, :, 1], 0), t[:, :, 2]
        s = np.einsum("bhai,bhaj->bhij", q, k)                                   # similarity of query i and key j
        o = np.einsum("bhij,bhcj->bhci", s, v) / (s.sum(-1)[:, :, None, :] + eps)
        att.append(o.reshape(B, Cp, H, W))
    out = np.einsum("oc,bchw->bohw", w["w_proj"], np.concatenate(att, axis=1))
    return out if bias is None else out + bias[None, :, None, None]


@pytest.mark.parametrize("shape", [(1, 8, 5, 6, 1, 16, 5, 3, 8), (2, 6, 4, 7, 2, 2, 3, 5, 10), (1, 4, 3, 3, 1, 1, 5, 5, 4)])
def test_three_branches_against_an_independent_composition(shape):
    B, C, H, W, heads, d, k1, k2, C_out = shape
    rng = np.random.default_rng(sum(shape))
    x = rng.standard_normal((B, C, H, W))
    w = _weights(rng, C, heads, d, k1, k2, C_out)
    bias = rng.standard_normal(C_out)
    got = _fwd3(x, w, heads, d, bias)
    ref = _independent(x, w, heads, d, bias)
    assert np.abs(got - ref).max() <= 1e-10 * np.abs(ref).max()


def test_a_silent_third_branch_gives_the_two_branch_module():
    """Zero columns of w_proj for branch 2: the pinned two-branch function, bit for bit."""
    rng = np.random.default_rng(7)
    heads, d, C = 2, 16, 12
    x = rng.standard_normal((1, C, 6, 5))
    w = _weights(rng, C, heads, d, 5, 3, C)
    w["w_proj"][:, 2 * heads * d:] = 0.0
    two = oracle.msla_forward(x, w["w_qkv"], w["w_dw"], w["w_pw"], np.ascontiguousarray(w["w_proj"][:, :2 * heads * d]), heads=heads, d=d)
    assert np.array_equal(_fwd3(x, w, heads, d), two)


def test_branches_with_identity_aggregation_repeat_the_first():
    """Centre-delta taps and identity 1x1 in both aggregated branches: the three branches hold the same heads, so the
    output equals the one-branch attention projected with the three column blocks of w_proj added up."""
    rng = np.random.default_rng(8)
    heads, d, C = 1, 16, 8
    Cp = heads * d
    x = rng.standard_normal((1, C, 5, 5))
    w = _weights(rng, C, heads, d, 5, 3, C)
    for k, name in ((5, "w_dw"), (3, "w_dw2")):
        w[name][:] = 0.0
        w[name][:, k // 2, k // 2] = 1.0
    eye = np.tile(np.eye(d), (3 * heads, 1))
    w["w_pw"], w["w_pw2"] = eye.copy(), eye.copy()
    got = _fwd3(x, w, heads, d)
    summed = w["w_proj"][:, :Cp] + w["w_proj"][:, Cp:2 * Cp] + w["w_proj"][:, 2 * Cp:]
    two_cols = np.concatenate([summed, np.zeros_like(summed)], axis=1)
    ref = oracle.msla_forward(x, w["w_qkv"], np.pad(w["w_dw2"], ((0, 0), (1, 1), (1, 1))), w["w_pw"], two_cols, heads=heads, d=d)
    assert np.abs(got - ref).max() <= 1e-12 * np.abs(ref).max()


def test_head_order_is_branch_major():
    """An identity-like w_proj exposes the concat order: the third block of output channels carries branch 2 only."""
    rng = np.random.default_rng(9)
    heads, d, C = 1, 2, 4
    Cp = heads * d
    x = rng.standard_normal((1, C, 4, 4))
    w = _weights(rng, C, heads, d, 3, 5, 3 * Cp)
    w["w_proj"] = np.eye(3 * Cp)
    base = _fwd3(x, w, heads, d)
    w2 = dict(w, w_dw2=w["w_dw2"] * 2.0)                 # only branch 2 changes
    got = _fwd3(x, w2, heads, d)
    assert np.array_equal(got[:, :2 * Cp], base[:, :2 * Cp]) and not np.allclose(got[:, 2 * Cp:], base[:, 2 * Cp:])
    w1 = dict(w, w_pw=w["w_pw"] * -1.0)                  # only branch 1 changes
    got = _fwd3(x, w1, heads, d)
    assert np.array_equal(got[:, :Cp], base[:, :Cp]) and np.array_equal(got[:, 2 * Cp:], base[:, 2 * Cp:])
    assert not np.allclose(got[:, Cp:2 * Cp], base[:, Cp:2 * Cp])
