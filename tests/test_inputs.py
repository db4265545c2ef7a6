"""Host logic of the seeded input generator (CPU only)."""
import numpy as np
import torch

from paper_2205_14756_b200 import inputs


def test_elements_depend_only_on_seed_stream_index():
    a = inputs.normal(3, 1, 1000)
    b = inputs.normal(3, 1, 5_000_000)          # crosses the internal chunk boundary
    assert np.array_equal(a, b[:1000])
    assert not np.array_equal(a, inputs.normal(3, 2, 1000))
    assert not np.array_equal(a, inputs.normal(4, 1, 1000))
    c = inputs.normal(3, 1, 4_200_000)
    assert np.array_equal(c, b[:4_200_000])


def test_normal_moments():
    a = inputs.normal(0, 0, 2_000_000)
    assert abs(a.mean()) < 3e-3 and abs(a.std() - 1.0) < 3e-3
    assert abs((a ** 3).mean()) < 1e-2 and abs((a ** 4).mean() - 3.0) < 3e-2
    assert np.all(np.isfinite(a))


def test_bf16_rounding_is_rne_and_matches_torch():
    a = inputs.normal(1, 0, 100_000).astype(np.float32)
    bits = inputs.round_to_bf16_bits(a)
    ref = torch.from_numpy(a).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, ref)
    # ties to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    tie = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8], dtype=np.float32)
    back = inputs.bf16_bits_to_f32(inputs.round_to_bf16_bits(tie))
    assert back[0] == 1.0 and back[1] == np.float32(1.0 + 2.0 ** -6)


def test_config_shapes_and_weight_scale():
    s = inputs.CONFIG1
    t = inputs.module_inputs(s)
    assert t["x"].shape == (1, 64, 16, 16) and t["w_qkv"].shape == (192, 64)
    assert t["w_dw"].shape == (192, 5, 5) and t["w_pw"].shape == (192, 16)
    assert t["w_proj"].shape == (64, 128)
    assert abs(t["w_qkv"].std() - 64 ** -0.5) < 0.01
    assert abs(t["w_dw"].std() - 0.2) < 0.01
    assert all(v.dtype == np.float32 for v in t.values())
    s3 = inputs.CONFIG3
    assert (s3.Cp, s3.N, 3 * s3.heads) == (192, 8192, 18)
    assert (inputs.CONFIG4.Cp, 3 * inputs.CONFIG4.heads) == (256, 24)
    assert [c.N for c in inputs.CONFIG5] == [1024, 4096, 16384, 65536, 262144]
    small = inputs.CoreShape("t", "bf16", 1, 2, 8, 32, seed=9)
    c = inputs.core_inputs(small)
    assert c["q"].shape == (1, 2, 8, 32)
    # already representable in bf16
    assert np.array_equal(inputs.quantise(c["k"], "bf16"), c["k"])
