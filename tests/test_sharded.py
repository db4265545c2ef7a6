"""Token-sharded forward: one image cut into bands of rows over the ranks of a process group.

CPU: the split, and the whole host path (halo exchange, all-gather in band order) on gloo ranks with the band
arithmetic done by the oracle's step functions, against the oracle's forward of the whole image.
GPU: the library's two band calls, the ranks taken one after the other on one GPU, against the oracle."""
import os
import subprocess
import sys

import numpy as np
import pytest

from paper_2205_14756_b200 import sharded

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("H,world", [(16, 1), (16, 2), (17, 3), (64, 8), (9, 4), (8, 4)])
def test_bands_tile_the_image(H, world):
    rows = [sharded.band_rows(H, world, r) for r in range(world)]
    assert rows[0][0] == 0 and rows[-1][1] == H
    for (a0, a1), (b0, b1) in zip(rows, rows[1:]):
        assert a1 == b0                                   # no gap, no overlap
    sizes = [b - a for a, b in rows]
    assert min(sizes) >= sharded.HALO and max(sizes) - min(sizes) <= 1
    assert sizes == sorted(sizes, reverse=True)           # the longer bands first


def test_bands_too_thin_are_refused():
    with pytest.raises(ValueError):
        sharded.band_rows(7, 4, 0)                        # a band of one row could not give a two-row halo
    with pytest.raises(ValueError):
        sharded.band_rows(16, 2, 2)


def test_halos_are_absent_at_the_image_border():
    assert sharded.band_halos(1, 0) == (0, 0)
    assert sharded.band_halos(3, 0) == (0, 2)
    assert sharded.band_halos(3, 1) == (2, 2)
    assert sharded.band_halos(3, 2) == (2, 0)


# What a rank computes on its band, written with the oracle's step functions (fp64): the stand-in for the
# library's two band calls in the CPU test of the host path.
ORACLE_BAND = r"""
import numpy as np, torch
import oracle

class OracleBand:
    def __init__(self, t, heads, d, eps=1e-15):
        self.t, self.heads, self.d, self.eps = t, heads, d, eps
    def states(self, x_ext, top, bottom):
        t, h, d = self.t, self.heads, self.d
        x = x_ext.numpy().astype(np.float64)
        qkv = oracle.conv1x1(x, t["w_qkv"])
        agg = oracle.group1x1(oracle.dwconv(qkv, t["w_dw"]), t["w_pw"])
        ms = np.concatenate([qkv, agg], axis=1)[:, :, top:x.shape[2] - bottom]
        B, _, rows, W = ms.shape
        ms = ms.reshape(B, 2 * h, 3, d, rows * W)
        self.q, k, v = np.maximum(ms[:, :, 0], 0), np.maximum(ms[:, :, 1], 0), ms[:, :, 2]
        self.rows, self.W = rows, W
        st = np.empty((B, 2 * h, d, d + 1))
        st[..., :d] = np.einsum("bhan,bhcn->bhac", k, v)
        st[..., d] = k.sum(-1)
        return torch.from_numpy(st)
    def output(self, states, top, bottom):
        d = self.d
        S = np.zeros(states.shape[1:])
        for r in range(states.shape[0]):
            S = S + states[r].numpy()
        num = np.einsum("bhan,bhac->bhcn", self.q, S[..., :d])
        den = np.einsum("bhan,bha->bhn", self.q, S[..., d]) + self.eps
        att = (num / den[:, :, None]).reshape(num.shape[0], -1, self.rows, self.W)
        return torch.from_numpy(oracle.conv1x1(att, self.t["w_proj"]))
"""

WORKER = ORACLE_BAND + r"""
import os, sys
import torch.distributed as dist
from paper_2205_14756_b200 import inputs, sharded
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
s = inputs.ModuleShape("t", "f32", 2, 16, int(os.environ["MSLA_H"]), 6, 1, 16, seed=11)
t = inputs.module_inputs(s)
r0, r1 = sharded.band_rows(s.H, world, rank)
x_band = torch.from_numpy(np.ascontiguousarray(t["x"][:, :, r0:r1]))
out = sharded.sharded_forward(OracleBand(t, s.heads, s.d), x_band)
assert out.shape == (s.B, s.C_out, r1 - r0, s.W)
np.save(os.path.join(os.environ["MSLA_OUT"], f"out{rank}.npy"), out.numpy())
dist.barrier()
dist.destroy_process_group()
"""


@pytest.mark.parametrize("world,H", [(2, 9), (3, 8)])
def test_gloo_ranks_reproduce_the_whole_image(tmp_path, world, H):
    """Bands of 5+4 rows on two ranks; 3+3+2 on three (a middle band with both halos, bands as thin as the halo)."""
    import oracle
    from paper_2205_14756_b200 import inputs
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, PYTHONPATH=ROOT, MSLA_OUT=str(tmp_path), MSLA_H=str(H), OMP_NUM_THREADS="1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={world}", "--master-addr", "127.0.0.1",
           "--master-port", str(29741 + world), str(script)]
    r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-3000:]
    s = inputs.ModuleShape("t", "f32", 2, 16, H, 6, 1, 16, seed=11)
    t = inputs.module_inputs(s)
    ref = oracle.msla_forward(t["x"], t["w_qkv"], t["w_dw"], t["w_pw"], t["w_proj"], heads=s.heads, d=s.d)
    got = np.concatenate([np.load(tmp_path / f"out{r}.npy") for r in range(world)], axis=2)
    assert got.shape == ref.shape
    assert np.abs(got - ref).max() <= 1e-12 * np.abs(ref).max()


def test_a_band_without_its_halo_is_wrong():
    """The pin that the halo matters: the same arithmetic with the halo rows left out differs at the band edges only."""
    import oracle
    from paper_2205_14756_b200 import inputs
    ns = {}
    exec(ORACLE_BAND, ns)
    import torch
    s = inputs.ModuleShape("t", "f32", 1, 16, 8, 6, 1, 16, seed=3)
    t = inputs.module_inputs(s)
    x = torch.from_numpy(t["x"])
    ref = oracle.msla_forward(t["x"], t["w_qkv"], t["w_dw"], t["w_pw"], t["w_proj"], heads=s.heads, d=s.d)
    bands = [ns["OracleBand"](t, s.heads, s.d) for _ in range(2)]
    st = torch.stack([bands[0].states(x[:, :, :4], 0, 0), bands[1].states(x[:, :, 4:], 0, 0)])   # no halo exchanged
    got = np.concatenate([b.output(st, 0, 0).numpy() for b in bands], axis=2)
    assert np.abs(got - ref).max() > 1e-3 * np.abs(ref).max()
    st = torch.stack([bands[0].states(x[:, :, :6], 0, 2), bands[1].states(x[:, :, 2:], 2, 0)])   # with it
    got = np.concatenate([bands[0].output(st, 0, 2).numpy(), bands[1].output(st, 2, 0).numpy()], axis=2)
    assert np.abs(got - ref).max() <= 1e-12 * np.abs(ref).max()


# ----------------------------------------------------------------------------- GPU
def _run_bands(t, s, world, dtype):
    """The ranks of a `world`-way split taken one after the other on this GPU (no kernel waits on another)."""
    import torch
    td = torch.bfloat16 if dtype == "bf16" else torch.float32
    dev = {k: torch.from_numpy(v).to("cuda").to(td) for k, v in t.items()}
    comps, states, halos = [], [], []
    for r in range(world):
        r0, r1 = sharded.band_rows(s.H, world, r)
        top, bottom = sharded.band_halos(world, r)
        c = sharded.CudaBandCompute(dev["w_qkv"], dev["w_dw"], dev["w_pw"], dev["w_proj"], dev.get("b_proj"), heads=s.heads, d=s.d)
        states.append(c.states(dev["x"][:, :, r0 - top:r1 + bottom].contiguous(), top, bottom).clone())
        comps.append(c)
        halos.append((top, bottom))
    gathered = torch.stack(states)
    outs = [c.output(gathered, *h) for c, h in zip(comps, halos)]
    torch.cuda.synchronize()
    return torch.cat(outs, dim=2).float().cpu().numpy(), gathered


@pytest.mark.gpu
@pytest.mark.parametrize("world", [1, 2, 3])
def test_bands_on_the_gpu_match_the_oracle_bf16(world):
    import oracle
    import util
    from paper_2205_14756_b200 import binding, inputs
    s = inputs.ModuleShape("bands_bf16", "bf16", 2, 64, 50, 40, 2, 32, seed=21)     # 17+17+16 rows of 40 tokens
    t = inputs.module_inputs(s)
    ref = oracle.msla_forward(t["x"], t["w_qkv"], t["w_dw"], t["w_pw"], t["w_proj"], heads=s.heads, d=s.d)
    got, _ = _run_bands(t, s, world, "bf16")
    util.assert_close(got, ref, "bf16", block=util.MODULE_BLOCK)
    assert binding.msla_debug_wait_timeouts() == 0


@pytest.mark.gpu
def test_bands_on_the_gpu_match_the_oracle_f32_and_unfused_shapes():
    import oracle
    import util
    from paper_2205_14756_b200 import inputs
    s = inputs.ModuleShape("bands_f32", "f32", 1, 32, 12, 10, 2, 16, seed=22)
    t = inputs.module_inputs(s)
    ref = oracle.msla_forward(t["x"], t["w_qkv"], t["w_dw"], t["w_pw"], t["w_proj"], heads=s.heads, d=s.d)
    got, _ = _run_bands(t, s, 3, "f32")
    util.assert_close(got, ref, "f32")
    # bf16 with more output channels than the fused steps 4+5 take: apply kernel + projection GEMM on a band
    s = inputs.ModuleShape("bands_bf16_wide", "bf16", 1, 64, 24, 32, 2, 32, seed=23)
    t = inputs.module_inputs(s)
    t["w_proj"] = inputs.quantise(inputs.normal(23, 9, 264 * 128, 128 ** -0.5).reshape(264, 128), "bf16")
    ref = oracle.msla_forward(t["x"], t["w_qkv"], t["w_dw"], t["w_pw"], t["w_proj"], heads=s.heads, d=s.d)
    got, _ = _run_bands(t, s, 2, "bf16")
    util.assert_close(got, ref, "bf16", block=util.MODULE_BLOCK)


@pytest.mark.gpu
def test_band_states_sum_to_the_oracle_state():
    """Eq. 3's sums over tokens, band by band: the gathered states add up to ReLU(K)^T [V | 1] of the whole image."""
    import oracle
    from paper_2205_14756_b200 import inputs
    s = inputs.ModuleShape("bands_state", "bf16", 1, 64, 32, 32, 2, 32, seed=24)
    t = inputs.module_inputs(s)
    _, gathered = _run_bands(t, s, 2, "bf16")
    qkv = oracle.conv1x1(t["x"], t["w_qkv"])
    agg = oracle.group1x1(oracle.dwconv(qkv, t["w_dw"]), t["w_pw"])
    ms = np.concatenate([qkv, agg], axis=1).reshape(s.B, 2 * s.heads, 3, s.d, s.N)
    k, v = np.maximum(ms[:, :, 1], 0), ms[:, :, 2]
    ref = np.concatenate([np.einsum("bhan,bhcn->bhac", k, v), k.sum(-1)[..., None]], axis=-1)
    got = gathered.double().sum(0).cpu().numpy()
    assert np.linalg.norm(got - ref) <= 1e-2 * np.linalg.norm(ref)


@pytest.mark.gpu
def test_band_calls_reject_bad_halos():
    import torch
    from paper_2205_14756_b200 import binding
    bf = torch.bfloat16
    x = torch.zeros(1, 32, 4, 8, device="cuda", dtype=bf)
    w = [torch.zeros(n, device="cuda", dtype=bf) for n in (96 * 32, 96 * 25, 96 * 32, 32 * 64)]
    d0 = binding.make_desc(1, 32, 4, 8, 1, 32, 32, binding.MSLA_BF16)
    ws = torch.empty(binding.msla_forward_workspace_bytes(d0), dtype=torch.uint8, device="cuda")
    desc = binding.make_desc(1, 32, 4, 8, 1, 32, 32, binding.MSLA_BF16, workspace=ws)
    st = torch.zeros(1, 2, 32, 33, device="cuda")
    with pytest.raises(binding.MslaError):
        binding.msla_band_states(desc, x, binding.make_weights(*w), 2, 2, st)     # no row left
    with pytest.raises(binding.MslaError):
        binding.msla_band_states(desc, x, binding.make_weights(*w), -1, 0, st)
