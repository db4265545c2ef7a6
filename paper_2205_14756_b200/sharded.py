"""One image's module forward spread over the ranks of a process group, by bands of image rows.

The module is linear in the number of tokens (Section 3.1), so a single high-resolution image is the case worth
spreading over several GPUs.  Two things couple the bands: the 5x5 window of the multi-scale aggregation, which
reaches two rows into the neighbouring bands, and Eq. 3's two sums over all tokens (the d x (d+1) state of each
head).  So a forward is

    1. every rank sends its two top rows of x to the rank above and its two bottom rows to the rank below
       (point-to-point; the image border gets no halo: that is where the aggregation pads with zeros),
    2. steps 1-3 on the band with its halo (`msla_band_states`): the band's share of every head's state,
    3. one all-gather of the states (<= 68 KB per rank), band 0 first,
    4. the sum of the gathered states in band order and steps 4-5 on the band (`msla_band_output`).

Step 3 is an all-gather followed by a sum in a fixed order, not an all-reduce, so that every rank forms bit-identical
states whatever the collective's internal reduction order would have been.

This module holds the host logic only: the split, the halo exchange and the gather, over `torch.distributed`
(NCCL between GPUs; any backend works).  What runs on a band is behind `BandCompute`; `CudaBandCompute` is the
library's two C-ABI calls.
"""
from __future__ import annotations

from typing import List, Optional, Protocol, Tuple

import torch
import torch.distributed as dist

HALO = 2  # rows the 5x5 aggregation reaches beyond a band (Section 3.1: small-kernel depthwise convolution, 5x5)


def band_rows(H: int, world: int, rank: int) -> Tuple[int, int]:
    """Rows [r0, r1) of the image that `rank` owns: H rows dealt out as evenly as possible, the first H % world
    bands one row longer.  Every band must be at least as tall as the halo, so that a halo comes from the direct
    neighbour only."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError(f"rank {rank} of {world}")
    if H < HALO * world:
        raise ValueError(f"{H} rows cannot be cut into {world} bands of at least {HALO} rows")
    base, extra = divmod(H, world)
    r0 = rank * base + min(rank, extra)
    return r0, r0 + base + (1 if rank < extra else 0)


def band_halos(world: int, rank: int) -> Tuple[int, int]:
    """(rows above, rows below) that the band needs from its neighbours."""
    return (0 if rank == 0 else HALO), (0 if rank == world - 1 else HALO)


class BandCompute(Protocol):
    def states(self, x_ext: torch.Tensor, halo_top: int, halo_bottom: int) -> torch.Tensor:
        """x_ext [B, C, halo_top + rows + halo_bottom, W] -> fp32 [B, 2*heads, d, d+1], the band's share of Eq. 3's sums."""

    def output(self, states: torch.Tensor, halo_top: int, halo_bottom: int) -> torch.Tensor:
        """states [R, B, 2*heads, d, d+1], band 0 first -> out [B, C_out, rows, W] for the band of the last `states` call."""


def exchange_halo(x_band: torch.Tensor, rank: int, world: int, group=None) -> torch.Tensor:
    """x_band [B, C, rows, W] -> [B, C, halo_top + rows + halo_bottom, W] with the neighbours' edge rows attached."""
    top, bottom = band_halos(world, rank)
    if x_band.shape[2] < HALO and world > 1:
        raise ValueError("a band must have at least two rows")
    B, C, rows, W = x_band.shape
    x_ext = x_band.new_empty((B, C, top + rows + bottom, W))
    x_ext[:, :, top:top + rows] = x_band
    ops: List[dist.P2POp] = []
    recv_top = recv_bottom = None
    if top:      # the band above: gets my first rows, gives me its last rows
        send_up = x_band[:, :, :HALO].contiguous()
        recv_top = x_band.new_empty((B, C, HALO, W))
        ops += [dist.P2POp(dist.isend, send_up, _global_rank(rank - 1, group), group),
                dist.P2POp(dist.irecv, recv_top, _global_rank(rank - 1, group), group)]
    if bottom:   # the band below: gets my last rows, gives me its first rows
        send_down = x_band[:, :, rows - HALO:].contiguous()
        recv_bottom = x_band.new_empty((B, C, HALO, W))
        ops += [dist.P2POp(dist.isend, send_down, _global_rank(rank + 1, group), group),
                dist.P2POp(dist.irecv, recv_bottom, _global_rank(rank + 1, group), group)]
    if ops:
        for req in dist.batch_isend_irecv(ops):
            req.wait()
    if top:
        x_ext[:, :, :top] = recv_top
    if bottom:
        x_ext[:, :, top + rows:] = recv_bottom
    return x_ext


def _global_rank(group_rank: int, group) -> int:
    return group_rank if group is None else dist.get_global_rank(group, group_rank)


def gather_states(state: torch.Tensor, world: int, group=None) -> torch.Tensor:
    """[...] -> [world, ...]: every rank's state, band 0 first, the same bytes on every rank."""
    state = state.contiguous()
    out = state.new_empty((world,) + tuple(state.shape))
    if world == 1:
        out[0] = state
        return out
    dist.all_gather_into_tensor(out.view(-1), state.view(-1), group=group)
    return out


def sharded_forward(compute: BandCompute, x_band: torch.Tensor, rank: Optional[int] = None, world: Optional[int] = None,
                    group=None) -> torch.Tensor:
    """The module forward of the image whose rows band_rows(H, world, rank) this rank holds in x_band.
    Returns this rank's rows of the output, [B, C_out, rows, W]."""
    if world is None:
        world = dist.get_world_size(group) if dist.is_initialized() else 1
    if rank is None:
        rank = dist.get_rank(group) if dist.is_initialized() else 0
    top, bottom = band_halos(world, rank)
    x_ext = exchange_halo(x_band, rank, world, group) if world > 1 else x_band
    state = compute.states(x_ext, top, bottom)
    return compute.output(gather_states(state, world, group), top, bottom)


class CudaBandCompute:
    """`BandCompute` on the library's kernels: `msla_band_states` and `msla_band_output` through the C ABI.
    Buffers are sized at the first call and reused while the band's shape stays the same."""

    def __init__(self, w_qkv, w_dw, w_pw, w_proj, b_proj=None, *, heads: int, d: int, eps: float = 1e-15, stream=None):
        from . import binding  # fails loudly when the library has not been built
        self.b = binding
        self.tensors = (w_qkv, w_dw, w_pw, w_proj, b_proj)
        self.weights = binding.make_weights(w_qkv, w_dw, w_pw, w_proj, b_proj)
        self.heads, self.d, self.eps, self.stream = heads, d, eps, stream
        self.C_out = w_proj.shape[0]
        self.dtype = binding.MSLA_BF16 if w_qkv.dtype == torch.bfloat16 else binding.MSLA_F32
        self._shape = None

    def _prepare(self, x_ext: torch.Tensor):
        if self._shape == tuple(x_ext.shape):
            return
        B, C, H, W = x_ext.shape
        b = self.b
        d0 = b.make_desc(B, C, H, W, self.heads, self.d, self.C_out, self.dtype, eps=self.eps)
        self.ws = torch.empty(b.msla_forward_workspace_bytes(d0), dtype=torch.uint8, device=x_ext.device)
        self.desc = b.make_desc(B, C, H, W, self.heads, self.d, self.C_out, self.dtype, eps=self.eps, workspace=self.ws)
        self.state = torch.empty(B, 2 * self.heads, self.d, self.d + 1, dtype=torch.float32, device=x_ext.device)
        self._shape = tuple(x_ext.shape)

    def states(self, x_ext, halo_top, halo_bottom):
        x_ext = x_ext.contiguous()
        self._prepare(x_ext)
        self._x = x_ext  # kept alive until the kernels that read it have been enqueued behind the next call
        self.b.msla_band_states(self.desc, x_ext, self.weights, halo_top, halo_bottom, self.state, self.stream)
        return self.state

    def output(self, states, halo_top, halo_bottom):
        B, _, H, W = self._shape
        out = torch.empty(B, self.C_out, H - halo_top - halo_bottom, W, dtype=self._x.dtype, device=self._x.device)
        self.b.msla_band_output(self.desc, self.weights, halo_top, halo_bottom, states.contiguous(), states.shape[0], out,
                                self.stream)
        return out
