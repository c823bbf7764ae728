"""Column-parallel MeteoRA linear: the output rows (d_out) of one layer split over the ranks of a process group.

Eq. 2 is row-wise in W0 and in every B_i: y[:, o0:o1] = W0[o0:o1] x + sum_j w_j B_{i_j}[o0:o1] (A_{i_j} x).  A rank
that holds W0[o0:o1], B[:, o0:o1, :] and full copies of A and Wg therefore produces its slice of y with no exchange
step: the gate (Eq. 3) and the shrink are replicated (about 1.5 % of the work at 4096 -> 4096), so every rank takes
the same routing decisions wherever the gate logits are not within rounding of a tie: ranks whose shards differ in
width may run different launch plans, which add the slices of the stacked shrink in a different fp32 order, and a
token whose k-th and (k+1)-th logits agree to the last bits can then get its picks from different adapters on
different ranks.  A caller that needs bit-identical routing on every rank cuts equal shards (same plan, same
order of sums) or computes the routing once with meteora_gate_topk and compares.  Only a consumer that wants the whole y on every rank pays an all-gather, which is
optional here.  Shards are cut at multiples of 128 rows, the row tile of the kernels, so that no rank works on a
partial tile the others also touch.

This module is plumbing around `meteora_linear_forward`: which rows a rank owns, contiguous copies of its shard
(B's slice is strided in the full tensor) and the optional gather.
"""
from typing import List, Optional, Tuple

import torch
import torch.distributed as dist

ROW_TILE = 128


def shard_bounds(d_out: int, world: int, rank: int, multiple: int = ROW_TILE) -> Tuple[int, int]:
    """Rows [o0, o1) of rank `rank`: whole row tiles dealt as evenly as possible, the ragged last tile (d_out no
    multiple of `multiple`) going to the rank that owns the last tile; ranks beyond the tile count get nothing."""
    if world < 1 or not 0 <= rank < world or d_out < 0:
        raise ValueError("bad shard request")
    tiles = (d_out + multiple - 1) // multiple
    t0, t1 = tiles * rank // world, tiles * (rank + 1) // world
    return min(t0 * multiple, d_out), min(t1 * multiple, d_out)


def shard_module(W0: torch.Tensor, B: torch.Tensor, world: int, rank: int):
    """Contiguous copies of this rank's rows of W0[d_out, d_in] and B[N, d_out, r] (made once, at load time)."""
    o0, o1 = shard_bounds(W0.shape[0], world, rank)
    return W0[o0:o1].contiguous(), B[:, o0:o1, :].contiguous()


def gather_columns(y_local: torch.Tensor, d_out: int, group=None) -> torch.Tensor:
    """All-gather of the ranks' slices into y[T, d_out] (every rank gets the whole).  Slices may differ in width:
    each is padded to the widest for the collective and trimmed afterwards."""
    world = dist.get_world_size(group)
    widths = [b - a for a, b in (shard_bounds(d_out, world, r) for r in range(world))]
    wmax = max(widths)
    T = y_local.shape[0]
    if y_local.shape[1] != widths[dist.get_rank(group)]:
        raise ValueError("y_local does not have this rank's width")
    padded = y_local if y_local.shape[1] == wmax else torch.nn.functional.pad(y_local, (0, wmax - y_local.shape[1]))
    parts: List[torch.Tensor] = [torch.empty((T, wmax), dtype=y_local.dtype, device=y_local.device) for _ in range(world)]
    dist.all_gather(parts, padded.contiguous(), group=group)
    return torch.cat([p[:, :w] for p, w in zip(parts, widths)], dim=1)


def column_parallel_forward(x, W0_shard, A, B_shard, Wg, k: int, temperature: float = 1.0, d_out: Optional[int] = None,
                            group=None, gather: bool = False, workspace: Optional[torch.Tensor] = None,
                            forward=None):
    """This rank's y[:, o0:o1] from its shard; with `gather`, the whole y[T, d_out] on every rank.

    `forward` is the single-GPU call (default: the CUDA library's `meteora_linear_forward`); a rank whose shard is
    empty (more ranks than row tiles) returns a [T, 0] tensor and still takes part in the gather."""
    if forward is None:
        from . import binding
        forward = binding.meteora_linear_forward
    T = x.shape[0]
    if W0_shard.shape[0] == 0:
        y_local = torch.empty((T, 0), dtype=x.dtype, device=x.device)
    elif workspace is not None:
        y_local = forward(x, W0_shard, A, B_shard, Wg, k, temperature, workspace=workspace)
    else:
        y_local = forward(x, W0_shard, A, B_shard, Wg, k, temperature)
    if not gather:
        return y_local
    if d_out is None:
        raise ValueError("gather needs the full d_out")
    return gather_columns(y_local, d_out, group)
