"""Head-sharded (tensor-parallel) prune step: each rank holds H / g query heads with their key / value heads.

The only exchange on the path is one all-reduce of the per-token scores (`sum n_vis` floats, a few KB:
latency bound on NVLink, nothing to fuse it with).  Each rank scores its own heads with `mvla_salience`
(the mean over ITS heads and the text queries), the all-reduce averages the ranks' means — equal shard
sizes, so that is the mean over all heads — and every rank then runs `mvla_select` on identical scores,
hence identical decisions, and `mvla_compact` on its own K / V shard and the replicated hidden rows.
Argument marshalling only; the arithmetic stays in the library's kernels and in the collective.
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist

from . import mvla


def head_shard(t: torch.Tensor, rank: int, world: int) -> torch.Tensor:
    """Rank's contiguous block of heads of a [rows, H, d] tensor, as its own contiguous tensor."""
    h = t.shape[1]
    assert h % world == 0, "heads must divide evenly over the ranks"
    n = h // world
    return t[:, rank * n:(rank + 1) * n].contiguous()


def average_over_ranks_(t: torch.Tensor, group=None) -> torch.Tensor:
    """In-place mean over the ranks of `group` (the result is bit-identical on every rank)."""
    if not dist.is_initialized() or dist.get_world_size(group) == 1:
        return t
    if dist.get_backend(group) == "nccl":
        dist.all_reduce(t, op=dist.ReduceOp.AVG, group=group)
    else:                                   # backends without an averaging reduction (CPU tests)
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
        t.div_(dist.get_world_size(group))
    return t


def prune_step_head_sharded(ctx: "mvla.PruneContext", prune_point: int, samples, mode: int,
                            q_local: torch.Tensor, k_local: torch.Tensor, v_local: Optional[torch.Tensor],
                            hidden: Optional[torch.Tensor], *, flags: int = 0, group=None,
                            out: Optional["mvla.StepOutputs"] = None, stream=None) -> "mvla.StepOutputs":
    """One prune point on a rank of a head-sharded group.  `ctx` was created with this rank's head counts
    (n_heads = H / g, n_kv_heads = H_kv / g); `q_local`, `k_local`, `v_local` are this rank's head blocks,
    `hidden` is replicated.  Returns the rank's outputs: kept positions (identical on every rank) and the
    compacted hidden rows and local K / V rows."""
    cs = samples if not isinstance(samples, (list, tuple)) else mvla.c_samples(samples)
    adaptive = mode == mvla.MODE_ADAPTIVE
    attn, l1 = ctx.salience(cs, q_local, k_local, hidden if adaptive else None, stream=stream)
    if stream is not None:
        with torch.cuda.stream(stream):
            average_over_ranks_(attn, group)
    else:
        average_over_ranks_(attn, group)
    if out is None:
        out = ctx.alloc_outputs(cs, hidden=hidden is not None, kv=v_local is not None, extras=True)
    ctx.select(prune_point, cs, mode, attn, l1, flags=flags, out=out, stream=stream)
    out.attn = attn
    total = sum(s.n_txt + s.n_2d + s.n_3d for s in cs)       # capacity; rows past out_offsets[batch] are not touched
    ctx.compact(cs, out.kept_idx, out.out_offsets, total, hidden, k_local, v_local, out_hidden=out.out_hidden,
                out_k=out.out_k, out_v=out.out_v, stream=stream)
    return out
