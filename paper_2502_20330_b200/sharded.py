"""Context-sharded verify attention: the keys of every sequence are spread over the ranks of a
process group (one GPU each), every rank attends over its own keys, the fp32 partial results are
all-gathered (the path's one exchange step) and combined by their log-sum-exp on every rank.

Only plumbing lives here (shard bounds, the all-gather); the attention and the merge run in the
library's kernels.  The rows' own keys (the R = gamma + 1 newest) stay together on the last rank,
so that rank alone applies the causal stair; all other ranks run with ``all_keys_visible``.
"""
from __future__ import annotations

from typing import List, Optional, Tuple

import torch
import torch.distributed as dist

from . import binding as _b


def context_shard_bounds(ctx_lens, gamma: int, world: int) -> List[List[Tuple[int, int]]]:
    """bounds[rank][b] = (start, end) of the keys of sequence b that rank holds.

    The L - R context keys are cut into ``world`` nearly equal runs in order; the last rank also holds
    the R newest keys.  Every rank gets at least one key of every sequence, which needs L - R >= world - 1.
    """
    R = gamma + 1
    out: List[List[Tuple[int, int]]] = [[] for _ in range(world)]
    for L in (int(x) for x in ctx_lens):
        body = L - R
        if body < world - 1 or L < R:
            raise ValueError(f"a sequence of {L} keys cannot be sharded over {world} ranks with gamma={gamma}")
        for r in range(world):
            s, e = r * body // world, (r + 1) * body // world
            if r == world - 1:
                e = L
            if e <= s:
                raise ValueError(f"rank {r} would hold no key of a sequence of {L} keys")
            out[r].append((s, e))
    return out


def exchange_partials(o32: torch.Tensor, lse: torch.Tensor, group=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """All-gather of this rank's (normalised fp32 output, log-sum-exp) -> ([P, ...], [P, ...]) in rank order."""
    world = dist.get_world_size(group)
    o_parts = torch.empty((world,) + tuple(o32.shape), dtype=o32.dtype, device=o32.device)
    l_parts = torch.empty((world,) + tuple(lse.shape), dtype=lse.dtype, device=lse.device)
    # the receive slots are the rows of one tensor, so the merge reads the gathered partials in place
    dist.all_gather(list(o_parts.unbind(0)), o32.contiguous(), group=group)
    dist.all_gather(list(l_parts.unbind(0)), lse.contiguous(), group=group)
    return o_parts, l_parts


def local_partial(q, k_local, v_local, local_lens, gamma, workspace, holds_newest: bool,
                  params: Optional[_b.AttnParams] = None, stream=None):
    """This rank's partial: (out_f32 [B,R,Hq,D], lse [B,R,Hq]) over its own keys.  The results are
    allocated on torch's current stream: make ``stream`` that stream (or pass None) when calling this directly."""
    B, R, Hq, D = q.shape
    o32 = torch.empty(B, R, Hq, D, dtype=torch.float32, device=q.device)
    lse = torch.empty(B, R, Hq, dtype=torch.float32, device=q.device)
    scratch = torch.empty_like(q)
    p = _b.AttnParams(scale=params.scale if params else 0.0, num_ctas=params.num_ctas if params else 0,
                      lse_out=lse, out_f32=o32, all_keys_visible=not holds_newest)
    _b.rapid_verify_attention(q, k_local, v_local, local_lens, gamma, scratch, workspace, p, stream)
    return o32, lse


def sharded_verify_attention(q, k_local, v_local, local_lens, gamma, out, workspace, group=None,
                             params: Optional[_b.AttnParams] = None, stream=None) -> None:
    """out[B,R,Hq,D] (bf16) <- verify attention over the union of all ranks' keys.

    ``k_local`` / ``v_local`` [B,Hkv,Lloc,D] hold this rank's run of every sequence's keys and
    ``local_lens`` [B] their counts (see ``context_shard_bounds``); q is the same on every rank.

    Everything runs on ``stream`` (default: the current stream).  The collective and the temporaries
    follow torch's current stream, so the whole call is made with ``stream`` current: the kernels, the
    all-gather and the allocator then agree on one order.  The inputs must be ready on that stream.
    """
    if stream is None:
        stream = torch.cuda.current_stream(q.device)
    with torch.cuda.stream(stream):
        rank, world = dist.get_rank(group), dist.get_world_size(group)
        o32, lse = local_partial(q, k_local, v_local, local_lens, gamma, workspace, rank == world - 1, params, stream)
        o_parts, l_parts = exchange_partials(o32, lse, group)
        _b.rapid_merge_partials(o_parts, l_parts, out=out, stream=stream)
