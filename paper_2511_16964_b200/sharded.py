"""Logits + softmax with the vocabulary (the columns of W) split over the GPUs of a process group.

Host-side plumbing only: which columns a rank owns, and the one exchange of the chain - an
all-gather of each rank's per-row (max, sum exp) pairs, 8*M bytes per rank - between the two
library calls.  All arithmetic runs in the library's kernels (`pike_linear_softmax_shard_local`,
`pike_linear_softmax_shard_finish`); one process drives one GPU.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import binding as _b


def vocab_shard_range(N: int, rank: int, world: int, multiple: int = 8) -> tuple[int, int]:
    """Columns [lo, hi) of an N-column weight owned by `rank` of `world`.

    Contiguous, disjoint, covering [0, N); every boundary is a multiple of `multiple` (the kernels need
    slices whose width is a multiple of 8) and widths differ by at most `multiple`.  N itself must be a
    multiple of `multiple`; a rank may own nothing when there are more ranks than blocks."""
    if N < 0 or N % multiple != 0:
        raise ValueError(f"N = {N} is not a multiple of {multiple}")
    if not 0 <= rank < world:
        raise ValueError(f"rank {rank} outside [0, {world})")
    blocks = N // multiple
    base, extra = divmod(blocks, world)
    lo = rank * base + min(rank, extra)
    hi = lo + base + (1 if rank < extra else 0)
    return lo * multiple, hi * multiple


def gather_row_stats(row_stats: torch.Tensor, group=None) -> torch.Tensor:
    """All-gather of every rank's row_stats [M,2] into [world, M, 2], rank-major (the layout
    `pike_linear_softmax_shard_finish` reads).  Runs on row_stats' device with the group's backend."""
    world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
    if world == 1:
        return row_stats.reshape(1, row_stats.shape[0], 2)
    row_stats = row_stats.contiguous()
    all_stats = torch.empty((world,) + tuple(row_stats.shape), dtype=row_stats.dtype, device=row_stats.device)
    dist.all_gather(list(all_stats.unbind(0)), row_stats, group=group)
    return all_stats


def linear_softmax_vocab_sharded(x, w_shard, bias_shard=None, *, group=None, act="none", scale=1.0, w_is_nk=False,
                                 out=None, workspace=None, stream=None):
    """This rank's columns of softmax(scale*act(x @ W + bias)) where W's columns are split over the group.

    x [M,K] is the same on every rank; w_shard is this rank's column slice of W ([K,N_r], or [N_r,K]
    with w_is_nk).  Returns out [M,N_r] fp32; concatenating the ranks' results along the columns gives
    the softmax over the whole vocabulary."""
    out, stats = _b.pike_linear_softmax_shard_local(x, w_shard, bias_shard, act=act, scale=scale, w_is_nk=w_is_nk,
                                                    out=out, workspace=workspace, stream=stream)
    if stream is not None:
        # the collective runs on torch's current stream: order it after the first half, and the second
        # half after it
        torch.cuda.current_stream().wait_stream(stream)
    all_stats = gather_row_stats(stats, group)
    if stream is not None:
        stream.wait_stream(torch.cuda.current_stream())
    return _b.pike_linear_softmax_shard_finish(out, all_stats, stream=stream)
