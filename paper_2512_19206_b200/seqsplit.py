"""Sequence-split decode for contexts that do not fit one GPU: the tokens of every sequence are spread over the ranks'
caches in contiguous ranges, each rank attends over its own range with the library's kernels on its own memory, one
all-gather moves the per-head results (output and log-denominator, 516 bytes per head), and every rank merges them
with the log-sum-exp identity.  No kernel is ever handed another GPU's memory.

The exchange is the only collective of the method, and only in this variant; plain batches shard by sequence with no
data-path collective (replicas.py)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_ranges(n_tokens: int, world: int, residual_len: int):
    """Contiguous token ranges [t0, t1) per rank.  Inner boundaries are multiples of the residual length, so that
    every rank but the last holds whole windows; the last rank (the owner of the newest tokens) takes the rest."""
    windows = n_tokens // residual_len
    per = windows // world
    ranges, t0 = [], 0
    for r in range(world):
        t1 = n_tokens if r == world - 1 else t0 + per * residual_len
        ranges.append((t0, t1))
        t0 = t1
    return ranges


def gather_partials(out: torch.Tensor, lse: torch.Tensor, group=None):
    """All-gather of this rank's (out [..., 128], lse [...]) -> (o_parts [W, ..., 128], lse_parts [W, ...]), rank-major:
    the layout the merge takes.  NCCL for CUDA tensors, gloo for CPU tensors."""
    world = dist.get_world_size(group)
    o_parts = torch.empty((world,) + tuple(out.shape), dtype=out.dtype, device=out.device)
    lse_parts = torch.empty((world,) + tuple(lse.shape), dtype=lse.dtype, device=lse.device)
    dist.all_gather(list(o_parts.unbind(0)), out.contiguous(), group=group)
    dist.all_gather(list(lse_parts.unbind(0)), lse.contiguous(), group=group)
    return o_parts, lse_parts


def split_attention(out: torch.Tensor, lse: torch.Tensor, merge, group=None):
    """This rank's partial -> attention over the whole context (identical on every rank)."""
    o_parts, lse_parts = gather_partials(out, lse, group)
    return merge(o_parts, lse_parts)


class SeqSplitDecoder:
    """One rank of a sequence-split decode.  `cache` holds this rank's range of every sequence; the last rank owns the
    newest tokens and is the only one that appends during decoding."""

    def __init__(self, cache, group=None):
        from . import binding          # the CUDA library: there is no other merge on this path
        self._merge = binding.merge_partials
        self.cache = cache
        self.group = group
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)

    @property
    def owner(self) -> bool:
        return self.rank == self.world - 1

    def attention(self, layer, q, scale):
        out, lse = self.cache.decode_attention_partial(layer, q, scale)
        return split_attention(out, lse, self._merge, self.group)

    def step(self, layer, k, v, q, scale):
        """k, v [B,Hkv,1,128], q [B,Hq,1,128] bf16, the same on every rank: the owner appends the token, all attend."""
        if self.owner:
            self.cache.quantize_append(layer, k, v, q)
        return self.attention(layer, q[:, :, 0].contiguous(), scale)
