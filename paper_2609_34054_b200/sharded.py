"""Context-sharded decode over several GPUs (one process per GPU): each rank keeps a contiguous,
page-aligned range of every request's tokens in its own caches, computes the split-KV record of its range
(``precc_lr_attend_decode_partial``), the records are all-gathered, and every rank merges them
(``precc_combine_partials``).  The exchange is ``(16 + 8 (hd + r_v)) * 4`` bytes per (request, kv head) and
rank, independent of the context length.  The paper is single-GPU; this is the natural way its path
shards when one GPU's HBM no longer holds a trajectory.

Only the plumbing lives here (range planning, the collective, buffer reuse); all arithmetic is in the two
kernels behind the C ABI.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import torch
import torch.distributed as dist

from .binding import Cache, LayerDesc, Precc
from .inputs import PAGE


def shard_ranges(ctx_len: Sequence[int], world: int, page: int = PAGE) -> List[List[Tuple[int, int]]]:
    """ranges[rank][request] = [start, end) token range held by that rank: whole pages, contiguous,
    in rank order, together covering [0, ctx) exactly once; a short request may leave late ranks empty."""
    out: List[List[Tuple[int, int]]] = [[] for _ in range(world)]
    for ctx in ctx_len:
        n_pages = (int(ctx) + page - 1) // page
        for r in range(world):
            p0, p1 = r * n_pages // world, (r + 1) * n_pages // world
            s, e = min(int(ctx), p0 * page), min(int(ctx), p1 * page)
            out[r].append((s, e))
    return out


def gather_records(local: torch.Tensor, group: Optional[dist.ProcessGroup] = None,
                   out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """All-gather of the per-rank record tensors: result[s] is rank s's ``local`` (any device the
    group's backend supports)."""
    world = dist.get_world_size(group)
    if out is None:
        out = torch.empty((world,) + tuple(local.shape), dtype=local.dtype, device=local.device)
    dist.all_gather_into_tensor(out.view(-1), local.contiguous().view(-1), group=group)
    return out


class ShardedDecoder:
    """Decode attention of one layer over context shards.  Buffers are allocated once per batch size."""

    def __init__(self, px: Precc, desc: LayerDesc, group: Optional[dist.ProcessGroup] = None):
        self.px, self.desc, self.group = px, desc, group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        self.rec_floats = px.partial_record_floats(desc)
        self._local = self._all = None

    def _buffers(self, B: int, device):
        shape = (B, self.desc.n_kv_heads, self.rec_floats)
        if self._local is None or self._local.shape != shape:
            self._local = torch.empty(shape, dtype=torch.float32, device=device)
            self._all = torch.empty((self.world,) + shape, dtype=torch.float32, device=device)
        return self._local, self._all

    def decode(self, q: torch.Tensor, agent_id: torch.Tensor, local_ctx_len: torch.Tensor, max_local_ctx: int, B_k, B_v,
               cache: Cache, out: torch.Tensor, workspace: torch.Tensor, block_table: Optional[torch.Tensor] = None,
               first_block: Optional[torch.Tensor] = None) -> torch.Tensor:
        """q, agent_id: the same on every rank; local_ctx_len: this rank's token counts; out: full result on every rank."""
        local, gathered = self._buffers(q.shape[0], q.device)
        self.px.lr_attend_decode_partial(self.desc, q, agent_id, local_ctx_len, max(1, max_local_ctx), B_k, cache, local,
                                         workspace, block_table, first_block)
        gather_records(local, self.group, gathered)
        self.px.combine_partials(self.desc, gathered, agent_id, B_v, out)
        return out
