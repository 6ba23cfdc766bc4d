"""Decode attention of one layer spread over several GPUs (one process per GPU), two ways.

Context sharding: each rank keeps a contiguous,
page-aligned range of every request's tokens in its own caches, computes the split-KV record of its range
(``precc_lr_attend_decode_partial``), the records are all-gathered, and every rank merges them
(``precc_combine_partials``).  The exchange is ``(16 + 8 (hd + r_v)) * 4`` bytes per (request, kv head) and
rank, independent of the context length.  The paper is single-GPU; this is the natural way its path
shards when one GPU's HBM no longer holds a trajectory.

Head sharding: each rank keeps the base cache of ``n_kv / world`` kv heads (and the matching columns of B_k and
B_v); the LR caches, a few percent of the bytes, are replicated.  A rank runs the ordinary decode call with the
descriptor of its slice (no new kernel: the heads of a layer never interact inside attention) and the outputs
``[B][n_q / world][hd]`` are all-gathered into ``[B][n_q][hd]``.

Only the plumbing lives here (range and head planning, the collectives, buffer reuse); all arithmetic is in the
kernels behind the C ABI.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import torch
import torch.distributed as dist

from .binding import Cache, LayerDesc, Precc
from .binding import layer_desc
from .inputs import PAGE, Geometry


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


# --------------------------------------------------------------------------------------------- head sharding

def head_shard_geometry(geo: Geometry, world: int) -> Geometry:
    """Geometry of one rank's slice: n_kv / world kv heads with their query heads; everything else unchanged."""
    if geo.n_kv % world:
        raise ValueError(f"{geo.n_kv} kv heads do not divide over {world} ranks")
    return Geometry(d_model=geo.d_model, n_q=geo.n_q // world, n_kv=geo.n_kv // world, hd=geo.hd, n_agents=geo.n_agents,
                    rank_k=geo.rank_k, rank_v=geo.rank_v, alpha=geo.alpha)


def head_slice(rank: int, world: int, n_heads: int) -> slice:
    """The heads (kv or query) that rank `rank` owns: a contiguous run, in rank order."""
    per = n_heads // world
    return slice(rank * per, (rank + 1) * per)


def shard_cache_heads(cache: Cache, geo: Geometry, rank: int, world: int) -> Cache:
    """One rank's caches cut out of full-width ones (for tests and for loading a sharded layout from a replicated
    one): base K/V of its kv heads (copied: the head axis is not the outermost), LR caches as they are."""
    hs = head_slice(rank, world, geo.n_kv)
    return Cache.from_tensors(head_shard_geometry(geo, world), cache.k_base[:, hs].contiguous(), cache.v_base[:, hs].contiguous(),
                              cache.lr_k, cache.lr_v)


def shard_b_heads(B: Optional[torch.Tensor], geo: Geometry, rank: int, world: int) -> Optional[torch.Tensor]:
    """Columns of B_k / B_v ([n_agents][rank][n_kv*hd]) that belong to the rank's kv heads."""
    if B is None:
        return None
    hs = head_slice(rank, world, geo.n_kv)
    return B[:, :, hs.start * geo.hd:hs.stop * geo.hd].contiguous()


def gather_heads(local_out: torch.Tensor, group: Optional[dist.ProcessGroup] = None,
                 staging: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """local_out [B][n_q_local][hd] of every rank -> [B][world * n_q_local][hd], rank r's heads at [r * n_q_local, ...)."""
    world = dist.get_world_size(group)
    B, hq, hd = local_out.shape
    if staging is None:
        staging = torch.empty((world, B, hq, hd), dtype=local_out.dtype, device=local_out.device)
    dist.all_gather_into_tensor(staging.view(-1), local_out.contiguous().view(-1), group=group)
    res = staging.permute(1, 0, 2, 3).reshape(B, world * hq, hd)
    if out is None:
        return res.contiguous()
    out.copy_(res)
    return out


class HeadShardedDecoder:
    """Decode attention of one layer with the kv heads divided over the ranks of `group`."""

    def __init__(self, px: Precc, geo: Geometry, group: Optional[dist.ProcessGroup] = None, softmax_scale: float = 0.0):
        self.px, self.geo, self.group = px, geo, group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        self.local_geo = head_shard_geometry(geo, self.world)
        self.desc = layer_desc(self.local_geo, softmax_scale)
        self._local = self._staging = None

    def decode(self, q: torch.Tensor, agent_id: torch.Tensor, ctx_len: torch.Tensor, max_ctx: int, B_k_local, B_v_local,
               cache_local: Cache, out: torch.Tensor, workspace: torch.Tensor, block_table: Optional[torch.Tensor] = None,
               first_block: Optional[torch.Tensor] = None) -> torch.Tensor:
        """q [B][n_q][hd] (the same on every rank; the rank's heads are cut out here), caches and B matrices of the
        rank's heads; out [B][n_q][hd]: the full result on every rank."""
        hs = head_slice(self.rank, self.world, self.geo.n_q)
        q_local = q[:, hs].contiguous()
        if self._local is None or self._local.shape != q_local.shape:
            self._local = torch.empty_like(q_local)
            self._staging = torch.empty((self.world,) + tuple(q_local.shape), dtype=q.dtype, device=q.device)
        self.px.lr_attend_decode(self.desc, q_local, agent_id, ctx_len, max_ctx, B_k_local, B_v_local, cache_local, self._local,
                                 workspace, block_table, first_block)
        return gather_heads(self._local, self.group, self._staging, out)
