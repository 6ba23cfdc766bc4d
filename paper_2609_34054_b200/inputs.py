"""Seeded synthetic inputs and workload shapes for the shared-base + low-rank KV path.

This module only draws random tensors and names shapes.  It holds none of the
method's arithmetic (no projections, no attention): both the CPU oracle's tests
and the CUDA path's tests/bench take their inputs from here so that they see
the same bit patterns.

All tensors are generated on the CPU with a per-tensor seeded ``torch.Generator``
(seed = f(workload seed, tensor name)) in fp32 and rounded once to bf16.
Conventions (paper notation, Section 2.1 / Eq. 1):

* ``H``      [T, d]                hidden states X (rows = tokens)
* ``W_k/W_v``[d, n_kv*hd]          frozen projections W0 (d_in x d_out)
* ``A_k/A_v``[N, d, r]             per-agent LoRA down-projections A_i
* ``B_k/B_v``[N, r, n_kv*hd]       per-agent LoRA up-projections B_i
* ``q``      [B, n_q, hd]          already-projected queries (the q projection is
                                   outside the KV path)
"""
from __future__ import annotations

import dataclasses
import zlib
from typing import Dict, Tuple

import torch

PAGE = 16  # tokens per cache block (the only supported page size)


@dataclasses.dataclass(frozen=True)
class Geometry:
    """One decoder layer's KV-path geometry."""

    d_model: int
    n_q: int
    n_kv: int
    hd: int
    n_agents: int
    rank_k: int
    rank_v: int
    alpha: float  # LoRA alpha; scale s = alpha / r (per projection)

    @property
    def group(self) -> int:
        return self.n_q // self.n_kv

    @property
    def kv_width(self) -> int:
        return self.n_kv * self.hd

    def scale(self, rank: int) -> float:
        return float(self.alpha) / rank if rank > 0 else 0.0

    @property
    def scale_k(self) -> float:
        return self.scale(self.rank_k)

    @property
    def scale_v(self) -> float:
        return self.scale(self.rank_v)


# The five workload families (shapes only).  C1 is the small parity case the
# oracle finishes in seconds; C2 is the benchmark workload.
C1 = Geometry(d_model=1024, n_q=8, n_kv=2, hd=128, n_agents=3, rank_k=8, rank_v=8, alpha=16.0)
C2 = Geometry(d_model=2048, n_q=32, n_kv=8, hd=64, n_agents=4, rank_k=16, rank_v=16, alpha=32.0)
C3 = Geometry(d_model=4096, n_q=32, n_kv=8, hd=128, n_agents=4, rank_k=32, rank_v=32, alpha=64.0)
C4 = Geometry(d_model=3584, n_q=28, n_kv=4, hd=128, n_agents=8, rank_k=16, rank_v=16, alpha=32.0)

C1_T = 256
C2_T, C2_LAYERS, C2_DECODE_STEPS = 8192, 16, 128
C3_T, C3_S, C3_LAYERS = 32768, 512, 32
C4_BATCH, C4_CTX_MIN, C4_CTX_MAX = 64, 4096, 32768


def c5_geometry(rank: int, n_agents: int) -> Geometry:
    """Sweep cell on Llama-3-8B layer shapes (alpha = 2r so that s = 2)."""
    return Geometry(d_model=4096, n_q=32, n_kv=8, hd=128, n_agents=n_agents,
                    rank_k=rank, rank_v=rank, alpha=2.0 * rank)


def _generator(seed: int, name: str) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed((zlib.crc32(name.encode()) * 1_000_003 + seed * 7_919 + 12_345) % (2**63 - 1))
    return g


def normal_bf16(shape: Tuple[int, ...], std: float, seed: int, name: str) -> torch.Tensor:
    """N(0, std^2) drawn in fp32 on the CPU, rounded once to bf16."""
    g = _generator(seed, name)
    x = torch.empty(shape, dtype=torch.float32)
    x.normal_(0.0, 1.0, generator=g)
    if std != 1.0:
        x.mul_(std)
    return x.to(torch.bfloat16)


def uniform_int(low: int, high_inclusive: int, n: int, seed: int, name: str) -> torch.Tensor:
    g = _generator(seed, name)
    return torch.randint(low, high_inclusive + 1, (n,), generator=g, dtype=torch.int32)


def permutation(n: int, seed: int, name: str) -> torch.Tensor:
    g = _generator(seed, name)
    return torch.randperm(n, generator=g).to(torch.int32)


def layer_weights(geo: Geometry, seed: int, tag: str = "L0") -> Dict[str, torch.Tensor]:
    """Frozen projections and all agents' adapters for one layer.

    W ~ N(0, 0.02^2); A ~ N(0, 1/d) (variance 1/d, so H.A has unit-variance
    entries); B ~ N(0, 0.02^2).
    """
    d, w, n = geo.d_model, geo.kv_width, geo.n_agents
    out = {
        "W_k": normal_bf16((d, w), 0.02, seed, f"{tag}.W_k"),
        "W_v": normal_bf16((d, w), 0.02, seed, f"{tag}.W_v"),
        "A_k": normal_bf16((n, d, geo.rank_k), d ** -0.5, seed, f"{tag}.A_k"),
        "A_v": normal_bf16((n, d, geo.rank_v), d ** -0.5, seed, f"{tag}.A_v"),
        "B_k": normal_bf16((n, geo.rank_k, w), 0.02, seed, f"{tag}.B_k"),
        "B_v": normal_bf16((n, geo.rank_v, w), 0.02, seed, f"{tag}.B_v"),
    }
    return out


def hidden_states(n_tokens: int, geo: Geometry, seed: int, tag: str = "L0.H") -> torch.Tensor:
    """Hidden states H ~ N(0,1), [n_tokens, d]."""
    return normal_bf16((n_tokens, geo.d_model), 1.0, seed, tag)


def queries(n_rows: int, geo: Geometry, seed: int, tag: str = "L0.q", gain: float = 1.0) -> torch.Tensor:
    """Already-projected queries q ~ N(0, gain^2), [n_rows, n_q, hd].

    ``gain`` > 1 gives the "peaked" variant: larger logits, so that the softmax
    has a few dominant tokens and outputs are O(0.1..1) even at long context.
    """
    return normal_bf16((n_rows, geo.n_q, geo.hd), gain, seed, tag)


def direct_caches(n_blocks: int, geo: Geometry, seed: int, tag: str = "cache") -> Dict[str, torch.Tensor]:
    """Cache contents drawn directly (serving-shaped timing runs).

    Base K/V ~ N(0, 0.02^2 d) (the distribution of H.W entries), LR ~ N(0,1)
    (the distribution of H.A entries).  Layouts are the library's HBM layouts:
    base ``[n_blocks, n_kv, PAGE, hd]``, LR ``[n_agents, n_blocks, PAGE, r]``.
    """
    sig = 0.02 * geo.d_model ** 0.5
    return {
        "k_base": normal_bf16((n_blocks, geo.n_kv, PAGE, geo.hd), sig, seed, f"{tag}.k_base"),
        "v_base": normal_bf16((n_blocks, geo.n_kv, PAGE, geo.hd), sig, seed, f"{tag}.v_base"),
        "lr_k": normal_bf16((geo.n_agents, n_blocks, PAGE, geo.rank_k), 1.0, seed, f"{tag}.lr_k"),
        "lr_v": normal_bf16((geo.n_agents, n_blocks, PAGE, geo.rank_v), 1.0, seed, f"{tag}.lr_v"),
    }


def direct_caches_device(n_blocks: int, geo: Geometry, seed: int, tag: str = "cache", device: str = "cuda") -> Dict[str, torch.Tensor]:
    """``direct_caches`` drawn on the device (large pools: seconds on the host, milliseconds there); same
    distributions and layouts, another stream of numbers.  Ranks of zero give no LR tensors."""
    g = torch.Generator(device=device)
    g.manual_seed((zlib.crc32(tag.encode()) * 1_000_003 + seed * 7_919 + 54_321) % (2**63 - 1))
    sig = 0.02 * geo.d_model ** 0.5

    def draw(shape, std):
        return (torch.randn(shape, device=device, generator=g) * std).to(torch.bfloat16)

    out = {"k_base": draw((n_blocks, geo.n_kv, PAGE, geo.hd), sig), "v_base": draw((n_blocks, geo.n_kv, PAGE, geo.hd), sig)}
    if geo.rank_k:
        out["lr_k"] = draw((geo.n_agents, n_blocks, PAGE, geo.rank_k), 1.0)
    if geo.rank_v:
        out["lr_v"] = draw((geo.n_agents, n_blocks, PAGE, geo.rank_v), 1.0)
    return out


def serving_batch(batch: int, ctx_min: int, ctx_max: int, n_agents: int, seed: int):
    """Agent ids uniform over the agents, context lengths uniform (inclusive)."""
    agent_id = uniform_int(0, n_agents - 1, batch, seed, "serve.agent_id")
    ctx_len = uniform_int(ctx_min, ctx_max, batch, seed, "serve.ctx_len")
    return agent_id, ctx_len


def block_tables(ctx_len: torch.Tensor, n_phys_blocks: int, seed: int) -> torch.Tensor:
    """Per-request block tables drawn from one seeded permutation of physical blocks.

    Request b owns ``ceil(ctx_len[b]/PAGE)`` distinct physical blocks; unused
    table entries hold -1.
    """
    need = [(int(c) + PAGE - 1) // PAGE for c in ctx_len.tolist()]
    total = sum(need)
    if total > n_phys_blocks:
        raise ValueError(f"need {total} blocks, pool has {n_phys_blocks}")
    perm = permutation(n_phys_blocks, seed, "serve.block_perm")
    table = torch.full((len(need), max(need) if need else 0), -1, dtype=torch.int32)
    at = 0
    for b, n in enumerate(need):
        table[b, :n] = perm[at:at + n]
        at += n
    return table


def rope_table(max_pos: int, hd: int, theta: float = 10000.0, device="cuda") -> torch.Tensor:
    """The position table that callers of the rotary-key entry points pass in: fp32 [max_pos][hd/2][2] =
    (cos, sin) of t * theta^(-2c/hd), angles evaluated in fp64 and rounded once."""
    inv = torch.pow(torch.tensor(theta, dtype=torch.float64), -torch.arange(hd // 2, dtype=torch.float64) * 2.0 / hd)
    ang = torch.arange(max_pos, dtype=torch.float64)[:, None] * inv[None, :]
    return torch.stack([torch.cos(ang), torch.sin(ang)], dim=-1).to(torch.float32).contiguous().to(device)
