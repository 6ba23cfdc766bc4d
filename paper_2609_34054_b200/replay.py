"""Turn-loop replay of controlled multi-agent traces through the KV-path kernels (Sections 3.1-3.2, 4.1).

A trace is a list of agent turns over one growing shared trajectory: turn = (agent j, n_in tokens that
arrive as input, n_out tokens the agent decodes).  For every layer the replay issues exactly the KV-path
work a sharing policy implies and nothing else (no MLP, no query/output projections, random hidden
states and queries), so its times are the KV-path share of a turn, not model latencies:

  prelr       PreLRShared: new tokens -> base rows + LR rows of ALL agents (one fused projection), then
              attention of agent j over base + own LR cache; the same per decoded token.
  rebase_lp   ReBaseShared with lazy prefill: during the turn only agent j's LR rows are written; after
              the turn one contiguous adapter-free pass over the turn's n_in + n_out tokens rewrites the
              base rows from neutral hidden states, writes the other agents' LR rows and runs plain
              attention over the neutral base cache.  That pass is outside TTFT and inside total time.
  fullshared  one shared full-width cache, no agent-specific part (the lower bound the paper compares to).
  nonshared   every agent keeps a private full-width cache and first processes all tokens it has not
              seen (everything the other agents appended since its last turn).
  rebase_db   ReBaseShared with double batching: every step of the turn carries two sequences over the same
              tokens, the adapted one (agent j: adapted base rows and its LR rows in private blocks that its
              block table splices in after the shared context; the LR rows are also written at the tokens' shared
              slots, where they stay) and the adapter-free one (neutral base
              rows into the shared cache, the other agents' LR rows).  Prefill runs both; every decode step
              is ONE two-row projection (per-row agent masks) and ONE attention launch of two requests (agent j and the
              adapter-free view, each with its own block table).  Nothing is left to do after the turn.

TTFT of a turn = its prefill phase (projection + prefill attention over all layers); the trace's TTFT is
the sum over turns; throughput = trajectory tokens / total time (Section 4.1).  Decode steps are one
CUDA graph per turn (all layers, device-side context length and slot), replayed n_out times.

Run:  python -m paper_2609_34054_b200.replay --lengths 1900,17300,66400 --layers 32
"""
from __future__ import annotations

import argparse
import json
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence

import torch

from . import inputs as I
from .binding import Cache, Precc, layer_desc

POLICIES = ("prelr", "rebase_lp", "rebase_db", "fullshared", "nonshared")


@dataclass(frozen=True)
class Turn:
    agent: int
    n_in: int
    n_out: int


def three_agent_trace(total_tokens: int, cycles: int = 2, prompt: int = 256, short_in: int = 64, n_out: int = 64) -> List[Turn]:
    """plan -> action -> reflect cycles; the action agent receives the retrieved context, which is the
    part that varies with the trajectory length; every call decodes a short segment."""
    fixed = prompt + cycles * (3 * n_out + 2 * short_in)
    retrieved = max(16, (total_tokens - fixed) // cycles)
    turns: List[Turn] = []
    for c in range(cycles):
        turns.append(Turn(0, (prompt if c == 0 else 0) + short_in, n_out))    # plan
        turns.append(Turn(1, retrieved, n_out))                               # action: tool observation arrives
        turns.append(Turn(2, short_in, n_out))                                # reflect
    return turns


def round_robin_trace(n_agents: int, n_turns: int = 8, retrieved: int = 8192, n_out: int = 64) -> List[Turn]:
    """Fixed retrieved context per turn, agents in round-robin order (the agent-count experiment)."""
    return [Turn(t % n_agents, retrieved, n_out) for t in range(n_turns)]


def trace_tokens(turns: Sequence[Turn]) -> int:
    return sum(t.n_in + t.n_out for t in turns)


class Stack:
    """Per-layer device state: caches, packed weights, B factors (distinct per layer unless
    ``shared_weights``, so that a layer's weights are not found in L2 by the next one).  Hidden states are
    random and indexed by trajectory position: ``H_adpt[t]`` is what the layer sees for token t under the
    current agent's adapter, ``H_neut[t]`` what it sees in the adapter-free pass; they and the queries are
    shared by all layers (their values do not affect the work done, but they make the final cache contents
    and outputs a function of the trace that a test can recompute)."""

    def __init__(self, px: Precc, geo: I.Geometry, n_layers: int, max_tokens: int, max_rows: int, seed: int = 0,
                 shared_weights: bool = False, private_tokens: int = 0):
        self.px, self.geo, self.n_layers = px, geo, n_layers
        self.desc = layer_desc(geo)
        n_blocks = (max_tokens + I.PAGE - 1) // I.PAGE
        # blocks [0, shared_blocks) hold the shared trajectory; the rest are private to the adapted sequence
        # of the current turn (double batching only)
        self.shared_blocks = n_blocks
        self.private_blocks = (private_tokens + I.PAGE - 1) // I.PAGE + 1 if private_tokens else 0
        self.caches = [Cache(geo, n_blocks + self.private_blocks, fill=0.0) for _ in range(n_layers)]
        n_w = 1 if shared_weights else n_layers
        self.WA, self.W, self.B_k, self.B_v = [], [], [], []
        for l in range(n_w):
            w = {k: v.cuda() for k, v in I.layer_weights(geo, seed, f"L{l}").items()}
            self.WA.append(px.pack_turn_weights(geo, w["W_k"], w["W_v"], w["A_k"], w["A_v"]))
            self.W.append(px.pack_base_weights(geo, w["W_k"], w["W_v"]))
            self.B_k.append(w["B_k"] if geo.rank_k else None)
            self.B_v.append(w["B_v"] if geo.rank_v else None)
        rows = n_blocks * I.PAGE
        self.H_adpt = I.normal_bf16((rows, geo.d_model), 1.0, seed, "replay.H_adpt").cuda()
        self.H_neut = I.normal_bf16((rows, geo.d_model), 1.0, seed, "replay.H_neut").cuda()
        self.H2 = torch.empty((max(max_rows, 2), geo.d_model), dtype=torch.bfloat16, device="cuda")   # two sequences in one batch
        self.stage = torch.empty((2, geo.d_model), dtype=torch.bfloat16, device="cuda")              # rows of one decode step
        self.q = I.queries(max_rows, geo, seed, "replay.q").cuda()
        self.out = torch.empty_like(self.q)
        self.ws = px.decode_workspace(self.desc, 2, max_tokens)      # up to two requests per launch (double batching)
        self.max_tokens = max_tokens

    def w(self, l: int) -> int:
        return l if len(self.WA) > 1 else 0


def _project(st: Stack, l: int, H: torch.Tensor, start: int, mask: Optional[int], slot_map=None):
    """Rows H -> slots start.. (or slot_map).  mask None: base rows only; else base rows + LR rows of the agents in `mask`."""
    px, k = st.px, st.w(l)
    if mask is None or (st.geo.rank_k == 0 and st.geo.rank_v == 0):
        px.rebase_project(st.desc, H, st.W[k], st.caches[l], start, slot_map)
    else:
        px.turn_project(st.desc, H, st.WA[k], st.caches[l], start, slot_map, mask)


def _prefill_phase(st: Stack, H: torch.Tensor, T: int, agent: int, mask: Optional[int]):
    """The n = len(H) tokens at positions T.. : projection into the caches, then attention of `agent` over them."""
    n = H.shape[0]
    for l in range(st.n_layers):
        _project(st, l, H, T, mask)
        k = st.w(l)
        st.px.lr_attend_prefill(st.desc, st.q[:n], agent, T, st.B_k[k], st.B_v[k], st.caches[l], st.out[:n])


class _DecodeGraph:
    """One decode step over all layers with device-side position; replayed once per generated token.  The
    hidden state of the token at position t is H_src[t], fetched into a staging row by a gather inside the graph."""

    def __init__(self, st: Stack, H_src: torch.Tensor, agent: int, mask: Optional[int], ctx0: int, max_ctx: int):
        dev = st.q.device
        self.ctx = torch.tensor([ctx0], dtype=torch.int32, device=dev)        # tokens attended (incl. the new one)
        self.slot = torch.tensor([ctx0 - 1], dtype=torch.int32, device=dev)   # where the new token's rows go
        self.pos = torch.tensor([ctx0 - 1], dtype=torch.int64, device=dev)    # its trajectory position (gather index)
        self.agent = torch.tensor([agent], dtype=torch.int32, device=dev)
        self.first = torch.zeros(1, dtype=torch.int32, device=dev)

        def step():
            torch.index_select(H_src, 0, self.pos, out=st.stage[:1])
            for l in range(st.n_layers):
                _project(st, l, st.stage[:1], 0, mask, self.slot)
                k = st.w(l)
                st.px.lr_attend_decode(st.desc, st.q[:1], self.agent, self.ctx, max_ctx, st.B_k[k], st.B_v[k], st.caches[l],
                                       st.out[:1], st.ws, None, self.first)
            self.ctx.add_(1)
            self.slot.add_(1)
            self.pos.add_(1)

        step()                                       # warm-up outside capture (also the first real step)
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            step()

    def run(self, n: int):
        for _ in range(n):
            self.graph.replay()


def _timed(fn) -> float:
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    fn()
    e1.record()
    e1.synchronize()
    return e0.elapsed_time(e1)


def _adapted_table(st: Stack, P: int, n_c: int) -> torch.Tensor:
    """Block table of the adapted sequence: the shared blocks of the context, then private blocks from the
    page that holds position P on (that boundary page is private too, so that the two sequences never
    write the same page)."""
    n_ctx = P // I.PAGE
    n_priv = (P % I.PAGE + n_c + I.PAGE - 1) // I.PAGE
    if n_priv > st.private_blocks:
        raise ValueError("turn longer than the private region of the stack")
    return torch.cat([torch.arange(n_ctx, dtype=torch.int32), st.shared_blocks + torch.arange(n_priv, dtype=torch.int32)]).cuda()


def _replay_db(st: Stack, turns: Sequence[Turn]) -> Dict[str, float]:
    geo, px = st.geo, st.px
    all_mask = (1 << geo.n_agents) - 1
    ttft = decode_ms = 0.0
    P = 0
    dev = st.q.device
    for t in turns:
        j, n, n_c = t.agent, t.n_in, t.n_in + t.n_out
        others = all_mask & ~(1 << j)
        table_a = _adapted_table(st, P, n_c)
        priv0 = st.shared_blocks * I.PAGE + P % I.PAGE                  # slot of position P in the private region
        slots_a = (priv0 + torch.arange(n, dtype=torch.int32)).to(dev)

        slots_2n = torch.cat([slots_a, (P + torch.arange(n, dtype=torch.int32)).to(dev)])
        masks_2n = torch.tensor([1 << j] * n + [others] * n, dtype=torch.int64, device=dev)
        # agent j's own LR rows also go to the tokens' shared slots: they outlive the private blocks
        copy_2n = torch.cat([P + torch.arange(n, dtype=torch.int32), torch.full((n,), -1, dtype=torch.int32)]).to(dev)

        st.H2[:n].copy_(st.H_adpt[P:P + n])                           # the two sequences of the turn, one batch
        st.H2[n:2 * n].copy_(st.H_neut[P:P + n])

        def prefill_both():
            for l in range(st.n_layers):
                k = st.w(l)
                if P % I.PAGE:
                    # the page that holds position P is private to the adapted sequence: it starts as a copy of the
                    # shared page, so that the context rows in front of P are there too
                    c, src, dst = st.caches[l], P // I.PAGE, st.shared_blocks
                    c.k_base[dst].copy_(c.k_base[src]); c.v_base[dst].copy_(c.v_base[src])
                    if c.lr_k is not None:
                        c.lr_k[:, dst].copy_(c.lr_k[:, src])
                    if c.lr_v is not None:
                        c.lr_v[:, dst].copy_(c.lr_v[:, src])
                # adapted rows and adapter-free rows of the turn in ONE projection (per-row agent masks)
                px.turn_project_rows(st.desc, st.H2[:2 * n], st.WA[k], st.caches[l], slots_2n, masks_2n, copy_2n)
                px.lr_attend_prefill(st.desc, st.q[:n], j, P, st.B_k[k], st.B_v[k], st.caches[l], st.out[:n], table_a)
                px.lr_attend_prefill(st.desc, st.q[:n], -1, P, st.B_k[k], st.B_v[k], st.caches[l], st.out[:n])

        ttft += _timed(prefill_both)
        if t.n_out > 0:
            max_ctx = P + n_c
            width = (max_ctx + I.PAGE - 1) // I.PAGE
            table2 = torch.zeros((2, width), dtype=torch.int32)
            table2[0, :table_a.numel()] = table_a.cpu()[:width]
            table2[1] = torch.arange(width, dtype=torch.int32)
            table2 = table2.to(dev)
            ctx = torch.full((2,), P + n + 1, dtype=torch.int32, device=dev)
            agent2 = torch.tensor([j, -1], dtype=torch.int32, device=dev)
            slot2 = torch.tensor([priv0 + n, P + n], dtype=torch.int32, device=dev)
            mask2 = torch.tensor([1 << j, others], dtype=torch.int64, device=dev)
            pos = torch.tensor([P + n], dtype=torch.int64, device=dev)
            copy2 = torch.tensor([P + n, -1], dtype=torch.int32, device=dev)

            def step():
                torch.index_select(st.H_adpt, 0, pos, out=st.stage[:1])
                torch.index_select(st.H_neut, 0, pos, out=st.stage[1:2])
                for l in range(st.n_layers):
                    k = st.w(l)
                    px.turn_project_rows(st.desc, st.stage, st.WA[k], st.caches[l], slot2, mask2, copy2)
                    px.lr_attend_decode(st.desc, st.q[:2], agent2, ctx, max_ctx, st.B_k[k], st.B_v[k], st.caches[l], st.out[:2],
                                        st.ws, table2)
                ctx.add_(1); slot2.add_(1); pos.add_(1); copy2[:1].add_(1)

            step()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                step()
            decode_ms += _timed(lambda: [g.replay() for _ in range(t.n_out - 1)]) * t.n_out / max(1, t.n_out - 1)
        P += n_c
    total = ttft + decode_ms
    per_tok = 2 * geo.n_kv * geo.hd * 2 + (geo.rank_k + geo.rank_v) * 2 * geo.n_agents
    return {"policy": "rebase_db", "tokens": P, "turns": len(turns), "prefilled_tokens": 2 * sum(t.n_in for t in turns),
            "ttft_ms": ttft, "decode_ms": decode_ms, "rebase_ms": 0.0, "total_ms": total, "tokens_per_s": P / total * 1e3,
            "cache_gb": per_tok * P * st.n_layers / 1e9}


def replay(st: Stack, turns: Sequence[Turn], policy: str) -> Dict[str, float]:
    """Replays one trace under one policy; returns milliseconds and token counts."""
    if policy not in POLICIES:
        raise ValueError(f"policy must be one of {POLICIES}")
    if policy == "rebase_db":
        return _replay_db(st, turns)
    geo = st.geo
    all_mask = (1 << geo.n_agents) - 1
    ttft = decode_ms = rebase_ms = 0.0
    P = 0                                            # shared trajectory length so far
    seen = [0] * geo.n_agents                        # nonshared: tokens each agent's private cache covers
    prefilled = 0
    for t in turns:
        j = t.agent
        if policy == "nonshared":
            start, n_pref, agent, mask = seen[j], P - seen[j] + t.n_in, -1, None
        elif policy == "fullshared":
            start, n_pref, agent, mask = P, t.n_in, -1, None
        elif policy == "prelr":
            start, n_pref, agent, mask = P, t.n_in, j, all_mask
        else:
            start, n_pref, agent, mask = P, t.n_in, j, 1 << j
        prefilled += n_pref
        ttft += _timed(lambda: _prefill_phase(st, st.H_adpt[start:start + n_pref], start, agent, mask))
        ctx0 = P + t.n_in + 1
        if t.n_out > 0:
            g = _DecodeGraph(st, st.H_adpt, agent, mask, ctx0, P + t.n_in + t.n_out)     # runs the first decode step itself
            decode_ms += _timed(lambda: g.run(t.n_out - 1)) * t.n_out / max(1, t.n_out - 1)
        if policy == "rebase_lp":
            n_c = t.n_in + t.n_out
            rebase_ms += _timed(lambda: _prefill_phase(st, st.H_neut[P:P + n_c], P, -1, all_mask & ~(1 << j)))
        P += t.n_in + t.n_out
        seen[j] = P
    total = ttft + decode_ms + rebase_ms
    per_tok = 2 * geo.n_kv * geo.hd * 2
    lr_tok = (geo.rank_k + geo.rank_v) * 2 * geo.n_agents
    cache_bytes = {"nonshared": per_tok * geo.n_agents, "fullshared": per_tok}.get(policy, per_tok + lr_tok) * P * st.n_layers
    return {"policy": policy, "tokens": P, "turns": len(turns), "prefilled_tokens": prefilled, "ttft_ms": ttft,
            "decode_ms": decode_ms, "rebase_ms": rebase_ms, "total_ms": total, "tokens_per_s": P / total * 1e3,
            "cache_gb": cache_bytes / 1e9}


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--lengths", default="1900,3000,5000,9100,17300,33700,66400")
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--agents", type=int, default=3)
    ap.add_argument("--rank", type=int, default=32)
    ap.add_argument("--policies", default=",".join(POLICIES))
    ap.add_argument("--round-robin", type=int, default=0, help="instead of the length sweep: N agents, 8 turns x 8192 tokens")
    args = ap.parse_args(argv)
    px = Precc(0)
    n_agents = args.round_robin or args.agents
    geo = I.Geometry(d_model=4096, n_q=32, n_kv=8, hd=128, n_agents=n_agents, rank_k=args.rank, rank_v=args.rank,
                     alpha=2.0 * args.rank)
    traces = [round_robin_trace(n_agents)] if args.round_robin else [three_agent_trace(int(x)) for x in args.lengths.split(",")]
    for turns in traces:
        total = trace_tokens(turns)
        rows = max(total, 64, 2 * max(t.n_in for t in turns))   # nonshared prefills nearly the whole trajectory at once; double batching 2 x n_in rows
        st = Stack(px, geo, args.layers, total + I.PAGE, rows, private_tokens=max(t.n_in + t.n_out for t in turns) + I.PAGE)
        for pol in args.policies.split(","):
            r = replay(st, turns, pol)
            r.update({"layers": args.layers, "n_agents": n_agents, "rank": args.rank})
            print(json.dumps({k: (round(v, 3) if isinstance(v, float) else v) for k, v in r.items()}), flush=True)
        del st
        torch.cuda.empty_cache()
    if px.poll_status() != 0:
        raise SystemExit("device status flagged an error")


if __name__ == "__main__":
    main()
