"""Sweep on Llama-3-8B layer shapes (d_model 4096, 32 q / 8 kv heads, head_dim 128): decode attention over
rank r x context T x batch, the LR precompute over agents N x rank r, and turn prefill over rank r x (S, T).  Seeded synthetic inputs generated
on the device; one JSON line per cell and a Markdown table at the end.

    python -m paper_2609_34054_b200.sweep [--decode-only | --precompute-only | --prefill-only] [--peak-gbs 6451.2] [--peak-tflops 1652.6]

Decode bytes per request do not depend on the number of agents (a request reads the base rows and its own
agent's LR rows), so the decode grid fixes N = 4; N enters through the precompute.  Small cells rotate over
several copies of the caches so that a launch never finds its data in L2 (the copies together exceed
126 MB); launches are timed back to back inside one CUDA graph with CUDA events.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import inputs as I
from .binding import Cache, Precc, layer_desc

RANKS = (8, 16, 32, 64)
AGENTS = (2, 4, 8, 16)
CONTEXTS = (1024, 8192, 32768, 131072)
BATCHES = (1, 32)
TURNS = ((512, 32768), (2048, 8192), (64, 65536))      # (new tokens S, context T)
L2_BYTES = 126e6


def _randn(shape, std, gen):
    return (torch.randn(shape, device="cuda", generator=gen) * std).to(torch.bfloat16)


def _graph_time_us(fn, per_graph: int, replays: int) -> float:
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for _ in range(per_graph):
            fn()
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(replays):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / (replays * per_graph) * 1e3


def decode_cell(px: Precc, r: int, B: int, T: int, seed: int = 0) -> dict:
    geo = I.c5_geometry(r, 4)
    desc = layer_desc(geo)
    gen = torch.Generator(device="cuda").manual_seed(seed)
    nb = B * (T // I.PAGE)
    per_tok = (2 * geo.kv_width + geo.rank_k + geo.rank_v) * 2
    cache_bytes = B * T * per_tok
    copies = 1 if cache_bytes > 2 * L2_BYTES else min(16, int(2 * L2_BYTES // cache_bytes) + 1)
    sig = 0.02 * geo.d_model ** 0.5                     # std of H W with H ~ N(0,1), W ~ N(0, 0.02)
    caches = []
    for _ in range(copies):
        caches.append(Cache.from_tensors(
            geo, _randn((nb, geo.n_kv, I.PAGE, geo.hd), sig, gen), _randn((nb, geo.n_kv, I.PAGE, geo.hd), sig, gen),
            _randn((geo.n_agents, nb, I.PAGE, r), 1.0, gen), _randn((geo.n_agents, nb, I.PAGE, r), 1.0, gen)))
    B_k = _randn((geo.n_agents, r, geo.kv_width), 0.02, gen)
    B_v = _randn((geo.n_agents, r, geo.kv_width), 0.02, gen)
    q = _randn((B, geo.n_q, geo.hd), 1.0, gen)
    out = torch.empty_like(q)
    aid = (torch.arange(B, device="cuda") % geo.n_agents).to(torch.int32)
    cl = torch.full((B,), T, dtype=torch.int32, device="cuda")
    first = (torch.arange(B, device="cuda") * (T // I.PAGE)).to(torch.int32)
    ws = px.decode_workspace(desc, B, T)
    it = [0]

    def run():
        c = caches[it[0] % copies]
        it[0] += 1
        px.lr_attend_decode(desc, q, aid, cl, T, B_k, B_v, c, out, ws, None, first)

    per_graph = max(copies, 4)
    us = _graph_time_us(run, per_graph, replays=max(2, int(2000 / max(1.0, cache_bytes / 6e6)) // per_graph + 1))
    byt = cache_bytes + B * 2 * geo.n_q * geo.hd * 2
    assert px.poll_status() == 0 and torch.isfinite(out.float()).all()
    return {"kind": "decode", "r": r, "B": B, "T": T, "us": us, "MB": byt / 1e6, "GBps": byt / us / 1e3, "copies": copies}


def precompute_cell(px: Precc, N: int, r: int, M: int = 32768, seed: int = 0) -> dict:
    geo = I.c5_geometry(r, N)
    desc = layer_desc(geo)
    gen = torch.Generator(device="cuda").manual_seed(seed)
    A_k = _randn((N, geo.d_model, r), geo.d_model ** -0.5, gen)
    A_v = _randn((N, geo.d_model, r), geo.d_model ** -0.5, gen)
    A = px.pack_adapters(geo, A_k, A_v)
    Hs = [_randn((M, geo.d_model), 1.0, gen) for _ in range(2)]     # 2 x 268 MB: never in L2
    nb = M // I.PAGE
    cache = Cache.__new__(Cache)                         # LR caches only: the precompute does not touch the base cache
    cache.geo, cache.n_blocks, cache.k_base, cache.v_base = geo, nb, None, None
    cache.lr_k = torch.empty((N, nb, I.PAGE, r), dtype=torch.bfloat16, device="cuda")
    cache.lr_v = torch.empty((N, nb, I.PAGE, r), dtype=torch.bfloat16, device="cuda")
    it = [0]

    def run():
        px.lr_precompute(desc, Hs[it[0] % 2], A, cache, 0)
        it[0] += 1

    us = _graph_time_us(run, 4, 5)
    n_out = N * 2 * r
    flops = 2.0 * M * geo.d_model * n_out
    byt = 2.0 * (M * geo.d_model + geo.d_model * n_out + M * n_out)
    assert px.poll_status() == 0
    return {"kind": "precompute", "N": N, "r": r, "n_out": n_out, "M": M, "us": us, "TFLOPs": flops / us / 1e6, "GBps": byt / us / 1e3}


def prefill_cell(px: Precc, r: int, S: int, T: int, seed: int = 0) -> dict:
    """r == 0: the adapter-free view (agent -1) of a rank-8 layer, i.e. the same kernel without LR columns."""
    agent = 1 if r else -1
    rr = r if r else 8
    geo = I.c5_geometry(rr, 4)
    desc = layer_desc(geo)
    c = I.direct_caches_device((T + S) // I.PAGE, geo, seed, "sweep.pf")
    cache = Cache.from_tensors(geo, c["k_base"], c["v_base"], c["lr_k"], c["lr_v"])
    gen = torch.Generator(device="cuda").manual_seed(seed)
    B_k = _randn((geo.n_agents, rr, geo.kv_width), 0.02, gen)
    B_v = _randn((geo.n_agents, rr, geo.kv_width), 0.02, gen)
    q = _randn((S, geo.n_q, geo.hd), 1.0, gen)
    out = torch.empty_like(q)
    us = _graph_time_us(lambda: px.lr_attend_prefill(desc, q, agent, T, B_k, B_v, cache, out), 2, 5)
    flops = 4.0 * geo.n_q * (geo.hd + r) * (S * T + S * (S + 1) / 2)      # scores + weighted sum over hd + r coordinates
    assert px.poll_status() == 0 and torch.isfinite(out.float()).all()
    return {"kind": "prefill", "r": r, "S": S, "T": T, "us": us, "TFLOPs": flops / us / 1e6}


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--decode-only", action="store_true")
    ap.add_argument("--precompute-only", action="store_true")
    ap.add_argument("--prefill-only", action="store_true")
    ap.add_argument("--peak-gbs", type=float, default=6451.2, help="measured copy bandwidth the fractions refer to")
    ap.add_argument("--peak-tflops", type=float, default=1652.6, help="measured dense bf16 burst rate")
    args = ap.parse_args(argv)
    px = Precc(0)
    dec, pre, pf = [], [], []
    if not (args.decode_only or args.precompute_only):
        for r in (0,) + tuple(RANKS):               # rank 0: the adapter-free view, for the LR overhead of the other rows
            for (S, T) in TURNS:
                c = prefill_cell(px, r, S, T)
                pf.append(c)
                print(json.dumps({k: (round(v, 2) if isinstance(v, float) else v) for k, v in c.items()}), flush=True)
                torch.cuda.empty_cache()
    if not (args.precompute_only or args.prefill_only):
        for r in RANKS:
            for B in BATCHES:
                for T in CONTEXTS:
                    c = decode_cell(px, r, B, T)
                    dec.append(c)
                    print(json.dumps({k: (round(v, 2) if isinstance(v, float) else v) for k, v in c.items()}), flush=True)
                    torch.cuda.empty_cache()
    if not (args.decode_only or args.prefill_only):
        for N in AGENTS:
            for r in RANKS:
                c = precompute_cell(px, N, r)
                pre.append(c)
                print(json.dumps({k: (round(v, 2) if isinstance(v, float) else v) for k, v in c.items()}), flush=True)
                torch.cuda.empty_cache()
    if dec:
        print("\n| r | B | " + " | ".join(f"T={T}" for T in CONTEXTS) + " |\n|---|---|" + "---|" * len(CONTEXTS))
        for r in RANKS:
            for B in BATCHES:
                cells = [c for c in dec if c["r"] == r and c["B"] == B]
                print(f"| {r} | {B} | " + " | ".join(
                    f"{c['us']:.1f} us, {c['GBps']:.0f} GB/s ({c['GBps'] / args.peak_gbs * 100:.0f} %)" for c in cells) + " |")
    if pf:
        print("\n| r | " + " | ".join(f"S={S}, T={T}" for (S, T) in TURNS) + " |\n|---|" + "---|" * len(TURNS))
        for r in (0,) + tuple(RANKS):
            cells = [c for c in pf if c["r"] == r]
            print(f"| {r} | " + " | ".join(f"{c['us']:.0f} us, {c['TFLOPs']:.0f} TF/s ({c['TFLOPs'] / args.peak_tflops * 100:.0f} %)" for c in cells) + " |")
    if pre:
        print("\n| N | " + " | ".join(f"r={r}" for r in RANKS) + " |\n|---|" + "---|" * len(RANKS))
        for N in AGENTS:
            cells = [c for c in pre if c["N"] == N]
            print(f"| {N} | " + " | ".join(
                f"{c['us']:.0f} us, {c['TFLOPs']:.0f} TF/s ({c['TFLOPs'] / args.peak_tflops * 100:.0f} %), {c['GBps']:.0f} GB/s" for c in cells) + " |")


if __name__ == "__main__":
    main()
