#!/usr/bin/env python
"""Benchmark of the shared-base + LR KV-cache path on B200.

Workload (one "step" = one pass of the hot path over one synthetic trajectory, single stream):
a Llama-3.2-1B-shaped stack (16 layers, d_model 2048, 32 q / 8 kv heads, head_dim 64), 4 agents,
LoRA rank 16 on K and V (scale alpha/r = 2), shared trajectory of 8192 tokens:
  phase A  per layer: one fused projection of the 8192 hidden states (precc_turn_project): base K/V rows
           into the shared cache and the LR rows of all 4 agents, the hidden states read once;
  phase B  per agent, 128 decode steps, each one LR-reconstructed decode attention per layer
           (precc_lr_attend_decode, batch 1, context 8192): 4 x 128 x 16 = 8192 launches,
           replayed from one CUDA graph.
The metric is the decode attention's algorithmic HBM bytes per second: per launch
ctx*(2*n_kv*hd + r_k + r_v)*2 + q/out + the agent's B slices, summed over the launches of the step and
divided by the WHOLE step time (phase A included).  Inputs are resident in HBM for `value`; `e2e`
repeats the step with the hidden states and queries copied from pinned host memory and the outputs
copied back inside the timed region.

Beside the timed step the line carries, at one GPU, the other rows of the metric with their own roofline
records (`rooflines`): serving-shaped decode (64 requests, 2.4 GB of cache per launch), the new-turn prefill
and the LR precompute of a Llama-3-8B-shaped layer, each with the oracle timed on a stated sample.

`--gpus N` (N > 1) without a launcher starts N ranks itself (torch.distributed.run on 127.0.0.1): independent
replicas, one per GPU; the only collective is the max-reduction of the step time.
`--impl reference` times the CPU oracle (oracle/lrkv_oracle.py, numpy float64) on a bounded sample
of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "lr_kv_decode_attention_GBps"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes per launch of the profiled kernels (dram__bytes_read.sum + dram__bytes_write.sum of one ncu
# capture each), kept as data beside the profile summaries
NCU_TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_dram_traffic.json")


def ncu_traffic(key: str):
    """The recorded capture `key`: {"dram_bytes": per launch, "algorithmic_bytes": of the captured case, ...} or None."""
    try:
        with open(NCU_TRAFFIC_FILE) as f:
            return json.load(f).get(key)
    except Exception:
        return None


def decode_bytes_per_launch(geo, ctx: int, batch: int = 1, distinct_agents: int = 1) -> int:
    """Algorithmic HBM bytes of one decode-attention launch (LR rows counted once, not per kv head)."""
    per_tok = (2 * geo.kv_width + geo.rank_k + geo.rank_v) * 2
    qo = 2 * geo.n_q * geo.hd * 2
    bmat = (geo.rank_k + geo.rank_v) * geo.kv_width * 2
    table = (ctx + 15) // 16 * 4
    return batch * (ctx * per_tok + qo + table) + distinct_agents * bmat


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            with open(p) as f:
                return float(json.load(f)["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def reduce_max_ms(ms: float, device="cpu") -> float:
    """Max over ranks of a per-rank duration (identity when torch.distributed is not initialised)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(bytes_per_rank_step: float, steps: int, ms_max: float, world: int) -> float:
    """Replicas: every rank processes the same number of units; GB/s of the whole job."""
    return world * bytes_per_rank_step * steps / (ms_max * 1e-3) / 1e9


def measured_tensor_peaks():
    """Dense bf16 TFLOP/s (burst, sustained) from MEASURED_PEAKS.json, else the fallback figures."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            d = json.load(f)
        return {"bf16_tflops_burst": float(d["bf16_tflops"]), "bf16_tflops_sustained": float(d["bf16_tflops_sustained"]),
                "peak_kind": "measured"}
    except Exception:
        return {"bf16_tflops_burst": 1590.0, "bf16_tflops_sustained": 1400.0, "peak_kind": "fallback"}


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled every 200 ms while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc = None
        self.gpu_index = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------ CPU arm

def oracle_sample(n_requests: int, seed: int = 0):
    """Time the oracle on `n_requests` decode requests of layer 0 (all 8 kv heads, context 8192)."""
    import numpy as np
    from oracle import lrkv_oracle as O
    from paper_2609_34054_b200 import inputs as I
    geo, T = I.C2, I.C2_T
    w = {k: v.float().numpy() for k, v in I.layer_weights(geo, seed, "L0").items()}
    H = I.hidden_states(T, geo, seed, "L0.H").float().numpy()
    q = I.queries(n_requests, geo, seed, "L0.q").float().numpy()
    agent_id = [i % geo.n_agents for i in range(n_requests)]
    t0 = time.perf_counter()
    out = O.lr_decode_reference(q, agent_id, [T] * n_requests, H, w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"],
                                geo.scale_k, geo.scale_v, geo.n_kv)
    dt = time.perf_counter() - t0
    assert np.isfinite(out).all()
    return n_requests * decode_bytes_per_launch(geo, T) / dt / 1e9, dt


def cpu_threads() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    per_step = 8
    for _ in range(args.warmup):
        oracle_sample(per_step)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_sample(per_step)
    dt = time.perf_counter() - t0
    from paper_2609_34054_b200 import inputs as I
    val = args.steps * per_step * decode_bytes_per_launch(I.C2, I.C2_T) / dt / 1e9
    sample = f"{per_step} decode requests of layer 0 per step (all 8 kv heads, context 8192), merged-weight K/V + naive softmax in float64"
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "C2 llama-3.2-1B-shaped stack, T=8192, N=4 agents, r=16 (bounded sample)", "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0



# ------------------------------------------------------------------------- other rows of the metric

def _event_us(torch, fn, iters, warm=3):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters * 1e3


def extra_serving_decode(px, batch: int, ctx_min: int, ctx_max: int, seed: int = 0, cpu_seconds: float = 0.0):
    """C4-shaped decode: `batch` requests, agents uniform over 8, contexts uniform in [ctx_min, ctx_max],
    paged-16 caches with every logical block on its own physical block (a seeded CPU pool of 4096 blocks
    tiled over the physical pool: values repeat, addresses do not, so every launch streams from HBM)."""
    import torch
    from paper_2609_34054_b200 import inputs as I
    from paper_2609_34054_b200.binding import Cache, layer_desc
    geo = I.C4
    agent_id, ctx_len = I.serving_batch(batch, ctx_min, ctx_max, geo.n_agents, seed)
    need = [(int(t) + 15) // 16 for t in ctx_len]
    n_phys = sum(need)
    pool = I.direct_caches(4096, geo, seed, "C4.pool")
    reps = (n_phys + 4095) // 4096
    tile = lambda t, dim: torch.cat([t.cuda()] * reps, dim=dim).narrow(dim, 0, n_phys).contiguous()
    cache = Cache.from_tensors(geo, tile(pool["k_base"], 0), tile(pool["v_base"], 0), tile(pool["lr_k"], 1), tile(pool["lr_v"], 1))
    table = I.block_tables(ctx_len, n_phys, seed).cuda()
    w = I.layer_weights(geo, seed, "C4")
    desc = layer_desc(geo)
    q = I.queries(batch, geo, seed, "C4.q").cuda()
    out = torch.empty_like(q)
    mx = int(ctx_len.max())
    ws = px.decode_workspace(desc, batch, mx)
    Bk, Bv, aid, cl = w["B_k"].cuda(), w["B_v"].cuda(), agent_id.cuda(), ctx_len.cuda()
    us = _event_us(torch, lambda: px.lr_attend_decode(desc, q, aid, cl, mx, Bk, Bv, cache, out, ws, table), iters=10)
    per_tok = (2 * geo.kv_width + geo.rank_k + geo.rank_v) * 2
    byt = int(ctx_len.sum()) * per_tok + batch * 2 * geo.n_q * geo.hd * 2 + sum(need) * 4 + geo.n_agents * (geo.rank_k + geo.rank_v) * geo.kv_width * 2
    peak, kind = measured_peak()
    gbs = byt / us / 1e3
    # DRAM traffic of a full launch: the ncu capture is a 16-request reduction of this workload (same kernel, same
    # page layout; traffic is proportional to the tokens streamed), scaled by the algorithmic bytes
    cap = ncu_traffic("decode_ticket_c4_reduced")
    traffic = int(cap["dram_bytes"] * byt / cap["algorithmic_bytes"]) if cap else None
    res = {"workload": f"C4 serving decode: B={batch}, ctx~U[{ctx_min},{ctx_max}], 28q/4kv hd=128, N=8 r=16, paged-16",
           "kernel": "lr_attend_decode_kernel<128,16,16> (ticket)", "us_per_launch": us, "algorithmic_bytes": byt,
           "GBps": gbs, "frac_of_peak": gbs / peak, "peak_kind": kind, "frac_of_nominal_8TBps": gbs / NOMINAL_HBM_GBS,
           "l2_policy": f"{byt / 1e6:.0f} MB of distinct cache per launch >> 126 MB L2",
           "roofline": {"bound": "hbm", "kernel": "lr_attend_decode_kernel<128,16,16> (ticket)", "achieved": gbs, "peak": peak,
                        "peak_kind": kind, "unit": "GB/s", "frac": gbs / peak, "frac_of_nominal_8TBps": gbs / NOMINAL_HBM_GBS,
                        "traffic": traffic, "traffic_note": "ncu capture of a 16-request reduction, scaled by algorithmic bytes",
                        "algorithmic_bytes_per_launch": byt, "avg_launch_us": us}}
    if cpu_seconds > 0:
        res["cpu_baseline"] = _oracle_serving_sample(geo, q, agent_id, ctx_len, table, cache, w, per_tok, cpu_seconds, out)
    return res


def _oracle_serving_sample(geo, q, agent_id, ctx_len, table, cache, w, per_tok, budget_s, gpu_out):
    """The oracle (attention from cache contents, float64) on whole requests of the batch until `budget_s` seconds
    of CPU time are spent; also checks those requests' GPU outputs against it."""
    import numpy as np
    import torch
    from oracle import lrkv_oracle as O
    G = geo.group
    f64 = lambda t: t.detach().float().cpu().numpy().astype(np.float64)
    spent, done_bytes, n_req, worst = 0.0, 0, 0, 0.0
    got = f64(gpu_out)
    for b in range(q.shape[0]):
        t, a = int(ctx_len[b]), int(agent_id[b])
        blocks = table[b, :(t + 15) // 16].long()
        kb = f64(cache.k_base[blocks].permute(0, 2, 1, 3).reshape(-1, geo.kv_width))[:t]
        vb = f64(cache.v_base[blocks].permute(0, 2, 1, 3).reshape(-1, geo.kv_width))[:t]
        lk = f64(cache.lr_k[a][blocks].reshape(-1, geo.rank_k))[:t]
        lv = f64(cache.lr_v[a][blocks].reshape(-1, geo.rank_v))[:t]
        t0 = time.perf_counter()
        ref = O.attend_from_caches(f64(q[b]), kb, vb, lk, lv, f64(w["B_k"][a]), f64(w["B_v"][a]), geo.scale_k, geo.scale_v, geo.n_kv)
        spent += time.perf_counter() - t0
        worst = max(worst, float(np.abs(got[b] - ref).max()))
        done_bytes += t * per_tok + 2 * geo.n_q * geo.hd * 2
        n_req += 1
        if spent >= budget_s:
            break
    return {"value": done_bytes / spent / 1e9, "unit": "GB/s", "cores": cpu_threads(), "kind": "oracle",
            "sample": f"{n_req} whole requests of the batch (all kv heads; attention from cache contents in float64), {spent:.1f} s",
            "gpu_max_abs_err_on_sample": worst}


def extra_turn(px, T: int, S: int, seed: int = 0, cpu_seconds: float = 0.0):
    """C3-shaped turn of one layer: LR precompute over the context (throughput), then the turn itself
    (base append + LR precompute of the S new tokens + prefill attention) and the ReBase re-projection."""
    import torch
    from paper_2609_34054_b200 import inputs as I
    from paper_2609_34054_b200.binding import Cache, layer_desc
    geo = I.C3
    desc = layer_desc(geo)
    w = {k: v.cuda() for k, v in I.layer_weights(geo, seed, "C3").items()}
    A_packed = px.pack_adapters(geo, w["A_k"], w["A_v"])
    W_packed = px.pack_base_weights(geo, w["W_k"], w["W_v"])
    WA_packed = px.pack_turn_weights(geo, w["W_k"], w["W_v"], w["A_k"], w["A_v"])
    cache = Cache(geo, (T + S + 15) // 16)
    H_ctx = [I.hidden_states(T, geo, seed + i, "C3.H_ctx").cuda() for i in range(2)]     # 2 x 268 MB: rotates past L2
    H_new = [I.hidden_states(S, geo, seed + i, "C3.H_new_adpt").cuda() for i in range(32)]
    H_neut = [I.hidden_states(S, geo, seed + i, "C3.H_new_neut").cuda() for i in range(32)]
    q = I.queries(S, geo, seed, "C3.q").cuda()
    out = torch.empty_like(q)
    it = [0]

    def ctx_pre():
        px.lr_precompute(desc, H_ctx[it[0] % 2], A_packed, cache, 0); it[0] += 1

    def ctx_base():
        px.rebase_project(desc, H_ctx[it[0] % 2], W_packed, cache, 0); it[0] += 1
    us_pre = _event_us(torch, ctx_pre, 10)
    us_base = _event_us(torch, ctx_base, 6)
    n_lr = geo.n_agents * (geo.rank_k + geo.rank_v)
    fl_pre = 2.0 * T * geo.d_model * n_lr
    cur = 1

    def turn():
        h = H_new[it[0] % 32]; it[0] += 1
        px.turn_project(desc, h, WA_packed, cache, T)
        px.lr_attend_prefill(desc, q, cur, T, w["B_k"], w["B_v"], cache, out)

    def turn_proj():
        h = H_new[it[0] % 32]; it[0] += 1
        px.turn_project(desc, h, WA_packed, cache, T)

    def ctx_fused():
        px.turn_project(desc, H_ctx[it[0] % 2], WA_packed, cache, 0); it[0] += 1

    def rebase():
        h = H_neut[it[0] % 32]; it[0] += 1
        px.turn_project(desc, h, WA_packed, cache, T, None, ~(1 << cur))
    us_turn = _event_us(torch, turn, 5)
    us_tproj = _event_us(torch, turn_proj, 10)
    us_cfused = _event_us(torch, ctx_fused, 6)
    us_attn = _event_us(torch, lambda: px.lr_attend_prefill(desc, q, cur, T, w["B_k"], w["B_v"], cache, out), 5)
    us_reb = _event_us(torch, rebase, 10)
    fl_attn = 4.0 * geo.n_q * S * (geo.hd + (geo.rank_k + geo.rank_v) / 2) * (T + S / 2)
    # a short turn over the same context (a tool observation of 128 tokens): the projection takes the split-K
    # kernel and the prefill splits its context over clusters
    S2 = 128
    H_short = [I.hidden_states(S2, geo, seed + i, "C3.H_short").cuda() for i in range(32)]
    q2 = I.queries(S2, geo, seed, "C3.q_short").cuda()
    out2 = torch.empty_like(q2)

    def short_proj():
        h = H_short[it[0] % 32]; it[0] += 1
        px.turn_project(desc, h, WA_packed, cache, T)

    def short_turn():
        short_proj()
        px.lr_attend_prefill(desc, q2, cur, T, w["B_k"], w["B_v"], cache, out2)
    us_sproj = _event_us(torch, short_proj, 10)
    us_sattn = _event_us(torch, lambda: px.lr_attend_prefill(desc, q2, cur, T, w["B_k"], w["B_v"], cache, out2), 10)
    us_sturn = _event_us(torch, short_turn, 10)
    short = {"S": S2, "projection_us": us_sproj, "prefill_attention_us": us_sattn, "turn_us_per_layer": us_sturn,
             "turn_ttft_ms_32_layers": us_sturn * C3_LAYERS_FOR_TTFT / 1e3}
    # rotary keys (Appendix D.2) on the same turn: the per-tile kernel, and the scratch form (adapted rotary keys of the
    # sequence written once, then the tensor-memory kernel); the cache contents are taken as they are - only times matter here
    table = I.rope_table(T + S, geo.hd)
    scratch = torch.empty(px.prefill_rope_scratch_bytes(desc, T, S), dtype=torch.uint8, device="cuda")
    us_rope_tile = _event_us(torch, lambda: px.lr_attend_prefill_rope(desc, q, cur, T, w["B_k"], w["B_v"], table, cache, out), 2)
    us_rope_scr = _event_us(torch, lambda: px.lr_attend_prefill_rope_scratch(desc, q, cur, T, w["B_k"], w["B_v"], table, cache, out, scratch), 5)
    rotary = {"prefill_per_tile_kernel_us": us_rope_tile, "prefill_through_scratch_us": us_rope_scr,
              "scratch_bytes": scratch.numel(), "position_free_us": us_attn}
    del scratch
    # a turn length that leaves SMs idle (384 new tokens of 8 kv heads = 96 blocks on 148 SMs): prefill with a workspace
    # puts helper blocks on them (the 512-token turn, 128 blocks, is left on the plain launch by the planner)
    S3 = 384
    q3 = q[:S3].contiguous()
    out3 = torch.empty_like(q3)
    wsb = max(px.prefill_ws_bytes(desc, S3), 256)
    pws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    helper = {"S": S3, "workspace_bytes": wsb,
              "plain_us": _event_us(torch, lambda: px.lr_attend_prefill(desc, q3, cur, T, w["B_k"], w["B_v"], cache, out3), 5),
              "with_workspace_us": _event_us(torch, lambda: px.lr_attend_prefill_ws(desc, q3, cur, T, w["B_k"], w["B_v"], cache, out3, pws), 5)}
    del pws
    pk = measured_tensor_peaks()
    hbm, hbm_kind = measured_peak()
    tf_attn = fl_attn / us_attn / 1e6
    tf_pre = fl_pre / us_pre / 1e6
    pre_bytes = 2.0 * (T * geo.d_model + geo.d_model * n_lr + T * n_lr)
    attainable = min(pk["bf16_tflops_burst"], fl_pre / pre_bytes * hbm / 1e3)      # min(tensor, intensity x HBM), TFLOP/s
    cap_pf, cap_pre = ncu_traffic("prefill_tc_c3_layer"), ncu_traffic("proj_gemm_c3_context")
    res = {"workload": f"C3 turn, one layer: d=4096 32q/8kv hd=128, N=4 r=32, T={T}, S={S}",
           "short_turn": short,
           "lr_precompute_context": {"us": us_pre, "tflops": tf_pre, "n_out": n_lr, "GBps": pre_bytes / us_pre / 1e3,
                                     "attainable_tflops": attainable, "frac_of_attainable": tf_pre / attainable},
           "base_projection_context": {"us": us_base, "tflops": 2.0 * T * geo.d_model * 2 * geo.kv_width / us_base / 1e6},
           "fused_projection_context": {"us": us_cfused, "tflops": 2.0 * T * geo.d_model * (2 * geo.kv_width + n_lr) / us_cfused / 1e6},
           "turn_projection_us": us_tproj,
           "turn_us_per_layer": us_turn, "turn_ttft_ms_32_layers": us_turn * C3_LAYERS_FOR_TTFT / 1e3,
           "prefill_attention": {"us": us_attn, "tflops": tf_attn},
           "rotary_prefill": rotary,
           "prefill_helper_blocks": helper,
           "rebase_us_per_layer": us_reb, "peaks": pk,
           "roofline_prefill": {"bound": "tensor", "kernel": "lr_attend_prefill_tc_kernel<128,32,32>", "achieved": tf_attn,
                                "peak": pk["bf16_tflops_burst"], "peak_kind": pk["peak_kind"] + " (burst)", "unit": "TFLOP/s",
                                "frac": tf_attn / pk["bf16_tflops_burst"], "frac_of_sustained": tf_attn / pk["bf16_tflops_sustained"],
                                "traffic": cap_pf["dram_bytes"] if cap_pf else None, "algorithmic_flops_per_launch": fl_attn,
                                "avg_launch_us": us_attn},
           "roofline_precompute": {"bound": "tensor", "kernel": "proj_gemm_kernel (mode 0, n_out 256)", "achieved": tf_pre,
                                   "peak": pk["bf16_tflops_burst"], "peak_kind": pk["peak_kind"] + " (burst)", "unit": "TFLOP/s",
                                   "frac": tf_pre / pk["bf16_tflops_burst"], "attainable_min_tensor_hbm": attainable,
                                   "frac_of_attainable": tf_pre / attainable,
                                   "traffic": cap_pre["dram_bytes"] if cap_pre else None, "algorithmic_flops_per_launch": fl_pre,
                                   "algorithmic_bytes_per_launch": pre_bytes, "avg_launch_us": us_pre}}
    if cpu_seconds > 0:
        res["cpu_baseline"] = _oracle_turn_sample(px, geo, desc, w, A_packed, W_packed, T, S, cur, seed, cpu_seconds)
    return res


def _oracle_turn_sample(px, geo, desc, w, A_packed, W_packed, T, S, cur, seed, budget_s):
    """The oracle on a sample of the turn's prefill (merged-weight K/V of two kv heads over all T + S tokens, then
    naive attention for a few query rows), timed; the GPU result for the same rows is checked against it."""
    import numpy as np
    import torch
    from oracle import lrkv_oracle as O
    from paper_2609_34054_b200 import inputs as I
    from paper_2609_34054_b200.binding import Cache
    f64 = lambda t: t.detach().float().cpu().numpy().astype(np.float64)
    H = torch.cat([I.hidden_states(T, geo, seed, "C3.H_ctx"), I.hidden_states(S, geo, seed, "C3.H_new_adpt")])
    cache = Cache(geo, (T + S + 15) // 16)
    px.rebase_project(desc, H.cuda(), W_packed, cache, 0)
    px.lr_precompute(desc, H.cuda(), A_packed, cache, 0)
    q = I.queries(S, geo, seed, "C3.q", gain=4.0)
    out = torch.empty_like(q, device="cuda")
    px.lr_attend_prefill(desc, q.cuda(), cur, T, w["B_k"], w["B_v"], cache, out)
    torch.cuda.synchronize()
    heads = [0, 5]
    rows = [0, 1, 17, 255, 256, 510, 511]
    wn = {k: f64(v) for k, v in w.items()}
    t0 = time.perf_counter()
    ref = O.lr_prefill_reference(f64(q), cur, T, f64(H), wn["W_k"], wn["W_v"], wn["A_k"], wn["B_k"], wn["A_v"], wn["B_v"],
                                 geo.scale_k, geo.scale_v, geo.n_kv, heads=heads, rows=rows)
    dt = time.perf_counter() - t0
    got = f64(out)
    m = ~np.isnan(ref)
    err = float(np.abs(got[m] - ref[m]).max())
    G = geo.group
    # work of the sample in the units of the GPU row: attention flops of the sampled (row, head) pairs, plus the
    # projection of the sampled heads' K and V columns that the oracle needs first
    fl_attn = sum(4.0 * G * len(heads) * (geo.hd + (geo.rank_k + geo.rank_v) / 2) * (T + r + 1) for r in rows)
    fl_proj = 2.0 * (T + S) * geo.d_model * 2 * len(heads) * geo.hd
    return {"value": (fl_attn + fl_proj) / dt / 1e12, "unit": "TFLOP/s", "cores": cpu_threads(), "kind": "oracle",
            "sample": f"kv heads {heads} x query rows {rows} of the {S}-token turn over {T} tokens: merged-weight K/V projection "
                      f"of those heads ({fl_proj / 1e9:.0f} GFLOP) + naive attention ({fl_attn / 1e9:.2f} GFLOP) in float64, {dt:.1f} s",
            "gpu_max_abs_err_on_sample": err, "budget_s": budget_s}


C3_LAYERS_FOR_TTFT = 32

# ------------------------------------------------------------------------------------------ GPU arm

class Workload:
    def __init__(self, px, seed: int, layers: int, steps: int, T: int):
        import torch
        from paper_2609_34054_b200 import inputs as I
        from paper_2609_34054_b200.binding import Cache, layer_desc
        self.torch, self.px = torch, px
        geo = self.geo = I.C2
        self.layers, self.dsteps, self.T = layers, steps, T
        self.desc = layer_desc(geo)
        nb = (T + 15) // 16
        self.H_host, self.H, self.WA_packed, self.B_k, self.B_v, self.cache = [], [], [], [], [], []
        for l in range(layers):
            w = I.layer_weights(geo, seed, f"L{l}")
            dev = {k: v.cuda() for k, v in w.items()}
            self.WA_packed.append(px.pack_turn_weights(geo, dev["W_k"], dev["W_v"], dev["A_k"], dev["A_v"]))
            self.B_k.append(dev["B_k"]); self.B_v.append(dev["B_v"])
            h = I.hidden_states(T, geo, seed, f"L{l}.H").pin_memory()
            self.H_host.append(h)
            self.H.append(h.cuda())
            self.cache.append(Cache(geo, nb))
        # queries of every (agent, decode step, layer): [N, steps, layers, n_q, hd]
        self.q_host = I.normal_bf16((geo.n_agents, steps, layers, geo.n_q, geo.hd), 1.0, seed, "q").pin_memory()
        self.q = self.q_host.cuda()
        self.out = torch.zeros_like(self.q)
        self.out_host = torch.empty_like(self.q_host).pin_memory()
        self.agent_ids = [torch.full((1,), a, dtype=torch.int32, device="cuda") for a in range(geo.n_agents)]
        self.ctx = torch.full((1,), T, dtype=torch.int32, device="cuda")
        self.ws = px.decode_workspace(self.desc, 1, T)
        self.graph = None
        self.launches_a = layers
        self.launches_b = geo.n_agents * steps * layers

    def phase_a(self):
        px = self.px
        for l in range(self.layers):           # base rows and all agents' LR rows in one pass over the hidden states
            px.turn_project(self.desc, self.H[l], self.WA_packed[l], self.cache[l], 0)

    def phase_b_eager(self):
        px, geo = self.px, self.geo
        for a in range(geo.n_agents):
            for s in range(self.dsteps):
                for l in range(self.layers):
                    px.lr_attend_decode(self.desc, self.q[a, s, l:l + 1], self.agent_ids[a], self.ctx, self.T,
                                        self.B_k[l], self.B_v[l], self.cache[l], self.out[a, s, l:l + 1], self.ws)

    def capture(self):
        torch = self.torch
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            self.phase_a()
            px, geo = self.px, self.geo
            for l in range(self.layers):          # one eager launch per layer sets the kernel attributes
                px.lr_attend_decode(self.desc, self.q[0, 0, l:l + 1], self.agent_ids[0], self.ctx, self.T,
                                    self.B_k[l], self.B_v[l], self.cache[l], self.out[0, 0, l:l + 1], self.ws)
        torch.cuda.current_stream().wait_stream(s)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self.phase_b_eager()
        self.graph = g

    def phase_b(self):
        if self.graph is not None:
            self.graph.replay()
        else:
            self.phase_b_eager()

    def step(self):
        self.phase_a()
        self.phase_b()

    def step_host(self):
        """The same step with inputs arriving from pinned host memory and outputs returned to it."""
        for l in range(self.layers):
            self.H[l].copy_(self.H_host[l], non_blocking=True)
        self.q.copy_(self.q_host, non_blocking=True)
        self.step()
        self.out_host.copy_(self.out, non_blocking=True)

    def run_host_pipelined(self, steps: int):
        """`steps` steps whose inputs arrive from pinned host memory and whose outputs return to it, with the copies on
        a second stream: the inputs of step i + 1 are uploaded (into the other of two device buffer sets) while step i
        computes, and the outputs of step i go back while step i + 1 projects.  Every step still uploads all of its
        inputs and downloads all of its outputs; only the first upload and the last download are not overlapped."""
        torch = self.torch
        cur = torch.cuda.current_stream()
        if not hasattr(self, "_cs"):
            self._cs = torch.cuda.Stream()
            self._H2 = [self.H, [torch.empty_like(h) for h in self.H]]
            self._q2 = [torch.empty_like(self.q), torch.empty_like(self.q)]
        cs = self._cs
        ready = [torch.cuda.Event(), torch.cuda.Event()]
        done = [None, None]
        d2h_done = None

        def upload(slot):
            with torch.cuda.stream(cs):
                if done[slot] is not None:
                    cs.wait_event(done[slot])           # the compute that last read this buffer set has finished
                for l in range(self.layers):
                    self._H2[slot][l].copy_(self.H_host[l], non_blocking=True)
                self._q2[slot].copy_(self.q_host, non_blocking=True)
                ready[slot].record(cs)

        cs.wait_stream(cur)
        upload(0)
        for i in range(steps):
            slot = i & 1
            cur.wait_event(ready[slot])
            if i + 1 < steps:
                upload(slot ^ 1)
            px = self.px
            for l in range(self.layers):
                px.turn_project(self.desc, self._H2[slot][l], self.WA_packed[l], self.cache[l], 0)
            if d2h_done is not None:
                cur.wait_event(d2h_done)                # the previous outputs have left `out`
            self.q.copy_(self._q2[slot], non_blocking=True)   # the decode graph reads q at a fixed address
            self.phase_b()
            done[slot] = torch.cuda.Event()
            done[slot].record(cur)
            with torch.cuda.stream(cs):
                cs.wait_event(done[slot])
                self.out_host.copy_(self.out, non_blocking=True)
                d2h_done = torch.cuda.Event()
                d2h_done.record(cs)
        cur.wait_stream(cs)

    def h2d_bytes(self):
        return sum(h.numel() * 2 for h in self.H_host) + self.q_host.numel() * 2

    def d2h_bytes(self):
        return self.out_host.numel() * 2

    def decode_bytes_per_step(self):
        return self.launches_b * decode_bytes_per_launch(self.geo, self.T)


def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2609_34054_b200 import inputs as I
    from paper_2609_34054_b200.binding import Precc

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the precc path has no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    ranks = None
    if world > 1:
        # evidence of the ranks that really ran: every rank reports its device
        mine = {"rank": rank, "local_rank": local, "device": torch.cuda.get_device_name(local)}
        ranks = [None] * world
        dist.all_gather_object(ranks, mine)
        if rank == 0:
            sys.stderr.write(f"bench.py: {world} ranks over NCCL: {ranks}\n")

    px = Precc(local)
    if args.extra_only:
        res = extra_serving_decode(px, args.c4_batch, args.c4_ctx_min, args.c4_ctx_max) if args.extra_only == "c4" \
            else extra_turn(px, args.c3_ctx, args.c3_new)
        assert px.poll_status() == 0
        print(json.dumps(res))
        return 0
    wl = Workload(px, seed=rank, layers=args.layers, steps=args.decode_steps, T=args.ctx)
    wl.step()                                        # first pass builds the caches (also a warm-up)
    torch.cuda.synchronize()
    if not args.no_graph:
        wl.capture()
    assert px.poll_status() == 0

    def timed(fn, steps, warmup, phases=False):
        for _ in range(warmup):
            fn()
        barrier()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        pa = pb = 0.0
        marks = []
        ev[0].record()
        for _ in range(steps):
            if phases:
                e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                e0.record(); wl.phase_a(); e1.record(); wl.phase_b(); e2.record()
                marks.append((e0, e1, e2))
            else:
                fn()
        ev[1].record()
        barrier()
        ms = ev[0].elapsed_time(ev[1])
        for e0, e1, e2 in marks:
            pa += e0.elapsed_time(e1); pb += e1.elapsed_time(e2)
        ms = reduce_max_ms(ms, "cuda")
        return ms, pa, pb

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms, pa, pb = timed(wl.step, args.steps, args.warmup, phases=True)
    clocks = sampler.stop() if rank == 0 else None
    e2e_steps = max(1, min(args.steps, 4))
    wl.step_host()                                                   # warm-up of the host path (pinned buffers touched)
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    wl.run_host_pipelined(e2e_steps)
    ev1.record()
    barrier()
    ms_e2e = reduce_max_ms(ev0.elapsed_time(ev1), "cuda")
    if not torch.equal(wl.out_host, wl.out.cpu()):                   # the host path returns what the device holds
        raise SystemExit("bench.py: the host-path outputs differ from the device-resident ones")
    status = px.poll_status()
    if status:
        raise SystemExit(f"bench.py: device status 0x{status:x}")

    geo = wl.geo
    step_bytes = wl.decode_bytes_per_step()
    value = whole_job_value(step_bytes, args.steps, ms, world)
    e2e_value = whole_job_value(step_bytes, e2e_steps, ms_e2e, world)
    per_launch = decode_bytes_per_launch(geo, wl.T)
    launch_us = pb / args.steps / wl.launches_b * 1e3
    achieved = per_launch / (launch_us * 1e-6) / 1e9
    peak, peak_kind = measured_peak()
    flops_a = wl.layers * 2.0 * wl.T * geo.d_model * (2 * geo.kv_width + geo.n_agents * (geo.rank_k + geo.rank_v))

    if rank == 0:
        cpu_val, cpu_dt = oracle_sample(args.cpu_requests) if world == 1 and not args.no_cpu else (None, None)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {
                "workload": f"C2 llama-3.2-1B-shaped stack: {wl.layers} layers d=2048 32q/8kv hd=64, N=4 agents r=16 on K,V, "
                            f"T={wl.T}: fused base projection + LR precompute of the trajectory, then {wl.dsteps} decode steps "
                            f"per agent (batch 1)",
                "parallelism": "replicas" if world > 1 else "single GPU",
                "l2_policy": f"decode cycles over {wl.layers} layers' caches = "
                             f"{wl.layers * per_launch / 1e6:.0f} MB > 126 MB L2; no explicit flush",
                "decode_launch": "CUDA graph replay" if not args.no_graph else "eager ctypes launches",
                "ranks": ranks,
            },
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": wl.h2d_bytes(), "d2h_bytes_per_step": wl.d2h_bytes(),
                    "ms_per_step": ms_e2e / e2e_steps, "steps": e2e_steps,
                    "how": "pinned host buffers -> device -> C-ABI calls -> pinned host; copies on a second stream, the next "
                           "step's upload and the previous step's download overlap the compute"},
            "gpu_launches": (wl.launches_a + wl.launches_b) * args.steps,
            "roofline": {"bound": "hbm", "kernel": "lr_attend_decode_cluster_kernel<64,16,16,8>", "achieved": achieved, "peak": peak,
                         "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak, "frac_of_nominal_8TBps": achieved / NOMINAL_HBM_GBS,
                         "traffic": (ncu_traffic("decode_cluster_c2_layer") or {}).get("dram_bytes"),
                         "algorithmic_bytes_per_launch": per_launch, "avg_launch_us": launch_us,
                         "note": "batch-1 launch of 17 MB: latency-bound by construction; the bandwidth-bound decode row is rooflines.decode_serving"},
            "phases": {"precompute_ms_per_step": pa / args.steps, "decode_ms_per_step": pb / args.steps,
                       "projection_tflops": flops_a / (pa / args.steps * 1e-3) / 1e12,
                       "decode_only_GBps": step_bytes / (pb / args.steps * 1e-3) / 1e9},
        }
        if world == 1 and not args.no_extra:
            del wl
            torch.cuda.empty_cache()
            cpu_s = 0.0 if args.no_cpu else 6.0
            line["extra"] = {"serving_decode": extra_serving_decode(px, 64, 4096, 32768, cpu_seconds=cpu_s),
                             "turn": extra_turn(px, 32768, 512, cpu_seconds=cpu_s)}
            # the other rows of the metric, each with its own roofline record (the timed step's is `roofline`)
            line["rooflines"] = {"decode_c2_layer": line["roofline"],
                                 "decode_serving": line["extra"]["serving_decode"]["roofline"],
                                 "prefill_turn": line["extra"]["turn"]["roofline_prefill"],
                                 "lr_precompute_context": line["extra"]["turn"]["roofline_precompute"]}
        if cpu_val is not None:
            line["cpu_baseline"] = {"value": cpu_val, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                                    "sample": f"{args.cpu_requests} decode requests of layer 0 (all kv heads, context {I.C2_T}), "
                                              f"{cpu_dt:.1f} s of numpy float64"}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def spawn_ranks(n: int, argv) -> int:
    """`bench.py --gpus N` run by hand: start N ranks of this script (one per GPU) under torch.distributed.run on
    127.0.0.1 and return the launcher's exit code.  Rank 0 prints the JSON line."""
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def run_stub(args) -> int:
    """The multi-rank plumbing of the benchmark without a GPU: gloo ranks, a sleep of (rank + 1) ms as the step, the
    same barrier / max-over-ranks / whole-job aggregation, one JSON line from rank 0."""
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time.sleep(1e-3 * (rank + 1))
    ms = reduce_max_ms((time.perf_counter() - t0) * 1e3)
    ranks = [None] * world
    if world > 1:
        dist.all_gather_object(ranks, {"rank": rank, "pid": os.getpid()})
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": whole_job_value(1e6, args.steps, ms, world), "unit": UNIT, "n_gpus": world,
                          "steps": args.steps, "ms_per_step": ms / args.steps, "stub": True, "scaling": "weak",
                          "config": {"workload": "stub", "parallelism": "replicas", "ranks": ranks}}))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="precc", choices=["precc", "reference"])
    ap.add_argument("--layers", type=int, default=16)
    ap.add_argument("--decode-steps", type=int, default=128)
    ap.add_argument("--ctx", type=int, default=8192)
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--cpu-requests", type=int, default=120)
    ap.add_argument("--no-extra", action="store_true", help="skip the C4 decode and C3 turn measurements")
    ap.add_argument("--extra-only", choices=["c3", "c4"], help="run only that measurement (used for profiling)")
    ap.add_argument("--c4-batch", type=int, default=64)
    ap.add_argument("--c4-ctx-min", type=int, default=4096)
    ap.add_argument("--c4-ctx-max", type=int, default=32768)
    ap.add_argument("--c3-ctx", type=int, default=32768)
    ap.add_argument("--c3-new", type=int, default=512)
    ap.add_argument("--stub-workload", action="store_true",
                    help="run the rank plumbing (launch, barrier, max-reduce, aggregation) on CPU over gloo with a sleep as the step")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_ranks(args.gpus, sys.argv[1:])          # started without a launcher: become one
    if args.impl == "reference":
        return run_reference(args)
    if args.stub_workload:
        return run_stub(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
