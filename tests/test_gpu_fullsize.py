"""Parity at the full sizes of the workload configurations, in the launch configurations the benchmark
times, on sampled outputs the oracle can compute one by one."""
import numpy as np
import pytest
import torch

from oracle import lrkv_oracle as O
from paper_2609_34054_b200 import inputs as I
from paper_2609_34054_b200.binding import Cache, Precc, layer_desc

from harness import Layer, assert_close, f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def px():
    p = Precc(0)
    yield p
    assert p.poll_status() == 0
    p.close()


def test_c2_layer_full_context_batch1(px):
    """One layer of the benchmark stack: caches built by the GEMM kernels, then batch-1 decode over all
    8192 tokens exactly as bench.py launches it (one request per call)."""
    geo, T = I.C2, I.C2_T
    L = Layer(px, geo, seed=0, n_blocks=T // 16, tag="L0")
    H = I.hidden_states(T, geo, 0, "L0.H")
    L.append(H)
    w, Hn = L.w_np, f64(H)
    ws = px.decode_workspace(L.desc, 1, T)
    for agent, gain in ((0, 1.0), (3, 4.0)):
        q = I.queries(1, geo, 0, f"q.a{agent}", gain=gain)
        out = f64(L.decode(q, [agent], [T], max_ctx=T, ws=ws))
        ref = O.lr_decode_reference(f64(q), [agent], [T], Hn, w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"],
                                    geo.scale_k, geo.scale_v, geo.n_kv)
        assert_close(out, ref, f"C2 decode agent {agent} gain {gain}")


def test_c3_turn_prefill_rebase_and_decode(px):
    """Llama-3-8B-shaped layer: context 32768 + a 512-token turn.  Prefill over base + LR of the current
    agent, then the adapter-free re-projection of the turn; checked on sampled kv heads and rows."""
    geo, T, S = I.C3, I.C3_T, I.C3_S
    cur = 1
    L = Layer(px, geo, seed=0, n_blocks=(T + S) // 16, tag="C3")
    H = torch.cat([I.hidden_states(T, geo, 0, "C3.H_ctx"), I.hidden_states(S, geo, 0, "C3.H_new_adpt")])
    L.append(H)
    w, Hn = L.w_np, f64(H)
    heads = [0, 5]
    rows = [0, 1, 2, 15, 16, 17, 255, 256, 510, 511]
    for gain in (1.0, 4.0):
        qs = I.queries(S, geo, 0, f"C3.q.{gain}", gain=gain)
        got = f64(L.prefill(qs, cur, T))
        ref = O.lr_prefill_reference(f64(qs), cur, T, Hn, w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"],
                                     geo.scale_k, geo.scale_v, geo.n_kv, heads=heads, rows=rows)
        assert_close(got, ref, f"C3 prefill gain {gain}")
    # decode at this shape (4 requests, one per agent, different lengths)
    ctx = [T + S, T, 20000, 4097]
    q = I.queries(4, geo, 0, "C3.qdec", gain=4.0)
    out = f64(L.decode(q, [0, 1, 2, 3], ctx))
    ref = O.lr_decode_reference(f64(q), [0, 1, 2, 3], ctx, Hn, w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"],
                                geo.scale_k, geo.scale_v, geo.n_kv, heads=[3])
    assert_close(out, ref, "C3-shape decode")
    # ReBase: adapter-free hidden states of the turn overwrite the base rows and the other agents' LR rows
    X_neut = I.hidden_states(S, geo, 0, "C3.H_new_neut")
    keep = L.cache.lr_v[cur].clone()
    px.rebase_project(L.desc, X_neut.cuda(), L.W_packed, L.cache, T)
    px.lr_precompute(L.desc, X_neut.cuda(), L.A_packed, L.cache, T, None, ~(1 << cur))
    torch.cuda.synchronize()
    assert torch.equal(L.cache.lr_v[cur], keep)
    g = heads[1]
    kb = f64(L.cache.k_base[T // 16:, g].reshape(S, geo.hd))
    refk = O.base_cache(f64(X_neut), w["W_k"][:, g * geo.hd:(g + 1) * geo.hd])
    assert (np.abs(kb - refk) <= 2.0 ** -8 * np.abs(refk) + 1e-3).all()
    lr0 = f64(L.cache.lr_k[0, T // 16:].reshape(S, geo.rank_k))
    refl = O.lr_cache(f64(X_neut), w["A_k"][0])
    assert (np.abs(lr0 - refl) <= 2.0 ** -8 * np.abs(refl) + 1e-3).all()


def test_c4_serving_batch_paged(px):
    """64 requests, agent ids uniform over 8, context lengths uniform in [4096, 32768], paged-16 caches
    filled directly.  The block tables draw from a pool smaller than the logical total (blocks are shared
    read-only between requests), which leaves the launch configuration unchanged."""
    geo = I.C4
    agent_id, ctx_len = I.serving_batch(I.C4_BATCH, I.C4_CTX_MIN, I.C4_CTX_MAX, geo.n_agents, 0)
    pool = 8192
    c = I.direct_caches(pool, geo, 0, "C4")
    cache = Cache.from_tensors(geo, c["k_base"].cuda(), c["v_base"].cuda(), c["lr_k"].cuda(), c["lr_v"].cuda())
    need = [(int(t) + 15) // 16 for t in ctx_len]
    table = torch.zeros((I.C4_BATCH, max(need)), dtype=torch.int32)
    for b, n in enumerate(need):
        table[b, :n] = I.uniform_int(0, pool - 1, n, 0, f"C4.table.{b}")
    w = I.layer_weights(geo, 0, "C4")
    desc = layer_desc(geo)
    q = I.queries(I.C4_BATCH, geo, 0, "C4.q", gain=4.0)
    out = torch.full_like(q, float("nan"), device="cuda")
    mx = int(ctx_len.max())
    ws = px.decode_workspace(desc, I.C4_BATCH, mx)
    px.lr_attend_decode(desc, q.cuda(), agent_id.cuda(), ctx_len.cuda(), mx, w["B_k"].cuda(), w["B_v"].cuda(), cache, out, ws,
                        table.cuda())
    torch.cuda.synchronize()
    out = f64(out)
    assert np.isfinite(out).all()
    G = geo.group
    longest, shortest = int(torch.argmax(ctx_len)), int(torch.argmin(ctx_len))
    for b, g in ((longest, 0), (shortest, 3), (7, 1), (33, 2), (63, 3)):
        t, a = int(ctx_len[b]), int(agent_id[b])
        blocks = table[b, :need[b]].long()
        rows = lambda x: f64(x[blocks].reshape(-1, x.shape[-1]))[:t]
        kb = f64(c["k_base"][blocks][:, g].reshape(-1, geo.hd))[:t]
        vb = f64(c["v_base"][blocks][:, g].reshape(-1, geo.hd))[:t]
        cols = slice(g * geo.hd, (g + 1) * geo.hd)
        ref = O.attend_from_caches(f64(q[b, g * G:(g + 1) * G]), kb, vb, rows(c["lr_k"][a]), rows(c["lr_v"][a]),
                                   f64(w["B_k"][a][:, cols]), f64(w["B_v"][a][:, cols]), geo.scale_k, geo.scale_v, 1)
        assert_close(out[b, g * G:(g + 1) * G], ref, f"C4 request {b} head {g}")


def test_c5_cell_long_context_rank64(px):
    """One sweep cell at the largest context: r = 64, T = 131072, batch 1, contiguous caches."""
    geo = I.c5_geometry(64, 2)
    T = 131072
    c = I.direct_caches(T // 16, geo, 1, "C5")
    cache = Cache.from_tensors(geo, c["k_base"].cuda(), c["v_base"].cuda(), c["lr_k"].cuda(), c["lr_v"].cuda())
    w = I.layer_weights(geo, 1, "C5")
    desc = layer_desc(geo)
    q = I.queries(1, geo, 1, "C5.q", gain=4.0)
    out = torch.full_like(q, float("nan"), device="cuda")
    ws = px.decode_workspace(desc, 1, T)
    px.lr_attend_decode(desc, q.cuda(), torch.tensor([1], dtype=torch.int32, device="cuda"),
                        torch.tensor([T], dtype=torch.int32, device="cuda"), T, w["B_k"].cuda(), w["B_v"].cuda(), cache, out, ws)
    torch.cuda.synchronize()
    g, G = 6, geo.group
    cols = slice(g * geo.hd, (g + 1) * geo.hd)
    ref = O.attend_from_caches(f64(q[0, g * G:(g + 1) * G]), f64(c["k_base"][:, g].reshape(T, geo.hd)),
                               f64(c["v_base"][:, g].reshape(T, geo.hd)), f64(c["lr_k"][1].reshape(T, 64)),
                               f64(c["lr_v"][1].reshape(T, 64)), f64(w["B_k"][1][:, cols]), f64(w["B_v"][1][:, cols]),
                               geo.scale_k, geo.scale_v, 1)
    assert_close(f64(out)[0, g * G:(g + 1) * G], ref, "C5 r=64 T=128k")
