"""Seeded random shapes: head_dim, group size, kv heads, ranks, agents, batch, context lengths (ragged, around
page and tile boundaries), paged or contiguous caches, adapter-free requests mixed in.  Decode and prefill
over directly filled caches against the oracle's cache-content form."""
import os

import numpy as np
import pytest
import torch

from oracle import lrkv_oracle as O
from paper_2609_34054_b200 import inputs as I
from paper_2609_34054_b200.binding import Cache, Precc, layer_desc

from harness import assert_close, f64

pytestmark = pytest.mark.gpu

N_CASES = int(os.environ.get("PRECC_FUZZ_CASES", "36"))      # a longer soak: PRECC_FUZZ_CASES=400


def _case(i: int):
    rng = np.random.default_rng(1000 + i)
    hd = int(rng.choice([64, 128]))
    G = int(rng.choice([1, 2, 4, 7, 8]))
    n_kv = int(rng.choice([1, 2, 3, 5]))
    r = int(rng.choice([0, 8, 16, 32, 64]))
    rk = r if rng.random() < 0.7 else 0
    N = int(rng.integers(1, 5))
    B = int(rng.integers(1, 6))
    edge = [1, 15, 16, 17, 127, 128, 129, 255, 257]
    ctx = [int(rng.choice(edge)) if rng.random() < 0.3 else int(rng.integers(1, 900)) for _ in range(B)]
    if i % 6 == 0:
        ctx[0] = int(rng.integers(3000, 6000))          # long enough for the split paths
    agents = [int(rng.integers(-1, N)) for _ in range(B)]
    paged = bool(rng.random() < 0.5)
    S = int(rng.integers(1, 90))
    T = int(rng.integers(0, 700)) if i % 5 else int(rng.integers(2000, 5000))
    return hd, G, n_kv, rk, r, N, B, ctx, agents, paged, S, T


@pytest.fixture(scope="module")
def px():
    p = Precc(0)
    yield p
    assert p.poll_status() == 0
    p.close()


@pytest.mark.parametrize("i", range(N_CASES))
def test_random_shapes(px, i):
    hd, G, n_kv, rk, rv, N, B, ctx, agents, paged, S, T = _case(i)
    geo = I.Geometry(d_model=64, n_q=G * n_kv, n_kv=n_kv, hd=hd, n_agents=N, rank_k=rk, rank_v=rv, alpha=2.0 * max(rv, 1))
    desc = layer_desc(geo)
    need = [(c + 15) // 16 for c in ctx]
    pool = sum(need) + 3
    c = I.direct_caches(pool, geo, 100 + i, f"fz{i}")
    dev = lambda t: None if t is None else t.cuda()
    cache = Cache.from_tensors(geo, c["k_base"].cuda(), c["v_base"].cuda(), dev(c.get("lr_k")), dev(c.get("lr_v")))
    w = I.layer_weights(geo, 100 + i, f"fz{i}")
    Bk = w["B_k"].cuda() if rk else None
    Bv = w["B_v"].cuda() if rv else None
    # ---------------------------------------------------------------- decode
    perm = I.permutation(pool, 100 + i, f"fz.perm{i}")
    table = torch.zeros((B, max(need)), dtype=torch.int32)
    first, at = [], 0
    for b, n in enumerate(need):
        table[b, :n] = perm[at:at + n] if paged else torch.arange(at, at + n)
        first.append(at)
        at += n
    q = I.queries(B, geo, 100 + i, f"fz.q{i}", gain=3.0)
    out = torch.full_like(q, float("nan"), device="cuda")
    mx = max(ctx)
    ws = px.decode_workspace(desc, B, mx)
    px.lr_attend_decode(desc, q.cuda(), torch.tensor(agents, dtype=torch.int32).cuda(), torch.tensor(ctx, dtype=torch.int32).cuda(),
                        mx, Bk, Bv, cache, out, ws, table.cuda() if paged else None,
                        None if paged else torch.tensor(first, dtype=torch.int32).cuda())
    torch.cuda.synchronize()
    out = f64(out)

    def rows(x, b, t):
        blocks = table[b, :need[b]].long()
        return f64(x[blocks].reshape(-1, x.shape[-1]))[:t]

    def base_rows_of(x, b, t):                              # [blocks, n_kv, 16, hd] -> [t, n_kv*hd]
        blocks = table[b, :need[b]].long()
        return f64(x[blocks].permute(0, 2, 1, 3).reshape(-1, n_kv * hd))[:t]

    zero_k = np.zeros((rk, n_kv * hd)); zero_v = np.zeros((rv, n_kv * hd))
    refs = []
    for b in range(B):
        t, a = ctx[b], agents[b]
        Lk = rows(c["lr_k"][max(a, 0)], b, t) if rk else np.zeros((t, 0))
        Lv = rows(c["lr_v"][max(a, 0)], b, t) if rv else np.zeros((t, 0))
        Bk_a = f64(w["B_k"][a]) if (rk and a >= 0) else zero_k
        Bv_a = f64(w["B_v"][a]) if (rv and a >= 0) else zero_v
        ref = O.attend_from_caches(f64(q[b]), base_rows_of(c["k_base"], b, t), base_rows_of(c["v_base"], b, t), Lk, Lv, Bk_a, Bv_a,
                                   geo.scale_k, geo.scale_v, n_kv)
        refs.append(ref)
        assert_close(out[b], ref, f"case {i} decode request {b} (hd{hd} G{G} kv{n_kv} r{rk}/{rv} ctx{t} agent{a} paged={paged})")
    if B > 1:
        # the same workspace serves a sub-batch (another split plan, possibly the other kernel)
        out2 = torch.full_like(q[1:], float("nan"), device="cuda")
        mx2 = max(ctx[1:])
        px.lr_attend_decode(desc, q[1:].cuda(), torch.tensor(agents[1:], dtype=torch.int32).cuda(),
                            torch.tensor(ctx[1:], dtype=torch.int32).cuda(), mx2, Bk, Bv, cache, out2, ws,
                            table[1:].contiguous().cuda() if paged else None,
                            None if paged else torch.tensor(first[1:], dtype=torch.int32).cuda())
        torch.cuda.synchronize()
        for b in range(1, B):
            assert_close(f64(out2[b - 1]), refs[b], f"case {i} sub-batch request {b}")
    # ---------------------------------------------------------------- prefill over a second, contiguous-or-paged sequence
    nb2 = (T + S + 15) // 16
    c2 = I.direct_caches(nb2 + 2, geo, 200 + i, f"fzp{i}")
    cache2 = Cache.from_tensors(geo, c2["k_base"].cuda(), c2["v_base"].cuda(), dev(c2.get("lr_k")), dev(c2.get("lr_v")))
    tab2 = I.permutation(nb2 + 2, 200 + i, f"fzp.perm{i}")[:nb2].to(torch.int32) if paged else torch.arange(1, nb2 + 1, dtype=torch.int32)
    agent = agents[0]
    qs = I.queries(S, geo, 200 + i, f"fzp.q{i}", gain=3.0)
    outp = torch.full_like(qs, float("nan"), device="cuda")
    px.lr_attend_prefill(desc, qs.cuda(), agent, T, Bk, Bv, cache2, outp, tab2.cuda() if paged else None, 0 if paged else 1)
    torch.cuda.synchronize()
    outp = f64(outp)
    blocks = tab2.long()
    kb = f64(c2["k_base"][blocks].permute(0, 2, 1, 3).reshape(-1, n_kv * hd))
    vb = f64(c2["v_base"][blocks].permute(0, 2, 1, 3).reshape(-1, n_kv * hd))
    Lk2 = f64(c2["lr_k"][max(agent, 0)][blocks].reshape(-1, rk)) if rk else np.zeros((nb2 * 16, 0))
    Lv2 = f64(c2["lr_v"][max(agent, 0)][blocks].reshape(-1, rv)) if rv else np.zeros((nb2 * 16, 0))
    Bk_a = f64(w["B_k"][agent]) if (rk and agent >= 0) else zero_k
    Bv_a = f64(w["B_v"][agent]) if (rv and agent >= 0) else zero_v
    for srow in sorted(set([0, S // 2, S - 1])):
        t = T + srow + 1
        ref = O.attend_from_caches(f64(qs[srow]), kb[:t], vb[:t], Lk2[:t], Lv2[:t], Bk_a, Bv_a, geo.scale_k, geo.scale_v, n_kv)
        assert_close(outp[srow], ref, f"case {i} prefill row {srow} (hd{hd} G{G} kv{n_kv} r{rk}/{rv} T{T} S{S} agent{agent} paged={paged})")


# ---------------------------------------------------------------------------------------------------------
# Projections and the rotary path, through the library's own calls (hidden states -> caches -> attention)

from harness import Layer, base_rows, lr_rows                     # noqa: E402
from paper_2609_34054_b200.inputs import rope_table               # noqa: E402

N_PROJ = max(12, N_CASES // 3)


def _proj_case(i: int):
    rng = np.random.default_rng(5000 + i)
    d = int(rng.choice([64, 128, 192, 320, 1024, 2048]))           # 1024 and 2048: deep enough for the split-K kernel
    hd = int(rng.choice([64, 128]))
    n_kv = int(rng.choice([1, 2, 3]))
    r = int(rng.choice([8, 16, 32, 64]))
    N = int(rng.integers(1, 6))
    kind = int(rng.integers(0, 4))
    M = [int(rng.integers(1, 65)), int(rng.integers(65, 400)), int(rng.integers(400, 1500)),
         int(rng.choice([1, 16, 17, 64, 65, 127, 128, 129, 256]))][kind]
    scattered = bool(rng.random() < 0.5)
    mask = int(rng.integers(1, 1 << N))
    return d, hd, n_kv, r, N, M, scattered, mask


@pytest.mark.parametrize("i", range(N_PROJ))
def test_random_projections(px, i):
    """rebase_project + lr_precompute against the definition on every row; the fused turn_project bit-equal
    to the two separate calls; masked-out agents and unaddressed slots untouched."""
    d, hd, n_kv, r, N, M, scattered, mask = _proj_case(i)
    geo = I.Geometry(d, 2 * n_kv, n_kv, hd, N, r, r, alpha=2.0 * r)
    H = I.hidden_states(M, geo, seed=300 + i, tag=f"pz{i}")
    nb = (M + 15) // 16 + 3
    start = 5 if not scattered else 0
    slots = I.permutation(nb * 16, 300 + i, f"pz.slots{i}")[:M].to(torch.int32) if scattered else None
    La = Layer(px, geo, seed=300 + i, n_blocks=nb, fill=float("nan"), tag=f"pz{i}")
    La.append(H, start_slot=start, slot_mapping=None if slots is None else slots.cuda(), agent_mask=mask)
    torch.cuda.synchronize()
    sl = slots.long() if scattered else torch.arange(start, start + M)
    w, Hn = La.w_np, f64(H)
    tol = lambda ref: 2.0 ** -8 * np.abs(ref) + 2e-3 * np.sqrt(d / 256)
    for got, ref in ((base_rows(La.cache.k_base)[sl], O.base_cache(Hn, w["W_k"])),
                     (base_rows(La.cache.v_base)[sl], O.base_cache(Hn, w["W_v"]))):
        assert (np.abs(got - ref) <= tol(ref)).all(), f"case {i} base (d{d} hd{hd} kv{n_kv} M{M})"
    for a in range(N):
        if mask >> a & 1:
            for name, A in (("lr_k", w["A_k"]), ("lr_v", w["A_v"])):
                got, ref = lr_rows(getattr(La.cache, name), a)[sl], O.lr_cache(Hn, A[a])
                assert (np.abs(got - ref) <= tol(ref)).all(), f"case {i} {name}[{a}] (d{d} r{r} M{M})"
        else:
            assert torch.isnan(La.cache.lr_k[a]).all() and torch.isnan(La.cache.lr_v[a]).all(), f"case {i}: masked agent {a} written"
    untouched = torch.ones(nb * 16, dtype=torch.bool); untouched[sl] = False
    assert torch.isnan(La.cache.k_base.permute(0, 2, 1, 3).reshape(nb * 16, -1)[untouched]).all()
    Lb = Layer(px, geo, seed=300 + i, n_blocks=nb, fill=float("nan"), tag=f"pz{i}")
    dev = {k: v.cuda() for k, v in Lb.w.items()}
    WA = px.pack_turn_weights(geo, dev["W_k"], dev["W_v"], dev["A_k"], dev["A_v"])
    px.turn_project(Lb.desc, H.cuda(), WA, Lb.cache, start, None if slots is None else slots.cuda(), mask)
    torch.cuda.synchronize()
    for name in ("k_base", "v_base", "lr_k", "lr_v"):
        a_, b_ = getattr(La.cache, name).view(torch.int16), getattr(Lb.cache, name).view(torch.int16)
        assert torch.equal(a_, b_), f"case {i}: fused projection differs in {name}"
    # one mask per row (double batching): a row's LR columns land only in the agents its mask names, with the
    # same bits as above; the base columns of every row are written
    rng = np.random.default_rng(7000 + i)
    row_masks = torch.from_numpy(rng.integers(0, 1 << N, size=M).astype(np.int64))
    Lc = Layer(px, geo, seed=300 + i, n_blocks=nb, fill=float("nan"), tag=f"pz{i}")
    slots_c = (slots if scattered else torch.arange(start, start + M, dtype=torch.int32)).cuda()
    px.turn_project_rows(Lc.desc, H.cuda(), WA, Lc.cache, slots_c, row_masks.cuda())
    full = Layer(px, geo, seed=300 + i, n_blocks=nb, fill=float("nan"), tag=f"pz{i}")
    px.turn_project(full.desc, H.cuda(), WA, full.cache, start, None if slots is None else slots.cuda())      # every agent
    torch.cuda.synchronize()
    assert torch.equal(Lc.cache.k_base.view(torch.int16), full.cache.k_base.view(torch.int16))
    assert torch.equal(Lc.cache.v_base.view(torch.int16), full.cache.v_base.view(torch.int16))
    for a in range(N):
        named = ((row_masks >> a) & 1).bool()
        for name in ("lr_k", "lr_v"):
            got = getattr(Lc.cache, name)[a].reshape(nb * 16, -1)[sl]
            want = getattr(full.cache, name)[a].reshape(nb * 16, -1)[sl]
            assert torch.equal(got[named].view(torch.int16), want[named].view(torch.int16)), f"case {i}: {name}[{a}] rows"
            assert torch.isnan(got[~named]).all(), f"case {i}: {name}[{a}] written for rows that do not name it"


def _rope_case(i: int):
    rng = np.random.default_rng(9000 + i)
    hd = int(rng.choice([64, 128]))
    G = int(rng.choice([1, 2, 4, 8]))
    n_kv = int(rng.choice([1, 2, 3]))
    r = int(rng.choice([8, 16, 32, 64]))
    T = int(rng.integers(1, 700)) if i % 4 else int(rng.integers(1500, 2600))
    S = int(rng.integers(1, 60))
    B = int(rng.integers(1, 4))
    ctx = [T + S] + [int(rng.integers(1, T + S + 1)) for _ in range(B - 1)]
    agents = [int(rng.integers(-1, 2)) for _ in range(B)]
    return hd, G, n_kv, r, T, S, ctx, agents


@pytest.mark.parametrize("i", range(N_PROJ))
def test_random_rope_shapes(px, i):
    """Rotary keys end to end: rotated base projection, un-rotated LR rows, rotary decode and prefill against
    the oracle's definition (adapted key = rotation of the full-width adapted projection)."""
    hd, G, n_kv, r, T, S, ctx, agents = _rope_case(i)
    geo = I.Geometry(d_model=128, n_q=G * n_kv, n_kv=n_kv, hd=hd, n_agents=2, rank_k=r, rank_v=r, alpha=2.0 * r)
    L = Layer(px, geo, seed=600 + i, n_blocks=(T + S + 15) // 16, tag=f"rz{i}")
    H = I.hidden_states(T + S, geo, 600 + i, f"rz.H{i}")
    table = rope_table(T + S + 1, hd)
    cos, sin = O.rope_tables(T + S + 1, hd)
    px.rebase_project_rope(L.desc, H.cuda(), L.W_packed, L.cache, table, 0)
    px.lr_precompute(L.desc, H.cuda(), L.A_packed, L.cache, 0)
    w = L.w_np
    args = (f64(H), w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"])
    q = I.queries(len(ctx), geo, 600 + i, f"rz.q{i}", gain=3.0)
    out = torch.full_like(q, float("nan"), device="cuda")
    ws = px.decode_workspace(L.desc, len(ctx), max(ctx))
    px.lr_attend_decode_rope(L.desc, q.cuda(), torch.tensor(agents, dtype=torch.int32).cuda(), torch.tensor(ctx, dtype=torch.int32).cuda(),
                             max(ctx), L.B_k, L.B_v, table, L.cache, out, ws)
    torch.cuda.synchronize()
    adapted = O.lr_decode_reference_rope(f64(q), [max(a, 0) for a in agents], ctx, *args, geo.scale_k, geo.scale_v, n_kv, cos, sin)
    neutral = O.lr_decode_reference_rope(f64(q), [0] * len(ctx), ctx, *args, 0.0, 0.0, n_kv, cos, sin)
    ref = np.where(np.array(agents)[:, None, None] < 0, neutral, adapted)
    assert_close(f64(out), ref, f"case {i} rope decode (hd{hd} G{G} kv{n_kv} r{r} ctx{ctx} agents{agents})")
    qs = I.queries(S, geo, 600 + i, f"rz.qs{i}", gain=3.0)
    outp = torch.full_like(qs, float("nan"), device="cuda")
    px.lr_attend_prefill_rope(L.desc, qs.cuda(), 1, T, L.B_k, L.B_v, table, L.cache, outp)
    torch.cuda.synchronize()
    refp = O.lr_prefill_reference_rope(f64(qs), 1, T, *args, geo.scale_k, geo.scale_v, n_kv, cos, sin)
    assert_close(f64(outp), refp, f"case {i} rope prefill (hd{hd} G{G} kv{n_kv} r{r} T{T} S{S})")
    # the same turn through the key scratch (adapted rotary keys written once, then the tensor-core kernel)
    scratch = torch.empty(px.prefill_rope_scratch_bytes(L.desc, T, S), dtype=torch.uint8, device="cuda")
    outs = torch.full_like(qs, float("nan"), device="cuda")
    px.lr_attend_prefill_rope_scratch(L.desc, qs.cuda(), 1, T, L.B_k, L.B_v, table, L.cache, outs, scratch)
    torch.cuda.synchronize()
    assert_close(f64(outs), refp, f"case {i} rope prefill through scratch (hd{hd} G{G} kv{n_kv} r{r} T{T} S{S})")


def _shard_case(i: int):
    rng = np.random.default_rng(13000 + i)
    hd = int(rng.choice([64, 128]))
    G = int(rng.choice([1, 2, 4, 8]))
    n_kv = int(rng.choice([1, 2, 3]))
    r = int(rng.choice([0, 8, 16, 32, 64]))
    world = int(rng.integers(1, 9))
    T = int(rng.integers(40, 900)) if i % 4 else int(rng.integers(2500, 4500))
    B = int(rng.integers(1, 5))
    ctx = [T] + [int(rng.integers(0, T + 1)) for _ in range(B - 1)]
    agents = [int(rng.integers(-1, 2)) for _ in range(B)]
    return hd, G, n_kv, r, world, T, ctx, agents


@pytest.mark.parametrize("i", range(N_PROJ))
def test_random_context_shards(px, i):
    """Context-sharded decode (shards run one after another on this GPU): partial records merged by the
    combine kernel equal attention over the whole context."""
    from paper_2609_34054_b200.sharded import shard_ranges
    hd, G, n_kv, r, world, T, ctx, agents = _shard_case(i)
    geo = I.Geometry(d_model=128, n_q=G * n_kv, n_kv=n_kv, hd=hd, n_agents=2, rank_k=r, rank_v=r, alpha=2.0 * max(r, 1))
    H = I.hidden_states(T, geo, 800 + i, f"sz.H{i}")
    q = I.queries(len(ctx), geo, 800 + i, f"sz.q{i}", gain=3.0)
    ranges = shard_ranges(ctx, world)
    aid = torch.tensor(agents, dtype=torch.int32).cuda()
    recs, first_layer = None, None
    for rk_ in range(world):
        local = [e - s for s, e in ranges[rk_]]
        L = Layer(px, geo, seed=800 + i, n_blocks=sum((l + 15) // 16 for l in local) + 1, tag=f"sz{i}")
        first, at = [], 0
        for (s, e) in ranges[rk_]:
            first.append(at)
            if e > s:
                L.append(H[s:e], start_slot=at * 16)
            at += (e - s + 15) // 16
        if recs is None:
            recs = torch.full((world, len(ctx), n_kv, px.partial_record_floats(L.desc)), float("nan"), dtype=torch.float32, device="cuda")
            first_layer = L
        mx = max(1, max(local))
        ws = px.decode_workspace(L.desc, len(ctx), mx)
        px.lr_attend_decode_partial(L.desc, q.cuda(), aid, torch.tensor(local, dtype=torch.int32).cuda(), mx, L.B_k, L.cache,
                                    recs[rk_], ws, None, torch.tensor(first, dtype=torch.int32).cuda())
    out = torch.full_like(q, float("nan"), device="cuda")
    px.combine_partials(first_layer.desc, recs, aid, first_layer.B_v, out)
    torch.cuda.synchronize()
    assert torch.isfinite(recs).all()
    w = first_layer.w_np
    args = (f64(H), w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"])
    live = [b for b, t in enumerate(ctx) if t > 0]
    adapted = O.lr_decode_reference(f64(q)[live], [max(agents[b], 0) for b in live], [ctx[b] for b in live], *args, geo.scale_k, geo.scale_v, n_kv)
    neutral = O.lr_decode_reference(f64(q)[live], [0] * len(live), [ctx[b] for b in live], *args, 0.0, 0.0, n_kv)
    ref = np.where(np.array([agents[b] for b in live])[:, None, None] < 0, neutral, adapted)
    assert_close(f64(out)[live], ref, f"case {i} sharded decode (hd{hd} G{G} kv{n_kv} r{r} world{world} ctx{ctx} agents{agents})")
    for b, t in enumerate(ctx):
        if t == 0:
            assert (out[b] == 0).all(), f"case {i}: empty request {b} not zero"


# ---------------------------------------------------------------------------------------------------------
# Large shapes (caches drawn on the device): batches up to 64 requests, contexts up to 70k tokens, turns of
# up to 2047 new tokens over up to 66k; sampled requests / rows against the oracle.

N_LARGE = max(6, N_CASES // 6)


def _weights_small(geo, seed, tag):
    w = I.layer_weights(geo, seed, tag)
    return (w["B_k"].cuda() if geo.rank_k else None, w["B_v"].cuda() if geo.rank_v else None, w)


@pytest.mark.parametrize("i", range(N_LARGE))
def test_random_large_decode(px, i):
    rng = np.random.default_rng(20000 + i)
    hd = int(rng.choice([64, 128])); G = int(rng.choice([1, 2, 4, 7, 8])); n_kv = int(rng.choice([1, 2, 4, 8]))
    r = int(rng.choice([0, 8, 16, 32, 64])); N = int(rng.integers(1, 5))
    B = int(rng.choice([1, 1, 2, 3, 5, 8, 16, 33, 64]))
    tmax = int(rng.choice([3000, 9000, 20000, 70000]))
    ctx = [int(rng.integers(1, tmax + 1)) for _ in range(B)]
    while sum(ctx) > 400000:
        ctx = [max(1, c // 2) for c in ctx]
    agents = [int(rng.integers(-1, N)) for _ in range(B)]
    paged = bool(rng.random() < 0.6)
    geo = I.Geometry(64, G * n_kv, n_kv, hd, N, r, r, alpha=2.0 * max(r, 1))
    desc = layer_desc(geo)
    need = [(c + 15) // 16 for c in ctx]
    pool = sum(need) + 5
    c = I.direct_caches_device(pool, geo, 400 + i, f"lz{i}")
    cache = Cache.from_tensors(geo, c["k_base"], c["v_base"], c.get("lr_k"), c.get("lr_v"))
    Bk, Bv, w = _weights_small(geo, 400 + i, f"lz{i}")
    perm = I.permutation(pool, 400 + i, f"lz.perm{i}")
    table = torch.zeros((B, max(need)), dtype=torch.int32)
    first, at = [], 0
    for b, n in enumerate(need):
        table[b, :n] = perm[at:at + n] if paged else torch.arange(at, at + n)
        first.append(at)
        at += n
    q = I.queries(B, geo, 400 + i, f"lz.q{i}", gain=3.0)
    out = torch.full_like(q, float("nan"), device="cuda")
    mx = max(ctx)
    ws = px.decode_workspace(desc, B, mx)
    px.lr_attend_decode(desc, q.cuda(), torch.tensor(agents, dtype=torch.int32).cuda(), torch.tensor(ctx, dtype=torch.int32).cuda(),
                        mx, Bk, Bv, cache, out, ws, table.cuda() if paged else None,
                        None if paged else torch.tensor(first, dtype=torch.int32).cuda())
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all()
    for b in sorted(set([0, B // 2, B - 1, int(np.argmax(ctx))])):
        t, a = ctx[b], agents[b]
        blocks = table[b, :need[b]].long().cuda()
        rows = lambda x: f64(x[blocks].permute(0, 2, 1, 3).reshape(-1, n_kv * hd))[:t]
        Lk = f64(c["lr_k"][max(a, 0)][blocks].reshape(-1, r))[:t] if r else np.zeros((t, 0))
        Lv = f64(c["lr_v"][max(a, 0)][blocks].reshape(-1, r))[:t] if r else np.zeros((t, 0))
        Bka = f64(w["B_k"][a]) if (r and a >= 0) else np.zeros((r, n_kv * hd))
        Bva = f64(w["B_v"][a]) if (r and a >= 0) else np.zeros((r, n_kv * hd))
        ref = O.attend_from_caches(f64(q[b]), rows(c["k_base"]), rows(c["v_base"]), Lk, Lv, Bka, Bva, geo.scale_k, geo.scale_v, n_kv)
        assert_close(f64(out[b]), ref, f"case {i} large decode request {b} (hd{hd} G{G} kv{n_kv} r{r} B{B} ctx{t} agent{a} paged={paged})")


@pytest.mark.parametrize("i", range(N_LARGE))
def test_random_large_prefill(px, i):
    rng = np.random.default_rng(40000 + i)
    hd = int(rng.choice([64, 128])); G = int(rng.choice([1, 2, 4, 8])); n_kv = int(rng.choice([1, 2, 4, 8]))
    r = int(rng.choice([0, 8, 16, 32, 64])); N = int(rng.integers(1, 4))
    S = int(rng.choice([1, 7, 16, 31, 32, 33, 64, 100, 128, 200, 256, 500, 512, 1000, 2047]))
    T = int(rng.choice([0, 1, 100, 127, 128, 1000, 4000, 9000, 30000, 66000]))
    if T > 100:
        T = int(rng.integers(T // 2, T + 1))
    agent = int(rng.integers(-1, N))
    paged = bool(rng.random() < 0.5)
    geo = I.Geometry(64, G * n_kv, n_kv, hd, N, r, r, alpha=2.0 * max(r, 1))
    desc = layer_desc(geo)
    nb = (T + S + 15) // 16
    c = I.direct_caches_device(nb + 3, geo, 500 + i, f"lp{i}")
    cache = Cache.from_tensors(geo, c["k_base"], c["v_base"], c.get("lr_k"), c.get("lr_v"))
    Bk, Bv, w = _weights_small(geo, 500 + i, f"lp{i}")
    tab = I.permutation(nb + 3, 500 + i, f"lp.perm{i}")[:nb].to(torch.int32) if paged else torch.arange(2, nb + 2, dtype=torch.int32)
    q = I.queries(S, geo, 500 + i, f"lp.q{i}", gain=3.0)
    out = torch.full_like(q, float("nan"), device="cuda")
    px.lr_attend_prefill(desc, q.cuda(), agent, T, Bk, Bv, cache, out, tab.cuda() if paged else None, 0 if paged else 2)
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all()
    blocks = tab.long().cuda()
    K = f64(c["k_base"][blocks].permute(0, 2, 1, 3).reshape(-1, n_kv * hd))
    V = f64(c["v_base"][blocks].permute(0, 2, 1, 3).reshape(-1, n_kv * hd))
    Lk = f64(c["lr_k"][max(agent, 0)][blocks].reshape(-1, r)) if r else np.zeros((nb * 16, 0))
    Lv = f64(c["lr_v"][max(agent, 0)][blocks].reshape(-1, r)) if r else np.zeros((nb * 16, 0))
    Bka = f64(w["B_k"][agent]) if (r and agent >= 0) else np.zeros((r, n_kv * hd))
    Bva = f64(w["B_v"][agent]) if (r and agent >= 0) else np.zeros((r, n_kv * hd))
    for srow in sorted(set([0, S // 3, S // 2, S - 1])):
        t = T + srow + 1
        ref = O.attend_from_caches(f64(q[srow]), K[:t], V[:t], Lk[:t], Lv[:t], Bka, Bva, geo.scale_k, geo.scale_v, n_kv)
        assert_close(f64(out[srow]), ref, f"case {i} large prefill row {srow} (hd{hd} G{G} kv{n_kv} r{r} S{S} T{T} agent{agent} paged={paged})")


@pytest.fixture(scope="module")
def px_helpers():
    """A context in which short contexts qualify for helper blocks too (the switch is read at creation)."""
    old = os.environ.get("PRECC_PREFILL_HELPER_MIN")
    os.environ["PRECC_PREFILL_HELPER_MIN"] = "8"
    p = Precc(0)
    if old is None:
        del os.environ["PRECC_PREFILL_HELPER_MIN"]
    else:
        os.environ["PRECC_PREFILL_HELPER_MIN"] = old
    yield p
    assert p.poll_status() == 0
    p.close()


@pytest.mark.parametrize("i", range(N_LARGE))
def test_random_prefill_with_helper_blocks(px_helpers, i):
    """Turn lengths that leave between a sixteenth and a half of the SMs without a block, contexts of 1k .. 40k tokens:
    the planner's own cuts (or its refusal), against the definition on rows across the turn, twice on one workspace."""
    px = px_helpers
    rng = np.random.default_rng(60000 + i)
    hd = int(rng.choice([64, 128])); G = int(rng.choice([1, 2, 4, 8])); n_kv = int(rng.choice([2, 4, 8]))
    r = int(rng.choice([0, 8, 16, 32, 64])); N = int(rng.integers(1, 4))
    tpt = 128 // G
    tiles = int(rng.integers(px.sm_count // 2 + 1, px.sm_count * 14 // 15))
    X = max(1, tiles // n_kv)
    S = int(min(4000, X * tpt - int(rng.integers(0, tpt))))
    T = int(rng.choice([1000, 3000, 9000, 20000, 40000]))
    T = int(rng.integers(T // 2, T + 1))
    agent = int(rng.integers(-1, N))
    paged = bool(rng.random() < 0.5)
    geo = I.Geometry(64, G * n_kv, n_kv, hd, N, r, r, alpha=2.0 * max(r, 1))
    desc = layer_desc(geo)
    nb = (T + S + 15) // 16
    c = I.direct_caches_device(nb + 3, geo, 600 + i, f"hp{i}")
    cache = Cache.from_tensors(geo, c["k_base"], c["v_base"], c.get("lr_k"), c.get("lr_v"))
    Bk, Bv, w = _weights_small(geo, 600 + i, f"hp{i}")
    tab = I.permutation(nb + 3, 600 + i, f"hp.perm{i}")[:nb].to(torch.int32) if paged else torch.arange(2, nb + 2, dtype=torch.int32)
    q = I.queries(S, geo, 600 + i, f"hp.q{i}", gain=3.0)
    ws = torch.full((max(px.prefill_ws_bytes(desc, S), 256),), 0x5A, dtype=torch.uint8, device="cuda")
    outs = []
    for _ in range(2):
        out = torch.full_like(q, float("nan"), device="cuda")
        px.lr_attend_prefill_ws(desc, q.cuda(), agent, T, Bk, Bv, cache, out, ws, tab.cuda() if paged else None, 0 if paged else 2)
        torch.cuda.synchronize()
        outs.append(out)
    assert torch.equal(outs[0], outs[1])
    out = outs[0]
    assert torch.isfinite(out.float()).all()
    blocks = tab.long().cuda()
    K = f64(c["k_base"][blocks].permute(0, 2, 1, 3).reshape(-1, n_kv * hd))
    V = f64(c["v_base"][blocks].permute(0, 2, 1, 3).reshape(-1, n_kv * hd))
    Lk = f64(c["lr_k"][max(agent, 0)][blocks].reshape(-1, r)) if r else np.zeros((nb * 16, 0))
    Lv = f64(c["lr_v"][max(agent, 0)][blocks].reshape(-1, r)) if r else np.zeros((nb * 16, 0))
    Bka = f64(w["B_k"][agent]) if (r and agent >= 0) else np.zeros((r, n_kv * hd))
    Bva = f64(w["B_v"][agent]) if (r and agent >= 0) else np.zeros((r, n_kv * hd))
    for srow in sorted(set([0, tpt - 1, S // 2, S - 1])):
        srow = min(srow, S - 1)
        t = T + srow + 1
        ref = O.attend_from_caches(f64(q[srow]), K[:t], V[:t], Lk[:t], Lv[:t], Bka, Bva, geo.scale_k, geo.scale_v, n_kv)
        assert_close(f64(out[srow]), ref, f"case {i} helper prefill row {srow} (hd{hd} G{G} kv{n_kv} r{r} S{S} T{T} agent{agent} paged={paged})")
