"""GPU parity: the CUDA path (through the C-ABI binding) against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import lrkv_oracle as O
from paper_2609_34054_b200 import inputs as I
from paper_2609_34054_b200.binding import Precc, PreccError

from harness import ATOL, RTOL, Layer, assert_close, base_rows, f64, lr_rows

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def px():
    p = Precc(0)
    yield p
    assert p.poll_status() == 0, "a kernel recorded a device status"
    p.close()


def _ref_decode(L: Layer, H, q, agent_id, ctx_len, heads=None, softmax_scale=None):
    w, g = L.w_np, L.geo
    return O.lr_decode_reference(f64(q), agent_id, ctx_len, f64(H), w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"],
                                 w["B_v"], L.desc.lora_scale_k, L.desc.lora_scale_v, g.n_kv, softmax_scale, heads)


def _cache_tol(ref):
    # one bf16 rounding of an fp32-accumulated value
    return 2.0 ** -8 * np.abs(ref) + 1e-3


# ------------------------------------------------------------------ C1: the whole chain

def test_c1_chain_precompute_rebase_decode(px):
    geo = I.C1
    T = I.C1_T
    L = Layer(px, geo, seed=0, n_blocks=T // 16)
    H = I.hidden_states(T, geo, seed=0)
    L.append(H)
    torch.cuda.synchronize()
    Hn = f64(H)
    kb, vb = base_rows(L.cache.k_base), base_rows(L.cache.v_base)
    rk, rv = O.base_cache(Hn, L.w_np["W_k"]), O.base_cache(Hn, L.w_np["W_v"])
    assert (np.abs(kb - rk) <= _cache_tol(rk)).all() and (np.abs(vb - rv) <= _cache_tol(rv)).all()
    for a in range(geo.n_agents):
        for cache_t, A in ((L.cache.lr_k, L.w_np["A_k"]), (L.cache.lr_v, L.w_np["A_v"])):
            ref = O.lr_cache(Hn, A[a])
            assert (np.abs(lr_rows(cache_t, a) - ref) <= _cache_tol(ref)).all()
    q = I.queries(geo.n_agents, geo, seed=0)
    agent_id, ctx_len = [0, 1, 2], [T, T, T]
    out = L.decode(q, agent_id, ctx_len)
    ref = _ref_decode(L, H, q, agent_id, ctx_len)
    assert_close(f64(out), ref, "C1 decode")
    # sensitivity: the adapter term must be visible at this tolerance
    base_only = O.lr_decode_reference(f64(q), agent_id, ctx_len, Hn, L.w_np["W_k"], L.w_np["W_v"], L.w_np["A_k"],
                                      L.w_np["B_k"], L.w_np["A_v"], L.w_np["B_v"], 0.0, 0.0, geo.n_kv)
    assert (np.abs(f64(out) - base_only) > ATOL + RTOL * np.abs(base_only)).any()
    # peaked variant (larger logits): outputs are O(0.1..1), so the bar bites
    qp = I.queries(geo.n_agents, geo, seed=0, tag="L0.q.peaked", gain=4.0)
    assert_close(f64(L.decode(qp, agent_id, ctx_len)), _ref_decode(L, H, qp, agent_id, ctx_len), "C1 decode peaked")


SMALL = [
    # d, n_q, n_kv, hd, N, rk, rv, T, ctx list
    (256, 8, 2, 128, 3, 8, 8, 100, [100, 1, 37]),
    (256, 8, 2, 64, 2, 16, 16, 200, [200, 16, 17]),
    (128, 28, 4, 128, 3, 16, 16, 90, [90, 33, 64]),          # group of 7 (Qwen-like)
    (192, 8, 8, 64, 2, 0, 0, 50, [50, 49, 2]),               # no adapters: plain attention
    (192, 16, 4, 128, 2, 0, 32, 77, [77, 5, 48]),            # adapters on V only (paper default QV)
    (256, 4, 1, 128, 2, 64, 64, 130, [130, 129, 15]),
    (128, 4, 2, 64, 5, 32, 32, 48, [48, 47, 1]),
    (128, 2, 2, 64, 2, 0, 8, 33, [33, 32, 31]),
    (128, 6, 2, 128, 2, 0, 64, 70, [70, 3, 69]),
]


@pytest.mark.parametrize("cfg", SMALL, ids=lambda c: "d%d_q%d_kv%d_hd%d_N%d_r%d-%d_T%d" % c[:8])
def test_small_shapes_decode_and_prefill(px, cfg):
    d, n_q, n_kv, hd, N, rk, rv, T, ctxs = cfg
    geo = I.Geometry(d, n_q, n_kv, hd, N, rk, rv, alpha=2.0 * max(rk, rv, 1))
    nb = (T + 15) // 16 + 2
    L = Layer(px, geo, seed=7, n_blocks=nb, fill=float("nan"))   # unwritten slots hold NaN: must never leak
    H = I.hidden_states(T, geo, seed=7)
    L.append(H)
    agent_id = [i % N for i in range(len(ctxs))]
    q = I.queries(len(ctxs), geo, seed=7, gain=2.0)
    out = L.decode(q, agent_id, ctxs)
    assert_close(f64(out), _ref_decode(L, H, q, agent_id, ctxs), "decode")
    # new-turn prefill: last S tokens are the turn
    S = min(T - 1, 21)
    Tc = T - S
    qs = I.queries(S, geo, seed=7, tag="q.turn", gain=2.0)
    w = L.w_np
    for agent in range(min(N, 2)):
        got = L.prefill(qs, agent, Tc)
        ref = O.lr_prefill_reference(f64(qs), agent, Tc, f64(H), w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"],
                                     L.desc.lora_scale_k, L.desc.lora_scale_v, n_kv)
        assert_close(f64(got), ref, f"prefill agent {agent}")


def test_softmax_scale_and_lora_scales_are_honoured(px):
    geo = I.Geometry(128, 4, 2, 64, 2, 16, 16, alpha=32.0)
    H = I.hidden_states(40, geo, seed=3)
    q = I.queries(2, geo, seed=3, gain=2.0)
    L = Layer(px, geo, seed=3, n_blocks=3, softmax_scale=0.31, scale_k=0.5, scale_v=3.0)
    L.append(H)
    out = L.decode(q, [0, 1], [40, 40])
    assert_close(f64(out), _ref_decode(L, H, q, [0, 1], [40, 40], softmax_scale=0.31), "custom scales")
    L1 = Layer(px, geo, seed=3, n_blocks=3, scale_k=1.0, scale_v=1.0)     # Eq. 1 literally
    L1.append(H)
    assert_close(f64(L1.decode(q, [0, 1], [40, 40])), _ref_decode(L1, H, q, [0, 1], [40, 40]), "s = 1")


def test_decode_many_splits_long_context(px):
    geo = I.Geometry(128, 8, 2, 128, 2, 16, 16, alpha=32.0)
    T = 6000 + 5
    L = Layer(px, geo, seed=11, n_blocks=(T + 15) // 16)
    H = I.hidden_states(T, geo, seed=11)
    L.append(H)
    q = I.queries(3, geo, seed=11, gain=4.0)
    ctx = [T, 4097, 333]
    assert_close(f64(L.decode(q, [1, 0, 1], ctx)), _ref_decode(L, H, q, [1, 0, 1], ctx), "long decode")
    # closed forms through the whole GPU path: q = 0 gives the mean adapted value row
    q0 = torch.zeros_like(q)
    out0 = f64(L.decode(q0, [1, 0, 1], ctx))
    w = L.w_np
    for b, a in enumerate([1, 0, 1]):
        mean_v = f64(H)[:ctx[b]].mean(0) @ (w["W_v"] + geo.scale_v * w["A_v"][a] @ w["B_v"][a])
        for h in range(geo.n_q):
            g = h // geo.group
            np.testing.assert_allclose(out0[b, h], mean_v[g * geo.hd:(g + 1) * geo.hd], atol=5e-3, rtol=2e-2)


def test_decode_is_deterministic_and_workspace_reusable(px):
    geo = I.Geometry(128, 8, 2, 64, 2, 8, 8, alpha=16.0)
    T = 3000
    L = Layer(px, geo, seed=5, n_blocks=(T + 15) // 16)
    L.append(I.hidden_states(T, geo, seed=5))
    q = I.queries(2, geo, seed=5)
    ws = px.decode_workspace(L.desc, 2, T)
    outs = [L.decode(q, [0, 1], [T, 1234], max_ctx=T, ws=ws) for _ in range(3)]
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])


# ------------------------------------------------------------------ paging: bit-exact

def test_paged_equals_contiguous_bitwise(px):
    geo = I.Geometry(256, 8, 2, 128, 3, 16, 16, alpha=32.0)
    ctx = [700, 50, 333]
    T = max(ctx)
    nb_seq = (T + 15) // 16
    H = I.hidden_states(T, geo, seed=21)
    q = I.queries(3, geo, seed=21)
    # contiguous: one shared sequence starting at block 0
    Lc = Layer(px, geo, seed=21, n_blocks=nb_seq)
    Lc.append(H)
    ref = Lc.decode(q, [0, 1, 2], ctx, max_ctx=T)
    # paged: same rows scattered over a larger pool through a random block permutation
    pool = 3 * nb_seq
    perm = I.permutation(pool, 21, "perm")[:nb_seq]
    slots = (perm.long()[:, None] * 16 + torch.arange(16)[None, :]).reshape(-1)[:T].to(torch.int32).cuda()
    Lp = Layer(px, geo, seed=21, n_blocks=pool, fill=float("nan"))
    Lp.append(H, slot_mapping=slots)
    table = perm.view(1, -1).repeat(3, 1).contiguous()
    got = Lp.decode(q, [0, 1, 2], ctx, max_ctx=T, block_table=table)
    assert torch.equal(got, ref)
    # written rows are bit-identical to the contiguous write, all other slots keep their fill
    tok = lambda c: c.permute(0, 2, 1, 3).reshape(-1, geo.kv_width)[:T].view(torch.int16)
    pidx = perm.long().cuda()
    assert torch.equal(tok(Lp.cache.k_base[pidx]), tok(Lc.cache.k_base))
    assert torch.equal(tok(Lp.cache.v_base[pidx]), tok(Lc.cache.v_base))
    for a in range(geo.n_agents):
        assert torch.equal(Lp.cache.lr_k[a][pidx].reshape(-1, 16)[:T].view(torch.int16),
                           Lc.cache.lr_k[a].reshape(-1, 16)[:T].view(torch.int16))
    untouched = torch.ones(pool, dtype=torch.bool)
    untouched[perm.long()] = False
    assert torch.isnan(Lp.cache.k_base[untouched.cuda()]).all() and torch.isnan(Lp.cache.lr_v[:, untouched.cuda()]).all()
    # the tail of the last block (slots >= T) is untouched too
    last = int(perm[-1])
    assert torch.isnan(Lp.cache.v_base[last, :, T % 16:]).all()
    # first_block addressing: the same sequence placed at an offset inside a bigger contiguous cache
    Lo = Layer(px, geo, seed=21, n_blocks=nb_seq + 9)
    Lo.append(H, start_slot=5 * 16)
    got2 = Lo.decode(q, [0, 1, 2], ctx, max_ctx=T, first_block=[5, 5, 5])
    assert torch.equal(got2, ref)
    # prefill: paged == contiguous, bitwise
    qs = I.queries(40, geo, seed=21, tag="turn")
    assert torch.equal(Lp.prefill(qs, 1, T - 40, block_table=perm), Lc.prefill(qs, 1, T - 40))
    assert torch.equal(Lo.prefill(qs, 1, T - 40, first_block=5), Lc.prefill(qs, 1, T - 40))


def test_agent_isolation_bitwise_and_agent_mask(px):
    geo = I.Geometry(128, 8, 2, 64, 3, 16, 16, alpha=32.0)
    T = 150
    H = I.hidden_states(T, geo, seed=9)
    q = I.queries(1, geo, seed=9)
    L = Layer(px, geo, seed=9, n_blocks=10)
    L.append(H)
    ref = L.decode(q, [1], [T])
    # clobber the other agents' LR caches and B matrices: agent 1's result must not move a bit
    for a in (0, 2):
        L.cache.lr_k[a].fill_(float("nan")); L.cache.lr_v[a].fill_(float("nan"))
        L.B_k[a].fill_(float("nan")); L.B_v[a].fill_(float("nan"))
    assert torch.equal(L.decode(q, [1], [T]), ref)
    # agent mask: write only agents 0 and 2 -> agent 1's rows keep their fill
    L2 = Layer(px, geo, seed=9, n_blocks=10, fill=float("nan"))
    L2.append(H, agent_mask=0b101)
    torch.cuda.synchronize()
    rows = slice(0, (T + 15) // 16)
    assert torch.isnan(L2.cache.lr_k[1]).all() and torch.isnan(L2.cache.lr_v[1]).all()
    assert torch.isfinite(L2.cache.lr_k[0].reshape(-1, 16)[:T]).all() and torch.isfinite(L2.cache.lr_v[2].reshape(-1, 16)[:T]).all()


def test_rebase_overwrites_segment_and_identity(px):
    geo = I.Geometry(256, 8, 2, 128, 2, 8, 8, alpha=16.0)
    T, S = 96, 40
    H = I.hidden_states(T, geo, seed=13)
    L = Layer(px, geo, seed=13, n_blocks=6)
    L.append(H)
    torch.cuda.synchronize()
    before_k, before_lr = L.cache.k_base.clone(), L.cache.lr_k.clone()
    # re-projecting the same hidden states leaves the cache unchanged: bitwise when the row count takes the
    # same kernel (T = 96 rows: tiled GEMM), within one bf16 rounding step when it does not (S = 40 rows take
    # the few-row split-K kernel, whose fp32 summation order differs)
    L.px.rebase_project(L.desc, H.cuda(), L.W_packed, L.cache, 0)
    torch.cuda.synchronize()
    assert torch.equal(L.cache.k_base, before_k)
    L.px.rebase_project(L.desc, H[T - S:].cuda(), L.W_packed, L.cache, T - S)
    torch.cuda.synchronize()
    a, b = L.cache.k_base.float(), before_k.float()
    assert ((a - b).abs() <= 2.0 ** -7 * b.abs() + 1e-6).all()
    L.cache.k_base.copy_(before_k)
    # adapter-free pass over the turn: base rows and the other agent's LR rows are rebuilt from X_neut,
    # the current agent's LR rows stay as they were (Section 3.2)
    X_neut = I.hidden_states(S, geo, seed=13, tag="neut")
    cur = 1
    L.px.rebase_project(L.desc, X_neut.cuda(), L.W_packed, L.cache, T - S)
    L.px.lr_precompute(L.desc, X_neut.cuda(), L.A_packed, L.cache, T - S, None, ~(1 << cur))
    torch.cuda.synchronize()
    kb = base_rows(L.cache.k_base)
    ref_new = O.base_cache(f64(X_neut), L.w_np["W_k"])
    assert (np.abs(kb[T - S:T] - ref_new) <= _cache_tol(ref_new)).all()
    assert torch.equal(L.cache.k_base.permute(0, 2, 1, 3).reshape(-1, 256)[:T - S],
                       before_k.permute(0, 2, 1, 3).reshape(-1, 256)[:T - S])
    assert torch.equal(L.cache.lr_k[cur], before_lr[cur])
    ref_lr = O.lr_cache(f64(X_neut), L.w_np["A_k"][0])
    assert (np.abs(lr_rows(L.cache.lr_k, 0)[T - S:T] - ref_lr) <= _cache_tol(ref_lr)).all()
    # token-by-token writes (double-batching order) == one segment write (lazy-prefill order), bitwise
    L2 = Layer(px, geo, seed=13, n_blocks=6)
    L2.append(H)
    for t in range(S):
        L2.px.rebase_project(L2.desc, X_neut[t:t + 1].cuda(), L2.W_packed, L2.cache, T - S + t)
    torch.cuda.synchronize()
    assert torch.equal(L2.cache.k_base, L.cache.k_base) and torch.equal(L2.cache.v_base, L.cache.v_base)


def test_prefill_row_matches_decode(px):
    geo = I.Geometry(256, 8, 2, 128, 2, 16, 16, alpha=32.0)
    T, S = 200, 70
    H = I.hidden_states(T + S, geo, seed=17)
    L = Layer(px, geo, seed=17, n_blocks=(T + S + 15) // 16)
    L.append(H)
    qs = I.queries(S, geo, seed=17, gain=3.0)
    pre = f64(L.prefill(qs, 0, T))
    for i in (0, 1, 15, 16, 17, S - 1):
        dec = f64(L.decode(qs[i:i + 1], [0], [T + i + 1]))[0]
        np.testing.assert_allclose(pre[i], dec, atol=1e-2, rtol=2e-2)


# ------------------------------------------------------------------ fused projection, adapter-free view

def test_turn_project_equals_the_two_separate_projections_bitwise(px):
    geo = I.Geometry(256, 8, 2, 128, 3, 16, 16, alpha=32.0)
    T = 200
    H = I.hidden_states(T, geo, seed=31)
    La = Layer(px, geo, seed=31, n_blocks=14, fill=float("nan"))
    La.append(H, start_slot=16, agent_mask=0b101)
    Lb = Layer(px, geo, seed=31, n_blocks=14, fill=float("nan"))
    dev = {k: v.cuda() for k, v in Lb.w.items()}
    WA = px.pack_turn_weights(geo, dev["W_k"], dev["W_v"], dev["A_k"], dev["A_v"])
    px.turn_project(Lb.desc, H.cuda(), WA, Lb.cache, 16, None, 0b101)
    torch.cuda.synchronize()
    for name in ("k_base", "v_base", "lr_k", "lr_v"):
        a, b = getattr(La.cache, name).view(torch.int16), getattr(Lb.cache, name).view(torch.int16)
        assert torch.equal(a, b), name


@pytest.mark.parametrize("M", [1, 7, 16, 17, 33, 64])
@pytest.mark.parametrize("d,hd,n_kv", [(192, 64, 2), (1024, 128, 2), (4096, 128, 1)])
def test_few_row_projection_kernel(px, M, d, hd, n_kv):
    """Decode-step projections (M <= 64 rows) take the weight-streaming split-K kernel: every mode against
    the definition, scattered slots, agent mask, and the fused call bit-equal to the two separate ones."""
    geo = I.Geometry(d, 2 * n_kv, n_kv, hd, 3, 16, 16, alpha=32.0)
    H = I.hidden_states(M, geo, seed=41, tag=f"few.{M}.{d}")
    nb = 12
    slots = I.permutation(nb * 16, 41, f"few.slots.{M}")[:M].to(torch.int32)
    La = Layer(px, geo, seed=41, n_blocks=nb, fill=float("nan"))
    La.append(H, slot_mapping=slots.cuda(), agent_mask=0b110)
    torch.cuda.synchronize()
    w, Hn = La.w_np, f64(H)
    sl = slots.long()
    kb = base_rows(La.cache.k_base)[sl]
    vb = base_rows(La.cache.v_base)[sl]
    for got, ref in ((kb, O.base_cache(Hn, w["W_k"])), (vb, O.base_cache(Hn, w["W_v"])),
                     (lr_rows(La.cache.lr_k, 1)[sl], O.lr_cache(Hn, w["A_k"][1])),
                     (lr_rows(La.cache.lr_v, 2)[sl], O.lr_cache(Hn, w["A_v"][2]))):
        assert (np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 2e-3 * np.sqrt(d / 256)).all()
    assert torch.isnan(La.cache.lr_k[0]).all()                     # masked-out agent untouched
    untouched = torch.ones(nb * 16, dtype=torch.bool); untouched[sl] = False
    assert torch.isnan(La.cache.k_base.permute(0, 2, 1, 3).reshape(nb * 16, -1)[untouched]).all()
    Lb = Layer(px, geo, seed=41, n_blocks=nb, fill=float("nan"))
    dev = {k: v.cuda() for k, v in Lb.w.items()}
    WA = px.pack_turn_weights(geo, dev["W_k"], dev["W_v"], dev["A_k"], dev["A_v"])
    px.turn_project(Lb.desc, H.cuda(), WA, Lb.cache, 0, slots.cuda(), 0b110)
    torch.cuda.synchronize()
    for name in ("k_base", "v_base", "lr_k", "lr_v"):
        a, b = getattr(La.cache, name).view(torch.int16), getattr(Lb.cache, name).view(torch.int16)
        assert torch.equal(a, b), name


def test_adapter_free_view_in_a_mixed_batch(px):
    """Double batching: adapted requests and adapter-free requests (agent id -1) in one launch."""
    geo = I.Geometry(256, 8, 2, 128, 2, 16, 16, alpha=32.0)
    T = 333
    H = I.hidden_states(T, geo, seed=33)
    L = Layer(px, geo, seed=33, n_blocks=(T + 15) // 16)
    L.append(H)
    L.cache.lr_k[1].fill_(float("nan"))          # the neutral requests must never touch an LR row
    q = I.queries(4, geo, seed=33, gain=2.0)
    agent_id, ctx = [0, -1, 0, -1], [T, T, 100, 17]
    out = f64(L.decode(q, agent_id, ctx))
    w = L.w_np
    args = (f64(H), w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"])
    adapted = O.lr_decode_reference(f64(q), [0, 0, 0, 0], ctx, *args, geo.scale_k, geo.scale_v, geo.n_kv)
    neutral = O.lr_decode_reference(f64(q), [0, 0, 0, 0], ctx, *args, 0.0, 0.0, geo.n_kv)
    assert_close(out[[0, 2]], adapted[[0, 2]], "adapted requests")
    assert_close(out[[1, 3]], neutral[[1, 3]], "adapter-free requests")
    # prefill: agent -1 is plain attention over the base cache
    qs = I.queries(30, geo, seed=33, tag="turn", gain=2.0)
    got = f64(L.prefill(qs, -1, T - 30))
    ref = O.lr_prefill_reference(f64(qs), 0, T - 30, *args, 0.0, 0.0, geo.n_kv)
    assert_close(got, ref, "adapter-free prefill")
    # a long, split context too (cluster path for the adapted one, same launch)
    T2 = 3000
    H2 = I.hidden_states(T2, geo, seed=34)
    L2 = Layer(px, geo, seed=34, n_blocks=(T2 + 15) // 16)
    L2.append(H2)
    q2 = I.queries(2, geo, seed=34, gain=3.0)
    out2 = f64(L2.decode(q2, [-1, 1], [T2, T2]))
    a2 = (f64(H2), L2.w_np["W_k"], L2.w_np["W_v"], L2.w_np["A_k"], L2.w_np["B_k"], L2.w_np["A_v"], L2.w_np["B_v"])
    assert_close(out2[:1], O.lr_decode_reference(f64(q2[:1]), [0], [T2], *a2, 0.0, 0.0, geo.n_kv), "neutral long")
    assert_close(out2[1:], O.lr_decode_reference(f64(q2[1:]), [1], [T2], *a2, geo.scale_k, geo.scale_v, geo.n_kv), "adapted long")


# ------------------------------------------------------------------ host-side validation

def test_invalid_arguments_are_rejected_without_launch(px):
    geo = I.Geometry(128, 8, 2, 64, 2, 16, 16, alpha=32.0)
    L = Layer(px, geo, seed=1, n_blocks=4, fill=7.0)
    H = I.hidden_states(32, geo, seed=1).cuda()
    snapshot = L.cache.k_base.clone()
    with pytest.raises(PreccError, match="INVALID_ARG"):
        px.rebase_project(L.desc, H, L.W_packed, L.cache, start_slot=4 * 16 - 8)      # runs past the cache
    with pytest.raises(PreccError, match="MISALIGNED"):
        px.rebase_project(L.desc, H.view(-1)[1:1 + 31 * 128].view(31, 128), L.W_packed, L.cache)
    bad = I.Geometry(128, 8, 2, 96, 2, 16, 16, alpha=32.0)
    from paper_2609_34054_b200.binding import layer_desc
    with pytest.raises(PreccError, match="UNSUPPORTED"):
        px.rebase_project(layer_desc(bad), H, L.W_packed, L.cache)
    with pytest.raises(PreccError, match="UNSUPPORTED"):
        px.lr_precompute(layer_desc(I.Geometry(128, 8, 2, 64, 2, 16, 8, alpha=1.0)), H, L.A_packed, L.cache)
    q = I.queries(1, geo, seed=1).cuda()
    out = torch.zeros_like(q)
    aid = torch.zeros(1, dtype=torch.int32, device="cuda"); cl = torch.full((1,), 32, dtype=torch.int32, device="cuda")
    tiny_ws = torch.zeros(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(PreccError, match="WORKSPACE"):
        px.lr_attend_decode(L.desc, q, aid, cl, 32, L.B_k, L.B_v, L.cache, out, tiny_ws)
    with pytest.raises(PreccError, match="INVALID_ARG"):
        px.lr_attend_prefill(L.desc, q, 5, 10, L.B_k, L.B_v, L.cache, out)             # agent out of range
    torch.cuda.synchronize()
    assert torch.equal(L.cache.k_base, snapshot) and (out == 0).all()
    # empty problems are no-ops
    px.rebase_project(L.desc, H[:0], L.W_packed, L.cache)
    px.lr_precompute(L.desc, H[:0], L.A_packed, L.cache)
    assert px.poll_status() == 0


def test_device_side_bad_indices_are_flagged_not_fatal(px):
    geo = I.Geometry(128, 8, 2, 64, 2, 16, 16, alpha=32.0)
    L = Layer(px, geo, seed=2, n_blocks=4, fill=1.0)
    H = I.hidden_states(16, geo, seed=2).cuda()
    slots = torch.arange(16, dtype=torch.int32)
    slots[3] = 10_000                   # outside the cache: skipped and recorded
    px.rebase_project(L.desc, H, L.W_packed, L.cache, 0, slots.cuda())
    assert px.poll_status() & 1
    assert (L.cache.k_base[0, :, 3] == 1.0).all()
    q = I.queries(2, geo, seed=2)
    out = L.decode(q, [0, 9], [16, 16])  # agent 9 does not exist: zeros + flag (-1 would be the adapter-free view)
    assert px.poll_status() & 1
    assert (out[1] == 0).all() and torch.isfinite(out[0]).all()
    assert px.poll_status() == 0


@pytest.mark.parametrize("B,T", [(2, 4096), (40, 1200)])     # the cluster kernel and the ticket kernel
def test_context_longer_than_the_host_bound_is_flagged_and_the_workspace_stays_usable(px, B, T):
    """ctx_len is device data; the host's max_ctx sized the grid, the split and the block table.  A request whose
    ctx_len exceeds it is rejected on the device like a bad agent id: zeros, BAD_INDEX, and the workspace is left
    ready, so the next call on it is correct."""
    geo = I.Geometry(256, 8, 2, 64, 2, 16, 16, alpha=32.0)
    nb = (T + 15) // 16
    c = I.direct_caches(nb, geo, 61, "over")
    from paper_2609_34054_b200.binding import Cache, layer_desc
    cache = Cache.from_tensors(geo, c["k_base"].cuda(), c["v_base"].cuda(), c["lr_k"].cuda(), c["lr_v"].cuda())
    w = I.layer_weights(geo, 61, "over")
    desc = layer_desc(geo)
    q = I.queries(B, geo, 61, "over.q").cuda()
    aid = torch.tensor([i % 2 for i in range(B)], dtype=torch.int32).cuda()
    good = torch.full((B,), T - 3, dtype=torch.int32)
    bad = good.clone()
    bad[1] = 8 * T                                        # far beyond max_ctx (and beyond the cache)
    ws = px.decode_workspace(desc, B, T)
    Bk, Bv = w["B_k"].cuda(), w["B_v"].cuda()
    ref = torch.full_like(q, float("nan"))
    px.lr_attend_decode(desc, q, aid, good.cuda(), T, Bk, Bv, cache, ref, ws)
    assert px.poll_status() == 0
    out = torch.full_like(q, float("nan"))
    px.lr_attend_decode(desc, q, aid, bad.cuda(), T, Bk, Bv, cache, out, ws)
    assert px.poll_status() & 1
    assert (out[1] == 0).all()
    keep = [i for i in range(B) if i != 1]
    assert torch.equal(out[keep], ref[keep])
    again = torch.full_like(q, float("nan"))
    px.lr_attend_decode(desc, q, aid, good.cuda(), T, Bk, Bv, cache, again, ws)      # same workspace, no re-init
    assert px.poll_status() == 0
    assert torch.equal(again, ref)


@pytest.mark.parametrize("M", [1, 7, 40])
def test_decode_launched_right_behind_the_append_of_its_newest_tokens(px, M):
    """Decode starts fetching a request's older pages while the kernel before it on the stream - here the few-row
    projection that appends the M newest tokens (Section 3.1: in-turn append) - may still be running.  The result
    must be bit-equal to running the two one after the other, for every one of many back-to-back repetitions with
    changing rows (a race on the appended rows, on q or on the output would show as a stale value)."""
    geo = I.Geometry(512, 32, 8, 64, 4, 16, 16, alpha=32.0)
    T = 4096 + 21
    L = Layer(px, geo, seed=77, n_blocks=(T + 15) // 16)
    dev = {k: v.cuda() for k, v in L.w.items()}
    WA = px.pack_turn_weights(geo, dev["W_k"], dev["W_v"], dev["A_k"], dev["A_v"])
    L.append(I.hidden_states(T, geo, 77, "pdl.H"))
    ws = px.decode_workspace(L.desc, 1, T)
    aid = torch.tensor([2], dtype=torch.int32).cuda()
    cl = torch.tensor([T], dtype=torch.int32).cuda()
    trials = 12
    Hn = [I.hidden_states(M, geo, 100 + i, "pdl.new").cuda() for i in range(trials)]
    qs = [I.queries(1, geo, 100 + i, "pdl.q", gain=3.0).cuda() for i in range(trials)]
    ref = []
    for i in range(trials):                                   # serialised order
        px.turn_project(L.desc, Hn[i], WA, L.cache, T - M)
        torch.cuda.synchronize()
        o = torch.full_like(qs[i], float("nan"))
        px.lr_attend_decode(L.desc, qs[i], aid, cl, T, L.B_k, L.B_v, L.cache, o, ws)
        torch.cuda.synchronize()
        ref.append(o)
    assert not torch.equal(ref[0], ref[1])
    got = [torch.full_like(qs[i], float("nan")) for i in range(trials)]
    for i in range(trials):                                   # back to back, nothing in between
        px.turn_project(L.desc, Hn[i], WA, L.cache, T - M)
        px.lr_attend_decode(L.desc, qs[i], aid, cl, T, L.B_k, L.B_v, L.cache, got[i], ws)
    torch.cuda.synchronize()
    for i in range(trials):
        assert torch.equal(got[i], ref[i]), f"repetition {i}"
    assert px.poll_status() == 0


@pytest.mark.parametrize("B,hd,n_kv", [(3, 64, 8), (5, 64, 8), (6, 128, 8), (9, 128, 4), (2, 128, 5)])
def test_decode_cluster_sizes_that_do_not_divide_the_head_dimension(px, B, hd, n_kv):
    """Few requests, long contexts: the splits of a (request, kv head) form a cluster of as many blocks as fit
    the machine in one wave (6, 3, 3, 4, 14 here), each finishing a slice of the output columns; the slices
    are uneven when the cluster size does not divide head_dim."""
    geo = I.Geometry(1024, 2 * n_kv, n_kv, hd, 3, 16, 16, alpha=32.0)
    T = 4096 + 16 * B + 5
    nb = (T + 15) // 16
    c = I.direct_caches(nb, geo, 51, f"cl.{B}")
    from paper_2609_34054_b200.binding import Cache, layer_desc
    cache = Cache.from_tensors(geo, c["k_base"].cuda(), c["v_base"].cuda(), c["lr_k"].cuda(), c["lr_v"].cuda())
    w = I.layer_weights(geo, 51, "cl")
    desc = layer_desc(geo)
    q = I.queries(B, geo, 51, f"cl.q{B}", gain=4.0)
    agents = [i % 3 for i in range(B)]
    ctx = [T - 37 * i for i in range(B)]
    out = torch.full_like(q, float("nan"), device="cuda")
    ws = px.decode_workspace(desc, B, T)
    args = (desc, q.cuda(), torch.tensor(agents, dtype=torch.int32).cuda(), torch.tensor(ctx, dtype=torch.int32).cuda(), T,
            w["B_k"].cuda(), w["B_v"].cuda(), cache, out, ws)
    px.lr_attend_decode(*args)
    torch.cuda.synchronize()
    first = out.clone()
    px.lr_attend_decode(*args)
    torch.cuda.synchronize()
    assert torch.equal(first, out)                                   # deterministic
    G = geo.group
    for b, g in ((0, 0), (B - 1, n_kv - 1), (B // 2, n_kv // 2)):
        t, a = ctx[b], agents[b]
        rows = lambda x: f64(x.reshape(-1, x.shape[-1]))[:t]
        cols = slice(g * hd, (g + 1) * hd)
        ref = O.attend_from_caches(f64(q[b, g * G:(g + 1) * G]), rows(c["k_base"][:, g]), rows(c["v_base"][:, g]),
                                   rows(c["lr_k"][a]), rows(c["lr_v"][a]), f64(w["B_k"][a][:, cols]), f64(w["B_v"][a][:, cols]),
                                   geo.scale_k, geo.scale_v, 1)
        assert_close(f64(out)[b, g * G:(g + 1) * G], ref, f"B={B} request {b} head {g}")


def test_one_workspace_serves_every_smaller_batch_and_context(px):
    """The workspace query is an upper bound: a buffer sized for (max_batch, max_ctx) must be accepted for any
    batch <= max_batch and any max_ctx below (smaller batches split each request further, so the need is not
    monotone in the batch size)."""
    geo = I.Geometry(256, 8, 2, 128, 2, 16, 16, alpha=32.0)
    T = 40000
    L = Layer(px, geo, seed=61, n_blocks=T // 16 + 1, fill=0.0)
    ws = px.decode_workspace(L.desc, 8, T)
    from paper_2609_34054_b200.binding import load_library
    import ctypes
    lib = load_library()
    q8 = I.queries(8, geo, 61, "ws.q").cuda()
    for B in (1, 2, 3, 5, 8):
        for ctx in (T, 33333, 8200, 4096, 100, 1):
            assert lib.precc_decode_workspace_bytes(ctypes.byref(L.desc), B, ctx, px.sm_count) <= ws.numel()
            out = torch.empty_like(q8[:B])
            px.lr_attend_decode(L.desc, q8[:B], torch.zeros(B, dtype=torch.int32, device="cuda"),
                                torch.full((B,), ctx, dtype=torch.int32, device="cuda"), ctx, L.B_k, L.B_v, L.cache, out, ws,
                                None, torch.zeros(B, dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    assert px.poll_status() == 0


@pytest.mark.parametrize("hd,n_q,n_kv,r,T,S,agent", [(128, 8, 2, 32, 2100, 40, 1), (128, 8, 2, 16, 4200, 33, 0), (64, 16, 4, 16, 9000, 20, 1),
                                                       (128, 8, 2, 32, 8300, 64, -1), (64, 8, 1, 32, 5000, 130, 0),
                                                       (128, 8, 2, 8, 3000, 50, 1), (128, 8, 2, 64, 4100, 45, 1), (64, 8, 2, 64, 2600, 70, 0),
                                                       (128, 16, 2, 64, 300, 500, 1)])
def test_prefill_short_turn_over_long_context_is_split_over_a_cluster(px, hd, n_q, n_kv, r, T, S, agent):
    """Few (row tile, kv head) blocks and many 128-token steps: the context is split over a cluster of 2, 4 or
    8 blocks and merged over distributed shared memory.  Against the definition, and bit-identical runs."""
    geo = I.Geometry(256, n_q, n_kv, hd, 2, r, r, alpha=2.0 * r)
    L = Layer(px, geo, seed=71, n_blocks=(T + S + 15) // 16, tag="sp")
    H = I.hidden_states(T + S, geo, 71, "sp.H")
    L.append(H)
    qs = I.queries(S, geo, 71, "sp.q", gain=4.0)
    got = L.prefill(qs, agent, T)
    again = L.prefill(qs, agent, T)
    assert torch.equal(got, again)
    w = L.w_np
    rows = sorted(set([0, 1, S // 2, S - 2, S - 1]))
    a = max(agent, 0)
    sk, sv = (geo.scale_k, geo.scale_v) if agent >= 0 else (0.0, 0.0)
    ref = O.lr_prefill_reference(f64(qs), a, T, f64(H), w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"], sk, sv, n_kv,
                                 rows=rows)
    assert_close(f64(got), ref, f"split prefill hd{hd} T{T} S{S}")


@pytest.mark.parametrize("hd,n_q,n_kv,r,T,S,agent,paged", [(128, 8, 2, 64, 2100, 40, 1, True), (128, 16, 2, 64, 1000, 260, 0, False),
                                                             (128, 8, 2, 64, 515, 130, 1, True), (128, 4, 2, 64, 77, 300, 1, False),
                                                             (128, 8, 2, 64, 8300, 64, 0, False)])
def test_prefill_value_ring_in_half_steps_is_bit_identical(monkeypatch, hd, n_q, n_kv, r, T, S, agent, paged):
    """Where shared memory holds one value stage but not two (head_dim 128, rank 64) the value ring works in units
    of 64 tokens.  The same MMAs in the same order: bit-identical to whole-step stages (the switch selects them),
    on contexts that end inside a unit, paged and contiguous, one block per tile and split over a cluster."""
    monkeypatch.setenv("PRECC_PREFILL_VHALF", "0")
    p_whole = Precc(0)
    monkeypatch.delenv("PRECC_PREFILL_VHALF")
    p_half = Precc(0)
    geo = I.Geometry(256, n_q, n_kv, hd, 2, r, r, alpha=2.0 * max(r, 1))
    nb = (T + S + 15) // 16
    L = Layer(p_half, geo, seed=75, n_blocks=nb + 5, tag="vh")
    H = I.hidden_states(T + S, geo, 75, "vh.H")
    bt = None
    if paged:
        bt = I.permutation(nb + 5, 75, "vh.perm")[:nb].to(torch.int32)
        slots = (bt.long()[:, None] * 16 + torch.arange(16)[None, :]).reshape(-1)[:T + S].to(torch.int32).cuda()
        L.append(H, slot_mapping=slots)
    else:
        L.append(H)
    qs = I.queries(S, geo, 75, "vh.q", gain=4.0)
    got = L.prefill(qs, agent, T, bt)
    ref = torch.full_like(got, float("nan"))
    p_whole.lr_attend_prefill(L.desc, qs.cuda(), agent, T, L.B_k, L.B_v, L.cache, ref, None if bt is None else bt.cuda(), 0)
    torch.cuda.synchronize()
    assert torch.equal(got, ref)
    w = L.w_np
    rows = sorted(set([0, S // 2, S - 1]))
    a = max(agent, 0)
    sk, sv = (geo.scale_k, geo.scale_v) if agent >= 0 and r else (0.0, 0.0)
    want = O.lr_prefill_reference(f64(qs), a, T, f64(H), w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"], sk, sv, n_kv,
                                  rows=rows)
    assert_close(f64(got), want, f"half-step value ring hd{hd} r{r} T{T} S{S}")
    assert p_half.poll_status() == 0


# (head_dim, q heads, kv heads, rank, context, new tokens, agent, paged): between 75 and 144 (row tile, kv head) blocks
_HELPER_CASES = [(128, 32, 8, 32, 1500, 384, 1, False), (64, 32, 8, 16, 2300, 512, 0, True), (128, 32, 8, 64, 1300, 300, 1, False),
                 (128, 32, 8, 8, 1100, 528, -1, False), (64, 16, 8, 0, 2000, 700, 0, True), (128, 28, 4, 16, 1800, 400, 1, False)]


@pytest.mark.parametrize("hd,n_q,n_kv,r,T,S,agent,paged", _HELPER_CASES)
def test_prefill_with_a_workspace_puts_helper_blocks_on_idle_sms(monkeypatch, hd, n_q, n_kv, r, T, S, agent, paged):
    """One wave that leaves SMs idle: with a workspace every block stops short of its context's end and helper
    blocks take the tails, several tile pieces each; the pieces meet through records in the workspace.  Against
    the definition on rows at both ends of the turn and at tile borders, bit-identical from run to run, the
    workspace reusable without clearing, and within rounding of the launch without a workspace."""
    monkeypatch.setenv("PRECC_PREFILL_HELPER_MIN", "8")          # contexts the oracle finishes in seconds qualify:
    n_steps = (T + S + 127) // 128                               # there the planner sees no gain, so the cut is given
    monkeypatch.setenv("PRECC_PREFILL_HELPER_P", str(n_steps - 5))
    p2 = Precc(0)
    geo = I.Geometry(256, n_q, n_kv, hd, 2, r, r, alpha=2.0 * max(r, 1))
    nb = (T + S + 15) // 16
    L = Layer(p2, geo, seed=73, n_blocks=nb + 7, tag="hw")
    H = I.hidden_states(T + S, geo, 73, "hw.H")
    bt = None
    if paged:
        perm = I.permutation(nb + 7, 73, "hw.perm")[:nb].to(torch.int32)
        slots = (perm.long()[:, None] * 16 + torch.arange(16)[None, :]).reshape(-1)[:T + S].to(torch.int32).cuda()
        L.append(H, slot_mapping=slots)
        bt = perm
    else:
        L.append(H)
    qs = I.queries(S, geo, 73, "hw.q", gain=4.0)
    nbytes = p2.prefill_ws_bytes(L.desc, S)
    assert nbytes > 0
    ws = torch.full((nbytes,), 0xA5, dtype=torch.uint8, device="cuda")     # contents on entry do not matter
    got = L.prefill_ws(qs, agent, T, ws, bt)
    again = L.prefill_ws(qs, agent, T, ws, bt)                             # the same workspace, not cleared
    assert torch.equal(got, again)
    plain = L.prefill(qs, agent, T, bt)
    assert not torch.equal(got, plain)                                     # the helper blocks did run: another summation order
    tol = 2e-2 + 1e-2 * plain.float().abs()
    assert ((got.float() - plain.float()).abs() <= tol).all()
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")            # too small a workspace: the plain launch, bit for bit
    assert torch.equal(L.prefill_ws(qs, agent, T, small, bt), plain)
    assert torch.equal(L.prefill_ws(qs, agent, T, None, bt), plain)
    with pytest.raises(PreccError, match="MISALIGNED|aligned"):
        L.prefill_ws(qs, agent, T, ws[16:], bt)                            # a workspace must start on a 256-byte boundary
    w = L.w_np
    tpt = 128 // geo.group
    rows = sorted(set([0, 1, tpt - 1, tpt, S // 2, S - tpt, S - 2, S - 1]))
    a = max(agent, 0)
    sk, sv = (geo.scale_k, geo.scale_v) if agent >= 0 and r else (0.0, 0.0)
    ref = O.lr_prefill_reference(f64(qs), a, T, f64(H), w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"], sk, sv, n_kv,
                                 rows=rows)
    assert_close(f64(got), ref, f"helper prefill hd{hd} T{T} S{S}")
    assert p2.poll_status() == 0


@pytest.mark.parametrize("n", [1, 10, 100])
def test_per_row_agent_masks_equal_two_separate_projections(px, n):
    """Double batching: adapted rows (current agent's LR rows, private slots) and adapter-free rows (the other
    agents' LR rows, shared slots) in one fused projection, bit-equal to one call per sequence."""
    geo = I.Geometry(256, 8, 2, 128, 3, 16, 16, alpha=32.0)
    nb = 40
    cur = 1
    others = 0b111 & ~(1 << cur)
    H_ad = I.hidden_states(n, geo, 81, f"db.ad{n}")
    H_nt = I.hidden_states(n, geo, 81, f"db.nt{n}")
    slots_ad = (20 * 16 + 3 + torch.arange(n)).to(torch.int32)          # private region, mid-page start
    slots_nt = (5 * 16 + 3 + torch.arange(n)).to(torch.int32)
    La = Layer(px, geo, seed=81, n_blocks=nb, fill=float("nan"))
    dev = {k: v.cuda() for k, v in La.w.items()}
    WA = px.pack_turn_weights(geo, dev["W_k"], dev["W_v"], dev["A_k"], dev["A_v"])
    px.turn_project(La.desc, H_ad.cuda(), WA, La.cache, 0, slots_ad.cuda(), 1 << cur)
    px.turn_project(La.desc, H_nt.cuda(), WA, La.cache, 0, slots_nt.cuda(), others)
    Lb = Layer(px, geo, seed=81, n_blocks=nb, fill=float("nan"))
    masks = torch.tensor([1 << cur] * n + [others] * n, dtype=torch.int64)
    px.turn_project_rows(Lb.desc, torch.cat([H_ad, H_nt]).cuda(), WA, Lb.cache, torch.cat([slots_ad, slots_nt]).cuda(), masks.cuda())
    torch.cuda.synchronize()
    for name in ("k_base", "v_base", "lr_k", "lr_v"):
        a, b = getattr(La.cache, name).view(torch.int16), getattr(Lb.cache, name).view(torch.int16)
        assert torch.equal(a, b), name
    assert not torch.isnan(Lb.cache.lr_k[cur].reshape(nb * 16, -1)[slots_ad.long()]).any()
    assert torch.isnan(Lb.cache.lr_k[cur].reshape(nb * 16, -1)[slots_nt.long()]).all()      # the neutral rows left agent `cur` alone


@pytest.mark.parametrize("hd,r", [(128, 8), (64, 16), (128, 32), (128, 64), (64, 64)])
def test_mma_sync_prefill_kernel_matches_too(monkeypatch, hd, r):
    """The tensor-memory kernel serves these shapes by default; the mma.sync kernel behind it (used for
    rotary keys and for oversized or unaligned caches) is forced here through the environment switch."""
    monkeypatch.setenv("PRECC_PREFILL", "simple")
    px2 = Precc(0)
    geo = I.Geometry(256, 8, 2, hd, 2, r, r, alpha=2.0 * r)
    T, S = 333, 77
    L = Layer(px2, geo, seed=91, n_blocks=(T + S + 15) // 16, tag="ms")
    H = I.hidden_states(T + S, geo, 91, "ms.H")
    L.append(H)
    qs = I.queries(S, geo, 91, "ms.q", gain=3.0)
    got = f64(L.prefill(qs, 1, T))
    w = L.w_np
    ref = O.lr_prefill_reference(f64(qs), 1, T, f64(H), w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"],
                                 geo.scale_k, geo.scale_v, 2)
    assert_close(got, ref, f"mma.sync prefill hd{hd} r{r}")
    assert px2.poll_status() == 0
    px2.close()


def test_decode_alternating_between_ring_layouts_of_one_shape(px):
    """A long context takes the one-block-per-SM ring layout of the cluster kernel, a short one the
    two-blocks-per-SM layout of the same kernel; going back and forth must keep working (the kernel's
    shared-memory limit may only grow)."""
    geo = I.Geometry(128, 6, 2, 64, 2, 0, 8, alpha=16.0)
    T = 5200
    L = Layer(px, geo, seed=63, n_blocks=(T + 15) // 16, tag="alt")
    H = I.hidden_states(T, geo, 63, "alt.H")
    L.append(H)
    q = I.queries(1, geo, 63, "alt.q", gain=3.0)
    w = L.w_np
    args = (f64(H), w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"])
    for ctx in (T, 600, T - 3, 777, 4100, 290):
        got = f64(L.decode(q, [1], [ctx]))
        ref = O.lr_decode_reference(f64(q), [1], [ctx], *args, geo.scale_k, geo.scale_v, geo.n_kv)
        assert_close(got, ref, f"alternating layouts, ctx {ctx}")
    assert px.poll_status() == 0


@pytest.mark.parametrize("M,d", [(41, 1024), (64, 2048), (100, 1024), (129, 2048), (300, 1024), (384, 4096), (450, 2048), (512, 4096)])
def test_short_turn_projection_split_over_a_cluster(monkeypatch, px, M, d):
    """41 to 512 rows (the tokens of a short turn): the K extent of every 128 x 256 tile is split over a cluster
    of 3 to 8 blocks (K slices need not be equal) whose partial accumulators are merged over distributed shared memory.  Against the
    definition, fused call bit-equal to the two separate ones, scattered slots, agent mask, untouched slots; and
    within one bf16 ulp (plus fp32 summation noise near zero) of the one-block-per-tile kernel."""
    geo = I.Geometry(d, 8, 2, 128, 3, 32, 32, alpha=64.0)
    H = I.hidden_states(M, geo, seed=81, tag=f"sk.{M}.{d}")
    nb = (M + 15) // 16 + 4
    slots = I.permutation(nb * 16, 81, f"sk.slots.{M}")[:M].to(torch.int32)
    La = Layer(px, geo, seed=81, n_blocks=nb, fill=float("nan"))
    La.append(H, slot_mapping=slots.cuda(), agent_mask=0b101)
    torch.cuda.synchronize()
    w, Hn, sl = La.w_np, f64(H), slots.long()
    tol = lambda ref: 2.0 ** -8 * np.abs(ref) + 2e-3 * np.sqrt(d / 256)
    for got, ref in ((base_rows(La.cache.k_base)[sl], O.base_cache(Hn, w["W_k"])), (base_rows(La.cache.v_base)[sl], O.base_cache(Hn, w["W_v"])),
                     (lr_rows(La.cache.lr_k, 0)[sl], O.lr_cache(Hn, w["A_k"][0])), (lr_rows(La.cache.lr_v, 2)[sl], O.lr_cache(Hn, w["A_v"][2]))):
        assert (np.abs(got - ref) <= tol(ref)).all()
    assert torch.isnan(La.cache.lr_k[1]).all()
    untouched = torch.ones(nb * 16, dtype=torch.bool); untouched[sl] = False
    assert torch.isnan(La.cache.v_base.permute(0, 2, 1, 3).reshape(nb * 16, -1)[untouched]).all()
    Lb = Layer(px, geo, seed=81, n_blocks=nb, fill=float("nan"))
    dev = {k: v.cuda() for k, v in Lb.w.items()}
    WA = px.pack_turn_weights(geo, dev["W_k"], dev["W_v"], dev["A_k"], dev["A_v"])
    px.turn_project(Lb.desc, H.cuda(), WA, Lb.cache, 0, slots.cuda(), 0b101)
    torch.cuda.synchronize()
    for name in ("k_base", "v_base", "lr_k", "lr_v"):
        assert torch.equal(getattr(La.cache, name).view(torch.int16), getattr(Lb.cache, name).view(torch.int16)), name
    monkeypatch.setenv("PRECC_GEMM_SPLITK", "0")
    monkeypatch.setenv("PRECC_GEMM", "tiled")
    px2 = Precc(0)
    Lc = Layer(px2, geo, seed=81, n_blocks=nb, fill=float("nan"))
    px2.turn_project(Lc.desc, H.cuda(), WA, Lc.cache, 0, slots.cuda(), 0b101)
    torch.cuda.synchronize()
    a, b = base_rows(Lb.cache.k_base)[sl], base_rows(Lc.cache.k_base)[sl]
    assert (np.abs(a - b) <= 2.0 ** -7 * np.abs(b) + 2e-4).all()      # another summation order: one bf16 ulp, or fp32 noise near zero
    assert px.poll_status() == 0 and px2.poll_status() == 0
    px2.close()


@pytest.mark.parametrize("ks,M,d", [(2, 100, 1024), (2, 777, 2048), (3, 384, 4096), (3, 130, 1024), (4, 512, 2048), (4, 64, 4096), (4, 1000, 1024),
                                    (5, 200, 2048), (6, 256, 4096), (7, 41, 2048), (8, 128, 1024), (8, 77, 4096)])
def test_split_k_merge_by_sends_equals_the_pulling_merge_bitwise(monkeypatch, ks, M, d):
    """The partial tiles of a split-K cluster are merged by sends into the owner's shared memory: whole slices by bulk
    copy (clusters of 2 to 4 blocks), or 16-byte pieces straight from registers (any cluster size; the default for
    finer splits of up to 64 rows).  The summation order is that of the pulling merge, so all three must agree bit for bit at the
    same split - and with the definition.  Scattered slots, agent mask, a fused width that is not a multiple of the tile."""
    geo = I.Geometry(d, 8, 2, 128, 3, 16, 16, alpha=32.0)          # fused width 2*256 + 3*32 = 608 columns: three tiles, the last 96 wide
    H = I.hidden_states(M, geo, seed=91, tag=f"push.{M}.{d}")
    nb = (M + 15) // 16 + 3
    slots = I.permutation(nb * 16, 91, f"push.slots.{M}")[:M].to(torch.int32)
    caches = []
    for push_max, direct in (("4", "1"), ("0", "2"), ("0", "0")):       # bulk copies where they apply | direct sends | pulling
        monkeypatch.setenv("PRECC_GEMM", "tiled")                      # keep the few-row kernel out of it
        monkeypatch.setenv("PRECC_GEMM_KS_MAX", str(ks))
        monkeypatch.setenv("PRECC_GEMM_KS_MIN", str(ks))
        monkeypatch.setenv("PRECC_GEMM_PUSH_MAX", push_max)
        monkeypatch.setenv("PRECC_GEMM_DIRECT", direct)
        pz = Precc(0)
        L = Layer(pz, geo, seed=91, n_blocks=nb, fill=float("nan"))
        dev = {k: v.cuda() for k, v in L.w.items()}
        WA = pz.pack_turn_weights(geo, dev["W_k"], dev["W_v"], dev["A_k"], dev["A_v"])
        pz.turn_project(L.desc, H.cuda(), WA, L.cache, 0, slots.cuda(), 0b110)
        torch.cuda.synchronize()
        assert pz.poll_status() == 0
        caches.append(L)
        pz.close()
    La, Lb, Lc = caches
    for name in ("k_base", "v_base", "lr_k", "lr_v"):
        assert torch.equal(getattr(La.cache, name).view(torch.int16), getattr(Lc.cache, name).view(torch.int16)), name
    for name in ("k_base", "v_base", "lr_k", "lr_v"):
        assert torch.equal(getattr(La.cache, name).view(torch.int16), getattr(Lb.cache, name).view(torch.int16)), name
    w, Hn, sl = La.w_np, f64(H), slots.long()
    tol = lambda ref: 2.0 ** -8 * np.abs(ref) + 2e-3 * np.sqrt(d / 256)
    for got, ref in ((base_rows(La.cache.k_base)[sl], O.base_cache(Hn, w["W_k"])), (base_rows(La.cache.v_base)[sl], O.base_cache(Hn, w["W_v"])),
                     (lr_rows(La.cache.lr_k, 1)[sl], O.lr_cache(Hn, w["A_k"][1])), (lr_rows(La.cache.lr_v, 2)[sl], O.lr_cache(Hn, w["A_v"][2]))):
        assert (np.abs(got - ref) <= tol(ref)).all()
    assert torch.isnan(La.cache.lr_k[0]).all()                     # agent 0 is masked out
    untouched = torch.ones(nb * 16, dtype=torch.bool); untouched[sl] = False
    assert torch.isnan(La.cache.k_base.permute(0, 2, 1, 3).reshape(nb * 16, -1)[untouched]).all()


@pytest.mark.parametrize("M,d,hd,n_kv,r", [(1000, 512, 128, 2, 32), (2125, 1024, 64, 8, 16), (640, 256, 128, 1, 8)])
def test_two_sm_projection_equals_the_one_block_kernel_bitwise(monkeypatch, px, M, d, hd, n_kv, r):
    """The cta_group::2 form of the projection GEMM (two SMs per 256-row tile, each staging half of the weight tile;
    opt-in) accumulates every output element over the same k steps in the same order as the one-block kernel: all
    caches agree bit for bit - fused, LR-only with an agent mask, scattered slots, a ragged last tile, and the rotary
    epilogue.  Run under a 20 ms wait limit so that a lost hand-off inside the pair would show as a timeout at once."""
    from paper_2609_34054_b200.inputs import rope_table
    geo = I.Geometry(d, 2 * n_kv, n_kv, hd, 3, r, r, alpha=2.0 * r)
    H = I.hidden_states(M, geo, seed=97, tag=f"pair.{M}").cuda()
    nb = (M + 15) // 16 + 3
    slots = I.permutation(nb * 16, 97, f"pair.slots.{M}")[:M].to(torch.int32).cuda()
    table = rope_table(M + 9, hd)
    monkeypatch.setenv("PRECC_GEMM", "pair")
    px2 = Precc(0)
    px2.set_wait_limit(40_000_000)
    out = []
    for p in (px, px2):
        L = Layer(p, geo, seed=97, n_blocks=nb, fill=float("nan"))
        dev = {k: v.cuda() for k, v in L.w.items()}
        WA = p.pack_turn_weights(geo, dev["W_k"], dev["W_v"], dev["A_k"], dev["A_v"])
        p.turn_project(L.desc, H, WA, L.cache, 0, slots, 0b101)
        Lr = Layer(p, geo, seed=97, n_blocks=nb, fill=float("nan"))
        p.turn_project_rope(Lr.desc, H, WA, Lr.cache, table, 0, None, 0b011, start_pos=5)
        Ll = Layer(p, geo, seed=97, n_blocks=nb, fill=float("nan"))
        p.lr_precompute(Ll.desc, H, Ll.A_packed, Ll.cache, 16, None, 0b110)
        torch.cuda.synchronize()
        assert p.poll_status() == 0
        out.append((L.cache, Lr.cache, Ll.cache))
    for a, b in zip(out[0], out[1]):
        for name in ("k_base", "v_base", "lr_k", "lr_v"):
            assert torch.equal(getattr(a, name).view(torch.int16), getattr(b, name).view(torch.int16)), name
    px2.close()


# ------------------------------------------------------------------ cluster merge under every layout switch

_LAYOUTS = [
    ({"PRECC_DECODE_CLUSTER": "15"}, 64, 8, 4, 16),                       # blocks 13, 14 own no output column
    ({"PRECC_DECODE_CLUSTER": "13"}, 64, 8, 4, 16),                       # the last block owns 4 of 5 columns
    ({"PRECC_DECODE_CLUSTER": "11", "PRECC_DEEP": "0"}, 64, 4, 3, 8),     # odd query group, rank 8 (half an MMA tile)
    ({"PRECC_DEEP": "2"}, 64, 8, 4, 16),                                  # one block per SM, four-page rings
    ({"PRECC_DEEP": "2", "PRECC_DECODE_CLUSTER": "7"}, 128, 8, 4, 64),    # adapter term after the block merge
    ({"PRECC_DEEP": "0"}, 128, 8, 2, 64),
    ({"PRECC_DECODE_PRE": "1"}, 64, 8, 4, 16),                            # one ring slot before the dependency wait
    ({"PRECC_DECODE_STAGES": "2", "PRECC_DEEP": "2"}, 128, 4, 4, 32),
    ({"PRECC_DEEP": "2", "PRECC_DECODE_CLUSTER": "6"}, 64, 8, 1, 0),      # no adapter at all, one query head per kv head
]


@pytest.mark.parametrize("env,hd,n_kv,G,r", _LAYOUTS, ids=lambda v: "-".join(f"{k[6:]}{x}" for k, x in v.items()) if isinstance(v, dict) else str(v))
def test_cluster_merge_under_every_layout_switch(monkeypatch, env, hd, n_kv, G, r):
    """The merge inside a cluster (sends to the block that owns a column) with cluster sizes that leave blocks
    without columns, both ring layouts, both places of the value-side adapter term, and the partial-record mode
    of the same kernel: every variant against the oracle, twice for determinism."""
    from paper_2609_34054_b200.binding import Cache, layer_desc
    for k, v in env.items():
        monkeypatch.setenv(k, v)
    p2 = Precc(0)                                        # the switches are read when a context is created
    try:
        geo = I.Geometry(1024, G * n_kv, n_kv, hd, 2, r, r, alpha=2.0 * max(r, 1))
        T = 5000 + 16 * n_kv + 3
        nb = (T + 15) // 16
        c = I.direct_caches(nb, geo, 77, f"lay.{hd}.{n_kv}.{r}")
        cache = Cache.from_tensors(geo, c["k_base"].cuda(), c["v_base"].cuda(), c["lr_k"].cuda() if r else None,
                                   c["lr_v"].cuda() if r else None)
        w = I.layer_weights(geo, 77, "lay")
        desc = layer_desc(geo)
        q = I.queries(1, geo, 77, "lay.q", gain=4.0)
        aid = torch.tensor([1], dtype=torch.int32).cuda()
        cl = torch.tensor([T], dtype=torch.int32).cuda()
        B_k = w["B_k"].cuda() if r else None
        B_v = w["B_v"].cuda() if r else None
        out = torch.full_like(q, float("nan"), device="cuda")
        ws = p2.decode_workspace(desc, 1, T)
        p2.lr_attend_decode(desc, q.cuda(), aid, cl, T, B_k, B_v, cache, out, ws)
        torch.cuda.synchronize()
        first = out.clone()
        p2.lr_attend_decode(desc, q.cuda(), aid, cl, T, B_k, B_v, cache, out, ws)
        torch.cuda.synchronize()
        assert torch.equal(first, out)
        # partial-record mode (one shard holding everything) + combine = the same attention
        R = p2.partial_record_floats(desc)
        rec = torch.full((1, 1, n_kv, R), float("nan"), dtype=torch.float32, device="cuda")
        p2.lr_attend_decode_partial(desc, q.cuda(), aid, cl, T, B_k, cache, rec[0], ws)
        out2 = torch.full_like(q, float("nan"), device="cuda")
        p2.combine_partials(desc, rec, aid, B_v, out2)
        torch.cuda.synchronize()
        assert torch.isfinite(rec).all()
        rows = lambda x: f64(x.reshape(-1, x.shape[-1]))[:T]
        zero = np.zeros((1, hd))
        for g in (0, n_kv - 1, n_kv // 2):
            cols = slice(g * hd, (g + 1) * hd)
            ref = O.attend_from_caches(f64(q[0, g * G:(g + 1) * G]), rows(c["k_base"][:, g]), rows(c["v_base"][:, g]),
                                       rows(c["lr_k"][1]) if r else np.zeros((T, 1)), rows(c["lr_v"][1]) if r else np.zeros((T, 1)),
                                       f64(w["B_k"][1][:, cols]) if r else zero, f64(w["B_v"][1][:, cols]) if r else zero,
                                       geo.scale_k if r else 0.0, geo.scale_v if r else 0.0, 1)
            assert_close(f64(out)[0, g * G:(g + 1) * G], ref, f"{env} head {g}")
            assert_close(f64(out2)[0, g * G:(g + 1) * G], ref, f"{env} head {g}, partial records + combine")
        assert p2.poll_status() == 0
    finally:
        p2.close()
