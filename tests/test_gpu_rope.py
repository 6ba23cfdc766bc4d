"""Parity of the rotary-key variant (Appendix D.2): rotated base keys written by the projection kernels,
un-rotated LR-K rows, and decode that expands, rotates and adds the rank-r key term page by page.
Expected values come from the merged-weight definition K_a[t] = RoPE_t(H_t (W_k + s A B))."""
import numpy as np
import pytest
import torch

from oracle import lrkv_oracle as O
from paper_2609_34054_b200 import inputs as I
from paper_2609_34054_b200.binding import PreccError
from paper_2609_34054_b200.inputs import rope_table

from harness import Layer, assert_close, base_rows, f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def px():
    from paper_2609_34054_b200.binding import Precc
    p = Precc(0)
    yield p
    assert p.poll_status() == 0
    p.close()


def _decode_rope(L, q, agent_id, ctx_len, table, max_ctx=None, block_table=None):
    qd = q.cuda()
    aid = torch.as_tensor(agent_id, dtype=torch.int32).cuda()
    cl = torch.as_tensor(ctx_len, dtype=torch.int32).cuda()
    max_ctx = int(max(ctx_len)) if max_ctx is None else max_ctx
    ws = L.px.decode_workspace(L.desc, qd.shape[0], max_ctx)
    out = torch.full_like(qd, float("nan"))
    bt = None if block_table is None else block_table.cuda()
    L.px.lr_attend_decode_rope(L.desc, qd, aid, cl, max_ctx, L.B_k, L.B_v, table, L.cache, out, ws, bt)
    torch.cuda.synchronize()
    return out


def test_rope_table_matches_the_definition():
    """The library-side table generator against the oracle's (independent code, same definition)."""
    t = rope_table(300, 64, device="cpu").double().numpy()
    cos, sin = O.rope_tables(300, 64)
    np.testing.assert_allclose(t[..., 0], cos, atol=1e-7)
    np.testing.assert_allclose(t[..., 1], sin, atol=1e-7)


@pytest.mark.parametrize("hd,n_kv,M", [(64, 2, 300), (128, 1, 130), (128, 4, 517),
                                      (64, 2, 1), (128, 2, 7), (128, 1, 40), (64, 4, 64), (128, 2, 16)])   # the last five: few-row kernel
def test_projection_rotates_keys_only(px, hd, n_kv, M):
    geo = I.Geometry(d_model=256, n_q=2 * n_kv, n_kv=n_kv, hd=hd, n_agents=2, rank_k=16, rank_v=16, alpha=32.0)
    nb = (M + 15) // 16 + 2
    L = Layer(px, geo, seed=3, n_blocks=nb, tag="rp", fill=0.0)
    H = I.hidden_states(M, geo, 3, "rp.H")
    table = rope_table(1024, hd)
    cos, sin = O.rope_tables(1024, hd)
    # plain projection first (keeps V for the bitwise check), then the rotary one with explicit positions
    px.rebase_project(L.desc, H.cuda(), L.W_packed, L.cache, 0)
    torch.cuda.synchronize()
    v_plain = L.cache.v_base.clone()
    pos = I.uniform_int(0, 1023, M, 3, "rp.pos").to(torch.int32)
    px.rebase_project_rope(L.desc, H.cuda(), L.W_packed, L.cache, table, 0, positions=pos.cuda())
    torch.cuda.synchronize()
    assert torch.equal(L.cache.v_base, v_plain)
    got = base_rows(L.cache.k_base)[:M]
    ref = O.rope_rotate(O.base_cache(f64(H), L.w_np["W_k"]), pos.numpy(), n_kv, cos, sin)
    err = np.abs(got - ref)
    assert (err <= 2.0 ** -8 * np.abs(ref) + 2e-3).all(), f"max err {err.max()}"
    # consecutive positions from start_pos, through the fused projection: bitwise equal to the two-call form
    px.rebase_project_rope(L.desc, H.cuda(), L.W_packed, L.cache, table, 0, start_pos=7)
    px.lr_precompute(L.desc, H.cuda(), L.A_packed, L.cache, 0)
    torch.cuda.synchronize()
    k2, lk2, v2, lv2 = L.cache.k_base.clone(), L.cache.lr_k.clone(), L.cache.v_base.clone(), L.cache.lr_v.clone()
    ref2 = O.rope_rotate(O.base_cache(f64(H), L.w_np["W_k"]), np.arange(M) + 7, n_kv, cos, sin)
    assert (np.abs(base_rows(k2)[:M] - ref2) <= 2.0 ** -8 * np.abs(ref2) + 2e-3).all()
    WA = px.pack_turn_weights(geo, L.w["W_k"].cuda(), L.w["W_v"].cuda(), L.w["A_k"].cuda(), L.w["A_v"].cuda())
    # the fused rotary projection (precc_turn_project_rope): every cache it writes equals the two-call form bit for
    # bit - rotated base K rows (checked against the oracle above), plain V rows, un-rotated LR rows of both sides
    for c in (L.cache.k_base, L.cache.v_base, L.cache.lr_k, L.cache.lr_v):
        c.zero_()
    px.turn_project_rope(L.desc, H.cuda(), WA, L.cache, table, 0, start_pos=7)
    torch.cuda.synchronize()
    assert torch.equal(L.cache.k_base, k2) and torch.equal(L.cache.lr_k, lk2)
    assert torch.equal(L.cache.v_base, v2) and torch.equal(L.cache.lr_v, lv2)
    assert_close(f64(L.cache.lr_k[1].reshape(-1, 16))[:M], O.lr_cache(f64(H), L.w_np["A_k"][1]), "LR-K rows stay un-rotated",
                 atol=2e-2, rtol=1e-2, norm_tol=1e-2)
    # with an agent mask only the selected agents' LR rows are written; the rotated base rows always are
    for c in (L.cache.k_base, L.cache.v_base, L.cache.lr_k, L.cache.lr_v):
        c.zero_()
    px.turn_project_rope(L.desc, H.cuda(), WA, L.cache, table, 0, None, 0b10, start_pos=7)
    torch.cuda.synchronize()
    assert torch.equal(L.cache.k_base, k2) and torch.equal(L.cache.lr_k[1], lk2[1]) and torch.equal(L.cache.lr_v[1], lv2[1])
    assert (L.cache.lr_k[0] == 0).all() and (L.cache.lr_v[0] == 0).all()


SHAPES = [
    # hd, n_q, n_kv, rank, T, agents
    (64, 8, 2, 16, 70, 2),
    (64, 16, 2, 8, 333, 3),
    (64, 4, 4, 32, 129, 2),
    (64, 8, 1, 64, 100, 2),
    (128, 8, 2, 8, 97, 3),
    (128, 8, 2, 16, 260, 2),
    (128, 4, 1, 32, 65, 2),
    (128, 8, 8, 64, 48, 2),
]


@pytest.mark.parametrize("hd,n_q,n_kv,r,T,N", SHAPES)
def test_decode_rope_small_shapes(px, hd, n_q, n_kv, r, T, N):
    geo = I.Geometry(d_model=192, n_q=n_q, n_kv=n_kv, hd=hd, n_agents=N, rank_k=r, rank_v=r, alpha=2.0 * r)
    L = Layer(px, geo, seed=5, n_blocks=(T + 15) // 16, tag="rd")
    H = I.hidden_states(T, geo, 5, "rd.H")
    table = rope_table(T + 5, hd)
    cos, sin = O.rope_tables(T + 5, hd)
    px.rebase_project_rope(L.desc, H.cuda(), L.W_packed, L.cache, table, 0)
    px.lr_precompute(L.desc, H.cuda(), L.A_packed, L.cache, 0)
    agents = [i % N for i in range(4)]
    ctx = [T, max(1, T // 2), 17, 1]
    w = L.w_np
    for gain in (1.0, 4.0):
        q = I.queries(4, geo, 5, f"rd.q{gain}", gain=gain)
        out = f64(_decode_rope(L, q, agents, ctx, table))
        ref = O.lr_decode_reference_rope(f64(q), agents, ctx, f64(H), w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"],
                                         geo.scale_k, geo.scale_v, n_kv, cos, sin)
        assert_close(out, ref, f"rope decode hd{hd} r{r} gain {gain}")


def test_decode_rope_differs_from_the_position_free_fold(px):
    """Guards against a vacuous test: on rotated base keys the position-free kernel (which folds the
    un-rotated rank-r term into the query) must NOT match the rotary definition."""
    geo = I.Geometry(d_model=192, n_q=8, n_kv=2, hd=64, n_agents=2, rank_k=16, rank_v=16, alpha=64.0)
    T = 200
    L = Layer(px, geo, seed=6, n_blocks=(T + 15) // 16, tag="rf")
    H = I.hidden_states(T, geo, 6, "rf.H")
    table = rope_table(T, 64)
    cos, sin = O.rope_tables(T, 64)
    px.rebase_project_rope(L.desc, H.cuda(), L.W_packed, L.cache, table, 0)
    px.lr_precompute(L.desc, H.cuda(), L.A_packed, L.cache, 0)
    q = I.queries(2, geo, 6, "rf.q", gain=4.0)
    w = L.w_np
    ref = O.lr_decode_reference_rope(f64(q), [0, 1], [T, T], f64(H), w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"],
                                     geo.scale_k, geo.scale_v, 2, cos, sin)
    assert_close(f64(_decode_rope(L, q, [0, 1], [T, T], table)), ref, "rotary decode")
    plain = f64(L.decode(q, [0, 1], [T, T]))
    assert np.max(np.abs(plain - ref)) > 5e-2
    # adapter-free view (agent -1) and position-free kernel agree bit for bit on the rotated base cache
    a = _decode_rope(L, q, [-1, -1], [T, T], table)
    b = L.decode(q, [-1, -1], [T, T])
    assert torch.equal(a, b)


def test_decode_rope_long_context_split_and_paged(px):
    """Benchmark-layer shape, 8192 tokens: batch 1 takes the cluster path, batch 24 over shuffled pages the
    ticket path with several splits; both against the definition."""
    geo, T = I.C2, 8192
    L = Layer(px, geo, seed=0, n_blocks=T // 16, tag="L0")
    H = I.hidden_states(T, geo, 0, "L0.H")
    table = rope_table(T, geo.hd)
    cos, sin = O.rope_tables(T, geo.hd)
    perm = I.permutation(T // 16, 0, "rope.perm").to(torch.int32)          # logical block -> physical block
    slots = (perm.long()[:, None] * 16 + torch.arange(16)[None, :]).reshape(-1).to(torch.int32)
    WA = px.pack_turn_weights(geo, L.w["W_k"].cuda(), L.w["W_v"].cuda(), L.w["A_k"].cuda(), L.w["A_v"].cuda())
    px.turn_project_rope(L.desc, H.cuda(), WA, L.cache, table, 0, slot_mapping=slots.cuda())
    w, Hn = L.w_np, f64(H)
    q = I.queries(1, geo, 0, "rope.q1", gain=4.0)
    out = f64(_decode_rope(L, q, [2], [T], table, block_table=perm[None, :]))
    ref = O.lr_decode_reference_rope(f64(q), [2], [T], Hn, w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"],
                                     geo.scale_k, geo.scale_v, geo.n_kv, cos, sin)
    assert_close(out, ref, "rope C2 batch 1")
    Bn = 24
    agents = [i % geo.n_agents for i in range(Bn)]
    ctx = [int(x) for x in I.uniform_int(1500, T, Bn, 0, "rope.ctx")]
    q = I.queries(Bn, geo, 0, "rope.q24", gain=4.0)
    out = f64(_decode_rope(L, q, agents, ctx, table, block_table=perm[None, :].repeat(Bn, 1)))
    sel = [0, 7, 23]
    ref = O.lr_decode_reference_rope(f64(q)[sel], [agents[i] for i in sel], [ctx[i] for i in sel], Hn, w["W_k"], w["W_v"],
                                     w["A_k"], w["B_k"], w["A_v"], w["B_v"], geo.scale_k, geo.scale_v, geo.n_kv, cos, sin)
    assert_close(out[sel], ref, "rope C2 batch 24")


@pytest.mark.parametrize("hd,n_q,n_kv,r,T,S", [(64, 8, 2, 16, 150, 37), (64, 4, 4, 8, 0, 70), (128, 8, 2, 32, 70, 64),
                                              (128, 8, 1, 64, 33, 20), (64, 16, 2, 32, 333, 5)])
def test_prefill_rope_shapes(px, hd, n_q, n_kv, r, T, S):
    geo = I.Geometry(d_model=192, n_q=n_q, n_kv=n_kv, hd=hd, n_agents=2, rank_k=r, rank_v=r, alpha=2.0 * r)
    L = Layer(px, geo, seed=8, n_blocks=(T + S + 15) // 16, tag="rpf")
    H = I.hidden_states(T + S, geo, 8, "rpf.H")
    table = rope_table(T + S + 3, hd)
    cos, sin = O.rope_tables(T + S + 3, hd)
    px.rebase_project_rope(L.desc, H.cuda(), L.W_packed, L.cache, table, 0)
    px.lr_precompute(L.desc, H.cuda(), L.A_packed, L.cache, 0)
    w = L.w_np
    q = I.queries(S, geo, 8, "rpf.q", gain=3.0)
    out = torch.full_like(q, float("nan"), device="cuda")
    px.lr_attend_prefill_rope(L.desc, q.cuda(), 1, T, L.B_k, L.B_v, table, L.cache, out)
    torch.cuda.synchronize()
    ref = O.lr_prefill_reference_rope(f64(q), 1, T, f64(H), w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"],
                                      geo.scale_k, geo.scale_v, n_kv, cos, sin)
    assert_close(f64(out), ref, f"rope prefill hd{hd} r{r}")
    # last row against the rotary decode kernel at the same context (two different kernels, same definition)
    dec = f64(_decode_rope(L, q[S - 1:], [1], [T + S], table))
    assert_close(dec, ref[S - 1:], "rope decode at the turn's last token")
    # adapter-free view: identical to the position-free prefill over the rotated base
    a = torch.full_like(q, float("nan"), device="cuda")
    px.lr_attend_prefill_rope(L.desc, q.cuda(), -1, T, L.B_k, L.B_v, table, L.cache, a)
    b = L.prefill(q, -1, T)
    assert torch.equal(a, b)


@pytest.mark.parametrize("hd,n_q,n_kv,r,T,S,paged", [(64, 8, 2, 16, 200, 40, False), (128, 8, 2, 32, 515, 130, True), (128, 4, 1, 8, 90, 7, False),
                                                     (128, 8, 1, 64, 33, 20, True), (64, 16, 2, 32, 333, 5, False), (128, 8, 2, 16, 2300, 33, True)])
def test_prefill_rope_through_a_key_scratch(px, hd, n_q, n_kv, r, T, S, paged):
    """The fast rotary prefill: the sequence's adapted rotary keys are written to a scratch area once, then the
    tensor-core kernel runs on them.  Against the definition, against the per-tile kernel, paged and contiguous,
    a short turn over a longer context (split over a cluster), scratch reuse, and the error paths."""
    geo = I.Geometry(d_model=192, n_q=n_q, n_kv=n_kv, hd=hd, n_agents=2, rank_k=r, rank_v=r, alpha=2.0 * r)
    nb = (T + S + 15) // 16
    pool = nb + 5 if paged else nb
    L = Layer(px, geo, seed=18, n_blocks=pool, tag="rps")
    H = I.hidden_states(T + S, geo, 18, "rps.H")
    table = rope_table(T + S + 3, hd)
    cos, sin = O.rope_tables(T + S + 3, hd)
    bt = I.permutation(pool, 18, "rps.bt")[:nb].to(torch.int32).cuda() if paged else None
    slots = (bt.long().cpu()[:, None] * 16 + torch.arange(16)[None, :]).reshape(-1)[:T + S].to(torch.int32).cuda() if paged else None
    pos = torch.arange(T + S, dtype=torch.int32).cuda()
    px.rebase_project_rope(L.desc, H.cuda(), L.W_packed, L.cache, table, 0, slots, positions=pos)
    px.lr_precompute(L.desc, H.cuda(), L.A_packed, L.cache, 0, slots)
    w = L.w_np
    q = I.queries(S, geo, 18, "rps.q", gain=3.0)
    nbytes = px.prefill_rope_scratch_bytes(L.desc, T, S)
    assert nbytes == ((nb + 7) // 8 * 8) * n_kv * 16 * hd * 2
    scratch = torch.full((nbytes + 256,), 0x7f, dtype=torch.uint8, device="cuda")       # NaN-ish fill, guard bytes behind
    out = torch.full_like(q, float("nan"), device="cuda")
    px.lr_attend_prefill_rope_scratch(L.desc, q.cuda(), 1, T, L.B_k, L.B_v, table, L.cache, out, scratch[:nbytes], bt)
    torch.cuda.synchronize()
    assert (scratch[nbytes:] == 0x7f).all()                                              # nothing written behind the area
    ref = O.lr_prefill_reference_rope(f64(q), 1, T, f64(H), w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"],
                                      geo.scale_k, geo.scale_v, n_kv, cos, sin)
    assert_close(f64(out), ref, f"rope prefill through scratch hd{hd} r{r}")
    slow = torch.full_like(q, float("nan"), device="cuda")
    px.lr_attend_prefill_rope(L.desc, q.cuda(), 1, T, L.B_k, L.B_v, table, L.cache, slow, bt)
    torch.cuda.synchronize()
    assert_close(f64(out), f64(slow), "scratch path against the per-tile kernel")
    # the scratch holds the adapted rotary keys of the sequence in logical order: check a few rows against the definition
    ks = scratch[:nbytes].view(torch.bfloat16).view(-1, n_kv, 16, hd)
    Ka = O.rope_rotate(O.adapted_projection(f64(H), w["W_k"], w["A_k"][1], w["B_k"][1], geo.scale_k), np.arange(T + S), n_kv, cos, sin)
    for t in (0, T - 1, T + S - 1):
        got = f64(ks[t // 16, :, t % 16, :]).reshape(-1)
        assert (np.abs(got - Ka[t]) <= 2.0 ** -7 * np.abs(Ka[t]) + 3e-3).all()
    # second call on the same scratch (another agent): the area is simply overwritten
    out2 = torch.full_like(q, float("nan"), device="cuda")
    px.lr_attend_prefill_rope_scratch(L.desc, q.cuda(), 0, T, L.B_k, L.B_v, table, L.cache, out2, scratch[:nbytes], bt)
    torch.cuda.synchronize()
    ref0 = O.lr_prefill_reference_rope(f64(q), 0, T, f64(H), w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"],
                                       geo.scale_k, geo.scale_v, n_kv, cos, sin)
    assert_close(f64(out2), ref0, "second agent through the same scratch")
    # adapter-free view: the scratch is not needed and not touched
    before = scratch.clone()
    a = torch.full_like(q, float("nan"), device="cuda")
    px.lr_attend_prefill_rope_scratch(L.desc, q.cuda(), -1, T, L.B_k, L.B_v, table, L.cache, a, scratch[:nbytes], bt)
    torch.cuda.synchronize()
    assert torch.equal(scratch, before)
    b = torch.full_like(q, float("nan"), device="cuda")
    px.lr_attend_prefill_rope(L.desc, q.cuda(), -1, T, L.B_k, L.B_v, table, L.cache, b, bt)
    assert torch.equal(a, b)
    with pytest.raises(PreccError):                      # too small
        px.lr_attend_prefill_rope_scratch(L.desc, q.cuda(), 1, T, L.B_k, L.B_v, table, L.cache, out, scratch[:nbytes - 128], bt)
    with pytest.raises(PreccError):                      # misaligned
        px.lr_attend_prefill_rope_scratch(L.desc, q.cuda(), 1, T, L.B_k, L.B_v, table, L.cache, out, scratch[64:nbytes + 64], bt)
    assert px.poll_status() == 0


def test_rope_invalid_arguments(px):
    geo = I.Geometry(d_model=192, n_q=8, n_kv=2, hd=64, n_agents=2, rank_k=16, rank_v=16, alpha=32.0)
    L = Layer(px, geo, seed=7, n_blocks=8, tag="ri", fill=0.0)
    H = I.hidden_states(100, geo, 7, "ri.H")
    table = rope_table(64, 64)
    with pytest.raises(PreccError):                      # positions 0..99 do not fit a 64-row table
        px.rebase_project_rope(L.desc, H.cuda(), L.W_packed, L.cache, table, 0)
    q = I.queries(1, geo, 7, "ri.q")
    with pytest.raises(PreccError):                      # max_ctx beyond the table
        _decode_rope(L, q, [0], [100], table)
    assert px.poll_status() == 0
