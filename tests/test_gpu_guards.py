"""Out-of-bounds writes: every output and cache buffer sits between guard regions filled with a sentinel
bit pattern; after each entry point has run at awkward sizes (ragged tails, partial pages, masked agents,
scattered slots) the guards must be untouched, and so must every cache row that was not addressed."""
import time

import pytest
import torch

from paper_2609_34054_b200 import inputs as I
from paper_2609_34054_b200.binding import Cache, Precc, layer_desc
from paper_2609_34054_b200.inputs import rope_table

pytestmark = pytest.mark.gpu

GUARD = 4096                      # bf16 elements on each side
SENTINEL = 0x7FC1                 # a NaN bit pattern no kernel produces


def guarded(shape, dtype=torch.bfloat16):
    """A tensor view of `shape` carved out of a larger buffer whose margins hold the sentinel."""
    n = 1
    for s in shape:
        n *= s
    assert dtype == torch.bfloat16
    raw = torch.full((n + 2 * GUARD,), SENTINEL, dtype=torch.int16, device="cuda")
    view = raw[GUARD:GUARD + n].view(torch.bfloat16).view(*shape)
    return raw, view


def guards_intact(raw) -> bool:
    return bool((raw[:GUARD] == SENTINEL).all() and (raw[-GUARD:] == SENTINEL).all())


@pytest.mark.parametrize("hd,r,M,S", [(64, 16, 37, 21), (128, 32, 130, 45), (128, 8, 5, 3), (64, 64, 70, 64)])
def test_all_entry_points_stay_inside_their_buffers(hd, r, M, S):
    px = Precc(0)
    geo = I.Geometry(d_model=256, n_q=8, n_kv=2, hd=hd, n_agents=3, rank_k=r, rank_v=r, alpha=2.0 * r)
    desc = layer_desc(geo)
    T = M + S
    nb = (T + 15) // 16 + 1
    raws, views = {}, {}
    for name, shape in (("k_base", (nb, geo.n_kv, 16, hd)), ("v_base", (nb, geo.n_kv, 16, hd)),
                        ("lr_k", (geo.n_agents, nb, 16, r)), ("lr_v", (geo.n_agents, nb, 16, r))):
        raws[name], views[name] = guarded(shape)
        views[name].view(torch.int16).fill_(SENTINEL)              # unaddressed rows must keep the sentinel too
    cache = Cache.from_tensors(geo, views["k_base"], views["v_base"], views["lr_k"], views["lr_v"])
    w = {k: v.cuda() for k, v in I.layer_weights(geo, 9, "g").items()}
    W = px.pack_base_weights(geo, w["W_k"], w["W_v"])
    A = px.pack_adapters(geo, w["A_k"], w["A_v"])
    WA = px.pack_turn_weights(geo, w["W_k"], w["W_v"], w["A_k"], w["A_v"])
    H = I.hidden_states(T, geo, 9, "g.H").cuda()
    table = rope_table(T + 1, hd)
    # projections: a tiled call (M rows), a few-row call (S rows), fused and rotary forms, one masked agent
    px.rebase_project(desc, H[:M], W, cache, 0)
    px.lr_precompute(desc, H[:M], A, cache, 0, None, 0b011)
    px.turn_project(desc, H[M:], WA, cache, M, None, 0b011)
    px.rebase_project_rope(desc, H[:M], W, cache, table, 0)
    px.turn_project_rope(desc, H[M:], WA, cache, table, M, None, 0b011, start_pos=M)
    torch.cuda.synchronize()
    flat = lambda t: t.view(torch.int16)
    # slots >= T were never addressed; agent 2 was masked out everywhere
    kb = flat(views["k_base"]).permute(0, 2, 1, 3).reshape(nb * 16, -1)
    assert (kb[T:] == SENTINEL).all() and not (kb[:T] == SENTINEL).any()
    assert (flat(views["lr_k"])[2] == SENTINEL).all() and (flat(views["lr_v"])[2] == SENTINEL).all()
    lk0 = flat(views["lr_k"])[0].reshape(nb * 16, -1)
    assert (lk0[T:] == SENTINEL).all() and not (lk0[:T] == SENTINEL).any()
    # attention outputs between guards: decode (batch 3, ragged lengths), prefill, their rotary forms
    B = 3
    q = I.queries(B, geo, 9, "g.q").cuda()
    aid = torch.tensor([0, 1, -1], dtype=torch.int32, device="cuda")
    cl = torch.tensor([T, min(17, T - 1), 1], dtype=torch.int32, device="cuda")
    ws = px.decode_workspace(desc, B, T)
    qs = I.queries(S, geo, 9, "g.qs").cuda()
    for rope in (False, True):
        raw_o, out = guarded((B, geo.n_q, hd))
        if rope:
            px.lr_attend_decode_rope(desc, q, aid, cl, T, w["B_k"], w["B_v"], table, cache, out, ws)
        else:
            px.lr_attend_decode(desc, q, aid, cl, T, w["B_k"], w["B_v"], cache, out, ws)
        raw_p, outp = guarded((S, geo.n_q, hd))
        if rope:
            px.lr_attend_prefill_rope(desc, qs, 1, M, w["B_k"], w["B_v"], table, cache, outp)
        else:
            px.lr_attend_prefill(desc, qs, 1, M, w["B_k"], w["B_v"], cache, outp)
        torch.cuda.synchronize()
        assert guards_intact(raw_o) and guards_intact(raw_p)
        assert torch.isfinite(out.float()).all() and torch.isfinite(outp.float()).all()
    for name, raw in raws.items():
        assert guards_intact(raw), name
    assert px.poll_status() == 0
    px.close()


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    """Failure detection without a fault: every wait inside the library's kernels has a limit.  A kernel whose
    barrier is never completed must end by itself once the limit (lowered here to about a millisecond) has passed,
    the status word must say TIMEOUT, nothing around the flag it writes may be touched, and the context must go on
    working: the same projection + attention calls give the same bits before and after."""
    px = Precc(0)
    geo = I.Geometry(d_model=256, n_q=8, n_kv=2, hd=128, n_agents=2, rank_k=16, rank_v=16, alpha=32.0)
    desc = layer_desc(geo)
    w = {k: v.cuda() for k, v in I.layer_weights(geo, 4, "to").items()}
    WA = px.pack_turn_weights(geo, w["W_k"], w["W_v"], w["A_k"], w["A_v"])
    T, S = 600, 96
    H = I.hidden_states(T, geo, 4, "to.H").cuda()
    q, qs = I.queries(2, geo, 4, "to.q").cuda(), I.queries(S, geo, 4, "to.qs").cuda()
    aid = torch.tensor([0, 1], dtype=torch.int32, device="cuda")
    cl = torch.tensor([T, 77], dtype=torch.int32, device="cuda")

    def ordinary():
        cache = Cache(geo, (T + 15) // 16 + 1, fill=0.0)
        px.turn_project(desc, H, WA, cache, 0)                      # tcgen05 GEMM: bounded mbarrier waits inside
        out = torch.full_like(q, float("nan"))
        px.lr_attend_decode(desc, q, aid, cl, T, w["B_k"], w["B_v"], cache, out, px.decode_workspace(desc, 2, T))
        outp = torch.full_like(qs, float("nan"))
        px.lr_attend_prefill(desc, qs, 1, T - S, w["B_k"], w["B_v"], cache, outp)   # tcgen05 prefill: bounded waits too
        torch.cuda.synchronize()
        return cache.k_base.clone(), out, outp

    before = ordinary()
    assert px.poll_status() == 0
    px.set_wait_limit(2_000_000)                                     # about 1 ms of SM clock
    raw = torch.full((2 * 64 + 1,), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    flag = raw[64:65]
    t0 = time.perf_counter()
    px.selftest_wait_timeout(flag)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    assert dt < 0.5, f"the wait did not give up at its limit ({dt:.2f} s)"
    assert flag.item() == 2                                          # expired, then ran to its end
    assert (raw[:64] == 0x5A5A5A5A).all() and (raw[65:] == 0x5A5A5A5A).all()
    assert px.poll_status() == 2                                     # PRECC_STATUS_TIMEOUT, nothing else
    assert px.poll_status() == 0                                     # cleared by the read
    after_low = ordinary()                                           # real kernels under the 1 ms limit: none of their waits runs out
    assert px.poll_status() == 0
    px.set_wait_limit(0)                                             # back to the default
    after = ordinary()
    assert px.poll_status() == 0
    for a, b, c in zip(before, after_low, after):
        assert torch.equal(a, b) and torch.equal(a, c)
    px.close()
