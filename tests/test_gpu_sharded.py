"""Context-sharded decode: the shards' partial records merged by the combine kernel equal attention over the
whole context.  The shards are emulated on one GPU one after another (each with its own caches holding its
token range from slot 0); nothing here waits on another launch."""
import numpy as np
import pytest
import torch

from oracle import lrkv_oracle as O
from paper_2609_34054_b200 import inputs as I
from paper_2609_34054_b200.binding import Precc, PreccError
from paper_2609_34054_b200.binding import layer_desc
from paper_2609_34054_b200.sharded import head_shard_geometry, head_slice, shard_b_heads, shard_cache_heads, shard_ranges

from harness import Layer, assert_close, f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def px():
    p = Precc(0)
    yield p
    assert p.poll_status() == 0
    p.close()


def _sharded_decode(px, geo, seed, H, q, agents, ctx, world):
    """Runs `world` shards sequentially and combines; returns (output, records)."""
    ranges = shard_ranges(ctx, world)
    Bn = q.shape[0]
    ref_layer = None
    R = None
    recs = None
    for r in range(world):
        local_len = [e - s for s, e in ranges[r]]
        # every request shares the trajectory H, so a shard's cache holds H[s:e] of the LONGEST range it owns;
        # requests with shorter contexts address a prefix of their own range, laid out request by request
        n_blocks = sum((l + 15) // 16 for l in local_len) + 1
        L = Layer(px, geo, seed=seed, n_blocks=n_blocks, tag="sh")
        first, at = [], 0
        for (s, e) in ranges[r]:
            first.append(at)
            if e > s:
                L.append(H[s:e], start_slot=at * 16)
            at += (e - s + 15) // 16
        if recs is None:
            R = px.partial_record_floats(L.desc)
            recs = torch.full((world, Bn, geo.n_kv, R), float("nan"), dtype=torch.float32, device="cuda")
            ref_layer = L
        mx = max(1, max(local_len))
        ws = px.decode_workspace(L.desc, Bn, mx)
        px.lr_attend_decode_partial(L.desc, q.cuda(), torch.tensor(agents, dtype=torch.int32).cuda(),
                                    torch.tensor(local_len, dtype=torch.int32).cuda(), mx, L.B_k, L.cache, recs[r], ws,
                                    None, torch.tensor(first, dtype=torch.int32).cuda())
    out = torch.full_like(q, float("nan"), device="cuda")
    px.combine_partials(ref_layer.desc, recs, torch.tensor(agents, dtype=torch.int32).cuda(), ref_layer.B_v, out)
    torch.cuda.synchronize()
    return out, recs, ref_layer


@pytest.mark.parametrize("hd,n_q,n_kv,r,world", [(64, 8, 2, 16, 2), (128, 8, 2, 32, 3), (128, 4, 1, 8, 4), (64, 16, 4, 0, 2),
                                                 (128, 8, 2, 64, 8)])
def test_sharded_equals_whole_context(px, hd, n_q, n_kv, r, world):
    geo = I.Geometry(d_model=192, n_q=n_q, n_kv=n_kv, hd=hd, n_agents=2, rank_k=r, rank_v=r, alpha=2.0 * max(r, 1))
    T = 700
    H = I.hidden_states(T, geo, 11, "sh.H")
    agents = [0, 1, -1, 1, 0]
    ctx = [T, 333, 50, 17, 1]                      # the short ones leave late shards empty
    q = I.queries(len(ctx), geo, 11, "sh.q", gain=4.0)
    out, recs, L = _sharded_decode(px, geo, 11, H, q, agents, ctx, world)
    assert torch.isfinite(recs).all()
    w = L.w_np
    args = (f64(H), w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"])
    adapted = O.lr_decode_reference(f64(q), [max(a, 0) for a in agents], ctx, *args, geo.scale_k, geo.scale_v, n_kv)
    neutral = O.lr_decode_reference(f64(q), [0] * len(ctx), ctx, *args, 0.0, 0.0, n_kv)
    ref = np.where(np.array(agents)[:, None, None] < 0, neutral, adapted)
    assert_close(f64(out), ref, f"sharded decode world {world}")
    # and against the single-GPU kernel over the whole context (same arithmetic up to summation order)
    whole = Layer(px, geo, seed=11, n_blocks=(T + 15) // 16, tag="sh")
    whole.append(H)
    one = whole.decode(q, agents, ctx)
    assert (one.float() - out.float()).abs().max() <= 2e-2


def test_one_shard_reproduces_the_plain_kernel_and_empty_requests_give_zeros(px):
    geo = I.Geometry(d_model=192, n_q=8, n_kv=2, hd=64, n_agents=2, rank_k=16, rank_v=16, alpha=32.0)
    T = 300
    H = I.hidden_states(T, geo, 12, "sh1.H")
    q = I.queries(3, geo, 12, "sh1.q", gain=2.0)
    agents, ctx = [0, 1, 1], [T, 40, 0]
    out, recs, L = _sharded_decode(px, geo, 12, H, q, agents, ctx, 1)
    assert (out[2] == 0).all()                                     # no token anywhere
    assert (recs[0, 2, :, :8] < -1e29).all() and (recs[0, 2, :, 8:] == 0).all()   # the neutral record
    whole = Layer(px, geo, seed=12, n_blocks=(T + 15) // 16, tag="sh")
    whole.append(H)
    one = whole.decode(q[:2], agents[:2], ctx[:2])
    assert (one.float() - out[:2].float()).abs().max() <= 1e-2
    with pytest.raises(PreccError):
        px.combine_partials(L.desc, recs.new_zeros((65,) + tuple(recs.shape[1:])), torch.tensor(agents, dtype=torch.int32).cuda(),
                            L.B_v, out)


def test_long_context_shards_take_the_cluster_path(px):
    """Benchmark-layer shape, one request, 8192 tokens over 2 shards: each shard's launch is the cluster
    kernel (few units, long context), whose blocks write column slices of the record."""
    geo, T = I.C2, 8192
    H = I.hidden_states(T, geo, 0, "L0.H")
    q = I.queries(2, geo, 0, "sh.q2", gain=4.0)
    agents, ctx = [3, -1], [T, 5000]
    out, recs, L = _sharded_decode(px, geo, 0, H, q, agents, ctx, 2)
    assert torch.isfinite(recs).all()
    w = L.w_np
    args = (f64(H), w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"])
    ref0 = O.lr_decode_reference(f64(q[:1]), [3], [T], *args, geo.scale_k, geo.scale_v, geo.n_kv)
    ref1 = O.lr_decode_reference(f64(q[1:]), [0], [5000], *args, 0.0, 0.0, geo.n_kv)
    assert_close(f64(out), np.concatenate([ref0, ref1]), "sharded C2 decode")


@pytest.mark.parametrize("hd,n_q,n_kv,r,world", [(64, 16, 4, 16, 2), (128, 16, 8, 32, 4), (128, 8, 8, 8, 8), (64, 8, 2, 0, 2)])
def test_head_sharded_equals_the_oracle_and_the_unsharded_call(px, hd, n_q, n_kv, r, world):
    """Head sharding: every rank runs the ordinary decode call on the caches of its kv heads (LR caches replicated)
    and the outputs are concatenated along the head axis.  The ranks are emulated one after another on one GPU; the
    result must meet the oracle's bar, and each rank's slice must equal the oracle's slice for its heads."""
    geo = I.Geometry(d_model=192, n_q=n_q, n_kv=n_kv, hd=hd, n_agents=2, rank_k=r, rank_v=r, alpha=2.0 * max(r, 1))
    T = 1500
    H = I.hidden_states(T, geo, 21, "hs.H")
    L = Layer(px, geo, seed=21, n_blocks=(T + 15) // 16, tag="hs")
    L.append(H)
    agents, ctx = [0, 1, -1, 1], [T, 777, 300, 16]
    q = I.queries(len(ctx), geo, 21, "hs.q", gain=4.0)
    aid = torch.tensor(agents, dtype=torch.int32).cuda()
    cl = torch.tensor(ctx, dtype=torch.int32).cuda()
    local_geo = head_shard_geometry(geo, world)
    desc = layer_desc(local_geo)
    parts = []
    for rank in range(world):
        cache_r = shard_cache_heads(L.cache, geo, rank, world)
        Bk, Bv = shard_b_heads(L.B_k, geo, rank, world), shard_b_heads(L.B_v, geo, rank, world)
        q_r = q[:, head_slice(rank, world, geo.n_q)].contiguous().cuda()
        out_r = torch.full_like(q_r, float("nan"))
        ws = px.decode_workspace(desc, len(ctx), T)
        px.lr_attend_decode(desc, q_r, aid, cl, T, Bk, Bv, cache_r, out_r, ws)
        parts.append(out_r)
    torch.cuda.synchronize()
    out = torch.cat(parts, dim=1)                        # what gather_heads builds from the all-gathered slices
    w, Hn = L.w_np, f64(H)
    ref = np.zeros((len(ctx), n_q, hd))
    for b, (a, t) in enumerate(zip(agents, ctx)):
        if a >= 0 and r > 0:
            ref[b] = O.lr_decode_reference(f64(q[b:b + 1]), [a], [t], Hn, w["W_k"], w["W_v"], w["A_k"], w["B_k"], w["A_v"], w["B_v"],
                                           geo.scale_k, geo.scale_v, geo.n_kv)[0]
        else:
            ref[b] = O.attend_decode_one(f64(q[b]), O.base_cache(Hn, w["W_k"]), O.base_cache(Hn, w["W_v"]), t, geo.n_kv)
    assert_close(f64(out), ref, f"head-sharded decode over {world} ranks")
    whole = f64(L.decode(q, agents, ctx))                # the unsharded call: same values up to fp32 summation order
    assert np.abs(f64(out) - whole).max() <= 2e-2
