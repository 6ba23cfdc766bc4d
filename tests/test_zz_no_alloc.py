"""The allocation-free decode entry point against the ordinary one.

Some callers of this library cannot allocate device memory when they call it: an engine whose KV-cache
pool took all of HBM at start-up, code that runs while a stream is being captured, a decode loop that
must not pay cudaMalloc's device-wide synchronisation.  For them `precc_lr_attend_decode_static` keeps
the split-merge scratch in an array built into the library.  This file is collected last on purpose, so
that a run that stops at the first failure has already run every other test.
"""
import pytest
import torch

from paper_2609_34054_b200 import inputs as I
from paper_2609_34054_b200.binding import Cache, Precc, PreccError, layer_desc

pytestmark = pytest.mark.gpu


def _case(px, geo, ctx_list, seed):
    """Caches filled directly; returns everything both entry points need."""
    B = len(ctx_list)
    need = [(c + I.PAGE - 1) // I.PAGE for c in ctx_list]
    nb = sum(need)
    c = I.direct_caches(nb, geo, seed)
    cache = Cache.from_tensors(geo, c["k_base"].cuda(), c["v_base"].cuda(), c["lr_k"].cuda(), c["lr_v"].cuda())
    w = I.layer_weights(geo, seed)
    table = I.block_tables(torch.tensor(ctx_list), nb, seed).cuda()
    q = I.queries(B, geo, seed, gain=2.0).cuda()
    aid = torch.tensor([i % geo.n_agents for i in range(B)], dtype=torch.int32, device="cuda")
    cl = torch.tensor(ctx_list, dtype=torch.int32, device="cuda")
    return dict(desc=layer_desc(geo), q=q, aid=aid, cl=cl, mx=max(ctx_list), Bk=w["B_k"].cuda(), Bv=w["B_v"].cuda(),
                cache=cache, table=table)


def _run_both(px, k):
    ws = px.decode_workspace(k["desc"], k["q"].shape[0], k["mx"])
    ref = torch.full_like(k["q"], float("nan"))
    px.lr_attend_decode(k["desc"], k["q"], k["aid"], k["cl"], k["mx"], k["Bk"], k["Bv"], k["cache"], ref, ws, k["table"])
    got = torch.full_like(k["q"], float("nan"))
    torch.cuda.synchronize()
    free_before, reserved_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_reserved()
    px.lr_attend_decode_static(k["desc"], k["q"], k["aid"], k["cl"], k["mx"], k["Bk"], k["Bv"], k["cache"], got, k["table"])
    torch.cuda.synchronize()
    # the call took no device memory: neither from the driver nor from torch's pool
    assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_reserved() == reserved_before
    return got, ref


def test_static_scratch_decode_matches_workspace_decode_twice_in_a_row():
    px = Precc(0)
    geo = I.Geometry(256, 8, 2, 128, 3, 16, 16, alpha=32.0)
    # 40 requests x 2 kv heads: more units than the short-latency path takes, so the split records and
    # arrival counters in the scratch are really used; the second case has different sizes, so it finds
    # the first call's leftovers in the shared array
    cases = [_case(px, geo, [1500 + 37 * i for i in range(40)], seed=3),
             _case(px, geo, [3000 - 61 * i for i in range(44)], seed=4)]
    warm = cases[0]                      # the first call on a device looks the array's address up: not measured
    px.lr_attend_decode_static(warm["desc"], warm["q"], warm["aid"], warm["cl"], warm["mx"], warm["Bk"], warm["Bv"],
                               warm["cache"], torch.empty_like(warm["q"]), warm["table"])
    for k in cases:
        got, ref = _run_both(px, k)
        assert torch.isfinite(got.float()).all()
        # same split schedule, same kernel, same summation order: the two entry points agree bit for bit
        # (which is inside the 2e-2 + 1e-2 |ref| bar the other tests use)
        assert torch.equal(got, ref), f"max abs diff {(got.float() - ref.float()).abs().max().item():.3e}"
    assert px.poll_status() == 0
    px.close()


def test_static_scratch_rejects_oversized_requests():
    px = Precc(0)
    geo = I.C4
    k = _case(px, I.Geometry(256, 8, 2, 128, 3, 16, 16, alpha=32.0), [64, 64], seed=5)
    big = layer_desc(geo)
    n = px.lib.precc_decode_workspace_bytes(big, 4096, 32768, px.sm_count)
    assert n > (8 << 20)
    q = torch.zeros((4096, geo.n_q, geo.hd), dtype=torch.bfloat16, device="cuda")
    ids = torch.zeros(4096, dtype=torch.int32, device="cuda")
    out = torch.full_like(q, 7.0)                      # sentinel: a rejected call must not touch its output
    with pytest.raises(PreccError, match="WORKSPACE.*built-in array"):
        px.lr_attend_decode_static(big, q, ids, ids, 32768, k["Bk"], k["Bv"], k["cache"], out)
    torch.cuda.synchronize()
    assert (out == 7.0).all() and px.poll_status() == 0
    px.close()
