"""The turn-loop replay issues the right work: token accounting per policy, cache contents after a
replay equal a one-shot projection of the same rows, no device-side error is flagged - and what a replayed
trace leaves in the caches and returns from its last attention calls is what the oracle computes from the same
hidden states (Sections 3.1-3.2: the two ReBaseShared schedules end in logically equal cache states)."""
import numpy as np
import pytest
import torch

from oracle import lrkv_oracle as O
from harness import assert_close, base_rows, f64, lr_rows

from paper_2609_34054_b200 import inputs as I
from paper_2609_34054_b200 import replay as R
from paper_2609_34054_b200.binding import Cache, Precc

pytestmark = pytest.mark.gpu


def test_trace_recipes():
    t = R.three_agent_trace(17300)
    assert [x.agent for x in t] == [0, 1, 2, 0, 1, 2]
    assert abs(R.trace_tokens(t) - 17300) <= 2
    rr = R.round_robin_trace(4)
    assert len(rr) == 8 and R.trace_tokens(rr) == 8 * (8192 + 64) and [x.agent for x in rr[:5]] == [0, 1, 2, 3, 0]


def test_replay_policies_small():
    px = Precc(0)
    geo = I.Geometry(d_model=256, n_q=8, n_kv=2, hd=64, n_agents=3, rank_k=16, rank_v=16, alpha=32.0)
    turns = [R.Turn(0, 70, 5), R.Turn(1, 200, 4), R.Turn(2, 33, 3), R.Turn(0, 64, 2)]
    total = R.trace_tokens(turns)
    st = R.Stack(px, geo, n_layers=2, max_tokens=total + 16, max_rows=2 * total, private_tokens=220)
    res = {p: R.replay(st, turns, p) for p in R.POLICIES}
    for p, r in res.items():
        assert r["tokens"] == total and r["ttft_ms"] > 0 and r["decode_ms"] > 0 and r["total_ms"] >= r["ttft_ms"]
        assert (r["rebase_ms"] > 0) == (p == "rebase_lp")
    assert res["rebase_db"]["prefilled_tokens"] == 2 * sum(t.n_in for t in turns)        # both sequences
    n_in = sum(t.n_in for t in turns)
    assert res["prelr"]["prefilled_tokens"] == n_in == res["fullshared"]["prefilled_tokens"]
    # nonshared: agent 0 sees 75 new, agent 1 all 75 + 200, agent 2 all 279 + 33, agent 0 again everything since its turn
    assert res["nonshared"]["prefilled_tokens"] == 70 + (75 + 200) + (75 + 204 + 33) + (204 + 36 + 64)
    assert res["nonshared"]["cache_gb"] > res["prelr"]["cache_gb"] > res["fullshared"]["cache_gb"]
    # after the prelr replay the rows of the last turn's input equal a one-shot fused projection of the same rows
    R.replay(st, turns, "prelr")
    P_last = total - turns[-1].n_in - turns[-1].n_out
    ref = Cache(geo, st.caches[1].n_blocks, fill=0.0)
    px.turn_project(st.desc, st.H_adpt[P_last:P_last + 64], st.WA[1], ref, P_last)
    torch.cuda.synchronize()
    blk = slice(P_last // 16 + 1, (P_last + 64) // 16)       # whole blocks inside [P_last, P_last + 64)
    assert torch.equal(st.caches[1].k_base[blk], ref.k_base[blk])
    assert torch.equal(st.caches[1].lr_v[:, blk], ref.lr_v[:, blk])
    assert px.poll_status() == 0
    px.close()


def _expected_rebase_state(st, turns, layer):
    """What ReBaseShared leaves in the shared caches of `layer` (float64, token-major): base rows from the
    adapter-free hidden states everywhere; agent k's LR rows from the adapted hidden states on the turns k
    produced itself and from the adapter-free ones elsewhere."""
    geo = st.geo
    total = R.trace_tokens(turns)
    w = {k: f64(v) for k, v in I.layer_weights(geo, 0, f"L{layer}").items()}
    Ha, Hn = f64(st.H_adpt[:total]), f64(st.H_neut[:total])
    owner = np.concatenate([np.full(t.n_in + t.n_out, t.agent) for t in turns])
    exp = {"k": O.base_cache(Hn, w["W_k"]), "v": O.base_cache(Hn, w["W_v"]), "lk": [], "lv": [], "w": w, "Ha": Ha, "owner": owner}
    for k in range(geo.n_agents):
        Hk = np.where((owner == k)[:, None], Ha, Hn)
        exp["lk"].append(O.lr_cache(Hk, w["A_k"][k]))
        exp["lv"].append(O.lr_cache(Hk, w["A_v"][k]))
    return exp


def _check_shared_state(st, exp, layer, total, what):
    c = st.caches[layer]
    for name, got, ref in (("base K", base_rows(c.k_base)[:total], exp["k"]), ("base V", base_rows(c.v_base)[:total], exp["v"])):
        assert_close(got, ref, f"{what}: {name}", atol=1e-2, rtol=1e-2, norm_tol=1e-2)
    for k in range(st.geo.n_agents):
        assert_close(lr_rows(c.lr_k, k)[:total], exp["lk"][k], f"{what}: LR-K agent {k}", atol=2e-2, rtol=1e-2, norm_tol=1e-2)
        assert_close(lr_rows(c.lr_v, k)[:total], exp["lv"][k], f"{what}: LR-V agent {k}", atol=2e-2, rtol=1e-2, norm_tol=1e-2)


def test_replayed_rebase_schedules_match_the_oracle_and_each_other():
    px = Precc(0)
    geo = I.Geometry(d_model=256, n_q=8, n_kv=2, hd=64, n_agents=3, rank_k=16, rank_v=16, alpha=32.0)
    turns = [R.Turn(0, 70, 5), R.Turn(1, 200, 4), R.Turn(2, 33, 3), R.Turn(0, 64, 2)]
    total = R.trace_tokens(turns)
    last = turns[-1]
    P = total - last.n_in - last.n_out
    n_c = last.n_in + last.n_out
    layer = 1
    state = {}
    for policy in ("rebase_lp", "rebase_db"):
        st = R.Stack(px, geo, n_layers=2, max_tokens=total + 16, max_rows=2 * total, private_tokens=220)
        R.replay(st, turns, policy)
        torch.cuda.synchronize()
        exp = _expected_rebase_state(st, turns, layer)
        _check_shared_state(st, exp, layer, total, policy)
        w, j = exp["w"], last.agent
        if policy == "rebase_lp":
            # the last call of the replay: the adapter-free pass over the last turn's tokens (neutral prefill)
            ref = O.attend_prefill(f64(st.q[:n_c]), exp["k"], exp["v"], P, geo.n_kv)
            assert_close(f64(st.out[:n_c]), ref, "rebase_lp: adapter-free pass of the last turn")
        else:
            # the last decode step carried two requests: agent j over the shared context + its private adapted rows,
            # and the adapter-free view over the shared (neutral) rows; both attend all `total` tokens
            k_ad = np.concatenate([exp["k"][:P], O.base_cache(exp["Ha"][P:], w["W_k"])])
            v_ad = np.concatenate([exp["v"][:P], O.base_cache(exp["Ha"][P:], w["W_v"])])
            ref_ad = O.attend_from_caches(f64(st.q[0]), k_ad, v_ad, exp["lk"][j], exp["lv"][j], w["B_k"][j], w["B_v"][j],
                                          geo.scale_k, geo.scale_v, geo.n_kv)
            ref_nt = O.attend_decode_one(f64(st.q[1]), exp["k"], exp["v"], total, geo.n_kv)
            assert_close(f64(st.out[0]), ref_ad, "rebase_db: last adapted decode step")
            assert_close(f64(st.out[1]), ref_nt, "rebase_db: last adapter-free decode step")
        full = total // 16                      # whole blocks of the shared trajectory
        state[policy] = {n: (getattr(st.caches[layer], n)[:full] if n in ("k_base", "v_base")
                             else getattr(st.caches[layer], n)[:, :full]).float().cpu() for n in ("k_base", "v_base", "lr_k", "lr_v")}
        assert px.poll_status() == 0
        del st
    # lazy prefill and double batching end in the same shared cache state: equal up to the last bf16 bit (the two
    # schedules project a token in calls of different size, i.e. on kernels with different fp32 summation orders)
    for n in ("k_base", "v_base", "lr_k", "lr_v"):
        a, b = state["rebase_lp"][n], state["rebase_db"][n]
        # one bf16 ulp of the larger value, plus the fp32 round-off of a 256-term sum for entries that cancel to ~0
        ulp = torch.maximum(a.abs(), b.abs()) * 2.0 ** -7 + 1e-4
        assert ((a - b).abs() <= ulp).all(), f"{n}: lazy prefill and double batching differ by more than one bf16 ulp"
        assert (a == b).float().mean() > 0.9, f"{n}: most entries agree bit for bit"
    px.close()
