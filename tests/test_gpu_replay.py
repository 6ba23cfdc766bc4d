"""The turn-loop replay issues the right work: token accounting per policy, cache contents after a
replay equal a one-shot projection of the same rows, and no device-side error is flagged."""
import pytest
import torch

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
    px.turn_project(st.desc, st.H[:64], st.WA[1], ref, P_last)
    torch.cuda.synchronize()
    blk = slice(P_last // 16 + 1, (P_last + 64) // 16)       # whole blocks inside [P_last, P_last + 64)
    assert torch.equal(st.caches[1].k_base[blk], ref.k_base[blk])
    assert torch.equal(st.caches[1].lr_v[:, blk], ref.lr_v[:, blk])
    assert px.poll_status() == 0
    px.close()
