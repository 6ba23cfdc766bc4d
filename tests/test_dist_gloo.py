"""The N > 1 path of the benchmark is "independent replicas": each rank runs the same workload, the
step time is the max over ranks and the value sums the ranks' units.  Covered here on CPU with gloo."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms = bench.reduce_max_ms(10.0 + 5.0 * rank)          # rank 1 is the slow one
    val = bench.whole_job_value(1e9, 2, ms, world)
    # every rank generates its own replica's inputs from its own seed: they must differ
    from paper_2609_34054_b200 import inputs as I
    h = I.hidden_states(4, I.C1, seed=rank)
    gathered = [torch.zeros_like(h, dtype=torch.float32) for _ in range(world)]
    dist.all_gather(gathered, h.float())
    out[rank] = (ms, val, bool(torch.equal(gathered[0], gathered[1])))
    dist.destroy_process_group()


def test_replica_aggregation_world_size_2():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 15.0                 # max over ranks
    assert abs(res[0][1] - 2 * 1e9 * 2 / 15e-3 / 1e9) < 1e-9 and res[0][1] == res[1][1]
    assert res[0][2] is False                             # replicas see different seeded inputs


def test_bench_gpus_flag_starts_that_many_ranks():
    """`python bench.py --gpus 2` without a launcher re-executes itself under torch.distributed.run with two ranks;
    here with the stub step on gloo: the line must come from rank 0, count two ranks with different pids, take the
    slower rank's time and sum the ranks' units."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "5", "--stub-workload"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                      # rank 0 alone prints
    d = lines[0]
    assert d["n_gpus"] == 2 and d["stub"] and d["scaling"] == "weak"
    ranks = d["config"]["ranks"]
    assert [x["rank"] for x in ranks] == [0, 1] and ranks[0]["pid"] != ranks[1]["pid"]
    assert d["ms_per_step"] >= 2.0                              # rank 1 sleeps 2 ms per step: the max over ranks
    assert abs(d["value"] - 2 * 1e6 * 5 / (d["ms_per_step"] * 5e-3) / 1e9) < 1e-9


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max_ms(3.5) == 3.5
    assert bench.whole_job_value(2e9, 1, 1000.0, 1) == 2.0


def test_reference_arm_is_silent_on_nonzero_ranks(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import bench
    import argparse
    monkeypatch.setenv("RANK", "1")
    assert bench.run_reference(argparse.Namespace(gpus=2, steps=1, warmup=0)) == 0
    assert capsys.readouterr().out == ""


# ---------------------------------------------------------------- context-sharded decode: host logic

def test_shard_ranges_cover_every_token_once():
    sys.path.insert(0, ROOT)
    from paper_2609_34054_b200.sharded import shard_ranges
    ctx = [0, 1, 15, 16, 17, 100, 4097, 32768]
    for world in (1, 2, 3, 4, 8):
        ranges = shard_ranges(ctx, world)
        assert len(ranges) == world and all(len(r) == len(ctx) for r in ranges)
        for i, c in enumerate(ctx):
            pos = 0
            for r in range(world):
                s, e = ranges[r][i]
                assert s == pos and e >= s and (s % 16 == 0 or s == c)      # contiguous, rank order, page-aligned starts
                pos = e
            assert pos == c                                                 # exactly [0, ctx)
        sizes = [ranges[r][-1][1] - ranges[r][-1][0] for r in range(world)]
        assert max(sizes) - min(sizes) <= 16                                # balanced to within a page


def _gather_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2609_34054_b200.sharded import gather_records
    local = torch.full((3, 2, 24), float(rank + 1), dtype=torch.float32)
    local[0, 0, 0] = 100.0 + rank
    got = gather_records(local)
    reuse = torch.empty((world, 3, 2, 24), dtype=torch.float32)
    again = gather_records(local, None, reuse)
    out[rank] = (tuple(got.shape), [float(got[s, 1, 1, 5]) for s in range(world)], [float(got[s, 0, 0, 0]) for s in range(world)],
                 again.data_ptr() == reuse.data_ptr() and bool(torch.equal(again, got)))
    dist.destroy_process_group()


def test_gather_records_layout_world_size_2():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_gather_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    for r in range(world):
        shape, vals, tags, reused = res[r]
        assert shape == (2, 3, 2, 24) and vals == [1.0, 2.0] and tags == [100.0, 101.0] and reused   # slot s holds rank s's records


def _gather_heads_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2609_34054_b200.sharded import gather_heads
    B, hq, hd = 3, 2, 4
    local = torch.arange(B * hq * hd, dtype=torch.float32).reshape(B, hq, hd) + 1000.0 * rank
    got = gather_heads(local)
    buf = torch.empty((B, world * hq, hd), dtype=torch.float32)
    again = gather_heads(local, None, None, buf)
    out[rank] = (tuple(got.shape), [float(got[1, r * hq + 1, 2]) for r in range(world)], bool(torch.equal(again, got)),
                 again.data_ptr() == buf.data_ptr())
    dist.destroy_process_group()


def test_gather_heads_layout_world_size_2():
    """Head-sharded decode: rank r's query heads land at [r * n_q_local, (r + 1) * n_q_local) of every request."""
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_gather_heads_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    for r in range(world):
        shape, vals, same, reused = res[r]
        assert shape == (3, 4, 4) and vals == [14.0, 1014.0] and same and reused


def test_head_shard_planning():
    sys.path.insert(0, ROOT)
    from paper_2609_34054_b200 import inputs as I
    from paper_2609_34054_b200.sharded import head_shard_geometry, head_slice
    g = head_shard_geometry(I.C3, 4)
    assert (g.n_q, g.n_kv, g.hd, g.rank_k, g.n_agents, g.d_model) == (8, 2, 128, 32, 4, 4096) and g.scale_k == I.C3.scale_k
    assert [head_slice(r, 4, 8) for r in range(4)] == [slice(0, 2), slice(2, 4), slice(4, 6), slice(6, 8)]
    try:
        head_shard_geometry(I.C3, 3)
        assert False
    except ValueError:
        pass
