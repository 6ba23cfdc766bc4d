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
