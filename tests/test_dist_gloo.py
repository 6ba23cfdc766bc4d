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
