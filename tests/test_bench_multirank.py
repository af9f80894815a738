"""Host logic of the N>1 benchmark path (independent replicas, max-over-ranks timing) on CPU with
the gloo backend, world size 2."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank 1 is the slower replica for the first number, rank 0 for the second
    got = bench.max_over_ranks([10.0 + rank, 5.0 - rank], dist, torch.device("cpu"))
    dist.barrier()
    out[rank] = got
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_with_gloo():
    world = 2
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, 29533, out), nprocs=world, join=True)
        assert out[0] == out[1] == [11.0, 5.0]
    sys.path.insert(0, ROOT)
    import bench
    # two replicas of 1 TFLOP each finishing within 1 ms -> 2000 TFLOP/s for the whole job
    assert abs(bench.aggregate_tflops(2, 1e12, 1.0) - 2000.0) < 1e-9
    assert bench.max_over_ranks([3.0, 4.0], None, None) == [3.0, 4.0]


def test_reference_arm_exits_silently_on_nonzero_rank(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import bench
    monkeypatch.setenv("RANK", "1")
    bench.run_reference(None)
    assert capsys.readouterr().out == ""
