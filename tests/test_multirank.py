"""The N > 1 path of the benchmark on CPU: two gloo ranks, each with its own batch (the path shards by
batch with no data-path collective), timing reduced as the maximum over ranks."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # each rank "measured" different times: the slowest decides
    mine = [10.0 + rank, 20.0 - rank, 0.5 * (rank + 1)]
    red = bench.max_over_ranks(mine, dist, "cpu")
    dist.barrier()
    value = bench.whole_job_throughput(16, world, red[0] / 100)
    torch.save({"red": red, "value": value}, out + f".{rank}")
    dist.destroy_process_group()


def test_two_rank_max_reduce_and_weak_scaling(tmp_path):
    port, out = _free_port(), str(tmp_path / "r")
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    r0, r1 = torch.load(out + ".0"), torch.load(out + ".1")
    assert r0["red"] == r1["red"] == [11.0, 20.0, 1.0]
    # 2 ranks x 16 sequences per step, step time = slowest rank's 0.11 ms
    assert r0["value"] == pytest.approx(2 * 16 / 0.11e-3)


def test_single_rank_is_identity():
    import bench
    assert bench.max_over_ranks([1.0, 2.0]) == [1.0, 2.0]
    assert bench.whole_job_throughput(16, 1, 0.2) == pytest.approx(80000.0)
    w = bench.W.CONFIGS[3]
    assert bench.decode_bytes(w) == 570425344 and bench.decode_units(w) == 4194304
