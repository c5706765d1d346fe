"""Host logic of the multi-GPU bench path on CPU ranks (gloo, world size 2):
one parameter set is partitioned over the ranks, the slowest rank sets the step
time (MAX-reduce), and the whole-job value is the work of the one job over that
time."""

import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2502_16982_b200 import workloads as wl

    # every rank draws the same parameter set (same seeds): the job is one set, partitioned
    spec = wl.GroupSpec(16, 24, 3)
    W, G, M = wl.make_group(spec, 3000, "cpu")
    gathered = [torch.zeros_like(G, dtype=torch.float32) for _ in range(world)]
    dist.all_gather(gathered, G.float())
    same = torch.equal(gathered[0], gathered[1])
    # the slowest rank sets the step time
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    val = bench.whole_job_value(2.0e12, ms)
    if rank == 0:
        torch.save({"same": same, "ms": ms, "value": val, "shape": tuple(G.shape)}, out)
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.timeout(600)
def test_two_cpu_ranks_shard_and_reduce(tmp_path):
    out = str(tmp_path / "r0.pt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    res = torch.load(out)
    assert res["same"]
    assert res["shape"] == (3, 16, 24)
    assert res["ms"] == 15.0
    # a 2 TFLOP job in 15 ms
    assert abs(res["value"] - 2.0 / 15e-3) < 1e-9


def test_single_process_identity():
    import bench

    assert bench.max_over_ranks(3.5, None, torch.device("cpu")) == 3.5
    assert abs(bench.whole_job_value(14.8e12, 14.0) - 14.8 / 14.0e-3) < 1e-9
