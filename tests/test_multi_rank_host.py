"""Host logic of the multi-GPU bench path on CPU ranks (gloo, world size 2):
matrices are independent units, so every rank owns its own shard and the only
cross-rank step is the MAX-reduce of the step time; the whole-job value is the
work of all ranks over the slowest rank's time."""

import os
import socket
import sys

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

    # each rank draws its own shard: same shapes, different values
    spec = wl.GroupSpec(16, 24, 3)
    W, G, M = wl.make_group(spec, bench.rank_seed(3, 0, rank), "cpu")
    gathered = [torch.zeros_like(G, dtype=torch.float32) for _ in range(world)]
    dist.all_gather(gathered, G.float())
    distinct = not torch.equal(gathered[0], gathered[1])
    # the slowest rank sets the step time
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    val = bench.whole_job_value(2.0e12, world, ms)
    if rank == 0:
        torch.save({"distinct": distinct, "ms": ms, "value": val, "shape": tuple(G.shape)}, out)
    dist.barrier()
    dist.destroy_process_group()


def test_two_cpu_ranks_shard_and_reduce(tmp_path):
    out = str(tmp_path / "r0.pt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    res = torch.load(out)
    assert res["distinct"]
    assert res["shape"] == (3, 16, 24)
    assert res["ms"] == 15.0
    # 2 ranks x 2 TFLOP in 15 ms
    assert abs(res["value"] - 2 * 2.0 / 15e-3) < 1e-9


def test_single_process_identity():
    import bench

    assert bench.max_over_ranks(3.5, None, torch.device("cpu")) == 3.5
    assert bench.rank_seed(3, 1, 0) == 3001 and bench.rank_seed(3, 1, 2) == 203001
