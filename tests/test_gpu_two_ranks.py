"""Distributed Muon (Sec. 2.3, Algorithm 1) as two real ranks on one GPU: two
processes share cuda:0, each steps the matrices it owns through the C-ABI
library (muon_step_bucket on the compute stream), and the exchanges - the
gradient reduce-scatter and the in-place all-gather of the updated weights, on
the side stream - go through torch.distributed.  With one GPU the process group
is gloo, whose collectives on CUDA tensors are broadcast and all-reduce; the
wrapper expresses both exchanges through them there (NCCL, which needs one GPU
per rank, takes all_gather_into_tensor / reduce_scatter_tensor on the same
storage).  No kernel of one rank waits for a kernel of the other.

The result must be the single-process result bit for bit: two steps of a plain
context over all matrices, on the summed gradients.
"""

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

pytestmark = pytest.mark.gpu

# two orientations of one bucket (odd number of row blocks: tiles shared by two matrices), a square
# bucket with fewer matrices than would divide evenly, fp32 weights, and a bucket only one rank owns
SHAPES = [(328, 200, 5, torch.bfloat16, torch.bfloat16), (200, 328, 2, torch.bfloat16, torch.bfloat16),
          (256, 256, 3, torch.bfloat16, torch.bfloat16), (136, 264, 2, torch.float32, torch.bfloat16),
          (384, 520, 1, torch.bfloat16, torch.bfloat16)]


def _grad(rows, cols, gen, scale):
    # multiples of 2^-13 below 2^-6 in magnitude: the sum over ranks is exact in bf16
    return torch.randint(-64, 65, (rows, cols), generator=gen).float() * (2.0 ** -13) * scale


def _fill(weights, grads, seed, scale, only_grads=False):
    gen = torch.Generator().manual_seed(seed)
    for gi, (rows, cols, n, wd, gd) in enumerate(SHAPES):
        for j in range(n):
            w = (torch.randn(rows, cols, generator=gen) * 0.02).to(wd)
            if not only_grads:
                weights[gi][j].copy_(w)
            grads[gi][j].copy_(_grad(rows, cols, gen, scale).to(gd))


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
    torch.cuda.set_device(0)
    from paper_2502_16982_b200 import binding
    from paper_2502_16982_b200.distributed import DistributedMuon

    dm = DistributedMuon(SHAPES, "cuda:0", dist=dist)
    hp = binding.Hyper(lr=1e-2, wd=0.1)
    timing = {}
    for step in range(2):
        # every rank contributes (rank + 1) x the step's base gradient
        _fill(dm.weights, dm.grads, 500 + step, float(rank + 1), only_grads=bool(step))
        dm.step(hp, reduce_grads=True, timing=timing)
    torch.cuda.synchronize()
    status = dm.status()
    total_ms = timing["start"].elapsed_time(timing["end"])
    exch_ms = sum(a.elapsed_time(b) for a, b in timing["exchanges"])
    torch.save({"w": [w.cpu().clone() for ws in dm.weights for w in ws], "status": status, "owned": len(dm.owned),
                "launches": dm._ctx.muon_last_launch_count() if dm._ctx is not None else 0,
                "exchanges": len(timing["exchanges"]), "total_ms": total_ms, "exch_ms": exch_ms,
                "bytes": dm.gather_bytes_per_rank}, out % rank)
    dm.close()
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.timeout(600)
def test_two_processes_on_one_gpu_give_the_single_process_bits(tmp_path):
    from paper_2502_16982_b200 import binding, workloads as wl

    out = str(tmp_path / "rank%d.pt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    r0, r1 = torch.load(out % 0), torch.load(out % 1)
    assert r0["status"][0] == 0 and r1["status"][0] == 0
    total = sum(s[2] for s in SHAPES)
    assert r0["owned"] + r1["owned"] == total and min(r0["owned"], r1["owned"]) >= total // 2 - 2
    assert r0["launches"] > 0 and r1["launches"] > 0           # both ranks ran the CUDA step
    n_buckets = 4
    assert r0["exchanges"] == r1["exchanges"] == 2 * n_buckets  # a reduce-scatter and a gather per bucket
    assert r0["bytes"] == r1["bytes"] > 0

    # single process: plain context over all matrices, gradients 3 x the base (1 x + 2 x)
    W = [torch.zeros((n, r, c), dtype=wd, device="cuda") for (r, c, n, wd, gd) in SHAPES]
    G = [torch.zeros((n, r, c), dtype=gd, device="cuda") for (r, c, n, wd, gd) in SHAPES]
    M = [torch.zeros((n, r, c), dtype=torch.float32, device="cuda") for (r, c, n, wd, gd) in SHAPES]
    ctx = binding.MuonContext([(wl.views(w), wl.views(g), wl.views(m)) for w, g, m in zip(W, G, M)])
    try:
        hp = binding.Hyper(lr=1e-2, wd=0.1)
        for step in range(2):
            _fill([wl.views(w) for w in W], [wl.views(g) for g in G], 500 + step, 3.0, only_grads=bool(step))
            ctx.muon_step(hp)
        assert ctx.muon_status()[0] == 0
        single = [w.cpu() for ws in W for w in ws]
    finally:
        ctx.muon_destroy()
    assert len(single) == len(r0["w"]) == len(r1["w"])
    for a, b_, c in zip(r0["w"], r1["w"], single):
        assert torch.equal(a, c) and torch.equal(b_, c)
