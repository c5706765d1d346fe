"""Owner-computes partition and weight all-gather (Sec. 2.3) on CPU: the
partition is pure host code in the C library; the gather runs on two gloo
ranks with a stand-in for the per-matrix step."""

import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def test_partition_covers_balances_and_is_deterministic():
    from paper_2502_16982_b200 import binding as b

    shapes = [(2048, 1408, 132), (1408, 2048, 66), (2048, 2048, 27), (2048, 11264, 2), (512, 4096, 27)]
    total = sum(n for _, _, n in shapes)
    for world in (1, 2, 3, 8):
        owners, loads = b.muon_partition(shapes, world)
        assert len(owners) == total and set(owners) <= set(range(world))
        assert b.muon_partition(shapes, world)[0] == owners
        # recompute the loads from the table with the same cost model
        cost = []
        for r, c, n in shapes:
            m_, n_ = min(r, c), max(r, c)
            cost += [3.0 * m_ * m_ * n_ + float(m_) ** 3] * n
        mine = [sum(c for c, o in zip(cost, owners) if o == rk) for rk in range(world)]
        assert all(abs(a - l) <= 1e-6 * max(l, 1.0) for a, l in zip(mine, loads))
        # longest-first greedy: no rank exceeds the mean by more than one heaviest matrix
        assert max(loads) - sum(loads) / world <= max(cost) * (1 + 1e-12)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _fake_step(mats, hp):
    # stand-in for the CUDA step: deterministic, touches owned weights and momentum only
    for w, g, m in mats:
        m.mul_(0.5).add_(g.float())
        w.sub_((hp * m).to(w.dtype))


def _make_groups(seed):
    # 16x8 and 8x16 share a bucket (same short and long side); the 4x4 bf16 and fp32
    # groups do not (dtypes differ); the single 32x8 matrix is a bucket only one rank owns
    gen = torch.Generator().manual_seed(seed)
    groups = []
    for rows, cols, n, dtype in ((8, 12, 3, torch.float32), (16, 8, 2, torch.float32), (4, 4, 4, torch.bfloat16),
                                 (8, 16, 3, torch.float32), (32, 8, 1, torch.float32), (4, 4, 2, torch.float32)):
        ws = [torch.randn(rows, cols, generator=gen).to(dtype) for _ in range(n)]
        gs = [torch.randn(rows, cols, generator=gen).to(dtype) for _ in range(n)]
        groups.append((ws, gs))
    return groups


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2502_16982_b200.distributed import DistributedMuon

    groups = _make_groups(123)  # identical on every rank, like replicated weights and reduced gradients
    dm = DistributedMuon(groups, dist=dist, step_fn=_fake_step)
    for _ in range(2):
        dm.step(0.1)
    n_owned = len(dm.owned)
    n_mom = sum(len(ms) for _, _, ms in dm.local_groups)
    torch.save({"w": [w.clone() for ws, _ in groups for w in ws], "owned": n_owned, "mom": n_mom,
                "units": dm.n_units, "unit_of": dm.unit_of,
                "stepped": [len(ms) for ms in dm.unit_mats]}, out % rank)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_end_with_the_single_process_weights(tmp_path):
    out = str(tmp_path / "rank%d.pt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    r0, r1 = torch.load(out % 0), torch.load(out % 1)
    # single process: every matrix stepped locally
    from paper_2502_16982_b200.distributed import DistributedMuon

    groups = _make_groups(123)
    dm = DistributedMuon(groups, dist=None, step_fn=_fake_step)
    for _ in range(2):
        dm.step(0.1)
    single = [w for ws, _ in groups for w in ws]
    assert r0["owned"] + r1["owned"] == len(single) and r0["owned"] > 0 and r1["owned"] > 0
    assert r0["mom"] == r0["owned"] and r1["mom"] == r1["owned"]  # momentum only for owned matrices
    # the gather's units: five buckets, the same on both ranks; the two orientations share one
    assert r0["units"] == r1["units"] == 5 and r0["unit_of"] == r1["unit_of"]
    u = r0["unit_of"]
    assert u[3] == u[4] == u[9] == u[10] == u[11] and u[5] != u[13] and len(set(u)) == 5
    # each unit's matrices are stepped by exactly one rank each, and the one-matrix unit by one rank alone
    both = [a + b_ for a, b_ in zip(r0["stepped"], r1["stepped"])]
    assert both == [u.count(k) for k in range(5)]
    assert sorted((r0["stepped"][u[12]], r1["stepped"][u[12]])) == [0, 1]
    for a, b_, c in zip(r0["w"], r1["w"], single):
        assert torch.equal(a, c) and torch.equal(b_, c)
