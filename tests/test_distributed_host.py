"""Owner-computes partition and weight all-gather (Sec. 2.3) on CPU: the
partition is pure host code in the C library; the gather runs on two gloo
ranks with a stand-in for the per-matrix step."""

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


def test_slot_partition_is_consistent_and_balanced():
    """muon_partition_slots: every matrix of a bucket has a distinct (owner,
    position) below the slot capacity, the owners of a bucket appear in runs,
    the counts per rank differ by at most one within a bucket, and the longer
    runs go to the ranks that were least loaded before the bucket."""
    from paper_2502_16982_b200 import binding as b

    bf, f32 = b.MUON_DTYPE_BF16, b.MUON_DTYPE_FP32
    shapes = [(2048, 1408, 132, bf, bf), (1408, 2048, 66, bf, bf), (2048, 2048, 27, bf, bf),
              (2048, 11264, 2, bf, bf), (11264, 2048, 1, bf, bf), (512, 4096, 27, f32, bf)]
    bucket_of, n_buckets = b.muon_plan_buckets(shapes)
    for world in (1, 2, 3, 8):
        owners, pos, share, loads = b.muon_partition_slots(shapes, world)
        assert b.muon_partition_slots(shapes, world)[:3] == (owners, pos, share)
        cost = []
        for r, c, n, _, _ in shapes:
            m_, n_ = min(r, c), max(r, c)
            cost += [3.0 * m_ * m_ * n_ + float(m_) ** 3] * n
        for u in range(n_buckets):
            members = [i for i, bu in enumerate(bucket_of) if bu == u]
            assert share[u] == -(-len(members) // world)
            cells = {(owners[i], pos[i]) for i in members}
            assert len(cells) == len(members) and all(0 <= p < share[u] for _, p in cells)
            per_rank = [sum(1 for i in members if owners[i] == rk) for rk in range(world)]
            assert max(per_rank) - min(per_rank) <= 1
            for rk in range(world):  # a slot fills from the front
                assert sorted(pos[i] for i in members if owners[i] == rk) == list(range(per_rank[rk]))
            assert [owners[i] for i in members] == sorted(owners[i] for i in members)  # consecutive runs
        mine = [sum(c for c, o in zip(cost, owners) if o == rk) for rk in range(world)]
        assert all(abs(a - l) <= 1e-6 * max(l, 1.0) for a, l in zip(mine, loads))
        assert max(loads) - min(loads) <= max(cost) * (1 + 1e-12) + 1e-6 * max(loads)


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


# 16x8 and 8x16 share a bucket (same short and long side); the 4x4 bf16 and fp32 groups do not
# (dtypes differ); the single 32x8 matrix is a bucket only one rank owns
SHAPES = [(8, 12, 3, torch.float32, torch.float32), (16, 8, 2, torch.float32, torch.float32),
          (4, 4, 4, torch.bfloat16, torch.bfloat16), (8, 16, 3, torch.float32, torch.float32),
          (32, 8, 1, torch.float32, torch.float32), (4, 4, 2, torch.float32, torch.float32)]


def _fill(dm, seed, grad_scale=1.0):
    """The same weights and gradients on every rank, whatever the slot layout."""
    gen = torch.Generator().manual_seed(seed)
    for gi, (rows, cols, n, wd, gd) in enumerate(SHAPES):
        for j in range(n):
            dm.weights[gi][j].copy_(torch.randn(rows, cols, generator=gen).to(wd))
            dm.grads[gi][j].copy_(_grad(rows, cols, gen, grad_scale).to(gd))


def _grad(rows, cols, gen, scale):
    # multiples of 1/16 in [-1, 1]: sums over the ranks are exact in bf16, so a reduce-scatter of
    # (rank + 1) x g gives the bits of 3 x g in any order of summation
    return torch.randint(-16, 17, (rows, cols), generator=gen).float() / 16.0 * scale


def _worker(rank, world, port, out, reduce_grads):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2502_16982_b200.distributed import DistributedMuon

    dm = DistributedMuon(SHAPES, "cpu", dist=dist, step_fn=_fake_step)
    # with reduce_grads every rank contributes (rank + 1) x the base gradient: the sum is 3 x
    _fill(dm, 123, grad_scale=float(rank + 1) if reduce_grads else 1.0)
    for step in range(2):
        if step and reduce_grads:
            _fill_grads_only(dm, 124, float(rank + 1))
        dm.step(0.1, reduce_grads=reduce_grads)
    n_mom = sum(len(ms) for _, _, ms in dm.local_groups)
    torch.save({"w": [w.clone() for ws in dm.weights for w in ws], "owned": len(dm.owned), "mom": n_mom,
                "units": dm.n_units, "unit_of": dm.unit_of, "share": dm.share,
                "stepped": [len(ms) for ms in dm.unit_mats]}, out % rank)
    dist.barrier()
    dist.destroy_process_group()


def _fill_grads_only(dm, seed, grad_scale):
    gen = torch.Generator().manual_seed(seed)
    for gi, (rows, cols, n, wd, gd) in enumerate(SHAPES):
        for j in range(n):
            dm.grads[gi][j].copy_(_grad(rows, cols, gen, grad_scale).to(gd))


@pytest.mark.timeout(600)
@pytest.mark.parametrize("reduce_grads", [False, True])
def test_two_ranks_end_with_the_single_process_weights(tmp_path, reduce_grads):
    out = str(tmp_path / "rank%d.pt")
    mp.spawn(_worker, args=(2, _free_port(), out, reduce_grads), nprocs=2, join=True)
    r0, r1 = torch.load(out % 0), torch.load(out % 1)
    # single process: every matrix stepped locally, on the summed gradients
    from paper_2502_16982_b200.distributed import DistributedMuon

    dm = DistributedMuon(SHAPES, "cpu", dist=None, step_fn=_fake_step)
    scale = 3.0 if reduce_grads else 1.0
    _fill(dm, 123, grad_scale=scale)
    for step in range(2):
        if step and reduce_grads:
            _fill_grads_only(dm, 124, scale)
        dm.step(0.1)
    single = [w for ws in dm.weights for w in ws]
    assert r0["owned"] + r1["owned"] == len(single) and r0["owned"] > 0 and r1["owned"] > 0
    assert r0["mom"] == r0["owned"] and r1["mom"] == r1["owned"]  # momentum only for owned matrices
    # the exchange's units: five buckets, the same on both ranks; the two orientations share one
    assert r0["units"] == r1["units"] == 5 and r0["unit_of"] == r1["unit_of"] and r0["share"] == r1["share"]
    u = r0["unit_of"]
    assert u[3] == u[4] == u[9] == u[10] == u[11] and u[5] != u[13] and len(set(u)) == 5
    assert r0["share"] == [-(-u.count(k) // 2) for k in range(5)]
    # each unit's matrices are stepped by exactly one rank each, and the one-matrix unit by one rank alone
    both = [a + b_ for a, b_ in zip(r0["stepped"], r1["stepped"])]
    assert both == [u.count(k) for k in range(5)]
    assert sorted((r0["stepped"][u[12]], r1["stepped"][u[12]])) == [0, 1]
    for a, b_, c in zip(r0["w"], r1["w"], single):
        assert torch.equal(a, c) and torch.equal(b_, c)
