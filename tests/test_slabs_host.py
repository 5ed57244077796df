"""Slab decomposition, host side: the plane ranges and halo transfer lists (pure arithmetic), and
the exchange itself between two gloo ranks on CPU tensors (no kernels: every rank fills its own
planes with their global plane number and checks what lands in its halo)."""
import os
import socket
import sys

import numpy as np
import pytest

from paper_2607_18020_b200 import binding as B
from paper_2607_18020_b200 import slabs as S
from paper_2607_18020_b200 import workloads as W

torch = pytest.importorskip("torch")


def _expected_plane(plan, local):
    return (plan.wide[0] + local) % plan.shape[0]


@pytest.mark.parametrize("op,shape,world", [(W.NS_3D_T, (16, 4, 4, 8), 1), (W.NS_3D_T, (16, 4, 4, 8), 2),
                                            (W.NS_3D_T, (17, 4, 4, 8), 3), (W.HELMHOLTZ_3D_O4, (19, 6, 8), 3),
                                            (W.POISSON_2D, (11, 8), 4), (W.NS_3D_STEADY, (9, 5, 8), 2),
                                            (W.GRAYSCOTT_2D, (10, 8), 2)])
def test_ranges_and_transfers(op, shape, world):
    ps = S.plans(op, shape, world)
    R = ps[0].radius
    covered = []
    for p in ps:
        x0, x1 = p.owned
        covered += list(range(x0, x1))
        t0, t1 = p.tight
        w0, w1 = p.wide
        assert w0 <= t0 <= x0 < x1 <= t1 <= w1
        if p.periodic:
            assert (t0, t1, w0, w1) == (x0 - R, x1 + R, x0 - 2 * R, x1 + 2 * R)
        else:
            assert t0 == max(0, x0 - R) and w1 == min(shape[0], x1 + 2 * R)
        for halo in (R, 2 * R):
            lo, hi = p._range(halo)
            got = np.full(p.local_shape[0], -1)
            for t in p.halo_transfers(halo):
                a, b = ps[t.peer].owned_of(t.peer)
                assert a <= t.start and t.start + t.count <= b          # one owner per run
                got[t.dst:t.dst + t.count] = np.arange(t.start, t.start + t.count)
            for g in list(range(lo, x0)) + list(range(x1, hi)):
                assert got[p.local_of(g)] == g % shape[0]
            for g in range(x0, x1):
                assert got[p.local_of(g)] == -1                         # own planes are never overwritten
    assert covered == list(range(shape[0]))


def test_too_thin_slabs_are_refused():
    with pytest.raises(ValueError):
        S.plans(W.HELMHOLTZ_3D_O4, (12, 6, 8), 4)       # 3 planes per rank < 2 * radius
    with pytest.raises(ValueError):
        S.plans(W.BURGERS_1D_T, (16, 8), 2)             # no slab form


def test_local_exchange_on_cpu_tensors():
    for op, shape, world in [(W.NS_3D_T, (13, 2, 2, 4), 3), (W.HELMHOLTZ_3D_O4, (14, 3, 4), 3)]:
        ps = S.plans(op, shape, world)
        arrs = []
        for p in ps:
            a = torch.full(p.local_shape, -1.0)
            x0, x1 = p.owned
            for g in range(x0, x1):
                a[p.local_of(g)] = float(g)
            arrs.append([a])
        S.exchange_local(ps, arrs, 2 * ps[0].radius)
        for p, (a,) in zip(ps, arrs):
            for l in range(p.local_shape[0]):
                assert float(a[l].flatten()[0]) == _expected_plane(p, l)
        # stacked form: one tensor per rank holding two arrays
        stacks = []
        for p in ps:
            st = torch.full((2,) + tuple(p.local_shape), -1.0)
            x0, x1 = p.owned
            for g in range(x0, x1):
                st[0, p.local_of(g)] = float(g)
                st[1, p.local_of(g)] = float(g) + 100.0
            stacks.append(st)
        S.exchange_local(ps, stacks, 2 * ps[0].radius)
        for p, st in zip(ps, stacks):
            for l in range(p.local_shape[0]):
                assert float(st[0, l].flatten()[0]) == _expected_plane(p, l)
                assert float(st[1, l].flatten()[0]) == _expected_plane(p, l) + 100.0


def _rank_main(rank, world, port, op, shape):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        plan = S.plans(op, shape, world)[rank]
        arrs = []
        for k in range(2):                                   # two arrays per exchange, as with several fields
            a = torch.full(plan.local_shape, -1.0)
            x0, x1 = plan.owned
            for g in range(x0, x1):
                a[plan.local_of(g)] = float(g) + 100.0 * k
            arrs.append(a)
        S.exchange_dist(plan, arrs, 2 * plan.radius, dist)
        for k, a in enumerate(arrs):
            for l in range(plan.local_shape[0]):
                assert float(a[l].flatten()[0]) == _expected_plane(plan, l) + 100.0 * k, (rank, k, l)
        # the same through one stacked tensor and a posted exchange that is waited for later
        st = torch.full((2,) + tuple(plan.local_shape), -1.0)
        x0, x1 = plan.owned
        for k in range(2):
            for g in range(x0, x1):
                st[k, plan.local_of(g)] = float(g) + 100.0 * k
        ex = S.post_exchange(plan, st, 2 * plan.radius, dist)
        ex.wait()
        for k in range(2):
            for l in range(plan.local_shape[0]):
                assert float(st[k, l].flatten()[0]) == _expected_plane(plan, l) + 100.0 * k, (rank, k, l)
        sums = torch.tensor([float(rank + 1), 2.0 * (rank + 1)], dtype=torch.float64)
        dist.all_reduce(sums, op=dist.ReduceOp.SUM)
        assert sums.tolist() == [3.0, 6.0]
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("op,shape", [(W.NS_3D_T, (12, 2, 2, 4)), (W.HELMHOLTZ_3D_O4, (13, 3, 4))])
def test_exchange_between_two_gloo_ranks(op, shape):
    import torch.multiprocessing as mp
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    mp.spawn(_rank_main, args=(2, port, op, shape), nprocs=2, join=True)


def test_chunk_plan_keeps_inner_launches_off_the_halo_planes():
    """The launches queued while the halo planes are in flight must neither cover nor read a plane an
    exchange fills: checked plane by plane from the chunk length the library reports."""
    for shape, world in (((128, 128, 128, 16), 2), ((128, 128, 128, 16), 4), ((121, 16, 16, 16), 1), ((50, 8, 8, 8), 2)):
        for plan in S.plans(W.NS_3D_T, shape, world):
            rank = S.SlabRank(torch, B, plan, (0.1,) * 4, (0.01,), device="cpu")
            cp = rank.chunk_plan()
            assert cp is not None, (shape, world)
            R = plan.radius
            for (K, lo, hi), n, halo_lo in ((cp[0], plan.tight_shape[0], range(0, R)),
                                            (cp[1], plan.local_shape[0], range(R, 2 * R))):
                P = B.plane_chunk(plan.local_op, (n,) + tuple(shape[1:]))
                assert K == -(-n // P) and 1 <= lo < hi < K
                halo = set(halo_lo) | {n - 1 - h for h in halo_lo}
                read = set()
                for a in range(lo * P, min(hi * P, n)):
                    read.update(range(a - R, a + R + 1))
                assert not (read & halo), (shape, world, plan.rank, sorted(read & halo))
    # an operator without launches over plane ranges, and a slab too short to have inner chunks
    short = S.SlabRank(torch, B, S.plans(W.NS_3D_T, (8, 8, 8, 8), 2)[0], (0.1,) * 4, (0.01,), device="cpu")
    assert short.chunk_plan() is None
    hh = S.SlabRank(torch, B, S.plans(W.HELMHOLTZ_3D_O4, (64, 16, 16), 2)[0], (0.1,) * 3, (1.0,), device="cpu")
    assert hh.chunk_plan() is None
