"""Slab decomposition on the GPU: several x-slabs of one grid processed in one process (the
kernels of different slabs run one after the other, halos are copied between the slabs' arrays)
must reproduce the whole-grid kernels, and the oracle on the whole grid."""
import numpy as np
import pytest

import oracle
from paper_2607_18020_b200 import binding as B
from paper_2607_18020_b200 import slabs as S
from paper_2607_18020_b200 import workloads as W

from gpu_util import LOSS_TOL, assert_close, run_bwd, run_fwd

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

CASES = [
    ("ns_tgv_128x16", (16, 8, 8, 8), 1),          # one slab: its halo planes are its own far planes
    ("ns_tgv_128x16", (16, 8, 8, 8), 2),
    ("ns_tgv_128x16", (37, 12, 8, 16), 3),        # uneven slabs, several plane chunks per slab
    ("helmholtz_256", (23, 10, 16), 3),
    ("poisson_1024", (40, 36), 4),
    ("ns2d_steady_4096", (30, 40), 2),
    ("ns3d_steady_256", (14, 6, 8), 3),
    ("grayscott_4096", (64, 96), 1),
    ("grayscott_4096", (67, 200), 3),
]


def _random_cases():
    """Randomly drawn (shape, number of slabs) per slab-capable operator, fixed seed."""
    rng = np.random.RandomState(20260719)
    out = []
    for name in ("ns_tgv_128x16", "helmholtz_256", "poisson_1024", "ns2d_steady_4096", "ns3d_steady_256", "grayscott_4096"):
        cfg = W.CONFIGS[name]
        nd = len(cfg["shape"])
        radius = S.RADIUS[cfg["op"]]
        for _ in range(6):
            world = int(rng.randint(1, 6))
            shape = [int(rng.randint(max(2 * radius * world, 4 * radius + 1), 2 * radius * world + 30))]
            for a in range(1, nd):
                if a == nd - 1:
                    shape.append(4 * int(rng.randint(2, 5 if nd == 4 else 30)))
                else:
                    shape.append(int(rng.randint(2 * radius + 1, 12)))
            out.append((name, tuple(shape), world))
    return out


@pytest.mark.parametrize("name,shape,world", CASES + _random_cases())
def test_slabs_reproduce_the_whole_grid(name, shape, world):
    w = W.make(name, seed=42, shape=shape, kind="randn")
    plan_list = S.plans(w.op, w.shape, world)
    ranks = [S.SlabRank(torch, B, p, w.spacing, w.coeffs) for p in plan_list]
    for r in ranks:
        r.load_owned(w.fields, w.sources)
    loss = S.step_local(ranks)
    torch.cuda.synchronize()
    # assemble the owned planes
    res = [torch.cat([r.owned(r.res)[e] for r in ranks]).cpu().numpy() for e in range(ranks[0].ne)]
    grads = [torch.cat([r.owned(r.grads)[f] for r in ranks]).cpu().numpy() for f in range(ranks[0].nf)]
    # (a) the whole-grid kernels: the same arithmetic per node, so identical bits
    fields, sources, res_w, loss_w = run_fwd(torch, w)
    rows = B.row_count(w.op, w.shape)
    grads_w = run_bwd(torch, w, fields, [r.view for r in res_w], [2.0 / rows] * len(res_w))
    for e, r in enumerate(res_w):
        assert np.array_equal(res[e], r.view.cpu().numpy()), "residual %d differs from the whole-grid kernel" % e
    for f, g in enumerate(grads_w):
        assert np.array_equal(grads[f], g.view.cpu().numpy()), "gradient %d differs from the whole-grid kernel" % f
    # (b) the oracle on the whole grid
    R_ref, loss_ref, g_ref, rows_ref = oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    assert rows == rows_ref == sum(r.rows_local for r in ranks)
    L = loss.cpu().numpy()
    assert np.all(np.abs(L - loss_ref) <= LOSS_TOL * np.abs(loss_ref) + 1e-300), (L, loss_ref)
    for e in range(len(res)):
        assert_close(res[e], R_ref[e], "%s slabs residual %d" % (name, e))
    for f in range(len(grads)):
        assert_close(grads[f], g_ref[f], "%s slabs gradient %d" % (name, f))


def test_step_dist_with_one_rank():
    """The per-process step on one rank (no process group needed: a periodic slab's halos are its
    own far planes)."""
    w = W.make("ns_tgv_128x16", seed=43, shape=(12, 8, 8, 8), kind="randn")
    rank = S.SlabRank(torch, B, S.plans(w.op, w.shape, 1)[0], w.spacing, w.coeffs)
    rank.load_owned(w.fields, w.sources)
    loss = S.step_dist(rank, dist=None)
    torch.cuda.synchronize()
    _, loss_ref, g_ref, _ = oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    assert abs(float(loss[-1]) - loss_ref[-1]) <= LOSS_TOL * abs(loss_ref[-1])
    for f, g in enumerate(rank.owned(rank.grads)):
        assert_close(g.cpu().numpy(), g_ref[f], "one-rank slab gradient %d" % f)


@pytest.mark.parametrize("name,shape", [("ns_tgv_128x16", (23, 8, 8, 8)), ("ns_tgv_xslab_34", (30, 6, 8, 16)),
                                        ("ns_tgv_xslab_34", (34, 128, 128, 16))])   # short and wide: a shortened chunk
def test_launches_over_plane_chunks_add_up_to_the_full_launch(name, shape):
    """fpde_fwd_chunks / fpde_bwd_chunks over a partition of the chunks of x-planes, in any order, write
    what one full launch writes, bit for bit, and the loss formed by the last call is the full launch's."""
    w = W.make(name, seed=44, shape=shape, kind="randn")
    fields, sources, res_w, loss_w = run_fwd(torch, w)
    rows = B.row_count(w.op, w.shape)
    grads_w = run_bwd(torch, w, fields, [r.view for r in res_w], [2.0 / rows] * len(res_w))
    P = B.plane_chunk(w.op, w.shape)
    assert P > 0
    K = -(-shape[0] // P)
    assert K >= 3
    res = [torch.full(shape, 7.0, dtype=torch.float32, device="cuda") for _ in res_w]
    grads = [torch.full(shape, 9.0, dtype=torch.float32, device="cuda") for _ in fields]
    loss = torch.full((len(res) + 1,), -1.0, dtype=torch.float64, device="cuda")
    ws = torch.empty(B.workspace_bytes(w.op, shape), dtype=torch.uint8, device="cuda")
    parts = [(1, K - 1), (K - 1, K), (0, 1)]                    # inner chunks first, then the two ends
    for i, (lo, hi) in enumerate(parts):
        B.fpde_fwd_chunks(w.op, fields, sources, res, loss, shape, w.spacing, w.coeffs, w.bc, ws, 0, lo, hi,
                          i == len(parts) - 1)
    for lo, hi in parts:
        B.fpde_bwd_chunks(w.op, fields, res, [2.0 / rows] * len(res), grads, shape, w.spacing, w.coeffs, w.bc, lo, hi)
    torch.cuda.synchronize()
    for a, b in zip(res, res_w):
        assert torch.equal(a, b.view)
    for a, b in zip(grads, grads_w):
        assert torch.equal(a, b.view)
    # the loss: the same partial sums when the ranged launches use the full launch's own chunk length
    # (the first two grids); a shortened chunk sums the same squares in other groups
    assert torch.allclose(loss, loss_w, rtol=1e-6, atol=0.0)
    if shape[1] < 128:
        assert torch.equal(loss, loss_w)
    assert B.plane_chunk(W.HELMHOLTZ_3D_O4, (32, 32, 32)) == 0


def test_step_dist_overlap_plan_on_one_rank():
    """One rank, a slab long enough to have chunks of planes away from its halos: the step that queues
    those chunks before waiting for the halo planes gives the oracle's loss and gradients."""
    w = W.make("ns_tgv_128x16", seed=45, shape=(26, 8, 8, 8), kind="randn")
    rank = S.SlabRank(torch, B, S.plans(w.op, w.shape, 1)[0], w.spacing, w.coeffs)
    rank.load_owned(w.fields, w.sources)
    plan = rank.chunk_plan()
    assert plan is not None and plan[0][1] >= 1 and plan[0][2] < plan[0][0] and plan[1][2] > plan[1][1]
    loss = S.step_dist(rank, dist=None, overlap=True)
    torch.cuda.synchronize()
    _, loss_ref, g_ref, _ = oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    assert np.all(np.abs(loss.cpu().numpy() - loss_ref) <= LOSS_TOL * np.abs(loss_ref))
    for f, g in enumerate(rank.owned(rank.grads)):
        assert_close(g.cpu().numpy(), g_ref[f], "overlapped one-rank slab gradient %d" % f)
