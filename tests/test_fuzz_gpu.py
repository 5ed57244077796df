"""Randomly drawn grid shapes (fixed seed) for every operator: residuals, loss, gradients of the
two-call path and of fpde_fwd_bwd against the fp64 CPU oracle.  The hand-picked cases of the other
files aim at known edges (warp boundaries, ragged tails, chunk ends); this sweep is there for the
combinations nobody thought of."""
import numpy as np
import pytest

import oracle
from paper_2607_18020_b200 import binding as B
from paper_2607_18020_b200 import workloads as W

from gpu_util import LOSS_TOL, assert_close, run_bwd, run_fwd, to_dev

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

CONFIG_OF = ["burgers_256x128", "poisson_1024", "grayscott_4096", "helmholtz_256", "ns_tgv_128x16",
             "ns2d_steady_4096", "ns3d_steady_256", "ns_tgv_xslab_34", "grayscott_xslab_1026"]
PER_OP = 25
MAX_POINTS = 100000


def _draw_shapes():
    rng = np.random.RandomState(20260718)
    cases = []
    for name in CONFIG_OF:
        cfg = W.CONFIGS[name]
        radius = 2 if cfg["op"] == W.HELMHOLTZ_3D_O4 else 1
        nd = len(cfg["shape"])
        got = 0
        while got < PER_OP:
            shape = []
            for a in range(nd):
                lo = 4 if cfg["bc"][a] == W.ONE_SIDED else 2 * radius + 1
                if a == nd - 1:
                    top = 6 if nd == 4 else 80
                    n = 4 * rng.randint((lo + 3) // 4, top + 1)
                else:
                    n = rng.randint(lo, 14 if nd == 4 else (40 if nd == 3 else 150))
                shape.append(int(n))
            if int(np.prod(shape)) <= MAX_POINTS:
                cases.append((name, tuple(shape), int(rng.randint(1, 1 << 30))))
                got += 1
    return cases


CASES = _draw_shapes()


@pytest.mark.parametrize("name,shape,seed", CASES, ids=["%s-%s" % (n, "x".join(map(str, s))) for n, s, _ in CASES])
def test_random_shape(name, shape, seed):
    w = W.make(name, seed=seed, shape=shape, kind="randn")
    tag = "%s%s seed %d" % (name, shape, seed)
    R_ref, loss_ref, g_ref, rows = oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    assert rows == B.row_count(w.op, w.shape)
    fields, sources, res, loss = run_fwd(torch, w)
    for e, (r, rr) in enumerate(zip(res, R_ref)):
        assert_close(r.view.cpu().numpy(), rr, "%s residual %d" % (tag, e))
    L = loss.cpu().numpy()
    assert np.all(np.abs(L - loss_ref) <= LOSS_TOL * np.abs(loss_ref) + 1e-300), (tag, L, loss_ref)
    grads = run_bwd(torch, w, fields, [r.view for r in res], [2.0 / rows] * len(res))
    for f, (g, gr) in enumerate(zip(grads, g_ref)):
        assert_close(g.view.cpu().numpy(), gr, "%s gradient %d" % (tag, f))
    # the one-call path (single-pass kernel where there is one)
    g1 = [torch.full(w.shape, 3.0, dtype=torch.float32, device="cuda") for _ in w.fields]
    r1 = [torch.full(w.shape, 5.0, dtype=torch.float32, device="cuda") for _ in res]
    l1 = torch.zeros(len(res) + 1, dtype=torch.float64, device="cuda")
    ws = torch.empty(max(16, B.fwd_bwd_workspace_bytes(w.op, w.shape)), dtype=torch.uint8, device="cuda")
    B.fpde_fwd_bwd(w.op, fields, sources, r1, g1, l1, w.shape, w.spacing, w.coeffs, w.bc, ws)
    torch.cuda.synchronize()
    assert np.all(np.abs(l1.cpu().numpy() - loss_ref) <= LOSS_TOL * np.abs(loss_ref) + 1e-300), tag
    for f, (g, gr) in enumerate(zip(g1, g_ref)):
        assert_close(g.cpu().numpy(), gr, "%s one-call gradient %d" % (tag, f))
    for e, (r, rr) in enumerate(zip(r1, R_ref)):
        assert_close(r.cpu().numpy(), rr, "%s one-call residual %d" % (tag, e))


@pytest.mark.parametrize("name,shape,seed", CASES[::3], ids=["%s-%s" % (n, "x".join(map(str, s))) for n, s, _ in CASES[::3]])
def test_random_shape_adjoint_of_arbitrary_upstream_arrays(name, shape, seed):
    """fpde_bwd and its double-precision twin on upstream arrays that are not residuals (non-zero at
    nodes without a row, where they must be ignored), unequal spacings and unequal scales."""
    rng = np.random.RandomState(seed)
    h = tuple(float(x) for x in rng.uniform(0.05, 0.4, size=len(shape)))
    w = W.make(name, seed=seed, shape=shape, kind="randn", spacing=h)
    G = W.random_sensitivities(w, seed=seed + 1)
    gscale = [float(x) for x in rng.uniform(0.2, 2.0, size=len(G))]
    ref = oracle.bwd(w.op, w.fields, [s * g.astype(np.float64) for s, g in zip(gscale, G)], w.shape, w.spacing, w.coeffs)
    fields = to_dev(torch, w.fields)
    grads = run_bwd(torch, w, fields, to_dev(torch, G), gscale)
    for f, (g, gr) in enumerate(zip(grads, ref)):
        assert_close(g.view.cpu().numpy(), gr, "%s%s adjoint %d" % (name, shape, f))
    f64 = [torch.from_numpy(np.ascontiguousarray(a, dtype=np.float64)).cuda() for a in w.fields]
    g64 = [torch.from_numpy(np.ascontiguousarray(a, dtype=np.float64)).cuda() for a in G]
    out = [torch.empty(w.shape, dtype=torch.float64, device="cuda") for _ in w.fields]
    B.fpde_bwd_f64(w.op, f64, g64, gscale, out, w.shape, w.spacing, w.coeffs, w.bc)
    torch.cuda.synchronize()
    ref64 = oracle.bwd(w.op, [a.astype(np.float64) for a in w.fields],
                       [s * g.astype(np.float64) for s, g in zip(gscale, G)], w.shape, w.spacing, w.coeffs)
    for f, (g, gr) in enumerate(zip(out, ref64)):
        d = np.abs(g.cpu().numpy() - gr).max()
        assert d <= 1e-11 * max(1.0, np.abs(gr).max()), "%s%s fp64 adjoint %d: %g" % (name, shape, f, d)


def _staged_helmholtz_shapes():
    """Randomly drawn grids wide enough for the shared-memory staged Helmholtz engine (z lines of 136
    floats and more, 40 rows and more), fixed seed: ragged tiles in y and z, few and many planes."""
    rng = np.random.RandomState(20261125)
    out = []
    for _ in range(10):
        out.append((int(rng.randint(8, 40)), int(rng.randint(40, 90)), 4 * int(rng.randint(34, 100))))
    return out


@pytest.mark.parametrize("shape", _staged_helmholtz_shapes())
def test_fuzz_staged_helmholtz_engine(shape, monkeypatch):
    """Forward on the staged engine too (FPDE_STAR3D_TMA_FWD=1), adjoint of the residuals and of an
    arbitrary upstream array with entries off the rows, against the oracle."""
    monkeypatch.setenv("FPDE_STAR3D_TMA", "1")
    monkeypatch.setenv("FPDE_STAR3D_TMA_FWD", "1")
    w = W.make("helmholtz_256", seed=50, shape=shape, kind="randn")
    R_ref, loss_ref, g_ref, rows = oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    fields, sources, res, loss = run_fwd(torch, w)
    assert_close(res[0].view.cpu().numpy(), R_ref[0], "staged helmholtz %s residual" % (shape,))
    assert np.all(np.abs(loss.cpu().numpy() - loss_ref) <= LOSS_TOL * np.abs(loss_ref))
    grads = run_bwd(torch, w, fields, [res[0].view], [2.0 / rows])
    assert_close(grads[0].view.cpu().numpy(), g_ref[0], "staged helmholtz %s gradient" % (shape,))
    rng = np.random.default_rng(7)
    G = rng.standard_normal(shape).astype(np.float32)
    g2_ref = oracle.bwd(w.op, w.fields, [G.astype(np.float64) * 0.5], w.shape, w.spacing, w.coeffs)
    grads2 = run_bwd(torch, w, fields, to_dev(torch, [G]), [0.5])
    assert_close(grads2[0].view.cpu().numpy(), g2_ref[0], "staged helmholtz %s arbitrary upstream" % (shape,))
    assert B.diag_tma_timeouts() == 0
