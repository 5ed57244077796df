"""GPU parity of the loss-specialised pass fpde_fwd_bwd (loss + dL/dfield from one call) against
the fp64 CPU oracle: single-pass kernels where the operator has one, the two-kernel sequence
elsewhere.  Same tolerances as the two-call path."""
import numpy as np
import pytest

import oracle
from paper_2607_18020_b200 import binding as B
from paper_2607_18020_b200 import workloads as W

from gpu_util import LOSS_TOL, Guarded, assert_close, to_dev

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

SINGLE_PASS = [
    ("poisson_1024", (3, 4)),
    ("poisson_1024", (5, 8)),
    ("poisson_1024", (36, 40)),
    ("poisson_1024", (203, 300)),          # ragged column group (75 float4 = 2.5 warps), several row chunks
    ("poisson_1024", (64, 484)),           # 121 float4: one column past four full warps
    ("poisson_1024", None),
    ("grayscott_4096", (3, 4)),
    ("grayscott_4096", (17, 12)),
    ("grayscott_4096", (70, 120)),         # exactly one warp's 30 float4
    ("grayscott_4096", (67, 124)),         # 31 float4: the wrap-around neighbour sits in another warp
    ("grayscott_4096", (1000, 1032)),
    ("ns2d_steady_4096", (3, 4)),
    ("ns2d_steady_4096", (36, 40)),
    ("ns2d_steady_4096", (203, 300)),
    ("ns2d_steady_4096", (128, 128)),
]
TWO_KERNEL = [
    ("burgers_256x128", (37, 23)),
    ("helmholtz_256", (12, 20, 24)),
    ("helmholtz_256", (70, 45, 136)),              # ragged z line: the adjoint runs without zero-extension here
    ("helmholtz_256", (5, 5, 8)),
    ("helmholtz_256", (41, 128, 128)),             # build with the y and z extents fixed
    ("ns_tgv_128x16", (8, 12, 16, 8)),
    ("ns3d_steady_256", (7, 5, 132)),
    ("ns3d_steady_256", (37, 22, 136)),
    ("ns3d_steady_256", (3, 3, 4)),
]


def _run(w, store, with_loss=True):
    """store: which residual arrays to ask for (list of bool)."""
    fields = to_dev(torch, w.fields)
    sources = to_dev(torch, w.sources)
    ne = len(W.OP_META[w.op]["residuals"])
    res = [Guarded(torch, w.shape, fill=7.0) if s else None for s in store]
    grads = [Guarded(torch, w.shape, fill=9.0) for _ in w.fields]
    loss = torch.full((ne + 1,), -1.0, dtype=torch.float64, device="cuda") if with_loss else None
    ws = torch.empty(B.fwd_bwd_workspace_bytes(w.op, w.shape), dtype=torch.uint8, device="cuda")
    B.fpde_fwd_bwd(w.op, fields, sources, [r.view if r is not None else None for r in res] if any(store) else None,
                   [g.view for g in grads], loss, w.shape, w.spacing, w.coeffs, w.bc, ws)
    torch.cuda.synchronize()
    for a in res + grads:
        if a is not None:
            a.check()
    return res, grads, loss


def _check(w, tag, store):
    R_ref, loss_ref, g_ref, rows = oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    res, grads, loss = _run(w, store)
    L = loss.cpu().numpy()
    assert np.all(np.abs(L - loss_ref) <= LOSS_TOL * np.abs(loss_ref) + 1e-300), (tag, L, loss_ref)
    for f, (g, gr) in enumerate(zip(grads, g_ref)):
        assert_close(g.view.cpu().numpy(), gr, "%s gradient %d" % (tag, f))
    for e, r in enumerate(res):
        if r is not None:
            assert_close(r.view.cpu().numpy(), R_ref[e], "%s residual %d" % (tag, e))
    return grads, loss


@pytest.mark.parametrize("name,shape", SINGLE_PASS)
def test_single_pass_config_fields(name, shape):
    w = W.make(name, seed=42, shape=shape)
    assert B.has_single_pass(w.op)
    ne = len(W.OP_META[w.op]["residuals"])
    _check(w, "%s%s" % (name, shape or ""), [False] * ne)


@pytest.mark.parametrize("name,shape", SINGLE_PASS[:-1])
@pytest.mark.parametrize("seed", [42, 43])
def test_single_pass_randn_fields_with_residuals(name, shape, seed):
    if shape is None:
        pytest.skip("covered by the config-field case")
    w = W.make(name, seed=seed, shape=shape, kind="randn")
    ne = len(W.OP_META[w.op]["residuals"])
    _check(w, "%s%s randn" % (name, shape), [True] * ne)
    if ne > 1:                                       # only some residual arrays asked for
        _check(w, "%s%s randn partial" % (name, shape), [e == 1 for e in range(ne)])


@pytest.mark.parametrize("name", ["grayscott_4096", "ns2d_steady_4096"])
def test_single_pass_full_size(name):
    w = W.make(name, seed=42)
    ne = len(W.OP_META[w.op]["residuals"])
    _check(w, name + " full size", [False] * ne)


def test_single_pass_unequal_spacing():
    for name, shape, h in [("poisson_1024", (20, 24), (0.3, 0.07)), ("grayscott_4096", (9, 8), (0.01, 0.02)),
                           ("ns2d_steady_4096", (9, 12), (0.3, 0.2))]:
        w = W.make(name, seed=45, shape=shape, kind="randn", spacing=h)
        _check(w, name + " unequal spacing", [True] * len(W.OP_META[w.op]["residuals"]))


def test_single_pass_matches_two_call_path_and_is_reproducible():
    w = W.make("grayscott_4096", seed=42, shape=(512, 512))
    _, g1, l1 = _run(w, [False, False])
    _, g2, l2 = _run(w, [True, True])
    assert torch.equal(l1, l2)                       # fixed-order loss: bit-identical across calls
    for a, b in zip(g1, g2):
        assert torch.equal(a.view, b.view)
    _, g3, _ = _run(w, [False, False], with_loss=False)
    for a, b in zip(g1, g3):
        assert torch.equal(a.view, b.view)


@pytest.mark.parametrize("name,shape", TWO_KERNEL)
def test_two_kernel_operators(name, shape):
    w = W.make(name, seed=42, shape=shape, kind="randn")
    assert not B.has_single_pass(w.op)
    ne = len(W.OP_META[w.op]["residuals"])
    _check(w, "%s%s" % (name, shape), [True] * ne)
    # these operators need the residual arrays as the intermediate
    fields = to_dev(torch, w.fields)
    grads = [torch.empty(w.shape, dtype=torch.float32, device="cuda") for _ in w.fields]
    st = B.fwd_bwd_status(w.op, fields, to_dev(torch, w.sources), None, grads, None, w.shape, w.spacing, w.coeffs,
                          w.bc, None, 0, None)
    assert st == 2


@pytest.mark.parametrize("shape", [(9, 16, 128), (21, 45, 128), (12, 24, 256), (37, 50, 256)])
@pytest.mark.parametrize("store_res", [False, True])
def test_helmholtz_single_pass_prototype(shape, store_res, monkeypatch):
    """FPDE_STAR3D_SINGLE_PASS=1: residual, loss and gradient of the Helmholtz operator from one kernel
    (planes of r handed from the forward star to the adjoint star through shared memory) on grids
    whose z lines are 128 or 256 floats; ragged row tiles, CTAs whose share spans several tiles."""
    monkeypatch.setenv("FPDE_STAR3D_SINGLE_PASS", "1")
    w = W.make("helmholtz_256", seed=49, shape=shape, kind="randn")
    R_ref, loss_ref, g_ref, _ = oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    fields, sources = to_dev(torch, w.fields), to_dev(torch, w.sources)
    res = Guarded(torch, shape, fill=7.0) if store_res else None
    grad = Guarded(torch, shape, fill=9.0)
    loss = torch.full((2,), -1.0, dtype=torch.float64, device="cuda")
    ws = torch.empty(B.fwd_bwd_workspace_bytes(w.op, shape), dtype=torch.uint8, device="cuda")
    B.fpde_fwd_bwd(w.op, fields, sources, [res.view] if store_res else None, [grad.view], loss, shape, w.spacing,
                   w.coeffs, w.bc, ws)
    torch.cuda.synchronize()
    grad.check()
    assert_close(grad.view.cpu().numpy(), g_ref[0], "helmholtz single pass %s gradient" % (shape,))
    L = loss.cpu().numpy()
    assert np.all(np.abs(L - loss_ref) <= LOSS_TOL * np.abs(loss_ref)), (L, loss_ref)
    if store_res:
        res.check()
        assert_close(res.view.cpu().numpy(), R_ref[0], "helmholtz single pass %s residual" % (shape,))
    assert B.diag_tma_timeouts() == 0


@pytest.mark.parametrize("name,shape", [("poisson_1024", (40, 48)), ("ns_tgv_128x16", (9, 8, 8, 8)), ("grayscott_4096", (48, 64))])
def test_prepared_step_is_the_same_calls_with_the_arguments_marshalled_once(name, shape):
    """PreparedStep.fwd / bwd / fwd_bwd give bit for bit what fpde_fwd / fpde_bwd / fpde_fwd_bwd give."""
    w = W.make(name, seed=51, shape=shape, kind="randn")
    fields, sources = to_dev(torch, w.fields), to_dev(torch, w.sources)
    ne = len(W.OP_META[w.op]["residuals"])
    mk = lambda n: [torch.full(shape, 3.0, dtype=torch.float32, device="cuda") for _ in range(n)]
    res_a, res_b, g_a, g_b, g_c, g_d = mk(ne), mk(ne), mk(len(fields)), mk(len(fields)), mk(len(fields)), mk(len(fields))
    loss_a = torch.zeros(ne + 1, dtype=torch.float64, device="cuda"); loss_b = loss_a.clone() - 1
    loss_c = loss_a.clone() - 2; loss_d = loss_a.clone() - 3
    ws = torch.empty(B.workspace_bytes(w.op, shape), dtype=torch.uint8, device="cuda")
    ws2 = torch.empty(B.fwd_bwd_workspace_bytes(w.op, shape), dtype=torch.uint8, device="cuda")
    rows = B.row_count(w.op, shape)
    B.fpde_fwd(w.op, fields, sources, res_a, loss_a, shape, w.spacing, w.coeffs, w.bc, ws)
    B.fpde_bwd(w.op, fields, res_a, [2.0 / rows] * ne, g_a, shape, w.spacing, w.coeffs, w.bc)
    step = B.PreparedStep(w.op, fields, sources, res_b, g_b, loss_b, shape, w.spacing, w.coeffs, w.bc, workspace=ws,
                          fwd_bwd_workspace=ws2)
    step.fwd(); step.bwd()
    torch.cuda.synchronize()
    for a, b in zip(res_a + g_a, res_b + g_b):
        assert torch.equal(a, b)
    assert torch.equal(loss_a, loss_b)
    # the one-call entry point, through the binding and through the prepared step
    store = not B.has_single_pass(w.op)
    res_c, res_d = mk(ne), mk(ne)
    B.fpde_fwd_bwd(w.op, fields, sources, res_c if store else None, g_c, loss_c, shape, w.spacing, w.coeffs, w.bc, ws2)
    step2 = B.PreparedStep(w.op, fields, sources, res_d, g_d, loss_d, shape, w.spacing, w.coeffs, w.bc, workspace=ws,
                           fwd_bwd_workspace=ws2)
    step2.fwd_bwd(store_residuals=store)
    torch.cuda.synchronize()
    for a, b in zip(g_c, g_d):
        assert torch.equal(a, b)
    assert torch.equal(loss_c, loss_d)
