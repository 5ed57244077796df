"""GPU parity of the double-precision verification path (fpde_fwd_f64 / fpde_bwd_f64) against the
fp64 CPU oracle.  Both sides compute in double, so only the order of a handful of additions per
node differs: tolerance 1e-12 relative to the largest entry of each array."""
import numpy as np
import pytest

import oracle
from paper_2607_18020_b200 import binding as B
from paper_2607_18020_b200 import workloads as W

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

TOL = 1e-12
CASES = [
    ("burgers_256x128", (4, 4)), ("burgers_256x128", (5, 9)), ("burgers_256x128", (37, 23)),
    ("poisson_1024", (3, 4)), ("poisson_1024", (36, 40)),
    ("grayscott_4096", (3, 4)), ("grayscott_4096", (17, 12)),
    ("helmholtz_256", (5, 5, 8)), ("helmholtz_256", (12, 20, 24)),
    ("ns_tgv_128x16", (3, 3, 3, 4)), ("ns_tgv_128x16", (5, 6, 7, 12)),
    ("ns2d_steady_4096", (3, 4)), ("ns2d_steady_4096", (36, 40)),
    ("ns3d_steady_256", (3, 3, 4)), ("ns3d_steady_256", (7, 5, 12)),
    ("ns_tgv_xslab_34", (3, 3, 3, 4)), ("ns_tgv_xslab_34", (6, 5, 4, 8)),
    ("grayscott_xslab_1026", (3, 4)), ("grayscott_xslab_1026", (9, 12)),
]


def _close(a, b, what):
    a = np.asarray(a, dtype=np.float64); b = np.asarray(b, dtype=np.float64)
    scale = np.abs(b).max() if b.size and np.abs(b).max() > 0 else 1.0
    err = np.abs(a - b).max() / scale
    assert err <= TOL, "%s: max error %.3e relative to the largest entry" % (what, err)


def _dev(arrs):
    return [torch.from_numpy(np.ascontiguousarray(a, dtype=np.float64)).cuda() for a in arrs]


@pytest.mark.parametrize("name,shape", CASES)
@pytest.mark.parametrize("seed", [42, 43])
def test_f64_path_against_oracle(name, shape, seed):
    w = W.make(name, seed=seed, shape=shape, kind="randn")
    # the oracle sees the same doubles the GPU gets (fp32 inputs widened)
    R_ref, loss_ref, g_ref, rows = oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    fields, sources = _dev(w.fields), _dev(w.sources)
    ne = len(W.OP_META[w.op]["residuals"])
    res = [torch.full(w.shape, 7.0, dtype=torch.float64, device="cuda") for _ in range(ne)]
    loss = torch.full((ne + 1,), -1.0, dtype=torch.float64, device="cuda")
    ws = torch.empty(B.workspace_bytes_f64(w.op, w.shape), dtype=torch.uint8, device="cuda")
    B.fpde_fwd_f64(w.op, fields, sources, res, loss, w.shape, w.spacing, w.coeffs, w.bc, ws)
    grads = [torch.full(w.shape, 9.0, dtype=torch.float64, device="cuda") for _ in w.fields]
    B.fpde_bwd_f64(w.op, fields, res, [2.0 / rows] * ne, grads, w.shape, w.spacing, w.coeffs, w.bc)
    torch.cuda.synchronize()
    for e in range(ne):
        _close(res[e].cpu().numpy(), R_ref[e], "%s residual %d" % (name, e))
    L = loss.cpu().numpy()
    assert np.all(np.abs(L - loss_ref) <= 1e-12 * np.abs(loss_ref) + 1e-300), (L, loss_ref)
    for f in range(len(w.fields)):
        _close(grads[f].cpu().numpy(), g_ref[f], "%s gradient %d" % (name, f))


def test_f64_adjoint_ignores_upstream_entries_without_a_row():
    w = W.make("helmholtz_256", seed=44, shape=(9, 10, 12), kind="randn")
    Gs = W.random_sensitivities(w, seed=7)
    ref = oracle.bwd(w.op, w.fields, [0.5 * g.astype(np.float64) for g in Gs], w.shape, w.spacing, w.coeffs)
    grads = [torch.empty(w.shape, dtype=torch.float64, device="cuda")]
    B.fpde_bwd_f64(w.op, _dev(w.fields), _dev(Gs), [0.5], grads, w.shape, w.spacing, w.coeffs, w.bc)
    torch.cuda.synchronize()
    _close(grads[0].cpu().numpy(), ref[0], "helmholtz adjoint on arbitrary upstream")


def test_f32_kernels_agree_with_the_f64_path():
    """The fast fp32 kernels against the fp64 GPU path on the same inputs: the two GPU
    implementations of the formulas, held against each other."""
    w = W.make("ns_tgv_128x16", seed=42, shape=(8, 12, 16, 8))
    ne, rows = 4, B.row_count(w.op, w.shape)
    f32 = [torch.from_numpy(f).cuda() for f in w.fields]
    r32 = [torch.empty(w.shape, dtype=torch.float32, device="cuda") for _ in range(ne)]
    B.fpde_fwd(w.op, f32, [], r32, None, w.shape, w.spacing, w.coeffs, w.bc, None)
    f64 = _dev(w.fields)
    r64 = [torch.empty(w.shape, dtype=torch.float64, device="cuda") for _ in range(ne)]
    B.fpde_fwd_f64(w.op, f64, [], r64, None, w.shape, w.spacing, w.coeffs, w.bc, None)
    torch.cuda.synchronize()
    for a, b in zip(r32, r64):
        d = (a.double() - b).norm() / b.norm()
        assert float(d) <= 1e-5
