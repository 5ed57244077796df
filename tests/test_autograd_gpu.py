"""The torch.autograd.Function wrappers: gradients that flow through torch's autograd must be the
oracle's J^T G (arbitrary downstream loss) and the oracle's loss gradient (fused loss)."""
import numpy as np
import pytest

import oracle
from paper_2607_18020_b200 import workloads as W

from gpu_util import LOSS_TOL, assert_close

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

CASES = [("poisson_1024", (36, 40)), ("grayscott_4096", (24, 32)), ("helmholtz_256", (12, 10, 16)),
         ("ns_tgv_128x16", (6, 8, 8, 8)), ("burgers_256x128", (9, 7)), ("ns2d_steady_4096", (10, 12)),
         ("ns3d_steady_256", (6, 5, 8))]


@pytest.mark.parametrize("name,shape", CASES)
def test_fused_loss_backward(name, shape):
    from paper_2607_18020_b200.autograd import fused_residual_loss
    w = W.make(name, seed=45, shape=shape, kind="randn")
    fields = [torch.from_numpy(f).cuda().requires_grad_(True) for f in w.fields]
    sources = [torch.from_numpy(s).cuda() for s in w.sources]
    loss = fused_residual_loss(w.op, fields, sources, w.spacing, w.coeffs, w.bc)
    (3.0 * loss).backward()
    _, L, g, _ = oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    assert abs(loss.item() - L[-1]) <= LOSS_TOL * abs(L[-1])
    for f, gr in zip(fields, g):
        assert_close(f.grad.cpu().numpy(), 3.0 * gr, name + " autograd loss gradient")


@pytest.mark.parametrize("name,shape", CASES)
def test_residuals_with_downstream_loss(name, shape):
    from paper_2607_18020_b200.autograd import fused_residual
    w = W.make(name, seed=46, shape=shape, kind="randn")
    fields = [torch.from_numpy(f).cuda().requires_grad_(True) for f in w.fields]
    sources = [torch.from_numpy(s).cuda() for s in w.sources]
    res = fused_residual(w.op, fields, sources, w.spacing, w.coeffs, w.bc)
    wts = W.random_sensitivities(w, seed=9)
    total = sum((r * torch.from_numpy(wt).cuda()).sum() for r, wt in zip(res, wts))
    total.backward()
    R, _, _ = oracle.fwd(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    for r, rr in zip(res, R):
        assert_close(r.detach().cpu().numpy(), rr, name + " autograd residual")
    ref = oracle.bwd(w.op, w.fields, [x.astype(np.float64) for x in wts], w.shape, w.spacing, w.coeffs)
    for f, gr in zip(fields, ref):
        assert_close(f.grad.cpu().numpy(), gr, name + " autograd J^T w")


@pytest.mark.parametrize("name,shape", [("grayscott_4096", (5, 8)), ("ns2d_steady_4096", (5, 8)), ("burgers_256x128", (6, 5)),
                                        ("ns3d_steady_256", (4, 4, 4))])
def test_gradcheck_in_double_precision(name, shape):
    """fp64 tensors go through the double-precision kernels, so torch's own finite-difference
    check of the adjoint applies (the paper's fp64 verification mode)."""
    from paper_2607_18020_b200.autograd import fused_residual, fused_residual_loss
    w = W.make(name, seed=47, shape=shape, kind="randn")
    fields = [torch.from_numpy(f.astype(np.float64)).cuda().requires_grad_(True) for f in w.fields]
    sources = [torch.from_numpy(s.astype(np.float64)).cuda() for s in w.sources]
    assert torch.autograd.gradcheck(lambda *f: fused_residual(w.op, f, sources, w.spacing, w.coeffs, w.bc), fields,
                                    eps=1e-6, atol=1e-6, rtol=1e-6, nondet_tol=0.0)
    assert torch.autograd.gradcheck(lambda *f: fused_residual_loss(w.op, f, sources, w.spacing, w.coeffs, w.bc), fields,
                                    eps=1e-6, atol=1e-5, rtol=1e-5, nondet_tol=0.0)
