"""Helpers for the GPU parity tests: run a workload through the C ABI, compare with the oracle."""
import numpy as np

from paper_2607_18020_b200 import binding as B
from paper_2607_18020_b200 import workloads as W

REL_L2_TOL = 1e-5      # ||a-b||_2 / ||b||_2 per output array
MAX_REL_TOL = 1e-4     # ||a-b||_inf / ||b||_inf per output array
LOSS_TOL = 1e-5        # |L - L_ref| / |L_ref|

GUARD = 64             # floats of canary on each side of every output array


def errors(a, b):
    a = np.asarray(a, dtype=np.float64).reshape(-1)
    b = np.asarray(b, dtype=np.float64).reshape(-1)
    d = a - b
    n2 = np.linalg.norm(b)
    ni = np.abs(b).max() if b.size else 0.0
    l2 = np.linalg.norm(d) / n2 if n2 > 0 else np.linalg.norm(d)
    mx = np.abs(d).max() / ni if ni > 0 else (np.abs(d).max() if d.size else 0.0)
    return float(l2), float(mx)


def assert_close(a, b, what):
    l2, mx = errors(a, b)
    assert l2 <= REL_L2_TOL and mx <= MAX_REL_TOL, "%s: rel-L2 %.3e (tol %.0e), max-rel %.3e (tol %.0e)" % (
        what, l2, REL_L2_TOL, mx, MAX_REL_TOL)
    return l2, mx


class Guarded:
    """An fp32 device array with NaN-free canary bands before and after it (stands in for a
    memory checker: any write outside the array is detected)."""

    def __init__(self, torch, shape, fill=None):
        n = int(np.prod(shape))
        self.buf = torch.full((n + 2 * GUARD,), -12345.5, dtype=torch.float32, device="cuda")
        self.view = self.buf[GUARD:GUARD + n].view(*shape)
        assert self.view.data_ptr() % 16 == 0
        if fill is not None:
            self.view.fill_(fill)

    def check(self):
        lo = self.buf[:GUARD]
        hi = self.buf[-GUARD:]
        assert bool((lo == -12345.5).all()) and bool((hi == -12345.5).all()), "guard band overwritten"


def to_dev(torch, arrs):
    return [torch.from_numpy(np.ascontiguousarray(a)).cuda() for a in arrs]


def run_fwd(torch, w: W.Workload, with_loss=True, stream=None):
    fields = to_dev(torch, w.fields)
    sources = to_dev(torch, w.sources)
    ne = len(W.OP_META[w.op]["residuals"])
    res = [Guarded(torch, w.shape, fill=7.0) for _ in range(ne)]
    loss = torch.full((ne + 1,), -1.0, dtype=torch.float64, device="cuda") if with_loss else None
    ws = torch.empty(B.workspace_bytes(w.op, w.shape), dtype=torch.uint8, device="cuda")
    B.fpde_fwd(w.op, fields, sources, [r.view for r in res], loss, w.shape, w.spacing, w.coeffs, w.bc, ws, stream)
    torch.cuda.synchronize()
    for r in res:
        r.check()
    return fields, sources, res, loss


def run_bwd(torch, w: W.Workload, fields, gres, gscale, stream=None):
    nf = len(w.fields)
    grads = [Guarded(torch, w.shape, fill=9.0) for _ in range(nf)]
    B.fpde_bwd(w.op, fields, gres, gscale, [g.view for g in grads], w.shape, w.spacing, w.coeffs, w.bc, None, stream)
    torch.cuda.synchronize()
    for g in grads:
        g.check()
    return grads
