"""Grids close to the 2^31-node limit of the 32-bit element offsets: the kernels' results are
checked on sampled windows (start of the array, middle, far corner) that the oracle evaluates as
small grids of their own.  The operators are local, so a window's interior must agree with the
big grid wherever the window's own edges are out of reach (margin = 2 * radius + 1)."""
import numpy as np
import pytest

import oracle
from paper_2607_18020_b200 import binding as B
from paper_2607_18020_b200 import workloads as W

from gpu_util import assert_close

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

CASES = [
    # op, shape, spacing, coeffs, bc, window extents
    (W.POISSON_2D, (46000, 46000), (1e-3, 2e-3), (), (W.INTERIOR,) * 2, (24, 32)),
    (W.HELMHOLTZ_3D_O4, (1280, 1280, 1280), (1e-2, 2e-2, 1.5e-2), (3.0,), (W.INTERIOR,) * 3, (14, 14, 24)),
    (W.NS_3D_T, (128, 256, 256, 128), (0.05, 0.04, 0.06, 0.1), (0.01,), (W.PERIODIC,) * 3 + (W.INTERIOR,), (9, 9, 9, 16)),
]


def _windows(shape, ext):
    lo = tuple(0 for _ in shape)
    mid = tuple((n - e) // 2 for n, e in zip(shape, ext))
    hi = tuple(n - e for n, e in zip(shape, ext))
    return [lo, mid, hi]


@pytest.mark.parametrize("op,shape,h,c,bc,ext", CASES)
def test_near_max_size_sampled_windows(op, shape, h, c, bc, ext):
    need = int(np.prod(shape)) * 4
    info = B.op_info(op)
    narr = 2 * info.nfields + info.nsources + info.nresiduals
    free, _ = torch.cuda.mem_get_info()
    if free < narr * need + (4 << 30):
        pytest.skip("not enough free device memory for %d arrays of %.1f GB" % (narr, need / 2 ** 30))
    torch.cuda.empty_cache()
    gen = torch.Generator(device="cuda").manual_seed(1234)
    mk = lambda: torch.randn(shape, generator=gen, dtype=torch.float32, device="cuda")
    fields = [mk() for _ in range(info.nfields)]
    sources = [mk() for _ in range(info.nsources)]
    res = [torch.empty(shape, dtype=torch.float32, device="cuda") for _ in range(info.nresiduals)]
    grads = [torch.empty(shape, dtype=torch.float32, device="cuda") for _ in range(info.nfields)]
    loss = torch.zeros(info.nresiduals + 1, dtype=torch.float64, device="cuda")
    ws = torch.empty(B.workspace_bytes(op, shape), dtype=torch.uint8, device="cuda")
    rows = B.row_count(op, shape)
    gs = [2.0 / rows] * info.nresiduals
    B.fpde_fwd(op, fields, sources, res, loss, shape, h, c, bc, ws)
    B.fpde_bwd(op, fields, res, gs, grads, shape, h, c, bc)
    torch.cuda.synchronize()
    grad_sets = [("pair", grads)]
    if B.has_single_pass(op) and torch.cuda.mem_get_info()[0] > info.nfields * need + (2 << 30):
        # the single-pass kernel on the same grid: same loss, gradients checked on the same windows
        grads1 = [torch.empty(shape, dtype=torch.float32, device="cuda") for _ in range(info.nfields)]
        loss1 = torch.zeros(info.nresiduals + 1, dtype=torch.float64, device="cuda")
        ws1 = torch.empty(B.fwd_bwd_workspace_bytes(op, shape), dtype=torch.uint8, device="cuda")
        B.fpde_fwd_bwd(op, fields, sources, None, grads1, loss1, shape, h, c, bc, ws1)
        torch.cuda.synchronize()
        assert torch.all((loss1 - loss).abs() <= 1e-6 * loss.abs())
        grad_sets.append(("single pass", grads1))
    # the reducer against a library reduction of the residuals it was given
    for e, r in enumerate(res):
        ref = float((r.double() ** 2).sum().item()) / rows
        assert abs(loss[e].item() - ref) <= 1e-6 * ref
    m = 2 * info.radius + 1
    for w0 in _windows(shape, ext):
        sl = tuple(slice(a, a + e) for a, e in zip(w0, ext))
        fw = [f[sl].cpu().numpy() for f in fields]
        sw = [s[sl].cpu().numpy() for s in sources]
        gw = [r[sl].cpu().numpy().astype(np.float64) * g for r, g in zip(res, gs)]
        R, _, _ = oracle.fwd(op, fw, sw, ext, h, c)
        G = oracle.bwd(op, fw, gw, ext, h, c)
        inner = tuple(slice(m, e - m) for e in ext)
        # nodes of the window interior that carry a row in the big grid too
        big_row = np.ones(ext, dtype=bool)
        for a, (n, b) in enumerate(zip(shape, bc)):
            if b == W.INTERIOR:
                idx = np.arange(w0[a], w0[a] + ext[a])
                keep = (idx >= info.radius) & (idx < n - info.radius)
                shp = [1] * len(ext); shp[a] = ext[a]
                big_row &= keep.reshape(shp)
        for e, (r, rr) in enumerate(zip(res, R)):
            got = r[sl].cpu().numpy()
            mask = big_row[inner]
            if mask.any():
                assert_close(got[inner][mask], rr[inner][mask], "window %s residual %d" % (w0, e))
            assert np.all(got[~big_row] == 0.0)
        # the gradient only where the window sees every row the node touches: its own interior,
        # and away from the big grid's band (there the window's rows and the grid's rows differ)
        band_free = np.ones(ext, dtype=bool)
        for a, (n, b) in enumerate(zip(shape, bc)):
            if b == W.INTERIOR:
                idx = np.arange(w0[a], w0[a] + ext[a])
                keep = (idx >= 2 * info.radius) & (idx < n - 2 * info.radius)
                shp = [1] * len(ext); shp[a] = ext[a]
                band_free &= keep.reshape(shp)
        for tag, gset in grad_sets:
            for f, (g, gg) in enumerate(zip(gset, G)):
                got = g[sl].cpu().numpy()
                mask = band_free[inner]
                if mask.any():
                    assert_close(got[inner][mask], gg[inner][mask], "%s: window %s gradient %d" % (tag, w0, f))
    del fields, sources, res, grads, grad_sets
    torch.cuda.empty_cache()
