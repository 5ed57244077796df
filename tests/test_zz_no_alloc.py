"""fpde_fwd_noalloc: the forward pass for callers that have no way to allocate a workspace (a
plug-in that receives tensors but no allocator, a region where cudaMalloc must not be called).
Its scratch is a fixed array inside the library, so the checks are: same residuals and loss as
fpde_fwd (which uses a caller workspace), on two calls in a row that share that array, and a
clear refusal of grids that need more scratch than the array holds."""
import numpy as np
import pytest

from paper_2607_18020_b200 import binding as B
from paper_2607_18020_b200 import workloads as W

from gpu_util import LOSS_TOL, assert_close

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _both(w):
    fields = [torch.from_numpy(f).cuda() for f in w.fields]
    sources = [torch.from_numpy(s).cuda() for s in w.sources]
    ne = len(W.OP_META[w.op]["residuals"])
    ref = [torch.empty(w.shape, dtype=torch.float32, device="cuda") for _ in range(ne)]
    got = [torch.full(w.shape, 5.0, dtype=torch.float32, device="cuda") for _ in range(ne)]
    loss_ref = torch.zeros(ne + 1, dtype=torch.float64, device="cuda")
    loss_got = torch.full((ne + 1,), -1.0, dtype=torch.float64, device="cuda")
    ws = torch.empty(B.workspace_bytes(w.op, w.shape), dtype=torch.uint8, device="cuda")
    B.fpde_fwd(w.op, fields, sources, ref, loss_ref, w.shape, w.spacing, w.coeffs, w.bc, ws)
    B.fpde_fwd_noalloc(w.op, fields, sources, got, loss_got, w.shape, w.spacing, w.coeffs, w.bc)
    torch.cuda.synchronize()
    return ref, got, loss_ref.cpu().numpy(), loss_got.cpu().numpy()


def test_noalloc_matches_workspace_entry_point_twice_in_a_row():
    # two different operators / grids back to back: the second call finds the first one's partial
    # sums in the shared array and must not be affected by them
    for name, shape, seed in (("ns_tgv_128x16", (24, 20, 16, 16), 42), ("grayscott_4096", (96, 128), 43),
                              ("ns_tgv_128x16", (24, 20, 16, 16), 44)):
        w = W.make(name, seed=seed, shape=shape)
        assert B.workspace_bytes(w.op, w.shape) <= B.NOALLOC_SCRATCH_BYTES
        ref, got, lr, lg = _both(w)
        for e, (a, b) in enumerate(zip(got, ref)):
            assert_close(a.cpu().numpy(), b.cpu().numpy().astype(np.float64), "%s residual %d" % (name, e))
            # same kernels, same slots of partial sums, only the scratch differs: every bit agrees
            assert torch.equal(a, b), "%s residual %d differs from fpde_fwd" % (name, e)
        assert np.all(np.abs(lg - lr) <= LOSS_TOL * np.abs(lr)), (lg, lr)
        assert np.array_equal(lg, lr), (lg, lr)


def test_noalloc_against_the_oracle_and_without_a_loss():
    import oracle
    w = W.make("ns_tgv_128x16", seed=45, shape=(12, 8, 8, 8))
    _, got, _, lg = _both(w)
    res, loss, _ = oracle.fwd(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    for e, a in enumerate(got):
        assert_close(a.cpu().numpy(), res[e], "residual %d vs oracle" % e)
    assert np.all(np.abs(lg - loss) <= LOSS_TOL * np.abs(loss)), (lg, loss)
    # no loss asked for: no scratch is touched, the residuals are the same
    fields = [torch.from_numpy(f).cuda() for f in w.fields]
    again = [torch.full(w.shape, 5.0, dtype=torch.float32, device="cuda") for _ in got]
    B.fpde_fwd_noalloc(w.op, fields, [], again, None, w.shape, w.spacing, w.coeffs, w.bc)
    torch.cuda.synchronize()
    for a, b in zip(again, got):
        assert torch.equal(a, b)


def test_noalloc_refuses_grids_beyond_its_scratch():
    shape = (512, 512, 64, 16)                 # needs more partial sums than the fixed array holds
    assert B.workspace_bytes(W.NS_3D_T, shape) > B.NOALLOC_SCRATCH_BYTES
    p = torch.empty(16, dtype=torch.float32, device="cuda")     # never dereferenced: the call is refused first
    loss = torch.full((5,), -1.0, dtype=torch.float64, device="cuda")
    st = B.fwd_noalloc_status(W.NS_3D_T, [p] * 4, [], [p] * 4, loss, shape, (0.1,) * 4, (0.01,),
                              (W.PERIODIC,) * 3 + (W.INTERIOR,), None)
    assert st == 9
    torch.cuda.synchronize()
    assert bool((loss == -1.0).all())
