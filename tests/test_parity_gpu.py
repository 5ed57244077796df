"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle on the same
seeded fp32 inputs.  Tolerances: relative L2 <= 1e-5 and infinity-norm-relative <= 1e-4 per
output array, |dL|/L <= 1e-5; zero-pattern (nodes without a row) exact."""
import numpy as np
import pytest

import oracle
from paper_2607_18020_b200 import binding as B
from paper_2607_18020_b200 import workloads as W

from gpu_util import LOSS_TOL, assert_close, run_bwd, run_fwd, to_dev

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")

# (config name, shape or None for the full configuration)
MEDIUM = [
    ("burgers_256x128", None),
    ("burgers_256x128", (37, 23)),
    ("poisson_1024", None),
    ("poisson_1024", (203, 300)),          # several row chunks and column blocks, ragged tails
    ("grayscott_4096", (1000, 1032)),
    ("helmholtz_256", (70, 45, 136)),
    ("helmholtz_256", (45, 128, 128)),      # the builds with the y and z extents fixed at compile time:
    ("helmholtz_256", (13, 256, 256)),      # interior and band blocks, several plane items in the adjoint
    ("helmholtz_256", (9, 512, 512)),
    ("ns_tgv_128x16", (36, 21, 20, 16)),
    ("ns2d_steady_4096", (128, 128)),
    ("ns2d_steady_4096", (203, 300)),
    ("ns3d_steady_256", (37, 22, 136)),     # ragged plane chunks, y blocks and a partial warp
    ("ns3d_steady_256", (20, 9, 260)),      # warp edges inside a z line, a ragged column block
    ("ns_tgv_xslab_34", (34, 21, 20, 16)),  # slab form: first / last x-plane without rows, three plane chunks
    ("ns_tgv_xslab_34", (17, 8, 8, 12)),    # t groups that straddle warps
    ("grayscott_xslab_1026", (203, 300)),   # slab form: first / last row without residual rows, periodic columns
]
TINY = [
    ("burgers_256x128", (4, 4)),
    ("burgers_256x128", (5, 9)),
    ("poisson_1024", (3, 4)),
    ("poisson_1024", (36, 40)),
    ("grayscott_4096", (3, 4)),
    ("grayscott_4096", (17, 12)),
    ("helmholtz_256", (5, 5, 8)),
    ("helmholtz_256", (12, 20, 24)),
    ("ns_tgv_128x16", (3, 3, 3, 4)),
    ("ns_tgv_128x16", (8, 12, 16, 8)),
    ("ns_tgv_128x16", (5, 6, 7, 12)),
    ("ns2d_steady_4096", (3, 4)),
    ("ns2d_steady_4096", (36, 40)),
    ("ns3d_steady_256", (3, 3, 4)),
    ("ns3d_steady_256", (5, 6, 8)),
    ("ns3d_steady_256", (7, 5, 132)),
    ("ns_tgv_xslab_34", (3, 3, 3, 4)),
    ("ns_tgv_xslab_34", (5, 6, 7, 12)),
    ("grayscott_xslab_1026", (3, 4)),
    ("grayscott_xslab_1026", (17, 12)),
]
FULL = [
    ("grayscott_4096", None),
    ("helmholtz_256", None),
    ("ns_tgv_128x16", None),
    ("ns2d_steady_4096", None),
    ("ns3d_steady_256", None),
]


def _row_mask(w):
    """True at the nodes that carry a residual row: on an interior axis the outer `radius` layers
    carry none (geometry only; independent of the data)."""
    radius = B.op_info(w.op).radius
    mask = np.ones(w.shape, dtype=bool)
    for a, (n, b) in enumerate(zip(w.shape, w.bc)):
        if b == W.INTERIOR:
            idx = np.arange(n)
            keep = (idx >= radius) & (idx < n - radius)
            shp = [1] * len(w.shape); shp[a] = n
            mask &= keep.reshape(shp)
    return mask


def _check_case(w, tag):
    R_ref, loss_ref, g_ref, rows = oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    assert rows == B.row_count(w.op, w.shape)
    fields, sources, res, loss = run_fwd(torch, w)
    for e, (r, rr) in enumerate(zip(res, R_ref)):
        got = r.view.cpu().numpy()
        assert_close(got, rr, "%s residual %d" % (tag, e))
        assert np.all(got[~_row_mask(w)] == 0.0), "%s: nodes without a row must hold exactly 0" % tag
        assert np.all(rr[~_row_mask(w)] == 0.0)
    L = loss.cpu().numpy()
    assert np.all(np.abs(L - loss_ref) <= LOSS_TOL * np.abs(loss_ref) + 1e-300), (tag, L, loss_ref)
    # gradient of the fused loss: upstream = the residual arrays the forward wrote, scale 2/N_r
    grads = run_bwd(torch, w, fields, [r.view for r in res], [2.0 / rows] * len(res))
    for f, (g, gr) in enumerate(zip(grads, g_ref)):
        assert_close(g.view.cpu().numpy(), gr, "%s gradient %d" % (tag, f))


@pytest.mark.parametrize("name,shape", MEDIUM)
def test_config_fields(name, shape):
    _check_case(W.make(name, seed=42, shape=shape), "%s%s" % (name, shape or ""))


WIDE_ADDRESS_SWITCHES = ("FPDE_LAP2D_OFF32", "FPDE_FUSED2D_OFF32", "FPDE_STAR3D_OFF32", "FPDE_NS2D_OFF32",
                         "FPDE_NS3D_OFF32", "FPDE_NS_OFF32")


@pytest.mark.parametrize("name,shape", [c for c in MEDIUM if c[1] is not None])
def test_builds_with_64_bit_addressing(name, shape, monkeypatch):
    """Arrays above 2^30 floats run kernel builds with 64-bit offsets; the switches select those
    builds on grids small enough for the oracle (the 3-D+T, steady NS and single-pass kernels have
    no other test at such sizes)."""
    for k in WIDE_ADDRESS_SWITCHES:
        monkeypatch.setenv(k, "0")
    w = W.make(name, seed=48, shape=shape, kind="randn")
    _check_case(w, "%s%s 64-bit offsets" % (name, shape))
    if B.has_single_pass(w.op):
        _, _, g_ref, _ = oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
        grads = [torch.empty(w.shape, dtype=torch.float32, device="cuda") for _ in w.fields]
        ws = torch.empty(B.fwd_bwd_workspace_bytes(w.op, w.shape), dtype=torch.uint8, device="cuda")
        B.fpde_fwd_bwd(w.op, to_dev(torch, w.fields), to_dev(torch, w.sources), None, grads, None, w.shape,
                       w.spacing, w.coeffs, w.bc, ws)
        torch.cuda.synchronize()
        for f, (g, gr) in enumerate(zip(grads, g_ref)):
            assert_close(g.cpu().numpy(), gr, "%s%s single pass, 64-bit offsets, gradient %d" % (name, shape, f))


@pytest.mark.parametrize("name,shape", TINY)
@pytest.mark.parametrize("seed", [42, 43, 44, 45, 46])
def test_randn_fields_tiny(name, shape, seed):
    _check_case(W.make(name, seed=seed, shape=shape, kind="randn"), "%s%s randn seed %d" % (name, shape, seed))


@pytest.mark.parametrize("name,shape", MEDIUM[1:])
def test_adjoint_alone_random_upstream(name, shape):
    """The adjoint on arbitrary upstream arrays (not a residual): non-zero entries at nodes
    without a row must be ignored, and gscale applied."""
    w = W.make(name, seed=44, shape=shape, kind="randn")
    G = W.random_sensitivities(w, seed=7)
    gscale = [0.5 + 0.25 * e for e in range(len(G))]
    ref = oracle.bwd(w.op, w.fields, [s * g.astype(np.float64) for s, g in zip(gscale, G)], w.shape, w.spacing, w.coeffs)
    fields = to_dev(torch, w.fields)
    grads = run_bwd(torch, w, fields, to_dev(torch, G), gscale)
    for f, (g, gr) in enumerate(zip(grads, ref)):
        assert_close(g.view.cpu().numpy(), gr, "%s adjoint %d" % (name, f))


def test_unequal_spacing():
    for name, shape, h in [("poisson_1024", (20, 24), (0.3, 0.07)), ("helmholtz_256", (9, 10, 12), (0.2, 0.15, 0.11)),
                           ("ns_tgv_128x16", (5, 6, 7, 8), (0.3, 0.2, 0.25, 0.1)), ("grayscott_4096", (9, 8), (0.01, 0.02)),
                           ("burgers_256x128", (11, 7), (0.05, 0.02)), ("ns2d_steady_4096", (9, 12), (0.3, 0.2)),
                           ("ns3d_steady_256", (6, 7, 8), (0.3, 0.2, 0.25))]:
        _check_case(W.make(name, seed=45, shape=shape, kind="randn", spacing=h), name + " unequal spacing")


@pytest.mark.parametrize("name,shape", FULL)
def test_full_size_configs(name, shape):
    """The configurations' full sizes in the launch configuration the bench times; the C oracle is fast
    enough to check every element."""
    _check_case(W.make(name, seed=42), name + " full size")


def test_loss_is_bitwise_reproducible():
    w = W.make("ns_tgv_128x16", seed=42, shape=(32, 32, 32, 16))
    fields = to_dev(torch, w.fields)
    res = [torch.empty(w.shape, dtype=torch.float32, device="cuda") for _ in range(4)]
    ws = torch.empty(B.workspace_bytes(w.op, w.shape), dtype=torch.uint8, device="cuda")
    seen = set()
    for _ in range(20):
        loss = torch.zeros(5, dtype=torch.float64, device="cuda")
        B.fpde_fwd(w.op, fields, [], res, loss, w.shape, w.spacing, w.coeffs, w.bc, ws)
        torch.cuda.synchronize()
        seen.add(loss.cpu().numpy().tobytes())
    assert len(seen) == 1


def test_loss_can_be_skipped_and_stream_is_honoured():
    w = W.make("grayscott_4096", seed=42, shape=(64, 64))
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        fields, sources, res, loss = run_fwd(torch, w, with_loss=False, stream=s)
    R_ref, _, _ = oracle.fwd(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    assert loss is None
    for r, rr in zip(res, R_ref):
        assert_close(r.view.cpu().numpy(), rr, "no-loss forward")


def test_invalid_arguments_launch_nothing():
    w = W.make("poisson_1024", seed=42, shape=(16, 16))
    fields = to_dev(torch, w.fields); sources = to_dev(torch, w.sources)
    out = torch.full(w.shape, 3.0, dtype=torch.float32, device="cuda")
    loss = torch.full((2,), -1.0, dtype=torch.float64, device="cuda")
    ws = torch.empty(B.workspace_bytes(w.op, w.shape), dtype=torch.uint8, device="cuda")
    st = B.fwd_status(w.op, fields, sources, [out], loss, w.shape, w.spacing, w.coeffs, w.bc, ws, 2, None)
    assert st == 9      # workspace too small
    st = B.fwd_status(w.op, fields, sources, [out.view(-1)[1:].data_ptr()], None, w.shape, w.spacing, w.coeffs, w.bc, None, 0, None)
    assert st == 5      # misaligned
    torch.cuda.synchronize()
    assert bool((out == 3.0).all()) and bool((loss == -1.0).all())


def test_loss_grad_from_host_buffers():
    """The host-buffer entry point (copies + forward + adjoint in one call) against the oracle."""
    w = W.make("ns_tgv_128x16", seed=43, shape=(12, 10, 8, 8))
    _, loss_ref, g_ref, rows = oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    hf = [torch.from_numpy(f).pin_memory() for f in w.fields]
    hg = [torch.empty(w.shape, dtype=torch.float32).pin_memory() for _ in w.fields]
    hl = torch.zeros(5, dtype=torch.float64).pin_memory()
    arena = torch.empty(B.host_arena_bytes(w.op, w.shape), dtype=torch.uint8, device="cuda")
    assert arena.data_ptr() % 256 == 0
    B.fpde_loss_grad_host(w.op, hf, [], hg, hl, w.shape, w.spacing, w.coeffs, w.bc, arena)
    torch.cuda.synchronize()
    assert np.all(np.abs(hl.numpy() - loss_ref) <= LOSS_TOL * np.abs(loss_ref))
    for f, (g, gr) in enumerate(zip(hg, g_ref)):
        assert_close(g.numpy(), gr, "host entry gradient %d" % f)
    st = B.loss_grad_host_status(w.op, hf, [], hg, hl, w.shape, w.spacing, w.coeffs, w.bc, arena, 1024, None)
    assert st == 9


@pytest.mark.parametrize("shape", [(48, 10, 8, 8), (53, 6, 8, 16), (128, 4, 8, 8), (29, 6, 8, 8), (33, 4, 8, 8)])
def test_pipelined_host_entry_for_navier_stokes(shape, monkeypatch):
    """Grids of 29 or more x-planes (six or more chunks) take the pipelined form of the host-buffer
    entry (transfers of x-planes go up, through forward and adjoint launches over item ranges, and
    down again on three streams; 29 planes is the smallest such grid, with 33 the last chunk is a
    single plane and the last transfer empty).  It must match the oracle, give bit-identical gradients to the plain
    form (the same arithmetic per node), leave the copy streams covered by the caller's stream,
    and be repeatable back to back."""
    w = W.make("ns_tgv_128x16", seed=47, shape=shape, kind="randn")
    _, loss_ref, g_ref, rows = oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    hf = [torch.from_numpy(f).pin_memory() for f in w.fields]
    arena = torch.empty(B.host_arena_bytes(w.op, w.shape), dtype=torch.uint8, device="cuda")
    outs = {}
    for mode in ("1", "0", "1"):
        monkeypatch.setenv("FPDE_HOST_PIPELINE", mode)
        hg = [torch.full(w.shape, 7.0, dtype=torch.float32).pin_memory() for _ in w.fields]
        hl = torch.zeros(5, dtype=torch.float64).pin_memory()
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            B.fpde_loss_grad_host(w.op, hf, [], hg, hl, w.shape, w.spacing, w.coeffs, w.bc, arena)
            B.fpde_loss_grad_host(w.op, hf, [], hg, hl, w.shape, w.spacing, w.coeffs, w.bc, arena)   # back to back
        s.synchronize()                                   # only the caller's stream is synchronised
        assert np.all(np.abs(hl.numpy() - loss_ref) <= LOSS_TOL * np.abs(loss_ref)), (mode, hl, loss_ref)
        for f, (g, gr) in enumerate(zip(hg, g_ref)):
            assert_close(g.numpy(), gr, "host entry (pipeline=%s) gradient %d" % (mode, f))
        outs.setdefault(mode, [g.numpy().copy() for g in hg])
    for a, b in zip(outs["1"], outs["0"]):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("shape", [(48, 10, 8, 8), (33, 4, 8, 8)])
def test_pipelined_host_entry_with_arrays_that_are_slices_of_one_buffer(shape, monkeypatch):
    """When the host arrays of a kind are slices of ONE pinned buffer (evenly spaced, one allocation) the
    pipelined host entry moves a range of planes of all of them in one strided copy; the results are bit
    for bit those of separate buffers (which take one copy per array), and of FPDE_HOST_STRIDED=0."""
    w = W.make("ns_tgv_128x16", seed=48, shape=shape, kind="randn")
    arena = torch.empty(B.host_arena_bytes(w.op, w.shape), dtype=torch.uint8, device="cuda")
    outs = []
    for stacked, switch in ((True, "1"), (True, "0"), (False, "1")):
        monkeypatch.setenv("FPDE_HOST_STRIDED", switch)
        if stacked:
            hf_all = torch.stack([torch.from_numpy(f) for f in w.fields]).pin_memory()
            hg_all = torch.full((len(w.fields),) + tuple(shape), 7.0, dtype=torch.float32).pin_memory()
            hf, hg = list(hf_all.unbind(0)), list(hg_all.unbind(0))
        else:
            hf = [torch.from_numpy(f).pin_memory() for f in w.fields]
            hg = [torch.full(shape, 7.0, dtype=torch.float32).pin_memory() for _ in w.fields]
        hl = torch.zeros(5, dtype=torch.float64).pin_memory()
        B.fpde_loss_grad_host(w.op, hf, [], hg, hl, w.shape, w.spacing, w.coeffs, w.bc, arena)
        torch.cuda.current_stream().synchronize()
        outs.append(([g.numpy().copy() for g in hg], hl.numpy().copy()))
    _, loss_ref, g_ref, _ = oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    for f, g in enumerate(outs[0][0]):
        assert_close(g, g_ref[f], "host entry, stacked buffers, gradient %d" % f)
    for gs, l in outs[1:]:
        for a, b in zip(gs, outs[0][0]):
            assert np.array_equal(a, b)
        assert np.array_equal(l, outs[0][1])


@pytest.mark.parametrize("shape", [(8, 12, 16, 8), (19, 8, 8, 16), (6, 4, 4, 32), (7, 16, 32, 16), (5, 12, 48, 8)])
def test_ns_tma_and_l1_staged_kernels_agree_with_oracle(shape, monkeypatch):
    """FPDE_NS_TMA=1 runs grids that tile exactly on the TMA-staged kernels (one-box tiles away from
    the periodic wrap, five-box tiles on it); the default is the L1-staged kernels.  Both must
    match the oracle, and no bounded barrier wait may have given up."""
    for tma in ("1", "0"):
        monkeypatch.setenv("FPDE_NS_TMA", tma)
        _check_case(W.make("ns_tgv_128x16", seed=46, shape=shape, kind="randn"), "ns %s tma=%s" % (shape, tma))
    assert B.diag_tma_timeouts() == 0


@pytest.mark.parametrize("name,shape", [("ns_tgv_128x16", (16, 16, 16, 8)), ("ns3d_steady_256", (16, 16, 32))])
@pytest.mark.parametrize("cells", [128, 2048])
def test_ns_adjoint_on_smooth_fields_at_fine_spacing(name, shape, cells):
    """Noise-free analytic fields on a spacing of 2 pi / cells: the upstream arrays are smooth, the
    second differences of the adjoint cancel to a part in nu/h^2 (about 1000 at 2048 cells), which is
    where a stencil sum evaluated with merged weights loses the most; the tolerances still hold."""
    w = W.make(name, seed=42, shape=shape)
    h = list(w.spacing)
    for a in range(3):
        h[a] = 2 * np.pi / cells
    idx = np.meshgrid(*[np.arange(n) for n in shape], indexing="ij")
    X, Y, Z = (idx[a] * h[a] + 0.3 * (a + 1) for a in range(3))
    dec = np.exp(-0.1 * idx[3] * h[3]) if len(shape) == 4 else 1.0
    f = [np.sin(X) * np.cos(Y) * np.cos(Z) * dec + 0.5, -np.cos(X) * np.sin(Y) * np.cos(Z) * dec - 0.3,
         0.2 * np.sin(X + Y + Z) * dec + 0.1, 0.25 * (np.cos(2 * X) + np.cos(2 * Y)) * dec]
    w.fields = [np.ascontiguousarray(a.astype(np.float32)) for a in f]
    w.spacing = tuple(h)
    R_ref, loss_ref, g_ref, _ = oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    fields, _, res, loss = run_fwd(torch, w)
    for e, r in enumerate(res):
        assert_close(r.view.cpu().numpy(), R_ref[e], "%s smooth residual %d" % (name, e))
    rows = B.row_count(w.op, w.shape)
    grads = run_bwd(torch, w, fields, [r.view for r in res], [2.0 / rows] * len(res))
    for k, g in enumerate(grads):
        assert_close(g.view.cpu().numpy(), g_ref[k], "%s smooth gradient %d (2 pi / %d)" % (name, k, cells))


@pytest.mark.parametrize("shape", [(20, 40, 136), (9, 45, 260), (37, 72, 256), (12, 130, 392)])
@pytest.mark.parametrize("engine", ["l1", "tma", "tma_fwd"])
def test_helmholtz_engines_agree_with_oracle(shape, engine, monkeypatch):
    """The Helmholtz operator has two engines: plane tiles staged through L1 and registers, and plane
    tiles staged through shared memory by the copy engine (default for the adjoint; the forward pass
    with FPDE_STAR3D_TMA_FWD=1).  Shapes with ragged tiles in y and z, grids of fewer tile-planes than
    CTAs would take and grids where one CTA's share spans two tiles; forward, the adjoint of the
    residuals (through both entry points) and the adjoint of an arbitrary upstream array."""
    monkeypatch.setenv("FPDE_STAR3D_TMA", "0" if engine == "l1" else "1")
    monkeypatch.setenv("FPDE_STAR3D_TMA_FWD", "1" if engine == "tma_fwd" else "0")
    w = W.make("helmholtz_256", seed=47, shape=shape, kind="randn")
    _check_case(w, "helmholtz %s engine %s" % (shape, engine))
    # arbitrary upstream array with entries off the rows, and the one-call entry point
    rng = np.random.default_rng(5)
    G = rng.standard_normal(shape).astype(np.float32)
    Gz = G.astype(np.float64).copy()
    Gz[:2] = 0; Gz[-2:] = 0; Gz[:, :2] = 0; Gz[:, -2:] = 0; Gz[:, :, :2] = 0; Gz[:, :, -2:] = 0
    g_ref = oracle.bwd(w.op, w.fields, [0.37 * Gz], w.shape, w.spacing, w.coeffs)
    fields = to_dev(torch, w.fields)
    grads = run_bwd(torch, w, fields, to_dev(torch, [G]), [0.37])
    assert_close(grads[0].view.cpu().numpy(), g_ref[0], "helmholtz %s engine %s arbitrary upstream" % (shape, engine))
    _, loss_ref, g2_ref, _ = oracle.loss_and_grad(w.op, w.fields, w.sources, w.shape, w.spacing, w.coeffs)
    res = [torch.empty(shape, dtype=torch.float32, device="cuda")]
    gr = [torch.empty(shape, dtype=torch.float32, device="cuda")]
    loss = torch.zeros(2, dtype=torch.float64, device="cuda")
    ws = torch.empty(B.fwd_bwd_workspace_bytes(w.op, shape), dtype=torch.uint8, device="cuda")
    B.fpde_fwd_bwd(w.op, fields, to_dev(torch, w.sources), res, gr, loss, shape, w.spacing, w.coeffs, w.bc, ws)
    torch.cuda.synchronize()
    assert_close(gr[0].cpu().numpy(), g2_ref[0], "helmholtz %s engine %s one call" % (shape, engine))
    assert abs(loss[-1].item() - loss_ref[-1]) <= 1e-5 * abs(loss_ref[-1])
    assert B.diag_tma_timeouts() == 0
