"""Host-side checks that need no GPU: the shared library builds, loads, exports every symbol the
public header declares, and rejects bad arguments with the documented status codes."""
import ctypes
import os
import re

import pytest

from paper_2607_18020_b200 import binding as B
from paper_2607_18020_b200 import build as fbuild
from paper_2607_18020_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    fbuild.build()


def _declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            txt = open(os.path.join(ROOT, "include", fn)).read()
            txt = re.sub(r"/\*.*?\*/", "", txt, flags=re.S)
            names |= set(re.findall(r"\b(fpde_[a-z0-9_]+)\s*\(", txt))
    return names


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(B.LIB_PATH)
    names = _declared_symbols()
    assert {"fpde_fwd", "fpde_bwd", "fpde_op_info", "fpde_strerror", "fpde_workspace_bytes", "fpde_row_count"} <= names
    for n in names:
        assert hasattr(lib, n), n


def test_registry():
    expect = {W.BURGERS_1D_T: (2, 1, 0, 1, 1, 1), W.POISSON_2D: (2, 1, 1, 1, 0, 1), W.GRAYSCOTT_2D: (2, 2, 0, 2, 4, 1),
              W.HELMHOLTZ_3D_O4: (3, 1, 1, 1, 1, 2), W.NS_3D_T: (4, 4, 0, 4, 1, 1),
              W.NS_2D_STEADY: (2, 3, 0, 3, 1, 1), W.NS_3D_STEADY: (3, 4, 0, 4, 1, 1),
              W.NS_3D_T_XSLAB: (4, 4, 0, 4, 1, 1), W.GRAYSCOTT_2D_XSLAB: (2, 2, 0, 2, 4, 1)}
    for op, e in expect.items():
        i = B.op_info(op)
        assert (i.ndim, i.nfields, i.nsources, i.nresiduals, i.ncoeffs, i.radius) == e
        cfg = next(c for c in W.CONFIGS.values() if c["op"] == op)
        assert [B.BC_IDS[b] for b in cfg["bc"]] == list(i.bc)[:i.ndim]
        assert len(W.OP_META[op]["fields"]) == i.nfields and len(W.DEFAULT_COEFFS[op]) == i.ncoeffs
    with pytest.raises(B.FpdeError):
        B.op_info(99)
    assert "unknown" in B.strerror(1234)


def test_row_counts_and_workspace():
    assert B.row_count(W.BURGERS_1D_T, (256, 128)) == 256 * 128
    assert B.row_count(W.POISSON_2D, (1024, 1024)) == 1022 * 1022
    assert B.row_count(W.GRAYSCOTT_2D, (4096, 4096)) == 4096 * 4096
    assert B.row_count(W.HELMHOLTZ_3D_O4, (256, 256, 256)) == 252 ** 3
    assert B.row_count(W.NS_3D_T, (128, 128, 128, 16)) == 128 ** 3 * 14
    assert B.row_count(W.POISSON_2D, (1024, 1023)) == 0          # x4 rule
    assert B.row_count(W.NS_2D_STEADY, (128, 128)) == 126 * 126
    assert B.row_count(W.NS_3D_STEADY, (64, 32, 16)) == 62 * 30 * 14
    assert B.row_count(W.NS_3D_T_XSLAB, (34, 8, 8, 16)) == 32 * 8 * 8 * 14
    assert B.row_count(W.GRAYSCOTT_2D_XSLAB, (18, 32)) == 16 * 32
    for name in W.CONFIG_ORDER + W.EXTRA_CONFIGS + W.SLAB_CONFIGS:
        c = W.CONFIGS[name]
        assert 0 < B.workspace_bytes(c["op"], c["shape"]) < (64 << 20)
    assert B.workspace_bytes(W.NS_3D_T, (2, 8, 8, 8)) == 0


def test_argument_validation_without_a_gpu():
    """Every check that precedes a launch; pointers are fake (never dereferenced on the host)."""
    P = 0x1000
    ok = dict(op=W.POISSON_2D, fields=[P], sources=[P], residuals=[P], loss_out=None, shape=(16, 16),
              spacing=(0.1, 0.1), coeffs=(), bc=(W.INTERIOR, W.INTERIOR), workspace=None, workspace_bytes_=0,
              stream=None)
    def call(**kw):
        a = dict(ok); a.update(kw)
        return B.fwd_status(**a)
    assert call(op=17) == 1
    assert call(fields=None) == 2
    assert call(fields=[None]) == 2
    assert call(sources=None) == 2
    assert call(residuals=[None]) == 2
    assert call(ndim=3) == 3
    assert call(shape=(2, 16)) == 4
    assert call(shape=(16, 18)) == 4
    assert call(shape=(1 << 16, 1 << 16)) == 4
    assert call(fields=[P + 4]) == 5
    assert call(spacing=(0.1, 0.0)) == 6
    assert call(spacing=(float("nan"), 0.1)) == 6
    assert call(coeffs=(1.0,)) == 7
    assert call(bc=(W.PERIODIC, W.INTERIOR)) == 8
    assert call(loss_out=P, workspace=None) == 9
    assert call(loss_out=P, workspace=P, workspace_bytes_=2) == 9
    assert call(op=W.HELMHOLTZ_3D_O4, shape=(4, 8, 8), spacing=(.1, .1, .1), coeffs=(1.0,), bc=(W.INTERIOR,) * 3) == 4
    assert call(op=W.BURGERS_1D_T, shape=(3, 8), coeffs=(0.1,), bc=(W.ONE_SIDED,) * 2, sources=None) == 4
    okb = dict(op=W.GRAYSCOTT_2D, fields=[P, P], gres=[P, P], gscale=None, gfields=[P, P], shape=(8, 8),
               spacing=(0.1, 0.1), coeffs=(1, 1, 1, 1), bc=(W.PERIODIC, W.PERIODIC), workspace=None,
               workspace_bytes_=0, stream=None)
    def callb(**kw):
        a = dict(okb); a.update(kw)
        return B.bwd_status(**a)
    assert callb(gres=None) == 2
    assert callb(gfields=[P, None]) == 2
    assert callb(gres=[P, P + 8]) == 5
    assert callb(gscale=(1.0, float("inf"))) == 6
    assert callb(coeffs=(1, 1, 1)) == 7
    assert callb(bc=(W.PERIODIC, W.ONE_SIDED)) == 8


def test_fwd_bwd_and_f64_validation_without_a_gpu():
    """The loss-specialised pass and the fp64 path check their arguments before any launch."""
    P = 0x1000
    ok = dict(op=W.GRAYSCOTT_2D, fields=[P, P], sources=None, residuals=None, gfields=[P, P], loss_out=None,
              shape=(8, 8), spacing=(0.1, 0.1), coeffs=(1, 1, 1, 1), bc=(W.PERIODIC, W.PERIODIC), workspace=None,
              workspace_bytes_=0, stream=None)
    def call(**kw):
        a = dict(ok); a.update(kw)
        return B.fwd_bwd_status(**a)
    assert B.has_single_pass(W.GRAYSCOTT_2D) and B.has_single_pass(W.POISSON_2D) and B.has_single_pass(W.NS_2D_STEADY)
    assert not B.has_single_pass(W.NS_3D_T) and not B.has_single_pass(W.HELMHOLTZ_3D_O4)
    assert call(op=23) == 1
    assert call(gfields=None) == 2
    assert call(gfields=[P, None]) == 2
    assert call(residuals=[P + 4, None]) == 5            # an optional residual array, if given, must be aligned
    assert call(gfields=[P, P + 8]) == 5
    assert call(shape=(8, 10)) == 4
    assert call(coeffs=(1, 1, 1)) == 7
    assert call(loss_out=P) == 9                          # loss wanted, no workspace
    assert call(loss_out=P, workspace=P, workspace_bytes_=4) == 9
    # operators without a single-pass kernel need every residual array
    assert call(op=W.HELMHOLTZ_3D_O4, fields=[P], sources=[P], gfields=[P], shape=(8, 8, 8), spacing=(.1, .1, .1),
                coeffs=(1.0,), bc=(W.INTERIOR,) * 3) == 2
    assert call(op=W.HELMHOLTZ_3D_O4, fields=[P], sources=[P], residuals=[None], gfields=[P], shape=(8, 8, 8),
                spacing=(.1, .1, .1), coeffs=(1.0,), bc=(W.INTERIOR,) * 3) == 2
    # workspace sizes are host-only queries and do not depend on a device being present
    assert 0 < B.fwd_bwd_workspace_bytes(W.GRAYSCOTT_2D, (4096, 4096)) < (1 << 20)
    assert B.fwd_bwd_workspace_bytes(W.NS_3D_T, (128, 128, 128, 16)) == B.workspace_bytes(W.NS_3D_T, (128, 128, 128, 16))
    assert 0 < B.workspace_bytes_f64(W.HELMHOLTZ_3D_O4, (64, 64, 64)) < (1 << 20)
    L = B.lib()
    import ctypes
    vpp = ctypes.POINTER(ctypes.c_void_p)
    one = (ctypes.c_void_p * 1)(P)
    sh = (ctypes.c_int64 * 2)(16, 16); h = (ctypes.c_double * 2)(0.1, 0.1); bc = (ctypes.c_int * 2)(1, 1)
    st = L.fpde_fwd_f64(1, ctypes.cast(one, vpp), ctypes.cast(one, vpp), None, None, 2, sh, h, None, 0, bc, None, 0, None)
    assert st == 2                                        # residuals missing
    st = L.fpde_bwd_f64(1, ctypes.cast(one, vpp), None, None, ctypes.cast(one, vpp), 2, sh, h, None, 0, bc, None)
    assert st == 2
    st = L.fpde_bwd_f64(1, ctypes.cast(one, vpp), ctypes.cast(one, vpp), None, ctypes.cast(one, vpp), 3, sh, h, None, 0, bc, None)
    assert st == 3


def test_host_pipeline_plan_covers_every_plane_once_ahead_of_its_chunk(monkeypatch):
    """The plan of the pipelined host path: chunks tile [0, n0) in whole 4-plane work items, the
    upload transfers tile [0, n0-1) (plane n0-1 goes first, on its own), and transfer c ends one
    plane past chunk c, which is what lets the forward launch of chunk c wait for transfer c alone."""
    monkeypatch.delenv("FPDE_HOST_PIPELINE", raising=False)
    monkeypatch.delenv("FPDE_HOST_PIPE_PLANES", raising=False)
    assert B.host_pipeline_plan(28) == [] and B.host_pipeline_plan(1) == [] and B.host_pipeline_plan(0) == []
    for n0 in (29, 30, 32, 33, 48, 53, 64, 127, 128, 129, 1000):
        plan = B.host_pipeline_plan(n0)
        K = len(plan)
        assert K >= 6, n0
        starts = [p[0] for p in plan] + [n0]
        assert starts[0] == 0 and all(a < b for a, b in zip(starts, starts[1:])), (n0, starts)
        assert all(s % 4 == 0 for s in starts[:-1])
        sizes = [b - a for a, b in zip(starts, starts[1:])]
        assert max(sizes) <= 8 and sizes[0] == sizes[1] == 4 and sizes[-2] <= 4 and sizes[-1] <= 4, (n0, sizes)
        covered = []
        for c, (first, lo, hi) in enumerate(plan):
            assert 0 <= lo <= hi <= n0
            covered += list(range(lo, hi))
            end = starts[c + 1]
            if c < K - 1:
                assert hi == end + 1, (n0, c)            # one plane ahead of the chunk
            # everything chunk c reads (its planes and one either side, periodic) is up by then
            need = set(range(first, end)) | {(first - 1) % n0, end % n0}
            assert need <= set(covered) | {n0 - 1}, (n0, c, sorted(need - set(covered)))
        assert sorted(set(covered) | {n0 - 1}) == list(range(n0)), n0
        assert len([p for p in covered if p != n0 - 1]) == len(set(covered) - {n0 - 1})   # nothing twice but the wrap plane
    L = B.lib()
    small = (ctypes.c_int * 6)()
    assert L.fpde_host_pipeline_plan(128, small, 2) == -len(B.host_pipeline_plan(128))
    monkeypatch.setenv("FPDE_HOST_PIPELINE", "0")
    assert B.host_pipeline_plan(128) == []


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "nope.so"))
    monkeypatch.setattr(B, "_lib", None)
    with pytest.raises(RuntimeError, match="no fallback"):
        B.lib()


def test_ns_tma_geometry_predicate_requires_aligned_slots_and_a_ring_that_fits():
    """The shared-memory-staged NS kernels copy each array's tile to `slot`-sized regions of a stage;
    the copy engine needs every region on a 128-byte boundary.  slot = (128 + 2 n_t)(rows + 2)
    floats, so the rule is checked here from that formula, independently of the library."""
    limit = 227 * 1024
    for ty in (4, 8):
        for nt in (4, 8, 16, 32, 64):
            for na in (4, 7):
                shape = (16, 32, 64, nt)
                slot_bytes = (128 + 2 * nt) * (ty + 2) * 4
                ring = 4 * na * slot_bytes + 128
                lanes_ok = (ty * nt) % 32 == 0 and 32 % (nt // 4) == 0
                want = lanes_ok and slot_bytes % 128 == 0 and (na * slot_bytes) % 128 == 0 and ring <= limit
                got = B.diag_ns_tma_geometry(shape, ty, na, limit)
                assert got == want, (ty, nt, na, slot_bytes, ring)
    # the case that used to pass the gate with 64-byte-aligned slots
    assert not B.diag_ns_tma_geometry((16, 32, 64, 4), 8, 4, limit)
    # the adjoint ring of the widest t extent does not fit, the forward ring does
    assert B.diag_ns_tma_geometry((16, 32, 64, 64), 8, 4, limit)
    assert not B.diag_ns_tma_geometry((16, 32, 64, 64), 8, 7, limit)
    # rows that do not tile, t extent beyond the one-box limit
    assert not B.diag_ns_tma_geometry((16, 30, 64, 16), 4, 4, limit)
    assert not B.diag_ns_tma_geometry((16, 32, 64, 128), 4, 4, limit)


def test_fwd_rows_rejects_a_row_count_below_one():
    """fpde_fwd_rows divides the loss by a row count the caller names; 0 or a negative count is refused
    before anything else is looked at."""
    st = B.fwd_status(W.POISSON_2D, [16], [16], [16], None, (8, 8), (0.1, 0.1), (), (W.INTERIOR, W.INTERIOR), None, 0,
                      None, loss_rows=0)
    assert st == 4
