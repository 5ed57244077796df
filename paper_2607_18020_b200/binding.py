"""ctypes binding of libfpde.so: same names as the C ABI, argument marshalling only.

Every step of the path (residuals, loss, adjoint, boundary correction) runs in the library's
CUDA kernels; this module turns torch tensors into device pointers and host scalars into C
arrays.  There is no fallback: if the shared library is missing or a call is refused, an
exception is raised.
"""
from __future__ import annotations

import ctypes
import functools
import os
from typing import List, Optional, Sequence

from . import workloads as _w

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfpde.so")

# numeric ids of include/fpde.h
OP_IDS = {_w.BURGERS_1D_T: 0, _w.POISSON_2D: 1, _w.GRAYSCOTT_2D: 2, _w.HELMHOLTZ_3D_O4: 3, _w.NS_3D_T: 4, _w.NS_2D_STEADY: 5,
          _w.NS_3D_STEADY: 6, _w.NS_3D_T_XSLAB: 7, _w.GRAYSCOTT_2D_XSLAB: 8}
BC_IDS = {_w.PERIODIC: 0, _w.INTERIOR: 1, _w.ONE_SIDED: 2}
FPDE_OK = 0


class FpdeError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: status %d (%s)" % (where, status, strerror(status)))


class OpInfo(ctypes.Structure):
    _fields_ = [("ndim", ctypes.c_int), ("nfields", ctypes.c_int), ("nsources", ctypes.c_int),
                ("nresiduals", ctypes.c_int), ("ncoeffs", ctypes.c_int), ("radius", ctypes.c_int),
                ("bc", ctypes.c_int * 4)]


_lib = None


def lib():
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libfpde.so is missing (%s): build it with "
                               "`python -m paper_2607_18020_b200.build`; there is no fallback path" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vpp = ctypes.POINTER(ctypes.c_void_p)
        L.fpde_op_info.restype = ctypes.c_int
        L.fpde_op_info.argtypes = [ctypes.c_int, ctypes.POINTER(OpInfo)]
        L.fpde_strerror.restype = ctypes.c_char_p
        L.fpde_strerror.argtypes = [ctypes.c_int]
        L.fpde_row_count.restype = ctypes.c_int64
        L.fpde_row_count.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_int64)]
        L.fpde_workspace_bytes.restype = ctypes.c_size_t
        L.fpde_workspace_bytes.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_int64)]
        L.fpde_fwd.restype = ctypes.c_int
        L.fpde_fwd.argtypes = [ctypes.c_int, vpp, vpp, vpp, ctypes.c_void_p, ctypes.c_int,
                               ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_double),
                               ctypes.POINTER(ctypes.c_double), ctypes.c_int, ctypes.POINTER(ctypes.c_int),
                               ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
        L.fpde_fwd_rows.restype = ctypes.c_int
        L.fpde_fwd_rows.argtypes = L.fpde_fwd.argtypes + [ctypes.c_int64]
        L.fpde_plane_chunk.restype = ctypes.c_int
        L.fpde_plane_chunk.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_int64)]
        L.fpde_fwd_chunks.restype = ctypes.c_int
        L.fpde_fwd_chunks.argtypes = L.fpde_fwd.argtypes + [ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int]
        L.fpde_bwd.restype = ctypes.c_int
        L.fpde_bwd.argtypes = [ctypes.c_int, vpp, vpp, ctypes.POINTER(ctypes.c_double), vpp, ctypes.c_int,
                               ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_double),
                               ctypes.POINTER(ctypes.c_double), ctypes.c_int, ctypes.POINTER(ctypes.c_int),
                               ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
        L.fpde_bwd_chunks.restype = ctypes.c_int
        L.fpde_bwd_chunks.argtypes = [ctypes.c_int, vpp, vpp, ctypes.POINTER(ctypes.c_double), vpp, ctypes.c_int,
                                      ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_double),
                                      ctypes.POINTER(ctypes.c_double), ctypes.c_int, ctypes.POINTER(ctypes.c_int),
                                      ctypes.c_void_p, ctypes.c_int, ctypes.c_int]
        L.fpde_has_single_pass.restype = ctypes.c_int
        L.fpde_has_single_pass.argtypes = [ctypes.c_int]
        L.fpde_fwd_bwd_workspace_bytes.restype = ctypes.c_size_t
        L.fpde_fwd_bwd_workspace_bytes.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_int64)]
        L.fpde_fwd_bwd.restype = ctypes.c_int
        L.fpde_fwd_bwd.argtypes = [ctypes.c_int, vpp, vpp, vpp, vpp, ctypes.c_void_p, ctypes.c_int,
                                   ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_double),
                                   ctypes.POINTER(ctypes.c_double), ctypes.c_int, ctypes.POINTER(ctypes.c_int),
                                   ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
        L.fpde_workspace_bytes_f64.restype = ctypes.c_size_t
        L.fpde_workspace_bytes_f64.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_int64)]
        L.fpde_fwd_f64.restype = ctypes.c_int
        L.fpde_fwd_f64.argtypes = L.fpde_fwd.argtypes
        L.fpde_bwd_f64.restype = ctypes.c_int
        L.fpde_bwd_f64.argtypes = [ctypes.c_int, vpp, vpp, ctypes.POINTER(ctypes.c_double), vpp, ctypes.c_int,
                                   ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_double),
                                   ctypes.POINTER(ctypes.c_double), ctypes.c_int, ctypes.POINTER(ctypes.c_int),
                                   ctypes.c_void_p]
        L.fpde_host_arena_bytes.restype = ctypes.c_size_t
        L.fpde_host_arena_bytes.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_int64)]
        L.fpde_host_pipeline_plan.restype = ctypes.c_int
        L.fpde_host_pipeline_plan.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_int), ctypes.c_int]
        L.fpde_loss_grad_host.restype = ctypes.c_int
        L.fpde_loss_grad_host.argtypes = [ctypes.c_int, vpp, vpp, vpp, ctypes.c_void_p, ctypes.c_int,
                                          ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_double),
                                          ctypes.POINTER(ctypes.c_double), ctypes.c_int,
                                          ctypes.POINTER(ctypes.c_int), ctypes.c_void_p, ctypes.c_size_t,
                                          ctypes.c_void_p]
        L.fpde_fwd_noalloc.restype = ctypes.c_int
        L.fpde_fwd_noalloc.argtypes = [ctypes.c_int, vpp, vpp, vpp, ctypes.c_void_p, ctypes.c_int,
                                       ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_double),
                                       ctypes.POINTER(ctypes.c_double), ctypes.c_int, ctypes.POINTER(ctypes.c_int),
                                       ctypes.c_void_p]
        L.fpde_diag_tma_timeouts.restype = ctypes.c_uint
        L.fpde_diag_tma_timeouts.argtypes = []
        L.fpde_diag_ns_tma_geometry.restype = ctypes.c_int
        L.fpde_diag_ns_tma_geometry.argtypes = [ctypes.POINTER(ctypes.c_int64), ctypes.c_int, ctypes.c_int,
                                                ctypes.c_size_t]
        _lib = L
    return _lib


def _opid(op) -> int:
    return OP_IDS[op] if isinstance(op, str) else int(op)


def _ptr_array(ptrs: Sequence[Optional[int]]):
    # a ctypes array is accepted where the prototype says POINTER(c_void_p): no cast needed
    return (ctypes.c_void_p * max(1, len(ptrs)))(*ptrs)


def _dev_ptrs(tensors) -> List[int]:
    out = []
    for t in tensors:
        if hasattr(t, "data_ptr"):
            out.append(t.data_ptr())
        else:
            out.append(int(t) if t is not None else None)
    return out


# The small host arrays of a call (shape, spacings, coefficients, boundary kinds) are read-only
# for the library and repeat from call to call: built once per distinct value.
@functools.lru_cache(maxsize=512)
def _i64_of(t: tuple):
    return (ctypes.c_int64 * max(1, len(t)))(*t)


@functools.lru_cache(maxsize=512)
def _f64_of(t: tuple):
    return (ctypes.c_double * max(1, len(t)))(*t)


@functools.lru_cache(maxsize=512)
def _bcs_of(t: tuple):
    return (ctypes.c_int * max(1, len(t)))(*[BC_IDS[b] if isinstance(b, str) else int(b) for b in t])


def _i64(v):
    return _i64_of(tuple(int(x) for x in v))


def _f64(v):
    return _f64_of(tuple(float(x) for x in v))


def _bcs(bc):
    return _bcs_of(tuple(bc))


def strerror(status: int) -> str:
    return lib().fpde_strerror(int(status)).decode()


def op_info(op) -> OpInfo:
    info = OpInfo()
    st = lib().fpde_op_info(_opid(op), ctypes.byref(info))
    if st != FPDE_OK:
        raise FpdeError(st, "fpde_op_info")
    return info


def row_count(op, shape) -> int:
    return int(lib().fpde_row_count(_opid(op), len(shape), _i64(shape)))


def workspace_bytes(op, shape) -> int:
    return int(lib().fpde_workspace_bytes(_opid(op), len(shape), _i64(shape)))


def fwd_status(op, fields, sources, residuals, loss_out, shape, spacing, coeffs, bc, workspace,
               workspace_bytes_, stream, ndim=None, ncoeffs=None, loss_rows=None) -> int:
    """Raw call: returns the status code (used by the error-path tests).  With loss_rows the call
    is fpde_fwd_rows (the loss divides by that row count)."""
    fn = lib().fpde_fwd if loss_rows is None else lib().fpde_fwd_rows
    extra = () if loss_rows is None else (int(loss_rows),)
    return fn(_opid(op),
                          _ptr_array(_dev_ptrs(fields)) if fields is not None else None,
                          _ptr_array(_dev_ptrs(sources)) if sources is not None else None,
                          _ptr_array(_dev_ptrs(residuals)) if residuals is not None else None,
                          _dev_ptrs([loss_out])[0] if loss_out is not None else None,
                          len(shape) if ndim is None else ndim,
                          _i64(shape) if shape is not None else None,
                          _f64(spacing) if spacing is not None else None,
                          _f64(coeffs) if coeffs is not None else None,
                          len(coeffs) if ncoeffs is None else ncoeffs,
                          _bcs(bc) if bc is not None else None,
                          _dev_ptrs([workspace])[0] if workspace is not None else None,
                          int(workspace_bytes_), stream, *extra)


def bwd_status(op, fields, gres, gscale, gfields, shape, spacing, coeffs, bc, workspace,
               workspace_bytes_, stream, ndim=None, ncoeffs=None) -> int:
    return lib().fpde_bwd(_opid(op),
                          _ptr_array(_dev_ptrs(fields)) if fields is not None else None,
                          _ptr_array(_dev_ptrs(gres)) if gres is not None else None,
                          _f64(gscale) if gscale is not None else None,
                          _ptr_array(_dev_ptrs(gfields)) if gfields is not None else None,
                          len(shape) if ndim is None else ndim,
                          _i64(shape) if shape is not None else None,
                          _f64(spacing) if spacing is not None else None,
                          _f64(coeffs) if coeffs is not None else None,
                          len(coeffs) if ncoeffs is None else ncoeffs,
                          _bcs(bc) if bc is not None else None,
                          _dev_ptrs([workspace])[0] if workspace is not None else None,
                          int(workspace_bytes_), stream)


def has_single_pass(op) -> bool:
    return bool(lib().fpde_has_single_pass(_opid(op)))


def fwd_bwd_workspace_bytes(op, shape) -> int:
    return int(lib().fpde_fwd_bwd_workspace_bytes(_opid(op), len(shape), _i64(shape)))


def fwd_bwd_status(op, fields, sources, residuals, gfields, loss_out, shape, spacing, coeffs, bc, workspace,
                   workspace_bytes_, stream, ndim=None, ncoeffs=None) -> int:
    return lib().fpde_fwd_bwd(_opid(op),
                              _ptr_array(_dev_ptrs(fields)) if fields is not None else None,
                              _ptr_array(_dev_ptrs(sources)) if sources is not None else None,
                              _ptr_array(_dev_ptrs(residuals)) if residuals is not None else None,
                              _ptr_array(_dev_ptrs(gfields)) if gfields is not None else None,
                              _dev_ptrs([loss_out])[0] if loss_out is not None else None,
                              len(shape) if ndim is None else ndim,
                              _i64(shape) if shape is not None else None,
                              _f64(spacing) if spacing is not None else None,
                              _f64(coeffs) if coeffs is not None else None,
                              len(coeffs) if ncoeffs is None else ncoeffs,
                              _bcs(bc) if bc is not None else None,
                              _dev_ptrs([workspace])[0] if workspace is not None else None,
                              int(workspace_bytes_), stream)


def _stream_handle(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if hasattr(stream, "cuda_stream"):
        return stream.cuda_stream
    return int(stream)


class _on_device_of:
    """Context for one call: every tensor argument must live on one CUDA device, and that device
    is made current for the call (the library launches on the current device, so a tensor of
    another GPU would be dereferenced there as a foreign address)."""

    def __init__(self, *groups):
        dev = None
        for g in groups:
            if g is None:
                continue
            for t in (g if isinstance(g, (list, tuple)) else [g]):
                d = getattr(t, "device", None)
                if d is None or not hasattr(t, "data_ptr"):
                    continue
                if d.type != "cuda":
                    raise ValueError("fpde: tensor on %s, expected a CUDA tensor" % (d,))
                if dev is None:
                    dev = d
                elif d != dev:
                    raise ValueError("fpde: tensors of one call live on different devices (%s and %s)" % (dev, d))
        self._ctx = None
        if dev is not None:
            import torch
            self._ctx = torch.cuda.device(dev)

    def __enter__(self):
        if self._ctx is not None:
            self._ctx.__enter__()
        return self

    def __exit__(self, *exc):
        if self._ctx is not None:
            return self._ctx.__exit__(*exc)
        return False


def fpde_fwd(op, fields, sources, residuals, loss_out, shape, spacing, coeffs, bc, workspace, stream=None):
    """Queue the fused forward residual + loss on `stream` (default: torch's current stream).

    fields / sources / residuals: sequences of fp32 CUDA tensors of the grid shape;
    loss_out: fp64 CUDA tensor with nresiduals+1 entries, or None; workspace: a CUDA tensor of at
    least workspace_bytes(op, shape) bytes (uint8 or any dtype)."""
    wsb = workspace.numel() * workspace.element_size() if workspace is not None else 0
    with _on_device_of(fields, sources, residuals, loss_out, workspace):
        st = fwd_status(op, fields, sources, residuals, loss_out, shape, spacing, coeffs, bc, workspace, wsb,
                        _stream_handle(stream))
    if st != FPDE_OK:
        raise FpdeError(st, "fpde_fwd")


def fpde_fwd_rows(op, fields, sources, residuals, loss_out, shape, spacing, coeffs, bc, workspace, loss_rows,
                  stream=None):
    """fpde_fwd whose loss divides by `loss_rows` (the row count of the whole grid when this array
    is one slab of it): the ranks' loss vectors then add up to the loss of the whole grid."""
    wsb = workspace.numel() * workspace.element_size() if workspace is not None else 0
    with _on_device_of(fields, sources, residuals, loss_out, workspace):
        st = fwd_status(op, fields, sources, residuals, loss_out, shape, spacing, coeffs, bc, workspace, wsb,
                        _stream_handle(stream), loss_rows=loss_rows)
    if st != FPDE_OK:
        raise FpdeError(st, "fpde_fwd_rows")


def fpde_fwd_bwd(op, fields, sources, residuals, gfields, loss_out, shape, spacing, coeffs, bc, workspace,
                 stream=None):
    """Queue the loss-specialised pass: loss and dL/dfield (and the residual arrays, where given).

    residuals: None, or a sequence with None entries for residual arrays that need not be stored
    (only where has_single_pass(op); the other operators need all of them).  workspace: a CUDA
    tensor of at least fwd_bwd_workspace_bytes(op, shape) bytes."""
    wsb = workspace.numel() * workspace.element_size() if workspace is not None else 0
    with _on_device_of(fields, sources, residuals, gfields, loss_out, workspace):
        st = fwd_bwd_status(op, fields, sources, residuals, gfields, loss_out, shape, spacing, coeffs, bc, workspace,
                            wsb, _stream_handle(stream))
    if st != FPDE_OK:
        raise FpdeError(st, "fpde_fwd_bwd")


def plane_chunk(op, shape) -> int:
    """Planes per chunk of the ranged launches for this operator and grid (0: the operator has none)."""
    return int(lib().fpde_plane_chunk(_opid(op), len(shape), _i64(shape)))


def fpde_fwd_chunks(op, fields, sources, residuals, loss_out, shape, spacing, coeffs, bc, workspace, loss_rows,
                    chunk_lo, chunk_hi, finish, stream=None):
    """fpde_fwd_rows over the chunks [chunk_lo, chunk_hi) of x-planes only (chunk length: plane_chunk());
    `finish`: form the loss vector from the partial sums of all chunks (the last call of a set that
    covers every chunk).  loss_rows = 0: the array's own row count."""
    wsb = workspace.numel() * workspace.element_size() if workspace is not None else 0
    with _on_device_of(fields, sources, residuals, loss_out, workspace):
        st = lib().fpde_fwd_chunks(_opid(op), _ptr_array(_dev_ptrs(fields)), _ptr_array(_dev_ptrs(sources)),
                                   _ptr_array(_dev_ptrs(residuals)),
                                   _dev_ptrs([loss_out])[0] if loss_out is not None else None, len(shape), _i64(shape),
                                   _f64(spacing), _f64(coeffs), len(coeffs), _bcs(bc),
                                   _dev_ptrs([workspace])[0] if workspace is not None else None, int(wsb),
                                   _stream_handle(stream), int(loss_rows), int(chunk_lo), int(chunk_hi), int(bool(finish)))
    if st != FPDE_OK:
        raise FpdeError(st, "fpde_fwd_chunks")


def fpde_bwd_chunks(op, fields, gres, gscale, gfields, shape, spacing, coeffs, bc, chunk_lo, chunk_hi, stream=None):
    """fpde_bwd over the chunks [chunk_lo, chunk_hi) of x-planes only."""
    with _on_device_of(fields, gres, gfields):
        st = lib().fpde_bwd_chunks(_opid(op), _ptr_array(_dev_ptrs(fields)), _ptr_array(_dev_ptrs(gres)),
                                   _f64(gscale) if gscale is not None else None, _ptr_array(_dev_ptrs(gfields)),
                                   len(shape), _i64(shape), _f64(spacing), _f64(coeffs), len(coeffs), _bcs(bc),
                                   _stream_handle(stream), int(chunk_lo), int(chunk_hi))
    if st != FPDE_OK:
        raise FpdeError(st, "fpde_bwd_chunks")


class PreparedStep:
    """The arguments of fpde_fwd / fpde_bwd / fpde_fwd_bwd for one set of tensors, marshalled ONCE.

    Turning tensors into pointer arrays costs more host time than a small grid's kernels take on the
    GPU (tens of microseconds per call against a few); a training loop calls the same operator on the
    same tensors every step, so this object builds the C arguments once and each `fwd()` / `bwd()` /
    `fwd_bwd()` is then a single foreign call on torch's current stream.  Pure marshalling: every
    step still runs in the library's kernels.  The tensors must stay alive and in place."""

    def __init__(self, op, fields, sources, residuals, gfields, loss_out, shape, spacing, coeffs, bc,
                 workspace=None, gscale=None, fwd_bwd_workspace=None):
        self._keep = (fields, sources, residuals, gfields, loss_out, workspace, fwd_bwd_workspace)
        _on_device_of(fields, sources, residuals, gfields, loss_out, workspace, fwd_bwd_workspace)   # one device?
        self._idx = fields[0].device.index
        L = lib()
        self._op = _opid(op)
        self._nd = len(shape)
        self._f, self._s = _ptr_array(_dev_ptrs(fields)), _ptr_array(_dev_ptrs(sources))
        self._r = _ptr_array(_dev_ptrs(residuals)) if residuals is not None else None
        self._g = _ptr_array(_dev_ptrs(gfields)) if gfields is not None else None
        self._loss = _dev_ptrs([loss_out])[0] if loss_out is not None else None
        self._shape, self._h, self._c, self._nc, self._bc = _i64(shape), _f64(spacing), _f64(coeffs), len(coeffs), _bcs(bc)
        self._ws = _dev_ptrs([workspace])[0] if workspace is not None else None
        self._wsb = workspace.numel() * workspace.element_size() if workspace is not None else 0
        self._ws2 = _dev_ptrs([fwd_bwd_workspace])[0] if fwd_bwd_workspace is not None else None
        self._wsb2 = fwd_bwd_workspace.numel() * fwd_bwd_workspace.element_size() if fwd_bwd_workspace is not None else 0
        if gscale is None and residuals is not None:
            rows = L.fpde_row_count(self._op, self._nd, self._shape)
            gscale = [2.0 / rows] * len(residuals)
        self._gs = _f64(gscale) if gscale is not None else None
        self._fwd, self._bwd, self._fb = L.fpde_fwd, L.fpde_bwd, L.fpde_fwd_bwd
        import torch
        self._torch = torch

    def _call(self, fn, name, *args):
        t = self._torch
        if t.cuda.current_device() == self._idx:        # the usual case: no device switch needed
            st = fn(*args, t.cuda.current_stream().cuda_stream)
        else:
            with t.cuda.device(self._idx):
                st = fn(*args, t.cuda.current_stream().cuda_stream)
        if st != FPDE_OK:
            raise FpdeError(st, name)

    def fwd(self):
        """fpde_fwd(fields, sources -> residuals, loss) on the current stream."""
        self._call(self._fwd, "fpde_fwd", self._op, self._f, self._s, self._r, self._loss, self._nd, self._shape,
                   self._h, self._c, self._nc, self._bc, self._ws, self._wsb)

    def bwd(self):
        """fpde_bwd with the residual arrays as upstream arrays and the prepared scales (default 2/N_r:
        the gradient of the fused loss) -> gfields."""
        self._call(self._bwd, "fpde_bwd", self._op, self._f, self._r, self._gs, self._g, self._nd, self._shape,
                   self._h, self._c, self._nc, self._bc, None, 0)

    def fwd_bwd(self, store_residuals=True):
        """fpde_fwd_bwd: loss and gradient from one call."""
        self._call(self._fb, "fpde_fwd_bwd", self._op, self._f, self._s, self._r if store_residuals else None, self._g,
                   self._loss, self._nd, self._shape, self._h, self._c, self._nc, self._bc, self._ws2, self._wsb2)


def workspace_bytes_f64(op, shape) -> int:
    return int(lib().fpde_workspace_bytes_f64(_opid(op), len(shape), _i64(shape)))


def fpde_fwd_f64(op, fields, sources, residuals, loss_out, shape, spacing, coeffs, bc, workspace, stream=None):
    """fpde_fwd on fp64 CUDA tensors (verification path)."""
    wsb = workspace.numel() * workspace.element_size() if workspace is not None else 0
    with _on_device_of(fields, sources, residuals, loss_out, workspace):
        st = lib().fpde_fwd_f64(_opid(op), _ptr_array(_dev_ptrs(fields)), _ptr_array(_dev_ptrs(sources)),
                                _ptr_array(_dev_ptrs(residuals)),
                                _dev_ptrs([loss_out])[0] if loss_out is not None else None, len(shape), _i64(shape),
                                _f64(spacing), _f64(coeffs), len(coeffs), _bcs(bc),
                                _dev_ptrs([workspace])[0] if workspace is not None else None, int(wsb),
                                _stream_handle(stream))
    if st != FPDE_OK:
        raise FpdeError(st, "fpde_fwd_f64")


def fpde_bwd_f64(op, fields, gres, gscale, gfields, shape, spacing, coeffs, bc, stream=None):
    """fpde_bwd on fp64 CUDA tensors (verification path)."""
    with _on_device_of(fields, gres, gfields):
        st = lib().fpde_bwd_f64(_opid(op), _ptr_array(_dev_ptrs(fields)), _ptr_array(_dev_ptrs(gres)),
                                _f64(gscale) if gscale is not None else None, _ptr_array(_dev_ptrs(gfields)),
                                len(shape), _i64(shape), _f64(spacing), _f64(coeffs), len(coeffs), _bcs(bc),
                                _stream_handle(stream))
    if st != FPDE_OK:
        raise FpdeError(st, "fpde_bwd_f64")


def fpde_bwd(op, fields, gres, gscale, gfields, shape, spacing, coeffs, bc, workspace=None, stream=None):
    """Queue the gather-form adjoint (with its boundary correction) on `stream`."""
    wsb = workspace.numel() * workspace.element_size() if workspace is not None else 0
    with _on_device_of(fields, gres, gfields, workspace):
        st = bwd_status(op, fields, gres, gscale, gfields, shape, spacing, coeffs, bc, workspace, wsb,
                        _stream_handle(stream))
    if st != FPDE_OK:
        raise FpdeError(st, "fpde_bwd")


def host_arena_bytes(op, shape) -> int:
    return int(lib().fpde_host_arena_bytes(_opid(op), len(shape), _i64(shape)))


def host_pipeline_plan(n0: int):
    """Chunks of the pipelined host path for n0 x-planes: list of (first plane of the chunk, first
    plane of its upload transfer, one past the transfer's last plane); empty if the plain form runs."""
    L = lib()
    k = L.fpde_host_pipeline_plan(int(n0), None, 0)
    if k <= 0:
        return []
    buf = (ctypes.c_int * (3 * k))()
    got = L.fpde_host_pipeline_plan(int(n0), buf, k)
    if got != k:
        raise FpdeError("fpde_host_pipeline_plan", got)
    return [(buf[3 * c], buf[3 * c + 1], buf[3 * c + 2]) for c in range(k)]


def loss_grad_host_status(op, h_fields, h_sources, h_gfields, h_loss, shape, spacing, coeffs, bc, arena,
                          arena_bytes, stream) -> int:
    return lib().fpde_loss_grad_host(_opid(op),
                                     _ptr_array(_dev_ptrs(h_fields)) if h_fields is not None else None,
                                     _ptr_array(_dev_ptrs(h_sources)) if h_sources is not None else None,
                                     _ptr_array(_dev_ptrs(h_gfields)) if h_gfields is not None else None,
                                     _dev_ptrs([h_loss])[0] if h_loss is not None else None,
                                     len(shape), _i64(shape), _f64(spacing), _f64(coeffs), len(coeffs), _bcs(bc),
                                     _dev_ptrs([arena])[0] if arena is not None else None, int(arena_bytes), stream)


def fpde_loss_grad_host(op, h_fields, h_sources, h_gfields, h_loss, shape, spacing, coeffs, bc, arena, stream=None):
    """Loss and dL/dfield from HOST tensors (pinned CPU tensors recommended): H2D copies, forward,
    adjoint and D2H copies are queued on `stream`; synchronise it before reading the results.
    `arena` is a CUDA tensor of at least host_arena_bytes(op, shape) bytes."""
    ab = arena.numel() * arena.element_size()
    with _on_device_of(arena):
        st = loss_grad_host_status(op, h_fields, h_sources, h_gfields, h_loss, shape, spacing, coeffs, bc, arena, ab,
                                   _stream_handle(stream))
    if st != FPDE_OK:
        raise FpdeError(st, "fpde_loss_grad_host")


NOALLOC_SCRATCH_BYTES = 256 * 1024      # FPDE_NOALLOC_SCRATCH_BYTES of include/fpde.h


def fwd_noalloc_status(op, fields, sources, residuals, loss_out, shape, spacing, coeffs, bc, stream) -> int:
    return lib().fpde_fwd_noalloc(_opid(op), _ptr_array(_dev_ptrs(fields)), _ptr_array(_dev_ptrs(sources)),
                                  _ptr_array(_dev_ptrs(residuals)),
                                  _dev_ptrs([loss_out])[0] if loss_out is not None else None,
                                  len(shape), _i64(shape), _f64(spacing), _f64(coeffs), len(coeffs), _bcs(bc),
                                  stream)


def fpde_fwd_noalloc(op, fields, sources, residuals, loss_out, shape, spacing, coeffs, bc, stream=None):
    """fpde_fwd for callers that cannot allocate a workspace (no allocator at hand, or a region
    where cudaMalloc must not be called): the loss partial sums live in a fixed array inside the
    library.  Grids needing more than NOALLOC_SCRATCH_BYTES of scratch raise FpdeError (status 9).
    Calls on one device share that array, so keep them ordered on the GPU; make the first call on
    a device outside stream capture."""
    with _on_device_of(fields, sources, residuals, loss_out):
        st = fwd_noalloc_status(op, fields, sources, residuals, loss_out, shape, spacing, coeffs, bc,
                                _stream_handle(stream))
    if st != FPDE_OK:
        raise FpdeError(st, "fpde_fwd_noalloc")


def diag_ns_tma_geometry(shape, tile_rows: int, narrays: int, smem_limit: int) -> bool:
    """Host-only: would the shared-memory-staged NS kernels take this (x,y,z,t) grid?"""
    return bool(lib().fpde_diag_ns_tma_geometry(_i64(shape), int(tile_rows), int(narrays), int(smem_limit)))


def diag_tma_timeouts() -> int:
    """Bounded barrier waits that gave up on the current device (0 in a healthy run)."""
    return int(lib().fpde_diag_tma_timeouts())
