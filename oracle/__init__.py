"""fp64 CPU oracle for the fused finite-difference PDE-residual operators -- TEST INFRASTRUCTURE.

Only ``tests/``, the smoke check and the bench's CPU-baseline / reference legs may import this
package.  It shares nothing with the CUDA library: its own C source (``fpde_oracle.c``), its
own operator ids, its own build.  Inputs are the fp32 arrays a workload holds, promoted to
double here; nothing is regenerated.

``fwd`` evaluates every residual row from its definition and the mean-square loss
(Section 2.1 of the paper for the residual structure, with the per-operator readings listed in
the design notes); ``bwd`` forms ``J^T G`` by scatter over rows (Section 2.2 / Appendix A.3).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fpde_oracle.c")
_LIB = os.path.join(_HERE, "libfpde_oracle.so")

OP_IDS = {"burgers_1d_t": 0, "poisson_2d": 1, "grayscott_2d": 2, "helmholtz_3d_o4": 3, "ns_3d_t": 4, "ns_2d_steady": 5, "ns_3d_steady": 6,
          "ns_3d_t_xslab": 7, "grayscott_2d_xslab": 8}

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, strict IEEE: no -ffast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        pp = ctypes.POINTER(ctypes.c_void_p)
        lib.fpde_oracle_fwd.restype = ctypes.c_longlong
        lib.fpde_oracle_fwd.argtypes = [ctypes.c_int, pp, pp, pp, ctypes.c_void_p, ctypes.c_int,
                                        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        lib.fpde_oracle_bwd.restype = ctypes.c_longlong
        lib.fpde_oracle_bwd.argtypes = [ctypes.c_int, pp, pp, pp, ctypes.c_int,
                                        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        _lib = lib
    return _lib


def _ptrs(arrs: Sequence[np.ndarray]):
    a = (ctypes.c_void_p * max(1, len(arrs)))()
    for i, x in enumerate(arrs):
        a[i] = x.ctypes.data
    return ctypes.cast(a, ctypes.POINTER(ctypes.c_void_p))


def _f64(arrs) -> List[np.ndarray]:
    return [np.ascontiguousarray(a, dtype=np.float64) for a in arrs]


def fwd(op: str, fields, sources, shape, spacing, coeffs) -> Tuple[List[np.ndarray], np.ndarray, int]:
    """Residual arrays (fp64, zero at nodes without a row), ``loss`` = [L_e..., L], row count."""
    lib = _load()
    opi = OP_IDS[op]
    shape = tuple(int(s) for s in shape)
    F, S = _f64(fields), _f64(sources)
    for a in F + S:
        assert a.shape == shape, (a.shape, shape)
    ne = {0: 1, 1: 1, 2: 2, 3: 1, 4: 4, 5: 3, 6: 4, 7: 4, 8: 2}[opi]
    R = [np.empty(shape, dtype=np.float64) for _ in range(ne)]
    loss = np.zeros(ne + 1, dtype=np.float64)
    shp = np.asarray(shape, dtype=np.int64)
    sp = np.asarray(spacing, dtype=np.float64)
    co = np.asarray(list(coeffs) + [0.0], dtype=np.float64)
    rows = lib.fpde_oracle_fwd(opi, _ptrs(F), _ptrs(S), _ptrs(R), loss.ctypes.data, len(shape),
                               shp.ctypes.data, sp.ctypes.data, co.ctypes.data)
    if rows < 0:
        raise ValueError("oracle rejected the problem (code %d)" % rows)
    return R, loss, int(rows)


def bwd(op: str, fields, G, shape, spacing, coeffs) -> List[np.ndarray]:
    """``J^T G`` for upstream sensitivities ``G`` (one full-shape array per residual)."""
    lib = _load()
    opi = OP_IDS[op]
    shape = tuple(int(s) for s in shape)
    F, Gd = _f64(fields), _f64(G)
    for a in F + Gd:
        assert a.shape == shape, (a.shape, shape)
    g = [np.empty(shape, dtype=np.float64) for _ in range(len(F))]
    shp = np.asarray(shape, dtype=np.int64)
    sp = np.asarray(spacing, dtype=np.float64)
    co = np.asarray(list(coeffs) + [0.0], dtype=np.float64)
    rows = lib.fpde_oracle_bwd(opi, _ptrs(F), _ptrs(Gd), _ptrs(g), len(shape),
                               shp.ctypes.data, sp.ctypes.data, co.ctypes.data)
    if rows < 0:
        raise ValueError("oracle rejected the problem (code %d)" % rows)
    return g


def loss_and_grad(op: str, fields, sources, shape, spacing, coeffs):
    """Forward, then ``G_e = (2/N_r) r_e``, then backward: residuals, loss vector, dL/du."""
    R, loss, rows = fwd(op, fields, sources, shape, spacing, coeffs)
    G = [r * (2.0 / rows) for r in R]
    return R, loss, bwd(op, fields, G, shape, spacing, coeffs), rows
