"""Seeded synthetic workloads for the fused finite-difference PDE-residual operators.

This module only *describes inputs*: grid shapes, spacings, PDE coefficients, boundary kinds
and the field arrays (an analytic profile plus seeded noise).  It contains none of the method's
arithmetic (no difference formula, no residual, no adjoint) and depends on numpy alone, so both
the CUDA path's tests and the CPU oracle's tests may draw their inputs from it.

Grids are row-major, axes in the order a workload names its coordinates, last axis contiguous
(space-time grids have ``t`` fastest).  A non-periodic axis on ``[a, b]`` has nodes
``a + i*(b-a)/(n-1)`` (both end points are nodes); a periodic axis on ``[a, b)`` has nodes
``a + i*(b-a)/n``.

Fields are generated in fp64 and rounded once to fp32; that fp32 array is what the GPU reads and
what the oracle promotes to double.

Random numbers come from a counter-based generator (a SplitMix64-style hash of
``(seed, stream, linear index)``), so any element can be regenerated on its own and results do
not depend on a library's implementation-defined distributions.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

# Operator names (strings on purpose: the CUDA binding and the oracle each map them to their
# own numeric ids).
BURGERS_1D_T = "burgers_1d_t"
POISSON_2D = "poisson_2d"
GRAYSCOTT_2D = "grayscott_2d"
HELMHOLTZ_3D_O4 = "helmholtz_3d_o4"
NS_3D_T = "ns_3d_t"
NS_2D_STEADY = "ns_2d_steady"
NS_3D_STEADY = "ns_3d_steady"
NS_3D_T_XSLAB = "ns_3d_t_xslab"     # NS_3D_T with a non-periodic x axis: the form of one slab of a grid split along x
GRAYSCOTT_2D_XSLAB = "grayscott_2d_xslab"   # the same for Gray-Scott
OPS = (BURGERS_1D_T, POISSON_2D, GRAYSCOTT_2D, HELMHOLTZ_3D_O4, NS_3D_T, NS_2D_STEADY, NS_3D_STEADY, NS_3D_T_XSLAB,
       GRAYSCOTT_2D_XSLAB)

# Boundary kinds per array axis.
PERIODIC = "periodic"      # rows at every node, wrap-around neighbours
INTERIOR = "interior"      # rows only where the full stencil fits; shell nodes are data
ONE_SIDED = "one_sided"    # rows at every node, second-order one-sided formulas at the edges

_U64 = np.uint64
_MASK53 = (1 << 53) - 1


def _mix64(z: np.ndarray) -> np.ndarray:
    """SplitMix64 finaliser on uint64 arrays (wrap-around arithmetic)."""
    z = z.copy()
    z ^= z >> _U64(30)
    z *= _U64(0xBF58476D1CE4E5B9)
    z ^= z >> _U64(27)
    z *= _U64(0x94D049BB133111EB)
    z ^= z >> _U64(31)
    return z


def _key(seed: int, stream: int) -> np.uint64:
    k = (seed * 0x9E3779B97F4A7C15 + stream * 0xD1B54A32D192ED03 + 0x2545F4914F6CDD1D) & 0xFFFFFFFFFFFFFFFF
    return _mix64(np.array([k], dtype=_U64))[0]


def uniform01(seed: int, stream: int, n: int, start: int = 0) -> np.ndarray:
    """``n`` doubles in the open interval (0, 1), elements ``start .. start+n-1`` of the
    stream ``(seed, stream)``."""
    idx = np.arange(start, start + n, dtype=_U64)
    with np.errstate(over="ignore"):
        z = _mix64(idx * _U64(0x9E3779B97F4A7C15) + _key(seed, stream))
    return ((z >> _U64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal01(seed: int, stream: int, n: int, start: int = 0) -> np.ndarray:
    """Standard normals by Box-Muller from two independent uniform streams."""
    u1 = uniform01(seed, 2 * stream + 1000003, n, start)
    u2 = uniform01(seed, 2 * stream + 1000004, n, start)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)


def axis_nodes(n: int, lo: float, hi: float, periodic: bool) -> Tuple[np.ndarray, float]:
    h = (hi - lo) / n if periodic else (hi - lo) / (n - 1)
    return lo + h * np.arange(n, dtype=np.float64), h


@dataclass
class Workload:
    name: str
    op: str
    shape: Tuple[int, ...]
    spacing: Tuple[float, ...]
    coeffs: Tuple[float, ...]
    bc: Tuple[str, ...]
    fields: List[np.ndarray]                 # fp32, C-contiguous, full grid shape
    sources: List[np.ndarray] = field(default_factory=list)
    field_names: Tuple[str, ...] = ()
    residual_names: Tuple[str, ...] = ()
    seed: int = 42
    kind: str = "config"

    @property
    def npoints(self) -> int:
        return int(np.prod(self.shape))


# name -> (op, default shape, domain per axis (lo, hi), bc per axis)
CONFIGS: Dict[str, dict] = {
    "burgers_256x128": dict(op=BURGERS_1D_T, shape=(256, 128),
                            domain=((-1.0, 1.0), (0.0, 1.0)), bc=(ONE_SIDED, ONE_SIDED)),
    "poisson_1024": dict(op=POISSON_2D, shape=(1024, 1024),
                         domain=((0.0, 1.0), (0.0, 1.0)), bc=(INTERIOR, INTERIOR)),
    "grayscott_4096": dict(op=GRAYSCOTT_2D, shape=(4096, 4096),
                           domain=((0.0, 1.0), (0.0, 1.0)), bc=(PERIODIC, PERIODIC)),
    "helmholtz_256": dict(op=HELMHOLTZ_3D_O4, shape=(256, 256, 256),
                          domain=((0.0, 1.0),) * 3, bc=(INTERIOR,) * 3),
    "ns_tgv_128x16": dict(op=NS_3D_T, shape=(128, 128, 128, 16),
                          domain=((0.0, 2 * math.pi),) * 3 + ((0.0, 1.0),),
                          bc=(PERIODIC, PERIODIC, PERIODIC, INTERIOR)),
}
# beyond the five baseline configurations: the paper's own worked operator (steady 2-D
# Navier-Stokes, its lid-driven-cavity case) on a grid large enough to measure against HBM
CONFIGS["ns2d_steady_4096"] = dict(op=NS_2D_STEADY, shape=(4096, 4096),
                                   domain=((0.0, 1.0), (0.0, 1.0)), bc=(INTERIOR, INTERIOR))
CONFIGS["ns3d_steady_256"] = dict(op=NS_3D_STEADY, shape=(256, 256, 256),
                                  domain=((0.0, 1.0),) * 3, bc=(INTERIOR,) * 3)
# one of four x-slabs of the 128^3 x 16 Navier-Stokes grid, with its two halo planes
CONFIGS["ns_tgv_xslab_34"] = dict(op=NS_3D_T_XSLAB, shape=(34, 128, 128, 16),
                                  domain=((0.0, 2 * math.pi * 33 / 128),) + ((0.0, 2 * math.pi),) * 2 + ((0.0, 1.0),),
                                  bc=(INTERIOR, PERIODIC, PERIODIC, INTERIOR))
# one of four x-slabs of the 4096^2 Gray-Scott grid, with its two halo rows
CONFIGS["grayscott_xslab_1026"] = dict(op=GRAYSCOTT_2D_XSLAB, shape=(1026, 4096),
                                       domain=((0.0, 1025.0 / 4096.0), (0.0, 1.0)), bc=(INTERIOR, PERIODIC))
EXTRA_CONFIGS = ("ns2d_steady_4096", "ns3d_steady_256")
SLAB_CONFIGS = ("ns_tgv_xslab_34", "grayscott_xslab_1026")
CONFIG_ORDER = ("burgers_256x128", "poisson_1024", "grayscott_4096", "helmholtz_256", "ns_tgv_128x16")

OP_META = {
    BURGERS_1D_T: dict(fields=("u",), sources=(), residuals=("r",), ncoeffs=1),
    POISSON_2D: dict(fields=("u",), sources=("f",), residuals=("r",), ncoeffs=0),
    GRAYSCOTT_2D: dict(fields=("u", "v"), sources=(), residuals=("r_u", "r_v"), ncoeffs=4),
    HELMHOLTZ_3D_O4: dict(fields=("u",), sources=("f",), residuals=("r",), ncoeffs=1),
    NS_3D_T: dict(fields=("u", "v", "w", "p"), sources=(),
                  residuals=("mom_x", "mom_y", "mom_z", "continuity"), ncoeffs=1),
    NS_2D_STEADY: dict(fields=("u", "v", "p"), sources=(), residuals=("res_u", "res_v", "res_div"), ncoeffs=1),
    NS_3D_STEADY: dict(fields=("u", "v", "w", "p"), sources=(),
                       residuals=("mom_x", "mom_y", "mom_z", "continuity"), ncoeffs=1),
    NS_3D_T_XSLAB: dict(fields=("u", "v", "w", "p"), sources=(),
                        residuals=("mom_x", "mom_y", "mom_z", "continuity"), ncoeffs=1),
    GRAYSCOTT_2D_XSLAB: dict(fields=("u", "v"), sources=(), residuals=("r_u", "r_v"), ncoeffs=4),
}
DEFAULT_COEFFS = {
    BURGERS_1D_T: (0.01 / math.pi,),
    POISSON_2D: (),
    GRAYSCOTT_2D: (2e-5, 1e-5, 0.04, 0.06),
    HELMHOLTZ_3D_O4: (4 * math.pi,),
    NS_3D_T: (0.01,),
    NS_2D_STEADY: (0.01,),
    NS_3D_STEADY: (0.01,),
    NS_3D_T_XSLAB: (0.01,),
    GRAYSCOTT_2D_XSLAB: (2e-5, 1e-5, 0.04, 0.06),
}


def _noise(seed, stream, shape, sigma):
    n = int(np.prod(shape))
    return (sigma * normal01(seed, stream, n)).reshape(shape)


def _grids(shape, domain, bc):
    axes, hs = [], []
    for n, (lo, hi), b in zip(shape, domain, bc):
        x, h = axis_nodes(n, lo, hi, b == PERIODIC)
        axes.append(x)
        hs.append(h)
    return axes, tuple(hs)


def _bcast(axes, a):
    """Axis ``a``'s node coordinates shaped for broadcasting over the full grid."""
    shp = [1] * len(axes)
    shp[a] = -1
    return axes[a].reshape(shp)


def analytic_fields(op: str, axes: Sequence[np.ndarray], coeffs: Sequence[float]) -> Tuple[List[np.ndarray], List[np.ndarray]]:
    """Noise-free fp64 fields and sources of each workload's recipe on the given node coordinates."""
    shape = tuple(len(a) for a in axes)
    if op == BURGERS_1D_T:
        x, t = _bcast(axes, 0), _bcast(axes, 1)
        return [np.broadcast_to(-np.sin(math.pi * x) * np.exp(-t), shape).copy()], []
    if op == POISSON_2D:
        x, y = _bcast(axes, 0), _bcast(axes, 1)
        us = np.sin(math.pi * x) * np.sin(math.pi * y)
        return [us.copy()], [2 * math.pi ** 2 * us]
    if op in (GRAYSCOTT_2D, GRAYSCOTT_2D_XSLAB):
        return [np.full(shape, 0.95), np.full(shape, 0.05)], []
    if op == HELMHOLTZ_3D_O4:
        x, y, z = (_bcast(axes, a) for a in range(3))
        us = np.sin(2 * math.pi * x) * np.sin(2 * math.pi * y) * np.sin(2 * math.pi * z)
        k = coeffs[0]
        return [us.copy()], [(k * k - 12 * math.pi ** 2) * us]
    if op in (NS_3D_T, NS_3D_T_XSLAB):
        x, y, z, t = (_bcast(axes, a) for a in range(4))
        nu = coeffs[0]
        e2, e4 = np.exp(-2 * nu * t), np.exp(-4 * nu * t)
        u = np.sin(x) * np.cos(y) * np.cos(z) * e2
        v = -np.cos(x) * np.sin(y) * np.cos(z) * e2
        w = np.zeros(shape)
        p = (np.cos(2 * x) + np.cos(2 * y)) * (np.cos(2 * z) + 2.0) / 16.0 * e4
        return [np.broadcast_to(a, shape).copy() for a in (u, v, w, p)], []
    if op == NS_2D_STEADY:
        x, y = _bcast(axes, 0), _bcast(axes, 1)
        u = np.sin(math.pi * x) * np.cos(math.pi * y)
        v = -np.cos(math.pi * x) * np.sin(math.pi * y)
        p = 0.25 * (np.cos(2 * math.pi * x) + np.cos(2 * math.pi * y))
        return [np.broadcast_to(a, shape).copy() for a in (u, v, p)], []
    if op == NS_3D_STEADY:
        x, y, z = (_bcast(axes, a) for a in range(3))
        pi = math.pi
        u = np.sin(pi * x) * np.cos(pi * y) * np.cos(pi * z)
        v = -0.5 * np.cos(pi * x) * np.sin(pi * y) * np.cos(pi * z)
        w = -0.5 * np.cos(pi * x) * np.cos(pi * y) * np.sin(pi * z)
        p = 0.25 * (np.cos(2 * pi * x) + np.cos(2 * pi * y) + np.cos(2 * pi * z))
        return [np.broadcast_to(a, shape).copy() for a in (u, v, w, p)], []
    raise ValueError(op)


_NOISE_SIGMA = {BURGERS_1D_T: 0.01, POISSON_2D: 0.05, HELMHOLTZ_3D_O4: 0.05, NS_3D_T: 0.01, NS_2D_STEADY: 0.01, NS_3D_STEADY: 0.01,
                NS_3D_T_XSLAB: 0.01}


def make(name: str, seed: int = 42, shape: Optional[Sequence[int]] = None, kind: str = "config",
         spacing: Optional[Sequence[float]] = None, coeffs: Optional[Sequence[float]] = None) -> Workload:
    """Build a workload.

    ``name``  one of ``CONFIG_ORDER`` (or an operator name, which selects that operator's config).
    ``shape`` overrides the grid extents (same domain, spacing follows from the extents).
    ``kind``  ``"config"``: the named recipe (analytic profile + seeded noise);
              ``"randn"``: independent standard-normal entries in every field and source (the
              paper's verification inputs, seeds 42-46).
    ``spacing`` overrides the spacings (used for unequal-spacing stress cases; the analytic
              profile is then evaluated on the nodes ``lo + i*h``).
    """
    if name in OPS:
        name = next(k for k in CONFIG_ORDER + EXTRA_CONFIGS + SLAB_CONFIGS if CONFIGS[k]["op"] == name)
    cfg = CONFIGS[name]
    op = cfg["op"]
    shape = tuple(int(s) for s in (shape if shape is not None else cfg["shape"]))
    if len(shape) != len(cfg["shape"]):
        raise ValueError("shape rank mismatch")
    meta = OP_META[op]
    coeffs = tuple(float(c) for c in (coeffs if coeffs is not None else DEFAULT_COEFFS[op]))
    axes, hs = _grids(shape, cfg["domain"], cfg["bc"])
    if spacing is not None:
        hs = tuple(float(h) for h in spacing)
        axes = [lo + h * np.arange(n, dtype=np.float64) for n, (lo, _), h in zip(shape, cfg["domain"], hs)]
    nf, ns = len(meta["fields"]), len(meta["sources"])
    if kind == "randn":
        fields = [_noise(seed, 10 + i, shape, 1.0) for i in range(nf)]
        sources = [_noise(seed, 50 + i, shape, 1.0) for i in range(ns)]
    elif kind == "config":
        fields, sources = analytic_fields(op, axes, coeffs)
        if op in (GRAYSCOTT_2D, GRAYSCOTT_2D_XSLAB):
            n = int(np.prod(shape))
            fields = [0.9 + 0.1 * uniform01(seed, 10, n).reshape(shape),
                      0.1 * uniform01(seed, 11, n).reshape(shape)]
        else:
            sig = _NOISE_SIGMA[op]
            fields = [f + _noise(seed, 10 + i, shape, sig) for i, f in enumerate(fields)]
    else:
        raise ValueError(kind)
    f32 = [np.ascontiguousarray(f, dtype=np.float32) for f in fields]
    s32 = [np.ascontiguousarray(s, dtype=np.float32) for s in sources]
    return Workload(name=name, op=op, shape=shape, spacing=hs, coeffs=coeffs, bc=tuple(cfg["bc"]),
                    fields=f32, sources=s32, field_names=meta["fields"],
                    residual_names=meta["residuals"], seed=seed, kind=kind)


def random_sensitivities(w: Workload, seed: int = 7) -> List[np.ndarray]:
    """Seeded standard-normal upstream arrays ``dL/dr_e`` (fp32, full grid shape) for testing the
    adjoint on its own."""
    ne = len(OP_META[w.op]["residuals"])
    return [np.ascontiguousarray(_noise(seed, 90 + e, w.shape, 1.0), dtype=np.float32) for e in range(ne)]
