"""Pins for the fp64 CPU oracle: every check compares it with something that is NOT the oracle.

  * polynomial exactness of the difference formulas (closed-form residuals at every row,
    edges and corners included);
  * closed forms on trigonometric / exponential fields (they are eigenfunctions of the centred
    differences, so the discrete residual is known exactly);
  * convergence order on manufactured smooth fields (2nd order, 4th for Helmholtz);
  * the adjoint identity <J du, w> = <du, J^T w>, with J du obtained from the forward only;
  * brute-force central finite differences of the loss on tiny grids;
  * the paper's printed u-adjoint of steady 2-D Navier-Stokes (Eq. 1 / Appendix A.3), to which
    the 3-D unsteady operator must reduce for fields constant in z and t;
  * special cases and symmetries; two hand-worked fixtures under tests/golden/.
"""
import math
import os

import zlib

import numpy as np
import pytest

import oracle
from paper_2607_18020_b200 import workloads as W

pi = math.pi
rng = np.random.default_rng(1234)


def _mesh(shape, spacing, lo=None):
    lo = lo or [0.0] * len(shape)
    ax = [l + h * np.arange(n) for n, h, l in zip(shape, spacing, lo)]
    return np.meshgrid(*ax, indexing="ij")


def _rel(a, b):
    return float(np.max(np.abs(a - b)) / max(np.max(np.abs(b)), 1e-300))


# --------------------------------------------------------------------------------------------
# 1. polynomial exactness
# --------------------------------------------------------------------------------------------
def test_poisson_cubic_exact():
    shape, h = (9, 12), (0.3, 0.07)
    x, y = _mesh(shape, h, [0.5, -1.0])
    u = x ** 3 - 2 * y ** 3 + 3 * x * x * y + x * y + 1.5
    f = 0.25 * x - y
    R, loss, rows = oracle.fwd(W.POISSON_2D, [u], [f], shape, h, ())
    exact = -(6 * x + 6 * y - 12 * y) - f          # -(u_xx + u_yy) - f
    r = R[0]
    assert rows == 7 * 10
    assert np.allclose(r[1:-1, 1:-1], exact[1:-1, 1:-1], rtol=0, atol=1e-9)
    # ring nodes carry no row
    mask = np.ones(shape, bool); mask[1:-1, 1:-1] = False
    assert np.all(r[mask] == 0.0)
    assert abs(loss[0] - np.sum(exact[1:-1, 1:-1] ** 2) / 70) < 1e-9 * loss[0]
    assert loss[1] == loss[0]


def test_helmholtz_quintic_exact():
    shape, h = (9, 8, 10), (0.2, 0.15, 0.11)
    x, y, z = _mesh(shape, h, [0.1, 0.2, -0.4])
    u = x ** 4 + 2 * y ** 4 - z ** 4 + x ** 5 - 0.5 * z ** 5 + x * y * z + 3 * y ** 3
    f = x - 2 * y + z * z
    k = 1.7
    R, loss, rows = oracle.fwd(W.HELMHOLTZ_3D_O4, [u], [f], shape, h, (k,))
    lap = 12 * x ** 2 + 24 * y ** 2 - 12 * z ** 2 + 20 * x ** 3 - 10 * z ** 3 + 18 * y
    exact = lap + k * k * u - f
    r = R[0]
    assert rows == 5 * 4 * 6
    inner = (slice(2, -2),) * 3
    assert np.allclose(r[inner], exact[inner], rtol=0, atol=2e-9 * np.abs(exact).max())
    mask = np.ones(shape, bool); mask[inner] = False
    assert np.all(r[mask] == 0.0)


def test_burgers_quadratic_exact_all_nodes():
    """All first-derivative formulas (centred and one-sided) are exact on quadratics, and so are
    both second-derivative formulas: the residual is known at every node, corners included."""
    shape, h = (7, 6), (0.25, 0.4)
    x, t = _mesh(shape, h, [-1.0, 0.0])
    a, b, c, d, e, m = 0.3, -1.2, 0.7, 0.9, -0.35, 0.2
    u = a + b * x + c * x * x + d * t + e * t * t + m * x * t
    nu = 0.37
    R, loss, rows = oracle.fwd(W.BURGERS_1D_T, [u], [], shape, h, (nu,))
    exact = (d + 2 * e * t + m * x) + u * (b + 2 * c * x + m * t) - nu * 2 * c
    assert rows == 42
    assert np.allclose(R[0], exact, rtol=0, atol=1e-11)
    assert abs(loss[0] - np.mean(exact ** 2)) < 1e-12


def test_burgers_second_difference_exact_on_cubics_incl_edges():
    """Isolate D_xx by differencing two runs in nu: r(nu1) - r(nu2) = -(nu1 - nu2) D_xx u.
    The four-point one-sided rule (2,-5,4,-1)/h^2 is exact on cubics, the three-point one is
    not, so this tells them apart."""
    shape, h = (8, 5), (0.3, 0.2)
    x, t = _mesh(shape, h, [-0.7, 0.0])
    u = x ** 3 - 2 * x * x + 0.5 * x + t
    r1 = oracle.fwd(W.BURGERS_1D_T, [u], [], shape, h, (1.0,))[0][0]
    r2 = oracle.fwd(W.BURGERS_1D_T, [u], [], shape, h, (3.0,))[0][0]
    dxx = -(r1 - r2) / (1.0 - 3.0)
    assert np.allclose(dxx, 6 * x - 4, rtol=0, atol=1e-10)


def test_ns_quadratic_exact_away_from_wrap():
    shape, h = (6, 7, 5, 6), (0.3, 0.2, 0.25, 0.1)
    x, y, z, t = _mesh(shape, h)
    def quad(c):
        return (c[0] + c[1] * x + c[2] * y + c[3] * z + c[4] * t + c[5] * x * y + c[6] * y * z
                + c[7] * x * x + c[8] * z * z + c[9] * t * t + c[10] * x * t + c[11] * y * y)
    def grad(c):
        return dict(x=c[1] + c[5] * y + 2 * c[7] * x + c[10] * t, y=c[2] + c[5] * x + c[6] * z + 2 * c[11] * y,
                    z=c[3] + c[6] * y + 2 * c[8] * z, t=c[4] + 2 * c[9] * t + c[10] * x,
                    lap=2 * c[7] + 2 * c[8] + 2 * c[11])
    cs = [rng.standard_normal(12) for _ in range(4)]
    u, v, w, p = (quad(c) for c in cs)
    gu, gv, gw, gp = (grad(c) for c in cs)
    nu = 0.13
    R, loss, rows = oracle.fwd(W.NS_3D_T, [u, v, w, p], [], shape, h, (nu,))
    ex = [g["t"] + u * g["x"] + v * g["y"] + w * g["z"] + gp[a] - nu * g["lap"]
          for g, a in ((gu, "x"), (gv, "y"), (gw, "z"))]
    ex.append(gu["x"] + gv["y"] + gw["z"])
    inner = (slice(1, -1),) * 4
    assert rows == 6 * 7 * 5 * 4
    for r, e in zip(R, ex):
        assert np.allclose(r[inner], e[inner], rtol=0, atol=1e-10)
        assert np.all(r[..., 0] == 0) and np.all(r[..., -1] == 0)   # t = first/last: no row


def test_grayscott_quadratic_exact_away_from_wrap():
    shape, h = (7, 9), (0.2, 0.3)
    x, y = _mesh(shape, h)
    u = 1 + 0.3 * x - 0.2 * y + 0.5 * x * x + 0.1 * x * y - 0.4 * y * y
    v = 0.2 - 0.1 * x + 0.25 * y * y + 0.05 * x * x
    Du, Dv, F, k = 0.7, 0.3, 0.04, 0.06
    R, loss, rows = oracle.fwd(W.GRAYSCOTT_2D, [u, v], [], shape, h, (Du, Dv, F, k))
    eu = Du * (1.0 - 0.8) - u * v * v + F * (1 - u)
    ev = Dv * (0.5 + 0.1) + u * v * v - (F + k) * v
    inner = (slice(1, -1),) * 2
    assert rows == 63
    assert np.allclose(R[0][inner], eu[inner], atol=1e-11, rtol=0)
    assert np.allclose(R[1][inner], ev[inner], atol=1e-11, rtol=0)
    assert abs(loss[2] - (loss[0] + loss[1])) < 1e-15


# --------------------------------------------------------------------------------------------
# 2. closed forms on trigonometric fields (fp64 inputs, noise off)
# --------------------------------------------------------------------------------------------
def _m1(kappa, h):   # centred first difference of sin/cos(kappa x): derivative factor
    return math.sin(kappa * h) / h
def _m2(kappa, h):   # centred second difference: -m2 * f
    return 4.0 / (h * h) * math.sin(kappa * h / 2) ** 2


def test_poisson_trig_closed_form():
    n = 65
    h = 1.0 / (n - 1)
    x, y = _mesh((n, n), (h, h))
    us = np.sin(pi * x) * np.sin(pi * y)
    R, _, _ = oracle.fwd(W.POISSON_2D, [us], [2 * pi ** 2 * us], (n, n), (h, h), ())
    exact = (2 * _m2(pi, h) - 2 * pi ** 2) * us
    assert np.allclose(R[0][1:-1, 1:-1], exact[1:-1, 1:-1], rtol=0, atol=1e-9)


def test_helmholtz_trig_closed_form():
    n = 33
    h = 1.0 / (n - 1)
    x, y, z = _mesh((n,) * 3, (h,) * 3)
    us = np.sin(2 * pi * x) * np.sin(2 * pi * y) * np.sin(2 * pi * z)
    k = 4 * pi
    f = (k * k - 12 * pi * pi) * us
    R, _, _ = oracle.fwd(W.HELMHOLTZ_3D_O4, [us], [f], (n,) * 3, (h,) * 3, (k,))
    s4 = (-2 * math.cos(4 * pi * h) + 32 * math.cos(2 * pi * h) - 30) / (12 * h * h)
    exact = (3 * s4 + 12 * pi * pi) * us
    inner = (slice(2, -2),) * 3
    assert np.allclose(R[0][inner], exact[inner], rtol=0, atol=1e-8)
    assert np.abs(exact).max() > 1e-3      # the check is not vacuous at this resolution


def test_tgv_closed_form():
    shape = (16, 16, 12, 7)
    w = W.make("ns_tgv_128x16", shape=shape)
    hx, hy, hz, dt = w.spacing
    nu = w.coeffs[0]
    x, y, z, t = _mesh(shape, w.spacing)
    E2, E4 = np.exp(-2 * nu * t), np.exp(-4 * nu * t)
    u = np.sin(x) * np.cos(y) * np.cos(z) * E2
    v = -np.cos(x) * np.sin(y) * np.cos(z) * E2
    wv = np.zeros(shape)
    p = (np.cos(2 * x) + np.cos(2 * y)) * (np.cos(2 * z) + 2) / 16 * E4
    R, _, _ = oracle.fwd(W.NS_3D_T, [u, v, wv, p], [], shape, w.spacing, (nu,))
    dtf = -math.sinh(2 * nu * dt) / dt
    ux = np.cos(x) * np.cos(y) * np.cos(z) * E2 * _m1(1, hx)
    uy = -np.sin(x) * np.sin(y) * np.cos(z) * E2 * _m1(1, hy)
    vx = np.sin(x) * np.sin(y) * np.cos(z) * E2 * _m1(1, hx)
    vy = -np.cos(x) * np.cos(y) * np.cos(z) * E2 * _m1(1, hy)
    px = -np.sin(2 * x) * _m1(2, hx) * (np.cos(2 * z) + 2) / 16 * E4
    py = -np.sin(2 * y) * _m1(2, hy) * (np.cos(2 * z) + 2) / 16 * E4
    pz = -(np.cos(2 * x) + np.cos(2 * y)) * np.sin(2 * z) * _m1(2, hz) / 16 * E4
    lapf = -(_m2(1, hx) + _m2(1, hy) + _m2(1, hz))
    ex_u = dtf * u + u * ux + v * uy + px - nu * lapf * u
    ex_v = dtf * v + u * vx + v * vy + py - nu * lapf * v
    ex_w = pz
    ex_c = ux + vy
    tin = (Ellipsis, slice(1, -1))
    for r, e in zip(R, (ex_u, ex_v, ex_w, ex_c)):
        assert np.allclose(r[tin], e[tin], rtol=0, atol=1e-13)
    assert np.abs(R[3]).max() < 1e-13 and np.abs(ex_u).max() > 0.05


def test_burgers_trig_closed_form_interior():
    shape = (41, 23)
    w = W.make("burgers_256x128", shape=shape)
    hx, dt = w.spacing
    x, t = _mesh(shape, w.spacing, [-1.0, 0.0])
    u = -np.sin(pi * x) * np.exp(-t)
    nu = w.coeffs[0]
    R, _, _ = oracle.fwd(W.BURGERS_1D_T, [u], [], shape, w.spacing, (nu,))
    ut = -u * math.sinh(dt) / dt
    ux = -np.cos(pi * x) * np.exp(-t) * _m1(pi, hx)
    uxx = -_m2(pi, hx) * u
    exact = ut + u * ux - nu * uxx
    inner = (slice(1, -1),) * 2
    assert np.allclose(R[0][inner], exact[inner], rtol=0, atol=1e-12)


# --------------------------------------------------------------------------------------------
# 3. convergence order (noise-free analytic fields; Burgers/TGV against the continuous residual)
# --------------------------------------------------------------------------------------------
def _poisson_err(n):
    h = 1.0 / (n - 1)
    x, y = _mesh((n, n), (h, h))
    us = np.sin(pi * x) * np.sin(pi * y)
    R, _, _ = oracle.fwd(W.POISSON_2D, [us], [2 * pi ** 2 * us], (n, n), (h, h), ())
    return np.abs(R[0]).max()


def test_poisson_second_order():
    assert 3.9 < _poisson_err(33) / _poisson_err(65) < 4.1


def _helm_err(n):
    h = 1.0 / (n - 1)
    x, y, z = _mesh((n,) * 3, (h,) * 3)
    us = np.sin(2 * pi * x) * np.sin(2 * pi * y) * np.sin(2 * pi * z)
    k = 4 * pi
    R, _, _ = oracle.fwd(W.HELMHOLTZ_3D_O4, [us], [(k * k - 12 * pi * pi) * us], (n,) * 3, (h,) * 3, (k,))
    return np.abs(R[0]).max()


def test_helmholtz_fourth_order():
    r = _helm_err(33) / _helm_err(65)
    assert 14.0 < r < 17.0


def _burgers_err(nx, nt):
    w = W.make("burgers_256x128", shape=(nx, nt))
    x, t = _mesh((nx, nt), w.spacing, [-1.0, 0.0])
    u = -np.sin(pi * x) * np.exp(-t)
    nu = w.coeffs[0]
    R, _, _ = oracle.fwd(W.BURGERS_1D_T, [u], [], (nx, nt), w.spacing, (nu,))
    cont = -u + u * (-pi * np.cos(pi * x) * np.exp(-t)) - nu * (pi * pi * np.sin(pi * x) * np.exp(-t))
    e = np.abs(R[0] - cont)
    edge = max(e[0].max(), e[-1].max(), e[:, 0].max(), e[:, -1].max())
    return e[1:-1, 1:-1].max(), edge


def test_burgers_second_order_interior_and_edges():
    (i1, e1), (i2, e2) = _burgers_err(33, 17), _burgers_err(65, 33)
    assert 3.7 < i1 / i2 < 4.3
    assert 3.3 < e1 / e2 < 4.8       # the one-sided rows are second order too


def _tgv_err(n, nt):
    shape = (n, n, n, nt)
    w = W.make("ns_tgv_128x16", shape=shape)
    nu = w.coeffs[0]
    x, y, z, t = _mesh(shape, w.spacing)
    F, _ = W.analytic_fields(W.NS_3D_T, [np.arange(s) * h for s, h in zip(shape, w.spacing)], w.coeffs)
    R, _, _ = oracle.fwd(W.NS_3D_T, F, [], shape, w.spacing, (nu,))
    E2, E4 = np.exp(-2 * nu * t), np.exp(-4 * nu * t)
    u, v = F[0], F[1]
    ux = np.cos(x) * np.cos(y) * np.cos(z) * E2
    uy = -np.sin(x) * np.sin(y) * np.cos(z) * E2
    px = -2 * np.sin(2 * x) * (np.cos(2 * z) + 2) / 16 * E4
    cont = -2 * nu * u + u * ux + v * uy + px + 3 * nu * u
    return np.abs(R[0] - cont)[..., 1:-1].max()


def test_tgv_second_order():
    assert 3.8 < _tgv_err(16, 9) / _tgv_err(32, 17) < 4.2


# --------------------------------------------------------------------------------------------
# 4. adjoint identity, J du from the forward routine only
# --------------------------------------------------------------------------------------------
CASES = [
    (W.BURGERS_1D_T, (9, 7), (0.21, 0.13), (0.3,)),
    (W.POISSON_2D, (8, 9), (0.2, 0.3), ()),
    (W.GRAYSCOTT_2D, (6, 7), (0.2, 0.3), (0.7, 0.3, 0.04, 0.06)),
    (W.HELMHOLTZ_3D_O4, (8, 7, 9), (0.2, 0.3, 0.25), (1.3,)),
    (W.NS_3D_T, (5, 6, 5, 6), (0.3, 0.2, 0.25, 0.15), (0.13,)),
    (W.NS_2D_STEADY, (8, 9), (0.2, 0.3), (0.17,)),
    (W.NS_3D_STEADY, (6, 7, 5), (0.2, 0.3, 0.25), (0.17,)),
    (W.NS_3D_T_XSLAB, (6, 5, 4, 6), (0.3, 0.2, 0.25, 0.15), (0.13,)),
    (W.GRAYSCOTT_2D_XSLAB, (7, 6), (0.2, 0.3), (0.7, 0.3, 0.04, 0.06)),
]


def _rand_problem(op, shape):
    nf = len(W.OP_META[op]["fields"]); ns = len(W.OP_META[op]["sources"]); ne = len(W.OP_META[op]["residuals"])
    r = np.random.default_rng(zlib.crc32(op.encode()) % 1000 + 5)   # fixed per operator: the cases repeat run to run
    F = [r.standard_normal(shape) for _ in range(nf)]
    S = [r.standard_normal(shape) for _ in range(ns)]
    dF = [r.standard_normal(shape) for _ in range(nf)]
    Wt = [r.standard_normal(shape) for _ in range(ne)]
    return F, S, dF, Wt


def _jvp(op, F, S, dF, shape, h, c):
    """J dF from forward evaluations only.  Residuals are polynomials of degree <= 3 in the
    fields, so a two-step Richardson combination of central differences is exact."""
    def Rr(eps):
        return oracle.fwd(op, [f + eps * d for f, d in zip(F, dF)], S, shape, h, c)[0]
    D1 = [a - b for a, b in zip(Rr(1.0), Rr(-1.0))]
    D2 = [a - b for a, b in zip(Rr(0.5), Rr(-0.5))]
    return [(8 * d2 - d1) / 6 for d1, d2 in zip(D1, D2)]


@pytest.mark.parametrize("op,shape,h,c", CASES)
def test_adjoint_identity(op, shape, h, c):
    F, S, dF, Wt = _rand_problem(op, shape)
    Jd = _jvp(op, F, S, dF, shape, h, c)
    JtW = oracle.bwd(op, F, Wt, shape, h, c)
    rows_mask = [r != 0 for r in oracle.fwd(op, F, S, shape, h, c)[0]]
    lhs = sum(float(np.sum(j * w_)) for j, w_ in zip(Jd, Wt))      # J d vanishes off the rows
    rhs = sum(float(np.sum(d * g)) for d, g in zip(dF, JtW))
    assert abs(lhs - rhs) <= 1e-12 * max(abs(lhs), abs(rhs), 1.0) * 10
    assert abs(lhs) > 1e-3
    assert all(m.any() for m in rows_mask)


# --------------------------------------------------------------------------------------------
# 5. brute-force finite differences of the loss
# --------------------------------------------------------------------------------------------
TINY = [
    (W.BURGERS_1D_T, (7, 6), (0.21, 0.13), (0.3,)),
    (W.POISSON_2D, (7, 7), (0.2, 0.3), ()),
    (W.GRAYSCOTT_2D, (5, 6), (0.2, 0.3), (0.7, 0.3, 0.04, 0.06)),
    (W.HELMHOLTZ_3D_O4, (7, 6, 7), (0.2, 0.3, 0.25), (1.3,)),
    (W.NS_3D_T, (4, 5, 4, 5), (0.3, 0.2, 0.25, 0.15), (0.13,)),
    (W.NS_2D_STEADY, (6, 7), (0.2, 0.3), (0.17,)),
    (W.NS_3D_STEADY, (5, 4, 5), (0.2, 0.3, 0.25), (0.17,)),
    (W.NS_3D_T_XSLAB, (5, 4, 4, 5), (0.3, 0.2, 0.25, 0.15), (0.13,)),
    (W.GRAYSCOTT_2D_XSLAB, (6, 5), (0.2, 0.3), (0.7, 0.3, 0.04, 0.06)),
]


@pytest.mark.parametrize("op,shape,h,c", TINY)
def test_loss_gradient_brute_force(op, shape, h, c):
    F, S, _, _ = _rand_problem(op, shape)
    _, loss, g, rows = oracle.loss_and_grad(op, F, S, shape, h, c)
    eps = 1e-5
    gmax = max(np.abs(x).max() for x in g)
    worst = 0.0
    for fi in range(len(F)):
        flat = F[fi].reshape(-1)
        num = np.empty_like(flat)
        for k in range(flat.size):
            old = flat[k]
            flat[k] = old + eps
            lp = oracle.fwd(op, F, S, shape, h, c)[1][-1]
            flat[k] = old - eps
            lm = oracle.fwd(op, F, S, shape, h, c)[1][-1]
            flat[k] = old
            num[k] = (lp - lm) / (2 * eps)
        worst = max(worst, np.abs(num - g[fi].reshape(-1)).max() / gmax)
    assert worst < 2e-7, worst


# --------------------------------------------------------------------------------------------
# 6. the paper's printed u-adjoint (Eq. 1): steady 2-D Navier-Stokes
# --------------------------------------------------------------------------------------------
def test_ns_adjoint_reduces_to_printed_2d_equation():
    nx, ny, nz, nt = 7, 6, 4, 7
    dx, dy, dz, dt = 0.3, 0.2, 0.4, 0.1
    nu = 0.17
    r = np.random.default_rng(3)
    def ext(a2):    # constant in z and t
        return np.broadcast_to(a2[:, :, None, None], (nx, ny, nz, nt)).copy()
    u2, v2, p2 = (r.standard_normal((nx, ny)) for _ in range(3))
    Gu2, Gv2, Gd2 = (r.standard_normal((nx, ny)) for _ in range(3))
    Gw = r.standard_normal((nx, ny))
    F = [ext(u2), ext(v2), np.zeros((nx, ny, nz, nt)), ext(p2)]
    G = [ext(Gu2), ext(Gv2), ext(Gw), ext(Gd2)]
    g = oracle.bwd(W.NS_3D_T, F, G, (nx, ny, nz, nt), (dx, dy, dz, dt), (nu,))
    xm = lambda a: np.roll(a, 1, 0)     # value at i-1 (periodic)
    xp = lambda a: np.roll(a, -1, 0)
    ym = lambda a: np.roll(a, 1, 1)
    yp = lambda a: np.roll(a, -1, 1)
    u_x = (xp(u2) - xm(u2)) / (2 * dx)
    v_x = (xp(v2) - xm(v2)) / (2 * dx)
    printed = (Gu2 * (u_x + 2 * nu / dx ** 2 + 2 * nu / dy ** 2)
               + xm(Gu2) * (xm(u2) / (2 * dx) - nu / dx ** 2)
               + xp(Gu2) * (-xp(u2) / (2 * dx) - nu / dx ** 2)
               + ym(Gu2) * (ym(v2) / (2 * dy) - nu / dy ** 2)
               + yp(Gu2) * (-yp(v2) / (2 * dy) - nu / dy ** 2)
               + Gv2 * v_x
               + (xm(Gd2) - xp(Gd2)) / (2 * dx))
    # rows exist for t-index 1..nt-2; at t-index 2..nt-3 the t-terms of constant-in-t G cancel
    for k in range(nz):
        for m in range(2, nt - 2):
            assert np.allclose(g[0][:, :, k, m], printed, rtol=0, atol=1e-12)
    # and the pressure gradient is the transposed centred pressure derivatives
    gp = (xm(Gu2) - xp(Gu2)) / (2 * dx) + (ym(Gv2) - yp(Gv2)) / (2 * dy)
    assert np.allclose(g[3][:, :, 1, 3], gp, rtol=0, atol=1e-12)


def test_ns2d_steady_printed_u_adjoint_directly():
    """The operator the paper spells out: at nodes whose four neighbours all carry rows, the
    oracle's dL/du must be the printed Eq. (1) term by term (no reduction needed here)."""
    nx, ny, dx, dy, nu = 9, 8, 0.3, 0.2, 0.17
    r = np.random.default_rng(21)
    u, v, p = (r.standard_normal((nx, ny)) for _ in range(3))
    Gu, Gv, Gd = (r.standard_normal((nx, ny)) for _ in range(3))
    g = oracle.bwd(W.NS_2D_STEADY, [u, v, p], [Gu, Gv, Gd], (nx, ny), (dx, dy), (nu,))
    for i in range(2, nx - 2):
        for j in range(2, ny - 2):
            u_x = (u[i + 1, j] - u[i - 1, j]) / (2 * dx)
            v_x = (v[i + 1, j] - v[i - 1, j]) / (2 * dx)
            printed = (Gu[i, j] * (u_x + 2 * nu / dx ** 2 + 2 * nu / dy ** 2)
                       + Gu[i - 1, j] * (u[i - 1, j] / (2 * dx) - nu / dx ** 2)
                       + Gu[i + 1, j] * (-u[i + 1, j] / (2 * dx) - nu / dx ** 2)
                       + Gu[i, j - 1] * (v[i, j - 1] / (2 * dy) - nu / dy ** 2)
                       + Gu[i, j + 1] * (-v[i, j + 1] / (2 * dy) - nu / dy ** 2)
                       + Gv[i, j] * v_x
                       + (Gd[i - 1, j] - Gd[i + 1, j]) / (2 * dx))
            assert abs(g[0][i, j] - printed) < 1e-11
    # corner nodes of the ring are read by no row
    assert g[0][0, 0] == 0 and g[1][-1, -1] == 0 and g[2][0, -1] == 0


def test_ns3d_steady_reduces_to_printed_2d_equation_and_is_quadratic_exact():
    # (a) fields constant in z, w = 0: at nodes whose neighbours carry rows, dL/du is Eq. (1)
    nx, ny, nz, dx, dy, dz, nu = 8, 7, 6, 0.3, 0.2, 0.4, 0.17
    r = np.random.default_rng(5)
    ext = lambda a2: np.broadcast_to(a2[:, :, None], (nx, ny, nz)).copy()
    u2, v2, p2, Gu2, Gv2, Gw2, Gd2 = (r.standard_normal((nx, ny)) for _ in range(7))
    g = oracle.bwd(W.NS_3D_STEADY, [ext(u2), ext(v2), np.zeros((nx, ny, nz)), ext(p2)],
                   [ext(Gu2), ext(Gv2), ext(Gw2), ext(Gd2)], (nx, ny, nz), (dx, dy, dz), (nu,))
    for i in range(2, nx - 2):
        for j in range(2, ny - 2):
            u_x = (u2[i + 1, j] - u2[i - 1, j]) / (2 * dx)
            v_x = (v2[i + 1, j] - v2[i - 1, j]) / (2 * dx)
            printed = (Gu2[i, j] * (u_x + 2 * nu / dx ** 2 + 2 * nu / dy ** 2)
                       + Gu2[i - 1, j] * (u2[i - 1, j] / (2 * dx) - nu / dx ** 2)
                       + Gu2[i + 1, j] * (-u2[i + 1, j] / (2 * dx) - nu / dx ** 2)
                       + Gu2[i, j - 1] * (v2[i, j - 1] / (2 * dy) - nu / dy ** 2)
                       + Gu2[i, j + 1] * (-v2[i, j + 1] / (2 * dy) - nu / dy ** 2)
                       + Gv2[i, j] * v_x + (Gd2[i - 1, j] - Gd2[i + 1, j]) / (2 * dx))
            for k in range(2, nz - 2):      # z neighbours carry rows too: their terms cancel
                assert abs(g[0][i, j, k] - printed) < 1e-11
    # (b) quadratic fields: every centred difference is exact
    shape, h = (6, 5, 7), (0.25, 0.2, 0.3)
    x, y, z = _mesh(shape, h, [0.1, -0.3, 0.2])
    def quad(c):
        return c[0] + c[1] * x + c[2] * y + c[3] * z + c[4] * x * y + c[5] * y * z + c[6] * x * x + c[7] * y * y + c[8] * z * z
    def der(c):
        return dict(x=c[1] + c[4] * y + 2 * c[6] * x, y=c[2] + c[4] * x + c[5] * z + 2 * c[7] * y,
                    z=c[3] + c[5] * y + 2 * c[8] * z, lap=2 * (c[6] + c[7] + c[8]))
    cs = [np.random.default_rng(41 + k).standard_normal(9) for k in range(4)]
    u, v, w, p = (quad(c) for c in cs)
    du, dv, dw, dp = (der(c) for c in cs)
    R, loss, rows = oracle.fwd(W.NS_3D_STEADY, [u, v, w, p], [], shape, h, (0.23,))
    ex = [u * d["x"] + v * d["y"] + w * d["z"] + dp[a] - 0.23 * d["lap"] for d, a in ((du, "x"), (dv, "y"), (dw, "z"))]
    ex.append(du["x"] + dv["y"] + dw["z"])
    inner = (slice(1, -1),) * 3
    assert rows == 4 * 3 * 5
    for rr, e in zip(R, ex):
        assert np.allclose(rr[inner], e[inner], rtol=0, atol=1e-11)
        mask = np.ones(shape, bool); mask[inner] = False
        assert np.all(rr[mask] == 0.0)


def test_ns2d_steady_quadratic_exact():
    shape, h = (7, 8), (0.25, 0.2)
    x, y = _mesh(shape, h, [0.1, -0.3])
    def quad(c):
        return c[0] + c[1] * x + c[2] * y + c[3] * x * y + c[4] * x * x + c[5] * y * y
    def der(c):
        return dict(x=c[1] + c[3] * y + 2 * c[4] * x, y=c[2] + c[3] * x + 2 * c[5] * y, lap=2 * c[4] + 2 * c[5])
    cs = [np.random.default_rng(31 + k).standard_normal(6) for k in range(3)]
    u, v, p = (quad(c) for c in cs)
    du, dv, dp = (der(c) for c in cs)
    nu = 0.23
    R, loss, rows = oracle.fwd(W.NS_2D_STEADY, [u, v, p], [], shape, h, (nu,))
    ex = [u * du["x"] + v * du["y"] + dp["x"] - nu * du["lap"],
          u * dv["x"] + v * dv["y"] + dp["y"] - nu * dv["lap"],
          du["x"] + dv["y"]]
    inner = (slice(1, -1),) * 2
    assert rows == 5 * 6
    for rr, e in zip(R, ex):
        assert np.allclose(rr[inner], e[inner], rtol=0, atol=1e-11)
        mask = np.ones(shape, bool); mask[inner] = False
        assert np.all(rr[mask] == 0.0)
    assert abs(loss[3] - sum(np.sum(e[inner] ** 2) for e in ex) / rows) < 1e-10


# --------------------------------------------------------------------------------------------
# 7. special cases, symmetries, hand-worked fixtures
# --------------------------------------------------------------------------------------------
def test_grayscott_special_cases():
    shape, h, c = (6, 8), (0.2, 0.3), (0.7, 0.3, 0.04, 0.06)
    one, zero = np.ones(shape), np.zeros(shape)
    R, loss, _ = oracle.fwd(W.GRAYSCOTT_2D, [one, zero], [], shape, h, c)
    assert np.all(R[0] == 0) and np.all(R[1] == 0) and loss[2] == 0
    # D = 0: pointwise reaction terms only
    r = np.random.default_rng(8)
    u, v = r.standard_normal(shape), r.standard_normal(shape)
    R, _, _ = oracle.fwd(W.GRAYSCOTT_2D, [u, v], [], shape, h, (0.0, 0.0, 0.04, 0.06))
    assert np.allclose(R[0], -u * v * v + 0.04 * (1 - u), atol=1e-15)
    assert np.allclose(R[1], u * v * v - 0.1 * v, atol=1e-15)
    # periodic shift equivariance, wrap rows/columns included
    R0, _, _ = oracle.fwd(W.GRAYSCOTT_2D, [u, v], [], shape, h, c)
    R1, _, _ = oracle.fwd(W.GRAYSCOTT_2D, [np.roll(u, (2, 3), (0, 1)), np.roll(v, (2, 3), (0, 1))], [], shape, h, c)
    assert np.allclose(np.roll(R0[0], (2, 3), (0, 1)), R1[0], atol=1e-12)
    assert np.allclose(np.roll(R0[1], (2, 3), (0, 1)), R1[1], atol=1e-12)
    # wrap check against numpy's roll Laplacian (library routine as the definition of "periodic")
    lap = ((np.roll(u, 1, 0) - 2 * u + np.roll(u, -1, 0)) / h[0] ** 2
           + (np.roll(u, 1, 1) - 2 * u + np.roll(u, -1, 1)) / h[1] ** 2)
    assert np.allclose(R0[0], c[0] * lap - u * v * v + c[2] * (1 - u), atol=1e-11)


def test_ns_constant_flow_and_shift():
    shape, h = (5, 6, 4, 5), (0.3, 0.2, 0.25, 0.15)
    const = [np.full(shape, a) for a in (0.3, -1.2, 0.8, 2.0)]
    R, loss, _ = oracle.fwd(W.NS_3D_T, const, [], shape, h, (0.1,))
    assert all(np.abs(r).max() < 1e-14 for r in R)
    r = np.random.default_rng(5)
    F = [r.standard_normal(shape) for _ in range(4)]
    R0, _, _ = oracle.fwd(W.NS_3D_T, F, [], shape, h, (0.1,))
    sh = ((1, 2, 3), (0, 1, 2))
    R1, _, _ = oracle.fwd(W.NS_3D_T, [np.roll(f, *sh) for f in F], [], shape, h, (0.1,))
    for a, b in zip(R0, R1):
        assert np.allclose(np.roll(a, *sh), b, atol=1e-12)


def test_symmetric_linear_operators():
    """Poisson / Helmholtz: the Jacobian restricted to fields vanishing on the shell is
    symmetric, so <A a, b> = <a, A b>."""
    r = np.random.default_rng(11)
    shape, h = (8, 9), (0.2, 0.3)
    a, b = r.standard_normal(shape), r.standard_normal(shape)
    for q in (a, b):
        q[0] = q[-1] = 0; q[:, 0] = q[:, -1] = 0
    z = np.zeros(shape)
    Aa = oracle.fwd(W.POISSON_2D, [a], [z], shape, h, ())[0][0]
    Ab = oracle.fwd(W.POISSON_2D, [b], [z], shape, h, ())[0][0]
    assert abs(np.sum(Aa * b) - np.sum(a * Ab)) < 1e-10 * abs(np.sum(Aa * b))
    shape, h = (8, 9, 7), (0.2, 0.3, 0.25)
    a, b = r.standard_normal(shape), r.standard_normal(shape)
    for q in (a, b):
        q[:2] = q[-2:] = 0; q[:, :2] = q[:, -2:] = 0; q[:, :, :2] = q[:, :, -2:] = 0
    z = np.zeros(shape)
    Aa = oracle.fwd(W.HELMHOLTZ_3D_O4, [a], [z], shape, h, (1.1,))[0][0]
    Ab = oracle.fwd(W.HELMHOLTZ_3D_O4, [b], [z], shape, h, (1.1,))[0][0]
    assert abs(np.sum(Aa * b) - np.sum(a * Ab)) < 1e-10 * abs(np.sum(Aa * b))


def _read_fixture(name):
    """tests/golden/*.txt: '#' comment lines, then 'key: v v v ...' lines."""
    out = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", name)) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split(":", 1)
            out[k.strip()] = [float(t) for t in v.split()]
    return out


def test_hand_worked_poisson_3x3():
    fx = _read_fixture("poisson_3x3_hand.txt")
    u = np.array(fx["u"]).reshape(3, 3)
    f = np.array(fx["f"]).reshape(3, 3)
    R, loss, g, rows = oracle.loss_and_grad(W.POISSON_2D, [u], [f], (3, 3), fx["h"], ())
    assert rows == 1
    assert abs(R[0][1, 1] - fx["r_center"][0]) < 1e-12
    assert abs(loss[0] - fx["loss"][0]) < 1e-9
    assert np.allclose(g[0].reshape(-1), fx["grad"], atol=1e-9, rtol=0)


def test_hand_worked_burgers_corner_4x4():
    fx = _read_fixture("burgers_4x4_hand.txt")
    u = np.array(fx["u"]).reshape(4, 4)
    R, _, _ = oracle.fwd(W.BURGERS_1D_T, [u], [], (4, 4), fx["h"], fx["nu"])
    assert abs(R[0][0, 0] - fx["r_00"][0]) < 1e-12
    assert abs(R[0][3, 3] - fx["r_33"][0]) < 1e-12
    assert abs(R[0][1, 2] - fx["r_12"][0]) < 1e-12


def test_inputs_are_seeded_and_reproducible():
    a = W.make("poisson_1024", shape=(16, 20), seed=42)
    b = W.make("poisson_1024", shape=(16, 20), seed=42)
    c = W.make("poisson_1024", shape=(16, 20), seed=43)
    assert np.array_equal(a.fields[0], b.fields[0]) and not np.array_equal(a.fields[0], c.fields[0])
    z = W.normal01(42, 3, 200000)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1) < 0.01
    u = W.uniform01(42, 3, 200000)
    assert 0 < u.min() and u.max() < 1 and abs(u.mean() - 0.5) < 0.005
    # counter-based: a slice can be regenerated on its own
    assert np.array_equal(W.normal01(42, 3, 10, start=1000), z[1000:1010])


def test_ns3dt_xslab_is_the_periodic_operator_on_its_inner_planes():
    """The slab form (x not periodic, rows at x-index 1..n-2) against the periodic operator on
    the same array: identical residuals on the inner planes, none on the two outer ones; and for
    upstream arrays that vanish on the outer planes, the same adjoint at every node."""
    shape, h, c = (7, 5, 4, 6), (0.3, 0.2, 0.25, 0.15), (0.13,)
    r = np.random.default_rng(77)
    F = [r.standard_normal(shape) for _ in range(4)]
    Rp, _, rows_p = oracle.fwd(W.NS_3D_T, F, [], shape, h, c)
    Rs, _, rows_s = oracle.fwd(W.NS_3D_T_XSLAB, F, [], shape, h, c)
    assert rows_p == 7 * 5 * 4 * 4 and rows_s == 5 * 5 * 4 * 4
    for a, b in zip(Rp, Rs):
        assert np.array_equal(a[1:-1], b[1:-1])
        assert np.all(b[0] == 0.0) and np.all(b[-1] == 0.0)
        assert np.any(a[0] != 0.0)
    G = [r.standard_normal(shape) for _ in range(4)]
    G0 = [g.copy() for g in G]
    for g in G0:
        g[0] = 0.0; g[-1] = 0.0
    gs = oracle.bwd(W.NS_3D_T_XSLAB, F, G, shape, h, c)          # outer planes of G are ignored
    gp = oracle.bwd(W.NS_3D_T, F, G0, shape, h, c)
    for a, b in zip(gs, gp):
        assert np.allclose(a, b, rtol=0, atol=1e-12)


def test_grayscott_xslab_is_the_periodic_operator_on_its_inner_rows():
    shape, h, c = (7, 8), (0.2, 0.3), (0.7, 0.3, 0.04, 0.06)
    r = np.random.default_rng(78)
    F = [r.standard_normal(shape) for _ in range(2)]
    Rp, _, rows_p = oracle.fwd(W.GRAYSCOTT_2D, F, [], shape, h, c)
    Rs, _, rows_s = oracle.fwd(W.GRAYSCOTT_2D_XSLAB, F, [], shape, h, c)
    assert rows_p == 56 and rows_s == 40
    for a, b in zip(Rp, Rs):
        assert np.array_equal(a[1:-1], b[1:-1]) and np.all(b[0] == 0.0) and np.all(b[-1] == 0.0)
    G = [r.standard_normal(shape) for _ in range(2)]
    G0 = [g.copy() for g in G]
    for g in G0:
        g[0] = 0.0; g[-1] = 0.0
    gs = oracle.bwd(W.GRAYSCOTT_2D_XSLAB, F, G, shape, h, c)
    gp = oracle.bwd(W.GRAYSCOTT_2D, F, G0, shape, h, c)
    for a, b in zip(gs, gp):
        assert np.allclose(a, b, rtol=0, atol=1e-12)
