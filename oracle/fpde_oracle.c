/*
 * fpde_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, fp64 CPU statement of what the fused finite-difference PDE-residual operators
 * compute: every residual row from its definition, the mean-square residual loss, and the
 * gradient dL/du by SCATTER (for every residual row, for every node that row reads, add
 * G(row) * d r(row) / d u(node)).  No tiling, no fusion, no gather-form adjoint, no sharing of
 * code, tables or constants with the CUDA library.  Only tests, the smoke check and the bench's
 * CPU-baseline leg may call it.
 *
 * What is computed follows the paper's Section 2.1 (residuals assembled from centred finite
 * differences of grid-aligned fields), Section 2.2 and Appendix A.3 (the gradient is the action
 * of the transposed discrete Jacobian on the upstream sensitivities G = dL/dres), and Appendix
 * A.5 (near-boundary rows differ because of prescribed values, one-sided formulas or omitted
 * neighbours).  The paper spells out only the steady 2-D Navier-Stokes operator; the other row
 * definitions used here are the readings listed in this repository's design notes.
 *
 * Conventions
 *   - arrays are row-major, axis 0 slowest, last axis contiguous; every array has the full
 *     grid shape; residuals are 0 at nodes that carry no row.
 *   - 1-D difference formulas are produced as explicit (index, weight) lists by d1(), d2() and
 *     d2_o4(); the forward pass applies a list, the backward pass scatters through the same
 *     list, so a transposition can only go wrong in one visible place.
 *   - loss: L_e = (1/N_r) * sum over rows of r_e^2,  L = sum_e L_e,  N_r = number of rows.
 *
 * Every function here is pinned by tests/test_oracle_pins.py (polynomial exactness, closed
 * forms on trigonometric fields, convergence order, <J du, w> = <du, J^T w>, brute-force
 * finite differences of the loss, and the paper's printed u-adjoint, Eq. (1)).
 */
#include <stddef.h>
#include <string.h>

typedef long long i64;

enum { OP_BURGERS_1D_T = 0, OP_POISSON_2D = 1, OP_GRAYSCOTT_2D = 2, OP_HELMHOLTZ_3D_O4 = 3,
       OP_NS_3D_T = 4, OP_NS_2D_STEADY = 5, OP_NS_3D_STEADY = 6, OP_NS_3D_T_XSLAB = 7,
       OP_GRAYSCOTT_2D_XSLAB = 8,
       OP_COUNT = 9 };
enum { BC_PERIODIC = 0, BC_INTERIOR = 1, BC_ONE_SIDED = 2 };

/* A 1-D difference formula at one node: value = sum_k w[k] * q[idx[k]] along one axis. */
typedef struct { int n; i64 idx[6]; double w[6]; } stencil;

static i64 wrap(i64 i, i64 n) { return ((i % n) + n) % n; }

/* First derivative, second order (Appendix A.3 centred formula q_x = (q[i+1]-q[i-1])/(2h);
 * one-sided rows: (-3,4,-1)/(2h) and (3,-4,1)/(2h)).  Returns 0 where the axis carries no row. */
static int d1(int bc, i64 i, i64 n, double h, stencil* s) {
    double c = 1.0 / (2.0 * h);
    if (bc == BC_PERIODIC) {
        s->n = 2; s->idx[0] = wrap(i + 1, n); s->w[0] = c; s->idx[1] = wrap(i - 1, n); s->w[1] = -c;
        return 1;
    }
    if (i >= 1 && i <= n - 2) {
        s->n = 2; s->idx[0] = i + 1; s->w[0] = c; s->idx[1] = i - 1; s->w[1] = -c;
        return 1;
    }
    if (bc == BC_INTERIOR) return 0;
    s->n = 3;
    if (i == 0) {
        s->idx[0] = 0; s->w[0] = -3.0 * c; s->idx[1] = 1; s->w[1] = 4.0 * c; s->idx[2] = 2; s->w[2] = -c;
    } else {
        s->idx[0] = n - 1; s->w[0] = 3.0 * c; s->idx[1] = n - 2; s->w[1] = -4.0 * c; s->idx[2] = n - 3; s->w[2] = c;
    }
    return 1;
}

/* Second derivative, second order (Appendix A.3: q_xx = (q[i+1]-2q[i]+q[i-1])/h^2; one-sided
 * rows use the four-point second-order formula (2,-5,4,-1)/h^2). */
static int d2(int bc, i64 i, i64 n, double h, stencil* s) {
    double c = 1.0 / (h * h);
    if (bc == BC_PERIODIC || (i >= 1 && i <= n - 2)) {
        i64 ip = i + 1, im = i - 1;
        if (bc == BC_PERIODIC) { ip = wrap(ip, n); im = wrap(im, n); }
        s->n = 3; s->idx[0] = ip; s->w[0] = c; s->idx[1] = i; s->w[1] = -2.0 * c; s->idx[2] = im; s->w[2] = c;
        return 1;
    }
    if (bc == BC_INTERIOR) return 0;
    s->n = 4;
    {
        i64 dir = (i == 0) ? 1 : -1;
        s->idx[0] = i;           s->w[0] = 2.0 * c;
        s->idx[1] = i + dir;     s->w[1] = -5.0 * c;
        s->idx[2] = i + 2 * dir; s->w[2] = 4.0 * c;
        s->idx[3] = i + 3 * dir; s->w[3] = -c;
    }
    return 1;
}

/* Second derivative, fourth order, five points: (-1,16,-30,16,-1)/(12 h^2). */
static int d2_o4(int bc, i64 i, i64 n, double h, stencil* s) {
    double c = 1.0 / (12.0 * h * h);
    static const double wt[5] = { -1.0, 16.0, -30.0, 16.0, -1.0 };
    int k;
    if (bc == BC_ONE_SIDED) return 0;
    if (bc == BC_INTERIOR && (i < 2 || i > n - 3)) return 0;
    s->n = 5;
    for (k = 0; k < 5; ++k) {
        i64 j = i + (k - 2);
        s->idx[k] = (bc == BC_PERIODIC) ? wrap(j, n) : j;
        s->w[k] = wt[k] * c;
    }
    return 1;
}

/* value of a 1-D formula applied along an axis: q points at the start of the 1-D line,
 * stride is that axis' stride in elements */
static double apply(const stencil* s, const double* line, i64 stride) {
    double v = 0.0; int k;
    for (k = 0; k < s->n; ++k) v += s->w[k] * line[s->idx[k] * stride];
    return v;
}
/* scatter: line[idx[k]] += a * w[k] */
static void scatter(const stencil* s, double* line, i64 stride, double a) {
    int k;
    for (k = 0; k < s->n; ++k) line[s->idx[k] * stride] += a * s->w[k];
}

static const int OP_NDIM[OP_COUNT] = { 2, 2, 2, 3, 4, 2, 3, 4, 2 };
static const int OP_NF[OP_COUNT] = { 1, 1, 2, 1, 4, 3, 4, 4, 2 };
static const int OP_NS[OP_COUNT] = { 0, 1, 0, 1, 0, 0, 0, 0, 0 };
static const int OP_NE[OP_COUNT] = { 1, 1, 2, 1, 4, 3, 4, 4, 2 };
static const int OP_NC[OP_COUNT] = { 1, 0, 4, 1, 1, 1, 1, 1, 4 };
static const int OP_BC[OP_COUNT][4] = {
    { BC_ONE_SIDED, BC_ONE_SIDED, 0, 0 },
    { BC_INTERIOR, BC_INTERIOR, 0, 0 },
    { BC_PERIODIC, BC_PERIODIC, 0, 0 },
    { BC_INTERIOR, BC_INTERIOR, BC_INTERIOR, 0 },
    { BC_PERIODIC, BC_PERIODIC, BC_PERIODIC, BC_INTERIOR },
    { BC_INTERIOR, BC_INTERIOR, 0, 0 },
    { BC_INTERIOR, BC_INTERIOR, BC_INTERIOR, 0 },
    { BC_INTERIOR, BC_PERIODIC, BC_PERIODIC, BC_INTERIOR },
    { BC_INTERIOR, BC_PERIODIC, 0, 0 },
};

int fpde_oracle_info(int op, int* ndim, int* nf, int* ns, int* ne, int* nc) {
    if (op < 0 || op >= OP_COUNT) return 1;
    *ndim = OP_NDIM[op]; *nf = OP_NF[op]; *ns = OP_NS[op]; *ne = OP_NE[op]; *nc = OP_NC[op];
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * One routine per operator visits every node; mode 0 = forward (write residuals, count rows),
 * mode 1 = backward (scatter G through the row's partial derivatives into the gradients).
 * ---------------------------------------------------------------------------------------- */

/* Viscous Burgers on an (x,t) array: r = D_t u + u * D_x u - nu * D_xx u at EVERY node, with
 * centred formulas inside and one-sided second-order formulas on the first/last node of each
 * axis (per axis: an x-edge node with interior t uses one-sided x and centred t). */
static i64 burgers(int mode, const double* u, double* r, const double* G, double* g,
                   const i64* n, const double* h, const double* c) {
    i64 nx = n[0], nt = n[1], i, j, rows = 0;
    double nu = c[0];
    for (i = 0; i < nx; ++i) for (j = 0; j < nt; ++j) {
        stencil sx, sxx, st;
        i64 p = i * nt + j;
        double ux, uxx, ut;
        if (!d1(BC_ONE_SIDED, i, nx, h[0], &sx)) continue;
        if (!d2(BC_ONE_SIDED, i, nx, h[0], &sxx)) continue;
        if (!d1(BC_ONE_SIDED, j, nt, h[1], &st)) continue;
        ++rows;
        ux = apply(&sx, u + j, nt);          /* line along x through column j */
        uxx = apply(&sxx, u + j, nt);
        ut = apply(&st, u + i * nt, 1);      /* line along t through row i    */
        if (mode == 0) {
            r[p] = ut + u[p] * ux - nu * uxx;
        } else {
            double Gp = G[p];
            scatter(&st, g + i * nt, 1, Gp);            /* d r / d u through D_t        */
            g[p] += Gp * ux;                            /* the factor u in u * D_x u    */
            scatter(&sx, g + j, nt, Gp * u[p]);         /* D_x u inside u * D_x u       */
            scatter(&sxx, g + j, nt, -Gp * nu);         /* -nu * D_xx u                 */
        }
    }
    return rows;
}

/* 2-D Poisson: r = -(d_xx u + d_yy u) - f on nodes where both centred formulas fit. */
static i64 poisson(int mode, const double* u, const double* f, double* r, const double* G, double* g,
                   const i64* n, const double* h) {
    i64 nx = n[0], ny = n[1], i, j, rows = 0;
    for (i = 0; i < nx; ++i) for (j = 0; j < ny; ++j) {
        stencil sx, sy;
        i64 p = i * ny + j;
        if (!d2(BC_INTERIOR, i, nx, h[0], &sx)) continue;
        if (!d2(BC_INTERIOR, j, ny, h[1], &sy)) continue;
        ++rows;
        if (mode == 0) {
            r[p] = -(apply(&sx, u + j, ny) + apply(&sy, u + i * ny, 1)) - f[p];
        } else {
            scatter(&sx, g + j, ny, -G[p]);
            scatter(&sy, g + i * ny, 1, -G[p]);
        }
    }
    return rows;
}

/* Two-field steady Gray-Scott, periodic: r_u = Du*Lap u - u v^2 + F (1-u),
 * r_v = Dv*Lap v + u v^2 - (F+k) v, Lap = d_xx + d_yy (five points). */
static i64 grayscott(int mode, const double* u, const double* v, double* ru, double* rv,
                     const double* Gu, const double* Gv, double* gu, double* gv,
                     const i64* n, const double* h, const double* c, int bcx) {
    i64 nx = n[0], ny = n[1], i, j, rows = 0;
    double Du = c[0], Dv = c[1], F = c[2], k = c[3];
    for (i = 0; i < nx; ++i) for (j = 0; j < ny; ++j) {
        stencil sx, sy;
        i64 p = i * ny + j;
        if (!d2(bcx, i, nx, h[0], &sx)) continue;    /* bcx = BC_INTERIOR: the slab form, rows at x-index 1..nx-2 */
        d2(BC_PERIODIC, j, ny, h[1], &sy);
        ++rows;
        if (mode == 0) {
            double lu = apply(&sx, u + j, ny) + apply(&sy, u + i * ny, 1);
            double lv = apply(&sx, v + j, ny) + apply(&sy, v + i * ny, 1);
            ru[p] = Du * lu - u[p] * v[p] * v[p] + F * (1.0 - u[p]);
            rv[p] = Dv * lv + u[p] * v[p] * v[p] - (F + k) * v[p];
        } else {
            double a = Gu[p], b = Gv[p];
            /* row r_u */
            scatter(&sx, gu + j, ny, a * Du);
            scatter(&sy, gu + i * ny, 1, a * Du);
            gu[p] += a * (-v[p] * v[p] - F);
            gv[p] += a * (-2.0 * u[p] * v[p]);
            /* row r_v */
            scatter(&sx, gv + j, ny, b * Dv);
            scatter(&sy, gv + i * ny, 1, b * Dv);
            gu[p] += b * (v[p] * v[p]);
            gv[p] += b * (2.0 * u[p] * v[p] - (F + k));
        }
    }
    return rows;
}

/* 3-D Helmholtz, fourth order: r = sum_a d_aa^(4) u + k^2 u - f on nodes where the 13-point
 * star fits (indices 2 .. n-3 on every axis). */
static i64 helmholtz(int mode, const double* u, const double* f, double* r, const double* G, double* g,
                     const i64* n, const double* h, const double* c) {
    i64 nx = n[0], ny = n[1], nz = n[2], i, j, l, rows = 0;
    double k2 = c[0] * c[0];
    for (i = 0; i < nx; ++i) for (j = 0; j < ny; ++j) for (l = 0; l < nz; ++l) {
        stencil sx, sy, sz;
        i64 p = (i * ny + j) * nz + l;
        if (!d2_o4(BC_INTERIOR, i, nx, h[0], &sx)) continue;
        if (!d2_o4(BC_INTERIOR, j, ny, h[1], &sy)) continue;
        if (!d2_o4(BC_INTERIOR, l, nz, h[2], &sz)) continue;
        ++rows;
        if (mode == 0) {
            r[p] = apply(&sx, u + j * nz + l, ny * nz) + apply(&sy, u + i * ny * nz + l, nz)
                 + apply(&sz, u + (i * ny + j) * nz, 1) + k2 * u[p] - f[p];
        } else {
            scatter(&sx, g + j * nz + l, ny * nz, G[p]);
            scatter(&sy, g + i * ny * nz + l, nz, G[p]);
            scatter(&sz, g + (i * ny + j) * nz, 1, G[p]);
            g[p] += G[p] * k2;
        }
    }
    return rows;
}

/* Unsteady incompressible Navier-Stokes on an (x,y,z,t) array, space periodic, rows at the
 * interior t nodes.  With bcx = BC_INTERIOR the x axis is not periodic: rows only where the
 * centred x formulas fit (x-index 1..n_x-2), the first and last x-plane are data.  That is the
 * form one slab of a grid split along x takes (its outer planes are copies of the neighbours'
 * planes), and on the planes that carry rows it is the same formula.  Section 2.1's residuals extended by d_t, w and d_z:
 *   mom_q = d_t q + u d_x q + v d_y q + w d_z q + d_{a_q} p - nu (d_xx+d_yy+d_zz) q, q in (u,v,w),
 *           a_u = x, a_v = y, a_w = z;
 *   cont  = d_x u + d_y v + d_z w.
 * fld = {u,v,w,p}; res / G / grd index: 0..2 momentum x,y,z, 3 continuity. */
static i64 ns3dt(int mode, const double* const* fld, double* const* res, const double* const* G,
                 double* const* grd, const i64* n, const double* h, const double* c, int bcx) {
    i64 i[4], rows = 0;
    i64 st[4];
    double nu = c[0];
    st[3] = 1; st[2] = n[3]; st[1] = n[2] * n[3]; st[0] = n[1] * n[2] * n[3];
    for (i[0] = 0; i[0] < n[0]; ++i[0]) for (i[1] = 0; i[1] < n[1]; ++i[1])
    for (i[2] = 0; i[2] < n[2]; ++i[2]) for (i[3] = 0; i[3] < n[3]; ++i[3]) {
        stencil s1[3], s2[3], stt;
        i64 p = i[0] * st[0] + i[1] * st[1] + i[2] * st[2] + i[3];
        i64 base[4];     /* offset of the start of the 1-D line through p along each axis */
        double vel[3], dq[3][3], lap[3], dt[3], dp[3];
        int a, q;
        if (!d1(BC_INTERIOR, i[3], n[3], h[3], &stt)) continue;
        if (!d1(bcx, i[0], n[0], h[0], &s1[0])) continue;
        d2(bcx, i[0], n[0], h[0], &s2[0]);
        for (a = 1; a < 3; ++a) {
            d1(BC_PERIODIC, i[a], n[a], h[a], &s1[a]);
            d2(BC_PERIODIC, i[a], n[a], h[a], &s2[a]);
        }
        for (a = 0; a < 4; ++a) base[a] = p - i[a] * st[a];
        ++rows;
        for (q = 0; q < 3; ++q) {
            vel[q] = fld[q][p];
            lap[q] = 0.0;
            for (a = 0; a < 3; ++a) {
                dq[q][a] = apply(&s1[a], fld[q] + base[a], st[a]);      /* d_a q   */
                lap[q] += apply(&s2[a], fld[q] + base[a], st[a]);       /* d_aa q  */
            }
            dt[q] = apply(&stt, fld[q] + base[3], 1);                   /* d_t q   */
            dp[q] = apply(&s1[q], fld[3] + base[q], st[q]);             /* d_{a_q} p */
        }
        if (mode == 0) {
            for (q = 0; q < 3; ++q)
                res[q][p] = dt[q] + vel[0] * dq[q][0] + vel[1] * dq[q][1] + vel[2] * dq[q][2]
                          + dp[q] - nu * lap[q];
            res[3][p] = dq[0][0] + dq[1][1] + dq[2][2];
        } else {
            for (q = 0; q < 3; ++q) {
                double Gq = G[q][p];
                scatter(&stt, grd[q] + base[3], 1, Gq);                          /* d_t q            */
                for (a = 0; a < 3; ++a) {
                    grd[a][p] += Gq * dq[q][a];                                  /* factor c_a       */
                    scatter(&s1[a], grd[q] + base[a], st[a], Gq * vel[a]);       /* c_a * d_a q      */
                    scatter(&s2[a], grd[q] + base[a], st[a], -Gq * nu);          /* -nu d_aa q       */
                }
                scatter(&s1[q], grd[3] + base[q], st[q], Gq);                    /* d_{a_q} p        */
            }
            for (a = 0; a < 3; ++a)
                scatter(&s1[a], grd[a] + base[a], st[a], G[3][p]);               /* continuity row   */
        }
    }
    return rows;
}

/* Steady incompressible Navier-Stokes on an (x,y) array, exactly the paper's Section 2.1 system:
 *   res_u = u u_x + v u_y + p_x - nu (u_xx + u_yy),  res_v = u v_x + v v_y + p_y - nu (v_xx + v_yy),
 *   res_div = u_x + v_y,
 * centred differences (Appendix A.3), rows at the nodes where they fit (interior points); the
 * outer ring is data.  fld = {u,v,p}; res / G / grd index: 0 res_u, 1 res_v, 2 res_div. */
static i64 ns2d(int mode, const double* const* fld, double* const* res, const double* const* G,
                double* const* grd, const i64* n, const double* h, const double* c) {
    i64 nx = n[0], ny = n[1], i, j, rows = 0;
    double nu = c[0];
    for (i = 0; i < nx; ++i) for (j = 0; j < ny; ++j) {
        stencil s1x, s1y, s2x, s2y;
        i64 p = i * ny + j;
        double vel[2], dq[2][2], lap[2], dp[2];
        int q;
        if (!d1(BC_INTERIOR, i, nx, h[0], &s1x) || !d1(BC_INTERIOR, j, ny, h[1], &s1y)) continue;
        d2(BC_INTERIOR, i, nx, h[0], &s2x); d2(BC_INTERIOR, j, ny, h[1], &s2y);
        ++rows;
        for (q = 0; q < 2; ++q) {
            vel[q] = fld[q][p];
            dq[q][0] = apply(&s1x, fld[q] + j, ny);          /* d_x q  */
            dq[q][1] = apply(&s1y, fld[q] + i * ny, 1);      /* d_y q  */
            lap[q] = apply(&s2x, fld[q] + j, ny) + apply(&s2y, fld[q] + i * ny, 1);
        }
        dp[0] = apply(&s1x, fld[2] + j, ny);
        dp[1] = apply(&s1y, fld[2] + i * ny, 1);
        if (mode == 0) {
            for (q = 0; q < 2; ++q)
                res[q][p] = vel[0] * dq[q][0] + vel[1] * dq[q][1] + dp[q] - nu * lap[q];
            res[2][p] = dq[0][0] + dq[1][1];
        } else {
            for (q = 0; q < 2; ++q) {
                double Gq = G[q][p];
                grd[0][p] += Gq * dq[q][0];                                  /* factor u in u d_x q */
                grd[1][p] += Gq * dq[q][1];                                  /* factor v in v d_y q */
                scatter(&s1x, grd[q] + j, ny, Gq * vel[0]);                  /* u * d_x q           */
                scatter(&s1y, grd[q] + i * ny, 1, Gq * vel[1]);              /* v * d_y q           */
                scatter(&s2x, grd[q] + j, ny, -Gq * nu);                     /* -nu d_xx q          */
                scatter(&s2y, grd[q] + i * ny, 1, -Gq * nu);                 /* -nu d_yy q          */
            }
            scatter(&s1x, grd[2] + j, ny, G[0][p]);                          /* p_x in res_u        */
            scatter(&s1y, grd[2] + i * ny, 1, G[1][p]);                      /* p_y in res_v        */
            scatter(&s1x, grd[0] + j, ny, G[2][p]);                          /* u_x in res_div      */
            scatter(&s1y, grd[1] + i * ny, 1, G[2][p]);                      /* v_y in res_div      */
        }
    }
    return rows;
}

/* Steady incompressible Navier-Stokes on an (x,y,z) array: Section 2.1's system with w and d_z
 * added (the paper's 3-D steady operator), centred differences, rows at the interior nodes:
 *   mom_q = u d_x q + v d_y q + w d_z q + d_{a_q} p - nu (d_xx + d_yy + d_zz) q,  q in (u,v,w),
 *   cont  = d_x u + d_y v + d_z w.
 * fld = {u,v,w,p}; res / G / grd index: 0..2 momentum x,y,z, 3 continuity. */
static i64 ns3d(int mode, const double* const* fld, double* const* res, const double* const* G,
                double* const* grd, const i64* n, const double* h, const double* c) {
    i64 i[3], rows = 0, st[3];
    double nu = c[0];
    st[2] = 1; st[1] = n[2]; st[0] = n[1] * n[2];
    for (i[0] = 0; i[0] < n[0]; ++i[0]) for (i[1] = 0; i[1] < n[1]; ++i[1]) for (i[2] = 0; i[2] < n[2]; ++i[2]) {
        stencil s1[3], s2[3];
        i64 p = i[0] * st[0] + i[1] * st[1] + i[2];
        i64 base[3];
        double vel[3], dq[3][3], lap[3], dp[3];
        int a, q, ok = 1;
        for (a = 0; a < 3; ++a) {
            if (!d1(BC_INTERIOR, i[a], n[a], h[a], &s1[a])) ok = 0;
            else d2(BC_INTERIOR, i[a], n[a], h[a], &s2[a]);
        }
        if (!ok) continue;
        for (a = 0; a < 3; ++a) base[a] = p - i[a] * st[a];
        ++rows;
        for (q = 0; q < 3; ++q) {
            vel[q] = fld[q][p];
            lap[q] = 0.0;
            for (a = 0; a < 3; ++a) {
                dq[q][a] = apply(&s1[a], fld[q] + base[a], st[a]);
                lap[q] += apply(&s2[a], fld[q] + base[a], st[a]);
            }
            dp[q] = apply(&s1[q], fld[3] + base[q], st[q]);
        }
        if (mode == 0) {
            for (q = 0; q < 3; ++q)
                res[q][p] = vel[0] * dq[q][0] + vel[1] * dq[q][1] + vel[2] * dq[q][2] + dp[q] - nu * lap[q];
            res[3][p] = dq[0][0] + dq[1][1] + dq[2][2];
        } else {
            for (q = 0; q < 3; ++q) {
                double Gq = G[q][p];
                for (a = 0; a < 3; ++a) {
                    grd[a][p] += Gq * dq[q][a];                                  /* factor c_a       */
                    scatter(&s1[a], grd[q] + base[a], st[a], Gq * vel[a]);       /* c_a * d_a q      */
                    scatter(&s2[a], grd[q] + base[a], st[a], -Gq * nu);          /* -nu d_aa q       */
                }
                scatter(&s1[q], grd[3] + base[q], st[q], Gq);                    /* d_{a_q} p        */
            }
            for (a = 0; a < 3; ++a)
                scatter(&s1[a], grd[a] + base[a], st[a], G[3][p]);               /* continuity row   */
        }
    }
    return rows;
}

static i64 total(int ndim, const i64* n) { i64 N = 1; int a; for (a = 0; a < ndim; ++a) N *= n[a]; return N; }

static int check(int op, int ndim, const i64* n) {
    int a;
    if (op < 0 || op >= OP_COUNT) return 1;
    if (ndim != OP_NDIM[op]) return 2;
    for (a = 0; a < ndim; ++a) {
        int bc = OP_BC[op][a];
        i64 need = (bc == BC_ONE_SIDED) ? 4 : (op == OP_HELMHOLTZ_3D_O4 ? 5 : 3);
        if (n[a] < need) return 3;
    }
    return 0;
}

/* Forward: residual arrays (zero at nodes without a row) and loss[0..E-1] = L_e, loss[E] = L.
 * Returns the number of rows, or a negative error. */
i64 fpde_oracle_fwd(int op, const double* const* fields, const double* const* sources,
                    double* const* residuals, double* loss, int ndim, const i64* shape,
                    const double* spacing, const double* coeffs) {
    i64 N, rows = 0, p; int e, E;
    if (check(op, ndim, shape)) return -(i64)check(op, ndim, shape);
    N = total(ndim, shape); E = OP_NE[op];
    for (e = 0; e < E; ++e) memset(residuals[e], 0, (size_t)N * sizeof(double));
    switch (op) {
    case OP_BURGERS_1D_T: rows = burgers(0, fields[0], residuals[0], NULL, NULL, shape, spacing, coeffs); break;
    case OP_POISSON_2D: rows = poisson(0, fields[0], sources[0], residuals[0], NULL, NULL, shape, spacing); break;
    case OP_GRAYSCOTT_2D: rows = grayscott(0, fields[0], fields[1], residuals[0], residuals[1], NULL, NULL, NULL, NULL, shape, spacing, coeffs, BC_PERIODIC); break;
    case OP_GRAYSCOTT_2D_XSLAB: rows = grayscott(0, fields[0], fields[1], residuals[0], residuals[1], NULL, NULL, NULL, NULL, shape, spacing, coeffs, BC_INTERIOR); break;
    case OP_HELMHOLTZ_3D_O4: rows = helmholtz(0, fields[0], sources[0], residuals[0], NULL, NULL, shape, spacing, coeffs); break;
    case OP_NS_3D_T: rows = ns3dt(0, fields, residuals, NULL, NULL, shape, spacing, coeffs, BC_PERIODIC); break;
    case OP_NS_3D_T_XSLAB: rows = ns3dt(0, fields, residuals, NULL, NULL, shape, spacing, coeffs, BC_INTERIOR); break;
    case OP_NS_2D_STEADY: rows = ns2d(0, fields, residuals, NULL, NULL, shape, spacing, coeffs); break;
    case OP_NS_3D_STEADY: rows = ns3d(0, fields, residuals, NULL, NULL, shape, spacing, coeffs); break;
    }
    if (loss) {
        loss[E] = 0.0;
        for (e = 0; e < E; ++e) {
            double s = 0.0;
            for (p = 0; p < N; ++p) s += residuals[e][p] * residuals[e][p];   /* non-row nodes hold 0 */
            loss[e] = s / (double)rows;
            loss[E] += loss[e];
        }
    }
    return rows;
}

/* Backward: gfields = J^T G by scatter.  G[e] are the upstream sensitivities dL/dr_e (full
 * grid shape; entries at nodes without a row are never read). */
i64 fpde_oracle_bwd(int op, const double* const* fields, const double* const* G,
                    double* const* gfields, int ndim, const i64* shape,
                    const double* spacing, const double* coeffs) {
    i64 N, rows = 0; int f;
    if (check(op, ndim, shape)) return -(i64)check(op, ndim, shape);
    N = total(ndim, shape);
    for (f = 0; f < OP_NF[op]; ++f) memset(gfields[f], 0, (size_t)N * sizeof(double));
    switch (op) {
    case OP_BURGERS_1D_T: rows = burgers(1, fields[0], NULL, G[0], gfields[0], shape, spacing, coeffs); break;
    case OP_POISSON_2D: rows = poisson(1, fields[0], NULL, NULL, G[0], gfields[0], shape, spacing); break;
    case OP_GRAYSCOTT_2D: rows = grayscott(1, fields[0], fields[1], NULL, NULL, G[0], G[1], gfields[0], gfields[1], shape, spacing, coeffs, BC_PERIODIC); break;
    case OP_GRAYSCOTT_2D_XSLAB: rows = grayscott(1, fields[0], fields[1], NULL, NULL, G[0], G[1], gfields[0], gfields[1], shape, spacing, coeffs, BC_INTERIOR); break;
    case OP_HELMHOLTZ_3D_O4: rows = helmholtz(1, fields[0], NULL, NULL, G[0], gfields[0], shape, spacing, coeffs); break;
    case OP_NS_3D_T: rows = ns3dt(1, fields, NULL, G, gfields, shape, spacing, coeffs, BC_PERIODIC); break;
    case OP_NS_3D_T_XSLAB: rows = ns3dt(1, fields, NULL, G, gfields, shape, spacing, coeffs, BC_INTERIOR); break;
    case OP_NS_2D_STEADY: rows = ns2d(1, fields, NULL, G, gfields, shape, spacing, coeffs); break;
    case OP_NS_3D_STEADY: rows = ns3d(1, fields, NULL, G, gfields, shape, spacing, coeffs); break;
    }
    return rows;
}
