// Double-precision verification path: every operator's residual and gather-form adjoint with one
// thread per node, written for clarity, not speed (the paper trains and times in fp32 and uses
// fp64 only to verify its hand-derived adjoints; Section 4 setup).  It shares the registry and the
// argument checks with the fp32 path but none of its kernels: two implementations of the same
// formulas that can be held against each other and against a CPU reference.
//
// Conventions.  A node carries a residual row iff on every INTERIOR axis its index lies in
// [radius, n-1-radius].  The adjoint reads the upstream arrays through G(), which returns 0 at
// nodes without a row and outside the array (omitted neighbours, Appendix A.5); with that rule
// the gather formulas below hold at every node, boundary layers included (Section 2.3).
#include "fpde_common.cuh"
#include "fpde_internal.h"

namespace fpde {

struct F64Params {
    const double* in[MAX_F];    // fields
    const double* aux[MAX_F];   // fwd: sources ; bwd: upstream arrays
    double* out[MAX_F];
    double gs[MAX_F];
    int op, ndim;
    int n[MAX_D];
    int stride[MAX_D];
    int bc[MAX_D];              // 0 periodic, 1 interior, 2 one-sided
    int radius;
    double h[MAX_D];
    double coef[8];
    double* partials;           // fwd: one double per block and residual
    int nblocks;
    int N;
};

struct Node {
    int c[MAX_D];
    int idx;
};

__device__ __forceinline__ Node node_of(const F64Params& p, int idx) {
    Node q; q.idx = idx;
    int rem = idx;
#pragma unroll
    for (int a = 0; a < MAX_D; ++a) {
        if (a < p.ndim) { q.c[a] = rem / p.stride[a]; rem -= q.c[a] * p.stride[a]; }
        else q.c[a] = 0;
    }
    return q;
}

// does the node at coordinates c carry a row?
__device__ __forceinline__ bool has_row(const F64Params& p, const int* c) {
    bool ok = true;
#pragma unroll
    for (int a = 0; a < MAX_D; ++a)
        if (a < p.ndim && p.bc[a] == 1) ok = ok && c[a] >= p.radius && c[a] <= p.n[a] - 1 - p.radius;
    return ok;
}

// index of the node displaced by d along axis a: periodic axes wrap; on the other axes the
// index is clamped into the array and `inside` tells whether the true neighbour exists
__device__ __forceinline__ int shifted(const F64Params& p, const Node& q, int a, int d, bool& inside) {
    int c = q.c[a] + d;
    inside = true;
    if (p.bc[a] == 0) { if (c < 0) c += p.n[a]; else if (c >= p.n[a]) c -= p.n[a]; }
    else if (c < 0 || c >= p.n[a]) { inside = false; c = c < 0 ? 0 : p.n[a] - 1; }
    return q.idx + (c - q.c[a]) * p.stride[a];
}

// field value at the displaced node (clamped where the neighbour does not exist: such values
// only ever multiply a zero)
__device__ __forceinline__ double fld(const F64Params& p, const double* f, const Node& q, int a, int d) {
    bool in; return f[shifted(p, q, a, d, in)];
}

// upstream value at the displaced node, zero-extended
__device__ __forceinline__ double G(const F64Params& p, int e, const Node& q, int a, int d) {
    bool in;
    const int j = shifted(p, q, a, d, in);
    if (!in) return 0.0;
    Node t = q;
    int c = q.c[a] + d;
    if (p.bc[a] == 0) { if (c < 0) c += p.n[a]; else if (c >= p.n[a]) c -= p.n[a]; }
    t.c[a] = c;
    return has_row(p, t.c) ? p.gs[e] * p.aux[e][j] : 0.0;
}

__device__ __forceinline__ double d1c(const F64Params& p, const double* f, const Node& q, int a) {
    return (fld(p, f, q, a, 1) - fld(p, f, q, a, -1)) / (2.0 * p.h[a]);
}
__device__ __forceinline__ double d2c(const F64Params& p, const double* f, const Node& q, int a) {
    return (fld(p, f, q, a, 1) - 2.0 * f[q.idx] + fld(p, f, q, a, -1)) / (p.h[a] * p.h[a]);
}
// fourth-order second difference (-1, 16, -30, 16, -1) / (12 h^2)
__device__ __forceinline__ double d2o4(const F64Params& p, const double* f, const Node& q, int a) {
    return (-fld(p, f, q, a, -2) + 16.0 * fld(p, f, q, a, -1) - 30.0 * f[q.idx] + 16.0 * fld(p, f, q, a, 1)
            - fld(p, f, q, a, 2)) / (12.0 * p.h[a] * p.h[a]);
}
// the same differences of a zero-extended upstream array (symmetric stencils: own transpose)
__device__ __forceinline__ double G_d2c(const F64Params& p, int e, const Node& q, int a) {
    return (G(p, e, q, a, 1) - 2.0 * G(p, e, q, a, 0) + G(p, e, q, a, -1)) / (p.h[a] * p.h[a]);
}
__device__ __forceinline__ double G_d2o4(const F64Params& p, int e, const Node& q, int a) {
    return (-G(p, e, q, a, -2) + 16.0 * G(p, e, q, a, -1) - 30.0 * G(p, e, q, a, 0) + 16.0 * G(p, e, q, a, 1)
            - G(p, e, q, a, 2)) / (12.0 * p.h[a] * p.h[a]);
}
// transposed centred first difference of a zero-extended array w: [w(P-a) - w(P+a)] / (2h)
__device__ __forceinline__ double G_d1T(const F64Params& p, int e, const Node& q, int a) {
    return (G(p, e, q, a, -1) - G(p, e, q, a, 1)) / (2.0 * p.h[a]);
}

// ---- Burgers: one-sided rows, explicit transposes ------------------------------------------------
__device__ __forceinline__ double b_d1(const double* f, int i, int n, int s, double h) {
    if (i == 0) return (-3.0 * f[0] + 4.0 * f[s] - f[2 * s]) / (2.0 * h);
    if (i == n - 1) return (3.0 * f[(n - 1) * s] - 4.0 * f[(n - 2) * s] + f[(n - 3) * s]) / (2.0 * h);
    return (f[(i + 1) * s] - f[(i - 1) * s]) / (2.0 * h);
}
__device__ __forceinline__ double b_d2(const double* f, int i, int n, int s, double h) {
    if (i == 0) return (2.0 * f[0] - 5.0 * f[s] + 4.0 * f[2 * s] - f[3 * s]) / (h * h);
    if (i == n - 1)
        return (2.0 * f[(n - 1) * s] - 5.0 * f[(n - 2) * s] + 4.0 * f[(n - 3) * s] - f[(n - 4) * s]) / (h * h);
    return (f[(i + 1) * s] - 2.0 * f[i * s] + f[(i - 1) * s]) / (h * h);
}
// weight of column j in row i of the first / second difference matrices (times 2h / h^2)
__device__ __forceinline__ double b_w1(int i, int j, int n) {
    if (i == 0) return j == 0 ? -3.0 : (j == 1 ? 4.0 : (j == 2 ? -1.0 : 0.0));
    if (i == n - 1) return j == n - 1 ? 3.0 : (j == n - 2 ? -4.0 : (j == n - 3 ? 1.0 : 0.0));
    return j == i + 1 ? 1.0 : (j == i - 1 ? -1.0 : 0.0);
}
__device__ __forceinline__ double b_w2(int i, int j, int n) {
    if (i == 0) return j == 0 ? 2.0 : (j == 1 ? -5.0 : (j == 2 ? 4.0 : (j == 3 ? -1.0 : 0.0)));
    if (i == n - 1) return j == n - 1 ? 2.0 : (j == n - 2 ? -5.0 : (j == n - 3 ? 4.0 : (j == n - 4 ? -1.0 : 0.0)));
    return j == i ? -2.0 : ((j == i + 1 || j == i - 1) ? 1.0 : 0.0);
}
// (D^T w)_j = sum_i D[i][j] w_i: the rows that can reach column j are j-1, j, j+1 and the two
// one-sided rows 0 and n-1
template <class WF>
__device__ __forceinline__ double b_T(WF w, int j, int n, bool second) {
    double s = 0.0;
    int rows[5] = {j - 1, j, j + 1, 0, n - 1};
    for (int k = 0; k < 5; ++k) {
        const int i = rows[k];
        if (i < 0 || i >= n) continue;
        bool seen = false;
        for (int m = 0; m < k; ++m) seen = seen || rows[m] == i;
        if (seen) continue;
        s += (second ? b_w2(i, j, n) : b_w1(i, j, n)) * w(i);
    }
    return s;
}

// ---- residuals at a node ------------------------------------------------------------------------
__device__ void residual_at(const F64Params& p, const Node& q, double* r) {
    const int nv = p.op == 5 ? 2 : 3;                     // velocity components of the NS operators
    switch (p.op) {
    case 0: {                                             // Burgers: r = u_t + u u_x - nu u_xx, (x,t) array
        const int i = q.c[0], j = q.c[1], nt = p.n[1];
        const double* u = p.in[0];
        r[0] = b_d1(u + (size_t)i * nt, j, nt, 1, p.h[1]) + u[q.idx] * b_d1(u + j, i, p.n[0], nt, p.h[0])
             - p.coef[0] * b_d2(u + j, i, p.n[0], nt, p.h[0]);
        break;
    }
    case 1:                                               // Poisson
        r[0] = -(d2c(p, p.in[0], q, 0) + d2c(p, p.in[0], q, 1)) - p.aux[0][q.idx];
        break;
    case 2: case 8: {                                     // Gray-Scott (8: its slab form): coef = D_u, D_v, F, k
        const double u = p.in[0][q.idx], v = p.in[1][q.idx];
        r[0] = p.coef[0] * (d2c(p, p.in[0], q, 0) + d2c(p, p.in[0], q, 1)) - u * v * v + p.coef[2] * (1.0 - u);
        r[1] = p.coef[1] * (d2c(p, p.in[1], q, 0) + d2c(p, p.in[1], q, 1)) + u * v * v - (p.coef[2] + p.coef[3]) * v;
        break;
    }
    case 3:                                               // Helmholtz, fourth order
        r[0] = d2o4(p, p.in[0], q, 0) + d2o4(p, p.in[0], q, 1) + d2o4(p, p.in[0], q, 2)
             + p.coef[0] * p.coef[0] * p.in[0][q.idx] - p.aux[0][q.idx];
        break;
    default: {                                            // Navier-Stokes: 3-D+T (4, slab form 7), steady 2-D (5), steady 3-D (6)
        const double* pr = p.in[nv];
        double cont = 0.0;
        for (int c = 0; c < nv; ++c) {
            const double* f = p.in[c];
            double m = (p.op == 4 || p.op == 7) ? d1c(p, f, q, 3) : 0.0;
            for (int a = 0; a < nv; ++a) m += p.in[a][q.idx] * d1c(p, f, q, a) - p.coef[0] * d2c(p, f, q, a);
            r[c] = m + d1c(p, pr, q, c);
            cont += d1c(p, f, q, c);
        }
        r[nv] = cont;
        break;
    }
    }
}

__global__ void __launch_bounds__(256) f64_fwd_kernel(const F64Params p, int ne) {
    __shared__ double red[MAX_F][8];
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    double r[MAX_F] = {0.0, 0.0, 0.0, 0.0};
    if (idx < p.N) {
        const Node q = node_of(p, idx);
        if (has_row(p, q.c)) residual_at(p, q, r);
        for (int e = 0; e < ne; ++e) p.out[e][idx] = r[e];
    }
    if (p.partials == nullptr) return;
    // fixed-shape reduction: shuffle tree, then the eight warp sums in order
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int e = 0; e < ne; ++e) {
        double v = r[e] * r[e];
        for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(FULL_MASK, v, o);
        if (lane == 0) red[e][warp] = v;
    }
    __syncthreads();
    if (threadIdx.x < ne) {
        double s = 0.0;
        for (int w = 0; w < 8; ++w) s += red[threadIdx.x][w];
        p.partials[(size_t)threadIdx.x * p.nblocks + blockIdx.x] = s;
    }
}

// loss_out[e] = sum of the block partials (fixed order) / rows ; loss_out[ne] = their sum
__global__ void __launch_bounds__(256) f64_finalize_kernel(const double* partials, int nblocks, int ne, double inv_rows,
                                                           double* loss_out) {
    __shared__ double sm[256];
    __shared__ double tot[MAX_F];
    for (int e = 0; e < ne; ++e) {
        double s = 0.0;
        for (int i = threadIdx.x; i < nblocks; i += 256) s += partials[(size_t)e * nblocks + i];
        sm[threadIdx.x] = s;
        __syncthreads();
        for (int o = 128; o > 0; o >>= 1) {
            if ((int)threadIdx.x < o) sm[threadIdx.x] += sm[threadIdx.x + o];
            __syncthreads();
        }
        if (threadIdx.x == 0) tot[e] = sm[0] * inv_rows;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int e = 0; e < ne; ++e) { loss_out[e] = tot[e]; t += tot[e]; }
        loss_out[ne] = t;
    }
}

// ---- gather-form adjoint at a node --------------------------------------------------------------
__device__ void adjoint_at(const F64Params& p, const Node& q, double* g) {
    const int nv = p.op == 5 ? 2 : 3;
    switch (p.op) {
    case 0: {
        // g = D_t^T G + (D_x u) G + D_x^T (u G) - nu D_xx^T G, one-sided rows included in the D's
        const int i = q.c[0], j = q.c[1], nx = p.n[0], nt = p.n[1];
        const double* u = p.in[0];
        const double* Gr = p.aux[0];
        auto Gt = [&](int jj) { return Gr[(size_t)i * nt + jj]; };
        auto Gx = [&](int ii) { return Gr[(size_t)ii * nt + j]; };
        auto uGx = [&](int ii) { return u[(size_t)ii * nt + j] * Gr[(size_t)ii * nt + j]; };
        g[0] = p.gs[0] * (b_T(Gt, j, nt, false) / (2.0 * p.h[1]) + b_d1(u + j, i, nx, nt, p.h[0]) * Gr[q.idx]
                          + b_T(uGx, i, nx, false) / (2.0 * p.h[0]) - p.coef[0] * b_T(Gx, i, nx, true) / (p.h[0] * p.h[0]));
        break;
    }
    case 1:
        g[0] = -(G_d2c(p, 0, q, 0) + G_d2c(p, 0, q, 1));
        break;
    case 2: case 8: {
        const double u = p.in[0][q.idx], v = p.in[1][q.idx];
        const double a = G(p, 0, q, 0, 0), b = G(p, 1, q, 0, 0);
        g[0] = p.coef[0] * (G_d2c(p, 0, q, 0) + G_d2c(p, 0, q, 1)) + a * (-v * v - p.coef[2]) + b * v * v;
        g[1] = p.coef[1] * (G_d2c(p, 1, q, 0) + G_d2c(p, 1, q, 1)) + a * (-2.0 * u * v)
             + b * (2.0 * u * v - (p.coef[2] + p.coef[3]));
        break;
    }
    case 3:
        g[0] = G_d2o4(p, 0, q, 0) + G_d2o4(p, 0, q, 1) + G_d2o4(p, 0, q, 2) + p.coef[0] * p.coef[0] * G(p, 0, q, 0, 0);
        break;
    default: {
        // Eq. (1) / Appendix A.3 and their extension by w, d_z and d_t:
        //   g_c = sum_e G_e d_c(e)  +  sum_a D_a^T (u_a G_c)  -  nu sum_a D_aa G_c  +  D_t^T G_c  +  D_c^T G_div
        //   g_p = sum_c D_c^T G_c
        double gp = 0.0;
        for (int c = 0; c < nv; ++c) {
            double s = 0.0;
            for (int e = 0; e < nv; ++e) {                 // local terms: G_e(P) (d_c e)(P)
                const double ge = G(p, e, q, 0, 0);
                if (ge != 0.0) s += ge * d1c(p, p.in[e], q, c);
            }
            for (int a = 0; a < nv; ++a) {
                s += (G(p, c, q, a, -1) * fld(p, p.in[a], q, a, -1) - G(p, c, q, a, 1) * fld(p, p.in[a], q, a, 1))
                     / (2.0 * p.h[a]);
                s -= p.coef[0] * G_d2c(p, c, q, a);
            }
            if (p.op == 4 || p.op == 7) s += G_d1T(p, c, q, 3);
            s += G_d1T(p, nv, q, c);
            g[c] = s;
            gp += G_d1T(p, c, q, c);
        }
        g[nv] = gp;
        break;
    }
    }
}

__global__ void __launch_bounds__(256) f64_bwd_kernel(const F64Params p, int nf) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= p.N) return;
    const Node q = node_of(p, idx);
    double g[MAX_F] = {0.0, 0.0, 0.0, 0.0};
    adjoint_at(p, q, g);
    for (int f = 0; f < nf; ++f) p.out[f][idx] = g[f];
}

// ---- launchers ----------------------------------------------------------------------------------
static void f64_fill(const ProblemF64& q, F64Params& p) {
    p.op = q.op; p.ndim = q.ndim; p.radius = q.radius;
    int64_t N = 1;
    for (int a = 0; a < MAX_D; ++a) { p.n[a] = a < q.ndim ? q.n[a] : 1; p.h[a] = a < q.ndim ? q.h[a] : 1.0; p.bc[a] = a < q.ndim ? q.bc[a] : 0; }
    for (int a = q.ndim - 1; a >= 0; --a) { p.stride[a] = (int)N; N *= q.n[a]; }
    for (int a = q.ndim; a < MAX_D; ++a) p.stride[a] = 1;
    p.N = (int)N;
    for (int c = 0; c < 8; ++c) p.coef[c] = q.coef[c];
    for (int k = 0; k < MAX_F; ++k) { p.in[k] = q.in[k]; p.aux[k] = q.aux[k]; p.out[k] = q.out[k]; p.gs[k] = q.gscale[k]; }
    p.nblocks = (p.N + 255) / 256;
}

int f64_blocks(int64_t N) { return (int)((N + 255) / 256); }

cudaError_t launch_f64_fwd(const ProblemF64& q, int ne) {
    F64Params p{};
    f64_fill(q, p);
    p.partials = q.partials;
    f64_fwd_kernel<<<p.nblocks, 256, 0, q.stream>>>(p, ne);
    cudaError_t ce = cudaGetLastError();
    if (ce != cudaSuccess || q.partials == nullptr) return ce;
    f64_finalize_kernel<<<1, 256, 0, q.stream>>>(q.partials, p.nblocks, ne, 1.0 / (double)q.rows, q.loss_out);
    return cudaGetLastError();
}

cudaError_t launch_f64_bwd(const ProblemF64& q, int nf) {
    F64Params p{};
    f64_fill(q, p);
    f64_bwd_kernel<<<p.nblocks, 256, 0, q.stream>>>(p, nf);
    return cudaGetLastError();
}

}  // namespace fpde
