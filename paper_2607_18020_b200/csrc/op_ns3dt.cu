// Unsteady incompressible Navier-Stokes on an (x,y,z,t) array (t contiguous), space periodic,
// rows at interior t: four residuals (momentum x,y,z and continuity) from four fields
// (u,v,w,p).  This is Section 2.1's steady 2-D system extended by d_t, w and d_z; the adjoint
// below is Eq. (1) / Appendix A.2 extended the same way (drop w, z and t and it is the printed
// u-gradient term by term).
//
// Memory view: (x, y, row) with row = (z,t) flattened, n2*n3 contiguous floats.  Along a row,
// t+-1 is +-1 float and z+-1 is +-n3 floats with wrap-around over the row, so periodic z is a
// cyclic shift inside one contiguous line.
//
// Kernel shape (both directions): a thread owns one float4 (four consecutive t of one z) of a
// (y,row) tile and marches along x, the slowest axis, with a three-plane register window per
// array; y+-1 and z+-1 neighbours of the current plane are read through L1, t+-1 neighbours
// come from the adjacent lanes' registers.  Nodes at the first / last t carry no row: the
// forward pass writes 0 there, the adjoint treats the upstream arrays as 0 there (omitted
// neighbours, Appendix A.4), which is the boundary-gradient correction of the t axis.
#include "fpde_common.cuh"
#include "fpde_internal.h"

#include <algorithm>
#include <cstdlib>

namespace fpde {

struct NsParams {
    const float* f[4];    // u, v, w, p
    const float* g[4];    // adjoint: upstream G of mom_x, mom_y, mom_z, continuity
    float* out[4];
    float gs[4];
    int n0, n1, n3;       // x, y extents; t extent
    int C, C4, nt4;       // row length in floats / float4, float4 per z
    int planes_per_item, ncb, nmb, nitems;
    float ihx, ihy, ihz, iht;       // 1/(2h)
    float ihxx, ihyy, ihzz;         // 1/h^2
    float nu;
    float* partials;
};

struct NsIndex {
    int c4, m, zm4, zp4;       // own float4 column, y row, float4 columns of z-1 / z+1
    bool cvalid, valid;
    bool t_first, t_last;      // this float4 holds t = 0 (in .x) / t = n3-1 (in .w)
};

__device__ __forceinline__ NsIndex ns_index(const NsParams& p, int& a0, int& a1) {
    NsIndex ix;
    int item = blockIdx.x;
    const int cb = item % p.ncb; item /= p.ncb;
    const int mb = item % p.nmb;
    const int ab = item / p.nmb;
    ix.c4 = cb * blockDim.x + threadIdx.x;
    ix.m = mb * blockDim.y + threadIdx.y;
    ix.cvalid = ix.c4 < p.C4;
    ix.valid = ix.cvalid && ix.m < p.n1;
    const int c4c = ix.cvalid ? ix.c4 : 0;
    ix.zm4 = c4c - p.nt4; if (ix.zm4 < 0) ix.zm4 += p.C4;
    ix.zp4 = c4c + p.nt4; if (ix.zp4 >= p.C4) ix.zp4 -= p.C4;
    const int tq = c4c % p.nt4;
    ix.t_first = tq == 0;
    ix.t_last = tq == p.nt4 - 1;
    a0 = ab * p.planes_per_item;
    a1 = min(a0 + p.planes_per_item, p.n0);
    return ix;
}

__device__ __forceinline__ int wrapi(int i, int n) { return i < 0 ? i + n : (i >= n ? i - n : i); }

// ------------------------------------------------------------------------------------------
// forward
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) ns_fwd_kernel(const NsParams p) {
    int a0, a1;
    const NsIndex ix = ns_index(p, a0, a1);
    const int n0 = p.n0, n1 = p.n1;
    const size_t C = p.C;
    const int mrow = ix.m < n1 ? ix.m : 0;
    const int ym = wrapi(mrow - 1, n1), yp = wrapi(mrow + 1, n1);

    auto ld = [&](const float* base, int a, int mm, int col4) -> float4 {
        return ld4(base + ((size_t)a * n1 + mm) * C + 4 * col4);
    };
    const int c4 = ix.cvalid ? ix.c4 : 0;

    float4 W0[4], W1[4], W2[4];     // planes x-1, x, x+1 of u,v,w,p at the own column
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        W0[k] = ld(p.f[k], wrapi(a0 - 1, n0), mrow, c4);
        W1[k] = ld(p.f[k], a0, mrow, c4);
    }
    float acc[4] = {0.f, 0.f, 0.f, 0.f};

    for (int a = a0; a < a1; ++a) {
        const int ap = wrapi(a + 1, n0);
        float4 Ym[4], Yp[4], Zm[4], Zp[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            W2[k] = ld(p.f[k], ap, mrow, c4);
            Ym[k] = ld(p.f[k], a, ym, c4);
            Yp[k] = ld(p.f[k], a, yp, c4);
            Zm[k] = ld(p.f[k], a, mrow, ix.zm4);
            Zp[k] = ld(p.f[k], a, mrow, ix.zp4);
        }
        LR2 lr[3];
#pragma unroll
        for (int k = 0; k < 3; ++k)
            lr[k] = lane_neighbours<1>(p.f[k] + ((size_t)a * n1 + mrow) * C, ix.c4, p.C4, W1[k], false, 1.f);

        float o[4][4];
#pragma unroll
        for (int comp = 0; comp < 4; ++comp) {
            const float u = f4get(W1[0], comp), v = f4get(W1[1], comp), w = f4get(W1[2], comp);
            float res[3];
#pragma unroll
            for (int k = 0; k < 3; ++k) {
                const float c = f4get(W1[k], comp);
                const float xm = f4get(W0[k], comp), xp = f4get(W2[k], comp);
                const float ymv = f4get(Ym[k], comp), ypv = f4get(Yp[k], comp);
                const float zmv = f4get(Zm[k], comp), zpv = f4get(Zp[k], comp);
                const float tm = comp == 0 ? lr[k].l1 : f4get(W1[k], comp - 1);
                const float tp = comp == 3 ? lr[k].r1 : f4get(W1[k], comp + 1);
                const float lap = ((xm - c) + (xp - c)) * p.ihxx + ((ymv - c) + (ypv - c)) * p.ihyy
                                + ((zmv - c) + (zpv - c)) * p.ihzz;
                res[k] = (tp - tm) * p.iht + u * ((xp - xm) * p.ihx) + v * ((ypv - ymv) * p.ihy)
                       + w * ((zpv - zmv) * p.ihz) - p.nu * lap;
            }
            res[0] += (f4get(W2[3], comp) - f4get(W0[3], comp)) * p.ihx;     // d_x p
            res[1] += (f4get(Yp[3], comp) - f4get(Ym[3], comp)) * p.ihy;     // d_y p
            res[2] += (f4get(Zp[3], comp) - f4get(Zm[3], comp)) * p.ihz;     // d_z p
            const float div = (f4get(W2[0], comp) - f4get(W0[0], comp)) * p.ihx
                            + (f4get(Yp[1], comp) - f4get(Ym[1], comp)) * p.ihy
                            + (f4get(Zp[2], comp) - f4get(Zm[2], comp)) * p.ihz;
            o[0][comp] = res[0]; o[1][comp] = res[1]; o[2][comp] = res[2]; o[3][comp] = div;
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {          // t = 0 and t = n3-1 carry no row
            if (ix.t_first) o[e][0] = 0.f;
            if (ix.t_last) o[e][3] = 0.f;
        }
        if (ix.valid) {
            const size_t off = ((size_t)a * n1 + ix.m) * C + 4 * ix.c4;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float4 ov = make_float4(o[e][0], o[e][1], o[e][2], o[e][3]);
                st4(p.out[e] + off, ov);
                acc[e] += sq4(ov);
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) { W0[k] = W1[k]; W1[k] = W2[k]; }
    }
    if (p.partials != nullptr) block_reduce_store<4>(acc, p.partials, p.nitems, blockIdx.x);
}

// ------------------------------------------------------------------------------------------
// adjoint (gather form).  With G the upstream arrays (zero at the first / last t), c = (u,v,w),
// a_q the axis of momentum component q:
//   g_q(P) = sum_e G_e(P) * (d_{a_q} e)(P)                                     local terms
//          + sum_a [ (G_q c_a)(P-a) - (G_q c_a)(P+a) ] / (2 h_a)               transposed advection
//          - nu sum_a [ G_q(P-a) - 2 G_q(P) + G_q(P+a) ] / h_a^2               transposed diffusion
//          + [ G_q(P-t) - G_q(P+t) ] / (2 dt)                                  transposed d_t
//          + [ G_c(P-a_q) - G_c(P+a_q) ] / (2 h_{a_q})                         continuity row
//   g_p(P) = sum_q [ G_q(P-a_q) - G_q(P+a_q) ] / (2 h_{a_q})
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) ns_bwd_kernel(const NsParams p) {
    int a0, a1;
    const NsIndex ix = ns_index(p, a0, a1);
    const int n0 = p.n0, n1 = p.n1;
    const size_t C = p.C;
    const int mrow = ix.m < n1 ? ix.m : 0;
    const int ym = wrapi(mrow - 1, n1), yp = wrapi(mrow + 1, n1);
    const int c4 = ix.cvalid ? ix.c4 : 0;

    auto ldf = [&](int k, int a, int mm, int col4) -> float4 {
        return ld4(p.f[k] + ((size_t)a * n1 + mm) * C + 4 * col4);
    };
    // upstream array k, scaled, zeroed at the first / last t.  z-neighbours sit at the same t.
    auto ldg = [&](int k, int a, int mm, int col4) -> float4 {
        float4 v = f4scale(ld4(p.g[k] + ((size_t)a * n1 + mm) * C + 4 * col4), p.gs[k]);
        if (ix.t_first) v.x = 0.f;
        if (ix.t_last) v.w = 0.f;
        return v;
    };

    float4 F0[3], F1[3], F2[3];     // u,v,w at x-1, x, x+1
    float4 G0[4], G1[4], G2[4];     // G_u,G_v,G_w,G_c at x-1, x, x+1
    {
        const int am = wrapi(a0 - 1, n0);
#pragma unroll
        for (int k = 0; k < 3; ++k) { F0[k] = ldf(k, am, mrow, c4); F1[k] = ldf(k, a0, mrow, c4); }
#pragma unroll
        for (int k = 0; k < 4; ++k) { G0[k] = ldg(k, am, mrow, c4); G1[k] = ldg(k, a0, mrow, c4); }
    }

    for (int a = a0; a < a1; ++a) {
        const int ap = wrapi(a + 1, n0);
        float4 FYm[3], FYp[3], FZm[3], FZp[3], GYm[4], GYp[4], GZm[4], GZp[4];
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            F2[k] = ldf(k, ap, mrow, c4);
            FYm[k] = ldf(k, a, ym, c4); FYp[k] = ldf(k, a, yp, c4);
            FZm[k] = ldf(k, a, mrow, ix.zm4); FZp[k] = ldf(k, a, mrow, ix.zp4);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            G2[k] = ldg(k, ap, mrow, c4);
            GYm[k] = ldg(k, a, ym, c4); GYp[k] = ldg(k, a, yp, c4);
            GZm[k] = ldg(k, a, mrow, ix.zm4); GZp[k] = ldg(k, a, mrow, ix.zp4);
        }
        LR2 lr[3];
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            lr[k] = lane_neighbours<1>(p.g[k] + ((size_t)a * n1 + mrow) * C, ix.c4, p.C4, G1[k], false, p.gs[k]);
            // the neighbour across a z-group boundary is the other group's first / last t: no row
            if (ix.t_first) lr[k].l1 = 0.f;
            if (ix.t_last) lr[k].r1 = 0.f;
        }

        float o[4][4];
#pragma unroll
        for (int comp = 0; comp < 4; ++comp) {
            // centred first differences d_a e of the three velocity components
            float dx[3], dy[3], dz[3];
#pragma unroll
            for (int e = 0; e < 3; ++e) {
                dx[e] = (f4get(F2[e], comp) - f4get(F0[e], comp)) * p.ihx;
                dy[e] = (f4get(FYp[e], comp) - f4get(FYm[e], comp)) * p.ihy;
                dz[e] = (f4get(FZp[e], comp) - f4get(FZm[e], comp)) * p.ihz;
            }
            const float gu = f4get(G1[0], comp), gv = f4get(G1[1], comp), gw = f4get(G1[2], comp);
            // advecting velocities at the six neighbours: u at x-+1, v at y-+1, w at z-+1
            const float uxm = f4get(F0[0], comp), uxp = f4get(F2[0], comp);
            const float vym = f4get(FYm[1], comp), vyp = f4get(FYp[1], comp);
            const float wzm = f4get(FZm[2], comp), wzp = f4get(FZp[2], comp);
            float gq[3];
#pragma unroll
            for (int q = 0; q < 3; ++q) {
                const float c = f4get(G1[q], comp);
                const float xm = f4get(G0[q], comp), xp = f4get(G2[q], comp);
                const float ymv = f4get(GYm[q], comp), ypv = f4get(GYp[q], comp);
                const float zmv = f4get(GZm[q], comp), zpv = f4get(GZp[q], comp);
                const float tm = comp == 0 ? lr[q].l1 : f4get(G1[q], comp - 1);
                const float tp = comp == 3 ? lr[q].r1 : f4get(G1[q], comp + 1);
                const float adv = (xm * uxm - xp * uxp) * p.ihx + (ymv * vym - ypv * vyp) * p.ihy
                                + (zmv * wzm - zpv * wzp) * p.ihz;
                const float lap = ((xm - c) + (xp - c)) * p.ihxx + ((ymv - c) + (ypv - c)) * p.ihyy
                                + ((zmv - c) + (zpv - c)) * p.ihzz;
                gq[q] = adv - p.nu * lap + (tm - tp) * p.iht;
            }
            gq[0] += gu * dx[0] + gv * dx[1] + gw * dx[2] + (f4get(G0[3], comp) - f4get(G2[3], comp)) * p.ihx;
            gq[1] += gu * dy[0] + gv * dy[1] + gw * dy[2] + (f4get(GYm[3], comp) - f4get(GYp[3], comp)) * p.ihy;
            gq[2] += gu * dz[0] + gv * dz[1] + gw * dz[2] + (f4get(GZm[3], comp) - f4get(GZp[3], comp)) * p.ihz;
            const float gp = (f4get(G0[0], comp) - f4get(G2[0], comp)) * p.ihx
                           + (f4get(GYm[1], comp) - f4get(GYp[1], comp)) * p.ihy
                           + (f4get(GZm[2], comp) - f4get(GZp[2], comp)) * p.ihz;
            o[0][comp] = gq[0]; o[1][comp] = gq[1]; o[2][comp] = gq[2]; o[3][comp] = gp;
        }
        if (ix.valid) {
            const size_t off = ((size_t)a * n1 + ix.m) * C + 4 * ix.c4;
#pragma unroll
            for (int e = 0; e < 4; ++e)
                st4(p.out[e] + off, make_float4(o[e][0], o[e][1], o[e][2], o[e][3]));
        }
#pragma unroll
        for (int k = 0; k < 3; ++k) { F0[k] = F1[k]; F1[k] = F2[k]; }
#pragma unroll
        for (int k = 0; k < 4; ++k) { G0[k] = G1[k]; G1[k] = G2[k]; }
    }
}

static int env_int(const char* name, int dflt) {
    const char* s = std::getenv(name);
    if (!s || !*s) return dflt;
    const int v = std::atoi(s);
    return v > 0 ? v : dflt;
}

static void ns_geometry(const Problem& q, NsParams& p, dim3& block) {
    p.n0 = q.n[0]; p.n1 = q.n[1]; p.n3 = q.n[3];
    p.C = q.n[2] * q.n[3]; p.C4 = p.C / 4; p.nt4 = q.n[3] / 4;
    int tx = p.C4 >= 64 ? 64 : 32;
    tx = env_int("FPDE_NS_TX", tx);
    tx = std::max(32, std::min(256, (tx / 32) * 32));
    int ty = env_int("FPDE_NS_TY", 4);
    ty = std::max(1, std::min(256 / tx, ty));
    block = dim3(tx, ty, 1);
    p.planes_per_item = env_int("FPDE_NS_PLANES", 16);
    p.ncb = (p.C4 + tx - 1) / tx;
    p.nmb = (p.n1 + ty - 1) / ty;
    p.nitems = p.ncb * p.nmb * ((p.n0 + p.planes_per_item - 1) / p.planes_per_item);
    p.ihx = (float)(0.5 / q.h[0]); p.ihy = (float)(0.5 / q.h[1]); p.ihz = (float)(0.5 / q.h[2]);
    p.iht = (float)(0.5 / q.h[3]);
    p.ihxx = (float)(1.0 / (q.h[0] * q.h[0])); p.ihyy = (float)(1.0 / (q.h[1] * q.h[1]));
    p.ihzz = (float)(1.0 / (q.h[2] * q.h[2]));
    p.nu = (float)q.coef[0];
}

int ns_items(const int* n) {
    Problem q{};
    for (int a = 0; a < 4; ++a) { q.n[a] = n[a]; q.h[a] = 1.0; }
    NsParams p{}; dim3 block;
    ns_geometry(q, p, block);
    return p.nitems;
}

cudaError_t launch_ns_fwd(const Problem& q) {
    NsParams p{}; dim3 block;
    ns_geometry(q, p, block);
    for (int k = 0; k < 4; ++k) { p.f[k] = q.in[k]; p.out[k] = q.out[k]; }
    p.partials = q.partials;
    ns_fwd_kernel<<<p.nitems, block, 0, q.stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_ns_bwd(const Problem& q) {
    NsParams p{}; dim3 block;
    ns_geometry(q, p, block);
    for (int k = 0; k < 4; ++k) {
        p.f[k] = q.in[k]; p.g[k] = q.aux[k]; p.out[k] = q.out[k]; p.gs[k] = (float)q.gscale[k];
    }
    p.partials = nullptr;
    ns_bwd_kernel<<<p.nitems, block, 0, q.stream>>>(p);
    return cudaGetLastError();
}

}  // namespace fpde
