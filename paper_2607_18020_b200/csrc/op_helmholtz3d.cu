// Three-dimensional fourth-order Helmholtz operator, r = Lap4 u + k^2 u - f, with the 13-point
// star (-1,16,-30,16,-1)/(12 h^2) per axis: fused forward residual + loss partials (Section
// 2.1) and the gather-form adjoint with its two-cell boundary band (Sections 2.2, 2.3).
//
// The Jacobian is constant and the star is symmetric, so the adjoint is the same star applied
// to the upstream array treated as zero outside the rows (omitted neighbours, Appendix A.4);
// that one rule produces the gradient of the two outer layers and the truncated sums of layers
// 2 and 3.  Forward and adjoint are therefore two instances of one 2.5-D engine:
//
//   a thread owns one float4 of a (y,z) tile and marches along x, the slowest axis, holding the
//   five x-planes of its own column in registers; the y+-1, y+-2 neighbours of the current plane
//   are read through L1 (other threads of the same block loaded those lines two steps earlier);
//   z neighbours come from the adjacent lanes' registers.
#include "fpde_common.cuh"
#include "fpde_internal.h"

#include <algorithm>
#include <cstdlib>

namespace fpde {

struct Star3dParams {
    const float* hin;     // read with halo 2 (u forward, upstream G in the adjoint)
    const float* cin;     // read at the centre (f forward, unused in the adjoint)
    float* out;
    float hscale;
    int n0, n1, n2, nc4;
    int planes_per_item, ncb, nmb, nitems;
    float w0, w1, w2;     // 1/(12 h_a^2)
    float k2;
    float* partials;
};

template <bool FWD>
__global__ void __launch_bounds__(256) star3d_kernel(const Star3dParams p) {
    const int n0 = p.n0, n1 = p.n1, n2 = p.n2;
    int item = blockIdx.x;
    const int cb = item % p.ncb; item /= p.ncb;
    const int mb = item % p.nmb;
    const int ab = item / p.nmb;
    const int c4 = cb * blockDim.x + threadIdx.x;
    const int m = mb * blockDim.y + threadIdx.y;
    const bool cvalid = c4 < p.nc4;
    const bool valid = cvalid && m < n1;
    const bool first_col = c4 == 0, last_col = c4 == p.nc4 - 1;
    const int a0 = ab * p.planes_per_item;
    const int a1 = min(a0 + p.planes_per_item, n0);
    constexpr bool MASK_IN = !FWD;

    // does a (plane,row) pair of the halo input read as zero?
    auto dead = [&](int a, int mm) -> bool {
        if (a < 0 || a >= n0 || mm < 0 || mm >= n1) return true;
        if (MASK_IN && (a < 2 || a > n0 - 3 || mm < 2 || mm > n1 - 3)) return true;
        return false;
    };
    auto load_h = [&](int a, int mm) -> float4 {
        if (dead(a, mm) || !cvalid) return f4zero();
        float4 v = ld4(p.hin + ((size_t)a * n1 + mm) * n2 + 4 * c4);
        if (MASK_IN) {
            v = f4scale(v, p.hscale);
            if (first_col) { v.x = 0.f; v.y = 0.f; }
            if (last_col) { v.z = 0.f; v.w = 0.f; }
        }
        return v;
    };

    float4 q0 = load_h(a0 - 2, m), q1 = load_h(a0 - 1, m), q2 = load_h(a0, m), q3 = load_h(a0 + 1, m);
    float acc[1] = {0.f};

    for (int a = a0; a < a1; ++a) {
        const float4 q4 = load_h(a + 2, m);
        const float4 ym1 = load_h(a, m - 1), yp1 = load_h(a, m + 1);
        const float4 ym2 = load_h(a, m - 2), yp2 = load_h(a, m + 2);
        float4 src = f4zero();
        if (FWD && valid) src = ld4(p.cin + ((size_t)a * n1 + m) * n2 + 4 * c4);
        LR2 lr;
        if (!dead(a, m)) {     // uniform over a warp (a warp lies inside one row)
            lr = lane_neighbours<2>(p.hin + ((size_t)a * n1 + m) * n2, c4, p.nc4, q2, false,
                                    MASK_IN ? p.hscale : 1.f);
        } else {
            lr.l1 = lr.l2 = lr.r1 = lr.r2 = 0.f;
        }
        float o[4];
#pragma unroll
        for (int comp = 0; comp < 4; ++comp) {
            const float c = f4get(q2, comp);
            const float l1 = comp == 0 ? lr.l1 : f4get(q2, comp - 1);
            const float l2 = comp == 0 ? lr.l2 : (comp == 1 ? lr.l1 : f4get(q2, comp - 2));
            const float r1 = comp == 3 ? lr.r1 : f4get(q2, comp + 1);
            const float r2 = comp == 3 ? lr.r2 : (comp == 2 ? lr.r1 : f4get(q2, comp + 2));
            const float sx = 16.f * ((f4get(q1, comp) - c) + (f4get(q3, comp) - c))
                           - ((f4get(q0, comp) - c) + (f4get(q4, comp) - c));
            const float sy = 16.f * ((f4get(ym1, comp) - c) + (f4get(yp1, comp) - c))
                           - ((f4get(ym2, comp) - c) + (f4get(yp2, comp) - c));
            const float sz = 16.f * ((l1 - c) + (r1 - c)) - ((l2 - c) + (r2 - c));
            float v = sx * p.w0 + sy * p.w1 + sz * p.w2 + p.k2 * c;
            if (FWD) v -= f4get(src, comp);
            o[comp] = v;
        }
        if (FWD) {   // nodes of the two outer layers carry no row
            if (a < 2 || a > n0 - 3 || m < 2 || m > n1 - 3) { o[0] = o[1] = o[2] = o[3] = 0.f; }
            if (first_col) { o[0] = 0.f; o[1] = 0.f; }
            if (last_col) { o[2] = 0.f; o[3] = 0.f; }
        }
        if (valid) {
            const float4 ov = make_float4(o[0], o[1], o[2], o[3]);
            st4(p.out + ((size_t)a * n1 + m) * n2 + 4 * c4, ov);
            if (FWD) acc[0] += sq4(ov);
        }
        q0 = q1; q1 = q2; q2 = q3; q3 = q4;
    }
    if (FWD && p.partials != nullptr) block_reduce_store<1>(acc, p.partials, p.nitems, blockIdx.x);
}

static int env_int(const char* name, int dflt) {
    const char* s = std::getenv(name);
    if (!s || !*s) return dflt;
    const int v = std::atoi(s);
    return v > 0 ? v : dflt;
}

static void star3d_geometry(const Problem& q, Star3dParams& p, dim3& block) {
    p.n0 = q.n[0]; p.n1 = q.n[1]; p.n2 = q.n[2]; p.nc4 = q.n[2] / 4;
    int tx = p.nc4 >= 64 ? 64 : 32;
    tx = env_int("FPDE_STAR3D_TX", tx);
    tx = std::max(32, std::min(128, (tx / 32) * 32));
    int ty = env_int("FPDE_STAR3D_TY", 4);
    ty = std::max(1, std::min(256 / tx, ty));
    block = dim3(tx, ty, 1);
    p.planes_per_item = env_int("FPDE_STAR3D_PLANES", 32);
    p.ncb = (p.nc4 + tx - 1) / tx;
    p.nmb = (p.n1 + ty - 1) / ty;
    p.nitems = p.ncb * p.nmb * ((p.n0 + p.planes_per_item - 1) / p.planes_per_item);
    p.w0 = (float)(1.0 / (12.0 * q.h[0] * q.h[0]));
    p.w1 = (float)(1.0 / (12.0 * q.h[1] * q.h[1]));
    p.w2 = (float)(1.0 / (12.0 * q.h[2] * q.h[2]));
    p.k2 = (float)(q.coef[0] * q.coef[0]);
}

int star3d_items(const int* n) {
    Problem q{}; q.n[0] = n[0]; q.n[1] = n[1]; q.n[2] = n[2]; q.h[0] = q.h[1] = q.h[2] = 1.0;
    Star3dParams p{}; dim3 block;
    star3d_geometry(q, p, block);
    return p.nitems;
}

cudaError_t launch_helmholtz_fwd(const Problem& q) {
    Star3dParams p{}; dim3 block;
    star3d_geometry(q, p, block);
    p.hin = q.in[0]; p.cin = q.aux[0]; p.out = q.out[0]; p.hscale = 1.f;
    p.partials = q.partials;
    star3d_kernel<true><<<p.nitems, block, 0, q.stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_helmholtz_bwd(const Problem& q) {
    Star3dParams p{}; dim3 block;
    star3d_geometry(q, p, block);
    p.hin = q.aux[0]; p.cin = nullptr; p.out = q.out[0]; p.hscale = (float)q.gscale[0];
    p.partials = nullptr;
    star3d_kernel<false><<<p.nitems, block, 0, q.stream>>>(p);
    return cudaGetLastError();
}

}  // namespace fpde
