// Steady incompressible Navier-Stokes on an (x,y,z) array (z contiguous): Section 2.1's system
// with the third velocity component w and d_z added.  Four residuals (momentum x,y,z and
// continuity) from four fields (u,v,w,p); rows at the nodes where all three centred stencils
// fit, i.e. the interior [1,n-2]^3; the outer shell of the array is data.
//
//   mom_q = u d_x q + v d_y q + w d_z q + d_{a_q} p - nu (d_xx + d_yy + d_zz) q     q in (u,v,w)
//   cont  = d_x u + d_y v + d_z w
//
// The adjoint is Eq. (1) / Appendix A.2 extended the same way (ns_math.cuh writes it out); the
// boundary-gradient correction of Section 2.3 is the zero extension of the upstream arrays
// outside the rows: a shell node receives only the terms of the interior rows that read it, an
// interior node next to the shell loses the terms of the rows that do not exist.
//
// Kernel shape (both directions): a thread owns one float4 (four consecutive z) of a (y,z)
// tile and marches along x with a three-plane register window per array, rotated by unrolling;
// y+-1 neighbours of the current plane are read through L1, z+-1 neighbours come from the
// adjacent lanes' registers (the first / last lane of a warp fetch one float).  Arithmetic is
// packed fp32x2 and shared with the unsteady operator (its d_t terms get a zero constant).
#include "fpde_common.cuh"
#include "fpde_internal.h"
#include "ns_math.cuh"

#include <algorithm>
#include <cstdlib>

namespace fpde {

struct Ns3dParams {
    const float* a[7];    // forward: u,v,w,p ; adjoint: u,v,w, upstream of mom_x, mom_y, mom_z, continuity
    float* out[4];
    int n0, n1, n2, nc4;
    int planes_per_item, ncb, nmb, nitems;
    NsConsts k;
    float* partials;
    int prefetch;
};

__device__ __forceinline__ void ns3d_prefetch_l2(const float* ptr) {
    asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
}

template <bool BWD, int MINB>
__global__ void __launch_bounds__(128, MINB) ns3d_kernel(const Ns3dParams p) {
    constexpr int NA = BWD ? 7 : 4;
    constexpr int G0 = 3;                            // adjoint: first upstream array
    pdl_wait_then_trigger();
    const int n0 = p.n0, n1 = p.n1, n2 = p.n2, nc4 = p.nc4;
    int item = blockIdx.x;
    const int cb = item % p.ncb; item /= p.ncb;
    const int mb = item % p.nmb;
    const int ab = item / p.nmb;
    const int c4 = cb * blockDim.x + threadIdx.x;
    const int m = mb * blockDim.y + threadIdx.y;
    const bool valid = c4 < nc4 && m < n1;
    const int c4c = c4 < nc4 ? c4 : 0, mc = m < n1 ? m : 0;   // out-of-range threads shadow (0,0)
    const int col = 4 * c4c;
    const bool first_col = c4c == 0, last_col = c4c == nc4 - 1;
    const int lane = threadIdx.x & 31;
    const bool lfetch = lane == 0 && !first_col;
    const bool rfetch = lane == 31 && !last_col;
    const int PS = n1 * n2;
    const int rowoff = mc * n2 + col;
    const int ymoff = max(mc - 1, 0) * n2 + col;
    const int ypoff = min(mc + 1, n1 - 1) * n2 + col;
    // rows of y that carry no residual: upstream arrays count as zero there
    const bool y_dead = mc < 1 || mc > n1 - 2;
    const bool ym_dead = mc - 1 < 1, yp_dead = mc + 1 > n1 - 2;
    const int a0 = ab * p.planes_per_item;
    const int a1 = min(a0 + p.planes_per_item, n0);

    // zero extension of an upstream float4: whole vector when its plane / row is outside the rows,
    // else the elements at z = 0 and z = n2-1
    auto mask = [&](V4 v, bool dead) -> V4 {
        if (dead) v = v4zero();
        if (first_col) v.lo.x = 0.f;
        if (last_col) v.hi.y = 0.f;
        return v;
    };
    auto load_own = [&](int k, int r) -> V4 {
        const int rr = max(0, min(n0 - 1, r));
        V4 v = ldv4(p.a[k] + rr * PS + rowoff);
        if (BWD && k >= G0) v = mask(v, y_dead || r < 1 || r > n0 - 2);
        return v;
    };

    V4 A[NA], B[NA], Cc[NA];
#pragma unroll
    for (int k = 0; k < NA; ++k) { A[k] = load_own(k, a0 - 1); B[k] = load_own(k, a0); }
    float2 acc[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[e] = make_float2(0.f, 0.f);

    // one x step: W0 = plane a-1, W1 = plane a, W2 receives plane a+1
    auto step = [&](int a, const V4 (&W0)[NA], const V4 (&W1)[NA], V4 (&W2)[NA]) {
        const int pl = a * PS;
        const bool x_dead = a < 1 || a > n0 - 2;
        if (p.prefetch > 0 && (threadIdx.x & 7) == 0 && a + 1 + p.prefetch <= min(a1, n0 - 1)) {
            const int po = (a + 1 + p.prefetch) * PS + rowoff;
#pragma unroll
            for (int k = 0; k < NA; ++k) ns3d_prefetch_l2(p.a[k] + po);
        }
        V4 Ym[NA], Yp[NA], Zm[NA], Zp[NA];
#pragma unroll
        for (int k = 0; k < NA; ++k) {
            W2[k] = load_own(k, a + 1);
            Ym[k] = ldv4(p.a[k] + pl + ymoff);
            Yp[k] = ldv4(p.a[k] + pl + ypoff);
            if (BWD && k >= G0) { Ym[k] = mask(Ym[k], x_dead || ym_dead); Yp[k] = mask(Yp[k], x_dead || yp_dead); }
            float l1 = __shfl_up_sync(FULL_MASK, W1[k].hi.y, 1);
            float r1 = __shfl_down_sync(FULL_MASK, W1[k].lo.x, 1);
            const bool dead = BWD && k >= G0 && (x_dead || y_dead);
            if (lfetch) l1 = dead ? 0.f : __ldg(p.a[k] + pl + rowoff - 1);
            if (rfetch) r1 = dead ? 0.f : __ldg(p.a[k] + pl + rowoff + 4);
            if (BWD && k >= G0) { if (first_col) l1 = 0.f; if (last_col) r1 = 0.f; }
            Zm[k] = shift_left(W1[k], l1);
            Zp[k] = shift_right(W1[k], r1);
        }
        float2 o[4][2];
        const float2 nodt[3] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float2 w0[NA], w1[NA], w2[NA], ym[NA], yp[NA], zm[NA], zp[NA], oo[4];
            v4_half<NA>(W0, h, w0); v4_half<NA>(W1, h, w1); v4_half<NA>(W2, h, w2);
            v4_half<NA>(Ym, h, ym); v4_half<NA>(Yp, h, yp); v4_half<NA>(Zm, h, zm); v4_half<NA>(Zp, h, zp);
            if constexpr (BWD) ns_bwd_pair(p.k, w0, w1, w2, ym, yp, zm, zp, nodt, oo);
            else ns_fwd_pair(p.k, w0, w1, w2, ym, yp, zm, zp, nodt, oo);
#pragma unroll
            for (int e = 0; e < 4; ++e) o[e][h] = oo[e];
        }
        if (!BWD) {                                  // the outer shell carries no row
            const bool rowless = x_dead || y_dead;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (rowless) { o[e][0] = make_float2(0.f, 0.f); o[e][1] = o[e][0]; }
                if (first_col) o[e][0].x = 0.f;
                if (last_col) o[e][1].y = 0.f;
            }
        }
        if (valid) {
            const int off = pl + rowoff;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                stv4(p.out[e] + off, o[e][0], o[e][1]);
                if (!BWD) acc[e] = fma2(o[e][0], o[e][0], fma2(o[e][1], o[e][1], acc[e]));
            }
        }
    };

    for (int a = a0; a < a1; a += 3) {
        step(a, A, B, Cc);
        if (a + 1 < a1) step(a + 1, B, Cc, A);
        if (a + 2 < a1) step(a + 2, Cc, A, B);
    }
    if (!BWD && p.partials != nullptr) {
        float s[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) s[e] = acc[e].x + acc[e].y;
        block_reduce_store<4>(s, p.partials, p.nitems, blockIdx.x);
    }
}

static int env_int(const char* name, int dflt) {
    const char* s = std::getenv(name);
    if (!s || !*s) return dflt;
    const int v = std::atoi(s);
    return v > 0 ? v : dflt;
}

static void ns3d_geometry(const int* n, Ns3dParams& p, dim3& block) {
    p.n0 = n[0]; p.n1 = n[1]; p.n2 = n[2]; p.nc4 = n[2] / 4;
    int tx = env_int("FPDE_NS3D_TX", 32);
    tx = std::max(32, std::min(128, (tx / 32) * 32));
    int ty = env_int("FPDE_NS3D_TY", 4);
    ty = std::max(1, std::min(128 / tx, ty));
    block = dim3(tx, ty, 1);
    p.planes_per_item = env_int("FPDE_NS3D_PLANES", 16);
    p.ncb = (p.nc4 + tx - 1) / tx;
    p.nmb = (p.n1 + ty - 1) / ty;
    p.nitems = p.ncb * p.nmb * ((p.n0 + p.planes_per_item - 1) / p.planes_per_item);
    const char* pf = std::getenv("FPDE_NS3D_PREFETCH");
    p.prefetch = pf && *pf ? std::atoi(pf) : 3;
    if (p.prefetch < 0 || p.prefetch >= p.n0) p.prefetch = 0;
}

int ns3d_items(const int* n) {
    Ns3dParams p{}; dim3 block;
    ns3d_geometry(n, p, block);
    return p.nitems;
}

// the unsteady operator's constants with every d_t constant zero
static void ns3d_consts(const Problem& q, const double* gscale, NsConsts& k) {
    const double h4[4] = {q.h[0], q.h[1], q.h[2], 1.0};
    ns_fill_consts(k, h4, q.coef[0], gscale);
    k.iht = make_float2(0.f, 0.f);
    for (int e = 0; e < 3; ++e) k.a_t[e] = make_float2(0.f, 0.f);
}

cudaError_t launch_ns3d_fwd(const Problem& q) {
    Ns3dParams p{}; dim3 block;
    ns3d_geometry(q.n, p, block);
    for (int k = 0; k < 4; ++k) { p.a[k] = q.in[k]; p.out[k] = q.out[k]; }
    const double ones[4] = {1.0, 1.0, 1.0, 1.0};
    ns3d_consts(q, ones, p.k);
    p.partials = q.partials;
    if (env_int("FPDE_NS3D_MINB_F", 3) == 4) return launch_kernel(ns3d_kernel<false, 4>, dim3(p.nitems), block, q.stream, p);
    return launch_kernel(ns3d_kernel<false, 3>, dim3(p.nitems), block, q.stream, p);
}

cudaError_t launch_ns3d_bwd(const Problem& q) {
    Ns3dParams p{}; dim3 block;
    ns3d_geometry(q.n, p, block);
    for (int k = 0; k < 3; ++k) p.a[k] = q.in[k];
    for (int k = 0; k < 4; ++k) { p.a[3 + k] = q.aux[k]; p.out[k] = q.out[k]; }
    ns3d_consts(q, q.gscale, p.k);
    p.partials = nullptr;
    if (env_int("FPDE_NS3D_MINB_B", 2) == 3) return launch_kernel(ns3d_kernel<true, 3>, dim3(p.nitems), block, q.stream, p);
    return launch_kernel(ns3d_kernel<true, 2>, dim3(p.nitems), block, q.stream, p);
}

}  // namespace fpde
