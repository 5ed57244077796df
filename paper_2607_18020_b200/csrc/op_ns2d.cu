// Steady incompressible Navier-Stokes on an (x,y) array: the operator the paper works through
// (Section 2.1 residuals, Eq. 1 / Appendix A.3 adjoint, Appendix A.4 pseudocode).
//   res_u = u u_x + v u_y + p_x - nu (u_xx + u_yy)
//   res_v = u v_x + v v_y + p_y - nu (v_xx + v_yy)
//   res_div = u_x + v_y
// centred differences, rows at the interior nodes; the outer ring is data.
//
// Adjoint in gather form (Eq. 1 for u; v and p derived the same way), G = upstream arrays,
// zero outside the rows (the boundary-gradient correction of Section 2.3 is that zero
// extension: ring nodes receive only the terms of the interior rows that read them):
//   g_u = G_u u_x + G_v v_x + [(G_u u)(i-1) - (G_u u)(i+1)]/(2dx) + [(G_u v)(j-1) - (G_u v)(j+1)]/(2dy)
//         - nu Lap G_u + [G_d(i-1) - G_d(i+1)]/(2dx)
//   g_v = G_u u_y + G_v v_y + [(G_v u)(i-1) - (G_v u)(i+1)]/(2dx) + [(G_v v)(j-1) - (G_v v)(j+1)]/(2dy)
//         - nu Lap G_v + [G_d(j-1) - G_d(j+1)]/(2dy)
//   g_p = [G_u(i-1) - G_u(i+1)]/(2dx) + [G_v(j-1) - G_v(j+1)]/(2dy)
//
// Kernel shape: as the other 2-D kernels, a thread owns a float4 column, marches down a chunk of
// rows (axis 0 = x) with a three-row register window per array; y neighbours come from the
// adjacent lanes.  Arithmetic is packed fp32x2; second differences are formed as
// (q[-1]-q[0]) + (q[+1]-q[0]) because the viscous term is small against the others.
#include "fpde_common.cuh"
#include "fpde_internal.h"

#include <algorithm>
#include <cstdlib>

namespace fpde {

struct Ns2dParams {
    const float* in[5];     // forward: u,v,p ; adjoint: u,v, upstream of res_u, res_v, res_div
    float* out[3];
    float2 gs[3];           // adjoint: upstream scales
    float2 ihx, ihy;        // 1/(2h)
    float2 nvx, nvy;        // -nu/h^2
    int n0, n1, nc4;
    int rows_per_item, ncb, nitems;
    float* partials;
    int prefetch;           // rows ahead of the window to pull into L2 (0 = off)
};

template <bool BWD, bool O32 = false>
__global__ void __launch_bounds__(128) ns2d_kernel(const Ns2dParams p) {
    constexpr int NA = BWD ? 5 : 3;
    pdl_wait_then_trigger();
    const int n0 = p.n0, n1 = p.n1, nc4 = p.nc4;
    const int item = blockIdx.x;
    const int cb = item % p.ncb, rc = item / p.ncb;
    const int c4 = cb * blockDim.x + threadIdx.x;
    const int lane = threadIdx.x & 31;
    const bool cvalid = c4 < nc4;
    const int col = cvalid ? 4 * c4 : 0;
    const bool first_col = c4 == 0, last_col = c4 == nc4 - 1;
    const int a0 = rc * p.rows_per_item;
    const int a1 = min(a0 + p.rows_per_item, n0);
    // The one float beyond the float4 that the first / last lane of a warp cannot get by shuffle:
    // one predicated load per array, issued with the other loads of the row (a load inside a
    // divergent branch would be waited for on its own).  At the ends of a row it stays 0.
    const bool efetch = cvalid && ((lane == 0 && !first_col) || (lane == 31 && !last_col));
    const int eoff = col + (lane == 0 ? -1 : 4);

    // array k at row r (clamped into the grid).  Upstream arrays (adjoint, k >= 2) are scaled and
    // read as zero outside the rows of the operator.
    auto load = [&](int k, int r) -> V4 {
        const int rr = max(0, min(n0 - 1, r));
        V4 v = ldv4(at_off<O32>(p.in[k], rr * n1 + col));
        if (BWD && k >= 2) {
            v = v4mul(v, p.gs[k - 2]);
            if (r < 1 || r > n0 - 2) v = v4zero();
            if (first_col) v.lo.x = 0.f;
            if (last_col) v.hi.y = 0.f;
        }
        return v;
    };

    auto prefetch_row = [&](int r) {                 // one lane per 128-byte line
        if ((threadIdx.x & 7) == 0 && cvalid && r < n0) {
#pragma unroll
            for (int k = 0; k < NA; ++k) asm volatile("prefetch.global.L2 [%0];" ::"l"(at_off<O32>(p.in[k], r * n1 + col)));
        }
    };
    if (p.prefetch > 0)
        for (int d = 1; d <= p.prefetch; ++d) if (a0 + d <= a1) prefetch_row(a0 + d);
    V4 prev[NA], cur[NA], nxt[NA];
#pragma unroll
    for (int k = 0; k < NA; ++k) { prev[k] = load(k, a0 - 1); cur[k] = load(k, a0); }
    float2 acc[3];
#pragma unroll
    for (int e = 0; e < 3; ++e) acc[e] = make_float2(0.f, 0.f);

    for (int row = a0; row < a1; ++row) {
        if (p.prefetch > 0 && row + 1 + p.prefetch <= a1) prefetch_row(row + 1 + p.prefetch);
        V4 L[NA], R[NA];
        float E[NA];
#pragma unroll
        for (int k = 0; k < NA; ++k) {
            nxt[k] = load(k, row + 1);
            E[k] = 0.f;
            if (efetch) E[k] = __ldg(at_off<O32>(p.in[k], row * n1 + eoff));
        }
#pragma unroll
        for (int k = 0; k < NA; ++k) {
            if (BWD && k >= 2) {
                E[k] *= p.gs[k - 2].x;
                if (row < 1 || row > n0 - 2) E[k] = 0.f;
            }
            float l1 = __shfl_up_sync(FULL_MASK, cur[k].hi.y, 1);
            float r1 = __shfl_down_sync(FULL_MASK, cur[k].lo.x, 1);
            if (lane == 0) l1 = E[k];
            if (lane == 31) r1 = E[k];
            if (last_col) r1 = 0.f;                   // a ragged row ends inside a warp
            L[k] = shift_left(cur[k], l1);
            R[k] = shift_right(cur[k], r1);
        }
        float2 o[3][2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            auto H = [&](const V4& v) -> float2 { return h == 0 ? v.lo : v.hi; };
            if (!BWD) {
                const float2 u = H(cur[0]), v = H(cur[1]);
                const float2 us = mul2(u, p.ihx), vs = mul2(v, p.ihy);
                float2 dxs[2], dys[2];
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    const float2 c = H(cur[q]);
                    const float2 xm = sub2(H(prev[q]), c), xp = sub2(H(nxt[q]), c);
                    const float2 ym = sub2(H(L[q]), c), yp = sub2(H(R[q]), c);
                    const float2 dx = sub2(xp, xm), dy = sub2(yp, ym);
                    float2 r = mul2(add2(xm, xp), p.nvx);
                    r = fma2(add2(ym, yp), p.nvy, r);
                    r = fma2(us, dx, r);
                    r = fma2(vs, dy, r);
                    dxs[q] = dx; dys[q] = dy;
                    o[q][h] = r;
                }
                o[0][h] = fma2(sub2(H(nxt[2]), H(prev[2])), p.ihx, o[0][h]);     // p_x
                o[1][h] = fma2(sub2(H(R[2]), H(L[2])), p.ihy, o[1][h]);          // p_y
                o[2][h] = fma2(dys[1], p.ihy, mul2(dxs[0], p.ihx));              // u_x + v_y
            } else {
                // velocities and upstream arrays at the four neighbours
                const float2 uxm = H(prev[0]), uxp = H(nxt[0]);
                const float2 vym = H(L[1]), vyp = H(R[1]);
                const float2 gu = H(cur[2]), gv = H(cur[3]);
                const float2 du_dx = sub2(uxp, uxm), dv_dx = sub2(H(nxt[1]), H(prev[1]));
                const float2 du_dy = sub2(H(R[0]), H(L[0])), dv_dy = sub2(vyp, vym);
                float2 gq[2];
                float2 gp = make_float2(0.f, 0.f);
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    const float2 c = H(cur[2 + q]);
                    const float2 gxm = H(prev[2 + q]), gxp = H(nxt[2 + q]);
                    const float2 gym = H(L[2 + q]), gyp = H(R[2 + q]);
                    const float2 advx = sub2(mul2(gxm, uxm), mul2(gxp, uxp));
                    const float2 advy = sub2(mul2(gym, vym), mul2(gyp, vyp));
                    const float2 dxm = sub2(gxm, c), dxp = sub2(gxp, c);
                    const float2 dym = sub2(gym, c), dyp = sub2(gyp, c);
                    float2 r = mul2(advx, p.ihx);
                    r = fma2(advy, p.ihy, r);
                    r = fma2(add2(dxm, dxp), p.nvx, r);
                    r = fma2(add2(dym, dyp), p.nvy, r);
                    gq[q] = r;
                    // pressure gradient: G_u along x, G_v along y
                    if (q == 0) gp = fma2(sub2(dxm, dxp), p.ihx, gp);
                    else gp = fma2(sub2(dym, dyp), p.ihy, gp);
                }
                // local terms and continuity row
                gq[0] = fma2(fma2(gv, dv_dx, mul2(gu, du_dx)), p.ihx, gq[0]);
                gq[0] = fma2(sub2(H(prev[4]), H(nxt[4])), p.ihx, gq[0]);
                gq[1] = fma2(fma2(gv, dv_dy, mul2(gu, du_dy)), p.ihy, gq[1]);
                gq[1] = fma2(sub2(H(L[4]), H(R[4])), p.ihy, gq[1]);
                o[0][h] = gq[0]; o[1][h] = gq[1]; o[2][h] = gp;
            }
        }
        if (!BWD) {                                   // the outer ring carries no row
            const bool rowless = row < 1 || row > n0 - 2;
#pragma unroll
            for (int e = 0; e < 3; ++e) {
                if (rowless) { o[e][0] = make_float2(0.f, 0.f); o[e][1] = o[e][0]; }
                if (first_col) o[e][0].x = 0.f;
                if (last_col) o[e][1].y = 0.f;
            }
        }
        if (cvalid) {
#pragma unroll
            for (int e = 0; e < 3; ++e) {
                stv4(at_off<O32>(p.out[e], row * n1 + col), o[e][0], o[e][1]);
                if (!BWD) acc[e] = fma2(o[e][0], o[e][0], fma2(o[e][1], o[e][1], acc[e]));
            }
        }
#pragma unroll
        for (int k = 0; k < NA; ++k) { prev[k] = cur[k]; cur[k] = nxt[k]; }
    }
    if (!BWD && p.partials != nullptr) {
        float s[3];
#pragma unroll
        for (int e = 0; e < 3; ++e) s[e] = acc[e].x + acc[e].y;
        block_reduce_store<3>(s, p.partials, p.nitems, item);
    }
}

static int env_int(const char* name, int dflt) {
    const char* s = std::getenv(name);
    if (!s || !*s) return dflt;
    const int v = std::atoi(s);
    return v > 0 ? v : dflt;
}

static float2 sp(double v) { return make_float2((float)v, (float)v); }

static void ns2d_geometry(const int* n, Ns2dParams& p, int& block) {
    p.n0 = n[0]; p.n1 = n[1]; p.nc4 = n[1] / 4;
    block = 128;
    p.rows_per_item = env_int("FPDE_NS2D_ROWS", 4);
    p.ncb = (p.nc4 + block - 1) / block;
    p.nitems = p.ncb * ((p.n0 + p.rows_per_item - 1) / p.rows_per_item);
    const char* pf = std::getenv("FPDE_NS2D_PREFETCH");
    p.prefetch = pf && *pf ? std::atoi(pf) : 1;
    if (p.prefetch < 0) p.prefetch = 0;
}

// 32-bit byte offsets are enough for arrays of at most 2^30 floats
static bool ns2d_off32(const Problem& q) {
    const char* s = std::getenv("FPDE_NS2D_OFF32");
    return !(s && s[0] == '0') && (int64_t)q.n[0] * q.n[1] <= ((int64_t)1 << 30);
}

int ns2d_items(const int* n) {
    Ns2dParams p{}; int block;
    ns2d_geometry(n, p, block);
    return p.nitems;
}

static void ns2d_consts(const Problem& q, Ns2dParams& p) {
    p.ihx = sp(0.5 / q.h[0]); p.ihy = sp(0.5 / q.h[1]);
    p.nvx = sp(-q.coef[0] / (q.h[0] * q.h[0])); p.nvy = sp(-q.coef[0] / (q.h[1] * q.h[1]));
}

cudaError_t launch_ns2d_fwd(const Problem& q) {
    Ns2dParams p{}; int block;
    ns2d_geometry(q.n, p, block);
    ns2d_consts(q, p);
    for (int k = 0; k < 3; ++k) { p.in[k] = q.in[k]; p.out[k] = q.out[k]; }
    p.partials = q.partials;
    if (ns2d_off32(q)) return launch_kernel(ns2d_kernel<false, true>, dim3(p.nitems), dim3(block), q.stream, p);
    return launch_kernel(ns2d_kernel<false>, dim3(p.nitems), dim3(block), q.stream, p);
}

cudaError_t launch_ns2d_bwd(const Problem& q) {
    Ns2dParams p{}; int block;
    ns2d_geometry(q.n, p, block);
    ns2d_consts(q, p);
    p.in[0] = q.in[0]; p.in[1] = q.in[1];
    for (int k = 0; k < 3; ++k) { p.in[2 + k] = q.aux[k]; p.out[k] = q.out[k]; p.gs[k] = sp(q.gscale[k]); }
    p.partials = nullptr;
    if (ns2d_off32(q)) return launch_kernel(ns2d_kernel<true, true>, dim3(p.nitems), dim3(block), q.stream, p);
    return launch_kernel(ns2d_kernel<true>, dim3(p.nitems), dim3(block), q.stream, p);
}

}  // namespace fpde
