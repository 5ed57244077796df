// Per-node arithmetic of the unsteady Navier-Stokes operator, shared by the kernels that stage
// their neighbours through L1 and those that stage them through shared memory.  Everything is
// packed fp32x2: a float4 (four consecutive t of one z) is two register-aligned pairs.
//
// Forward (Section 2.1 extended by d_t, w, d_z), per momentum component q along axis a_q:
//   mom_q = d_t q + u d_x q + v d_y q + w d_z q + d_{a_q} p - nu (d_xx + d_yy + d_zz) q
//   cont  = d_x u + d_y v + d_z w
// Adjoint (Eq. 1 / Appendix A.3 extended the same way), G = upstream arrays (zero at the first
// and last t), c = (u,v,w):
//   g_q(P) = sum_e G_e(P) (d_{a_q} e)(P)                                   local terms
//          + sum_a [ (G_q c_a)(P-a) - (G_q c_a)(P+a) ] / (2 h_a)           transposed advection
//          - nu sum_a [ G_q(P-a) - 2 G_q(P) + G_q(P+a) ] / h_a^2           transposed diffusion
//          + [ G_q(P-t) - G_q(P+t) ] / (2 dt)                              transposed d_t
//          + [ G_c(P-a_q) - G_c(P+a_q) ] / (2 h_{a_q})                     continuity row
//   g_p(P) = sum_q [ G_q(P-a_q) - G_q(P+a_q) ] / (2 h_{a_q})
// with G_e = gscale_e * gres_e; the scales are folded into the constants.
//
// Second differences are formed as (q[-1]-q[0]) + (q[+1]-q[0]) before scaling: the viscous term
// is small against the other terms and must not carry the rounding of the large centre value.
//
// Nodes at the first / last t carry no row.  Every spatial read of an output node happens at the
// node's own t, so in the adjoint that rule only changes (i) the t-neighbour of the nodes next
// to the two end planes and (ii) the end planes themselves, where only the transposed d_t term
// survives: the boundary-gradient correction of this operator is a fix-up of two lanes.
#pragma once
#include "fpde_common.cuh"

namespace fpde {

struct NsConsts {
    // forward, splatted
    float2 ih[3];         // 1/(2 h_a)
    float2 iht;           // 1/(2 dt)
    float2 nv[3];         // -nu / h_a^2
    // adjoint (upstream scales folded in), splatted
    float2 a_ih[3][3];    // [q][a]  gs_q / (2 h_a)
    float2 a_nv[3][3];    // [q][a]  -nu gs_q / h_a^2
    float2 a_t[3];        // [q]     gs_q / (2 dt)
    float2 l_g[3];        // [e]     gs_e
    float2 c_ih[3];       // [a]     gs_c / (2 h_a)
    float2 nih[3];        // [a]     -1/(2 h_a)
    float2 nv2c;          //         2 nu sum_a 1/h_a^2
};

// ---- one packed pair (two consecutive t of one z) of every array -----------------------------
// w0/w1/w2: planes x-1, x, x+1 at the own column; ym/yp/zm/zp: y-+1 and z-+1 neighbours of plane x.
// Forward: arrays u,v,w,p; dt[q] = q(t+1) - q(t-1) for the pair.  o[e]: mom_x, mom_y, mom_z, continuity.
__device__ __forceinline__ void ns_fwd_pair(const NsConsts& k, const float2 (&w0)[4], const float2 (&w1)[4],
                                            const float2 (&w2)[4], const float2 (&ym)[4], const float2 (&yp)[4],
                                            const float2 (&zm)[4], const float2 (&zp)[4], const float2 (&dt)[3],
                                            float2 (&o)[4]) {
    const float2 us = mul2(w1[0], k.ih[0]);     // advecting velocities, pre-scaled by 1/(2h)
    const float2 vs = mul2(w1[1], k.ih[1]);
    const float2 ws = mul2(w1[2], k.ih[2]);
    float2 dself[3];                            // d_x u, d_y v, d_z w (raw differences)
#pragma unroll
    for (int q = 0; q < 3; ++q) {
        const float2 c = w1[q];
        const float2 xm = sub2(w0[q], c), xp = sub2(w2[q], c);
        const float2 ymd = sub2(ym[q], c), ypd = sub2(yp[q], c);
        const float2 zmd = sub2(zm[q], c), zpd = sub2(zp[q], c);
        const float2 dx = sub2(xp, xm), dy = sub2(ypd, ymd), dz = sub2(zpd, zmd);
        float2 r = mul2(add2(xm, xp), k.nv[0]);
        r = fma2(add2(ymd, ypd), k.nv[1], r);
        r = fma2(add2(zmd, zpd), k.nv[2], r);
        r = fma2(us, dx, r);
        r = fma2(vs, dy, r);
        r = fma2(ws, dz, r);
        r = fma2(dt[q], k.iht, r);
        dself[q] = q == 0 ? dx : (q == 1 ? dy : dz);
        o[q] = r;
    }
    o[0] = fma2(sub2(w2[3], w0[3]), k.ih[0], o[0]);     // d_x p
    o[1] = fma2(sub2(yp[3], ym[3]), k.ih[1], o[1]);     // d_y p
    o[2] = fma2(sub2(zp[3], zm[3]), k.ih[2], o[2]);     // d_z p
    o[3] = fma2(dself[2], k.ih[2], fma2(dself[1], k.ih[1], mul2(dself[0], k.ih[0])));
}

// Adjoint: arrays 0..2 = u,v,w ; 3..6 = upstream of mom_x, mom_y, mom_z, continuity;
// dt[q] = G_q(t-1) - G_q(t+1) for the pair (end planes already counted as zero).  o[f]: g_u, g_v, g_w, g_p.
// MERGED: transposed advection and diffusion of component q share their neighbours,
//   sum_a [ G_q(P-a) (c_a(P-a)/(2h_a) - nu/h_a^2) + G_q(P+a) (-c_a(P+a)/(2h_a) - nu/h_a^2) ] + 2 nu sum_a 1/h_a^2 G_q(P),
// and the six coefficients are the same for the three components: two multiply-adds per
// neighbour instead of six instructions.  This is a plain weighted stencil sum: its rounding error
// is eps * sum |w_i G_i|, i.e. it grows with nu/h^2 when the upstream array is smooth (measured on
// smooth fields: gradient rel-L2 2e-7 at nu/h^2 = 4, 5e-6 at nu/h^2 = 1000, steady operator).  The
// other form differences first, (G(P-a) - G(P)) + (G(P+a) - G(P)), and keeps separate products:
// error relative to the differences, three more instructions per neighbour pair.
template <bool MERGED = false>
__device__ __forceinline__ void ns_bwd_pair(const NsConsts& k, const float2 (&w0)[7], const float2 (&w1)[7],
                                            const float2 (&w2)[7], const float2 (&ym)[7], const float2 (&yp)[7],
                                            const float2 (&zm)[7], const float2 (&zp)[7], const float2 (&dt)[3],
                                            float2 (&o)[4]) {
    // neighbours of array i along axis a: minus / plus
    auto NM = [&](int i, int a_) -> float2 { return a_ == 0 ? w0[i] : (a_ == 1 ? ym[i] : zm[i]); };
    auto NP = [&](int i, int a_) -> float2 { return a_ == 0 ? w2[i] : (a_ == 1 ? yp[i] : zp[i]); };
    float2 gs[3];                               // scaled centre sensitivities
#pragma unroll
    for (int e = 0; e < 3; ++e) gs[e] = mul2(w1[3 + e], k.l_g[e]);
    float2 cm[3], ncp[3];                       // advecting velocity at P-a, minus the one at P+a
#pragma unroll
    for (int a_ = 0; a_ < 3; ++a_) {
        cm[a_] = NM(a_, a_);
        const float2 cp = NP(a_, a_);
        ncp[a_] = make_float2(-cp.x, -cp.y);
    }
    float2 am[3], apl[3];                       // MERGED: what G_q(P-a) and G_q(P+a) are multiplied by
    if (MERGED) {
#pragma unroll
        for (int a_ = 0; a_ < 3; ++a_) {
            am[a_] = fma2(cm[a_], k.ih[a_], k.nv[a_]);
            apl[a_] = fma2(NP(a_, a_), k.nih[a_], k.nv[a_]);
        }
    }
    float2 gp = make_float2(0.f, 0.f);
#pragma unroll
    for (int q = 0; q < 3; ++q) {
        const float2 c = w1[3 + q];
        float2 r = mul2(dt[q], k.a_t[q]);
        if (MERGED) {
            float2 T = mul2(c, k.nv2c);
#pragma unroll
            for (int a_ = 0; a_ < 3; ++a_) {
                const float2 gm = NM(3 + q, a_), gpl = NP(3 + q, a_);
                T = fma2(gm, am[a_], T);
                T = fma2(gpl, apl[a_], T);
                if (a_ == q) gp = fma2(sub2(gm, gpl), k.a_ih[q][q], gp);
            }
            r = fma2(T, k.l_g[q], r);
        } else {
#pragma unroll
            for (int a_ = 0; a_ < 3; ++a_) {
                const float2 gm = NM(3 + q, a_), gpl = NP(3 + q, a_);
                const float2 adv = fma2(gpl, ncp[a_], mul2(gm, cm[a_]));
                r = fma2(adv, k.a_ih[q][a_], r);
                const float2 dm = sub2(gm, c), dp = sub2(gpl, c);
                r = fma2(add2(dm, dp), k.a_nv[q][a_], r);
                if (a_ == q) gp = fma2(sub2(dm, dp), k.a_ih[q][q], gp);
            }
        }
        // local terms and continuity row along this component's own axis
        float2 loc = mul2(gs[0], sub2(NP(0, q), NM(0, q)));
        loc = fma2(gs[1], sub2(NP(1, q), NM(1, q)), loc);
        loc = fma2(gs[2], sub2(NP(2, q), NM(2, q)), loc);
        r = fma2(loc, k.ih[q], r);
        r = fma2(sub2(NM(6, q), NP(6, q)), k.c_ih[q], r);
        o[q] = r;
    }
    o[3] = gp;
}

// ---- a float4 (four consecutive t) per thread: two pairs -------------------------------------
// l1/r1: t-1 of lane x and t+1 of lane w for u,v,w (forward) / the momentum upstream arrays.
__device__ __forceinline__ void ns_fwd_math(const NsConsts& k, const V4 (&W0)[4], const V4 (&W1)[4], const V4 (&W2)[4],
                                            const V4 (&Ym)[4], const V4 (&Yp)[4], const V4 (&Zm)[4], const V4 (&Zp)[4],
                                            const float (&l1)[3], const float (&r1)[3], bool t_first, bool t_last,
                                            float2 (&o)[4][2]) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        float2 w0[4], w1[4], w2[4], ym[4], yp[4], zm[4], zp[4], dt[3], oo[4];
        v4_half<4>(W0, h, w0); v4_half<4>(W1, h, w1); v4_half<4>(W2, h, w2);
        v4_half<4>(Ym, h, ym); v4_half<4>(Yp, h, yp); v4_half<4>(Zm, h, zm); v4_half<4>(Zp, h, zp);
#pragma unroll
        for (int q = 0; q < 3; ++q) {           // q(t+1) - q(t-1)
            const V4 c = W1[q];
            dt[q] = h == 0 ? make_float2(c.lo.y - l1[q], c.hi.x - c.lo.x) : make_float2(c.hi.y - c.lo.y, r1[q] - c.hi.x);
        }
        ns_fwd_pair(k, w0, w1, w2, ym, yp, zm, zp, dt, oo);
#pragma unroll
        for (int e = 0; e < 4; ++e) o[e][h] = oo[e];
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {               // t = 0 and t = n3-1 carry no row
        if (t_first) o[e][0].x = 0.f;
        if (t_last) o[e][1].y = 0.f;
    }
}

__device__ __forceinline__ void ns_bwd_math(const NsConsts& k, const V4 (&W0)[7], const V4 (&W1)[7], const V4 (&W2)[7],
                                            const V4 (&Ym)[7], const V4 (&Yp)[7], const V4 (&Zm)[7], const V4 (&Zp)[7],
                                            const float (&l1)[3], const float (&r1)[3], bool t_first, bool t_last,
                                            float2 (&o)[4][2]) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        float2 w0[7], w1[7], w2[7], ym[7], yp[7], zm[7], zp[7], dt[3], oo[4];
        v4_half<7>(W0, h, w0); v4_half<7>(W1, h, w1); v4_half<7>(W2, h, w2);
        v4_half<7>(Ym, h, ym); v4_half<7>(Yp, h, yp); v4_half<7>(Zm, h, zm); v4_half<7>(Zp, h, zp);
#pragma unroll
        for (int q = 0; q < 3; ++q) {           // G_q(t-1) - G_q(t+1), end planes counted as 0
            const V4 c = W1[3 + q];
            const float tm_y = t_first ? 0.f : c.lo.x;       // t-1 of lane y is the end plane t = 0
            const float tp_z = t_last ? 0.f : c.hi.y;        // t+1 of lane z is the end plane t = n3-1
            dt[q] = h == 0 ? make_float2(l1[q] - c.lo.y, tm_y - c.hi.x) : make_float2(c.lo.y - tp_z, c.hi.x - r1[q]);
        }
        ns_bwd_pair<true>(k, w0, w1, w2, ym, yp, zm, zp, dt, oo);
#pragma unroll
        for (int e = 0; e < 4; ++e) o[e][h] = oo[e];
    }
    // end planes of t: only the transposed d_t term exists there, and no pressure gradient
#pragma unroll
    for (int q = 0; q < 3; ++q) {
        const V4 c = W1[3 + q];
        if (t_first) o[q][0].x = -c.lo.y * k.a_t[q].x;
        if (t_last) o[q][1].y = c.hi.x * k.a_t[q].x;
    }
    if (t_first) o[3][0].x = 0.f;
    if (t_last) o[3][1].y = 0.f;
}

// Host side: fill the constants from spacings, viscosity and upstream scales.
inline void ns_fill_consts(NsConsts& k, const double* h, double nu, const double* gscale) {
    auto sp = [](double v) { return make_float2((float)v, (float)v); };
    for (int a = 0; a < 3; ++a) {
        k.ih[a] = sp(0.5 / h[a]);
        k.nv[a] = sp(-nu / (h[a] * h[a]));
        k.c_ih[a] = sp(gscale[3] * 0.5 / h[a]);
        k.nih[a] = sp(-0.5 / h[a]);
    }
    k.nv2c = sp(2.0 * nu * (1.0 / (h[0] * h[0]) + 1.0 / (h[1] * h[1]) + 1.0 / (h[2] * h[2])));
    k.iht = sp(0.5 / h[3]);
    for (int q = 0; q < 3; ++q) {
        k.a_t[q] = sp(gscale[q] * 0.5 / h[3]);
        k.l_g[q] = sp(gscale[q]);
        for (int a = 0; a < 3; ++a) {
            k.a_ih[q][a] = sp(gscale[q] * 0.5 / h[a]);
            k.a_nv[q][a] = sp(-nu * gscale[q] / (h[a] * h[a]));
        }
    }
}

}  // namespace fpde
