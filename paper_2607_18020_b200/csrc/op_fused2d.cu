// Loss-specialised single pass for the two-dimensional operators: residual (Section 2.1), the
// mean-square loss, and the loss gradient through the gather-form adjoint (Sections 2.2, 2.3)
// in ONE launch, without the residual arrays ever going to memory and coming back.  With the
// mean-square loss the upstream array of the adjoint is G_e = (2/N_r) r_e, so the adjoint at a
// node needs r at the node and its four neighbours; nothing else of the forward pass.
//
// How r gets to the adjoint without a round trip:
//   * along x (the marching axis) by pipelining: a thread owns a float4 column and marches down
//     the rows; in step i it forms r(i+1) from the field rows i, i+1, i+2 it holds in registers
//     and then g(i) from r(i-1), r(i), r(i+1), which it also holds.  Each r is computed once.
//   * along y (the contiguous axis) by shuffles inside a warp.  Warps overlap by one float4 on
//     each side: lanes 1..30 own their columns, lanes 0 and 31 only supply r to their neighbour
//     (so no value ever has to cross a warp, and no shared memory or barrier is needed).  The
//     overlap costs 2/32 of the arithmetic and of the L1 traffic, nothing in DRAM traffic.
// A chunk of rows recomputes r on one row above and below itself.
//
// Boundary handling is the zero extension of r outside the rows of the operator (omitted
// neighbours, Appendix A.5): on interior axes r is forced to 0 on the outer ring and outside
// the array, on periodic axes row and column indices wrap.
//
// Field rows are requested one step before they are first used (five-slot rotation, unrolled).
#include "fpde_common.cuh"
#include "fpde_internal.h"

#include <algorithm>
#include <cstdlib>

namespace fpde {

struct Fused2dParams {
    const float* f[3];      // fields
    const float* src[1];    // sources
    float* res[3];          // residual arrays, NULL = not stored
    float* g[3];            // dL/dfield
    float2 c[8];            // operator constants, splatted
    float2 gs;              // 2 / N_r
    int n0, n1, nc4;
    int rows_per_item, ncg, ncb, nitems;
    float* partials;
    int prefetch;           // rows ahead of the newest requested row to pull into L2 (0 = off)
};

constexpr int FUSED2D_OWN = 30;     // float4 columns a warp owns (lanes 1..30)

// ---- operators: one packed pair (two consecutive y) per call -----------------------------------
// fwd: field neighbours m/p along x (rows i-1, i+1), l/r along y  ->  residuals
// bwd: the same for the fields plus the residual neighbourhood     ->  dL/dfield / (2/N_r)

struct FusedPoisson {       // r = -Lap u - f ; g = -Lap G
    static constexpr int NF = 1, NS = 1, NE = 1;
    static constexpr bool PERIODIC = false, FIELD_LATERAL_IN_BWD = false, LATERAL_SUM = true;
    // l: the SUM of the two lateral neighbours (LATERAL_SUM operators get it in fl / rl; fr / rr unused)
    __device__ static __forceinline__ float2 lap(const float2* c, float2 m, float2 z, float2 p, float2 l, float2) {
        const float2 m2 = splat2(-2.f);
        return fma2(fma2(z, m2, add2(m, p)), c[0], mul2(fma2(z, m2, l), c[1]));
    }
    __device__ static __forceinline__ void fwd(const float2* c, const float2* fm, const float2* f0, const float2* fp,
                                               const float2* fl, const float2* fr, const float2* s, float2* r) {
        r[0] = fma2(lap(c, fm[0], f0[0], fp[0], fl[0], fr[0]), splat2(-1.f), make_float2(-s[0].x, -s[0].y));
    }
    __device__ static __forceinline__ void bwd(const float2* c, const float2* fm, const float2* f0, const float2* fp,
                                               const float2* fl, const float2* fr, const float2* rm, const float2* r0,
                                               const float2* rp, const float2* rl, const float2* rr, float2* g) {
        const float2 t = lap(c, rm[0], r0[0], rp[0], rl[0], rr[0]);
        g[0] = make_float2(-t.x, -t.y);
    }
};

struct FusedGrayScott {     // c: 1/h0^2, 1/h1^2, D_u, D_v, F, F+k
    static constexpr int NF = 2, NS = 0, NE = 2;
    static constexpr bool PERIODIC = true, FIELD_LATERAL_IN_BWD = false, LATERAL_SUM = true;
    __device__ static __forceinline__ void fwd(const float2* c, const float2* fm, const float2* f0, const float2* fp,
                                               const float2* fl, const float2* fr, const float2* s, float2* r) {
        const float2 u = f0[0], w = f0[1];
        const float2 lu = FusedPoisson::lap(c, fm[0], u, fp[0], fl[0], fr[0]);
        const float2 lw = FusedPoisson::lap(c, fm[1], w, fp[1], fl[1], fr[1]);
        const float2 uww = mul2(mul2(u, w), w);
        const float2 t = fma2(u, make_float2(-c[4].x, -c[4].y), c[4]);           // F (1 - u)
        r[0] = sub2(fma2(lu, c[2], t), uww);
        r[1] = fma2(lw, c[3], fma2(w, make_float2(-c[5].x, -c[5].y), uww));
    }
    // g_u = D_u Lap G_u + G_u (-v^2 - F) + G_v v^2 ;  g_v = D_v Lap G_v + G_u (-2uv) + G_v (2uv - (F+k))
    __device__ static __forceinline__ void bwd(const float2* c, const float2* fm, const float2* f0, const float2* fp,
                                               const float2* fl, const float2* fr, const float2* rm, const float2* r0,
                                               const float2* rp, const float2* rl, const float2* rr, float2* g) {
        const float2 u = f0[0], w = f0[1], a = r0[0], b = r0[1];
        const float2 la = FusedPoisson::lap(c, rm[0], a, rp[0], rl[0], rr[0]);
        const float2 lb = FusedPoisson::lap(c, rm[1], b, rp[1], rl[1], rr[1]);
        const float2 ww = mul2(w, w), uw2 = mul2(add2(u, u), w), bma = sub2(b, a);
        g[0] = fma2(la, c[2], fma2(ww, bma, mul2(a, make_float2(-c[4].x, -c[4].y))));
        g[1] = fma2(lb, c[3], fma2(uw2, bma, mul2(b, make_float2(-c[5].x, -c[5].y))));
    }
};

struct FusedNs2d {          // c: 1/(2 h0), 1/(2 h1), -nu/h0^2, -nu/h1^2 ; fields u,v,p ; residuals mom_x, mom_y, div
    static constexpr int NF = 3, NS = 0, NE = 3;
    static constexpr bool PERIODIC = false, FIELD_LATERAL_IN_BWD = true, LATERAL_SUM = false;
    __device__ static __forceinline__ void fwd(const float2* c, const float2* fm, const float2* f0, const float2* fp,
                                               const float2* fl, const float2* fr, const float2* s, float2* r) {
        const float2 us = mul2(f0[0], c[0]), vs = mul2(f0[1], c[1]);
        float2 dxs[2], dys[2];
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const float2 z = f0[q];
            const float2 xm = sub2(fm[q], z), xp = sub2(fp[q], z), ym = sub2(fl[q], z), yp = sub2(fr[q], z);
            const float2 dx = sub2(xp, xm), dy = sub2(yp, ym);
            float2 t = mul2(add2(xm, xp), c[2]);
            t = fma2(add2(ym, yp), c[3], t);
            t = fma2(us, dx, t);
            t = fma2(vs, dy, t);
            dxs[q] = dx; dys[q] = dy;
            r[q] = t;
        }
        r[0] = fma2(sub2(fp[2], fm[2]), c[0], r[0]);                 // p_x
        r[1] = fma2(sub2(fr[2], fl[2]), c[1], r[1]);                 // p_y
        r[2] = fma2(dys[1], c[1], mul2(dxs[0], c[0]));               // u_x + v_y
    }
    // Eq. (1) for u, and the analogous expressions for v and p, with G = r
    __device__ static __forceinline__ void bwd(const float2* c, const float2* fm, const float2* f0, const float2* fp,
                                               const float2* fl, const float2* fr, const float2* rm, const float2* r0,
                                               const float2* rp, const float2* rl, const float2* rr, float2* g) {
        const float2 uxm = fm[0], uxp = fp[0], vym = fl[1], vyp = fr[1];
        const float2 gu = r0[0], gv = r0[1];
        const float2 du_dx = sub2(uxp, uxm), dv_dx = sub2(fp[1], fm[1]);
        const float2 du_dy = sub2(fr[0], fl[0]), dv_dy = sub2(vyp, vym);
        float2 gq[2];
        float2 gp = make_float2(0.f, 0.f);
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const float2 z = r0[q];
            const float2 advx = sub2(mul2(rm[q], uxm), mul2(rp[q], uxp));
            const float2 advy = sub2(mul2(rl[q], vym), mul2(rr[q], vyp));
            const float2 dxm = sub2(rm[q], z), dxp = sub2(rp[q], z), dym = sub2(rl[q], z), dyp = sub2(rr[q], z);
            float2 t = mul2(advx, c[0]);
            t = fma2(advy, c[1], t);
            t = fma2(add2(dxm, dxp), c[2], t);
            t = fma2(add2(dym, dyp), c[3], t);
            gq[q] = t;
            if (q == 0) gp = fma2(sub2(dxm, dxp), c[0], gp);
            else gp = fma2(sub2(dym, dyp), c[1], gp);
        }
        gq[0] = fma2(fma2(gv, dv_dx, mul2(gu, du_dx)), c[0], gq[0]);
        gq[0] = fma2(sub2(rm[2], rp[2]), c[0], gq[0]);
        gq[1] = fma2(fma2(gv, dv_dy, mul2(gu, du_dy)), c[1], gq[1]);
        gq[1] = fma2(sub2(rl[2], rr[2]), c[1], gq[1]);
        g[0] = gq[0]; g[1] = gq[1]; g[2] = gp;
    }
};

// ---- engine ------------------------------------------------------------------------------------
template <class OP, int MINB, bool O32 = false>
__global__ void __launch_bounds__(128, MINB) fused2d_kernel(const Fused2dParams p) {
    constexpr int NF = OP::NF, NS = OP::NS, NE = OP::NE;
    constexpr int NSA = NS > 0 ? NS : 1;
    constexpr bool PER = OP::PERIODIC;
    pdl_wait_then_trigger();
    const int n0 = p.n0, n1 = p.n1, nc4 = p.nc4;
    const int item = blockIdx.x;
    const int cb = item % p.ncb, rc = item / p.ncb;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int wg = cb * 4 + warp;                           // column group of this warp
    const int c4 = wg * FUSED2D_OWN - 1 + lane;             // float4 column this lane holds
    const bool inside = c4 >= 0 && c4 < nc4;
    const bool own = lane >= 1 && lane <= FUSED2D_OWN && c4 < nc4;
    int c4r;                                                // column read from
    if (PER) { c4r = c4 % nc4; if (c4r < 0) c4r += nc4; }
    else c4r = max(0, min(nc4 - 1, c4));
    const int col = 4 * c4r;
    const bool first_col = c4 == 0, last_col = c4 == nc4 - 1;
    const int a0 = rc * p.rows_per_item;
    const int a1 = min(a0 + p.rows_per_item, n0);

    // row read for index j in [-2, n0 + 1] (what the march asks for): wrapped once, no division
    auto row_of = [&](int j) -> int {
        if (PER) return j < 0 ? j + n0 : (j >= n0 ? j - n0 : j);
        return max(0, min(n0 - 1, j));
    };
    auto load_row = [&](int j, V4 (&F)[NF], V4 (&S)[NSA]) {
        const int off = row_of(j) * n1 + col;
#pragma unroll
        for (int k = 0; k < NF; ++k) F[k] = ldv4(at_off<O32>(p.f[k], off));
#pragma unroll
        for (int k = 0; k < NS; ++k) S[k] = ldv4(at_off<O32>(p.src[k], off));
    };
    // left / right neighbours along y of a row held in registers (lanes 0 / 31 get their own
    // value back on the outer side: what depends on it is never used)
    auto lateral = [&](const V4& c, V4& L, V4& R) {
        const float l1 = __shfl_up_sync(FULL_MASK, c.hi.y, 1);
        const float r1 = __shfl_down_sync(FULL_MASK, c.lo.x, 1);
        if (OP::LATERAL_SUM) {                           // only l + r is wanted: four scalar adds, no shifted copies
            L.lo = make_float2(l1 + c.lo.y, c.lo.x + c.hi.x);
            L.hi = make_float2(c.lo.y + c.hi.y, c.hi.x + r1);
            R = L;
        } else {
            L = shift_left(c, l1);
            R = shift_right(c, r1);
        }
    };
    // r at row j from the field rows j-1, j, j+1; zero where the operator has no row
    auto residual_row = [&](int j, const V4 (&Fm)[NF], const V4 (&F0)[NF], const V4 (&Fp)[NF], const V4 (&S0)[NSA],
                            V4 (&R)[NE]) {
        V4 FL[NF], FR[NF];
#pragma unroll
        for (int k = 0; k < NF; ++k) lateral(F0[k], FL[k], FR[k]);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float2 fm[NF], f0[NF], fp[NF], fl[NF], fr[NF], s[NSA], r[NE];
            v4_half<NF>(Fm, h, fm); v4_half<NF>(F0, h, f0); v4_half<NF>(Fp, h, fp);
            v4_half<NF>(FL, h, fl); v4_half<NF>(FR, h, fr);
#pragma unroll
            for (int k = 0; k < NSA; ++k) s[k] = NS > 0 ? (h == 0 ? S0[k].lo : S0[k].hi) : make_float2(0.f, 0.f);
            OP::fwd(p.c, fm, f0, fp, fl, fr, s, r);
#pragma unroll
            for (int e = 0; e < NE; ++e) { if (h == 0) R[e].lo = r[e]; else R[e].hi = r[e]; }
        }
        if (!PER) {
            const bool rowless = j < 1 || j > n0 - 2 || !inside;
#pragma unroll
            for (int e = 0; e < NE; ++e) {
                if (rowless) R[e] = v4zero();
                if (first_col) R[e].lo.x = 0.f;
                if (last_col) R[e].hi.y = 0.f;
            }
        }
    };

    V4 F[5][NF], S[5][NSA], R[5][NE];
    // slots at step i (s = (i - a0) mod 5): F[s] row i-1, F[s+1] row i, F[s+2] row i+1, F[s+3] row i+2,
    // F[s+4] receives row i+3; R[s] = r(i-1), R[s+1] = r(i), R[s+2] receives r(i+1)
    load_row(a0 - 2, F[4], S[4]);
    load_row(a0 - 1, F[0], S[0]);
    load_row(a0, F[1], S[1]);
    load_row(a0 + 1, F[2], S[2]);
    load_row(a0 + 2, F[3], S[3]);
    residual_row(a0 - 1, F[4], F[0], F[1], S[0], R[0]);
    residual_row(a0, F[0], F[1], F[2], S[1], R[1]);
    float2 acc[NE];
#pragma unroll
    for (int e = 0; e < NE; ++e) acc[e] = make_float2(0.f, 0.f);

    auto step = [&](int i, const V4 (&Fm)[NF], const V4 (&F0)[NF], const V4 (&Fp)[NF], const V4 (&Fpp)[NF],
                    V4 (&Fnew)[NF], const V4 (&Sp)[NSA], V4 (&Snew)[NSA], const V4 (&Rm)[NE], const V4 (&R0)[NE],
                    V4 (&Rp)[NE]) {
        if (i + 1 < a1) load_row(i + 3, Fnew, Snew);
        if (p.prefetch > 0 && (lane & 7) == 0 && i + 3 + p.prefetch <= a1 + 1) {
            const int off = row_of(i + 3 + p.prefetch) * n1 + col;
#pragma unroll
            for (int k = 0; k < NF; ++k) asm volatile("prefetch.global.L2 [%0];" ::"l"(at_off<O32>(p.f[k], off)));
#pragma unroll
            for (int k = 0; k < NS; ++k) asm volatile("prefetch.global.L2 [%0];" ::"l"(at_off<O32>(p.src[k], off)));
        }
        residual_row(i + 1, F0, Fp, Fpp, Sp, Rp);
        V4 RL[NE], RR[NE], FL[NF], FR[NF];
#pragma unroll
        for (int e = 0; e < NE; ++e) lateral(R0[e], RL[e], RR[e]);
#pragma unroll
        for (int k = 0; k < NF; ++k) {
            if (OP::FIELD_LATERAL_IN_BWD) lateral(F0[k], FL[k], FR[k]);
            else { FL[k] = F0[k]; FR[k] = F0[k]; }
        }
        float2 g[NF][2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float2 fm[NF], f0[NF], fp[NF], fl[NF], fr[NF], rm[NE], r0[NE], rp[NE], rl[NE], rr[NE], gg[NF];
            v4_half<NF>(Fm, h, fm); v4_half<NF>(F0, h, f0); v4_half<NF>(Fp, h, fp);
            v4_half<NF>(FL, h, fl); v4_half<NF>(FR, h, fr);
            v4_half<NE>(Rm, h, rm); v4_half<NE>(R0, h, r0); v4_half<NE>(Rp, h, rp);
            v4_half<NE>(RL, h, rl); v4_half<NE>(RR, h, rr);
            OP::bwd(p.c, fm, f0, fp, fl, fr, rm, r0, rp, rl, rr, gg);
#pragma unroll
            for (int k = 0; k < NF; ++k) g[k][h] = mul2(gg[k], p.gs);
        }
        if (own) {
            const int off = i * n1 + col;
#pragma unroll
            for (int k = 0; k < NF; ++k) stv4(at_off<O32>(p.g[k], off), g[k][0], g[k][1]);
#pragma unroll
            for (int e = 0; e < NE; ++e) {
                if (p.res[e] != nullptr) stv4(at_off<O32>(p.res[e], off), R0[e].lo, R0[e].hi);
                acc[e] = fma2(R0[e].lo, R0[e].lo, fma2(R0[e].hi, R0[e].hi, acc[e]));
            }
        }
    };

    for (int i = a0; i < a1; i += 5) {
#pragma unroll
        for (int s = 0; s < 5; ++s) {
            if (i + s < a1)
                step(i + s, F[s % 5], F[(s + 1) % 5], F[(s + 2) % 5], F[(s + 3) % 5], F[(s + 4) % 5], S[(s + 2) % 5],
                     S[(s + 4) % 5], R[s % 5], R[(s + 1) % 5], R[(s + 2) % 5]);
        }
    }
    if (p.partials != nullptr) {
        float sum[NE];
#pragma unroll
        for (int e = 0; e < NE; ++e) sum[e] = acc[e].x + acc[e].y;
        block_reduce_store<NE>(sum, p.partials, p.nitems, item);
    }
}

static int env_int(const char* name, int dflt) {
    const char* s = std::getenv(name);
    if (!s || !*s) return dflt;
    const int v = std::atoi(s);
    return v > 0 ? v : dflt;
}

static float2 sp(double v) { return make_float2((float)v, (float)v); }

bool fused2d_supported(int op) {
    return op == 1 || op == 2 || op == 5;            // Poisson 2-D, Gray-Scott, steady 2-D Navier-Stokes
}

static int sm_count() {                              // initialised once, thread-safe
    static const int n = [] {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) return v;
        return 148;
    }();
    return n;
}

static int fused2d_minb(int op) {                   // resident blocks per SM the kernel is compiled for
    const int dflt = op == 1 ? 4 : (op == 2 ? 4 : 3);
    const int v = env_int("FPDE_FUSED2D_MINB", dflt);
    return op == 1 ? 4 : (op == 2 ? (v == 3 ? 3 : 4) : (v == 2 ? 2 : 3));
}
static int fused2d_blocks_per_sm(int op) { return fused2d_minb(op); }

// Rows per work item: every item recomputes r on two extra rows, and the last wave of items
// should be nearly full; pick the row count with the smallest (waves x rows marched per item).
static void fused2d_geometry(int op, const int* n, Fused2dParams& p) {
    p.n0 = n[0]; p.n1 = n[1]; p.nc4 = n[1] / 4;
    p.ncg = (p.nc4 + FUSED2D_OWN - 1) / FUSED2D_OWN;
    p.ncb = (p.ncg + 3) / 4;
    int rows = env_int("FPDE_FUSED2D_ROWS", 0);
    if (rows > 0 && rows < 4) rows = 4;
    if (rows == 0) {
        const long slots = (long)sm_count() * fused2d_blocks_per_sm(op);
        long best = -1;
        for (int r = 4; r <= 96; ++r) {
            const long items = (long)p.ncb * ((p.n0 + r - 1) / r);
            const long cost = ((items + slots - 1) / slots) * (r + 4);
            if (best < 0 || cost < best) { best = cost; rows = r; }
        }
    }
    p.rows_per_item = rows;
    const char* pf = std::getenv("FPDE_FUSED2D_PREFETCH");
    p.prefetch = pf && *pf ? std::atoi(pf) : 2;
    if (p.prefetch < 0) p.prefetch = 0;
    p.nitems = p.ncb * ((p.n0 + rows - 1) / rows);
}

// upper bound of the item count over every row count the geometry can choose (>= 4 rows per
// item), for workspace sizing that does not depend on the device the query runs on
int fused2d_max_items(const int* n) {
    const int nc4 = n[1] / 4, ncg = (nc4 + FUSED2D_OWN - 1) / FUSED2D_OWN, ncb = (ncg + 3) / 4;
    return ncb * ((n[0] + 3) / 4);
}

int fused2d_items(int op, const int* n) {
    Fused2dParams p{};
    fused2d_geometry(op, n, p);
    return p.nitems;
}

// q.in = fields, q.aux = sources, q.out = dL/dfield; `res` = residual arrays (entries may be NULL)
cudaError_t launch_fused2d(const Problem& q, float* const* res) {
    Fused2dParams p{};
    fused2d_geometry(q.op, q.n, p);
    p.partials = q.partials;
    p.gs = sp(2.0 / (double)q.rows);
    // 32-bit byte offsets from the array bases for arrays of at most 2^30 floats
    const char* o32s = std::getenv("FPDE_FUSED2D_OFF32");
    const bool o32 = !(o32s && o32s[0] == '0') && (int64_t)q.n[0] * q.n[1] <= ((int64_t)1 << 30);
    const double h0 = q.h[0], h1 = q.h[1];
    switch (q.op) {
    case 1:
        p.f[0] = q.in[0]; p.src[0] = q.aux[0]; p.g[0] = q.out[0]; p.res[0] = res ? res[0] : nullptr;
        p.c[0] = sp(1.0 / (h0 * h0)); p.c[1] = sp(1.0 / (h1 * h1));
        if (o32) return launch_kernel(fused2d_kernel<FusedPoisson, 4, true>, dim3(p.nitems), dim3(128), q.stream, p);
        return launch_kernel(fused2d_kernel<FusedPoisson, 4>, dim3(p.nitems), dim3(128), q.stream, p);
    case 2:
        for (int k = 0; k < 2; ++k) { p.f[k] = q.in[k]; p.g[k] = q.out[k]; p.res[k] = res ? res[k] : nullptr; }
        p.c[0] = sp(1.0 / (h0 * h0)); p.c[1] = sp(1.0 / (h1 * h1));
        p.c[2] = sp(q.coef[0]); p.c[3] = sp(q.coef[1]); p.c[4] = sp(q.coef[2]); p.c[5] = sp(q.coef[2] + q.coef[3]);
        if (fused2d_minb(2) == 3) return launch_kernel(fused2d_kernel<FusedGrayScott, 3>, dim3(p.nitems), dim3(128), q.stream, p);
        if (o32) return launch_kernel(fused2d_kernel<FusedGrayScott, 4, true>, dim3(p.nitems), dim3(128), q.stream, p);
        return launch_kernel(fused2d_kernel<FusedGrayScott, 4>, dim3(p.nitems), dim3(128), q.stream, p);
    case 5:
        for (int k = 0; k < 3; ++k) { p.f[k] = q.in[k]; p.g[k] = q.out[k]; p.res[k] = res ? res[k] : nullptr; }
        p.c[0] = sp(0.5 / h0); p.c[1] = sp(0.5 / h1);
        p.c[2] = sp(-q.coef[0] / (h0 * h0)); p.c[3] = sp(-q.coef[0] / (h1 * h1));
        if (fused2d_minb(5) == 3) {
            if (o32) return launch_kernel(fused2d_kernel<FusedNs2d, 3, true>, dim3(p.nitems), dim3(128), q.stream, p);
            return launch_kernel(fused2d_kernel<FusedNs2d, 3>, dim3(p.nitems), dim3(128), q.stream, p);
        }
        return launch_kernel(fused2d_kernel<FusedNs2d, 2>, dim3(p.nitems), dim3(128), q.stream, p);
    }
    return cudaErrorInvalidValue;
}

}  // namespace fpde
