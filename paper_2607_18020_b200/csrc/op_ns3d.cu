// Steady incompressible Navier-Stokes on an (x,y,z) array (z contiguous): Section 2.1's system
// with the third velocity component w and d_z added.  Four residuals (momentum x,y,z and
// continuity) from four fields (u,v,w,p); rows at the nodes where all three centred stencils
// fit, i.e. the interior [1,n-2]^3; the outer shell of the array is data.
//
//   mom_q = u d_x q + v d_y q + w d_z q + d_{a_q} p - nu (d_xx + d_yy + d_zz) q     q in (u,v,w)
//   cont  = d_x u + d_y v + d_z w
//
// The adjoint is Eq. (1) / Appendix A.3 extended the same way (ns_math.cuh writes it out); the
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

// per-thread constants of a launch
struct Ns3dThread {
    int n0, PS;
    int rowoff, eoff, ymoff, ypoff;    // element offsets inside a plane: own float4, edge float, y-1, y+1
    int a1;
    bool valid, first_col, last_col, efetch, lane_first, lane_last;
    bool y_dead, ym_dead, yp_dead;     // own row / y-1 / y+1 carry no residual row
};

// zero extension of an upstream float4 along z (elements z = 0 and z = n2-1)
__device__ __forceinline__ V4 ns3d_zmask(const Ns3dThread& t, V4 v) {
    if (t.first_col) v.lo.x = 0.f;
    if (t.last_col) v.hi.y = 0.f;
    return v;
}

// array k at plane r (clamped into the array) at the thread's own float4; with `check`, an
// upstream float4 whose plane or row is outside the rows reads as zero
template <bool BWD, bool PRE, bool O32>
__device__ __forceinline__ V4 ns3d_load_own(const Ns3dParams& p, const Ns3dThread& t, int k, int r, bool check) {
    const int rr = max(0, min(t.n0 - 1, r));
    V4 v = ldv4(at_off<O32>(p.a[k], rr * t.PS + t.rowoff));
    if (BWD && !PRE && k >= 3) {
        v = ns3d_zmask(t, v);
        if (check && (t.y_dead || r < 1 || r > t.n0 - 2)) v = v4zero();
    }
    return v;
}

// One x step: W0 = plane a-1, W1 = plane a, W2 receives plane a+1.  EDGE: some float4 the block
// reads in this step lies outside the rows (a block-uniform property), so the whole-vector
// zero extension has to be looked at; the other steps skip those selects.
// PRE (adjoint only): the upstream arrays are already zero off the rows (residual arrays the
// forward kernel of the same call wrote), so nothing is zero-extended here; clamped reads beyond
// the array land in the zero shell.
template <bool BWD, bool EDGE, int NA, bool PRE, bool O32>
__device__ __forceinline__ void ns3d_step(const Ns3dParams& p, const Ns3dThread& t, int a, const V4 (&W0)[NA],
                                          const V4 (&W1)[NA], V4 (&W2)[NA], float2 (&acc)[4]) {
    constexpr int G0 = 3;                            // adjoint: first upstream array
    const int pl = a * t.PS;
    const bool x_dead = a < 1 || a > t.n0 - 2;
    if (p.prefetch > 0 && (threadIdx.x & 7) == 0 && a + 1 + p.prefetch <= min(t.a1, t.n0 - 1)) {
        const int po = (a + 1 + p.prefetch) * t.PS + t.rowoff;
#pragma unroll
        for (int k = 0; k < NA; ++k) ns3d_prefetch_l2(at_off<O32>(p.a[k], po));
    }
    V4 Ym[NA], Yp[NA], Zm[NA], Zp[NA];
    float E[NA];
#pragma unroll
    for (int k = 0; k < NA; ++k) {
        W2[k] = ns3d_load_own<BWD, PRE, O32>(p, t, k, a + 1, EDGE);
        Ym[k] = ldv4(at_off<O32>(p.a[k], pl + t.ymoff));
        Yp[k] = ldv4(at_off<O32>(p.a[k], pl + t.ypoff));
        E[k] = 0.f;
        if (t.efetch) E[k] = __ldg(at_off<O32>(p.a[k], pl + t.eoff));
    }
#pragma unroll
    for (int k = 0; k < NA; ++k) {
        if (BWD && !PRE && k >= G0) {
            Ym[k] = ns3d_zmask(t, Ym[k]); Yp[k] = ns3d_zmask(t, Yp[k]);
            if (EDGE) {
                if (x_dead || t.ym_dead) Ym[k] = v4zero();
                if (x_dead || t.yp_dead) Yp[k] = v4zero();
                if (x_dead || t.y_dead) E[k] = 0.f;
            }
        }
        float l1 = __shfl_up_sync(FULL_MASK, W1[k].hi.y, 1);
        float r1 = __shfl_down_sync(FULL_MASK, W1[k].lo.x, 1);
        if (t.lane_first) l1 = E[k];
        if (t.lane_last) r1 = E[k];
        // (a z line that ends inside a warp: the lane after it shadows column 0, whose upstream
        // lo.x is zero-extended, so r1 of the last column is 0 there as well)
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
        if constexpr (BWD) ns_bwd_pair<true>(p.k, w0, w1, w2, ym, yp, zm, zp, nodt, oo);
        else ns_fwd_pair(p.k, w0, w1, w2, ym, yp, zm, zp, nodt, oo);
#pragma unroll
        for (int e = 0; e < 4; ++e) o[e][h] = oo[e];
    }
    if (!BWD) {                                      // the outer shell carries no row
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (EDGE && (x_dead || t.y_dead)) { o[e][0] = make_float2(0.f, 0.f); o[e][1] = o[e][0]; }
            if (t.first_col) o[e][0].x = 0.f;
            if (t.last_col) o[e][1].y = 0.f;
        }
    }
    if (t.valid) {
        const int off = pl + t.rowoff;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            stv4(at_off<O32>(p.out[e], off), o[e][0], o[e][1]);
            if (!BWD) acc[e] = fma2(o[e][0], o[e][0], fma2(o[e][1], o[e][1], acc[e]));
        }
    }
}

// O32: 32-bit byte offsets from the array bases (arrays of at most 2^30 floats): in the forward
// kernel, the adjoint without zero-extension, and the interior steps of the masking adjoint (with
// its shell steps as well that build spills 200 bytes; as it is, 16 bytes of stack at 255
// registers, which the timed loop does not notice)
template <bool BWD, int MINB, bool PRE = false, bool O32 = false>
__global__ void __launch_bounds__(128, MINB) ns3d_kernel(const Ns3dParams p) {
    constexpr int NA = BWD ? 7 : 4;
    pdl_wait_then_trigger();
    const int n1 = p.n1, n2 = p.n2, nc4 = p.nc4;
    int item = blockIdx.x;
    const int cb = item % p.ncb; item /= p.ncb;
    const int mb = item % p.nmb;
    const int ab = item / p.nmb;
    const int c4 = cb * blockDim.x + threadIdx.x;
    const int m = mb * blockDim.y + threadIdx.y;
    const int c4c = c4 < nc4 ? c4 : 0, mc = m < n1 ? m : 0;   // out-of-range threads shadow (0,0)
    const int col = 4 * c4c;
    const int lane = threadIdx.x & 31;
    Ns3dThread t;
    t.n0 = p.n0; t.PS = n1 * n2;
    t.valid = c4 < nc4 && m < n1;
    t.first_col = c4c == 0; t.last_col = c4c == nc4 - 1;
    t.lane_first = lane == 0; t.lane_last = lane == 31;
    // the one float beyond the float4 that the first / last lane of a warp cannot get by shuffle;
    // at the ends of a z line it stays 0 (zero extension; the velocities' value there is unused)
    t.efetch = (lane == 0 && !t.first_col) || (lane == 31 && !t.last_col);
    t.rowoff = mc * n2 + col;
    t.eoff = t.rowoff + (lane == 0 ? -1 : 4);
    t.ymoff = max(mc - 1, 0) * n2 + col;
    t.ypoff = min(mc + 1, n1 - 1) * n2 + col;
    t.y_dead = mc < 1 || mc > n1 - 2;
    t.ym_dead = mc - 1 < 1; t.yp_dead = mc + 1 > n1 - 2;
    // does any thread of this block touch a y row without residuals (its own or a y neighbour)?
    const int m_lo = mb * blockDim.y, m_hi = m_lo + blockDim.y - 1;
    const bool y_edge_block = m_lo <= 1 || m_hi >= n1 - 2;
    const int a0 = ab * p.planes_per_item;
    const int a1 = min(a0 + p.planes_per_item, p.n0);
    t.a1 = a1;

    // the planes the first steps load are not covered by the per-step prefetch: ask for them now
    if (p.prefetch > 0 && (threadIdx.x & 7) == 0) {
        for (int d = 1; d <= p.prefetch && a0 + d <= min(a1, p.n0 - 1); ++d) {
            const int po = (a0 + d) * t.PS + t.rowoff;
#pragma unroll
            for (int k = 0; k < NA; ++k) ns3d_prefetch_l2(at_off<O32>(p.a[k], po));
        }
    }
    V4 A[NA], B[NA], Cc[NA];
#pragma unroll
    for (int k = 0; k < NA; ++k) {
        A[k] = ns3d_load_own<BWD, PRE, O32>(p, t, k, a0 - 1, true);
        B[k] = ns3d_load_own<BWD, PRE, O32>(p, t, k, a0, true);
    }
    float2 acc[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[e] = make_float2(0.f, 0.f);

    auto step = [&](int a, const V4 (&W0)[NA], const V4 (&W1)[NA], V4 (&W2)[NA]) {
        if (!PRE && (y_edge_block || a <= 1 || a >= p.n0 - 2)) ns3d_step<BWD, true, NA, PRE, O32 && !BWD>(p, t, a, W0, W1, W2, acc);
        else ns3d_step<BWD, false, NA, PRE, O32>(p, t, a, W0, W1, W2, acc);
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
    int tx = env_int("FPDE_NS3D_TX", p.nc4 % 64 == 0 ? 64 : 32);
    tx = std::max(32, std::min(128, (tx / 32) * 32));
    int ty = env_int("FPDE_NS3D_TY", 128 / tx);
    ty = std::max(1, std::min(128 / tx, ty));
    block = dim3(tx, ty, 1);
    p.ncb = (p.nc4 + tx - 1) / tx;
    p.nmb = (p.n1 + ty - 1) / ty;
    p.planes_per_item = env_int("FPDE_NS3D_PLANES", planes_for_grid(p.n0, 24, (long)p.ncb * p.nmb, (long long)n[0] * n[1] * n[2]));
    p.nitems = p.ncb * p.nmb * ((p.n0 + p.planes_per_item - 1) / p.planes_per_item);
    const char* pf = std::getenv("FPDE_NS3D_PREFETCH");
    p.prefetch = pf && *pf ? std::atoi(pf) : 2;
    if (p.prefetch < 0 || p.prefetch >= p.n0) p.prefetch = 0;
}

// 32-bit byte offsets are enough for arrays of at most 2^30 floats
static bool ns3d_off32(const Problem& q) {
    const char* s = std::getenv("FPDE_NS3D_OFF32");
    return !(s && s[0] == '0') && (int64_t)q.n[0] * q.n[1] * q.n[2] <= ((int64_t)1 << 30);
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
    if (ns3d_off32(q)) return launch_kernel(ns3d_kernel<false, 3, false, true>, dim3(p.nitems), block, q.stream, p);
    return launch_kernel(ns3d_kernel<false, 3>, dim3(p.nitems), block, q.stream, p);
}

cudaError_t launch_ns3d_bwd(const Problem& q) {
    Ns3dParams p{}; dim3 block;
    ns3d_geometry(q.n, p, block);
    for (int k = 0; k < 3; ++k) p.a[k] = q.in[k];
    for (int k = 0; k < 4; ++k) { p.a[3 + k] = q.aux[k]; p.out[k] = q.out[k]; }
    ns3d_consts(q, q.gscale, p.k);
    p.partials = nullptr;
    if (q.gres_zero_off_rows) {
        if (ns3d_off32(q)) return launch_kernel(ns3d_kernel<true, 2, true, true>, dim3(p.nitems), block, q.stream, p);
        return launch_kernel(ns3d_kernel<true, 2, true>, dim3(p.nitems), block, q.stream, p);
    }
    if (env_int("FPDE_NS3D_MINB_B", 2) == 3) return launch_kernel(ns3d_kernel<true, 3>, dim3(p.nitems), block, q.stream, p);
    if (ns3d_off32(q)) return launch_kernel(ns3d_kernel<true, 2, false, true>, dim3(p.nitems), block, q.stream, p);
    return launch_kernel(ns3d_kernel<true, 2>, dim3(p.nitems), block, q.stream, p);
}

}  // namespace fpde
