// Unsteady incompressible Navier-Stokes on an (x,y,z,t) array (t contiguous), space periodic,
// rows at interior t: four residuals (momentum x,y,z and continuity) from four fields
// (u,v,w,p).  This is Section 2.1's steady 2-D system extended by d_t, w and d_z; the adjoint
// below is Eq. (1) / Appendix A.3 extended the same way (drop w, z and t and it is the printed
// u-gradient term by term).
//
// Memory view: (x, y, row) with row = (z,t) flattened, n2*n3 contiguous floats.  Along a row,
// t+-1 is +-1 float and z+-1 is +-n3 floats with wrap-around over the row, so periodic z is a
// cyclic shift inside one contiguous line.
//
// Kernel shape (both directions): a thread owns one float4 (four consecutive t of one z) of a
// (y,row) tile and marches along x, the slowest axis, with a three-plane register window per
// array (rotated by unrolling, not by moves); y+-1 and z+-1 neighbours of the current plane are
// read through L1, t+-1 neighbours come from the adjacent lanes' registers.  Arithmetic is
// packed fp32x2.  Second differences are formed as (q[-1]-q[0]) + (q[+1]-q[0]) before scaling:
// here the viscous term is small against the other terms and must not carry the rounding of
// the large centre value.
//
// Nodes at the first / last t carry no row: the forward pass writes 0 there; in the adjoint the
// upstream arrays count as 0 there (omitted neighbours, Appendix A.5).  Every spatial read of an
// output node happens at the node's own t, so that rule only changes (i) the t-neighbour of the
// nodes next to the two end planes and (ii) the end planes themselves, where only the
// transposed d_t term survives: that is the boundary-gradient correction of this operator, and
// it is applied as a fix-up of two lanes instead of masking every load.
#include "fpde_common.cuh"
#include "fpde_internal.h"
#include "ns_math.cuh"

#include <algorithm>
#include <cstdlib>

namespace fpde {

struct NsParams {
    const float* f[4];    // u, v, w, p
    const float* g[4];    // adjoint: upstream arrays of mom_x, mom_y, mom_z, continuity
    float* out[4];
    int n0, n1, n3;       // x, y extents; t extent
    int C, C4, nt4;       // row length in floats / float4, float4 per z
    int planes_per_item, ncb, nmb, nitems;
    int item_offset;      // first work item of this launch (launches over a range of plane chunks)
    NsConsts k;
    float* partials;
    int prefetch;         // planes ahead of the window to prefetch into L2 (0 = off)
    int xint;             // x axis not periodic: rows at x-index 1..n0-2 only (one slab of a split grid)
};

struct NsIndex {
    int col, rowoff;           // own column (floats) and m*C
    int ymoff, ypoff;          // (m-1)*C, (m+1)*C wrapped
    int zmcol, zpcol;          // columns of z-1 / z+1 (floats), wrapped over the row
    int m, c4;
    bool valid;
    bool t_first, t_last;      // this float4 holds t = 0 (in lo.x) / t = n3-1 (in hi.y)
};

__device__ __forceinline__ int wrapi(int i, int n) { return i < 0 ? i + n : (i >= n ? i - n : i); }
// x-plane a step reads: wrapped, or (non-periodic x) clamped into the array; a clamped plane only
// ever feeds an output that is zeroed or an upstream value that counts as zero
__device__ __forceinline__ int xplane(const NsParams& p, int a) {
    return p.xint ? max(0, min(p.n0 - 1, a)) : wrapi(a, p.n0);
}
__device__ __forceinline__ bool xdead(const NsParams& p, int a) { return p.xint && (a < 1 || a > p.n0 - 2); }
template <int NA>
__device__ __forceinline__ void zero_from(V4 (&W)[NA], int first) {
#pragma unroll
    for (int k = 0; k < NA; ++k) if (k >= first) W[k] = v4zero();
}

// Ask L2 for the line holding `ptr` (no register, no wait): hides most of the DRAM latency of
// the plane the register window will pull in a few steps later.
__device__ __forceinline__ void prefetch_l2(const float* ptr) {
    asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
}

__device__ __forceinline__ NsIndex ns_index(const NsParams& p, int& a0, int& a1) {
    NsIndex ix;
    int item = blockIdx.x + p.item_offset;
    const int cb = item % p.ncb; item /= p.ncb;
    const int mb = item % p.nmb;
    const int ab = item / p.nmb;
    ix.c4 = cb * blockDim.x + threadIdx.x;
    ix.m = mb * blockDim.y + threadIdx.y;
    ix.valid = ix.c4 < p.C4 && ix.m < p.n1;
    const int c4c = ix.c4 < p.C4 ? ix.c4 : 0;       // out-of-range threads shadow column 0 / row 0
    const int mc = ix.m < p.n1 ? ix.m : 0;
    ix.col = 4 * c4c;
    ix.rowoff = mc * p.C;
    ix.ymoff = wrapi(mc - 1, p.n1) * p.C;
    ix.ypoff = wrapi(mc + 1, p.n1) * p.C;
    ix.zmcol = 4 * wrapi(c4c - p.nt4, p.C4);
    ix.zpcol = 4 * wrapi(c4c + p.nt4, p.C4);
    const int tq = c4c % p.nt4;
    ix.t_first = tq == 0;
    ix.t_last = tq == p.nt4 - 1;
    a0 = ab * p.planes_per_item;
    a1 = min(a0 + p.planes_per_item, p.n0);
    return ix;
}

// t-1 / t+1 neighbours of a float4's outer lanes: lane-1's last / lane+1's first element.  When
// a warp boundary can fall inside a z group (TSAFE false) the outer lanes fetch them from memory.
template <bool TSAFE>
__device__ __forceinline__ void t_neighbours(const V4& c, const float* __restrict__ row, const NsIndex& ix,
                                             float& l1, float& r1) {
    l1 = __shfl_up_sync(FULL_MASK, c.hi.y, 1);
    r1 = __shfl_down_sync(FULL_MASK, c.lo.x, 1);
    if (!TSAFE) {
        const int lane = threadIdx.x & 31;
        if (lane == 0 && !ix.t_first) l1 = __ldg(row + ix.col - 1);
        if (lane == 31 && !ix.t_last) r1 = __ldg(row + ix.col + 4);
    }
}

// ------------------------------------------------------------------------------------------
// forward
// ------------------------------------------------------------------------------------------
template <bool TSAFE, int MINB, bool O32>
__global__ void __launch_bounds__(128, MINB) ns_fwd_kernel(const NsParams p) {
    pdl_wait_then_trigger();
    int a0, a1;
    const NsIndex ix = ns_index(p, a0, a1);
    const int PS = p.n1 * p.C;                      // plane stride
    const float* __restrict__ f0 = p.f[0];
    const float* __restrict__ f1 = p.f[1];
    const float* __restrict__ f2 = p.f[2];
    const float* __restrict__ f3 = p.f[3];
    const float* const fp[4] = {f0, f1, f2, f3};

    V4 A[4], B[4], Cc[4];                           // three x-planes of u,v,w,p at the own column
    {
        const int om = xplane(p, a0 - 1) * PS + ix.rowoff + ix.col;
        const int oc = a0 * PS + ix.rowoff + ix.col;
#pragma unroll
        for (int k = 0; k < 4; ++k) { A[k] = ldv4(at_off<O32>(fp[k], om)); B[k] = ldv4(at_off<O32>(fp[k], oc)); }
    }
    float2 acc[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[e] = make_float2(0.f, 0.f);

    // one x step: W0 = plane a-1, W1 = plane a, W2 receives plane a+1
    auto step = [&](int a, const V4 (&W0)[4], const V4 (&W1)[4], V4 (&W2)[4]) {
        const int pl = a * PS;
        const int ap = xplane(p, a + 1) * PS;
        if (p.prefetch > 0 && (threadIdx.x & 7) == 0 && a + 1 + p.prefetch <= a1) {   // one lane per 128-byte line
            const int af = xplane(p, a + 1 + p.prefetch);
            const int po = af * PS + ix.rowoff + ix.col;
#pragma unroll
            for (int k = 0; k < 4; ++k) prefetch_l2(at_off<O32>(fp[k], po));
        }
        V4 Ym[4], Yp[4], Zm[4], Zp[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            W2[k] = ldv4(at_off<O32>(fp[k], ap + ix.rowoff + ix.col));
            Ym[k] = ldv4(at_off<O32>(fp[k], pl + ix.ymoff + ix.col));
            Yp[k] = ldv4(at_off<O32>(fp[k], pl + ix.ypoff + ix.col));
            Zm[k] = ldv4(at_off<O32>(fp[k], pl + ix.rowoff + ix.zmcol));
            Zp[k] = ldv4(at_off<O32>(fp[k], pl + ix.rowoff + ix.zpcol));
        }
        float l1[3], r1[3];
#pragma unroll
        for (int k = 0; k < 3; ++k) t_neighbours<TSAFE>(W1[k], fp[k] + pl + ix.rowoff, ix, l1[k], r1[k]);
        float2 o[4][2];
        ns_fwd_math(p.k, W0, W1, W2, Ym, Yp, Zm, Zp, l1, r1, ix.t_first, ix.t_last, o);
        if (xdead(p, a)) {                          // the two outer x-planes of a slab carry no row
#pragma unroll
            for (int e = 0; e < 4; ++e) { o[e][0] = make_float2(0.f, 0.f); o[e][1] = o[e][0]; }
        }
        if (ix.valid) {
            const int off = pl + ix.rowoff + ix.col;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                stv4(at_off<O32>(p.out[e], off), o[e][0], o[e][1]);
                acc[e] = fma2(o[e][0], o[e][0], fma2(o[e][1], o[e][1], acc[e]));
            }
        }
    };

    for (int a = a0; a < a1; a += 3) {
        step(a, A, B, Cc);
        if (a + 1 < a1) step(a + 1, B, Cc, A);
        if (a + 2 < a1) step(a + 2, Cc, A, B);
    }
    if (p.partials != nullptr) {
        float s[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) s[e] = acc[e].x + acc[e].y;
        block_reduce_store<4>(s, p.partials, p.nitems, blockIdx.x + p.item_offset);
    }
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
// G_e = gscale_e * gres_e; the scales are folded into the constants.
// ------------------------------------------------------------------------------------------
template <bool TSAFE, int MINB, bool O32>
__global__ void __launch_bounds__(128, MINB) ns_bwd_kernel(const NsParams p) {
    pdl_wait_then_trigger();
    int a0, a1;
    const NsIndex ix = ns_index(p, a0, a1);
    const int PS = p.n1 * p.C;
    // arrays 0..2: u,v,w ; 3..6: upstream of mom_x, mom_y, mom_z, continuity
    const float* const ap[7] = {p.f[0], p.f[1], p.f[2], p.g[0], p.g[1], p.g[2], p.g[3]};

    V4 A[7], B[7], Cc[7];
    {
        const int om = xplane(p, a0 - 1) * PS + ix.rowoff + ix.col;
        const int oc = a0 * PS + ix.rowoff + ix.col;
#pragma unroll
        for (int k = 0; k < 7; ++k) { A[k] = ldv4(at_off<O32>(ap[k], om)); B[k] = ldv4(at_off<O32>(ap[k], oc)); }
        // upstream arrays count as zero on planes without rows
        if (xdead(p, a0 - 1)) zero_from<7>(A, 3);
        if (xdead(p, a0)) zero_from<7>(B, 3);
    }

    auto step = [&](int a, const V4 (&W0)[7], const V4 (&W1)[7], V4 (&W2)[7]) {
        const int pl = a * PS;
        const int apl = xplane(p, a + 1) * PS;
        if (p.prefetch > 0 && (threadIdx.x & 7) == 0 && a + 1 + p.prefetch <= a1) {
            const int af = xplane(p, a + 1 + p.prefetch);
            const int po = af * PS + ix.rowoff + ix.col;
#pragma unroll
            for (int k = 0; k < 7; ++k) prefetch_l2(at_off<O32>(ap[k], po));
        }
        V4 Ym[7], Yp[7], Zm[7], Zp[7];
#pragma unroll
        for (int k = 0; k < 7; ++k) {
            W2[k] = ldv4(at_off<O32>(ap[k], apl + ix.rowoff + ix.col));
            Ym[k] = ldv4(at_off<O32>(ap[k], pl + ix.ymoff + ix.col));
            Yp[k] = ldv4(at_off<O32>(ap[k], pl + ix.ypoff + ix.col));
            Zm[k] = ldv4(at_off<O32>(ap[k], pl + ix.rowoff + ix.zmcol));
            Zp[k] = ldv4(at_off<O32>(ap[k], pl + ix.rowoff + ix.zpcol));
        }
        if (xdead(p, a + 1)) zero_from<7>(W2, 3);
        if (xdead(p, a)) { zero_from<7>(Ym, 3); zero_from<7>(Yp, 3); zero_from<7>(Zm, 3); zero_from<7>(Zp, 3); }
        float l1[3], r1[3];
#pragma unroll
        for (int q = 0; q < 3; ++q) {
            t_neighbours<TSAFE>(W1[3 + q], ap[3 + q] + pl + ix.rowoff, ix, l1[q], r1[q]);
            if (xdead(p, a)) { l1[q] = 0.f; r1[q] = 0.f; }
        }
        float2 o[4][2];
        ns_bwd_math(p.k, W0, W1, W2, Ym, Yp, Zm, Zp, l1, r1, ix.t_first, ix.t_last, o);
        if (ix.valid) {
            const int off = pl + ix.rowoff + ix.col;
#pragma unroll
            for (int e = 0; e < 4; ++e) stv4(at_off<O32>(p.out[e], off), o[e][0], o[e][1]);
        }
    };

    for (int a = a0; a < a1; a += 3) {
        step(a, A, B, Cc);
        if (a + 1 < a1) step(a + 1, B, Cc, A);
        if (a + 2 < a1) step(a + 2, Cc, A, B);
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
    int tx = env_int("FPDE_NS_TX", p.C4 % 64 == 0 ? 64 : 32);
    tx = std::max(32, std::min(128, (tx / 32) * 32));
    int ty = env_int("FPDE_NS_TY", 128 / tx);
    ty = std::max(1, std::min(128 / tx, ty));
    block = dim3(tx, ty, 1);
    p.ncb = (p.C4 + tx - 1) / tx;
    p.nmb = (p.n1 + ty - 1) / ty;
    p.planes_per_item = q.planes_per_item > 0 ? q.planes_per_item
                                              : env_int("FPDE_NS_PLANES", planes_for_grid(p.n0, 24, (long)p.ncb * p.nmb, (long long)q.n[0] * q.n[1] * q.n[2] * q.n[3]));
    p.nitems = p.ncb * p.nmb * ((p.n0 + p.planes_per_item - 1) / p.planes_per_item);
    const char* pf = std::getenv("FPDE_NS_PREFETCH");
    p.prefetch = pf && *pf ? std::atoi(pf) : 2;
    if (p.prefetch < 0 || p.prefetch >= p.n0) p.prefetch = 0;
    p.xint = q.bc0_interior ? 1 : 0;
}

static bool ns_tsafe(const NsParams& p) { return 32 % p.nt4 == 0; }

// 32-bit byte offsets are enough for arrays of at most 2^30 floats (FPDE_NS_OFF32=0: never)
static bool ns_off32(const Problem& q) {
    const int64_t N = (int64_t)q.n[0] * q.n[1] * q.n[2] * q.n[3];
    const char* s = std::getenv("FPDE_NS_OFF32");
    return !(s && s[0] == '0') && N <= ((int64_t)1 << 30);
}

// Grid of a launch: all work items, or those of the plane chunks [chunk_lo, chunk_hi) of the
// problem (items are ordered with the plane chunk slowest, so a chunk range is an item range).
static dim3 ns_range(const Problem& q, NsParams& p) {
    const int per_chunk = p.ncb * p.nmb;
    if (q.chunk_hi > q.chunk_lo) {
        p.item_offset = q.chunk_lo * per_chunk;
        return dim3((q.chunk_hi - q.chunk_lo) * per_chunk);
    }
    p.item_offset = 0;
    return dim3(p.nitems);
}

int ns_items(const int* n, bool xint, int planes_per_item) {
    if (!xint && planes_per_item == 0 && ns_tma_wanted(n)) return ns_tma_items(n);
    Problem q{};
    for (int a = 0; a < 4; ++a) { q.n[a] = n[a]; q.h[a] = 1.0; }
    q.bc0_interior = xint;
    q.planes_per_item = planes_per_item;
    NsParams p{}; dim3 block;
    ns_geometry(q, p, block);
    return p.nitems;
}

// Planes per work item the launcher chooses for this grid when the caller names none.
int ns_plane_chunk(const int* n, bool xint) {
    Problem q{};
    for (int a = 0; a < 4; ++a) { q.n[a] = n[a]; q.h[a] = 1.0; }
    q.bc0_interior = xint;
    NsParams p{}; dim3 block;
    ns_geometry(q, p, block);
    return p.planes_per_item;
}

cudaError_t launch_ns_fwd(const Problem& q) {
    if (!q.bc0_interior && q.planes_per_item == 0) {
        bool launched = false;
        const cudaError_t ce = launch_ns_fwd_tma(q, launched);
        if (launched || ce != cudaSuccess) return ce;
    }
    NsParams p{}; dim3 block;
    ns_geometry(q, p, block);
    for (int k = 0; k < 4; ++k) { p.f[k] = q.in[k]; p.out[k] = q.out[k]; }
    const double ones[4] = {1.0, 1.0, 1.0, 1.0};
    ns_fill_consts(p.k, q.h, q.coef[0], ones);
    p.partials = q.partials;
    const int minb = env_int("FPDE_NS_MINB_F", 3);
    cudaError_t ce;
    const dim3 grid = ns_range(q, p);
    const bool o32 = ns_off32(q);
    if (!ns_tsafe(p)) ce = launch_kernel(ns_fwd_kernel<false, 3, false>, grid, block, q.stream, p);
    else if (minb != 3) ce = launch_kernel(ns_fwd_kernel<true, 4, false>, grid, block, q.stream, p);
    else if (o32) ce = launch_kernel(ns_fwd_kernel<true, 3, true>, grid, block, q.stream, p);
    else ce = launch_kernel(ns_fwd_kernel<true, 3, false>, grid, block, q.stream, p);
    return ce;
}

cudaError_t launch_ns_bwd(const Problem& q) {
    if (!q.bc0_interior && q.planes_per_item == 0) {
        bool launched = false;
        const cudaError_t ce = launch_ns_bwd_tma(q, launched);
        if (launched || ce != cudaSuccess) return ce;
    }
    NsParams p{}; dim3 block;
    ns_geometry(q, p, block);
    for (int k = 0; k < 4; ++k) { p.f[k] = q.in[k]; p.g[k] = q.aux[k]; p.out[k] = q.out[k]; }
    ns_fill_consts(p.k, q.h, q.coef[0], q.gscale);
    p.partials = nullptr;
    const int minb = env_int("FPDE_NS_MINB_B", 2);
    cudaError_t ce;
    const dim3 grid = ns_range(q, p);
    const bool o32 = ns_off32(q);
    if (!ns_tsafe(p)) ce = launch_kernel(ns_bwd_kernel<false, 2, false>, grid, block, q.stream, p);
    else if (minb == 3) ce = launch_kernel(ns_bwd_kernel<true, 3, false>, grid, block, q.stream, p);
    else if (o32) ce = launch_kernel(ns_bwd_kernel<true, 2, true>, grid, block, q.stream, p);
    else ce = launch_kernel(ns_bwd_kernel<true, 2, false>, grid, block, q.stream, p);
    return ce;
}

}  // namespace fpde
