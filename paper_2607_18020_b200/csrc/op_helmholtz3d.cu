// Three-dimensional fourth-order Helmholtz operator, r = Lap4 u + k^2 u - f, with the 13-point
// star (-1,16,-30,16,-1)/(12 h^2) per axis: fused forward residual + loss partials (Section
// 2.1) and the gather-form adjoint with its two-cell boundary band (Sections 2.2, 2.3).
//
// The Jacobian is constant and the star is symmetric, so the adjoint is the same star applied
// to the upstream array treated as zero outside the rows (omitted neighbours, Appendix A.5);
// that one rule produces the gradient of the two outer layers and the truncated sums of layers
// 2 and 3.  Forward and adjoint are therefore two instances of one 2.5-D engine:
//
//   a thread owns one float4 of a (y,z) tile and marches along x, the slowest axis, holding the
//   five x-planes of its own column in registers (rotated by unrolling); the y+-1, y+-2
//   neighbours of the current plane are read through L1 (other threads of the same block loaded
//   those lines two steps earlier); z neighbours come from the adjacent lanes' registers.  The
//   plane the window loads in the next step is prefetched into L2.  Arithmetic is packed
//   fp32x2; the star is evaluated as  sum_a w_a (16 (q[-1]+q[+1]) - (q[-2]+q[+2])) + K q  with
//   K = k^2 - 30 sum_a w_a.
#include "fpde_common.cuh"
#include "fpde_internal.h"

#include <algorithm>
#include <cstdlib>
#include <cstddef>
#include <type_traits>

namespace fpde {

struct Star3dParams {
    const float* hin;     // read with halo 2 (u forward, upstream array in the adjoint)
    const float* cin;     // read at the centre (f forward, unused in the adjoint)
    float* out;
    int n0, n1, n2, nc4;
    int planes_per_item, ncb, nmb, nitems;
    float2 w16[3];        // 16 s / (12 h_a^2), s = upstream scale (1 forward)
    float2 nw[3];         // -s / (12 h_a^2)
    float2 kc;            // s (k^2 - 30 sum_a 1/(12 h_a^2))
    float* partials;
    int prefetch;
};

__device__ __forceinline__ void prefetch_l2_line(const void* ptr) {
    asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
}

// EDGE: the block touches the two-cell band in x or y, where (adjoint) rows and planes of the
// upstream array read as zero; blocks away from the band run without those selects.  The first
// and last float4 of a row (the band in z) are handled in every block.
// MODE 0: forward.  MODE 1: adjoint of an arbitrary upstream array (zero-extended here).  MODE 2:
// adjoint of an upstream array that is already zero off the rows (the residual array the forward
// kernel of the same call wrote): the star itself, nothing to mask; clamped reads beyond the
// array land in the zero band.
// Addressing: a position is a byte offset from the array bases (the three arrays are reached from
// the same offset), 32-bit (O32) when every array is below 4 GiB; the y neighbours sit at
// per-thread distances from it that are constant over the march.  (Builds with the y and z
// extents fixed at compile time, where those distances become constants of the load
// instructions, execute a tenth fewer instructions and run no faster: the kernels wait on
// memory, not on issue slots.)
template <int MODE, bool EDGE, int MINB, bool O32>
__device__ __forceinline__ void star3d_body(const Star3dParams& p, int cb, int mb, int ab) {
    constexpr bool FWD = MODE == 0;
    using Off = typename std::conditional<O32, unsigned, size_t>::type;
    const int n0 = p.n0, n1 = p.n1, n2 = p.n2, nc4 = p.nc4;
    const int c4 = cb * blockDim.x + threadIdx.x;
    const int m = mb * blockDim.y + threadIdx.y;
    const int lane = threadIdx.x & 31;
    const bool valid = c4 < nc4 && m < n1;
    const int col = c4 < nc4 ? 4 * c4 : 0;
    const int mc = m < n1 ? m : 0;
    const bool first_col = c4 == 0, last_col = c4 == nc4 - 1;
    const int a0 = ab * p.planes_per_item;
    const int a1 = min(a0 + p.planes_per_item, n0);
    const Off PS4 = (Off)4 * (Off)n1 * (Off)n2;     // bytes per plane
    constexpr bool MASK_IN = MODE == 1;             // the adjoint zero-extends its input outside the rows
    constexpr bool ROWMASK = MASK_IN && EDGE;
    const char* __restrict__ hin = reinterpret_cast<const char*>(p.hin);
    const char* __restrict__ cin = reinterpret_cast<const char*>(p.cin);
    char* __restrict__ out = reinterpret_cast<char*>(p.out);
    using Pos = Off;
    auto h_at = [&](Pos pos, Off d) -> const char* { return hin + (Off)(pos + d); };
    auto c_at = [&](Pos pos, Off d) -> const char* { return cin + (Off)(pos + d); };
    auto o_at = [&](Pos pos) -> char* { return out + pos; };

    // element offsets of the own row and of the four y neighbours within a plane (clamped into the
    // grid: out of range rows only feed outputs that are masked, or are discarded by the selects
    // below); the neighbours as distances from the own row, constant over the march
    auto yoff = [&](int d) -> int { return (EDGE ? max(0, min(n1 - 1, mc + d)) : mc + d) * n2 + col; };
    auto ydead = [&](int d) -> bool { const int r = mc + d; return ROWMASK && (r < 2 || r > n1 - 3); };
    const int o_c = yoff(0);
    auto ydelta = [&](int d) -> Off { return (Off)(4 * (yoff(d) - o_c)); };   // d < 0: added modulo 2^32 / 2^64
    const Off dm1 = ydelta(-1), dp1 = ydelta(1), dm2 = ydelta(-2), dp2 = ydelta(2);
    const bool d0 = ydead(0), dm1d = ydead(-1), dp1d = ydead(1), dm2d = ydead(-2), dp2d = ydead(2);
    auto ld_at = [&](const char* ptr) -> V4 {
        const float4 t = __ldg(reinterpret_cast<const float4*>(ptr));
        V4 v; v.lo = make_float2(t.x, t.y); v.hi = make_float2(t.z, t.w);
        return v;
    };
    // Load of the upstream / field array; `dead` = reads as zero.
    // OWN: the thread's own column (the x window).  Only that one is masked in the first / last
    // float4 of a row (the band in z); the y neighbours are not, their contribution to the two
    // band columns is removed after the sums instead (see the step).
    auto load_h = [&](const char* ptr, bool dead, bool own) -> V4 {
        V4 v = ld_at(ptr);
        if (MASK_IN) {
            if ((ROWMASK && dead) || (own && first_col)) v.lo = make_float2(0.f, 0.f);
            if ((ROWMASK && dead) || (own && last_col)) v.hi = make_float2(0.f, 0.f);
        }
        return v;
    };
    // own column on plane a (clamped in the blocks that touch the ends of the x axis)
    auto ppos = [&](int a) -> Pos {
        return (Off)(EDGE ? max(0, min(n0 - 1, a)) : a) * PS4 + (Off)(4 * o_c);
    };
    auto pdead = [&](int a) -> bool { return ROWMASK && (a < 2 || a > n0 - 3); };
    // The two floats beyond the float4 that the first / last lane of a warp cannot get by shuffle:
    // one predicated 8-byte load, issued with the other loads of the step (a load inside a
    // divergent branch would be waited for on its own).  At the ends of a z line it stays 0.
    const bool efetch = (lane == 0 && c4 > 0 && c4 < nc4) || (lane == 31 && c4 < nc4 - 1);
    const Off eoff = lane == 0 ? (Off)(-8) : (Off)16;
    const bool pf_lane = p.prefetch > 0 && (threadIdx.x & 7) == 0;
    const int pf_last = min(a1 + 1, n0 - 1) - 2 - p.prefetch;      // last step that still prefetches
    const Off pf_h = (Off)(2 + p.prefetch) * PS4, pf_c = (Off)p.prefetch * PS4;

    V4 Q0 = load_h(h_at(ppos(a0 - 2), 0), d0 || pdead(a0 - 2), true), Q1 = load_h(h_at(ppos(a0 - 1), 0), d0 || pdead(a0 - 1), true);
    V4 Q2 = load_h(h_at(ppos(a0), 0), d0 || pdead(a0), true), Q3 = load_h(h_at(ppos(a0 + 1), 0), d0 || pdead(a0 + 1), true), Q4;
    Pos pos = ppos(a0);                              // own float4 on the current plane
    float2 acc = make_float2(0.f, 0.f);

    // one x step: q0..q3 = planes a-2..a+1, q4 receives plane a+2
    auto step = [&](int a, const V4& q0, const V4& q1, const V4& q2, const V4& q3, V4& q4) {
        if (pf_lane && a <= pf_last) {
            prefetch_l2_line(h_at(pos, pf_h));
            if (FWD) prefetch_l2_line(c_at(pos, pf_c));
        }
        const bool pd = pdead(a);
        q4 = load_h(EDGE ? h_at(ppos(a + 2), 0) : h_at(pos, 2 * PS4), d0 || pdead(a + 2), true);
        const V4 a1v = load_h(h_at(pos, dm1), dm1d || pd, false), b1v = load_h(h_at(pos, dp1), dp1d || pd, false);
        const V4 a2v = load_h(h_at(pos, dm2), dm2d || pd, false), b2v = load_h(h_at(pos, dp2), dp2d || pd, false);
        V4 src = v4zero();
        if (FWD) {
            // read once and by nobody else: streamed past L1, which the y neighbours' lines need
            const float4 t4 = __ldcs(reinterpret_cast<const float4*>(c_at(pos, 0)));
            src.lo = make_float2(t4.x, t4.y); src.hi = make_float2(t4.z, t4.w);
        }
        float2 E = make_float2(0.f, 0.f);
        if (efetch) E = __ldg(reinterpret_cast<const float2*>(h_at(pos, eoff)));
        if (ROWMASK && (d0 || pd)) E = make_float2(0.f, 0.f);
        // z neighbours from the adjacent lanes; the outer lanes of a warp take the fetched pair
        float l1 = __shfl_up_sync(FULL_MASK, q2.hi.y, 1), l2 = __shfl_up_sync(FULL_MASK, q2.hi.x, 1);
        float r1 = __shfl_down_sync(FULL_MASK, q2.lo.x, 1), r2 = __shfl_down_sync(FULL_MASK, q2.lo.y, 1);
        if (lane == 0) { l2 = E.x; l1 = E.y; }
        if (lane == 31) { r1 = E.x; r2 = E.y; }
        if (MASK_IN && last_col) { r1 = 0.f; r2 = 0.f; }   // a ragged row ends inside a warp
        const V4 s1x = v4add(q1, q3), s2x = v4add(q0, q4);
        const V4 s1y = v4add(a1v, b1v), s2y = v4add(a2v, b2v);
        V4 s1z, s2z;
        s1z.lo = make_float2(l1 + q2.lo.y, q2.lo.x + q2.hi.x);
        s1z.hi = make_float2(q2.lo.y + q2.hi.y, q2.hi.x + r1);
        s2z.lo = make_float2(l2 + q2.hi.x, l1 + q2.hi.y);
        s2z.hi = make_float2(q2.lo.x + r1, q2.lo.y + r2);
        V4 o = v4mul(q2, p.kc);
        o = v4fma(s1x, p.w16[0], o); o = v4fma(s2x, p.nw[0], o);
        o = v4fma(s1z, p.w16[2], o); o = v4fma(s2z, p.nw[2], o);
        const V4 oxz = o;                            // centre + x + z terms
        o = v4fma(s1y, p.w16[1], o); o = v4fma(s2y, p.nw[1], o);
        if (MASK_IN) {
            // band in z (adjoint): columns 0,1 / n-2,n-1 of the upstream array are zero.  The own
            // column was masked on load, so oxz is already right there; only the (unmasked) y
            // neighbours have to be taken out again.
            if (first_col) o.lo = oxz.lo;
            if (last_col) o.hi = oxz.hi;
        }
        if (FWD) {
            o = v4sub(o, src);
            // nodes of the two outer layers carry no row
            if (EDGE && (a < 2 || a > n0 - 3 || m < 2 || m > n1 - 3)) { o = v4zero(); }
            if (first_col) o.lo = make_float2(0.f, 0.f);
            if (last_col) o.hi = make_float2(0.f, 0.f);
        }
        if (valid) {
            *reinterpret_cast<float4*>(o_at(pos)) = make_float4(o.lo.x, o.lo.y, o.hi.x, o.hi.y);
            if (FWD) acc = fma2(o.lo, o.lo, fma2(o.hi, o.hi, acc));
        }
        pos += PS4;
    };

    for (int a = a0; a < a1; a += 5) {
        step(a, Q0, Q1, Q2, Q3, Q4);
        if (a + 1 < a1) step(a + 1, Q1, Q2, Q3, Q4, Q0);
        if (a + 2 < a1) step(a + 2, Q2, Q3, Q4, Q0, Q1);
        if (a + 3 < a1) step(a + 3, Q3, Q4, Q0, Q1, Q2);
        if (a + 4 < a1) step(a + 4, Q4, Q0, Q1, Q2, Q3);
    }
    if (FWD && p.partials != nullptr) {
        float s[1] = {acc.x + acc.y};
        block_reduce_store<1>(s, p.partials, p.nitems, blockIdx.x);
    }
}

template <int MODE, int MINB, bool O32>
__global__ void __launch_bounds__(256, MINB) star3d_kernel(const Star3dParams p) {
    pdl_wait_then_trigger();
    int item = blockIdx.x;
    const int cb = item % p.ncb; item /= p.ncb;
    const int mb = item % p.nmb;
    const int ab = item / p.nmb;
    const int m0 = mb * blockDim.y, a0 = ab * p.planes_per_item;
    // away from the band: every row m0-2 .. m0+TY+1 and plane a0-2 .. a1+1 is a row of the operator
    const bool interior = m0 >= 4 && m0 + (int)blockDim.y + 4 <= p.n1 && a0 >= 4 && a0 + p.planes_per_item + 4 <= p.n0;
    if (interior) star3d_body<MODE, false, MINB, O32>(p, cb, mb, ab);
    else star3d_body<MODE, true, MINB, O32>(p, cb, mb, ab);
}

static int env_int(const char* name, int dflt) {
    const char* s = std::getenv(name);
    if (!s || !*s) return dflt;
    const int v = std::atoi(s);
    return v > 0 ? v : dflt;
}

static float2 sp(double v) { return make_float2((float)v, (float)v); }

static void star3d_geometry(const Problem& q, Star3dParams& p, dim3& block, double scale, bool fwd) {
    p.n0 = q.n[0]; p.n1 = q.n[1]; p.n2 = q.n[2]; p.nc4 = q.n[2] / 4;
    int tx = p.nc4 > 32 ? 64 : 32;
    tx = env_int("FPDE_STAR3D_TX", tx);
    tx = std::max(32, std::min(128, (tx / 32) * 32));
    int ty = env_int("FPDE_STAR3D_TY", 4);
    ty = std::max(1, std::min(256 / tx, ty));
    block = dim3(tx, ty, 1);
    // the forward kernel (two input streams) runs best on long items, the adjoint on short ones
    p.ncb = (p.nc4 + tx - 1) / tx;
    p.nmb = (p.n1 + ty - 1) / ty;
    const long per_chunk = (long)p.ncb * p.nmb;
    const long long points = (long long)p.n0 * p.n1 * p.n2;
    // large grids: the tuned length, stretched until the blocks just fill whole waves of the 4 blocks
    // an SM holds (256^3 forward: 32 -> 29 planes, 512 -> 576 blocks for 592 slots, 33.9 -> 31.9 us)
    auto fitted = [&](int tuned) {
        const int pl = planes_for_grid(p.n0, tuned, per_chunk, points);
        return points >= (1ll << 22) ? fit_planes_to_waves(p.n0, pl, per_chunk, 4l * sm_count_or_default()) : pl;
    };
    p.planes_per_item = fwd ? env_int("FPDE_STAR3D_PLANES_F", fitted(32)) : env_int("FPDE_STAR3D_PLANES_B", fitted(10));
    p.nitems = p.ncb * p.nmb * ((p.n0 + p.planes_per_item - 1) / p.planes_per_item);
    double wsum = 0.0;
    for (int a = 0; a < 3; ++a) {
        const double w = 1.0 / (12.0 * q.h[a] * q.h[a]);
        p.w16[a] = sp(16.0 * w * scale);
        p.nw[a] = sp(-w * scale);
        wsum += w;
    }
    p.kc = sp((q.coef[0] * q.coef[0] - 30.0 * wsum) * scale);
    const char* pf = std::getenv("FPDE_STAR3D_PREFETCH");
    p.prefetch = pf && *pf ? std::atoi(pf) : 1;
    if (p.prefetch < 0) p.prefetch = 0;
}

static int star3d_l1_items(const int* n) {
    Problem q{}; q.n[0] = n[0]; q.n[1] = n[1]; q.n[2] = n[2]; q.h[0] = q.h[1] = q.h[2] = 1.0;
    Star3dParams p{}; dim3 block;
    star3d_geometry(q, p, block, 1.0, true);
    return p.nitems;
}

// Loss partial sums a forward launch may write: the larger of the two engines' item counts (which
// engine runs is decided per launch; the launcher reports the count it used).
int star3d_items(const int* n) {
    const int l1 = star3d_l1_items(n);
    return star3d_tma_wanted(n) ? std::max(l1, star3d_tma_items(n)) : l1;
}

// 32-bit byte offsets when every array is below 4 GiB (FPDE_STAR3D_OFF32=0 forces the 64-bit form)
template <int MODE>
static cudaError_t star3d_launch(const Problem& q, const Star3dParams& p, dim3 block) {
    const char* e = std::getenv("FPDE_STAR3D_OFF32");
    const bool o32 = !(e && *e == '0') && (long long)p.n0 * p.n1 * p.n2 <= (1ll << 30);
    if (o32) return launch_kernel(star3d_kernel<MODE, 4, true>, dim3(p.nitems), block, q.stream, p);
    return launch_kernel(star3d_kernel<MODE, 4, false>, dim3(p.nitems), block, q.stream, p);
}

cudaError_t launch_helmholtz_fwd(const Problem& q, int* items) {
    bool launched = false;
    cudaError_t ce = launch_star3d_tma(q, 0, items, launched);
    if (launched || ce != cudaSuccess) return ce;
    Star3dParams p{}; dim3 block;
    star3d_geometry(q, p, block, 1.0, true);
    p.hin = q.in[0]; p.cin = q.aux[0]; p.out = q.out[0];
    p.partials = q.partials;
    if (items) *items = p.nitems;
    return star3d_launch<0>(q, p, block);
}

cudaError_t launch_helmholtz_bwd(const Problem& q) {
    bool launched = false;
    cudaError_t ce = launch_star3d_tma(q, q.gres_zero_off_rows ? 2 : 1, nullptr, launched);
    if (launched || ce != cudaSuccess) return ce;
    Star3dParams p{}; dim3 block;
    star3d_geometry(q, p, block, q.gscale[0], false);      // the operator is linear: the scale goes into the weights
    p.hin = q.aux[0]; p.cin = nullptr; p.out = q.out[0];
    p.partials = nullptr;
    return q.gres_zero_off_rows ? star3d_launch<2>(q, p, block) : star3d_launch<1>(q, p, block);
}

}  // namespace fpde
