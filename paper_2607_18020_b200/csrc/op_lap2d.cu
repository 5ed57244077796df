// Two-dimensional five-point operators: 2-D Poisson and two-field Gray-Scott, forward
// (Section 2.1: fused residual, here with the loss partial sums) and gather-form adjoint
// (Section 2.2), all instances of one streaming engine.
//
// Engine.  A thread owns one float4 column of the array and marches down a chunk of rows with a
// three-row register window (previous / current / next), so every input element is loaded by
// exactly one thread; left/right neighbours come from the adjacent lanes' registers (the first
// and last lane of a warp fetch theirs with one predicated scalar load).  Rows are fetched U at
// a time so that each thread keeps U independent 128-bit loads per input in flight.  A work
// item is (row chunk, column block); the chunk's two halo rows are re-read from L2.
// Arithmetic is packed fp32x2 (two lanes of the float4 per instruction).  Inputs are of two
// kinds: "halo" inputs, read with their four neighbours (fields in the forward pass, upstream
// sensitivities in the adjoint), and "centre" inputs read only at the node itself (sources in
// the forward pass, fields in a nonlinear adjoint).
//
// The five-point sum is formed as ih0*((up+dn) - 2c) + ih1*((l+r) - 2c).
//
// Boundary handling (Section 2.3 / Appendix A.5) is part of the same launch:
//   periodic axes   - row and column indices wrap;
//   interior axes   - forward: nodes of the outer ring carry no row and get 0;
//                     adjoint: the upstream array is treated as 0 outside the rows (omitted
//                     neighbours), which also yields the gradient of the ring nodes.
#include "fpde_common.cuh"
#include "fpde_internal.h"

#include <algorithm>
#include <cstdlib>

namespace fpde {

struct Lap2dParams {
    const float* hin[2];
    const float* cin[2];
    float* out[2];
    float2 hscale[2];
    float2 ih0, ih1;     // 1/h0^2, 1/h1^2 (splatted)
    float2 c[4];
    int n0, n1, nc4;
    int rows_per_item, ncb, nitems;
    float* partials;
};

// out = -Lap u - f
struct PoissonFwd {
    static constexpr int NH = 1, NC = 1, NO = 1;
    static constexpr bool BWD = false;
    __device__ static __forceinline__ void eval(const float2* v, const float2* lap, const float2* cc,
                                                const float2* c, float2* o) {
        o[0] = fma2(lap[0], splat2(-1.f), make_float2(-cc[0].x, -cc[0].y));
    }
};
// g = -Lap G  (the Jacobian is constant and symmetric on the rows)
struct PoissonBwd {
    static constexpr int NH = 1, NC = 0, NO = 1;
    static constexpr bool BWD = true;
    __device__ static __forceinline__ void eval(const float2* v, const float2* lap, const float2* cc,
                                                const float2* c, float2* o) {
        o[0] = make_float2(-lap[0].x, -lap[0].y);
    }
};
// c = {D_u, D_v, F, F+k}
struct GrayScottFwd {
    static constexpr int NH = 2, NC = 0, NO = 2;
    static constexpr bool BWD = false;
    __device__ static __forceinline__ void eval(const float2* v, const float2* lap, const float2* cc,
                                                const float2* c, float2* o) {
        const float2 u = v[0], w = v[1];
        const float2 uww = mul2(mul2(u, w), w);
        // D_u lap_u + F (1 - u) - u w^2
        const float2 t = fma2(u, make_float2(-c[2].x, -c[2].y), c[2]);
        o[0] = sub2(fma2(lap[0], c[0], t), uww);
        // D_v lap_v + u w^2 - (F+k) w
        o[1] = fma2(lap[1], c[1], fma2(w, make_float2(-c[3].x, -c[3].y), uww));
    }
};
// g_u = D_u Lap G_u + G_u (-v^2 - F) + G_v v^2 ;  g_v = D_v Lap G_v + G_u (-2uv) + G_v (2uv - (F+k))
struct GrayScottBwd {
    static constexpr int NH = 2, NC = 2, NO = 2;
    static constexpr bool BWD = true;
    __device__ static __forceinline__ void eval(const float2* v, const float2* lap, const float2* cc,
                                                const float2* c, float2* o) {
        const float2 a = v[0], b = v[1], u = cc[0], w = cc[1];
        const float2 ww = mul2(w, w);
        const float2 uw2 = mul2(add2(u, u), w);
        // D_u lap_a + ww (b - a) - F a
        const float2 bma = sub2(b, a);
        o[0] = fma2(lap[0], c[0], fma2(ww, bma, mul2(a, make_float2(-c[2].x, -c[2].y))));
        // D_v lap_b + uw2 (b - a) - (F+k) b
        o[1] = fma2(lap[1], c[1], fma2(uw2, bma, mul2(b, make_float2(-c[3].x, -c[3].y))));
    }
};

// PX / PY: the row axis (x) / the column axis (y) is periodic.  Poisson: neither; Gray-Scott:
// both; the slab form of Gray-Scott (x not periodic: rows at x-index 1..n0-2): PY only.
template <class F, bool PX, bool PY, int U, bool O32 = false>
__global__ void __launch_bounds__(128) lap2d_kernel(const Lap2dParams p) {
    constexpr int NH = F::NH, NC = F::NC, NO = F::NO;
    constexpr int NCA = NC > 0 ? NC : 1;
    constexpr bool BWD = F::BWD;
    constexpr bool ROWS_MASK_IN = BWD && !PX;      // upstream array is zero on the first / last row and beyond
    constexpr bool COLS_MASK_IN = BWD && !PY;      // ... and on the first / last column and beyond
    constexpr bool ROWS_MASK_OUT = !BWD && !PX;    // nodes of the first / last row carry no residual row
    constexpr bool COLS_MASK_OUT = !BWD && !PY;    // nor do those of the first / last column
    pdl_wait_then_trigger();
    const int n0 = p.n0, n1 = p.n1, nc4 = p.nc4;
    const int item = blockIdx.x;
    const int cb = item % p.ncb, rc = item / p.ncb;
    const int c4 = cb * blockDim.x + threadIdx.x;
    const int lane = threadIdx.x & 31;
    const bool cvalid = c4 < nc4;
    const int col = cvalid ? 4 * c4 : 0;            // out-of-range threads read column 0, store nothing
    const bool first_col = c4 == 0, last_col = c4 == nc4 - 1;
    const int a0 = rc * p.rows_per_item;
    const int a1 = min(a0 + p.rows_per_item, n0);

    // columns the first / last lane of a warp fetch from memory (the others use shuffles)
    int lcol = col - 1, rcol = col + 4;
    if (PY) { if (lcol < 0) lcol += n1; if (rcol >= n1) rcol -= n1; }
    const bool lfetch = cvalid && (lane == 0 || first_col) && lcol >= 0;
    const bool rfetch = cvalid && (lane == 31 || last_col) && rcol < n1;
    const bool lzero = !PY && first_col, rzero = !PY && last_col;

    // row index a halo-input row is read from, or -1 if it reads as zero
    auto in_row = [&](int r) -> int {
        if (PX) return r < 0 ? r + n0 : (r >= n0 ? r - n0 : r);
        if (ROWS_MASK_IN) return (r < 1 || r > n0 - 2) ? -1 : r;
        return max(0, min(n0 - 1, r));              // forward: out-of-range rows only feed masked outputs
    };
    auto load_h = [&](int k, int r) -> V4 {
        const int rr = in_row(r);
        if (ROWS_MASK_IN && rr < 0) return v4zero();
        V4 v = BWD ? ldv4(p.hin[k] + rr * n1 + col) : ldv4(at_off<O32>(p.hin[k], rr * n1 + col));
        if (BWD) v = v4mul(v, p.hscale[k]);
        if (COLS_MASK_IN) {
            if (first_col) v.lo.x = 0.f;
            if (last_col) v.hi.y = 0.f;
        }
        return v;
    };

    V4 prev[NH], cur[NH];
#pragma unroll
    for (int k = 0; k < NH; ++k) { prev[k] = load_h(k, a0 - 1); cur[k] = load_h(k, a0); }
    float2 acc[NO];
#pragma unroll
    for (int e = 0; e < NO; ++e) acc[e] = make_float2(0.f, 0.f);
    const float2 m2 = splat2(-2.f);

    for (int a = a0; a < a1; a += U) {
        V4 nxt[U][NH];
        V4 cen[U][NCA];
        float le[U][NH], re[U][NH];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int row = min(a + u, a1 - 1);     // rows past the chunk repeat the last one (unused)
#pragma unroll
            for (int k = 0; k < NH; ++k) {
                nxt[u][k] = load_h(k, row + 1);
                const int rr = in_row(row);
                le[u][k] = 0.f; re[u][k] = 0.f;
                if (!(ROWS_MASK_IN && rr < 0)) {
                    if (BWD) {                    // (two forms of the same address: each direction keeps the one its build is faster with)
                        const float* rp = p.hin[k] + rr * n1;
                        if (lfetch) le[u][k] = __ldg(rp + lcol);
                        if (rfetch) re[u][k] = __ldg(rp + rcol);
                    } else {
                        if (lfetch) le[u][k] = __ldg(at_off<O32>(p.hin[k], rr * n1 + lcol));
                        if (rfetch) re[u][k] = __ldg(at_off<O32>(p.hin[k], rr * n1 + rcol));
                    }
                }
            }
#pragma unroll
            for (int k = 0; k < NC; ++k) cen[u][k] = BWD ? ldv4(p.cin[k] + row * n1 + col) : ldv4(at_off<O32>(p.cin[k], row * n1 + col));
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int row = a + u;
            if (row < a1) {                       // uniform over the block
                float2 lap_lo[NH], lap_hi[NH], v_lo[NH], v_hi[NH];
#pragma unroll
                for (int k = 0; k < NH; ++k) {
                    const V4 c = cur[k];
                    float l1 = __shfl_up_sync(FULL_MASK, c.hi.y, 1);
                    float r1 = __shfl_down_sync(FULL_MASK, c.lo.x, 1);
                    if (lfetch) l1 = BWD ? le[u][k] * p.hscale[k].x : le[u][k];
                    if (rfetch) r1 = BWD ? re[u][k] * p.hscale[k].x : re[u][k];
                    if (lzero) l1 = 0.f;
                    if (rzero) r1 = 0.f;
                    const V4 vs = v4add(prev[k], nxt[u][k]);
                    V4 hs;
                    hs.lo = make_float2(l1 + c.lo.y, c.lo.x + c.hi.x);
                    hs.hi = make_float2(c.lo.y + c.hi.y, c.hi.x + r1);
                    const V4 tv = v4fma(c, m2, vs), th = v4fma(c, m2, hs);
                    lap_lo[k] = fma2(tv.lo, p.ih0, mul2(th.lo, p.ih1));
                    lap_hi[k] = fma2(tv.hi, p.ih0, mul2(th.hi, p.ih1));
                    v_lo[k] = c.lo; v_hi[k] = c.hi;
                }
                float2 cc_lo[NCA], cc_hi[NCA], o_lo[NO], o_hi[NO];
#pragma unroll
                for (int k = 0; k < NC; ++k) { cc_lo[k] = cen[u][k].lo; cc_hi[k] = cen[u][k].hi; }
                F::eval(v_lo, lap_lo, cc_lo, p.c, o_lo);
                F::eval(v_hi, lap_hi, cc_hi, p.c, o_hi);
                if (ROWS_MASK_OUT || COLS_MASK_OUT) {
                    const bool rowless = ROWS_MASK_OUT && (row < 1 || row > n0 - 2);
#pragma unroll
                    for (int e = 0; e < NO; ++e) {
                        if (rowless) { o_lo[e] = make_float2(0.f, 0.f); o_hi[e] = o_lo[e]; }
                        if (COLS_MASK_OUT && first_col) o_lo[e].x = 0.f;
                        if (COLS_MASK_OUT && last_col) o_hi[e].y = 0.f;
                    }
                }
                if (cvalid) {
#pragma unroll
                    for (int e = 0; e < NO; ++e) {
                        if (BWD) stv4(p.out[e] + row * n1 + col, o_lo[e], o_hi[e]);
                        else stv4(at_off<O32>(p.out[e], row * n1 + col), o_lo[e], o_hi[e]);
                        if (!BWD) acc[e] = fma2(o_lo[e], o_lo[e], fma2(o_hi[e], o_hi[e], acc[e]));
                    }
                }
#pragma unroll
                for (int k = 0; k < NH; ++k) { prev[k] = cur[k]; cur[k] = nxt[u][k]; }
            }
        }
    }
    if (!BWD && p.partials != nullptr) {
        float s[NO];
#pragma unroll
        for (int e = 0; e < NO; ++e) s[e] = acc[e].x + acc[e].y;
        block_reduce_store<NO>(s, p.partials, p.nitems, item);
    }
}

static int env_int(const char* name, int dflt) {
    const char* s = std::getenv(name);
    if (!s || !*s) return dflt;
    const int v = std::atoi(s);
    return v > 0 ? v : dflt;
}

static void lap2d_geometry(const Problem& q, Lap2dParams& p, int& block) {
    p.n0 = q.n[0]; p.n1 = q.n[1]; p.nc4 = q.n[1] / 4;
    block = env_int("FPDE_LAP2D_BLOCK", 128);
    block = std::max(32, std::min(128, (block / 32) * 32));
    p.rows_per_item = env_int("FPDE_LAP2D_ROWS", 8);
    p.ncb = (p.nc4 + block - 1) / block;
    p.nitems = p.ncb * ((p.n0 + p.rows_per_item - 1) / p.rows_per_item);
    const float ih0 = (float)(1.0 / (q.h[0] * q.h[0])), ih1 = (float)(1.0 / (q.h[1] * q.h[1]));
    p.ih0 = make_float2(ih0, ih0);
    p.ih1 = make_float2(ih1, ih1);
}

int lap2d_items(const int* n) {
    Problem q{}; q.n[0] = n[0]; q.n[1] = n[1]; q.h[0] = q.h[1] = 1.0;
    Lap2dParams p{}; int block;
    lap2d_geometry(q, p, block);
    return p.nitems;
}

template <class F, bool PX, bool PY>
static cudaError_t launch(const Lap2dParams& p, int block, cudaStream_t s) {
    // 32-bit byte offsets from the array bases for arrays of at most 2^30 floats
    const char* o = std::getenv("FPDE_LAP2D_OFF32");
    if (!(o && o[0] == '0') && (int64_t)p.n0 * p.n1 <= ((int64_t)1 << 30))
        return launch_kernel(lap2d_kernel<F, PX, PY, 4, true>, dim3(p.nitems), dim3(block), s, p);
    return launch_kernel(lap2d_kernel<F, PX, PY, 4>, dim3(p.nitems), dim3(block), s, p);
}

static float2 sp(double v) { return make_float2((float)v, (float)v); }

cudaError_t launch_lap2d_fwd(const Problem& q) {
    Lap2dParams p{}; int block;
    lap2d_geometry(q, p, block);
    p.partials = q.partials;
    p.hin[0] = q.in[0]; p.out[0] = q.out[0];
    if (q.op != 1) {                                 // Gray-Scott: 2 periodic, 8 its slab form
        p.hin[1] = q.in[1]; p.out[1] = q.out[1];
        p.c[0] = sp(q.coef[0]); p.c[1] = sp(q.coef[1]); p.c[2] = sp(q.coef[2]); p.c[3] = sp(q.coef[2] + q.coef[3]);
        if (q.op == 2) return launch<GrayScottFwd, true, true>(p, block, q.stream);
        return launch<GrayScottFwd, false, true>(p, block, q.stream);
    }
    p.cin[0] = q.aux[0];
    return launch<PoissonFwd, false, false>(p, block, q.stream);
}

cudaError_t launch_lap2d_bwd(const Problem& q) {
    Lap2dParams p{}; int block;
    lap2d_geometry(q, p, block);
    p.partials = nullptr;
    p.hin[0] = q.aux[0]; p.out[0] = q.out[0]; p.hscale[0] = sp(q.gscale[0]);
    if (q.op != 1) {
        p.hin[1] = q.aux[1]; p.out[1] = q.out[1]; p.hscale[1] = sp(q.gscale[1]);
        p.cin[0] = q.in[0]; p.cin[1] = q.in[1];
        p.c[0] = sp(q.coef[0]); p.c[1] = sp(q.coef[1]); p.c[2] = sp(q.coef[2]); p.c[3] = sp(q.coef[2] + q.coef[3]);
        if (q.op == 2) return launch<GrayScottBwd, true, true>(p, block, q.stream);
        return launch<GrayScottBwd, false, true>(p, block, q.stream);
    }
    return launch<PoissonBwd, false, false>(p, block, q.stream);
}

}  // namespace fpde
