// Two-dimensional five-point operators: 2-D Poisson and two-field Gray-Scott, forward
// (Section 2.1: fused residual, here with the loss partial sums) and gather-form adjoint
// (Section 2.2), both instances of one streaming engine.
//
// Engine.  A thread owns one float4 column of the array and marches down a chunk of rows with a
// three-row register window (previous / current / next), so every input element is loaded by
// exactly one thread; left/right neighbours come from the adjacent lanes' registers.  A work
// item is (row chunk, column block); the chunk's two halo rows are re-read from L2.  Inputs are
// of two kinds: "halo" inputs, read with their four neighbours (fields in the forward pass,
// upstream sensitivities in the adjoint), and "centre" inputs read only at the node itself
// (sources in the forward pass, fields in a nonlinear adjoint).
//
// Boundary handling (Section 2.3 / Appendix A.4) is part of the same launch:
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
    float hscale[2];
    int n0, n1, nc4;
    int periodic, mask_in, mask_out;
    int rows_per_item, ncb, nitems;
    float ih0, ih1;      // 1/h0^2, 1/h1^2
    float c[4];
    float* partials;
};

// out = -Lap u - f
struct PoissonFwd {
    static constexpr int NH = 1, NC = 1, NO = 1;
    static constexpr bool SCALE = false;
    __device__ static void eval(const float* v, const float* lap, const float* cc, const float* c, float* o) {
        o[0] = -lap[0] - cc[0];
    }
};
// g = -Lap G  (the Jacobian is constant and symmetric on the rows)
struct PoissonBwd {
    static constexpr int NH = 1, NC = 0, NO = 1;
    static constexpr bool SCALE = true;
    __device__ static void eval(const float* v, const float* lap, const float* cc, const float* c, float* o) {
        o[0] = -lap[0];
    }
};
// c = {D_u, D_v, F, F+k}
struct GrayScottFwd {
    static constexpr int NH = 2, NC = 0, NO = 2;
    static constexpr bool SCALE = false;
    __device__ static void eval(const float* v, const float* lap, const float* cc, const float* c, float* o) {
        const float u = v[0], w = v[1], uww = u * w * w;
        o[0] = c[0] * lap[0] - uww + c[2] * (1.f - u);
        o[1] = c[1] * lap[1] + uww - c[3] * w;
    }
};
// g_u = D_u Lap G_u + G_u (-v^2 - F) + G_v v^2 ;  g_v = D_v Lap G_v + G_u (-2uv) + G_v (2uv - (F+k))
struct GrayScottBwd {
    static constexpr int NH = 2, NC = 2, NO = 2;
    static constexpr bool SCALE = true;
    __device__ static void eval(const float* v, const float* lap, const float* cc, const float* c, float* o) {
        const float a = v[0], b = v[1], u = cc[0], w = cc[1];
        const float ww = w * w, uw2 = 2.f * u * w;
        o[0] = c[0] * lap[0] + a * (-ww - c[2]) + b * ww;
        o[1] = c[1] * lap[1] - a * uw2 + b * (uw2 - c[3]);
    }
};

template <class F, int U>
__global__ void __launch_bounds__(256) lap2d_kernel(const Lap2dParams p) {
    constexpr int NH = F::NH, NC = F::NC, NO = F::NO;
    constexpr int NCA = NC > 0 ? NC : 1;
    const int item = blockIdx.x;
    const int cb = item % p.ncb, rc = item / p.ncb;
    const int c4 = cb * blockDim.x + threadIdx.x;
    const bool cvalid = c4 < p.nc4;
    const bool first_col = c4 == 0, last_col = c4 == p.nc4 - 1;
    const int n0 = p.n0, n1 = p.n1;
    const int a0 = rc * p.rows_per_item;
    const int a1 = min(a0 + p.rows_per_item, n0);

    // resolved row index of a halo-input row, or -1 if it reads as zero
    auto in_row = [&](int row) -> int {
        if (p.periodic) return row < 0 ? row + n0 : (row >= n0 ? row - n0 : row);
        if (row < 0 || row >= n0) return -1;
        if (p.mask_in && (row < 1 || row > n0 - 2)) return -1;
        return row;
    };
    auto load_h = [&](int k, int row) -> float4 {
        const int r = in_row(row);
        if (r < 0 || !cvalid) return f4zero();
        float4 v = ld4(p.hin[k] + (size_t)r * n1 + 4 * c4);
        if (F::SCALE) v = f4scale(v, p.hscale[k]);
        if (p.mask_in) {
            if (first_col) v.x = 0.f;
            if (last_col) v.w = 0.f;
        }
        return v;
    };

    float4 prev[NH], cur[NH];
#pragma unroll
    for (int k = 0; k < NH; ++k) { prev[k] = load_h(k, a0 - 1); cur[k] = load_h(k, a0); }
    float acc[NO];
#pragma unroll
    for (int e = 0; e < NO; ++e) acc[e] = 0.f;

    for (int a = a0; a < a1; a += U) {
        float4 nxt[U][NH];
        float4 cen[U][NCA];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const bool need = a + u < a1;
#pragma unroll
            for (int k = 0; k < NH; ++k) nxt[u][k] = need ? load_h(k, a + u + 1) : f4zero();
#pragma unroll
            for (int k = 0; k < NC; ++k)
                cen[u][k] = (need && cvalid) ? ld4(p.cin[k] + (size_t)(a + u) * n1 + 4 * c4) : f4zero();
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int row = a + u;
            if (row < a1) {                       // uniform over the block
                LR2 lr[NH];
                const int r = in_row(row);
#pragma unroll
                for (int k = 0; k < NH; ++k) {
                    if (r >= 0) {
                        lr[k] = lane_neighbours<1>(p.hin[k] + (size_t)r * n1, c4, p.nc4, cur[k],
                                                   p.periodic != 0, F::SCALE ? p.hscale[k] : 1.f);
                    } else {
                        lr[k].l1 = lr[k].r1 = lr[k].l2 = lr[k].r2 = 0.f;
                    }
                }
                float o[NO][4];
#pragma unroll
                for (int comp = 0; comp < 4; ++comp) {
                    float v[NH], lap[NH], cc[NCA], oo[NO];
#pragma unroll
                    for (int k = 0; k < NH; ++k) {
                        const float c = f4get(cur[k], comp);
                        const float left = comp == 0 ? lr[k].l1 : f4get(cur[k], comp - 1);
                        const float right = comp == 3 ? lr[k].r1 : f4get(cur[k], comp + 1);
                        const float up = f4get(prev[k], comp), dn = f4get(nxt[u][k], comp);
                        v[k] = c;
                        lap[k] = ((up - c) + (dn - c)) * p.ih0 + ((left - c) + (right - c)) * p.ih1;
                    }
#pragma unroll
                    for (int k = 0; k < NC; ++k) cc[k] = f4get(cen[u][k], comp);
                    F::eval(v, lap, cc, p.c, oo);
#pragma unroll
                    for (int e = 0; e < NO; ++e) o[e][comp] = oo[e];
                }
                if (p.mask_out) {
                    const bool rowless = row < 1 || row > n0 - 2;
#pragma unroll
                    for (int e = 0; e < NO; ++e) {
                        if (rowless) { o[e][0] = o[e][1] = o[e][2] = o[e][3] = 0.f; }
                        if (first_col) o[e][0] = 0.f;
                        if (last_col) o[e][3] = 0.f;
                    }
                }
                if (cvalid) {
#pragma unroll
                    for (int e = 0; e < NO; ++e) {
                        const float4 ov = make_float4(o[e][0], o[e][1], o[e][2], o[e][3]);
                        st4(p.out[e] + (size_t)row * n1 + 4 * c4, ov);
                        acc[e] += sq4(ov);
                    }
                }
#pragma unroll
                for (int k = 0; k < NH; ++k) { prev[k] = cur[k]; cur[k] = nxt[u][k]; }
            }
        }
    }
    if (p.partials != nullptr) block_reduce_store<NO>(acc, p.partials, p.nitems, item);
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
    block = std::max(32, std::min(256, (block / 32) * 32));
    p.rows_per_item = env_int("FPDE_LAP2D_ROWS", 16);
    p.ncb = (p.nc4 + block - 1) / block;
    p.nitems = p.ncb * ((p.n0 + p.rows_per_item - 1) / p.rows_per_item);
    p.ih0 = (float)(1.0 / (q.h[0] * q.h[0]));
    p.ih1 = (float)(1.0 / (q.h[1] * q.h[1]));
}

int lap2d_items(const int* n) {
    Problem q{}; q.n[0] = n[0]; q.n[1] = n[1]; q.h[0] = q.h[1] = 1.0;
    Lap2dParams p{}; int block;
    lap2d_geometry(q, p, block);
    return p.nitems;
}

template <class F>
static cudaError_t launch(const Lap2dParams& p, int block, cudaStream_t s) {
    lap2d_kernel<F, 4><<<p.nitems, block, 0, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_lap2d_fwd(const Problem& q) {
    Lap2dParams p{}; int block;
    lap2d_geometry(q, p, block);
    p.partials = q.partials;
    const bool gs = q.op == 2;
    p.periodic = gs; p.mask_in = 0; p.mask_out = !gs;
    p.hin[0] = q.in[0]; p.out[0] = q.out[0];
    if (gs) {
        p.hin[1] = q.in[1]; p.out[1] = q.out[1];
        p.c[0] = (float)q.coef[0]; p.c[1] = (float)q.coef[1]; p.c[2] = (float)q.coef[2];
        p.c[3] = (float)(q.coef[2] + q.coef[3]);
        return launch<GrayScottFwd>(p, block, q.stream);
    }
    p.cin[0] = q.aux[0];
    return launch<PoissonFwd>(p, block, q.stream);
}

cudaError_t launch_lap2d_bwd(const Problem& q) {
    Lap2dParams p{}; int block;
    lap2d_geometry(q, p, block);
    p.partials = nullptr;
    const bool gs = q.op == 2;
    p.periodic = gs; p.mask_in = !gs; p.mask_out = 0;
    p.hin[0] = q.aux[0]; p.out[0] = q.out[0]; p.hscale[0] = (float)q.gscale[0];
    if (gs) {
        p.hin[1] = q.aux[1]; p.out[1] = q.out[1]; p.hscale[1] = (float)q.gscale[1];
        p.cin[0] = q.in[0]; p.cin[1] = q.in[1];
        p.c[0] = (float)q.coef[0]; p.c[1] = (float)q.coef[1]; p.c[2] = (float)q.coef[2];
        p.c[3] = (float)(q.coef[2] + q.coef[3]);
        return launch<GrayScottBwd>(p, block, q.stream);
    }
    return launch<PoissonBwd>(p, block, q.stream);
}

}  // namespace fpde
