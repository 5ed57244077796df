// Fourth-order Helmholtz operator, loss-specialised single pass: residual (Section 2.1), mean-square
// loss and its gradient through the discrete adjoint (Sections 2.2, 2.3) in ONE kernel, with the
// residual planes handed from the forward stencil to the adjoint stencil through shared memory and
// never written to global memory (unless the caller asks for them).
//
//   g = S^T G,  G = (2/N_r) r on the rows, 0 elsewhere,  r = S u - f   (S: the 13-point star + k^2)
//
// Structure (one persistent CTA per SM, warp-specialised):
//   * a producer warp streams plane tiles of u (TYB + 8 rows: halo 4, because the rows of r the
//     adjoint needs reach two rows beyond the tile, and each of those needs u two rows further)
//     and of f (TYB + 4 rows) through a ring in shared memory with the copy engine;
//   * the A warps apply the star to u by partial sums along x (four partial outputs per thread in
//     registers, as in op_helmholtz3d_tma.cu), subtract f, zero the nodes without a row, add the
//     squares of the tile's own nodes to the loss, and store the finished plane of r (TYB + 4 rows)
//     into a second, small ring in shared memory;
//   * the B warps apply the star (scaled by 2/N_r) to those planes of r, again by partial sums
//     along x, and store the finished planes of g.
// A tile spans whole z lines (extents of 128 or 256), so r beyond the tile in z is r beyond the
// grid, i.e. zero, and needs no recomputation; in y the A warps recompute a ring of two rows, in
// x a segment of planes [a0, a1) streams u on [a0-4, a1+4).
//
// Every wait is bounded (tma_common.cuh); star3d_fused_timeouts() reports waits that gave up.
#include "fpde_common.cuh"
#include "fpde_internal.h"
#include "tma_common.cuh"

#include <algorithm>
#include <cstdlib>
#include <type_traits>

namespace fpde {

struct HfParams {
    CUtensorMap map_u;       // box NZ x (TYB+8) x 1
    CUtensorMap map_f;       // box NZ x (TYB+4) x 1
    float* g;
    float* r;                // residual array, or NULL = not stored
    int n0, n1, n2;
    int ntiles;
    long long work;          // ntiles * n0 tile-planes, shared out evenly over the CTAs
    float2 w16[3], nw[3], kc;        // forward star
    float2 gw16[3], gnw[3], gkc;     // adjoint star, scale 2/N_r folded in
    float* partials;
};

__device__ unsigned int g_star3d_fused_timeouts = 0;

struct HfSegment { int tile, a0, a1; };
__device__ __forceinline__ bool hf_next_segment(long long& pos, long long end, int n0, HfSegment& g) {
    if (pos >= end) return false;
    g.tile = (int)(pos / n0);
    g.a0 = (int)(pos - (long long)g.tile * n0);
    const long long left = end - pos;
    g.a1 = (int)((long long)(n0 - g.a0) < left ? n0 : g.a0 + left);
    pos += g.a1 - g.a0;
    return true;
}

struct HfWeights { float2 w16x, w16y, w16z, nwx, nwy, nwz, kc; };

// One plane arrives: L = rows -2 .. RY+1 around the thread's RY rows at its float4 column, zl / zr
// the two floats left / right of it.  A0..A3 hold the partial outputs of planes b-2 .. b+1; o
// receives the completed plane b-2, A0 the first term of plane b+2.
template <int RY>
__device__ __forceinline__ void hf_star_step(const V4 (&L)[RY + 4], const float2 (&zl)[RY], const float2 (&zr)[RY],
                                             const HfWeights& w, V4 (&A0)[RY], V4 (&A1)[RY], V4 (&A2)[RY],
                                             V4 (&A3)[RY], V4 (&o)[RY]) {
#pragma unroll
    for (int j = 0; j < RY; ++j) {
        const V4 c = L[j + 2];
        const V4 s1y = v4add(L[j + 1], L[j + 3]), s2y = v4add(L[j], L[j + 4]);
        V4 s1z, s2z;
        s1z.lo = make_float2(zl[j].y + c.lo.y, c.lo.x + c.hi.x);
        s1z.hi = make_float2(c.lo.y + c.hi.y, c.hi.x + zr[j].x);
        s2z.lo = add2(zl[j], c.hi);                          // (z-2, z-1) + (z+2, z+3): both register pairs
        s2z.hi = add2(c.lo, zr[j]);
        A2[j] = v4fma(s1y, w.w16y, A2[j]);
        A2[j] = v4fma(s2y, w.nwy, A2[j]);
        A2[j] = v4fma(c, w.kc, A2[j]);
        A2[j] = v4fma(s1z, w.w16z, A2[j]);
        A2[j] = v4fma(s2z, w.nwz, A2[j]);
        const V4 t = v4mul(c, w.nwx);
        o[j] = v4add(A0[j], t);
        A1[j] = v4fma(c, w.w16x, A1[j]);
        A3[j] = v4fma(c, w.w16x, A3[j]);
        A0[j] = t;
    }
}

// NZW: warps along a z line (n2 = 128 NZW).  TYB: rows of g per tile.  RY: rows per thread.
// ST: stages of the u / f ring.  RS: stages of the r ring.
template <int NZW, int TYB, int RY, int ST, int RS>
__global__ void __launch_bounds__(32 * (NZW * ((TYB + 4) / RY + TYB / RY) + 1), 1)
star3d_fused_kernel(const __grid_constant__ HfParams p) {
    constexpr int NZ = 128 * NZW;                          // floats per z line
    constexpr int NA = NZW * ((TYB + 4) / RY);             // warps of the forward stage
    constexpr int NB = NZW * (TYB / RY);                   // warps of the adjoint stage
    constexpr uint32_t UB = (uint32_t)((TYB + 8) * NZ * 4);
    constexpr uint32_t FB = (uint32_t)((TYB + 4) * NZ * 4);
    constexpr uint32_t STAGE = UB + FB;                    // multiples of 128 bytes
    constexpr uint32_t RB = (uint32_t)((TYB + 4) * NZ * 4);
    constexpr uint32_t ROW = (uint32_t)(NZ * 4);
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long bars[2 * ST + 2 * RS];   // full, empty, r_full, r_empty

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    // 128 bytes of slack in front: the first lane of a line reads (and discards) the 8 bytes before it
    const uint32_t base = ((smem_u32(smem_raw) + 127u) & ~127u) + 128u;
    const uint32_t rbase = base + (uint32_t)ST * STAGE;
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = full0 + 8u * ST;
    const uint32_t rfull0 = empty0 + 8u * ST, rempty0 = rfull0 + 8u * RS;
    long long pos = p.work * (long long)blockIdx.x / (long long)gridDim.x;
    const long long end = p.work * (long long)(blockIdx.x + 1) / (long long)gridDim.x;

    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < ST; ++s) { mbar_init(full0 + 8u * s, 1); mbar_init(empty0 + 8u * s, NA); }
#pragma unroll
        for (int s = 0; s < RS; ++s) { mbar_init(rfull0 + 8u * s, NA); mbar_init(rempty0 + 8u * s, NB); }
        mbar_fence_init();
    }
    __syncthreads();
    pdl_wait_then_trigger();

    bool gave_up = false;
    float2 acc = make_float2(0.f, 0.f);
    double acc_long = 0.0;
    HfSegment g;
    const float2 zero2 = make_float2(0.f, 0.f);
    const size_t PS = (size_t)p.n1 * p.n2;

    if (warp == NA + NB) {
        // ---- producer ----
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0; bool first_round = true;
            while (hf_next_segment(pos, end, p.n0, g)) {
                const int m0 = g.tile * TYB;
                const int nb = g.a1 - g.a0 + 8;            // planes a0-4 .. a1+3
                for (int s = 0; s < nb; ++s) {
                    if (!first_round) mbar_wait(empty0 + 8u * stage, phase ^ 1u, gave_up, &g_star3d_fused_timeouts);
                    const bool with_f = s >= 4;            // f of the plane of r this step completes (a0-6+s)
                    const uint32_t fb = full0 + 8u * stage, dst = base + (uint32_t)stage * STAGE;
                    mbar_expect_tx(fb, UB + (with_f ? FB : 0u));
                    tma_load_3d(dst, &p.map_u, 0, m0 - 4, g.a0 - 4 + s, fb);
                    if (with_f) tma_load_3d(dst + UB, &p.map_f, 0, m0 - 2, g.a0 - 6 + s, fb);
                    if (++stage == ST) { stage = 0; phase ^= 1u; first_round = false; }
                }
            }
        }
    } else if (warp < NA) {
        // ---- forward stage: rows m0-2 + wr RY + j of r, from u ----
        const int wz = warp % NZW, wr = warp / NZW;
        const int c4 = wz * 32 + lane;                     // float4 column of the z line
        const bool first_col = c4 == 0, last_col = c4 == NZ / 4 - 1;
        const uint32_t u_off = (uint32_t)((wr * RY) * NZ + 4 * c4) * 4u;     // u-tile row wr RY = global row m0-4+wr RY
        const uint32_t f_off = UB + (uint32_t)((wr * RY) * NZ + 4 * c4) * 4u;
        const uint32_t r_off = (uint32_t)((wr * RY) * NZ + 4 * c4) * 4u;
        HfWeights w;
        w.w16x = p.w16[0]; w.w16y = p.w16[1]; w.w16z = p.w16[2];
        w.nwx = p.nw[0]; w.nwy = p.nw[1]; w.nwz = p.nw[2]; w.kc = p.kc;
        int stage = 0; uint32_t phase = 0;
        int rstage = 0; uint32_t rphase = 0; bool rfirst = true;
        while (hf_next_segment(pos, end, p.n0, g)) {
            const int m0 = g.tile * TYB;
            const int mrow = m0 - 2 + wr * RY;             // first row of r of this thread
            bool keep_lo[RY], keep_hi[RY], own[RY];
#pragma unroll
            for (int j = 0; j < RY; ++j) {
                const int m = mrow + j;
                const bool row_in = m >= 2 && m <= p.n1 - 3;
                keep_lo[j] = row_in && !first_col;         // columns 0,1 / n-2,n-1 carry no row
                keep_hi[j] = row_in && !last_col;
                own[j] = m >= m0 && m < m0 + TYB && m < p.n1;     // the tile's own rows: counted in the loss here
            }
            float* rptr = p.r != nullptr ? p.r + ((size_t)g.a0 * p.n1 + (size_t)max(mrow, 0)) * (size_t)p.n2 + (size_t)(4 * c4) : nullptr;
            V4 R0[RY], R1[RY], R2[RY], R3[RY];
#pragma unroll
            for (int j = 0; j < RY; ++j) { R0[j] = v4zero(); R1[j] = v4zero(); R2[j] = v4zero(); R3[j] = v4zero(); }
            // Step s: plane a0-4+s of u arrives; from s = 4 on it completes plane a = a0-6+s of r.
            auto step = [&](auto emit_tag, int a, V4 (&A0)[RY], V4 (&A1)[RY], V4 (&A2)[RY], V4 (&A3)[RY]) {
                constexpr bool EMIT = decltype(emit_tag)::value;
                const uint32_t bar = full0 + 8u * (uint32_t)stage;
                mbar_wait(bar, phase, gave_up, &g_star3d_fused_timeouts);
                const uint32_t sb = base + (uint32_t)stage * STAGE;
                const uint32_t us = sb + u_off;
                V4 L[RY + 4];
#pragma unroll
                for (int i = 0; i < RY + 4; ++i) L[i] = ldsv4(us + (uint32_t)i * ROW);
                float2 zl[RY], zr[RY];
#pragma unroll
                for (int j = 0; j < RY; ++j) {
                    zl[j] = ldsv2(us + (uint32_t)(j + 2) * ROW - 8u);
                    zr[j] = ldsv2(us + (uint32_t)(j + 2) * ROW + 16u);
                    if (first_col) zl[j] = zero2;          // beyond the z line
                    if (last_col) zr[j] = zero2;
                }
                V4 src[RY];
                if (EMIT) {
#pragma unroll
                    for (int j = 0; j < RY; ++j) src[j] = ldsv4(sb + f_off + (uint32_t)j * ROW);
                }
                V4 o[RY];
                hf_star_step<RY>(L, zl, zr, w, A0, A1, A2, A3, o);
                // the u / f stage has been consumed
                __syncwarp();
                if (lane == 0) mbar_arrive(bar + 8u * ST);
                if (++stage == ST) { stage = 0; phase ^= 1u; }
                if (EMIT) {
                    const bool plane_in = a >= 2 && a <= p.n0 - 3;
                    const bool plane_own = a >= g.a0 && a < g.a1;
                    const uint32_t rb = rbase + (uint32_t)rstage * RB + r_off;
                    if (!rfirst) mbar_wait(rempty0 + 8u * (uint32_t)rstage, rphase ^ 1u, gave_up, &g_star3d_fused_timeouts);
#pragma unroll
                    for (int j = 0; j < RY; ++j) {
                        V4 r = v4sub(o[j], src[j]);
                        if (!(plane_in && keep_lo[j])) r.lo = zero2;
                        if (!(plane_in && keep_hi[j])) r.hi = zero2;
                        stsv4(rb + (uint32_t)j * ROW, r);
                        if (plane_own && own[j]) {
                            acc = fma2(r.lo, r.lo, fma2(r.hi, r.hi, acc));
                            if (rptr != nullptr) stv4(rptr + (size_t)(a - g.a0) * PS + (size_t)(mrow + j - max(mrow, 0)) * p.n2, r.lo, r.hi);
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(rfull0 + 8u * (uint32_t)rstage);      // release: the plane of r is in shared memory
                    if (++rstage == RS) { rstage = 0; rphase ^= 1u; rfirst = false; }
                }
            };
            using No = std::false_type;
            using Yes = std::true_type;
            step(No{}, 0, R0, R1, R2, R3);
            step(No{}, 0, R1, R2, R3, R0);
            step(No{}, 0, R2, R3, R0, R1);
            step(No{}, 0, R3, R0, R1, R2);
            int a = g.a0 - 2, group = 0;                   // planes a0-2 .. a1+1 of r
            const int a_end = g.a1 + 2;
            for (; a + 4 <= a_end; a += 4) {
                step(Yes{}, a, R0, R1, R2, R3);
                step(Yes{}, a + 1, R1, R2, R3, R0);
                step(Yes{}, a + 2, R2, R3, R0, R1);
                step(Yes{}, a + 3, R3, R0, R1, R2);
                if ((++group & 3) == 0) { acc_long += (double)(acc.x + acc.y); acc = zero2; }
            }
            if (a < a_end) step(Yes{}, a, R0, R1, R2, R3);
            if (a + 1 < a_end) step(Yes{}, a + 1, R1, R2, R3, R0);
            if (a + 2 < a_end) step(Yes{}, a + 2, R2, R3, R0, R1);
        }
    } else {
        // ---- adjoint stage: rows m0 + wr RY + j of g, from the planes of r in shared memory ----
        const int wb = warp - NA;
        const int wz = wb % NZW, wr = wb / NZW;
        const int c4 = wz * 32 + lane;
        const bool first_col = c4 == 0, last_col = c4 == NZ / 4 - 1;
        const uint32_t r_off = (uint32_t)((wr * RY) * NZ + 4 * c4) * 4u;    // r-tile row wr RY = global row m0-2+wr RY
        HfWeights w;
        w.w16x = p.gw16[0]; w.w16y = p.gw16[1]; w.w16z = p.gw16[2];
        w.nwx = p.gnw[0]; w.nwy = p.gnw[1]; w.nwz = p.gnw[2]; w.kc = p.gkc;
        int rstage = 0; uint32_t rphase = 0;
        while (hf_next_segment(pos, end, p.n0, g)) {
            const int m0 = g.tile * TYB;
            const int mrow = m0 + wr * RY;
            float* optr = p.g + ((size_t)g.a0 * p.n1 + mrow) * (size_t)p.n2 + (size_t)(4 * c4);
            bool row_ok[RY];
#pragma unroll
            for (int j = 0; j < RY; ++j) row_ok[j] = mrow + j < p.n1;
            V4 R0[RY], R1[RY], R2[RY], R3[RY];
#pragma unroll
            for (int j = 0; j < RY; ++j) { R0[j] = v4zero(); R1[j] = v4zero(); R2[j] = v4zero(); R3[j] = v4zero(); }
            // Step t: plane a0-2+t of r arrives; from t = 4 on it completes plane a0-4+t of g.
            auto step = [&](auto emit_tag, V4 (&A0)[RY], V4 (&A1)[RY], V4 (&A2)[RY], V4 (&A3)[RY]) {
                constexpr bool EMIT = decltype(emit_tag)::value;
                const uint32_t bar = rfull0 + 8u * (uint32_t)rstage;
                mbar_wait(bar, rphase, gave_up, &g_star3d_fused_timeouts);
                const uint32_t rs = rbase + (uint32_t)rstage * RB + r_off;
                V4 L[RY + 4];
#pragma unroll
                for (int i = 0; i < RY + 4; ++i) L[i] = ldsv4(rs + (uint32_t)i * ROW);
                float2 zl[RY], zr[RY];
#pragma unroll
                for (int j = 0; j < RY; ++j) {
                    zl[j] = ldsv2(rs + (uint32_t)(j + 2) * ROW - 8u);
                    zr[j] = ldsv2(rs + (uint32_t)(j + 2) * ROW + 16u);
                    if (first_col) zl[j] = zero2;
                    if (last_col) zr[j] = zero2;
                }
                V4 o[RY];
                hf_star_step<RY>(L, zl, zr, w, A0, A1, A2, A3, o);
                __syncwarp();
                if (lane == 0) mbar_arrive(bar + 8u * RS);
                if (++rstage == RS) { rstage = 0; rphase ^= 1u; }
                if (EMIT) {
#pragma unroll
                    for (int j = 0; j < RY; ++j)
                        if (row_ok[j]) stv4(optr + (size_t)j * p.n2, o[j].lo, o[j].hi);
                    optr += PS;
                }
            };
            using No = std::false_type;
            using Yes = std::true_type;
            step(No{}, R0, R1, R2, R3);
            step(No{}, R1, R2, R3, R0);
            step(No{}, R2, R3, R0, R1);
            step(No{}, R3, R0, R1, R2);
            int a = g.a0;
            for (; a + 4 <= g.a1; a += 4) {
                step(Yes{}, R0, R1, R2, R3);
                step(Yes{}, R1, R2, R3, R0);
                step(Yes{}, R2, R3, R0, R1);
                step(Yes{}, R3, R0, R1, R2);
            }
            if (a < g.a1) step(Yes{}, R0, R1, R2, R3);
            if (a + 1 < g.a1) step(Yes{}, R1, R2, R3, R0);
            if (a + 2 < g.a1) step(Yes{}, R2, R3, R0, R1);
        }
    }
    if (p.partials != nullptr) {
        float s[1] = {(float)(acc_long + (double)(acc.x + acc.y))};
        block_reduce_store<1>(s, p.partials, gridDim.x, blockIdx.x);
    }
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
constexpr int HF_MAX_CTAS = 1024;

// Grids the single-pass kernel takes: z lines of 128 or 256 floats (one tile spans the line), at
// least one full tile of rows and a few planes.
bool star3d_fused_supported(const int* n) {
    if (tma_encode_fn() == nullptr) return false;
    return (n[2] == 128 || n[2] == 256) && n[1] >= 16 && n[0] >= 8;
}

int star3d_fused_items(const int*) { return HF_MAX_CTAS; }

template <int NZW, int TYB, int RY, int ST, int RS>
static cudaError_t hf_launch(const Problem& q, HfParams& p, int* items) {
    constexpr int NZ = 128 * NZW;
    constexpr size_t smem = (size_t)ST * ((TYB + 8) * NZ * 4 + (TYB + 4) * NZ * 4) + (size_t)RS * ((TYB + 4) * NZ * 4) + 256;
    constexpr int threads = 32 * (NZW * ((TYB + 4) / RY + TYB / RY) + 1);
    auto kern = star3d_fused_kernel<NZW, TYB, RY, ST, RS>;
    static int slots_of[64];
    int dev = 0;
    cudaError_t ce = cudaGetDevice(&dev);
    if (ce != cudaSuccess) return ce;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (slots_of[dev] == 0) {
        ce = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (ce != cudaSuccess) return ce;
        int sms = 0, per_sm = 0;
        ce = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (ce != cudaSuccess) return ce;
        ce = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, threads, smem);
        if (ce != cudaSuccess) return ce;
        if (per_sm < 1) return cudaErrorLaunchOutOfResources;
        slots_of[dev] = sms * per_sm;
    }
    const long long G = std::max(1ll, std::min<long long>(std::min(slots_of[dev], HF_MAX_CTAS), p.work / 16));
    if (items) *items = (int)G;
    return launch_kernel_smem(kern, dim3((unsigned)G), dim3(threads, 1, 1), smem, q.stream, p);
}

// q.in[0] = u, q.aux[0] = f, q.out[0] = g; res = residual array or NULL.
cudaError_t launch_star3d_fused(const Problem& q, float* res, int* items) {
    constexpr int TYB = 8;
    HfParams p{};
    p.n0 = q.n[0]; p.n1 = q.n[1]; p.n2 = q.n[2];
    p.ntiles = (p.n1 + TYB - 1) / TYB;
    p.work = (long long)p.ntiles * p.n0;
    const long long n0 = p.n0, n1 = p.n1, n2 = p.n2;
    if (!tma_encode_3d(&p.map_u, q.in[0], n2, n1, n0, n2, n1 * n2, p.n2, TYB + 8)) return cudaErrorInvalidValue;
    if (!tma_encode_3d(&p.map_f, q.aux[0], n2, n1, n0, n2, n1 * n2, p.n2, TYB + 4)) return cudaErrorInvalidValue;
    const double gs = 2.0 / (double)q.rows;
    double wsum = 0.0;
    for (int a = 0; a < 3; ++a) {
        const double w = 1.0 / (12.0 * q.h[a] * q.h[a]);
        p.w16[a] = make_float2((float)(16.0 * w), (float)(16.0 * w));
        p.nw[a] = make_float2((float)(-w), (float)(-w));
        p.gw16[a] = make_float2((float)(16.0 * w * gs), (float)(16.0 * w * gs));
        p.gnw[a] = make_float2((float)(-w * gs), (float)(-w * gs));
        wsum += w;
    }
    const double kc = q.coef[0] * q.coef[0] - 30.0 * wsum;
    p.kc = make_float2((float)kc, (float)kc);
    p.gkc = make_float2((float)(kc * gs), (float)(kc * gs));
    p.g = q.out[0];
    p.r = res;
    p.partials = q.partials;
    if (p.n2 == 256) return hf_launch<2, TYB, 2, 4, 3>(q, p, items);
    return hf_launch<1, TYB, 2, 4, 3>(q, p, items);
}

unsigned int star3d_fused_timeouts() {
    unsigned int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_star3d_fused_timeouts, sizeof(v)) != cudaSuccess) { (void)cudaGetLastError(); return ~0u; }
    return v;
}

}  // namespace fpde
