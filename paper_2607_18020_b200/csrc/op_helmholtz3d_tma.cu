// Fourth-order Helmholtz star, r = Lap4 u + k^2 u - f (Section 2.1), and its gather-form adjoint
// with the two-cell boundary band (Sections 2.2, 2.3): the engine that stages plane tiles through
// shared memory with the copy engine (cp.async.bulk.tensor, each copy to the issuing CTA only).
//
// How it differs from the L1-staged engine (op_helmholtz3d.cu), which holds every load of a step in
// registers while it is in flight and issues five 128-bit loads per output float4:
//   * the data in flight lives in shared memory: a producer warp keeps a ring of ST plane tiles
//     (with their halo of 2 rows and 4 floats) filled ST-1 planes ahead of the consumers, so the
//     consumers only ever issue shared-memory loads of short, fixed latency;
//   * a thread owns RY adjacent rows of one float4 column: the RY+4 rows it reads per plane serve
//     RY outputs (3 loads per output at RY = 2, 2 at RY = 4, against 5);
//   * the x direction needs no window of planes at all: each arriving plane b is scattered into
//     the four partial outputs b-1 .. b+2 the thread keeps in registers and completes output b-2
//     (partial sums along the marching axis), so a plane is read from shared memory in the step
//     it arrives and never again;
//   * zero extension comes from the tensor map: a box that reaches beyond the array is filled
//     with zeros, and the adjoint of an arbitrary upstream array (whose entries off the rows must
//     read as zero) uses a map of the sub-array of rows in x and y, so its band in those axes costs
//     nothing; only the band in z (whose start is not 16-byte aligned) is masked in registers;
//   * the grid is persistent: one CTA per slot the device holds at once, each with an equal share
//     of the (tile, plane) pairs, so there is no partial last wave.
//
// What was measured on 256^3 (kernel durations, cold caches): the ring alone, with consumers that
// only hand the stages back, streams the adjoint's input in 16-18 us and the forward's two inputs
// in 30 us; the consumers alone, computing on whatever is in shared memory, take 21-23 us -- with
// about 90 executed instructions per output float4 (a third of them the packed arithmetic) they
// are bound by instruction issue at 0.4-0.5 per cycle and scheduler, as the L1-staged kernels
// are.  Together: adjoint 24.8 us (L1-staged: 29.5), forward 36 us (L1-staged: 34, within a
// tenth of its DRAM time), so the adjoint runs here by default and the forward pass does not.
//
// Every wait is bounded (tma_common.cuh); star3d_tma_timeouts() reports waits that gave up.
#include "fpde_common.cuh"
#include "fpde_internal.h"
#include "tma_common.cuh"

#include <algorithm>
#include <cstdlib>
#include <type_traits>

namespace fpde {

constexpr int S3T_TX = 32;                 // lanes along z: one warp spans a 128-float segment of a row
constexpr int S3T_TZ = 4 * S3T_TX;         // floats of z per tile
constexpr int S3T_WP = S3T_TZ + 8;         // row pitch of the halo tile in shared memory (floats)

struct Star3dTmaParams {
    CUtensorMap map_h;       // array read with halo: box (TZ+8) x (TYB+4) x 1
    CUtensorMap map_c;       // source array (forward): box TZ x TYB x 1
    float* out;
    int n0, n1, n2, nc4;
    int ox, oy;              // origin of map_h inside the grid (2,2 for the adjoint's sub-array of rows)
    int ncb, ntiles;         // tiles along z, tiles in all
    long long work;          // ntiles * n0 tile-planes, shared out evenly over the CTAs
    float2 w16[3], nw[3], kc;
    float* partials;
};

__device__ unsigned int g_star3d_tma_timeouts = 0;

// Work distribution: the (tile, plane) pairs, tile-major, form one sequence of `work` tile-planes;
// CTA k of G takes the contiguous range [k work / G, (k+1) work / G).  A range is one or more
// segments (runs of planes of one tile); a segment [a0, a1) passes planes a0-2 .. a1+1 through the
// ring.  Every CTA gets the same number of output planes to within one, whatever the grid and the
// number of SMs, and the assignment depends on nothing but G, so the loss partial sums (one per
// CTA) are reproducible.
struct S3tSegment { int tile, a0, a1; };
__device__ __forceinline__ bool s3t_next_segment(long long& pos, long long end, int n0, S3tSegment& g) {
    if (pos >= end) return false;
    g.tile = (int)(pos / n0);
    g.a0 = (int)(pos - (long long)g.tile * n0);
    const long long left = end - pos;
    g.a1 = (int)((long long)(n0 - g.a0) < left ? n0 : g.a0 + left);
    pos += g.a1 - g.a0;
    return true;
}

// MODE 0: forward.  MODE 1: adjoint of an arbitrary upstream array.  MODE 2: adjoint of an upstream
// array that is zero off the rows (the residual array the forward kernel of the same call wrote).
template <int MODE, int TYB, int RY, int ST, int MINB>
__global__ void __launch_bounds__(S3T_TX * (TYB / RY) + 32, MINB)
star3d_tma_kernel(const __grid_constant__ Star3dTmaParams p) {
    constexpr bool FWD = MODE == 0;
    constexpr int NCW = TYB / RY;                          // consumer warps
    constexpr uint32_t HB = (uint32_t)((TYB + 4) * S3T_WP * 4);          // bytes of a halo tile
    constexpr uint32_t CB = FWD ? (uint32_t)(TYB * S3T_TZ * 4) : 0u;     // bytes of a source tile
    constexpr uint32_t STAGE = ((HB + CB + 127u) / 128u) * 128u;
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long bars[2 * ST];          // full[0..ST), empty[ST..2ST)

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = full0 + 8u * ST;
    long long pos = p.work * (long long)blockIdx.x / (long long)gridDim.x;
    const long long end = p.work * (long long)(blockIdx.x + 1) / (long long)gridDim.x;

    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < ST; ++s) { mbar_init(full0 + 8u * s, 1); mbar_init(empty0 + 8u * s, NCW); }
        mbar_fence_init();
    }
    __syncthreads();
    pdl_wait_then_trigger();          // nothing of the previous kernel's output is read before this

    bool gave_up = false;
    float2 acc = make_float2(0.f, 0.f);
    double acc_long = 0.0;            // the fp32 sums of squares are folded into this every few steps
    int stage = 0;                    // ring position and its phase, running on across segments
    uint32_t phase = 0;
    S3tSegment g;

    if (warp == NCW) {
        // ---- producer: one lane keeps the ring filled ----
        if (lane == 0) {
            bool first_round = true;
            while (s3t_next_segment(pos, end, p.n0, g)) {
                const int z0 = (g.tile % p.ncb) * S3T_TZ, m0 = (g.tile / p.ncb) * TYB;
                const int nb = g.a1 - g.a0 + 4;
                for (int s = 0; s < nb; ++s) {
                    if (!first_round) mbar_wait(empty0 + 8u * stage, phase ^ 1u, gave_up, &g_star3d_tma_timeouts);
                    const bool with_src = FWD && s >= 4;       // the source tile of the plane this step completes
                    const uint32_t fb = full0 + 8u * stage, dst = base + (uint32_t)stage * STAGE;
                    mbar_expect_tx(fb, HB + (with_src ? CB : 0u));
                    tma_load_3d(dst, &p.map_h, z0 - 4, m0 - 2 - p.oy, g.a0 - 2 + s - p.ox, fb);
                    if (with_src) tma_load_3d(dst + HB, &p.map_c, z0, m0, g.a0 + s - 4, fb);
                    if (++stage == ST) { stage = 0; phase ^= 1u; first_round = false; }
                }
            }
        }
    } else {
        // ---- consumers: warp w owns rows m0 + w RY .. + RY-1, lane l the float4 at z0 + 4 l ----
        // byte offsets inside a stage: row warp*RY of the halo tile is global row mrow-2
        const uint32_t h_off = (uint32_t)((warp * RY) * S3T_WP + 4 + 4 * lane) * 4u;
        const uint32_t c_off = HB + (uint32_t)((warp * RY) * S3T_TZ + 4 * lane) * 4u;
        const size_t PS = (size_t)p.n1 * p.n2;
        // the weights live in registers (packed operands cannot come from the constant bank)
        const float2 w16x = p.w16[0], w16y = p.w16[1], w16z = p.w16[2];
        const float2 nwx = p.nw[0], nwy = p.nw[1], nwz = p.nw[2], kc = p.kc;
        const float2 zero2 = make_float2(0.f, 0.f);
        while (s3t_next_segment(pos, end, p.n0, g)) {
            const int cb = g.tile % p.ncb, m0 = (g.tile / p.ncb) * TYB;
            const int c4 = cb * S3T_TX + lane;
            const int mrow = m0 + warp * RY;
            const bool first_col = c4 == 0, last_col = c4 == p.nc4 - 1;
            float* optr = p.out + ((size_t)g.a0 * p.n1 + mrow) * (size_t)p.n2 + (size_t)(4 * c4);   // output (a0, mrow, col)
            // per thread and row, fixed over the segment: may the row be stored at all (ragged tiles),
            // and (forward) do its two halves carry residual rows
            bool row_ok[RY], keep_lo[RY], keep_hi[RY];
#pragma unroll
            for (int j = 0; j < RY; ++j) {
                const bool row_in = mrow + j >= 2 && mrow + j <= p.n1 - 3 && c4 < p.nc4;
                row_ok[j] = c4 < p.nc4 && mrow + j < p.n1;
                keep_lo[j] = row_in && !first_col;
                keep_hi[j] = row_in && !last_col;
            }
            V4 R0[RY], R1[RY], R2[RY], R3[RY];
#pragma unroll
            for (int j = 0; j < RY; ++j) { R0[j] = v4zero(); R1[j] = v4zero(); R2[j] = v4zero(); R3[j] = v4zero(); }

            // One step: plane b arrives.  A0..A3 hold the partial outputs of planes b-2 .. b+1; the step
            // completes b-2 (stored when `emit`: the first four planes of a segment only fill the
            // partial sums), adds to b-1, b, b+1 and starts b+2 in the registers of A0.
            // plane_in (forward): the completed plane carries residual rows.
            auto step = [&](auto emit_tag, bool plane_in, V4 (&A0)[RY], V4 (&A1)[RY], V4 (&A2)[RY], V4 (&A3)[RY]) {
                constexpr bool EMIT = decltype(emit_tag)::value;
                const uint32_t bar = full0 + 8u * (uint32_t)stage;
                mbar_wait(bar, phase, gave_up, &g_star3d_tma_timeouts);
                const uint32_t sb = base + (uint32_t)stage * STAGE;
                const uint32_t hs = sb + h_off;
                V4 L[RY + 4];
#pragma unroll
                for (int i = 0; i < RY + 4; ++i) L[i] = ldsv4(hs + (uint32_t)(i * S3T_WP * 4));
                float2 zl[RY], zr[RY];
#pragma unroll
                for (int j = 0; j < RY; ++j) {
                    zl[j] = ldsv2(hs + (uint32_t)((j + 2) * S3T_WP * 4) - 8u);
                    zr[j] = ldsv2(hs + (uint32_t)((j + 2) * S3T_WP * 4) + 16u);
                }
                V4 src[RY];
                if (FWD && EMIT) {
#pragma unroll
                    for (int j = 0; j < RY; ++j) src[j] = ldsv4(sb + c_off + (uint32_t)(j * S3T_TZ * 4));
                }
#pragma unroll
                for (int j = 0; j < RY; ++j) {
                    V4 c = L[j + 2];
                    if (MODE == 1) {                            // band in z: columns 0,1 / n-2,n-1 read as zero
                        if (first_col) c.lo = zero2;
                        if (last_col) c.hi = zero2;
                    }
                    const V4 s1y = v4add(L[j + 1], L[j + 3]), s2y = v4add(L[j], L[j + 4]);
                    V4 s1z, s2z;
                    s1z.lo = make_float2(zl[j].y + c.lo.y, c.lo.x + c.hi.x);
                    s1z.hi = make_float2(c.lo.y + c.hi.y, c.hi.x + zr[j].x);
                    s2z.lo = add2(zl[j], c.hi);                          // (z-2, z-1) + (z+2, z+3): both register pairs
                    s2z.hi = add2(c.lo, zr[j]);
                    if (MODE == 1) {
                        // the y neighbours in the z band are zero too: their sum is formed apart and masked
                        V4 py = v4mul(s1y, w16y);
                        py = v4fma(s2y, nwy, py);
                        if (first_col) py.lo = zero2;
                        if (last_col) py.hi = zero2;
                        A2[j] = v4add(A2[j], py);
                    } else {
                        A2[j] = v4fma(s1y, w16y, A2[j]);
                        A2[j] = v4fma(s2y, nwy, A2[j]);
                    }
                    A2[j] = v4fma(c, kc, A2[j]);
                    A2[j] = v4fma(s1z, w16z, A2[j]);
                    A2[j] = v4fma(s2z, nwz, A2[j]);
                    const V4 t = v4mul(c, nwx);
                    V4 o = v4add(A0[j], t);                     // output of plane b-2 is complete
                    A1[j] = v4fma(c, w16x, A1[j]);
                    A3[j] = v4fma(c, w16x, A3[j]);
                    A0[j] = t;                                  // first term of plane b+2
                    if (EMIT) {
                        if (FWD) {
                            o = v4sub(o, src[j]);
                            // nodes of the two outer layers carry no row
                            if (!(plane_in && keep_lo[j])) o.lo = zero2;
                            if (!(plane_in && keep_hi[j])) o.hi = zero2;
                            acc = fma2(o.lo, o.lo, fma2(o.hi, o.hi, acc));      // (rows never stored are zero here)
                        }
                        if (row_ok[j]) stv4(optr + (size_t)j * p.n2, o.lo, o.hi);
                    }
                }
                if (EMIT) optr += PS;
                // every value of the stage has been consumed by the arithmetic above: hand it back
                __syncwarp();
                if (lane == 0) mbar_arrive(bar + 8u * ST);
                if (++stage == ST) { stage = 0; phase ^= 1u; }
            };
            using No = std::false_type;
            using Yes = std::true_type;
            // planes a0-2 .. a0+1 fill the partial sums
            step(No{}, false, R0, R1, R2, R3);
            step(No{}, false, R1, R2, R3, R0);
            step(No{}, false, R2, R3, R0, R1);
            step(No{}, false, R3, R0, R1, R2);
            // each further plane completes one: a = a0 .. a1-1
            const int hi_in = p.n0 - 3;
            int a = g.a0, group = 0;
            for (; a + 4 <= g.a1; a += 4) {
                if (a >= 2 && a + 3 <= hi_in) {                 // all four planes carry rows (the common case)
                    step(Yes{}, true, R0, R1, R2, R3);
                    step(Yes{}, true, R1, R2, R3, R0);
                    step(Yes{}, true, R2, R3, R0, R1);
                    step(Yes{}, true, R3, R0, R1, R2);
                } else {
                    step(Yes{}, a >= 2 && a <= hi_in, R0, R1, R2, R3);
                    step(Yes{}, a + 1 >= 2 && a + 1 <= hi_in, R1, R2, R3, R0);
                    step(Yes{}, a + 2 >= 2 && a + 2 <= hi_in, R2, R3, R0, R1);
                    step(Yes{}, a + 3 >= 2 && a + 3 <= hi_in, R3, R0, R1, R2);
                }
                // a CTA's share of a large grid is thousands of planes: keep the fp32 partial sums
                // short (16 planes of RY float4 each) so that their rounding stays below 1e-6
                if (FWD && (++group & 3) == 0) { acc_long += (double)(acc.x + acc.y); acc = zero2; }
            }
            if (a < g.a1) step(Yes{}, a >= 2 && a <= hi_in, R0, R1, R2, R3);
            if (a + 1 < g.a1) step(Yes{}, a + 1 >= 2 && a + 1 <= hi_in, R1, R2, R3, R0);
            if (a + 2 < g.a1) step(Yes{}, a + 2 >= 2 && a + 2 <= hi_in, R2, R3, R0, R1);
        }
    }
    if (FWD && p.partials != nullptr) {
        float s[1] = {(float)(acc_long + (double)(acc.x + acc.y))};
        block_reduce_store<1>(s, p.partials, gridDim.x, blockIdx.x);
    }
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
static int env_int(const char* name, int dflt) {
    const char* s = std::getenv(name);
    if (!s || !*s) return dflt;
    const int v = std::atoi(s);
    return v >= 0 ? v : dflt;
}

constexpr int S3T_MAX_CTAS = 2048;       // upper bound of the grid (= loss partial sums a launch may write)

struct S3tShape { int tyb, ry; };
constexpr int S3T_STAGES = 6;            // ring depth (4, 6 and 8 measured within a microsecond of one another)

// Launch shape: rows per block / per thread.
static S3tShape s3t_shape() {
    S3tShape g;
    g.tyb = env_int("FPDE_STAR3D_TMA_TYB", 8) >= 16 ? 16 : 8;
    g.ry = env_int("FPDE_STAR3D_TMA_RY", 2) >= 4 ? 4 : 2;
    return g;
}

// The engine takes grids whose tiles are mostly full (it always moves whole boxes): at least one
// full tile in z and y.  FPDE_STAR3D_TMA=0 selects the L1-staged engine everywhere.
bool star3d_tma_wanted(const int* n) {
    if (env_int("FPDE_STAR3D_TMA", 1) == 0 || tma_encode_fn() == nullptr) return false;
    return n[2] >= S3T_WP && n[1] >= 16 + 8 && n[0] >= 8;
}

int star3d_tma_items(const int*) { return S3T_MAX_CTAS; }

template <int MODE, int TYB, int RY, int ST, int MINB>
static cudaError_t s3t_launch(const Problem& q, Star3dTmaParams& p, int* items) {
    constexpr uint32_t HB = (uint32_t)((TYB + 4) * S3T_WP * 4);
    constexpr uint32_t CB = MODE == 0 ? (uint32_t)(TYB * S3T_TZ * 4) : 0u;
    constexpr size_t smem = (size_t)ST * (((HB + CB + 127u) / 128u) * 128u) + 128;
    constexpr int threads = S3T_TX * (TYB / RY) + 32;
    auto kern = star3d_tma_kernel<MODE, TYB, RY, ST, MINB>;
    // CTAs the device holds at once (per device: the attribute and the occupancy are looked up once)
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
        // three CTAs per SM measured best on 256^3 (more CTAs mean shorter runs of planes per CTA,
        // each of which re-reads four halo planes)
        const int cap = env_int("FPDE_STAR3D_TMA_CTAS_PER_SM", 3);
        if (cap > 0) per_sm = std::min(per_sm, cap);
        slots_of[dev] = sms * per_sm;
    }
    // one CTA per slot; fewer on grids with less than 16 tile-planes per slot
    const long long G = std::max(1ll, std::min<long long>(std::min(slots_of[dev], S3T_MAX_CTAS), p.work / 16));
    if (items) *items = (int)G;
    return launch_kernel_smem(kern, dim3((unsigned)G), dim3(threads, 1, 1), smem, q.stream, p);
}

template <int MODE>
static cudaError_t s3t_dispatch(const Problem& q, Star3dTmaParams& p, const S3tShape& g, int* items) {
    // CTAs per SM the register budget is set for: 3 with 8-row tiles, 2 with 16-row tiles
    if (g.tyb == 16 && g.ry == 4) return s3t_launch<MODE, 16, 4, S3T_STAGES, 2>(q, p, items);
    if (g.tyb == 16) return s3t_launch<MODE, 16, 2, S3T_STAGES, 2>(q, p, items);
    if (g.ry == 4) return s3t_launch<MODE, 8, 4, S3T_STAGES, 3>(q, p, items);
    return s3t_launch<MODE, 8, 2, S3T_STAGES, 3>(q, p, items);
}

// mode as in the kernel.  `launched` false (with cudaSuccess) = this grid runs on the other engine.
// The adjoint runs here by default (measured on 256^3: 24.8 us against 29.5 us for the L1-staged
// engine); the forward pass, which streams a second input array and whose L1-staged kernel is
// already within a tenth of its DRAM time, only with FPDE_STAR3D_TMA_FWD=1 (36 us against 34 us).
cudaError_t launch_star3d_tma(const Problem& q, int mode, int* items, bool& launched) {
    launched = false;
    if (!star3d_tma_wanted(q.n)) return cudaSuccess;
    if (mode == 0 && env_int("FPDE_STAR3D_TMA_FWD", 0) == 0) return cudaSuccess;
    const bool fwd = mode == 0;
    const S3tShape g = s3t_shape();
    Star3dTmaParams p{};
    p.n0 = q.n[0]; p.n1 = q.n[1]; p.n2 = q.n[2]; p.nc4 = q.n[2] / 4;
    p.ncb = (p.n2 + S3T_TZ - 1) / S3T_TZ;
    p.ntiles = p.ncb * ((p.n1 + g.tyb - 1) / g.tyb);
    p.work = (long long)p.ntiles * p.n0;
    const float* hin = fwd ? q.in[0] : q.aux[0];
    const long long n1 = p.n1, n2 = p.n2, n0 = p.n0;
    bool ok;
    if (mode == 1) {
        // the sub-array of rows in x and y: everything outside it reads as zero
        p.ox = 2; p.oy = 2;
        ok = tma_encode_3d(&p.map_h, hin + (2 * n1 + 2) * n2, n2, n1 - 4, n0 - 4, n2, n1 * n2, S3T_WP, g.tyb + 4);
    } else {
        p.ox = 0; p.oy = 0;
        ok = tma_encode_3d(&p.map_h, hin, n2, n1, n0, n2, n1 * n2, S3T_WP, g.tyb + 4);
    }
    if (ok && fwd) ok = tma_encode_3d(&p.map_c, q.aux[0], n2, n1, n0, n2, n1 * n2, S3T_TZ, g.tyb);
    if (!ok) return cudaSuccess;                      // not encodable: the other engine takes it
    const double scale = fwd ? 1.0 : q.gscale[0];     // the operator is linear: the scale goes into the weights
    double wsum = 0.0;
    for (int a = 0; a < 3; ++a) {
        const double w = 1.0 / (12.0 * q.h[a] * q.h[a]);
        p.w16[a] = make_float2((float)(16.0 * w * scale), (float)(16.0 * w * scale));
        p.nw[a] = make_float2((float)(-w * scale), (float)(-w * scale));
        wsum += w;
    }
    const double kc = (q.coef[0] * q.coef[0] - 30.0 * wsum) * scale;
    p.kc = make_float2((float)kc, (float)kc);
    p.out = q.out[0];
    p.partials = fwd ? q.partials : nullptr;
    launched = true;
    if (mode == 0) return s3t_dispatch<0>(q, p, g, items);
    if (mode == 1) return s3t_dispatch<1>(q, p, g, items);
    return s3t_dispatch<2>(q, p, g, items);
}

unsigned int star3d_tma_timeouts() {
    unsigned int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_star3d_tma_timeouts, sizeof(v)) != cudaSuccess) { (void)cudaGetLastError(); return ~0u; }
    return v;
}

}  // namespace fpde
