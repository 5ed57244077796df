// Navier-Stokes forward / adjoint kernels whose plane tiles are staged through shared memory by
// TMA (cp.async.bulk.tensor, each copy to the issuing CTA only) in a four-stage ring, instead of through L1.
//
// Why: the L1 variants keep every load of a step in registers while it is in flight, and at
// 160-240 registers per thread only 2-3 small blocks fit on an SM, so DRAM / L2 latency is
// exposed (long-scoreboard stalls dominate).  Here the data in flight lives in shared memory:
// while the block computes plane a from stages (a, a+1), the copy engine fills the other two
// stages with planes a+2 and a+3, steps (microseconds) ahead of their use, and every load the
// threads issue is a shared-memory load of fixed, short latency.  There is no block-wide barrier
// in the loop: a stage is handed back to the copy engine through an "empty" mbarrier on which
// each warp arrives when it has consumed the stage, so warps drift freely within the ring.
//
// Tile: TY rows x TXF = 4*TX floats of the contiguous (z,t) row, plus its halo: the row above,
// the row below, and n_t floats left and right (z-1, z+1).  A tile that does not touch the
// periodic wrap (most of them) is ONE box per array and plane, (TXF + 2 n_t) x (TY + 2); a tile
// on the first / last rows or columns takes five boxes (centre, row above, row below, left,
// right) whose coordinates are wrapped.  The two layouts differ only in per-thread shared-memory
// offsets that are fixed before the loop.  Box shapes need one tensor map each.
// The x-neighbours stay in a three-plane register window as in the L1 variant; the arithmetic is
// shared (ns_math.cuh).
//
// Status: opt-in (FPDE_NS_TMA=1).  On the 128^3 x 16 grid it reaches 4.2 / 4.8 TB/s (adjoint /
// forward) against 4.6 / 4.9 TB/s for the L1-staged kernels: with loads at shared-memory latency
// both variants end up limited by the same thing, the LSU data pipe (five 128-bit loads per output
// float4 and array), so the simpler kernels stay the default.  What made the difference here was
// the number of boxes: five small boxes per array and plane ran at 3.3 TB/s, one box at 4.2.
//
// Every wait on an mbarrier is bounded: after the limit the kernel counts a timeout in a global
// word and carries on with whatever is in shared memory, so it always terminates.
#include "fpde_common.cuh"
#include "fpde_internal.h"
#include "ns_math.cuh"
#include "tma_common.cuh"

#include <algorithm>
#include <cstdlib>
#include <mutex>

namespace fpde {

constexpr int NS_TMA_STAGES = 4;      // power of two: stage index = sequence number & 3
constexpr int NS_TMA_TX = 32;       // lanes along the row: TXF = 128 floats

template <int NA>
struct NsTmaParams {
    CUtensorMap map_c[NA];   // centre box   TXF x TY x 1
    CUtensorMap map_r[NA];   // one-row box  TXF x 1  x 1
    CUtensorMap map_z[NA];   // z-halo box   n_t x TY x 1
    CUtensorMap map_w[NA];   // whole tile with halo, (TXF + 2 n_t) x (TY + 2) x 1 (tiles away from the wrap)
    const float* arr[NA];    // the same arrays as plain pointers (plane a0-1 of the window)
    float* out[4];
    NsConsts k;
    int n0, n1, n3, C;
    int planes_per_item, ncb, nmb, nitems;
    float* partials;
};

__device__ unsigned int g_ns_tma_timeouts = 0;   // number of bounded waits that gave up (0 in a healthy run)

__device__ __forceinline__ int wrapn(int i, int n) { return i < 0 ? i + n : (i >= n ? i - n : i); }

template <int NA, bool FWD, int TY, int MINB>
__global__ void __launch_bounds__(NS_TMA_TX * TY, MINB)
ns_tma_kernel(const __grid_constant__ NsTmaParams<NA> p) {
    constexpr int TX = NS_TMA_TX, TXF = 4 * TX, ST = NS_TMA_STAGES;
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long full_bar[ST];
    __shared__ __align__(8) unsigned long long empty_bar[ST];

    const int tx = threadIdx.x, ty = threadIdx.y;
    const int tid = ty * TX + tx;
    const int n0 = p.n0, n1 = p.n1, n3 = p.n3, C = p.C;
    int item = blockIdx.x;
    const int cb = item % p.ncb; item /= p.ncb;
    const int mb = item % p.nmb;
    const int ab = item / p.nmb;
    const int x0f = cb * TXF, y0 = mb * TY;
    const int a0 = ab * p.planes_per_item;
    const int a1 = min(a0 + p.planes_per_item, n0);
    const int nsteps = a1 - a0;

    // shared-memory layout (floats) of one array's slot inside a stage
    const int OFF_U = TY * TXF, OFF_D = OFF_U + TXF, OFF_L = OFF_D + TXF, OFF_R = OFF_L + TY * n3;
    const int SLOT5 = OFF_R + TY * n3;               // five-box layout
    const int WP = TXF + 2 * n3;                     // row pitch of the one-box layout
    const int SLOT1 = WP * (TY + 2);
    const bool one_box = cb > 0 && cb < p.ncb - 1 && mb > 0 && mb < p.nmb - 1;
    const int SLOT = SLOT1;                          // slot pitch (SLOT1 >= SLOT5)
    const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
    const uint32_t stage_bytes = (uint32_t)(NA * SLOT) * 4u;
    const uint32_t fill_bytes = (uint32_t)(NA * (one_box ? SLOT1 : SLOT5)) * 4u;
    const uint32_t full0 = smem_u32(&full_bar[0]), empty0 = smem_u32(&empty_bar[0]);

    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < ST; ++s) { mbar_init(full0 + 8u * s, 1); mbar_init(empty0 + 8u * s, TY); }
        mbar_fence_init();
    }
    __syncthreads();
    pdl_wait_then_trigger();          // nothing of the previous kernel's output is read before this

    // queue the five boxes of every array for plane index `seq` (a0 + seq, wrapped) into `stage`
    bool gave_up = false;
    // (first warp only) queue the five boxes of every array for plane a0 + seq (wrapped) into
    // stage seq & 3, once every warp has handed that stage back
    auto issue = [&](int seq) {
        const int stage = seq & (ST - 1);
        const uint32_t fb = full0 + 8u * stage;
        if (seq >= ST) mbar_wait(empty0 + 8u * stage, (uint32_t)(((seq / ST) - 1) & 1), gave_up, &g_ns_tma_timeouts);
        const int pl = wrapn(a0 + seq, n0);
        const uint32_t sb = base + (uint32_t)stage * stage_bytes;
        if (tx == 0) mbar_expect_tx(fb, fill_bytes);
        __syncwarp();
        if (tx < NA && one_box) {
            tma_load_3d(sb + (uint32_t)(tx * SLOT) * 4u, &p.map_w[tx], x0f - n3, y0 - 1, pl, fb);
        } else if (tx < NA) {
            const uint32_t d = sb + (uint32_t)(tx * SLOT) * 4u;
            tma_load_3d(d, &p.map_c[tx], x0f, y0, pl, fb);
            tma_load_3d(d + OFF_U * 4u, &p.map_r[tx], x0f, wrapn(y0 - 1, n1), pl, fb);
            tma_load_3d(d + OFF_D * 4u, &p.map_r[tx], x0f, wrapn(y0 + TY, n1), pl, fb);
            tma_load_3d(d + OFF_L * 4u, &p.map_z[tx], wrapn(x0f - n3, C), y0, pl, fb);
            tma_load_3d(d + OFF_R * 4u, &p.map_z[tx], wrapn(x0f + TXF, C), y0, pl, fb);
        }
    };
    if (ty == 0) {
#pragma unroll
        for (int s = 0; s < ST; ++s)
            if (s <= nsteps) issue(s);
    }

    // per-thread byte offsets inside an array's slot
    const int own = one_box ? (ty + 1) * WP + n3 + 4 * tx : ty * TXF + 4 * tx;
    const uint32_t o_own = own * 4u;
    uint32_t o_ym, o_yp, o_zm, o_zp;
    if (one_box) {
        o_ym = (own - WP) * 4u; o_yp = (own + WP) * 4u; o_zm = (own - n3) * 4u; o_zp = (own + n3) * 4u;
    } else {
        o_ym = (ty > 0 ? own - TXF : OFF_U + 4 * tx) * 4u;
        o_yp = (ty < TY - 1 ? own + TXF : OFF_D + 4 * tx) * 4u;
        o_zm = (4 * tx >= n3 ? own - n3 : OFF_L + ty * n3 + 4 * tx) * 4u;
        o_zp = (4 * tx + n3 < TXF ? own + n3 : OFF_R + ty * n3 + (4 * tx + n3 - TXF)) * 4u;
    }
    const int nt4 = n3 / 4;
    const int tq = tx % nt4;                         // TXF is a multiple of n3: groups start at lane multiples of nt4
    const bool t_first = tq == 0, t_last = tq == nt4 - 1;
    const int gcol = x0f + 4 * tx, grow = y0 + ty;
    const int PS = n1 * C;

    V4 A[NA], B[NA], Cc[NA];
    {
        const int om = wrapn(a0 - 1, n0) * PS + grow * C + gcol;
#pragma unroll
        for (int k = 0; k < NA; ++k) A[k] = ldv4(p.arr[k] + om);
    }
    mbar_wait(full0, 0, gave_up, &g_ns_tma_timeouts);
#pragma unroll
    for (int k = 0; k < NA; ++k) B[k] = ldsv4(base + (uint32_t)(k * SLOT) * 4u + o_own);

    float2 acc[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[e] = make_float2(0.f, 0.f);

    // step s: plane a0+s from stage S0 (neighbours), plane a0+s+1 from stage S1 (own column -> W2)
    auto step = [&](int s, const V4 (&W0)[NA], const V4 (&W1)[NA], V4 (&W2)[NA]) {
        const int S0 = s & (ST - 1), S1 = (s + 1) & (ST - 1);
        mbar_wait(full0 + 8u * S1, (uint32_t)(((s + 1) / ST) & 1), gave_up, &g_ns_tma_timeouts);
        const uint32_t b0 = base + (uint32_t)S0 * stage_bytes, b1 = base + (uint32_t)S1 * stage_bytes;
        V4 Ym[NA], Yp[NA], Zm[NA], Zp[NA];
#pragma unroll
        for (int k = 0; k < NA; ++k) {
            const uint32_t sk = (uint32_t)(k * SLOT) * 4u;
            W2[k] = ldsv4(b1 + sk + o_own);
            Ym[k] = ldsv4(b0 + sk + o_ym);
            Yp[k] = ldsv4(b0 + sk + o_yp);
            Zm[k] = ldsv4(b0 + sk + o_zm);
            Zp[k] = ldsv4(b0 + sk + o_zp);
        }
        float l1[3], r1[3];
#pragma unroll
        for (int q = 0; q < 3; ++q) {               // t neighbours of the outer lanes: adjacent lanes' registers
            const V4& c = W1[FWD ? q : 3 + q];
            l1[q] = __shfl_up_sync(FULL_MASK, c.hi.y, 1);
            r1[q] = __shfl_down_sync(FULL_MASK, c.lo.x, 1);
        }
        float2 o[4][2];
        if constexpr (FWD) ns_fwd_math(p.k, W0, W1, W2, Ym, Yp, Zm, Zp, l1, r1, t_first, t_last, o);
        else ns_bwd_math(p.k, W0, W1, W2, Ym, Yp, Zm, Zp, l1, r1, t_first, t_last, o);
        const int off = (a0 + s) * PS + grow * C + gcol;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            stv4(p.out[e] + off, o[e][0], o[e][1]);
            if (FWD) acc[e] = fma2(o[e][0], o[e][0], fma2(o[e][1], o[e][1], acc[e]));
        }
        // this warp is done with stage S0 (its values have been consumed by the arithmetic above)
        __syncwarp();
        if (tx == 0) mbar_arrive(empty0 + 8u * S0);
        if (ty == 0 && s + ST <= nsteps) issue(s + ST);
    };

    for (int s = 0; s < nsteps; s += 3) {
        step(s, A, B, Cc);
        if (s + 1 < nsteps) step(s + 1, B, Cc, A);
        if (s + 2 < nsteps) step(s + 2, Cc, A, B);
    }
    if (FWD && p.partials != nullptr) {
        float sres[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) sres[e] = acc[e].x + acc[e].y;
        block_reduce_store<4>(sres, p.partials, p.nitems, blockIdx.x);
    }
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
static bool encode_box(CUtensorMap* m, const float* ptr, int C, int n1, int n0, int bx, int by) {
    return tma_encode_3d(m, ptr, C, n1, n0, C, (long long)C * n1, bx, by);
}

static int env_int(const char* name, int dflt) {
    const char* s = std::getenv(name);
    if (!s || !*s) return dflt;
    const int v = std::atoi(s);
    return v >= 0 ? v : dflt;
}

// rows per tile: 8 when the grid allows it (fewer, larger boxes and less halo per byte), else 4
static int ns_tma_ty(const int* n) {
    const int want = env_int("FPDE_NS_TMA_TY", 4);
    return (want >= 8 && n[1] % 8 == 0) ? 8 : 4;
}

// Dynamic shared memory of a launch with `na` arrays per stage.
static size_t ns_tma_smem_bytes(const int* n, int ty, int na) {
    const size_t slot = (size_t)(4 * NS_TMA_TX + 2 * n[3]) * (ty + 2);
    return (size_t)NS_TMA_STAGES * na * slot * 4 + 128;
}

// Pure geometry: can a kernel with tiles of `ty` rows and `na` arrays per stage take this grid
// within `smem_limit` bytes of dynamic shared memory?  Exact tiling; t groups aligned to lanes;
// every bulk-copy destination (array slot, stage) on a 128-byte boundary, which the copy engine
// requires -- the slot is (128 + 2 n_t)(ty + 2) floats, a multiple of 32 floats only when n_t is
// a multiple of 8 for the even tile heights used here; the stage ring within the limit.
bool ns_tma_geometry_ok(const int* n, int ty, int na, size_t smem_limit) {
    const int n3 = n[3], C = n[2] * n[3], nt4 = n3 / 4;
    if (n3 % 4 != 0 || nt4 < 1 || 32 % nt4 != 0) return false;
    if (ty < 1 || n[1] % ty != 0 || C % (4 * NS_TMA_TX) != 0) return false;
    if ((ty * n3) % 32 != 0 || n3 > 64) return false;      // n3 <= 64: the one-box tile fits 256 elements
    const size_t slot_bytes = (size_t)(4 * NS_TMA_TX + 2 * n3) * (ty + 2) * 4;
    if (slot_bytes % 128 != 0 || (na * slot_bytes) % 128 != 0) return false;
    return ns_tma_smem_bytes(n, ty, na) <= smem_limit;
}

static size_t smem_optin_limit() {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    return (size_t)v;
}

// Can the TMA-staged kernels take this grid?  Both directions must fit (forward: 4 arrays per
// stage, adjoint: 7), because the loss workspace is sized for one launch shape per grid; anything
// else runs on the L1-staged kernels.
static bool ns_tma_applicable(const int* n) {
    if (env_int("FPDE_NS_TMA", 0) == 0 || tma_encode_fn() == nullptr) return false;
    const int ty = ns_tma_ty(n);
    const size_t limit = smem_optin_limit();
    return ns_tma_geometry_ok(n, ty, 4, limit) && ns_tma_geometry_ok(n, ty, 7, limit);
}

template <int NA, bool FWD, int TY, int MINB>
static cudaError_t launch_tma(const Problem& q, const float* const* arrays, const double* gscale, bool& launched) {
    launched = false;
    static NsTmaParams<NA> p;                      // large (tensor maps): keep it off the stack
    static std::mutex mtx;
    std::lock_guard<std::mutex> lock(mtx);
    p.n0 = q.n[0]; p.n1 = q.n[1]; p.n3 = q.n[3]; p.C = q.n[2] * q.n[3];
    const int TXF = 4 * NS_TMA_TX;
    for (int k = 0; k < NA; ++k) {
        p.arr[k] = arrays[k];
        if (!encode_box(&p.map_c[k], arrays[k], p.C, p.n1, p.n0, TXF, TY)) return cudaErrorInvalidValue;
        if (!encode_box(&p.map_r[k], arrays[k], p.C, p.n1, p.n0, TXF, 1)) return cudaErrorInvalidValue;
        if (!encode_box(&p.map_z[k], arrays[k], p.C, p.n1, p.n0, p.n3, TY)) return cudaErrorInvalidValue;
        // the wide box must fit the 256-element box limit and the row; grids too narrow for it have no
        // tile away from the wrap, so the map is never used there (encode a valid placeholder)
        const int wide = TXF + 2 * p.n3 <= 256 && TXF + 2 * p.n3 <= p.C ? TXF + 2 * p.n3 : TXF;
        if (!encode_box(&p.map_w[k], arrays[k], p.C, p.n1, p.n0, wide, std::min(TY + 2, p.n1))) return cudaErrorInvalidValue;
    }
    for (int e = 0; e < 4; ++e) p.out[e] = q.out[e];
    ns_fill_consts(p.k, q.h, q.coef[0], gscale);
    p.planes_per_item = std::max(1, env_int("FPDE_NS_PLANES", 16));
    p.ncb = p.C / TXF;
    p.nmb = p.n1 / TY;
    p.nitems = p.ncb * p.nmb * ((p.n0 + p.planes_per_item - 1) / p.planes_per_item);
    p.partials = FWD ? q.partials : nullptr;
    const size_t smem = ns_tma_smem_bytes(q.n, TY, NA);
    auto kern = ns_tma_kernel<NA, FWD, TY, MINB>;
    cudaError_t ce = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (ce != cudaSuccess) return ce;
    launched = true;
    return launch_kernel_smem(kern, dim3(p.nitems), dim3(NS_TMA_TX, TY, 1), smem, q.stream, p);
}

int ns_tma_items(const int* n) {
    const int C = n[2] * n[3];
    const int planes = std::max(1, env_int("FPDE_NS_PLANES", 16));
    return (C / (4 * NS_TMA_TX)) * (n[1] / ns_tma_ty(n)) * ((n[0] + planes - 1) / planes);
}

bool ns_tma_wanted(const int* n) { return ns_tma_applicable(n); }

cudaError_t launch_ns_fwd_tma(const Problem& q, bool& launched) {
    const float* arrays[4] = {q.in[0], q.in[1], q.in[2], q.in[3]};
    const double ones[4] = {1.0, 1.0, 1.0, 1.0};
    launched = false;
    if (!ns_tma_applicable(q.n)) return cudaSuccess;
    if (ns_tma_ty(q.n) == 8) {
        if (env_int("FPDE_NS_TMA_MINB_F", 2) >= 2) return launch_tma<4, true, 8, 2>(q, arrays, ones, launched);
        return launch_tma<4, true, 8, 1>(q, arrays, ones, launched);
    }
    return launch_tma<4, true, 4, 3>(q, arrays, ones, launched);
}

cudaError_t launch_ns_bwd_tma(const Problem& q, bool& launched) {
    const float* arrays[7] = {q.in[0], q.in[1], q.in[2], q.aux[0], q.aux[1], q.aux[2], q.aux[3]};
    launched = false;
    if (!ns_tma_applicable(q.n)) return cudaSuccess;
    if (ns_tma_ty(q.n) == 8) return launch_tma<7, false, 8, 1>(q, arrays, q.gscale, launched);
    return launch_tma<7, false, 4, 2>(q, arrays, q.gscale, launched);
}

unsigned int ns_tma_timeouts() {
    unsigned int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_ns_tma_timeouts, sizeof(v)) != cudaSuccess) { (void)cudaGetLastError(); return ~0u; }
    return v;
}

}  // namespace fpde
