// Device-side helpers shared by the operator kernels: 128-bit loads/stores, lane-neighbour
// exchange along the contiguous axis, and the deterministic loss reduction
// (per-thread fp32 -> warp shuffle tree -> shared-memory block tree -> one partial per CTA).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace fpde {

constexpr unsigned FULL_MASK = 0xffffffffu;

// Programmatic dependent launch: every kernel first waits until the kernel before it in the
// stream has completed and its writes are visible (a no-op when launched without the
// attribute), then lets the kernel after it start launching, so that launch latency and the
// tail of one kernel overlap with the head of the next.
__device__ __forceinline__ void pdl_wait_then_trigger() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
constexpr int MAX_RES = 4;        // most residual fields of any operator

__device__ __forceinline__ float4 ld4(const float* p) {
    return __ldg(reinterpret_cast<const float4*>(p));
}
__device__ __forceinline__ void st4(float* p, float4 v) {
    *reinterpret_cast<float4*>(p) = v;
}
__device__ __forceinline__ float4 f4zero() { return make_float4(0.f, 0.f, 0.f, 0.f); }
__device__ __forceinline__ float4 f4scale(float4 a, float s) {
    return make_float4(a.x * s, a.y * s, a.z * s, a.w * s);
}
__device__ __forceinline__ float f4get(const float4& a, int k) {
    return k == 0 ? a.x : k == 1 ? a.y : k == 2 ? a.z : a.w;
}
__device__ __forceinline__ float sq4(float4 a) {
    return a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
}


// ------------------------------------------------------------------------------------------
// Packed fp32x2 arithmetic (sm_100 FFMA2 / FADD2 / FMUL2): one instruction per two lanes of a
// thread's float4, which halves the issue slots the stencil arithmetic takes.  Per component
// the results are those of fmaf / add / mul in round-to-nearest.
// ------------------------------------------------------------------------------------------
struct V4 { float2 lo, hi; };           // a float4 as two register-aligned pairs

__device__ __forceinline__ float2 splat2(float a) { return make_float2(a, a); }
__device__ __forceinline__ float2 add2(float2 a, float2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ float2 mul2(float2 a, float2 b) { return __fmul2_rn(a, b); }
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ float2 sub2(float2 a, float2 b) {            // a - b, exactly rounded once
    return __ffma2_rn(b, make_float2(-1.f, -1.f), a);
}
__device__ __forceinline__ V4 ldv4(const float* p) {
    const float4 t = __ldg(reinterpret_cast<const float4*>(p));
    V4 v; v.lo = make_float2(t.x, t.y); v.hi = make_float2(t.z, t.w);
    return v;
}
__device__ __forceinline__ void stv4(float* p, float2 lo, float2 hi) {
    *reinterpret_cast<float4*>(p) = make_float4(lo.x, lo.y, hi.x, hi.y);
}
// The same accesses at an element offset from an array base.  OFF32: the byte offset is formed
// as an unsigned 32-bit number (arrays of at most 2^30 floats), which lets the address be a
// 64-bit base plus a 32-bit register instead of a 64-bit add per access; the kernels spend a
// sixth of their issue slots on addresses otherwise.
template <bool OFF32>
__device__ __forceinline__ const float* at_off(const float* base, int eoff) {
    if (OFF32) return reinterpret_cast<const float*>(reinterpret_cast<const char*>(base) + 4u * (unsigned)eoff);
    return base + eoff;
}
template <bool OFF32>
__device__ __forceinline__ float* at_off(float* base, int eoff) {
    if (OFF32) return reinterpret_cast<float*>(reinterpret_cast<char*>(base) + 4u * (unsigned)eoff);
    return base + eoff;
}

__device__ __forceinline__ V4 v4zero() { V4 v; v.lo = make_float2(0.f, 0.f); v.hi = v.lo; return v; }
__device__ __forceinline__ V4 v4add(V4 a, V4 b) { V4 r; r.lo = add2(a.lo, b.lo); r.hi = add2(a.hi, b.hi); return r; }
__device__ __forceinline__ V4 v4sub(V4 a, V4 b) { V4 r; r.lo = sub2(a.lo, b.lo); r.hi = sub2(a.hi, b.hi); return r; }
__device__ __forceinline__ V4 v4mul(V4 a, float2 s) { V4 r; r.lo = mul2(a.lo, s); r.hi = mul2(a.hi, s); return r; }
__device__ __forceinline__ V4 v4mulv(V4 a, V4 b) { V4 r; r.lo = mul2(a.lo, b.lo); r.hi = mul2(a.hi, b.hi); return r; }
// a * s + c
__device__ __forceinline__ V4 v4fma(V4 a, float2 s, V4 c) { V4 r; r.lo = fma2(a.lo, s, c.lo); r.hi = fma2(a.hi, s, c.hi); return r; }
// a * b + c
__device__ __forceinline__ V4 v4fmav(V4 a, V4 b, V4 c) { V4 r; r.lo = fma2(a.lo, b.lo, c.lo); r.hi = fma2(a.hi, b.hi, c.hi); return r; }

// half h (0: lo, 1: hi) of each float4 of an array
template <int NA>
__device__ __forceinline__ void v4_half(const V4 (&A)[NA], int h, float2 (&out)[NA]) {
#pragma unroll
    for (int i = 0; i < NA; ++i) out[i] = h == 0 ? A[i].lo : A[i].hi;
}

// a float4 shifted by one element to the left / right along the row
__device__ __forceinline__ V4 shift_left(const V4& c, float l1) {    // value at column j-1
    V4 r; r.lo = make_float2(l1, c.lo.x); r.hi = make_float2(c.lo.y, c.hi.x); return r;
}
__device__ __forceinline__ V4 shift_right(const V4& c, float r1) {   // value at column j+1
    V4 r; r.lo = make_float2(c.lo.y, c.hi.x); r.hi = make_float2(c.hi.y, r1); return r;
}

// Values one and two elements to the left / right of a thread's float4 along the contiguous
// axis.  Inside a warp they come from the neighbouring lane's registers; the first and last
// lane (and the first / last float4 of a row) fetch them from global memory, wrapped around
// the row when `periodic`, else 0 outside the row.  `row` points at element 0 of the row,
// `c4` is this thread's float4 index, `nc4` the row length in float4.  All 32 lanes must call
// this (lanes with c4 >= nc4 pass cur = 0 and get unspecified values).  `cur` is the value
// the thread holds in registers (already scaled / masked by the caller); values fetched from
// global memory are multiplied by `scale` to match.
struct LR2 { float l1, l2, r1, r2; };

template <int R>
__device__ __forceinline__ LR2 lane_neighbours(const float* __restrict__ row, int c4, int nc4,
                                               float4 cur, bool periodic, float scale) {
    LR2 o;
    const int lane = threadIdx.x & 31;
    o.l1 = __shfl_up_sync(FULL_MASK, cur.w, 1);
    o.r1 = __shfl_down_sync(FULL_MASK, cur.x, 1);
    if (R >= 2) {
        o.l2 = __shfl_up_sync(FULL_MASK, cur.z, 1);
        o.r2 = __shfl_down_sync(FULL_MASK, cur.y, 1);
    } else {
        o.l2 = 0.f; o.r2 = 0.f;
    }
    if (c4 < nc4) {
        const int n = nc4 * 4;
        if (lane == 0 || c4 == 0) {
            int j1 = 4 * c4 - 1, j2 = 4 * c4 - 2;
            if (periodic) { if (j1 < 0) j1 += n; if (j2 < 0) j2 += n; }
            o.l1 = j1 >= 0 ? scale * __ldg(row + j1) : 0.f;
            if (R >= 2) o.l2 = j2 >= 0 ? scale * __ldg(row + j2) : 0.f;
        }
        if (lane == 31 || c4 == nc4 - 1) {
            int j1 = 4 * c4 + 4, j2 = 4 * c4 + 5;
            if (periodic) { if (j1 >= n) j1 -= n; if (j2 >= n) j2 -= n; }
            o.r1 = j1 < n ? scale * __ldg(row + j1) : 0.f;
            if (R >= 2) o.r2 = j2 < n ? scale * __ldg(row + j2) : 0.f;
        }
    }
    return o;
}

// Deterministic block reduction of NE per-thread partial sums; thread 0 writes
// partials[e * stride + slot].  The shuffle tree and the shared-memory tree have a fixed shape,
// so the result depends only on the data, never on scheduling.
template <int NE>
__device__ __forceinline__ void block_reduce_store(const float (&acc)[NE], float* __restrict__ partials,
                                                   int stride, int slot) {
    __shared__ float red[NE][32];
    const int tid = threadIdx.x + blockDim.x * (threadIdx.y + blockDim.y * threadIdx.z);
    const int nthreads = blockDim.x * blockDim.y * blockDim.z;
    const int lane = tid & 31, warp = tid >> 5, nwarps = (nthreads + 31) >> 5;
#pragma unroll
    for (int e = 0; e < NE; ++e) {
        float v = acc[e];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(FULL_MASK, v, o);
        if (lane == 0) red[e][warp] = v;
    }
    __syncthreads();
    if (warp == 0) {
#pragma unroll
        for (int e = 0; e < NE; ++e) {
            float v = lane < nwarps ? red[e][lane] : 0.f;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(FULL_MASK, v, o);
            if (lane == 0) partials[(size_t)e * stride + slot] = v;
        }
    }
}

}  // namespace fpde
