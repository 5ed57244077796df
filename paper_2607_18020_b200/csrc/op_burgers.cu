// Viscous Burgers on an (x,t) array: r = D_t u + u D_x u - nu D_xx u at every node, with
// centred second-order differences inside and second-order one-sided differences on the first
// and last node of each axis (per axis).  Forward (Section 2.1) and gather-form adjoint with
// its boundary-gradient correction (Sections 2.2, 2.3): this is the operator whose correction
// terms come from one-sided formulas (Appendix A.5), not merely from omitted neighbours.
//
// Adjoint:  g = D_t^T G + (D_x u) . G + D_x^T (u . G) - nu D_xx^T G.
// A transposed difference matrix acts on w as
//     regular part    : the centred transpose, with w restricted to the centred rows 1..n-2;
//     edge correction : the columns of the two one-sided rows 0 and n-1, which reach nodes
//                       0..2 / n-3..n-1 (first derivative) and 0..3 / n-4..n-1 (second).
// The grid of this operator is small (latency-bound), so one thread handles one node.
#include "fpde_common.cuh"
#include "fpde_internal.h"

namespace fpde {

struct BurgersParams {
    const float* u;
    const float* g;      // adjoint: upstream G
    float* out;
    float gs;
    int nx, nt;
    float ihx, iht;      // 1/(2h)
    float ihxx;          // 1/hx^2
    float nu;
    float* partials;
    int nitems;
};

// First derivative at node i of a line q[i*stride], i in [0,n).
__device__ __forceinline__ float d1_at(const float* __restrict__ q, int i, int n, int stride, float ih2) {
    if (i == 0) return (-3.f * q[0] + 4.f * q[stride] - q[2 * stride]) * ih2;
    if (i == n - 1)
        return (3.f * q[(n - 1) * stride] - 4.f * q[(n - 2) * stride] + q[(n - 3) * stride]) * ih2;
    return (q[(i + 1) * stride] - q[(i - 1) * stride]) * ih2;
}
__device__ __forceinline__ float d2_at(const float* __restrict__ q, int i, int n, int stride, float ihh) {
    if (i == 0) return (2.f * q[0] - 5.f * q[stride] + 4.f * q[2 * stride] - q[3 * stride]) * ihh;
    if (i == n - 1)
        return (2.f * q[(n - 1) * stride] - 5.f * q[(n - 2) * stride] + 4.f * q[(n - 3) * stride]
                - q[(n - 4) * stride]) * ihh;
    const float c = q[i * stride];
    return ((q[(i + 1) * stride] - c) + (q[(i - 1) * stride] - c)) * ihh;
}

// (D^T w)_j for the first-derivative matrix; W(i) returns w at node i of the line.
template <class WF>
__device__ __forceinline__ float d1T_at(WF W, int j, int n, float ih2) {
    float s = 0.f;
    // regular part: centred rows i = j-1 (weight +1 at column j) and i = j+1 (weight -1)
    if (j - 1 >= 1 && j - 1 <= n - 2) s += W(j - 1);
    if (j + 1 >= 1 && j + 1 <= n - 2) s -= W(j + 1);
    // boundary correction: columns of the one-sided rows 0 and n-1
    if (j <= 2) s += W(0) * (j == 0 ? -3.f : (j == 1 ? 4.f : -1.f));
    if (j >= n - 3) s += W(n - 1) * (j == n - 1 ? 3.f : (j == n - 2 ? -4.f : 1.f));
    return s * ih2;
}
// (D2^T w)_j for the second-derivative matrix.
template <class WF>
__device__ __forceinline__ float d2T_at(WF W, int j, int n, float ihh) {
    float s = 0.f;
    if (j - 1 >= 1 && j - 1 <= n - 2) s += W(j - 1);
    if (j >= 1 && j <= n - 2) s -= 2.f * W(j);
    if (j + 1 >= 1 && j + 1 <= n - 2) s += W(j + 1);
    if (j <= 3) s += W(0) * (j == 0 ? 2.f : (j == 1 ? -5.f : (j == 2 ? 4.f : -1.f)));
    if (j >= n - 4) s += W(n - 1) * (j == n - 1 ? 2.f : (j == n - 2 ? -5.f : (j == n - 3 ? 4.f : -1.f)));
    return s * ihh;
}

__global__ void __launch_bounds__(256) burgers_fwd_kernel(const BurgersParams p) {
    pdl_wait_then_trigger();
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    const int N = p.nx * p.nt;
    float acc[1] = {0.f};
    if (idx < N) {
        const int i = idx / p.nt, j = idx - i * p.nt;
        const float ut = d1_at(p.u + (size_t)i * p.nt, j, p.nt, 1, p.iht);
        const float ux = d1_at(p.u + j, i, p.nx, p.nt, p.ihx);
        const float uxx = d2_at(p.u + j, i, p.nx, p.nt, p.ihxx);
        const float r = ut + p.u[idx] * ux - p.nu * uxx;
        p.out[idx] = r;
        acc[0] = r * r;
    }
    if (p.partials != nullptr) block_reduce_store<1>(acc, p.partials, p.nitems, blockIdx.x);
}

__global__ void __launch_bounds__(256) burgers_bwd_kernel(const BurgersParams p) {
    pdl_wait_then_trigger();
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    const int N = p.nx * p.nt;
    if (idx >= N) return;
    const int nt = p.nt, nx = p.nx;
    const int i = idx / nt, j = idx - i * nt;
    const float* __restrict__ u = p.u;
    const float* __restrict__ G = p.g;
    auto Gt = [&](int jj) { return G[(size_t)i * nt + jj]; };            // G along t through row i
    auto Gx = [&](int ii) { return G[(size_t)ii * nt + j]; };            // G along x through column j
    auto uGx = [&](int ii) { return u[(size_t)ii * nt + j] * G[(size_t)ii * nt + j]; };
    const float ux = d1_at(u + j, i, nx, nt, p.ihx);
    const float g = d1T_at(Gt, j, nt, p.iht) + ux * G[idx] + d1T_at(uGx, i, nx, p.ihx)
                  - p.nu * d2T_at(Gx, i, nx, p.ihxx);
    p.out[idx] = p.gs * g;
}

static void burgers_params(const Problem& q, BurgersParams& p) {
    p.nx = q.n[0]; p.nt = q.n[1];
    p.ihx = (float)(0.5 / q.h[0]); p.iht = (float)(0.5 / q.h[1]);
    p.ihxx = (float)(1.0 / (q.h[0] * q.h[0]));
    p.nu = (float)q.coef[0];
    p.nitems = (p.nx * p.nt + 255) / 256;
}

int burgers_items(const int* n) { return (n[0] * n[1] + 255) / 256; }

cudaError_t launch_burgers_fwd(const Problem& q) {
    BurgersParams p{};
    burgers_params(q, p);
    p.u = q.in[0]; p.out = q.out[0]; p.partials = q.partials;
    return launch_kernel(burgers_fwd_kernel, dim3(p.nitems), dim3(256), q.stream, p);
}

cudaError_t launch_burgers_bwd(const Problem& q) {
    BurgersParams p{};
    burgers_params(q, p);
    p.u = q.in[0]; p.g = q.aux[0]; p.out = q.out[0]; p.gs = (float)q.gscale[0];
    return launch_kernel(burgers_bwd_kernel, dim3(p.nitems), dim3(256), q.stream, p);
}

}  // namespace fpde
