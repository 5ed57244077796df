// Host-side internal interface between the C-ABI layer (validation, registry) and the
// per-operator launchers.  Not installed; the public interface is include/fpde.h.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace fpde {

constexpr int MAX_F = 4;   // most fields / residuals of any operator
constexpr int MAX_D = 4;   // most array axes

// A validated problem, as the launchers see it.
struct Problem {
    int op;
    int ndim;
    int n[MAX_D];            // extents, memory order
    double h[MAX_D];         // spacings
    double coef[8];          // operator coefficients
    const float* in[MAX_F];  // fwd: fields            bwd: fields
    const float* aux[MAX_F]; // fwd: sources           bwd: upstream dL/dr_e
    float* out[MAX_F];       // fwd: residuals         bwd: field gradients
    double gscale[MAX_F];    // bwd only
    float* partials;         // fwd: loss partial sums (NULL = no loss)
    double* loss_out;        // fwd: device, E+1 doubles
    int64_t rows;            // N_r
    cudaStream_t stream;
    bool bc0_interior;       // unsteady NS only: x axis not periodic (the slab form of the operator)
    // unsteady NS only: planes per work item (0 = the launcher's default) and the range of plane
    // chunks this launch covers (chunk_hi <= chunk_lo = all); the loss partial sums keep their
    // global slots, so several ranged launches add up to one full launch
    int planes_per_item, chunk_lo, chunk_hi;
    // bwd: the upstream arrays are residual arrays a forward kernel of this library wrote (exactly
    // zero at nodes without a row), so the adjoint need not zero-extend them itself
    bool gres_zero_off_rows;
};

// The same for the double-precision verification path (ops_f64.cu).
struct ProblemF64 {
    int op, ndim, radius;
    int n[MAX_D];
    int bc[MAX_D];
    double h[MAX_D];
    double coef[8];
    const double* in[MAX_F];
    const double* aux[MAX_F];
    double* out[MAX_F];
    double gscale[MAX_F];
    double* partials;        // fwd: one double per block and residual (NULL = no loss)
    double* loss_out;
    int64_t rows;
    cudaStream_t stream;
};
int f64_blocks(int64_t N);
cudaError_t launch_f64_fwd(const ProblemF64& p, int nresiduals);
cudaError_t launch_f64_bwd(const ProblemF64& p, int nfields);

// Launch with programmatic stream serialisation allowed (kernels call pdl_wait_then_trigger()).
// FPDE_PDL=0 in the environment falls back to plain stream order (for A/B measurements).
bool pdl_enabled();
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = 0; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = pdl_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Args&&>(args)...);
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel_smem(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem_bytes,
                                      cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem_bytes; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = pdl_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Args&&>(args)...);
}

// Planes per work item of the 2.5-D kernels: the length tuned on large grids, halved on grids that
// items of that length would not spread over the GPU, never below 4.  On small grids a step is
// latency-bound and what counts is how many items march concurrently: at least four per SM on
// grids whose arrays fit L2 several times over (under 2^22 points), two per SM above that, where
// longer items pay by re-reading fewer halo planes.
inline int planes_for_grid(int n0, int tuned, long items_per_chunk, long long points) {
    const long target = (points < (1ll << 22) ? 4 : 2) * 148;
    int planes = tuned;
    while (planes > 4 && items_per_chunk * ((n0 + planes - 1) / planes) < target) planes = planes / 2 < 4 ? 4 : planes / 2;
    return planes;
}

// SMs of the current device (148 when there is none to ask: host-only queries).
inline int sm_count_or_default() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
        (void)cudaGetLastError();
        return 148;
    }
    return n;
}

// Wave fitting for grids that fill the GPU: with `planes` planes per item a launch has
// items_per_chunk * ceil(n0 / planes) blocks, which run in ceil(blocks / slots) waves (slots = SMs x
// resident blocks per SM).  A last wave that is nearly empty, or a single wave that leaves some SMs
// with one block more than others, costs up to a full item; this returns the item length whose
// block count just fits the same number of waves (a little longer items, fewer blocks).
inline int fit_planes_to_waves(int n0, int planes, long items_per_chunk, long slots) {
    if (items_per_chunk < 1 || slots < 1) return planes;
    const long blocks = items_per_chunk * ((n0 + planes - 1) / planes);
    const long waves = (blocks + slots - 1) / slots;
    const long chunks = waves * slots / items_per_chunk;           // most chunks that still fit
    if (chunks < 1) return planes;
    const int fitted = (int)((n0 + chunks - 1) / chunks);
    return fitted >= planes ? fitted : planes;                      // never shorter than the tuned length
}

// Launchers: return cudaGetLastError() after queuing the kernels.
cudaError_t launch_burgers_fwd(const Problem& p);
cudaError_t launch_burgers_bwd(const Problem& p);
cudaError_t launch_lap2d_fwd(const Problem& p);     // Poisson 2-D and Gray-Scott
cudaError_t launch_lap2d_bwd(const Problem& p);
cudaError_t launch_helmholtz_fwd(const Problem& p, int* items);   // *items: loss partial sums written
cudaError_t launch_helmholtz_bwd(const Problem& p);
cudaError_t launch_ns2d_fwd(const Problem& p);    // steady 2-D Navier-Stokes
cudaError_t launch_ns2d_bwd(const Problem& p);
cudaError_t launch_ns3d_fwd(const Problem& p);    // steady 3-D Navier-Stokes
cudaError_t launch_ns3d_bwd(const Problem& p);
cudaError_t launch_ns_fwd(const Problem& p);
// Helmholtz engine staged through shared memory by the copy engine (op_helmholtz3d_tma.cu);
// `launched` false = this grid runs on the L1-staged engine
bool star3d_tma_wanted(const int* n);
int star3d_tma_items(const int* n);
cudaError_t launch_star3d_tma(const Problem& p, int mode, int* items, bool& launched);
unsigned int star3d_tma_timeouts();
// Helmholtz single pass (op_helmholtz3d_fused.cu): residual, loss partial sums and gradient in one
// kernel; `res` may be NULL (residuals not stored)
bool star3d_fused_supported(const int* n);
int star3d_fused_items(const int* n);
cudaError_t launch_star3d_fused(const Problem& p, float* res, int* items);
unsigned int star3d_fused_timeouts();
// TMA-staged variants (op_ns3dt_tma.cu); `launched` false = this grid is not eligible
bool ns_tma_wanted(const int* n);
bool ns_tma_geometry_ok(const int* n, int ty, int na, size_t smem_limit);
int ns_tma_items(const int* n);
cudaError_t launch_ns_fwd_tma(const Problem& p, bool& launched);
cudaError_t launch_ns_bwd_tma(const Problem& p, bool& launched);
unsigned int ns_tma_timeouts();
// single-pass residual + loss + gradient (op_fused2d.cu); `res` entries may be NULL
bool fused2d_supported(int op);
int fused2d_items(int op, const int* n);
int fused2d_max_items(const int* n);
cudaError_t launch_fused2d(const Problem& p, float* const* res);
cudaError_t launch_ns_bwd(const Problem& p);

// Final, fixed-order fp64 sum of the per-item partials: loss_out[e] = sum/N_r, loss_out[E] = total.
cudaError_t launch_loss_finalize(const float* partials, int nitems, int nres, int64_t rows,
                                 double* loss_out, cudaStream_t stream);

}  // namespace fpde
