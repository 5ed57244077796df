// C ABI of libfpde.so: operator registry, argument validation, conversion of host scalars to
// kernel parameters, dispatch to the per-operator launchers, and the final loss reduction.
// See include/fpde.h for the contract of every entry point.
#include <cuda.h>

#include "../../include/fpde.h"
#include "fpde_common.cuh"
#include "fpde_internal.h"

#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

namespace fpde {

int lap2d_items(const int* n);
int star3d_items(const int* n);
int ns_items(const int* n, bool xint, int planes_per_item = 0);
int ns_plane_chunk(const int* n, bool xint);
int burgers_items(const int* n);
int ns2d_items(const int* n);
int ns3d_items(const int* n);

struct OpEntry {
    int ndim, nf, ns, ne, nc, radius;
    int bc[MAX_D];
    bool x4;                // contiguous extent must be a multiple of 4
};

static const OpEntry REGISTRY[FPDE_OP_COUNT] = {
    /* BURGERS_1D_T    */ {2, 1, 0, 1, 1, 1, {FPDE_BC_ONE_SIDED, FPDE_BC_ONE_SIDED, 0, 0}, false},
    /* POISSON_2D      */ {2, 1, 1, 1, 0, 1, {FPDE_BC_INTERIOR, FPDE_BC_INTERIOR, 0, 0}, true},
    /* GRAYSCOTT_2D    */ {2, 2, 0, 2, 4, 1, {FPDE_BC_PERIODIC, FPDE_BC_PERIODIC, 0, 0}, true},
    /* HELMHOLTZ_3D_O4 */ {3, 1, 1, 1, 1, 2, {FPDE_BC_INTERIOR, FPDE_BC_INTERIOR, FPDE_BC_INTERIOR, 0}, true},
    /* NS_3D_T         */ {4, 4, 0, 4, 1, 1, {FPDE_BC_PERIODIC, FPDE_BC_PERIODIC, FPDE_BC_PERIODIC, FPDE_BC_INTERIOR}, true},
    /* NS_2D_STEADY    */ {2, 3, 0, 3, 1, 1, {FPDE_BC_INTERIOR, FPDE_BC_INTERIOR, 0, 0}, true},
    /* NS_3D_STEADY    */ {3, 4, 0, 4, 1, 1, {FPDE_BC_INTERIOR, FPDE_BC_INTERIOR, FPDE_BC_INTERIOR, 0}, true},
    /* NS_3D_T_XSLAB   */ {4, 4, 0, 4, 1, 1, {FPDE_BC_INTERIOR, FPDE_BC_PERIODIC, FPDE_BC_PERIODIC, FPDE_BC_INTERIOR}, true},
    /* GRAYSCOTT_XSLAB */ {2, 2, 0, 2, 4, 1, {FPDE_BC_INTERIOR, FPDE_BC_PERIODIC, 0, 0}, true},
};

static int check_shape(int op, int ndim, const int64_t* shape, int* n_out, int64_t* total, int64_t* rows) {
    if (op < 0 || op >= FPDE_OP_COUNT) return FPDE_ERR_BAD_OP;
    if (!shape) return FPDE_ERR_NULL;
    const OpEntry& e = REGISTRY[op];
    if (ndim != e.ndim) return FPDE_ERR_NDIM;
    int64_t N = 1, R = 1;
    for (int a = 0; a < ndim; ++a) {
        const int64_t n = shape[a];
        const int64_t need = e.bc[a] == FPDE_BC_ONE_SIDED ? 4 : 2 * e.radius + 1;
        if (n < need || n > (int64_t)1 << 30) return FPDE_ERR_SHAPE;
        N *= n;
        if (N >= (int64_t)1 << 31) return FPDE_ERR_SHAPE;
        R *= e.bc[a] == FPDE_BC_INTERIOR ? n - 2 * e.radius : n;
        if (n_out) n_out[a] = (int)n;
    }
    if (e.x4 && shape[ndim - 1] % 4 != 0) return FPDE_ERR_SHAPE;
    if (total) *total = N;
    if (rows) *rows = R;
    return FPDE_OK;
}

// Planes per chunk of the launches over ranges of x-planes (unsteady NS): the launcher's own choice
// for this grid, shortened on short arrays until there are at least four chunks (never below four
// planes), so that a slab of a grid split many ways still has chunks away from its halo planes.
static int ranged_plane_chunk(const int* n, bool xint) {
    int P = ns_plane_chunk(n, xint);
    while (P > 4 && (n[0] + P - 1) / P < 4) P = std::max(4, P / 2);
    return P;
}

static size_t workspace_need(int op, const int* n) {
    int items = 0;
    switch (op) {
    case FPDE_OP_BURGERS_1D_T: items = burgers_items(n); break;
    case FPDE_OP_POISSON_2D:
    case FPDE_OP_GRAYSCOTT_2D:
    case FPDE_OP_GRAYSCOTT_2D_XSLAB: items = lap2d_items(n); break;
    case FPDE_OP_HELMHOLTZ_3D_O4: items = star3d_items(n); break;
    // (the launches over ranges of plane chunks may use a shorter chunk, i.e. more partial sums)
    case FPDE_OP_NS_3D_T: items = std::max(ns_items(n, false), ns_items(n, false, ranged_plane_chunk(n, false))); break;
    case FPDE_OP_NS_3D_T_XSLAB: items = std::max(ns_items(n, true), ns_items(n, true, ranged_plane_chunk(n, true))); break;
    case FPDE_OP_NS_2D_STEADY: items = ns2d_items(n); break;
    case FPDE_OP_NS_3D_STEADY: items = ns3d_items(n); break;
    }
    return (size_t)items * REGISTRY[op].ne * sizeof(float);
}

bool pdl_enabled() {
    const char* s = std::getenv("FPDE_PDL");
    return !(s && s[0] == '0');
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Common validation of the arguments fwd and bwd share; fills the Problem.
static int validate(int op, const float* const* fields, int ndim, const int64_t* shape,
                    const double* spacing, const double* coeffs, int ncoeffs, const int* bc,
                    Problem& q) {
    int st = check_shape(op, ndim, shape, q.n, nullptr, &q.rows);
    if (st != FPDE_OK) return st;
    const OpEntry& e = REGISTRY[op];
    if (!fields || !spacing || !bc) return FPDE_ERR_NULL;
    if (ncoeffs != e.nc) return FPDE_ERR_COEFF_COUNT;
    if (e.nc > 0 && !coeffs) return FPDE_ERR_NULL;
    for (int a = 0; a < ndim; ++a) {
        if (!(spacing[a] > 0.0) || !std::isfinite(spacing[a])) return FPDE_ERR_SPACING;
        if (bc[a] != e.bc[a]) return FPDE_ERR_BC;
        q.h[a] = spacing[a];
    }
    for (int c = 0; c < e.nc; ++c) {
        if (!std::isfinite(coeffs[c])) return FPDE_ERR_SPACING;
        q.coef[c] = coeffs[c];
    }
    for (int f = 0; f < e.nf; ++f) {
        if (!fields[f]) return FPDE_ERR_NULL;
        if (!aligned16(fields[f])) return FPDE_ERR_ALIGN;
        q.in[f] = fields[f];
    }
    q.op = op; q.ndim = ndim;
    q.bc0_interior = op == FPDE_OP_NS_3D_T_XSLAB;
    return FPDE_OK;
}

// Fixed-order final sum.  Thread t adds partials t, t+T, ... (T = threads of the block, four
// independent loads in flight, combined in a fixed order) in fp64; then a shuffle tree inside each
// warp and one over the warp sums.  One block, so no inter-block ordering exists to vary: the
// result depends on the data and on T only, and T is a function of the number of partials.
__global__ void __launch_bounds__(1024) loss_finalize_kernel(const float* __restrict__ partials, int nitems,
                                                             int nres, double inv_rows,
                                                             double* __restrict__ loss_out) {
    __shared__ double sm[MAX_F][32];
    pdl_wait_then_trigger();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int T = blockDim.x, nwarps = T >> 5;
    double s[MAX_F];
#pragma unroll
    for (int e = 0; e < MAX_F; ++e) {
        s[e] = 0.0;
        if (e < nres) {
            const float* p = partials + (size_t)e * nitems;
            int i = tid;
            for (; i + 3 * T < nitems; i += 4 * T) {
                const float a = p[i], b = p[i + T], c = p[i + 2 * T], d = p[i + 3 * T];
                s[e] += ((double)a + (double)b) + ((double)c + (double)d);
            }
            for (; i < nitems; i += T) s[e] += (double)p[i];
        }
    }
#pragma unroll
    for (int e = 0; e < MAX_F; ++e) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s[e] += __shfl_down_sync(FULL_MASK, s[e], o);
        if (lane == 0) sm[e][warp] = s[e];
    }
    __syncthreads();
    if (warp == 0) {
        double total = 0.0;
#pragma unroll
        for (int e = 0; e < MAX_F; ++e) {
            double v = lane < nwarps ? sm[e][lane] : 0.0;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(FULL_MASK, v, o);
            if (e < nres) {
                const double le = v * inv_rows;
                if (lane == 0) loss_out[e] = le;
                total += le;
            }
        }
        if (lane == 0) loss_out[nres] = total;
    }
}

cudaError_t launch_loss_finalize(const float* partials, int nitems, int nres, int64_t rows,
                                 double* loss_out, cudaStream_t stream) {
    // a small block for few partial sums (it starts sooner and its tree is shorter), the full one
    // for many
    const char* e = std::getenv("FPDE_FINALIZE_THREADS");
    int threads = e && *e ? std::atoi(e) : (nitems <= 1024 ? 128 : (nitems <= 8192 ? 256 : 1024));
    threads = std::max(32, std::min(1024, (threads / 32) * 32));
    return launch_kernel(loss_finalize_kernel, dim3(1), dim3(threads), stream, partials, nitems, nres,
                         1.0 / (double)rows, loss_out);
}

}  // namespace fpde

using namespace fpde;

extern "C" {

int fpde_op_info(int op, fpde_op_info_t* out) {
    if (op < 0 || op >= FPDE_OP_COUNT) return FPDE_ERR_BAD_OP;
    if (!out) return FPDE_ERR_NULL;
    const OpEntry& e = REGISTRY[op];
    out->ndim = e.ndim; out->nfields = e.nf; out->nsources = e.ns; out->nresiduals = e.ne;
    out->ncoeffs = e.nc; out->radius = e.radius;
    for (int a = 0; a < 4; ++a) out->bc[a] = a < e.ndim ? e.bc[a] : 0;
    return FPDE_OK;
}

const char* fpde_strerror(int status) {
    switch (status) {
    case FPDE_OK: return "ok";
    case FPDE_ERR_BAD_OP: return "operator id out of range";
    case FPDE_ERR_NULL: return "a required pointer is NULL";
    case FPDE_ERR_NDIM: return "ndim does not match the operator";
    case FPDE_ERR_SHAPE: return "grid extent too small, too large, or contiguous extent not a multiple of 4";
    case FPDE_ERR_ALIGN: return "device pointer not 16-byte aligned";
    case FPDE_ERR_SPACING: return "spacing or coefficient not finite / not positive";
    case FPDE_ERR_COEFF_COUNT: return "ncoeffs does not match the operator";
    case FPDE_ERR_BC: return "boundary kinds not supported by the operator";
    case FPDE_ERR_WORKSPACE: return "workspace NULL, misaligned or too small";
    case FPDE_ERR_CUDA: return "CUDA runtime error";
    default: return "unknown status";
    }
}

int64_t fpde_row_count(int op, int ndim, const int64_t* shape) {
    int64_t rows = 0;
    if (check_shape(op, ndim, shape, nullptr, nullptr, &rows) != FPDE_OK) return 0;
    return rows;
}

size_t fpde_workspace_bytes(int op, int ndim, const int64_t* shape) {
    int n[MAX_D] = {0, 0, 0, 0};
    if (check_shape(op, ndim, shape, n, nullptr, nullptr) != FPDE_OK) return 0;
    // rounded up generously so that tile-shape tuning never outgrows a caller's allocation
    const size_t need = workspace_need(op, n);
    return ((need + 255) / 256) * 256 + 4096;
}

// chunk_hi > chunk_lo: only the work items of those chunks of x-planes are launched (operators whose
// launcher can do that), and the loss vector is formed only if `finish`.
static int fwd_impl(int op, const float* const* fields, const float* const* sources, float* const* residuals,
                    double* loss_out, int ndim, const int64_t* shape, const double* spacing,
                    const double* coeffs, int ncoeffs, const int* bc, void* workspace, size_t workspace_bytes,
                    void* stream, int64_t loss_rows, int chunk_lo = 0, int chunk_hi = 0, int finish = 1);

int fpde_fwd(int op, const float* const* fields, const float* const* sources, float* const* residuals,
             double* loss_out, int ndim, const int64_t* shape, const double* spacing,
             const double* coeffs, int ncoeffs, const int* bc, void* workspace, size_t workspace_bytes,
             void* stream) {
    return fwd_impl(op, fields, sources, residuals, loss_out, ndim, shape, spacing, coeffs, ncoeffs, bc, workspace,
                    workspace_bytes, stream, 0);
}

int fpde_fwd_rows(int op, const float* const* fields, const float* const* sources, float* const* residuals,
                  double* loss_out, int ndim, const int64_t* shape, const double* spacing,
                  const double* coeffs, int ncoeffs, const int* bc, void* workspace, size_t workspace_bytes,
                  void* stream, int64_t loss_rows) {
    if (loss_rows < 1) return FPDE_ERR_SHAPE;
    return fwd_impl(op, fields, sources, residuals, loss_out, ndim, shape, spacing, coeffs, ncoeffs, bc, workspace,
                    workspace_bytes, stream, loss_rows);
}

static bool has_plane_chunks(int op) { return op == FPDE_OP_NS_3D_T || op == FPDE_OP_NS_3D_T_XSLAB; }

// planes per chunk of the ranged launches: the launcher's own choice for this grid
static int plane_chunk_of(int op, const int* n) {
    if (!has_plane_chunks(op)) return 0;
    return ranged_plane_chunk(n, op == FPDE_OP_NS_3D_T_XSLAB);
}

static int fwd_impl(int op, const float* const* fields, const float* const* sources, float* const* residuals,
                    double* loss_out, int ndim, const int64_t* shape, const double* spacing,
                    const double* coeffs, int ncoeffs, const int* bc, void* workspace, size_t workspace_bytes,
                    void* stream, int64_t loss_rows, int chunk_lo, int chunk_hi, int finish) {
    Problem q;
    std::memset(&q, 0, sizeof(q));
    int st = validate(op, fields, ndim, shape, spacing, coeffs, ncoeffs, bc, q);
    if (st != FPDE_OK) return st;
    const OpEntry& e = REGISTRY[op];
    if (!residuals) return FPDE_ERR_NULL;
    if (e.ns > 0 && !sources) return FPDE_ERR_NULL;
    for (int s = 0; s < e.ns; ++s) {
        if (!sources[s]) return FPDE_ERR_NULL;
        if (!aligned16(sources[s])) return FPDE_ERR_ALIGN;
        q.aux[s] = sources[s];
    }
    for (int r = 0; r < e.ne; ++r) {
        if (!residuals[r]) return FPDE_ERR_NULL;
        if (!aligned16(residuals[r])) return FPDE_ERR_ALIGN;
        q.out[r] = residuals[r];
    }
    if (loss_out) {
        if (!aligned16(loss_out)) return FPDE_ERR_ALIGN;
        if (!workspace || !aligned16(workspace) || workspace_bytes < workspace_need(op, q.n))
            return FPDE_ERR_WORKSPACE;
        q.partials = static_cast<float*>(workspace);
        q.loss_out = loss_out;
    }
    q.stream = static_cast<cudaStream_t>(stream);
    cudaError_t ce = cudaSuccess;
    int items = 0;
    if (chunk_hi > chunk_lo) {
        // a range of plane chunks: fixed chunk length, partial sums in their global slots
        const int P = plane_chunk_of(op, q.n);
        if (P <= 0) return FPDE_ERR_BAD_OP;
        const int nchunks = (q.n[0] + P - 1) / P;
        if (chunk_lo < 0 || chunk_hi > nchunks) return FPDE_ERR_SHAPE;
        q.planes_per_item = P; q.chunk_lo = chunk_lo; q.chunk_hi = chunk_hi;
        if (loss_out && workspace_bytes < (size_t)ns_items(q.n, q.bc0_interior, P) * e.ne * sizeof(float))
            return FPDE_ERR_WORKSPACE;
        ce = launch_ns_fwd(q);
        if (ce != cudaSuccess) return FPDE_ERR_CUDA;
        if (loss_out && finish) {
            ce = launch_loss_finalize(q.partials, ns_items(q.n, q.bc0_interior, P), e.ne, loss_rows > 0 ? loss_rows : q.rows,
                                      loss_out, q.stream);
            if (ce != cudaSuccess) return FPDE_ERR_CUDA;
        }
        return FPDE_OK;
    }
    switch (op) {
    case FPDE_OP_BURGERS_1D_T: ce = launch_burgers_fwd(q); items = burgers_items(q.n); break;
    case FPDE_OP_POISSON_2D:
    case FPDE_OP_GRAYSCOTT_2D:
    case FPDE_OP_GRAYSCOTT_2D_XSLAB: ce = launch_lap2d_fwd(q); items = lap2d_items(q.n); break;
    case FPDE_OP_HELMHOLTZ_3D_O4: ce = launch_helmholtz_fwd(q, &items); break;
    case FPDE_OP_NS_3D_T: ce = launch_ns_fwd(q); items = ns_items(q.n, false); break;
    case FPDE_OP_NS_3D_T_XSLAB: ce = launch_ns_fwd(q); items = ns_items(q.n, true); break;
    case FPDE_OP_NS_2D_STEADY: ce = launch_ns2d_fwd(q); items = ns2d_items(q.n); break;
    case FPDE_OP_NS_3D_STEADY: ce = launch_ns3d_fwd(q); items = ns3d_items(q.n); break;
    }
    if (ce != cudaSuccess) return FPDE_ERR_CUDA;
    if (loss_out) {
        ce = launch_loss_finalize(q.partials, items, e.ne, loss_rows > 0 ? loss_rows : q.rows, loss_out, q.stream);
        if (ce != cudaSuccess) return FPDE_ERR_CUDA;
    }
    return FPDE_OK;
}

static int bwd_impl(int op, const float* const* fields, const float* const* gres, const double* gscale,
                    float* const* gfields, int ndim, const int64_t* shape, const double* spacing,
                    const double* coeffs, int ncoeffs, const int* bc, void* stream, bool gres_zero_off_rows,
                    int chunk_lo = 0, int chunk_hi = 0);

int fpde_bwd(int op, const float* const* fields, const float* const* gres, const double* gscale,
             float* const* gfields, int ndim, const int64_t* shape, const double* spacing,
             const double* coeffs, int ncoeffs, const int* bc, void* workspace, size_t workspace_bytes,
             void* stream) {
    (void)workspace; (void)workspace_bytes;
    return bwd_impl(op, fields, gres, gscale, gfields, ndim, shape, spacing, coeffs, ncoeffs, bc, stream, false);
}

int fpde_plane_chunk(int op, int ndim, const int64_t* shape) {
    int n[MAX_D] = {0, 0, 0, 0};
    if (check_shape(op, ndim, shape, n, nullptr, nullptr) != FPDE_OK) return 0;
    return plane_chunk_of(op, n);
}

int fpde_fwd_chunks(int op, const float* const* fields, const float* const* sources, float* const* residuals,
                    double* loss_out, int ndim, const int64_t* shape, const double* spacing,
                    const double* coeffs, int ncoeffs, const int* bc, void* workspace, size_t workspace_bytes,
                    void* stream, int64_t loss_rows, int chunk_lo, int chunk_hi, int finish) {
    if (op < 0 || op >= FPDE_OP_COUNT || !has_plane_chunks(op)) return FPDE_ERR_BAD_OP;
    if (chunk_hi <= chunk_lo || loss_rows < 0) return FPDE_ERR_SHAPE;
    return fwd_impl(op, fields, sources, residuals, loss_out, ndim, shape, spacing, coeffs, ncoeffs, bc, workspace,
                    workspace_bytes, stream, loss_rows, chunk_lo, chunk_hi, finish);
}

int fpde_bwd_chunks(int op, const float* const* fields, const float* const* gres, const double* gscale,
                    float* const* gfields, int ndim, const int64_t* shape, const double* spacing,
                    const double* coeffs, int ncoeffs, const int* bc, void* stream, int chunk_lo, int chunk_hi) {
    if (op < 0 || op >= FPDE_OP_COUNT || !has_plane_chunks(op)) return FPDE_ERR_BAD_OP;
    if (chunk_hi <= chunk_lo) return FPDE_ERR_SHAPE;
    return bwd_impl(op, fields, gres, gscale, gfields, ndim, shape, spacing, coeffs, ncoeffs, bc, stream, false,
                    chunk_lo, chunk_hi);
}

static int bwd_impl(int op, const float* const* fields, const float* const* gres, const double* gscale,
                    float* const* gfields, int ndim, const int64_t* shape, const double* spacing,
                    const double* coeffs, int ncoeffs, const int* bc, void* stream, bool gres_zero_off_rows,
                    int chunk_lo, int chunk_hi) {
    Problem q;
    std::memset(&q, 0, sizeof(q));
    int st = validate(op, fields, ndim, shape, spacing, coeffs, ncoeffs, bc, q);
    if (st != FPDE_OK) return st;
    const OpEntry& e = REGISTRY[op];
    if (!gres || !gfields) return FPDE_ERR_NULL;
    for (int r = 0; r < e.ne; ++r) {
        if (!gres[r]) return FPDE_ERR_NULL;
        if (!aligned16(gres[r])) return FPDE_ERR_ALIGN;
        q.aux[r] = gres[r];
        q.gscale[r] = gscale ? gscale[r] : 1.0;
        if (!std::isfinite(q.gscale[r])) return FPDE_ERR_SPACING;
    }
    for (int f = 0; f < e.nf; ++f) {
        if (!gfields[f]) return FPDE_ERR_NULL;
        if (!aligned16(gfields[f])) return FPDE_ERR_ALIGN;
        q.out[f] = gfields[f];
    }
    q.stream = static_cast<cudaStream_t>(stream);
    q.gres_zero_off_rows = gres_zero_off_rows;
    cudaError_t ce = cudaSuccess;
    if (chunk_hi > chunk_lo) {
        const int P = plane_chunk_of(op, q.n);
        if (P <= 0) return FPDE_ERR_BAD_OP;
        if (chunk_lo < 0 || chunk_hi > (q.n[0] + P - 1) / P) return FPDE_ERR_SHAPE;
        q.planes_per_item = P; q.chunk_lo = chunk_lo; q.chunk_hi = chunk_hi;
        return launch_ns_bwd(q) == cudaSuccess ? FPDE_OK : FPDE_ERR_CUDA;
    }
    switch (op) {
    case FPDE_OP_BURGERS_1D_T: ce = launch_burgers_bwd(q); break;
    case FPDE_OP_POISSON_2D:
    case FPDE_OP_GRAYSCOTT_2D:
    case FPDE_OP_GRAYSCOTT_2D_XSLAB: ce = launch_lap2d_bwd(q); break;
    case FPDE_OP_HELMHOLTZ_3D_O4: ce = launch_helmholtz_bwd(q); break;
    case FPDE_OP_NS_3D_T:
    case FPDE_OP_NS_3D_T_XSLAB: ce = launch_ns_bwd(q); break;
    case FPDE_OP_NS_2D_STEADY: ce = launch_ns2d_bwd(q); break;
    case FPDE_OP_NS_3D_STEADY: ce = launch_ns3d_bwd(q); break;
    }
    return ce == cudaSuccess ? FPDE_OK : FPDE_ERR_CUDA;
}

// The Helmholtz single-pass kernel is a measured prototype: slower than forward + adjoint on the
// grids tried (see the design notes), so it only runs when asked for (FPDE_STAR3D_SINGLE_PASS=1).
static bool helmholtz_single_pass_wanted(const int* n) {
    const char* s = std::getenv("FPDE_STAR3D_SINGLE_PASS");
    return s && s[0] == '1' && star3d_fused_supported(n);
}

int fpde_has_single_pass(int op) {
    return (op >= 0 && op < FPDE_OP_COUNT && fused2d_supported(op)) ? 1 : 0;
}

size_t fpde_fwd_bwd_workspace_bytes(int op, int ndim, const int64_t* shape) {
    int n[MAX_D] = {0, 0, 0, 0};
    if (check_shape(op, ndim, shape, n, nullptr, nullptr) != FPDE_OK) return 0;
    if (!fused2d_supported(op)) return fpde_workspace_bytes(op, ndim, shape);
    const size_t need = (size_t)fused2d_max_items(n) * REGISTRY[op].ne * sizeof(float);
    return ((need + 255) / 256) * 256 + 4096;
}

int fpde_fwd_bwd(int op, const float* const* fields, const float* const* sources, float* const* residuals,
                 float* const* gfields, double* loss_out, int ndim, const int64_t* shape, const double* spacing,
                 const double* coeffs, int ncoeffs, const int* bc, void* workspace, size_t workspace_bytes,
                 void* stream) {
    Problem q;
    std::memset(&q, 0, sizeof(q));
    int st = validate(op, fields, ndim, shape, spacing, coeffs, ncoeffs, bc, q);
    if (st != FPDE_OK) return st;
    const OpEntry& e = REGISTRY[op];
    if (!gfields) return FPDE_ERR_NULL;
    if (op == FPDE_OP_HELMHOLTZ_3D_O4 && helmholtz_single_pass_wanted(q.n)) {
        // one kernel: the planes of r go from the forward star to the adjoint star through shared memory
        if (!sources || !sources[0] || !gfields[0]) return FPDE_ERR_NULL;
        if (!aligned16(sources[0]) || !aligned16(gfields[0])) return FPDE_ERR_ALIGN;
        float* res = residuals ? residuals[0] : nullptr;
        if (res && !aligned16(res)) return FPDE_ERR_ALIGN;
        q.aux[0] = sources[0]; q.out[0] = gfields[0];
        if (loss_out) {
            if (!aligned16(loss_out)) return FPDE_ERR_ALIGN;
            if (!workspace || !aligned16(workspace) || workspace_bytes < (size_t)star3d_fused_items(q.n) * sizeof(float))
                return FPDE_ERR_WORKSPACE;
            q.partials = static_cast<float*>(workspace);
            q.loss_out = loss_out;
        }
        q.stream = static_cast<cudaStream_t>(stream);
        int items = 0;
        cudaError_t ce = launch_star3d_fused(q, res, &items);
        if (ce != cudaSuccess) return FPDE_ERR_CUDA;
        if (loss_out && launch_loss_finalize(q.partials, items, e.ne, q.rows, loss_out, q.stream) != cudaSuccess)
            return FPDE_ERR_CUDA;
        return FPDE_OK;
    }
    if (!fused2d_supported(op)) {
        // two kernels with the residual arrays as the intermediate
        if (!residuals) return FPDE_ERR_NULL;
        for (int f = 0; f < e.nf; ++f) {
            if (!gfields[f]) return FPDE_ERR_NULL;
            if (!aligned16(gfields[f])) return FPDE_ERR_ALIGN;
        }
        st = fpde_fwd(op, fields, sources, residuals, loss_out, ndim, shape, spacing, coeffs, ncoeffs, bc, workspace,
                      workspace_bytes, stream);
        if (st != FPDE_OK) return st;
        double gscale[MAX_F];
        for (int r = 0; r < e.ne; ++r) gscale[r] = 2.0 / (double)q.rows;
        // the upstream arrays are the residual arrays the forward kernel just wrote
        return bwd_impl(op, fields, residuals, gscale, gfields, ndim, shape, spacing, coeffs, ncoeffs, bc, stream, true);
    }
    if (e.ns > 0 && !sources) return FPDE_ERR_NULL;
    for (int s = 0; s < e.ns; ++s) {
        if (!sources[s]) return FPDE_ERR_NULL;
        if (!aligned16(sources[s])) return FPDE_ERR_ALIGN;
        q.aux[s] = sources[s];
    }
    float* res[MAX_F] = {nullptr, nullptr, nullptr, nullptr};
    for (int r = 0; r < e.ne; ++r) {
        res[r] = residuals ? residuals[r] : nullptr;
        if (res[r] && !aligned16(res[r])) return FPDE_ERR_ALIGN;
    }
    for (int f = 0; f < e.nf; ++f) {
        if (!gfields[f]) return FPDE_ERR_NULL;
        if (!aligned16(gfields[f])) return FPDE_ERR_ALIGN;
        q.out[f] = gfields[f];
    }
    const int items = fused2d_items(op, q.n);
    if (loss_out) {
        if (!aligned16(loss_out)) return FPDE_ERR_ALIGN;
        if (!workspace || !aligned16(workspace) || workspace_bytes < (size_t)items * e.ne * sizeof(float))
            return FPDE_ERR_WORKSPACE;
        q.partials = static_cast<float*>(workspace);
        q.loss_out = loss_out;
    }
    q.stream = static_cast<cudaStream_t>(stream);
    cudaError_t ce = launch_fused2d(q, res);
    if (ce != cudaSuccess) return FPDE_ERR_CUDA;
    if (loss_out) {
        ce = launch_loss_finalize(q.partials, items, e.ne, q.rows, loss_out, q.stream);
        if (ce != cudaSuccess) return FPDE_ERR_CUDA;
    }
    return FPDE_OK;
}

// ------------------------------------------------------------------------------------------
// double-precision verification path
// ------------------------------------------------------------------------------------------
static int validate_f64(int op, const double* const* fields, int ndim, const int64_t* shape, const double* spacing,
                        const double* coeffs, int ncoeffs, const int* bc, ProblemF64& q, int64_t* total) {
    int st = check_shape(op, ndim, shape, q.n, total, &q.rows);
    if (st != FPDE_OK) return st;
    const OpEntry& e = REGISTRY[op];
    if (!fields || !spacing || !bc) return FPDE_ERR_NULL;
    if (ncoeffs != e.nc) return FPDE_ERR_COEFF_COUNT;
    if (e.nc > 0 && !coeffs) return FPDE_ERR_NULL;
    for (int a = 0; a < ndim; ++a) {
        if (!(spacing[a] > 0.0) || !std::isfinite(spacing[a])) return FPDE_ERR_SPACING;
        if (bc[a] != e.bc[a]) return FPDE_ERR_BC;
        q.h[a] = spacing[a]; q.bc[a] = bc[a];
    }
    for (int c = 0; c < e.nc; ++c) {
        if (!std::isfinite(coeffs[c])) return FPDE_ERR_SPACING;
        q.coef[c] = coeffs[c];
    }
    for (int f = 0; f < e.nf; ++f) {
        if (!fields[f]) return FPDE_ERR_NULL;
        if (!aligned16(fields[f])) return FPDE_ERR_ALIGN;
        q.in[f] = fields[f];
    }
    q.op = op; q.ndim = ndim; q.radius = e.radius;
    return FPDE_OK;
}

size_t fpde_workspace_bytes_f64(int op, int ndim, const int64_t* shape) {
    int64_t N = 0;
    if (check_shape(op, ndim, shape, nullptr, &N, nullptr) != FPDE_OK) return 0;
    return (size_t)f64_blocks(N) * REGISTRY[op].ne * sizeof(double) + 256;
}

int fpde_fwd_f64(int op, const double* const* fields, const double* const* sources, double* const* residuals,
                 double* loss_out, int ndim, const int64_t* shape, const double* spacing, const double* coeffs,
                 int ncoeffs, const int* bc, void* workspace, size_t workspace_bytes, void* stream) {
    ProblemF64 q;
    std::memset(&q, 0, sizeof(q));
    int64_t N = 0;
    int st = validate_f64(op, fields, ndim, shape, spacing, coeffs, ncoeffs, bc, q, &N);
    if (st != FPDE_OK) return st;
    const OpEntry& e = REGISTRY[op];
    if (!residuals) return FPDE_ERR_NULL;
    if (e.ns > 0 && !sources) return FPDE_ERR_NULL;
    for (int s = 0; s < e.ns; ++s) {
        if (!sources[s]) return FPDE_ERR_NULL;
        if (!aligned16(sources[s])) return FPDE_ERR_ALIGN;
        q.aux[s] = sources[s];
    }
    for (int r = 0; r < e.ne; ++r) {
        if (!residuals[r]) return FPDE_ERR_NULL;
        if (!aligned16(residuals[r])) return FPDE_ERR_ALIGN;
        q.out[r] = residuals[r];
    }
    if (loss_out) {
        if (!aligned16(loss_out)) return FPDE_ERR_ALIGN;
        if (!workspace || !aligned16(workspace) ||
            workspace_bytes < (size_t)f64_blocks(N) * e.ne * sizeof(double))
            return FPDE_ERR_WORKSPACE;
        q.partials = static_cast<double*>(workspace);
        q.loss_out = loss_out;
    }
    q.stream = static_cast<cudaStream_t>(stream);
    return launch_f64_fwd(q, e.ne) == cudaSuccess ? FPDE_OK : FPDE_ERR_CUDA;
}

int fpde_bwd_f64(int op, const double* const* fields, const double* const* gres, const double* gscale,
                 double* const* gfields, int ndim, const int64_t* shape, const double* spacing, const double* coeffs,
                 int ncoeffs, const int* bc, void* stream) {
    ProblemF64 q;
    std::memset(&q, 0, sizeof(q));
    int st = validate_f64(op, fields, ndim, shape, spacing, coeffs, ncoeffs, bc, q, nullptr);
    if (st != FPDE_OK) return st;
    const OpEntry& e = REGISTRY[op];
    if (!gres || !gfields) return FPDE_ERR_NULL;
    for (int r = 0; r < e.ne; ++r) {
        if (!gres[r]) return FPDE_ERR_NULL;
        if (!aligned16(gres[r])) return FPDE_ERR_ALIGN;
        q.aux[r] = gres[r];
        q.gscale[r] = gscale ? gscale[r] : 1.0;
        if (!std::isfinite(q.gscale[r])) return FPDE_ERR_SPACING;
    }
    for (int f = 0; f < e.nf; ++f) {
        if (!gfields[f]) return FPDE_ERR_NULL;
        if (!aligned16(gfields[f])) return FPDE_ERR_ALIGN;
        q.out[f] = gfields[f];
    }
    q.stream = static_cast<cudaStream_t>(stream);
    return launch_f64_bwd(q, e.nf) == cudaSuccess ? FPDE_OK : FPDE_ERR_CUDA;
}

static size_t round256(size_t b) { return (b + 255) / 256 * 256; }

// scratch the host-buffer call needs: the loss partial sums of whichever launch shape it uses
// planes per work item of the pipelined host path's launches (the workspace is sized for it)
static constexpr int HOST_PIPE_ITEM_PLANES = 4;

static size_t host_workspace_bytes(int op, int ndim, const int64_t* shape) {
    size_t need = fpde_fwd_bwd_workspace_bytes(op, ndim, shape);
    int n[MAX_D] = {0, 0, 0, 0};
    if (op == FPDE_OP_NS_3D_T && check_shape(op, ndim, shape, n, nullptr, nullptr) == FPDE_OK)
        need = std::max(need, round256((size_t)ns_items(n, false, HOST_PIPE_ITEM_PLANES) * REGISTRY[op].ne * sizeof(float)) + 4096);
    return need;
}

size_t fpde_host_arena_bytes(int op, int ndim, const int64_t* shape) {
    int64_t N = 0;
    if (check_shape(op, ndim, shape, nullptr, &N, nullptr) != FPDE_OK) return 0;
    const OpEntry& e = REGISTRY[op];
    const size_t arr = round256((size_t)N * sizeof(float));
    return arr * (size_t)(2 * e.nf + e.ns + e.ne) + round256((e.ne + 1) * sizeof(double))
         + host_workspace_bytes(op, ndim, shape);
}

// ------------------------------------------------------------------------------------------
// fpde_loss_grad_host, pipelined form for the unsteady Navier-Stokes operator.
//
// The plain form queues H2D(all fields) -> kernels -> D2H(all gradients) on one stream, so the two
// copy directions never overlap and the step costs T_in + T_out.  Here the grid is cut into K
// chunks of x-planes.  The fields go up on a copy stream in transfers that run one plane ahead of
// the chunks (transfer c ends with the first plane of chunk c+1; the last plane of the grid, which
// chunk 0 reads through the periodic wrap, goes first), so the forward kernel of chunk c can run
// (on the caller's stream) as soon as transfer c has landed.  The adjoint of chunk c follows the
// forward of chunk c+1, and its gradients go down on a second copy stream while later transfers
// are still coming up.  Kernels are the ordinary ones launched over a range of work items (they
// read their x neighbours from the full arrays, periodic wrap included, and write only their own
// planes), so nothing is copied or recomputed on the device.
// What stays exposed is the lead (three transfers before the first gradients exist) and the tail
// (the gradients of the last two chunks and of chunk 0 wait for the last forward launch); the
// two chunks at either end are therefore half as long as the others.  The caller's stream waits
// for both copy streams at the end: synchronising it covers everything, as in the plain form.
// ------------------------------------------------------------------------------------------
static int host_pipe_planes() {                     // planes per chunk away from the ends: a multiple of the item
    const char* s = std::getenv("FPDE_HOST_PIPE_PLANES");
    const int v = s && *s ? std::atoi(s) : 8;
    return std::max(1, std::min(16, v / HOST_PIPE_ITEM_PLANES)) * HOST_PIPE_ITEM_PLANES;
}
// Item boundaries of the chunks: one-item chunks at the two ends (two each), host_pipe_planes()
// in between.
static std::vector<int> host_pipe_chunks(int n0) {
    const int G = HOST_PIPE_ITEM_PLANES, items = (n0 + G - 1) / G, mid = host_pipe_planes() / G;
    std::vector<int> ib{0};
    const int ends = items >= 8 ? 2 : 0;
    for (int i = 0; i < ends; ++i) ib.push_back(ib.back() + 1);
    while (ib.back() + mid <= items - ends) ib.push_back(ib.back() + mid);
    while (ib.back() < items) ib.push_back(ib.back() + 1);
    return ib;
}
// Per-device state of the pipelined host path, created on first use and kept until the process
// exits: the two copy streams and a pool of timing-free events (a call needs 2K+2 of them; making
// and destroying them on every call cost more than the launches they order).  Calls are queued
// under the mutex, one at a time; an event recorded again by a later call does not disturb the
// waits an earlier call queued on it (a stream wait captures the record that precedes it).
// Is [lo, hi) inside ONE allocation the driver knows (pinned host memory or device memory)?  A
// strided copy over several arrays is only valid when they are slices of one allocation; arrays that
// merely happen to be evenly spaced are not.  (Driver entry point through the runtime, no -lcuda.)
static bool one_allocation(const void* lo, const void* hi) {
    typedef CUresult (*GetAttrFn)(void*, CUpointer_attribute, CUdeviceptr);
    static GetAttrFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuPointerGetAttribute", &f, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return (GetAttrFn) nullptr;
        }
        return reinterpret_cast<GetAttrFn>(f);
    }();
    if (fn == nullptr) return false;
    CUdeviceptr start = 0;
    size_t size = 0;
    const CUdeviceptr p = reinterpret_cast<CUdeviceptr>(lo);
    if (fn(&start, CU_POINTER_ATTRIBUTE_RANGE_START_ADDR, p) != CUDA_SUCCESS ||
        fn(&size, CU_POINTER_ATTRIBUTE_RANGE_SIZE, p) != CUDA_SUCCESS)
        return false;
    return p >= start && reinterpret_cast<CUdeviceptr>(hi) <= start + size;
}

static std::mutex g_pipe_mutex;
struct HostPipeState {
    cudaStream_t in = nullptr, out = nullptr;
    std::vector<cudaEvent_t> events;
};
static HostPipeState g_pipe[64];

static bool host_pipeline_wanted(int op, const int* n) {
    const char* s = std::getenv("FPDE_HOST_PIPELINE");
    if (s && s[0] == '0') return false;
    return op == FPDE_OP_NS_3D_T && (int)host_pipe_chunks(n[0]).size() - 1 >= 6;
}

// Upload transfer c of a plan with item boundaries ib: planes [lo, hi).  Transfers run one plane
// ahead of the chunks; plane n0-1 goes up separately, first.
static void host_pipe_transfer(const std::vector<int>& ib, int n0, int c, int64_t* lo, int64_t* hi) {
    const int G = HOST_PIPE_ITEM_PLANES, K = (int)ib.size() - 1;
    auto end = [&](int k) { return std::min<int64_t>((int64_t)ib[k + 1] * G, n0); };
    *lo = c == 0 ? 0 : end(c - 1) + 1;
    *hi = c == K - 1 ? n0 - 1 : end(c) + 1;
    if (*hi < *lo) *hi = *lo;
}

int fpde_host_pipeline_plan(int n0, int* planes, int cap) {
    if (n0 < 1) return 0;
    const std::vector<int> ib = host_pipe_chunks(n0);
    const int K = (int)ib.size() - 1;
    const char* s = std::getenv("FPDE_HOST_PIPELINE");
    if ((s && s[0] == '0') || K < 6) return 0;
    if (planes) {
        if (cap < K) return -K;
        for (int c = 0; c < K; ++c) {
            int64_t lo, hi;
            host_pipe_transfer(ib, n0, c, &lo, &hi);
            planes[3 * c] = ib[c] * HOST_PIPE_ITEM_PLANES;
            planes[3 * c + 1] = (int)lo;
            planes[3 * c + 2] = (int)hi;
        }
    }
    return K;
}

// (g_pipe_mutex held)  The current device's state with at least `nevents` events in its pool.
static cudaError_t host_pipeline_state(int nevents, HostPipeState** out) {
    int dev = 0;
    cudaError_t ce = cudaGetDevice(&dev);
    if (ce != cudaSuccess) return ce;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    HostPipeState& st = g_pipe[dev];
    if (st.in == nullptr) {
        cudaStream_t a = nullptr, b = nullptr;
        ce = cudaStreamCreateWithFlags(&a, cudaStreamNonBlocking);
        if (ce != cudaSuccess) return ce;
        ce = cudaStreamCreateWithFlags(&b, cudaStreamNonBlocking);
        if (ce != cudaSuccess) { cudaStreamDestroy(a); return ce; }
        st.in = a; st.out = b;
    }
    while ((int)st.events.size() < nevents) {
        cudaEvent_t e = nullptr;
        ce = cudaEventCreateWithFlags(&e, cudaEventDisableTiming);
        if (ce != cudaSuccess) return ce;
        st.events.push_back(e);
    }
    *out = &st;
    return cudaSuccess;
}

// q: validated problem with device arrays set (in = fields, out unused); d_r / d_g device arrays
static int loss_grad_host_pipelined(Problem q, const float* const* h_fields, float* const* h_gfields, double* h_loss,
                                    float* const* d_f, float* const* d_r, float* const* d_g, double* d_loss,
                                    void* d_ws, int nf, int ne) {
    const int n0 = q.n[0], G = HOST_PIPE_ITEM_PLANES;
    const int64_t plane = (int64_t)q.n[1] * q.n[2] * q.n[3];
    const std::vector<int> ib = host_pipe_chunks(n0);
    const int K = (int)ib.size() - 1;
    std::lock_guard<std::mutex> lock(g_pipe_mutex);
    HostPipeState* hp = nullptr;
    if (host_pipeline_state(2 * K + 2, &hp) != cudaSuccess) { (void)cudaGetLastError(); return FPDE_ERR_CUDA; }
    cudaStream_t cs = q.stream, s_in = hp->in, s_out = hp->out;
    cudaEvent_t* ev = hp->events.data();
    cudaEvent_t* e_in = ev;                  // transfer c has landed
    cudaEvent_t* e_bwd = ev + K;             // gradients of chunk c are complete
    cudaEvent_t e_start = ev[2 * K], e_done = ev[2 * K + 1];
    bool ok = true;
    auto chk = [&](cudaError_t ce) { ok = ok && ce == cudaSuccess; };
    auto first = [&](int c) { return (int64_t)ib[c] * G; };                          // planes of chunk c: [first, end)
    auto end = [&](int c) { return std::min<int64_t>((int64_t)ib[c + 1] * G, n0); };

    // the copy streams start after whatever the caller queued before this call
    chk(cudaEventRecord(e_start, cs));
    chk(cudaStreamWaitEvent(s_in, e_start, 0));
    chk(cudaStreamWaitEvent(s_out, e_start, 0));
    // When the caller's arrays of a kind are evenly spaced in host memory (slices of one buffer), the
    // planes of all of them move in ONE strided copy per transfer instead of one copy per array: on a
    // link busy in both directions every copy costs about 10 us of dead time.
    auto even_stride = [&](const float* const* h, const float* const* d, ptrdiff_t* hs, ptrdiff_t* ds) {
        if (nf < 2) return false;
        const char* e = std::getenv("FPDE_HOST_STRIDED");
        if (e && e[0] == '0') return false;
        *hs = reinterpret_cast<const char*>(h[1]) - reinterpret_cast<const char*>(h[0]);
        *ds = reinterpret_cast<const char*>(d[1]) - reinterpret_cast<const char*>(d[0]);
        if (*hs <= 0 || *ds <= 0) return false;
        for (int f = 2; f < nf; ++f)
            if (reinterpret_cast<const char*>(h[f]) - reinterpret_cast<const char*>(h[f - 1]) != *hs ||
                reinterpret_cast<const char*>(d[f]) - reinterpret_cast<const char*>(d[f - 1]) != *ds)
                return false;
        const size_t arr_bytes = (size_t)plane * n0 * sizeof(float);
        if ((size_t)*hs < arr_bytes || (size_t)*ds < arr_bytes) return false;
        return one_allocation(h[0], reinterpret_cast<const char*>(h[nf - 1]) + arr_bytes) &&
               one_allocation(d[0], reinterpret_cast<const char*>(d[nf - 1]) + arr_bytes);
    };
    ptrdiff_t hs_in = 0, ds_in = 0, hs_out = 0, ds_out = 0;
    const bool strided_in = even_stride(h_fields, d_f, &hs_in, &ds_in);
    const bool strided_out = even_stride(h_gfields, d_g, &hs_out, &ds_out);
    auto up = [&](int64_t lo, int64_t hi) {
        if (hi <= lo) return;
        const size_t off = (size_t)(lo * plane), bytes = (size_t)((hi - lo) * plane) * sizeof(float);
        if (strided_in) {
            chk(cudaMemcpy2DAsync(d_f[0] + off, (size_t)ds_in, h_fields[0] + off, (size_t)hs_in, bytes, (size_t)nf,
                                  cudaMemcpyHostToDevice, s_in));
            return;
        }
        for (int f = 0; f < nf; ++f)
            chk(cudaMemcpyAsync(d_f[f] + off, h_fields[f] + off, bytes, cudaMemcpyHostToDevice, s_in));
    };
    // fields up: the wrap plane, then transfer c = planes up to and including the first of chunk c+1
    up(n0 - 1, n0);
    for (int c = 0; c < K; ++c) {
        int64_t lo, hi;
        host_pipe_transfer(ib, n0, c, &lo, &hi);
        up(lo, hi);
        chk(cudaEventRecord(e_in[c], s_in));
    }
    q.planes_per_item = G;
    q.partials = static_cast<float*>(d_ws);
    q.loss_out = d_loss;
    for (int f = 0; f < nf; ++f) q.in[f] = d_f[f];
    auto fwd = [&](int c) {
        chk(cudaStreamWaitEvent(cs, e_in[c], 0));
        Problem r = q;
        for (int e = 0; e < ne; ++e) r.out[e] = d_r[e];
        r.chunk_lo = ib[c]; r.chunk_hi = ib[c + 1];
        chk(launch_ns_fwd(r));
    };
    auto bwd = [&](int c) {
        Problem r = q;
        for (int e = 0; e < ne; ++e) { r.aux[e] = d_r[e]; r.gscale[e] = 2.0 / (double)q.rows; }
        for (int f = 0; f < nf; ++f) r.out[f] = d_g[f];
        r.partials = nullptr;
        r.chunk_lo = ib[c]; r.chunk_hi = ib[c + 1];
        chk(launch_ns_bwd(r));
        chk(cudaEventRecord(e_bwd[c], cs));
        chk(cudaStreamWaitEvent(s_out, e_bwd[c], 0));
        const size_t off = (size_t)(first(c) * plane), bytes = (size_t)((end(c) - first(c)) * plane) * sizeof(float);
        if (strided_out) {
            chk(cudaMemcpy2DAsync(h_gfields[0] + off, (size_t)hs_out, d_g[0] + off, (size_t)ds_out, bytes, (size_t)nf,
                                  cudaMemcpyDeviceToHost, s_out));
            return;
        }
        for (int f = 0; f < nf; ++f)
            chk(cudaMemcpyAsync(h_gfields[f] + off, d_g[f] + off, bytes, cudaMemcpyDeviceToHost, s_out));
    };
    // the adjoint of chunk c once the forward of c+1 is queued; the chunks next to the wrap
    // (the last one and chunk 0) need the last forward launch and come at the end
    fwd(0);
    fwd(1);
    for (int c = 2; c <= K - 1; ++c) {
        fwd(c);
        bwd(c - 1);
    }
    chk(launch_loss_finalize(q.partials, ns_items(q.n, false, G), ne, q.rows, d_loss, cs));
    bwd(K - 1);
    bwd(0);
    chk(cudaMemcpyAsync(h_loss, d_loss, (ne + 1) * sizeof(double), cudaMemcpyDeviceToHost, cs));
    // the caller's stream covers the copy streams
    chk(cudaEventRecord(e_done, s_out));
    chk(cudaStreamWaitEvent(cs, e_done, 0));
    return ok ? FPDE_OK : FPDE_ERR_CUDA;
}

int fpde_loss_grad_host(int op, const float* const* h_fields, const float* const* h_sources,
                        float* const* h_gfields, double* h_loss, int ndim, const int64_t* shape,
                        const double* spacing, const double* coeffs, int ncoeffs, const int* bc,
                        void* d_arena, size_t arena_bytes, void* stream) {
    int64_t N = 0, rows = 0;
    int st = check_shape(op, ndim, shape, nullptr, &N, &rows);
    if (st != FPDE_OK) return st;
    const OpEntry& e = REGISTRY[op];
    if (!h_fields || !h_gfields || !h_loss || (e.ns > 0 && !h_sources)) return FPDE_ERR_NULL;
    for (int f = 0; f < e.nf; ++f) if (!h_fields[f] || !h_gfields[f]) return FPDE_ERR_NULL;
    for (int s = 0; s < e.ns; ++s) if (!h_sources[s]) return FPDE_ERR_NULL;
    if (!d_arena || (reinterpret_cast<uintptr_t>(d_arena) & 255u) != 0 ||
        arena_bytes < fpde_host_arena_bytes(op, ndim, shape))
        return FPDE_ERR_WORKSPACE;
    // validate the remaining host arguments before the first copy is queued
    if (!spacing || !bc) return FPDE_ERR_NULL;
    if (ncoeffs != e.nc) return FPDE_ERR_COEFF_COUNT;
    if (e.nc > 0 && !coeffs) return FPDE_ERR_NULL;
    for (int a = 0; a < ndim; ++a) {
        if (!(spacing[a] > 0.0) || !std::isfinite(spacing[a])) return FPDE_ERR_SPACING;
        if (bc[a] != e.bc[a]) return FPDE_ERR_BC;
    }
    const size_t bytes = (size_t)N * sizeof(float), arr = round256(bytes);
    char* base = static_cast<char*>(d_arena);
    float* d_f[MAX_F]; float* d_s[MAX_F]; float* d_r[MAX_F]; float* d_g[MAX_F];
    for (int f = 0; f < e.nf; ++f) { d_f[f] = reinterpret_cast<float*>(base); base += arr; }
    for (int s = 0; s < e.ns; ++s) { d_s[s] = reinterpret_cast<float*>(base); base += arr; }
    for (int r = 0; r < e.ne; ++r) { d_r[r] = reinterpret_cast<float*>(base); base += arr; }
    for (int f = 0; f < e.nf; ++f) { d_g[f] = reinterpret_cast<float*>(base); base += arr; }
    double* d_loss = reinterpret_cast<double*>(base); base += round256((e.ne + 1) * sizeof(double));
    void* d_ws = base;
    const size_t ws_bytes = host_workspace_bytes(op, ndim, shape);
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    {
        int n[MAX_D] = {0, 0, 0, 0};
        check_shape(op, ndim, shape, n, nullptr, nullptr);
        if (host_pipeline_wanted(op, n)) {
            Problem q;
            std::memset(&q, 0, sizeof(q));
            st = validate(op, d_f, ndim, shape, spacing, coeffs, ncoeffs, bc, q);
            if (st != FPDE_OK) return st;
            q.stream = cs;
            return loss_grad_host_pipelined(q, h_fields, h_gfields, h_loss, d_f, d_r, d_g, d_loss, d_ws, e.nf, e.ne);
        }
    }
    for (int f = 0; f < e.nf; ++f)
        if (cudaMemcpyAsync(d_f[f], h_fields[f], bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess) return FPDE_ERR_CUDA;
    for (int s = 0; s < e.ns; ++s)
        if (cudaMemcpyAsync(d_s[s], h_sources[s], bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess) return FPDE_ERR_CUDA;
    // one kernel where the operator has a single-pass kernel (the staged residual arrays are
    // then not written), forward + adjoint through them otherwise
    st = fpde_fwd_bwd(op, d_f, d_s, fused2d_supported(op) ? nullptr : d_r, d_g, d_loss, ndim, shape, spacing, coeffs,
                      ncoeffs, bc, d_ws, ws_bytes, stream);
    if (st != FPDE_OK) return st;
    for (int f = 0; f < e.nf; ++f)
        if (cudaMemcpyAsync(h_gfields[f], d_g[f], bytes, cudaMemcpyDeviceToHost, cs) != cudaSuccess) return FPDE_ERR_CUDA;
    if (cudaMemcpyAsync(h_loss, d_loss, (e.ne + 1) * sizeof(double), cudaMemcpyDeviceToHost, cs) != cudaSuccess)
        return FPDE_ERR_CUDA;
    return FPDE_OK;
}

// ------------------------------------------------------------------------------------------
// fpde_fwd_noalloc: the forward pass with its scratch in a fixed array of the library image.
// In host code the array's name is only a handle; the device address comes from
// cudaGetSymbolAddress, looked up once per device with that device current.
// ------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_noalloc_scratch[FPDE_NOALLOC_SCRATCH_BYTES];

static constexpr int NOALLOC_MAX_DEVICES = 64;
static std::mutex g_noalloc_mutex;
static void* g_noalloc_addr[NOALLOC_MAX_DEVICES];      // per device, filled on first use

static cudaError_t noalloc_scratch_address(void** out) {
    int dev = -1;
    cudaError_t ce = cudaGetDevice(&dev);
    if (ce != cudaSuccess) return ce;
    if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (g_noalloc_addr[dev] == nullptr) {
        void* addr = nullptr;
        ce = cudaGetSymbolAddress(&addr, g_noalloc_scratch);
        if (ce != cudaSuccess) return ce;
        g_noalloc_addr[dev] = addr;
    }
    *out = g_noalloc_addr[dev];
    return cudaSuccess;
}

int fpde_fwd_noalloc(int op, const float* const* fields, const float* const* sources, float* const* residuals,
                     double* loss_out, int ndim, const int64_t* shape, const double* spacing,
                     const double* coeffs, int ncoeffs, const int* bc, void* stream) {
    // refuse grids beyond the fixed scratch before touching the device
    const size_t need = fpde_workspace_bytes(op, ndim, shape);
    if (need == 0) {                       // invalid op / shape: let the common validation name the error
        return fpde_fwd(op, fields, sources, residuals, nullptr, ndim, shape, spacing, coeffs, ncoeffs, bc,
                        nullptr, 0, stream);
    }
    if (loss_out != nullptr && need > FPDE_NOALLOC_SCRATCH_BYTES) return FPDE_ERR_WORKSPACE;
    void* scratch = nullptr;
    if (loss_out != nullptr) {
        if (noalloc_scratch_address(&scratch) != cudaSuccess) return FPDE_ERR_CUDA;
    }
    return fpde_fwd(op, fields, sources, residuals, loss_out, ndim, shape, spacing, coeffs, ncoeffs, bc,
                    scratch, scratch ? (size_t)FPDE_NOALLOC_SCRATCH_BYTES : 0, stream);
}

unsigned int fpde_diag_tma_timeouts(void) {
    const unsigned int a = ns_tma_timeouts(), b = star3d_tma_timeouts(), c = star3d_fused_timeouts();
    return (a == ~0u || b == ~0u || c == ~0u) ? ~0u : a + b + c;
}

int fpde_diag_ns_tma_geometry(const int64_t* shape, int tile_rows, int narrays, size_t smem_limit) {
    if (!shape) return 0;
    int n[MAX_D];
    for (int a = 0; a < 4; ++a) {
        if (shape[a] < 1 || shape[a] > (int64_t)1 << 30) return 0;
        n[a] = (int)shape[a];
    }
    return ns_tma_geometry_ok(n, tile_rows, narrays, smem_limit) ? 1 : 0;
}

}  // extern "C"
