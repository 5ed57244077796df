/*
 * fpde.h -- C ABI of the fused finite-difference PDE-residual operator library (libfpde.so).
 *
 * The library evaluates, on a regular Cartesian (space or space-time) grid, the discrete PDE
 * residuals of grid-aligned physical fields in one fused forward pass, and maps the upstream
 * sensitivities dL/dres back to dL/dfield with a hand-derived discrete adjoint in gather form.
 * It is the method of the paper's Section 2 ("Kernel design and discrete analytic adjoints"):
 * fused forward stencil (Section 2.1), analytic discrete-adjoint backward (Section 2.2,
 * Eq. 1, Appendix A.3) and boundary-gradient correction (Section 2.3, Appendix A.5).
 *
 * General rules (all entry points)
 *   - Plain C types only.  Nothing throws or aborts; every call returns an fpde_status.
 *   - Arrays are fp32, row-major, axis 0 slowest, last axis contiguous, all of the FULL grid
 *     shape.  Space-time grids keep t as the last (contiguous) axis.
 *   - "device" pointers are CUDA device memory owned by the caller, 16-byte aligned, not
 *     overlapping; "host" pointers are ordinary host memory read during the call only.
 *   - The library allocates no device memory.  The kernel entry points keep no state between
 *     calls.  Two entry points keep a little per device, created on first use and held until the
 *     process exits: fpde_loss_grad_host (two copy streams and a pool of events for its pipelined
 *     form) and fpde_fwd_noalloc (the address of its fixed scratch array).  Work is queued on
 *     `stream` (a cudaStream_t passed as void*; NULL = the legacy default stream) and the call
 *     returns without waiting for it.
 *   - On any status other than FPDE_OK nothing has been launched.  FPDE_ERR_CUDA reports a
 *     launch the CUDA runtime rejected.
 *   - With no CUDA device the entry points still load and validate, and a launch attempt
 *     returns FPDE_ERR_CUDA: there is no CPU fallback.
 */
#ifndef FPDE_H
#define FPDE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FPDE_OK = 0,
    FPDE_ERR_BAD_OP = 1,       /* operator id out of range                                   */
    FPDE_ERR_NULL = 2,         /* a required pointer (or array entry) is NULL                */
    FPDE_ERR_NDIM = 3,         /* ndim does not match the operator                           */
    FPDE_ERR_SHAPE = 4,        /* an extent is too small, too large, or breaks the x4 rule   */
    FPDE_ERR_ALIGN = 5,        /* a device pointer is not 16-byte aligned                    */
    FPDE_ERR_SPACING = 6,      /* a spacing is not finite and positive                       */
    FPDE_ERR_COEFF_COUNT = 7,  /* ncoeffs does not match the operator                        */
    FPDE_ERR_BC = 8,           /* boundary kinds not supported by the operator               */
    FPDE_ERR_WORKSPACE = 9,    /* workspace NULL, misaligned or smaller than required        */
    FPDE_ERR_CUDA = 10         /* the CUDA runtime reported an error                         */
} fpde_status;

/*
 * Operators.  Fields (differentiated inputs), sources (read-only inputs without gradient),
 * residuals and coefficients, in the order the arrays are passed:
 *
 *  FPDE_OP_BURGERS_1D_T     (x,t) array.  fields [u]; residuals [r]; coeffs [nu].
 *        r = D_t u + u D_x u - nu D_xx u at every node; centred second-order differences
 *        inside, second-order one-sided differences on the first/last node of each axis.
 *        bc = (ONE_SIDED, ONE_SIDED).
 *  FPDE_OP_POISSON_2D       (x,y) array.  fields [u]; sources [f]; residuals [r]; no coeffs.
 *        r = -(d_xx u + d_yy u) - f, five-point Laplacian, rows where it fits.
 *        bc = (INTERIOR, INTERIOR).
 *  FPDE_OP_GRAYSCOTT_2D     (x,y) array.  fields [u,v]; residuals [r_u,r_v];
 *        coeffs [D_u, D_v, F, k].  r_u = D_u Lap u - u v^2 + F (1-u),
 *        r_v = D_v Lap v + u v^2 - (F+k) v.  bc = (PERIODIC, PERIODIC).
 *  FPDE_OP_HELMHOLTZ_3D_O4  (x,y,z) array.  fields [u]; sources [f]; residuals [r];
 *        coeffs [k] (wavenumber).  r = Lap4 u + k^2 u - f with the fourth-order 13-point
 *        Laplacian (-1,16,-30,16,-1)/(12 h^2) per axis.  bc = (INTERIOR x3): rows at indices
 *        2..n-3; the two outer layers are data and receive gradient.
 *  FPDE_OP_NS_3D_T          (x,y,z,t) array.  fields [u,v,w,p];
 *        residuals [mom_x, mom_y, mom_z, continuity]; coeffs [nu].
 *        mom_q = d_t q + u d_x q + v d_y q + w d_z q + d_{a_q} p - nu Lap q, continuity =
 *        d_x u + d_y v + d_z w (Section 2.1's residuals extended by t, w and z), centred
 *        differences.  bc = (PERIODIC x3, INTERIOR): rows at t-index 1..n_t-2.
 *  FPDE_OP_NS_2D_STEADY    (x,y) array.  fields [u,v,p]; residuals [res_u, res_v, res_div];
 *        coeffs [nu].  The paper's worked operator (Section 2.1):
 *        res_u = u u_x + v u_y + p_x - nu Lap u, res_v = u v_x + v v_y + p_y - nu Lap v,
 *        res_div = u_x + v_y, centred differences; its adjoint is Eq. 1 (and the analogous
 *        expressions for v and p).  bc = (INTERIOR, INTERIOR): rows at the interior nodes, the
 *        outer ring is data and receives gradient.
 *  FPDE_OP_NS_3D_STEADY    (x,y,z) array.  fields [u,v,w,p];
 *        residuals [mom_x, mom_y, mom_z, continuity]; coeffs [nu].  Section 2.1's system with
 *        the third component: mom_q = u d_x q + v d_y q + w d_z q + d_{a_q} p - nu Lap q,
 *        continuity = d_x u + d_y v + d_z w, centred differences.  bc = (INTERIOR x3): rows at
 *        the interior nodes, the outer shell is data and receives gradient.
 *  FPDE_OP_NS_3D_T_XSLAB   FPDE_OP_NS_3D_T with a non-periodic x axis, bc = (INTERIOR, PERIODIC,
 *        PERIODIC, INTERIOR): rows at x-index 1..n_x-2 (and t-index 1..n_t-2), the first and last
 *        x-plane are data.  This is the form one slab of a grid split along x takes: its outer
 *        planes are copies of the neighbouring slabs' planes, and on the planes that carry rows
 *        the residuals are those of the periodic operator on the whole grid.
 *  FPDE_OP_GRAYSCOTT_2D_XSLAB  the same for FPDE_OP_GRAYSCOTT_2D, bc = (INTERIOR, PERIODIC): rows
 *        at x-index 1..n_x-2, the first and last row of the array are data.
 *
 * Shape rules: the contiguous extent must be a multiple of 4 (float4 path) except for
 * BURGERS_1D_T; PERIODIC / INTERIOR axes need n >= 2*radius+1, ONE_SIDED axes n >= 4; the
 * total number of nodes must stay below 2^31.
 */
typedef enum {
    FPDE_OP_BURGERS_1D_T = 0,
    FPDE_OP_POISSON_2D = 1,
    FPDE_OP_GRAYSCOTT_2D = 2,
    FPDE_OP_HELMHOLTZ_3D_O4 = 3,
    FPDE_OP_NS_3D_T = 4,
    FPDE_OP_NS_2D_STEADY = 5,
    FPDE_OP_NS_3D_STEADY = 6,
    FPDE_OP_NS_3D_T_XSLAB = 7,
    FPDE_OP_GRAYSCOTT_2D_XSLAB = 8,
    FPDE_OP_COUNT = 9
} fpde_op;

/* Boundary kind of one array axis (Appendix A.5 names the three causes of boundary terms:
 * prescribed values, one-sided formulas, omitted neighbours). */
typedef enum {
    FPDE_BC_PERIODIC = 0,   /* rows at every node, wrap-around neighbours                       */
    FPDE_BC_INTERIOR = 1,   /* rows only where the full stencil fits; the outer `radius` layers */
                            /* are ordinary input data (e.g. Dirichlet values) and do receive   */
                            /* gradient from the rows that read them                            */
    FPDE_BC_ONE_SIDED = 2   /* rows at every node, second-order one-sided formulas at the edges */
} fpde_bc;

typedef struct {
    int ndim, nfields, nsources, nresiduals, ncoeffs, radius;
    int bc[4];              /* the boundary kinds the operator accepts, per axis */
} fpde_op_info_t;

/* Describe an operator (host only).  FPDE_ERR_BAD_OP / FPDE_ERR_NULL on bad arguments. */
int fpde_op_info(int op, fpde_op_info_t* out);

/* Static, never-NULL description of a status code. */
const char* fpde_strerror(int status);

/* Number of nodes that carry a residual row (N_r, the divisor of each mean square); 0 if the
 * operator / shape is invalid.  Host only. */
int64_t fpde_row_count(int op, int ndim, const int64_t* shape);

/* Bytes of device scratch fpde_fwd needs for this operator and grid (loss partial sums); 0 if
 * the operator / shape is invalid.  fpde_bwd needs none.  Host only.
 * The figure follows the launch shape, which the FPDE_* tuning variables of the environment can
 * change (they are read on every call): size the workspace after setting them, not before.  A call
 * whose workspace has become too small is refused with FPDE_ERR_WORKSPACE, never run short. */
size_t fpde_workspace_bytes(int op, int ndim, const int64_t* shape);

/*
 * Fused forward residual + loss (Section 2.1; loss = mean square residual, summed over the
 * residual fields, which the paper evaluates outside its operator and this library fuses).
 *
 *   fields     host array of nfields   device pointers, read only
 *   sources    host array of nsources  device pointers, read only (may be NULL if nsources = 0)
 *   residuals  host array of nresiduals device pointers, overwritten: r_e at every node that
 *              carries a row, exactly 0.0f elsewhere
 *   loss_out   device, nresiduals+1 doubles, overwritten with L_0..L_{E-1} and their sum, where
 *              L_e = (1/N_r) sum over rows r_e^2.  The sum is taken in a fixed order: repeated
 *              calls give bit-identical results.  NULL skips the loss (workspace unused).
 *   ndim, shape, spacing, coeffs, ncoeffs, bc   host; see the operator list
 *   workspace  device scratch of at least fpde_workspace_bytes() bytes, contents arbitrary
 *              before and after; calls sharing a workspace must not overlap on the GPU
 *   stream     cudaStream_t
 */
int fpde_fwd(int op,
             const float* const* fields,
             const float* const* sources,
             float* const* residuals,
             double* loss_out,
             int ndim, const int64_t* shape,
             const double* spacing,
             const double* coeffs, int ncoeffs,
             const int* bc,
             void* workspace, size_t workspace_bytes,
             void* stream);

/*
 * fpde_fwd whose loss divides by a row count the caller names instead of this array's own:
 *   L_e = (1 / loss_rows) sum over the rows of THIS array of r_e^2.
 * For a grid split into slabs (Section 2.1's residual rows are independent, so a grid splits into
 * slabs of planes that only share halo planes): every rank passes the row count of the WHOLE grid,
 * and the sum of the ranks' loss vectors is the loss of the whole grid, so the ranks all-reduce the
 * vector itself.  loss_rows < 1 is FPDE_ERR_SHAPE; everything else as fpde_fwd.
 */
int fpde_fwd_rows(int op,
                  const float* const* fields,
                  const float* const* sources,
                  float* const* residuals,
                  double* loss_out,
                  int ndim, const int64_t* shape,
                  const double* spacing,
                  const double* coeffs, int ncoeffs,
                  const int* bc,
                  void* workspace, size_t workspace_bytes,
                  void* stream,
                  int64_t loss_rows);

/*
 * Launches over a range of x-planes, for overlapping the halo exchange of a grid split into slabs
 * with the work that does not read the halo planes (Sections 2.1 and 2.2: rows are independent, so
 * a launch may cover any subset of them).  Only FPDE_OP_NS_3D_T and FPDE_OP_NS_3D_T_XSLAB have
 * them (FPDE_ERR_BAD_OP otherwise).
 *
 *   fpde_plane_chunk   planes per chunk for this operator and grid (0 = no ranged launches);
 *                      chunk c covers planes [c * chunk, min((c + 1) * chunk, n_x)).  Host only.
 *   fpde_fwd_chunks    fpde_fwd_rows restricted to the chunks [chunk_lo, chunk_hi): residuals are
 *                      written on those planes only, their loss partial sums go to their own slots
 *                      of the workspace.  `finish` != 0: the loss vector is formed from the partial
 *                      sums of ALL chunks, so this must be the last of a set of calls that share
 *                      workspace and stream and together cover every chunk.  loss_rows = 0: the
 *                      array's own row count.
 *   fpde_bwd_chunks    fpde_bwd restricted to the chunks [chunk_lo, chunk_hi): gradients are written
 *                      on those planes only (they read the upstream arrays and fields one plane
 *                      beyond the range at either end).
 * FPDE_ERR_SHAPE for an empty or out-of-range chunk range.
 */
int fpde_plane_chunk(int op, int ndim, const int64_t* shape);
int fpde_fwd_chunks(int op,
                    const float* const* fields,
                    const float* const* sources,
                    float* const* residuals,
                    double* loss_out,
                    int ndim, const int64_t* shape,
                    const double* spacing,
                    const double* coeffs, int ncoeffs,
                    const int* bc,
                    void* workspace, size_t workspace_bytes,
                    void* stream,
                    int64_t loss_rows,
                    int chunk_lo, int chunk_hi, int finish);
int fpde_bwd_chunks(int op,
                    const float* const* fields,
                    const float* const* gres,
                    const double* gscale,
                    float* const* gfields,
                    int ndim, const int64_t* shape,
                    const double* spacing,
                    const double* coeffs, int ncoeffs,
                    const int* bc,
                    void* stream,
                    int chunk_lo, int chunk_hi);

/*
 * Discrete adjoint in gather form with boundary-gradient correction (Sections 2.2 and 2.3):
 * gfields[f] = sum_e J_{e,f}^T G_e with G_e = gscale[e] * gres[e] on the rows of residual e
 * and 0 elsewhere (entries of gres at nodes without a row are ignored).
 *
 *   fields     as in fpde_fwd (the Jacobian of a nonlinear operator depends on them)
 *   gres       host array of nresiduals device pointers: upstream dL/dr_e, read only.  Passing
 *              the residual arrays fpde_fwd wrote, with gscale[e] = 2/N_r, yields the gradient
 *              of the fused loss.
 *   gscale     host, nresiduals doubles; NULL means all 1
 *   gfields    host array of nfields device pointers, OVERWRITTEN (not accumulated) at every
 *              node, boundary layers included
 *   workspace  unused by the current kernels; may be NULL with workspace_bytes = 0
 * No atomics are used: every output element is written by exactly one thread.
 *
 * Accuracy limit of the Navier-Stokes adjoints (FPDE_OP_NS_3D_T, FPDE_OP_NS_3D_STEADY and the
 * slab form): their transposed advection and diffusion terms are evaluated as one weighted sum
 * over the six neighbours of an upstream array, whose fp32 rounding error is relative to
 * sum |w_i G_i| and therefore grows with nu / h^2 when the upstream array is smooth.  Measured
 * against the fp64 oracle on noise-free fields: gradient relative L2 error 2e-7 at
 * nu * max_a(1 / h_a^2) = 4, 5e-6 at 1000.  Keep nu * max_a(1 / h_a^2) at or below 1000 for
 * the 1e-5 tolerance this library is tested to; beyond it use fpde_bwd_f64.  The forward
 * kernels difference first and have no such limit.
 */
int fpde_bwd(int op,
             const float* const* fields,
             const float* const* gres,
             const double* gscale,
             float* const* gfields,
             int ndim, const int64_t* shape,
             const double* spacing,
             const double* coeffs, int ncoeffs,
             const int* bc,
             void* workspace, size_t workspace_bytes,
             void* stream);

/*
 * Loss-specialised single pass: residuals (Section 2.1), the mean-square loss and its gradient
 * through the discrete adjoint (Sections 2.2, 2.3) from one call,
 *   L = sum_e L_e,  L_e = (1/N_r) sum over rows r_e^2,   gfields[f] = dL/dfield_f
 * i.e. what fpde_fwd followed by fpde_bwd with gres = residuals, gscale[e] = 2/N_r computes.
 * Where fpde_has_single_pass(op) is 1 this is ONE kernel in which the residuals stay in
 * registers between the forward stencil and the adjoint (the upstream array of the adjoint is
 * (2/N_r) r, so nothing else of the forward pass is needed): it reads the fields and sources
 * and writes the gradients, and the residual arrays only if asked for.  For the other
 * operators it queues the forward kernel, the loss sum and the adjoint kernel.
 *
 *   fields, sources, ndim ... bc, stream   as in fpde_fwd
 *   residuals  host array of nresiduals device pointers, or NULL.  Single-pass operators: a
 *              NULL array or NULL entries mean "do not store that residual"; a non-NULL entry
 *              is overwritten as by fpde_fwd.  Other operators: every entry is required
 *              (FPDE_ERR_NULL otherwise), the arrays serve as the intermediate.
 *   gfields    host array of nfields device pointers, overwritten at every node
 *   loss_out   device, nresiduals+1 doubles (as in fpde_fwd), or NULL to skip the loss
 *   workspace  device scratch of at least fpde_fwd_bwd_workspace_bytes() bytes (needed only
 *              when loss_out is given)
 * Same status codes as fpde_fwd / fpde_bwd.
 */
int fpde_has_single_pass(int op);
size_t fpde_fwd_bwd_workspace_bytes(int op, int ndim, const int64_t* shape);
int fpde_fwd_bwd(int op,
                 const float* const* fields,
                 const float* const* sources,
                 float* const* residuals,
                 float* const* gfields,
                 double* loss_out,
                 int ndim, const int64_t* shape,
                 const double* spacing,
                 const double* coeffs, int ncoeffs,
                 const int* bc,
                 void* workspace, size_t workspace_bytes,
                 void* stream);

/*
 * Double-precision verification path (the paper trains and times in fp32 and uses fp64 only to
 * verify its hand-derived adjoints): fpde_fwd / fpde_bwd with every array in double, computed by
 * separate one-thread-per-node kernels written for clarity, not speed.  Same operators, shapes,
 * boundary kinds, status codes and semantics (rows, zero at nodes without a row, loss in a fixed
 * order, gradients overwritten at every node) as the fp32 entry points; pointers are device
 * pointers to doubles, 16-byte aligned.  fpde_workspace_bytes_f64 gives the scratch fpde_fwd_f64
 * needs when loss_out is given; fpde_bwd_f64 needs none.
 */
size_t fpde_workspace_bytes_f64(int op, int ndim, const int64_t* shape);
int fpde_fwd_f64(int op,
                 const double* const* fields,
                 const double* const* sources,
                 double* const* residuals,
                 double* loss_out,
                 int ndim, const int64_t* shape,
                 const double* spacing,
                 const double* coeffs, int ncoeffs,
                 const int* bc,
                 void* workspace, size_t workspace_bytes,
                 void* stream);
int fpde_bwd_f64(int op,
                 const double* const* fields,
                 const double* const* gres,
                 const double* gscale,
                 double* const* gfields,
                 int ndim, const int64_t* shape,
                 const double* spacing,
                 const double* coeffs, int ncoeffs,
                 const int* bc,
                 void* stream);

/*
 * Loss gradient from HOST buffers in one call: copies the fields (and sources) to the device,
 * runs fpde_fwd_bwd, i.e. the adjoint with the upstream sensitivities of the mean-square loss,
 * G_e = (2/N_r) r_e (Section 2.2: the operator receives G = dL/dres from the loss), and copies
 * dL/dfield and the loss vector back.  Everything is queued on `stream`; the host buffers may be
 * read / written until the stream has been synchronised (use page-locked memory for the copies to
 * run asynchronously).
 *
 *   h_fields   host array of nfields  HOST pointers, N floats each, read only
 *   h_sources  host array of nsources HOST pointers (may be NULL if nsources = 0)
 *   h_gfields  host array of nfields  HOST pointers, N floats each, overwritten with dL/dfield
 *   h_loss     HOST, nresiduals+1 doubles, overwritten with L_0..L_{E-1} and their sum
 *   d_arena    DEVICE scratch of at least fpde_host_arena_bytes() bytes, 256-byte aligned, owned
 *              by the caller (staging for fields, sources, residuals, gradients, loss, workspace)
 * Same status codes as fpde_fwd / fpde_bwd; FPDE_ERR_WORKSPACE if the arena is too small.
 * For FPDE_OP_NS_3D_T on grids that split into six or more chunks of x-planes (29 planes and up)
 * the call is pipelined: the fields are copied up on one internal stream in transfers that run one
 * plane ahead of the chunks, run through forward and adjoint launches over the chunks' work items
 * on `stream`, and the gradients are copied down on a second internal stream, so the two copy
 * directions overlap; `stream` waits for both internal streams before the call's work counts as
 * done on it, so synchronising `stream` is still all a caller has to do.  (FPDE_HOST_PIPELINE=0
 * in the environment selects the plain one-stream form.)  If the host arrays of a kind are slices
 * of ONE page-locked allocation at even spacing (e.g. h_fields[k] = base + k * stride), a range of
 * planes of all of them moves in one strided copy instead of one copy per array, which is worth
 * about 5 % of the step on a link busy in both directions; any other layout works as before.
 */
size_t fpde_host_arena_bytes(int op, int ndim, const int64_t* shape);

/*
 * The plan the pipelined form of fpde_loss_grad_host follows for a grid of n0 x-planes (host-only
 * query, no device needed).  Returns the number of chunks K, or 0 if such a grid takes the plain
 * form.  If `planes` is not NULL it receives 3 ints per chunk c (cap = number of chunks it has room
 * for; nothing is written and -K is returned if cap < K):
 *   planes[3c]   first x-plane of chunk c (the chunk ends where the next one starts, the last at n0)
 *   planes[3c+1] first x-plane of upload transfer c
 *   planes[3c+2] one past the last x-plane of upload transfer c (an empty transfer has both equal)
 * Plane n0-1 is uploaded before transfer 0.  The forward launch of chunk c follows transfer c; the
 * adjoint launch of chunk c follows the forward launch of chunk c+1 (chunks K-1 and 0: the last one).
 */
int fpde_host_pipeline_plan(int n0, int* planes, int cap);
int fpde_loss_grad_host(int op,
                        const float* const* h_fields,
                        const float* const* h_sources,
                        float* const* h_gfields,
                        double* h_loss,
                        int ndim, const int64_t* shape,
                        const double* spacing,
                        const double* coeffs, int ncoeffs,
                        const int* bc,
                        void* d_arena, size_t arena_bytes,
                        void* stream);

/*
 * fpde_fwd for callers that cannot allocate device memory.  (The paper has no counterpart; this
 * is a convenience of this library.)
 *
 * Who needs it: code that runs where a device allocation is forbidden or impossible -- inside a
 * region that must not synchronise the device (cudaMalloc does), in a plug-in that is handed
 * tensors but no allocator, or late in a job whose memory pool is already fully committed.  Such
 * callers can supply inputs and outputs but no workspace.
 *
 * Same arguments and results as fpde_fwd, without `workspace`: the loss partial sums go to a
 * fixed array that is part of the library image (FPDE_NOALLOC_SCRATCH_BYTES bytes of device
 * memory on every GPU that loads the library, held until the process exits).  The call makes no
 * cudaMalloc / cudaFree and calls no allocating routine.
 *
 *   - Grids whose forward pass needs more scratch than that (fpde_workspace_bytes() >
 *     FPDE_NOALLOC_SCRATCH_BYTES) are refused with FPDE_ERR_WORKSPACE; nothing is launched.  The
 *     need follows the launch shape, so a tuning variable that shortens the work items can turn
 *     an accepted grid into a refused one.
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  Make that first call outside any stream capture.
 *   - Every call on a device shares the one array.  The kernels overwrite every slot they later
 *     read, so nothing has to be cleared between calls, but two calls that overlap on the GPU
 *     (different streams, no ordering) race on it: order them, or use fpde_fwd with separate
 *     workspaces.
 */
#define FPDE_NOALLOC_SCRATCH_BYTES (256u * 1024u)
int fpde_fwd_noalloc(int op,
                     const float* const* fields,
                     const float* const* sources,
                     float* const* residuals,
                     double* loss_out,
                     int ndim, const int64_t* shape,
                     const double* spacing,
                     const double* coeffs, int ncoeffs,
                     const int* bc,
                     void* stream);

/*
 * Diagnostic.  The Navier-Stokes kernels that stage their tiles through shared memory with the
 * copy engine wait on memory barriers with an iteration limit instead of spinning for ever; this
 * returns how many such waits have given up on the current device since the library was loaded
 * (0 in a healthy run; results of a launch that timed out are garbage).  Synchronises the device.
 * Returns UINT_MAX if the counter cannot be read.
 */
unsigned int fpde_diag_tma_timeouts(void);

/*
 * Diagnostic, host only.  1 if the shared-memory-staged Navier-Stokes kernels (an opt-in variant,
 * FPDE_NS_TMA=1) can take an (x,y,z,t) grid of this shape with tiles of `tile_rows` rows (4 or 8)
 * and `narrays` arrays per pipeline stage (4 forward, 7 adjoint) inside `smem_limit` bytes of
 * dynamic shared memory; 0 otherwise, in which case fpde_fwd / fpde_bwd run the default kernels.
 * The rule includes the copy engine's requirement that every destination in shared memory starts
 * on a 128-byte boundary.
 */
int fpde_diag_ns_tma_geometry(const int64_t* shape, int tile_rows, int narrays, size_t smem_limit);

#ifdef __cplusplus
}
#endif
#endif /* FPDE_H */
