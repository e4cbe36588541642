/*
 * dn -- physics loss of a data-free generative PDE solver, as CUDA kernels for sm_100a.
 *
 * The paper trains a generator of full solution fields without data: the loss scores
 * a batch of generated fields against the PDE  A_nu(u) = f,  B(u) = b  on the unit
 * domain ("Mathematical preliminaries", Eq. (pde)), as an expectation over sampled
 * coefficients nu and boundary data b ("DiffNets", Eq. (pde_loss)), and the gradient
 * of that loss with respect to the field is what enters back-propagation
 * (Algorithm 1, local back-propagation step).  This library evaluates that loss for
 * the diffusion equation
 *
 *        -div( nu grad u ) = f   on [0,1]^d, d = 2 or 3,
 *        u = bc_x0 on x = 0,  u = bc_x1 on x = 1,  zero flux on the other faces,
 *
 * in its variational (Ritz/Galerkin) form on a uniform mesh of bilinear / trilinear
 * (Q1) elements with 2-point-per-axis Gauss quadrature:
 *
 *        J(u)  = sum_e sum_q W_q ( 1/2 nu_q |grad u_q|^2 - f_q u_q )          (energy)
 *        r     = dJ/du = K(nu) u - F,  set to 0 at the Dirichlet nodes         (residual)
 *
 * Conventions shared by all entry points
 *  - Fields are C-ordered [batch][nz][ny][nx] float32 (x fastest; nz = 1 in 2D).  Node
 *    (ix,iy,iz) sits at (ix*hx, iy*hy, iz*hz), h_a = 1/(n_a - 1).  Dirichlet nodes are
 *    those with ix == 0 or ix == nx-1.
 *  - Every pointer is a DEVICE pointer unless its name ends in _host; structs are read
 *    on the host.  The caller owns every buffer.  The library allocates no memory,
 *    keeps no state between calls that could change a result, and never synchronises.
 *    What it does keep: the *_host entry points return after their last copy has finished
 *    (also when they fail half-way); dn_energy_grad_static remembers, per device, the
 *    address of its built-in scratch array (looked up on the first call on that device; it
 *    goes stale if the device is reset); and every host thread remembers the launch geometry
 *    of the last problem shape it saw per kernel family (a pure function of the shape, the
 *    mode and the SM count, searched once instead of on every call).
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Work is
 *    enqueued on it in order; outputs are valid once that work has finished.
 *  - Return value: DN_OK or an error code; nothing is thrown, nothing aborts.  When
 *    validation fails nothing has been enqueued and no output is touched.
 *  - Results are deterministic: no atomics, fixed reduction order.
 */
#ifndef DN_H_
#define DN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DN_OK = 0,
    DN_ERR_NULL = 1,       /* a required pointer is NULL                                   */
    DN_ERR_DIM = 2,        /* dim is not 2 or 3                                            */
    DN_ERR_SIZE = 3,       /* a grid extent < 2, batch < 1, or an extent beyond the limits */
    DN_ERR_MODE = 4,       /* unknown nu_mode / bc mode, kl_modes outside 1..DN_MAX_KL_MODES */
    DN_ERR_WORKSPACE = 5,  /* workspace NULL, misaligned (256 B) or smaller than required  */
    DN_ERR_CUDA = 6,       /* a CUDA runtime call or kernel launch failed                  */
    DN_ERR_ALIAS = 7       /* r overlaps u                                                 */
} dn_status;

typedef enum {
    DN_NU_NODAL = 0,       /* nu given at the nodes, Q1-interpolated to the Gauss points    */
    DN_NU_KL_GAUSS = 1,    /* nu evaluated from the KL weights at the Gauss points; no field stored */
    DN_NU_KL_NODAL = 2     /* nu evaluated from the KL weights at the nodes inside the kernel, then Q1-interpolated
                              (the numbers of dn_kl_field + DN_NU_NODAL, without storing the field)          */
} dn_nu_mode;

/* dn_problem.flags */
#define DN_IMPOSE_BC_ON_LOAD 1u  /* read u as if its x faces held bc_x0 / bc_x1 (u itself is not written) */
#define DN_NO_MASK           2u  /* keep the raw residual at Dirichlet nodes (tests)                      */
#define DN_FORCE_GENERIC     4u  /* use the any-size kernels even where a tiled kernel applies (tests)    */

#define DN_MAX_KL_MODES 8        /* largest m (KL modes per axis)                                         */
#define DN_MAX_EXTENT 32768      /* largest nx, ny or nz                                                  */
#define DN_STATIC_SCRATCH_BYTES (1u << 20)  /* scratch built into the library for dn_energy_grad_static   */

typedef struct {
    int32_t dim;                 /* 2 or 3                                 */
    int32_t nx, ny, nz;          /* nodes per axis; nz is ignored when dim == 2 */
} dn_grid;

/* Statement of one batched problem: grid size, batch, diffusivity (KL coefficients or a
 * nodal field), boundary values and forcing. */
typedef struct {
    dn_grid grid;
    int32_t batch;               /* B >= 1                                                         */
    int32_t nu_mode;             /* dn_nu_mode                                                     */
    const float* nu;             /* [B][nz][ny][nx], used when nu_mode == DN_NU_NODAL              */
    int32_t kl_modes;            /* m, used when nu_mode is DN_NU_KL_GAUSS or DN_NU_KL_NODAL       */
    const float* kl_w;           /* [B][m]^dim, index [b][i-1][j-1]([k-1]); i <-> x, j <-> y, k <-> z */
    float f_const;               /* forcing when f == NULL                                         */
    const float* f;              /* optional nodal forcing [B][nz][ny][nx], Q1-interpolated        */
    float bc_x0, bc_x1;          /* Dirichlet values on x = 0 and x = 1                            */
    uint32_t flags;              /* DN_* flags above                                               */
    const float* bc_x0_b;        /* optional [B]: per-sample Dirichlet value on x = 0 (the paper samples the  */
    const float* bc_x1_b;        /* boundary data b per minibatch); each overrides its scalar when non-NULL   */
} dn_problem;

/* Bytes of device scratch that dn_energy / dn_energy_grad need for this problem (per-block
 * energy partials, cosine and coefficient tables and, for 3D grids, the contributions exchanged across
 * tile and chunk seams: up to about 1/3 of one field, plus 16 floats per element row of the grid for the
 * coefficient table of the KL modes).  0 if the problem is invalid.  The workspace must be
 * 256-byte aligned; its contents need not be preserved between calls, and two calls that
 * may overlap on the device need separate workspaces. */
size_t dn_workspace_bytes(const dn_problem* problem);

/* Bytes of device staging that dn_energy_grad_host needs (u, r, J, weights / nodal fields,
 * plus dn_workspace_bytes).  0 if the problem is invalid. */
size_t dn_host_staging_bytes(const dn_problem* problem);

/* Diffusivity sampling ("DiffNets": coefficients nu are sampled per minibatch): writes
 *   nu[b][node] = exp( sum_{i,j(,k)=1..m} w[b][i-1][j-1]([k-1]) cos(i pi x) cos(j pi y) (cos(k pi z))
 *                      / (1 + i^2 + j^2 (+ k^2)) )
 * at the nodes.  kl_w: [B][m]^dim floats; nu_out: [B][nz][ny][nx] floats.  Needs no workspace. */
dn_status dn_kl_field(const dn_grid* grid, int32_t batch, int32_t kl_modes, const float* kl_w,
                      float* nu_out, void* stream);

/* Energy only (Eq. (pde_loss) in its variational form): J[b], b < B.  u: [B][nz][ny][nx].
 * The same number as the J output of dn_energy_grad up to rounding (every kernel family sums element
 * energies here and takes J from the residual there).  Nothing but J and the workspace is written. */
dn_status dn_energy(const dn_problem* problem, const float* u, float* J, void* workspace,
                    size_t workspace_bytes, void* stream);

/* Energy and its exact gradient in one pass over u (Algorithm 1: loss, then its gradient
 * for back-propagation):  r = K(nu) u - F, zeroed at Dirichlet nodes unless DN_NO_MASK,
 * multiplied by gJ[b] when gJ != NULL (the upstream dLoss/dJ_b).
 * J may be NULL (residual only).  r must not overlap u.  gJ: [B] floats or NULL.
 * Errors found before anything is enqueued come back as a status and leave the outputs untouched.
 * The kernels contain no unbounded wait: where warps of the tiled 2D kernel hand values to one
 * another, the wait has an iteration limit, and should it ever run out the energy J[b] of that
 * sample is returned as NaN (its residual is then not to be trusted either; a residual-only call, J == NULL,
 * cannot report it: pass J where that check matters). */
dn_status dn_energy_grad(const dn_problem* problem, const float* u, const float* gJ, float* J, float* r,
                         void* workspace, size_t workspace_bytes, void* stream);

/* dn_energy_grad that also records two caller-owned CUDA events (cudaEvent_t passed as void*)
 * on `stream`: event_before just before the fused energy+residual kernel is enqueued and
 * event_after just after it, so that a caller can time that kernel alone while the table and
 * finaliser kernels of the same call are excluded.  Either event may be NULL.  A measurement
 * aid (Algorithm 1 has no counterpart); results are identical to dn_energy_grad. */
dn_status dn_energy_grad_traced(const dn_problem* problem, const float* u, const float* gJ, float* J, float* r,
                                void* workspace, size_t workspace_bytes, void* stream,
                                void* event_before, void* event_after);

/* dn_energy_grad without a workspace argument, for callers that are not allowed to allocate
 * device memory: code running inside another framework's memory plan, under a fixed memory
 * budget, or at a point where cudaMalloc would stall the device.  (The paper has no counterpart;
 * this is a calling convenience.)  The scratch that dn_energy_grad takes from the caller is here a
 * fixed array of DN_STATIC_SCRATCH_BYTES (1 MiB) inside the library image; every GPU that loads the
 * library holds it until the process exits.  The call itself allocates and frees nothing.
 *  - Inputs, outputs and results are exactly those of dn_energy_grad.
 *  - A problem that needs more scratch than the array holds (large grids on the any-size kernels,
 *    very large batches) is refused with DN_ERR_WORKSPACE and nothing is enqueued; use
 *    dn_energy_grad with your own workspace for those.  A wide 2D grid whose per-row coefficient
 *    table does not fit runs on another kernel family if that one's scratch fits, else it is refused
 *    the same way (e.g. 4096 x 4096 nodes, batch 16, 6 KL modes).
 *  - The first call on each device looks up the array's device address (one runtime query, with
 *    that device current); make that first call before starting any stream capture.
 *  - All calls on a device share the one array and it keeps whatever the previous call left in it.
 *    Nothing in it needs to start at zero (every entry is written before it is read), but two calls
 *    that may run on the GPU at the same time (different streams) race on it: serialise them, or
 *    use dn_energy_grad with separate workspaces. */
dn_status dn_energy_grad_static(const dn_problem* problem, const float* u, const float* gJ, float* J, float* r,
                                void* stream);

/* Boundary operator B(u) = b (Eq. (pde)): overwrites the two Dirichlet faces of a field in
 * place.  mode 0: field = bc_x0 at ix = 0 and bc_x1 at ix = nx-1;  mode 1: both faces = 0
 * (e.g. to mask a gradient). */
dn_status dn_apply_bc(const dn_grid* grid, int32_t batch, float bc_x0, float bc_x1, int32_t mode,
                      float* field_inout, void* stream);

/* dn_apply_bc (mode 0) with one pair of values per sample: field[b] = bc_x0_b[b] at ix = 0 and bc_x1_b[b] at
 * ix = nx-1.  bc_x0_b, bc_x1_b: [B] floats. */
dn_status dn_apply_bc_per_sample(const dn_grid* grid, int32_t batch, const float* bc_x0_b, const float* bc_x1_b,
                                 float* field_inout, void* stream);

/* dn_energy_grad with HOST buffers: copies u (and nu / f / kl_w / gJ when present) to the
 * device staging area, runs the same kernels, copies J and r back, and waits for the last
 * copy.  The batch is pipelined in chunks of whole samples over two internal copy streams (created
 * and destroyed inside the call) so that both directions of the host link overlap with the kernels.  In `problem`, nu / kl_w / f / bc_x0_b / bc_x1_b are HOST pointers here.  u_host, r_host: [B][..] floats;
 * J_host: [B] floats or NULL; staging: device memory of dn_host_staging_bytes(problem) bytes,
 * 256-byte aligned.  Use pinned host memory for full copy bandwidth. */
dn_status dn_energy_grad_host(const dn_problem* problem, const float* u_host, const float* gJ_host,
                              float* J_host, float* r_host, void* staging, size_t staging_bytes,
                              void* stream);

/* ---- The discrete FEM solution by matrix-free conjugate gradients ----------------------------------
 * The conventional-solver side of the paper's comparison ("Mathematical preliminaries": the PDE is usually
 * discretised and solved; the appendix sets the generator's fields against such solutions): solves
 * K(nu) u = F on the free nodes with u = bc_x0 / bc_x1 on the Dirichlet faces, by Jacobi-preconditioned
 * conjugate gradients whose operator is the fused energy+residual kernel of dn_energy_grad.  The result is
 * the minimiser of J, i.e. the lower bound of the loss a generator can reach for this nu.
 *  - u_inout: [B][nz][ny][nx]; its interior is the initial guess, its Dirichlet faces are overwritten.
 *  - Exactly max_iters iterations are enqueued (nothing is read back); a sample whose residual norm has
 *    fallen to rtol times its initial value stops changing.  relres_out: [B] floats = |r| / |r0| reached,
 *    iters_out: [B] int32 = iterations a sample took part in; either may be NULL.
 *  - problem->flags: DN_FORCE_GENERIC is honoured, the other flags are ignored.
 *  - workspace: dn_cg_workspace_bytes(problem) bytes (four fields + two fused-kernel workspaces), 256-byte aligned. */
size_t dn_cg_workspace_bytes(const dn_problem* problem);
dn_status dn_cg_solve(const dn_problem* problem, float* u_inout, int32_t max_iters, float rtol,
                      float* relres_out, int32_t* iters_out, void* workspace, size_t workspace_bytes,
                      void* stream);

/* ---- The paper's own example: finite-difference loss of the inviscid Burgers equation ------------
 *
 *        u_t + u u_x = 0 on (x,t) in [0,1] x [0,T],   u(x,0) = (1 - cos(2 pi c x)) / 2
 *
 * ("Introduction", Eq. (Inviscid_Burgers), Eq. (initial-condition)).  A generated field is scored by
 * L = L_p + lambda L_b ("DiffNets", Eq. (diffnetloss), Eq. (pde_loss), Eq. (boundaryloss)) with the
 * first derivatives taken by 3x3 Sobel stencils ("Implementing the forward model"):
 *
 *   field   u[b][j][i] at x_i = i hx, t_j = j ht,  hx = 1/(nx-1), ht = T/(nt-1)   (x fastest)
 *   u_x     = sum Sx[dj][di] u[j+dj][i+di] / (8 hx),  Sx = [[-1,0,1],[-2,0,2],[-1,0,1]];  u_t: Sx transposed, / (8 ht)
 *   res     = u_t + u u_x at the interior nodes (0 < i < nx-1, 0 < j < nt-1)
 *   L_p[b]  = hx ht sum_interior res^2
 *   L_b[b]  = hx sum_i (u[0][i] - u(x_i,0))^2 + ht sum_j u[j][0]^2      (initial row and inflow column)
 *   L[b]    = L_p[b] + lambda L_b[b],    g = dL/du at every node.
 *
 * The paper names the stencils only; the 1/(8h) normalisation (exact on linear fields), the discrete
 * norms and the inflow-only boundary term are this library's reading. */
typedef struct {
    int32_t nx, nt;              /* nodes in x and t, each in 3..DN_MAX_EXTENT                      */
    int32_t batch;               /* B >= 1                                                         */
    float T;                     /* final time (> 0); the paper's domain has T = 0.2               */
    float lambda;                /* weight of L_b                                                  */
    const float* c;              /* [B] wave numbers of the initial-condition family               */
    uint32_t flags;              /* DN_FORCE_GENERIC or 0                                          */
} dn_burgers;

/* Bytes of device scratch (per-warp loss partials) dn_burgers_loss_grad needs; 0 if invalid. */
size_t dn_burgers_workspace_bytes(const dn_burgers* problem);

/* Loss and its exact gradient in one pass over u (Algorithm 1: loss, then its gradient for
 * back-propagation).  u: [B][nt][nx];  L: [B] or NULL;  parts: [B][2] = (L_p, L_b) or NULL;
 * g: [B][nt][nx] or NULL (loss only), multiplied by gL[b] when gL != NULL; g must not overlap u.
 * Grids with nx % 4 == 0 and 16-byte aligned u and g take the row-marching kernel, all others an
 * any-size kernel.  event_before / event_after: optional caller-owned CUDA events recorded on
 * `stream` around the main kernel (a measurement aid), or NULL. */
dn_status dn_burgers_loss_grad(const dn_burgers* problem, const float* u, const float* gL, float* L,
                               float* parts, float* g, void* workspace, size_t workspace_bytes,
                               void* stream, void* event_before, void* event_after);

/* Bytes of device staging dn_burgers_loss_grad_host needs (u, g, c, gL, L, parts and the workspace); 0 if invalid. */
size_t dn_burgers_host_staging_bytes(const dn_burgers* problem);

/* dn_burgers_loss_grad with HOST buffers (problem->c is a HOST pointer here): copies c, gL and u to the
 * device staging area, runs the same kernels, copies L, parts and g back and waits for the last copy.
 * The batch flows in chunks of whole samples over two internal copy streams, as in dn_energy_grad_host.
 * g_host must not be NULL; L_host, parts_host, gL_host may be.  staging: device memory of
 * dn_burgers_host_staging_bytes(problem) bytes, 256-byte aligned.  Use pinned host memory. */
dn_status dn_burgers_loss_grad_host(const dn_burgers* problem, const float* u_host, const float* gL_host,
                                    float* L_host, float* parts_host, float* g_host, void* staging,
                                    size_t staging_bytes, void* stream);

/* Name of the kernel family dn_burgers_loss_grad would use for these pointers ("march", "generic"). */
const char* dn_burgers_path_name(const dn_burgers* problem, const float* u, const float* g);

/* Number of kernel launches the last-validated path of this problem enqueues per
 * dn_energy_grad call (for launch accounting); 0 if the problem is invalid. */
int32_t dn_launches_per_call(const dn_problem* problem);

/* Name of the kernel family that dn_energy_grad would use ("row2d", "strip2d", "strip3d", "tiled2d", "tiled3d", "generic"). */
const char* dn_path_name(const dn_problem* problem);

const char* dn_status_string(dn_status status);

#ifdef __cplusplus
}
#endif
#endif /* DN_H_ */
