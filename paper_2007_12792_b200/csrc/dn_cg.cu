// Matrix-free conjugate gradients on K(nu) u = F with the Dirichlet faces held at their values: the
// "conventional solver" side of the paper's comparison ("Mathematical preliminaries": the PDE is normally
// discretised and solved; the appendix compares the generator's fields with such solutions), built on the
// same fused energy+residual kernel that scores the generator.  Its result u* is the minimiser of the
// energy J, the lower bound of the loss any generator can reach.
//
// Per sample b (all samples advance together, each with its own scalars; Jacobi preconditioner D = diag K):
//     r = F - K u,  z = D^-1 r,  p = z,  rho = r.z
//     repeat:  q = K p;  alpha = rho / p.q;  u += alpha p;  r -= alpha q;  z = D^-1 r;
//              rho' = r.z;  beta = rho' / rho;  p = z + beta p;  rho = rho'
// K p is the fused kernel applied to p with zero forcing and zero boundary values (p vanishes on the
// Dirichlet faces), and p.q = 2 J(p) comes from the energy that kernel computes anyway, so an iteration is
// the fused kernel plus two streaming kernels (update + dot, new direction) and two one-block-per-sample
// scalar kernels.  Dot products are summed in fp64 in a fixed order.  A sample whose residual norm has
// dropped below rtol times its initial value is frozen (alpha = 0); the iteration count is fixed by the
// caller, so nothing is read back and the whole solve is one stream of launches.
#include "dn_internal.cuh"

namespace dn {
namespace {

constexpr int CG_THREADS = 256;
constexpr int CG_VEC = 4;                    // floats per thread per trip
constexpr int CG_BLOCK_NODES = CG_THREADS * CG_VEC * 4;

struct CgScalars {                           // per sample, in the workspace
    double rho, rr0, rr;
    float alpha, beta;
    int active, iters;
};

__device__ __forceinline__ void block_sum2(double& a, double& b) {
    __shared__ double sa[CG_THREADS / 32], sb[CG_THREADS / 32];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a += __shfl_down_sync(0xffffffffu, a, o);
        b += __shfl_down_sync(0xffffffffu, b, o);
    }
    if ((threadIdx.x & 31) == 0) { sa[threadIdx.x >> 5] = a; sb[threadIdx.x >> 5] = b; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double x = 0.0, y = 0.0;
        for (int w = 0; w < CG_THREADS / 32; ++w) { x += sa[w]; y += sb[w]; }
        a = x; b = y;
    }
}

// r = -r (the fused kernel returns K u - F), p = z = dinv r; partial sums of r.z and r.r per block.
__global__ void __launch_bounds__(CG_THREADS) cg_init_kernel(long long nodes, int nblk, float* __restrict__ r,
                                                             const float* __restrict__ dinv, float* __restrict__ p,
                                                             double* __restrict__ partials) {
    const int b = blockIdx.y;
    const long long base = (long long)b * nodes;
    const long long lo = (long long)blockIdx.x * CG_BLOCK_NODES;
    const long long hi = min(lo + (long long)CG_BLOCK_NODES, nodes);
    double s_rz = 0.0, s_rr = 0.0;
    for (long long i = lo + threadIdx.x; i < hi; i += CG_THREADS) {
        const float rv = -r[base + i];
        const float zv = rv * dinv[base + i];
        r[base + i] = rv;
        p[base + i] = zv;
        s_rz += (double)(rv * zv);
        s_rr += (double)(rv * rv);
    }
    block_sum2(s_rz, s_rr);
    if (threadIdx.x == 0) {
        partials[2 * ((long long)b * nblk + blockIdx.x)] = s_rz;
        partials[2 * ((long long)b * nblk + blockIdx.x) + 1] = s_rr;
    }
}

__device__ __forceinline__ void sum_pairs(const double* __restrict__ p, int n, double& a, double& b) {
    double x = 0.0, y = 0.0;
    for (int i = threadIdx.x; i < n; i += CG_THREADS) { x += p[2 * i]; y += p[2 * i + 1]; }
    block_sum2(x, y);
    a = x; b = y;                            // valid in thread 0
}

__global__ void __launch_bounds__(CG_THREADS) cg_start_kernel(const double* __restrict__ partials, int nblk,
                                                              CgScalars* __restrict__ sc) {
    double rz, rr;
    sum_pairs(partials + 2ll * blockIdx.x * nblk, nblk, rz, rr);
    if (threadIdx.x == 0) {
        CgScalars s;
        s.rho = rz; s.rr0 = rr; s.rr = rr; s.alpha = 0.f; s.beta = 0.f; s.iters = 0;
        s.active = (rr > 0.0 && rz > 0.0) ? 1 : 0;
        sc[blockIdx.x] = s;
    }
}

// alpha = rho / p.q with p.q = 2 (diffusion part - load part) of the fused kernel's energy of p.
__global__ void __launch_bounds__(CG_THREADS) cg_alpha_kernel(const double* __restrict__ op_partials, int op_nblk,
                                                              CgScalars* __restrict__ sc) {
    double d, l;
    sum_pairs(op_partials + 2ll * blockIdx.x * op_nblk, op_nblk, d, l);
    if (threadIdx.x == 0) {
        CgScalars& s = sc[blockIdx.x];
        const double pq = 2.0 * (d - l);
        s.alpha = (s.active && pq > 0.0) ? (float)(s.rho / pq) : 0.0f;
        if (!(pq > 0.0)) s.active = 0;
    }
}

// u += alpha p, r -= alpha q; partial sums of r.z (z = dinv r) and r.r.
__global__ void __launch_bounds__(CG_THREADS) cg_update_kernel(long long nodes, int nblk, float* __restrict__ u,
                                                               float* __restrict__ r, const float* __restrict__ p,
                                                               const float* __restrict__ q,
                                                               const float* __restrict__ dinv,
                                                               const CgScalars* __restrict__ sc,
                                                               double* __restrict__ partials) {
    const int b = blockIdx.y;
    const float alpha = sc[b].alpha;
    const long long base = (long long)b * nodes;
    const long long lo = (long long)blockIdx.x * CG_BLOCK_NODES;
    const long long hi = min(lo + (long long)CG_BLOCK_NODES, nodes);
    double s_rz = 0.0, s_rr = 0.0;
    if (alpha != 0.0f) {
        for (long long i = lo + threadIdx.x; i < hi; i += CG_THREADS) {
            const float pv = p[base + i], qv = q[base + i];
            const float rv = fmaf(-alpha, qv, r[base + i]);
            u[base + i] = fmaf(alpha, pv, u[base + i]);
            r[base + i] = rv;
            const float zv = rv * dinv[base + i];
            s_rz += (double)(rv * zv);
            s_rr += (double)(rv * rv);
        }
    }
    block_sum2(s_rz, s_rr);
    if (threadIdx.x == 0) {
        partials[2 * ((long long)b * nblk + blockIdx.x)] = s_rz;
        partials[2 * ((long long)b * nblk + blockIdx.x) + 1] = s_rr;
    }
}

__global__ void __launch_bounds__(CG_THREADS) cg_beta_kernel(const double* __restrict__ partials, int nblk, double rtol2,
                                                             CgScalars* __restrict__ sc) {
    double rz, rr;
    sum_pairs(partials + 2ll * blockIdx.x * nblk, nblk, rz, rr);
    if (threadIdx.x == 0) {
        CgScalars& s = sc[blockIdx.x];
        if (s.active && s.alpha != 0.0f) {
            s.beta = (float)(rz / s.rho);
            s.rho = rz; s.rr = rr; s.iters += 1;
            if (rr <= rtol2 * s.rr0 || !(rz > 0.0)) s.active = 0;
        } else {
            s.active = 0; s.alpha = 0.0f;    // frozen: u and r no longer change
        }
    }
}

// p = dinv r + beta p
__global__ void __launch_bounds__(CG_THREADS) cg_direction_kernel(long long nodes, const float* __restrict__ r,
                                                                  const float* __restrict__ dinv, float* __restrict__ p,
                                                                  const CgScalars* __restrict__ sc) {
    const int b = blockIdx.y;
    if (!sc[b].active) return;
    const float beta = sc[b].beta;
    const long long base = (long long)b * nodes;
    const long long lo = (long long)blockIdx.x * CG_BLOCK_NODES;
    const long long hi = min(lo + (long long)CG_BLOCK_NODES, nodes);
    for (long long i = lo + threadIdx.x; i < hi; i += CG_THREADS)
        p[base + i] = fmaf(beta, p[base + i], r[base + i] * dinv[base + i]);
}

// ---- diagonal of K by probing ------------------------------------------------------------------------
// Nodes whose indices agree modulo 3 on every axis share no element, so the fused kernel applied to the
// indicator of one such colour class returns K_ii at the nodes i of that class: 3^dim applications give the
// whole diagonal.  One block per x-row; only the rows of the class (iy, iz congruent to the colour) do work.
// phase 0: e = 1 on the free nodes of the class in this row, 0 elsewhere in the row (e is zero outside the class rows).
// phase 1: dinv = 1 / (K e) on the free nodes of the class, 0 on its Dirichlet nodes; the row of e is cleared again.
__global__ void __launch_bounds__(CG_THREADS) cg_probe_kernel(int nx, int ny, int nz, int colour, int phase,
                                                              float* __restrict__ e, const float* __restrict__ q,
                                                              float* __restrict__ dinv) {
    const long long row = blockIdx.x;
    const int iy = (int)(row % ny), iz = (int)((row / ny) % nz);
    const int cx = colour % 3, cy = (colour / 3) % 3, cz = colour / 9;
    if (iy % 3 != cy || iz % 3 != cz) return;
    const long long base = row * nx;
    for (int ix = threadIdx.x; ix < nx; ix += CG_THREADS) {
        const bool mine = ix % 3 == cx, face = ix == 0 || ix == nx - 1;
        if (phase == 0) {
            e[base + ix] = (mine && !face) ? 1.0f : 0.0f;
        } else {
            if (mine) dinv[base + ix] = face ? 0.0f : 1.0f / q[base + ix];
            e[base + ix] = 0.0f;
        }
    }
}

__global__ void cg_report_kernel(const CgScalars* __restrict__ sc, int batch, float* __restrict__ relres,
                                 int32_t* __restrict__ iters) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= batch) return;
    if (relres) relres[b] = sc[b].rr0 > 0.0 ? (float)sqrt(sc[b].rr / sc[b].rr0) : 0.0f;
    if (iters) iters[b] = sc[b].iters;
}

long long nodes_of(const dn_problem& p) { return (long long)p.grid.nx * p.grid.ny * (p.grid.dim == 3 ? p.grid.nz : 1); }
int vec_blocks(long long nodes) { return (int)((nodes + CG_BLOCK_NODES - 1) / CG_BLOCK_NODES); }

struct CgLayout { size_t r, q, p, dinv, partials, scalars, op, op_bytes, op1, op1_bytes, total; };

CgLayout cg_layout(const dn_problem& p) {
    CgLayout L{};
    const size_t field = align_up(sizeof(float) * (size_t)p.batch * nodes_of(p));
    size_t off = 0;
    L.r = off; off += field;
    L.q = off; off += field;
    L.p = off; off += field;
    L.dinv = off; off += field;
    L.partials = off; off += align_up(sizeof(double) * 2 * (size_t)p.batch * vec_blocks(nodes_of(p)));
    L.scalars = off; off += align_up(sizeof(CgScalars) * (size_t)p.batch);
    // Two fused-kernel workspaces: one for the operator on directions (no nodal forcing, aligned scratch fields) and one
    // for the caller's problem (initial residual), which may take another kernel family with another layout.
    dn_problem pop = p;
    pop.f = nullptr;
    L.op_bytes = dn_workspace_bytes(&pop);
    L.op = off; off += align_up(L.op_bytes);
    L.op1_bytes = dn_workspace_bytes(&p);
    L.op1 = off; off += align_up(L.op1_bytes);
    L.total = off;
    return L;
}

}  // namespace
}  // namespace dn

using namespace dn;

extern "C" {

size_t dn_cg_workspace_bytes(const dn_problem* p) {
    if (!p || dn_workspace_bytes(p) == 0) return 0;
    return cg_layout(*p).total;
}

dn_status dn_cg_solve(const dn_problem* p, float* u, int32_t max_iters, float rtol, float* relres, int32_t* iters,
                      void* ws, size_t ws_bytes, void* stream) {
    if (!p || !u) return DN_ERR_NULL;
    if (dn_workspace_bytes(p) == 0) {        // invalid problem: let the fused path name the reason
        float dummy;
        return dn_energy(p, u, &dummy, nullptr, 0, stream);
    }
    if (max_iters < 0 || !(rtol >= 0.0f)) return DN_ERR_MODE;
    const CgLayout L = cg_layout(*p);
    if (!ws || (reinterpret_cast<uintptr_t>(ws) % kAlign) != 0 || ws_bytes < L.total) return DN_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char* base = static_cast<char*>(ws);
    float* r = reinterpret_cast<float*>(base + L.r);
    float* q = reinterpret_cast<float*>(base + L.q);
    float* pd = reinterpret_cast<float*>(base + L.p);
    float* dinv = reinterpret_cast<float*>(base + L.dinv);
    double* partials = reinterpret_cast<double*>(base + L.partials);
    CgScalars* sc = reinterpret_cast<CgScalars*>(base + L.scalars);
    void* op_ws = base + L.op;
    const size_t op_bytes = L.op_bytes;
    void* op1_ws = base + L.op1;
    const size_t op1_bytes = L.op1_bytes;
    const long long nodes = nodes_of(*p);
    const int nvb = vec_blocks(nodes);
    const dim3 vgrid((unsigned)nvb, (unsigned)p->batch);

    // Dirichlet faces of u take their values; r = K u - F (masked) with the caller's forcing
    if (launch_apply_bc(p->grid, p->batch, p->bc_x0, p->bc_x1, 0, u, s, p->bc_x0_b, p->bc_x1_b) != cudaSuccess)
        return DN_ERR_CUDA;
    dn_status st = DN_OK;
    dn_problem p1 = *p;
    p1.flags &= ~(DN_NO_MASK | DN_IMPOSE_BC_ON_LOAD);
    // the operator on directions: zero forcing, zero boundary values, same diffusivity
    dn_problem p0 = p1;
    p0.f = nullptr; p0.f_const = 0.0f; p0.bc_x0 = 0.0f; p0.bc_x1 = 0.0f; p0.bc_x0_b = nullptr; p0.bc_x1_b = nullptr;
    // The KL tables are built once per solve for the direction operator (aligned scratch fields, no nodal forcing); the
    // caller's problem is applied once, in a workspace of its own with its own tables (it may take another family).
    st = build_tables(&p0, pd, q, op_ws, op_bytes, s);
    if (st != DN_OK) return st;
    st = run_operator(&p1, u, r, op1_ws, op1_bytes, s, true, nullptr, nullptr);
    if (st != DN_OK) return st;
    {   // Jacobi preconditioner: the diagonal of K, one colour class per application (p and q serve as scratch)
        const int nz = p->grid.dim == 3 ? p->grid.nz : 1;
        const unsigned rows = (unsigned)((long long)p->batch * nz * p->grid.ny);
        const int ncol = p->grid.dim == 3 ? 27 : 9;
        if (cudaMemsetAsync(pd, 0, sizeof(float) * (size_t)nodes * p->batch, s) != cudaSuccess) return DN_ERR_CUDA;
        for (int c = 0; c < ncol; ++c) {
            cg_probe_kernel<<<rows, CG_THREADS, 0, s>>>(p->grid.nx, p->grid.ny, nz, c, 0, pd, nullptr, nullptr);
            st = run_operator(&p0, pd, q, op_ws, op_bytes, s, false, nullptr, nullptr);
            if (st != DN_OK) return st;
            cg_probe_kernel<<<rows, CG_THREADS, 0, s>>>(p->grid.nx, p->grid.ny, nz, c, 1, pd, q, dinv);
        }
        if (cudaGetLastError() != cudaSuccess) return DN_ERR_CUDA;
    }
    cg_init_kernel<<<vgrid, CG_THREADS, 0, s>>>(nodes, nvb, r, dinv, pd, partials);
    cg_start_kernel<<<p->batch, CG_THREADS, 0, s>>>(partials, nvb, sc);
    if (cudaGetLastError() != cudaSuccess) return DN_ERR_CUDA;

    const double rtol2 = (double)rtol * (double)rtol;
    for (int it = 0; it < max_iters; ++it) {
        const double* op_partials = nullptr;
        int op_nblk = 0;
        st = run_operator(&p0, pd, q, op_ws, op_bytes, s, false, &op_partials, &op_nblk);
        if (st != DN_OK) return st;
        cg_alpha_kernel<<<p->batch, CG_THREADS, 0, s>>>(op_partials, op_nblk, sc);
        cg_update_kernel<<<vgrid, CG_THREADS, 0, s>>>(nodes, nvb, u, r, pd, q, dinv, sc, partials);
        cg_beta_kernel<<<p->batch, CG_THREADS, 0, s>>>(partials, nvb, rtol2, sc);
        cg_direction_kernel<<<vgrid, CG_THREADS, 0, s>>>(nodes, r, dinv, pd, sc);
        if (cudaGetLastError() != cudaSuccess) return DN_ERR_CUDA;
    }
    if (relres || iters) {
        cg_report_kernel<<<(p->batch + 127) / 128, 128, 0, s>>>(sc, p->batch, relres, iters);
        if (cudaGetLastError() != cudaSuccess) return DN_ERR_CUDA;
    }
    return DN_OK;
}

}  // extern "C"
