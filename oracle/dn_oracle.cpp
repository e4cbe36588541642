// TEST INFRASTRUCTURE -- not part of the product.
//
// Plain fp64 CPU statement of what the physics-loss path computes.  It is the
// definition written out with loops: no tiling, no fusion, no sharing of
// quantities between neighbouring elements.  The CUDA library shares no code,
// header, table or constant with this file.
//
// What is computed (paper: "Mathematical preliminaries", Eq. (pde): a PDE
// A_nu(u) = f with boundary operator B(u) = b on the unit square/cube; "DiffNets",
// Eq. (pde_loss): the loss is an expectation over a batch of full-field
// generator outputs).  The paper fixes the role of the loss only; the concrete
// PDE, discretisation and loss form used here are:
//
//   PDE        -div(nu grad u) = f on [0,1]^d, d in {2,3};
//              u = bc_x0 on x = 0, u = bc_x1 on x = 1, zero flux elsewhere.
//   mesh       uniform grid of nx*ny(*nz) nodes, Q1 (bi/tri-linear) elements,
//              h_a = 1/(n_a - 1).
//   energy     J(u) = sum_e sum_q W_q ( 1/2 nu_q |grad u_q|^2 - f_q u_q )
//              with tensor Gauss quadrature, 2 points per axis (3 for checks).
//   residual   r_i = dJ/du_i = sum_{e contains i} sum_q W_q
//                      ( nu_q grad u_q . grad N_i(x_q) - f_q N_i(x_q) )
//              = (K(nu) u - F)_i, then set to zero at Dirichlet nodes
//              (ix == 0 or ix == nx-1), then scaled by gJ[b] when given.
//   nu_q       mode 0: Q1 interpolation of a nodal field;
//              mode 1: the KL expansion
//                 nu(x) = exp( sum_{i,j(,k)=1..m} w_ij(k) cos(i pi x) cos(j pi y)
//                              (cos(k pi z)) / (1 + i^2 + j^2 (+ k^2)) )
//              evaluated at the physical Gauss point;
//              mode 2: the same KL expansion evaluated at the nodes (in double), then Q1 interpolation.
//
// Inputs are the same fp32 arrays the GPU gets, promoted to double on read.
// Arrays are C-ordered [B][nz][ny][nx], x fastest.
//
// Pins (tests/test_oracle_pins.py): closed-form energies, textbook element
// matrices, partition of unity, Euler identity, quadratic-in-t, finite
// differences, 3-point-rule cross-check, dense direct solve.  The KL-at-Gauss
// mode is pinned by Gauss sums typed out point by point: for u = 1 - x, and for
// the Q1 fields u = 2x + xy and u = x + xyz, whose gradient differs at every Gauss
// point of an element (energy, and the residual at one node).

#include <cmath>
#include <cstddef>
#include <cstdint>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

enum { ORC_NU_NODAL = 0, ORC_NU_KL_GAUSS = 1, ORC_NU_KL_NODAL = 2 };
enum { ORC_IMPOSE_BC_ON_LOAD = 1u, ORC_NO_MASK = 2u };

struct orc_problem {
    int32_t dim, nx, ny, nz, batch;
    int32_t nu_mode;
    int32_t kl_modes;
    int32_t nquad;        // Gauss points per axis: 2 (the method) or 3 (cross-check)
    uint32_t flags;
    int32_t u_f64;        // 1: the u argument holds doubles (used by the solver/finite-difference pins)
    double f_const;
    double bc_x0, bc_x1;
    const float* nu;      // [B][nz][ny][nx] when nu_mode == ORC_NU_NODAL
    const float* kl_w;    // [B][m]^dim, index [b][i-1][j-1]([k-1]); i<->x, j<->y, k<->z
    const float* f;       // nodal forcing [B][..] or NULL -> f_const
};

}  // extern "C"

namespace {

const double kPi = 3.14159265358979323846264338327950288;

struct Rule { int n; double xi[3]; double wt[3]; };

Rule gauss_rule(int n) {
    Rule r{};
    r.n = n;
    if (n == 2) {
        r.xi[0] = -1.0 / std::sqrt(3.0); r.xi[1] = 1.0 / std::sqrt(3.0);
        r.wt[0] = 1.0; r.wt[1] = 1.0;
    } else {  // n == 3
        r.xi[0] = -std::sqrt(3.0 / 5.0); r.xi[1] = 0.0; r.xi[2] = std::sqrt(3.0 / 5.0);
        r.wt[0] = 5.0 / 9.0; r.wt[1] = 8.0 / 9.0; r.wt[2] = 5.0 / 9.0;
    }
    return r;
}

struct Geo {
    int dim, nx, ny, nz;
    long nodes;           // per sample
    double h[3];
    int nc;               // corners per element
};

Geo make_geo(const orc_problem& p) {
    Geo g{};
    g.dim = p.dim; g.nx = p.nx; g.ny = p.ny; g.nz = (p.dim == 3) ? p.nz : 1;
    g.nodes = (long)g.nx * g.ny * g.nz;
    g.h[0] = 1.0 / (g.nx - 1);
    g.h[1] = 1.0 / (g.ny - 1);
    g.h[2] = (p.dim == 3) ? 1.0 / (g.nz - 1) : 1.0;
    g.nc = (p.dim == 3) ? 8 : 4;
    return g;
}

inline long node_index(const Geo& g, int ix, int iy, int iz) {
    return ((long)iz * g.ny + iy) * g.nx + ix;
}

// KL diffusivity at a physical point of sample b.
double kl_nu(const orc_problem& p, int b, double x, double y, double z) {
    const int m = p.kl_modes;
    double s = 0.0;
    if (p.dim == 2) {
        const float* w = p.kl_w + (size_t)b * m * m;
        for (int i = 1; i <= m; ++i)
            for (int j = 1; j <= m; ++j)
                s += (double)w[(i - 1) * m + (j - 1)] * std::cos(i * kPi * x) * std::cos(j * kPi * y) /
                     (1.0 + (double)i * i + (double)j * j);
    } else {
        const float* w = p.kl_w + (size_t)b * m * m * m;
        for (int i = 1; i <= m; ++i)
            for (int j = 1; j <= m; ++j)
                for (int k = 1; k <= m; ++k)
                    s += (double)w[((i - 1) * m + (j - 1)) * m + (k - 1)] * std::cos(i * kPi * x) *
                         std::cos(j * kPi * y) * std::cos(k * kPi * z) /
                         (1.0 + (double)i * i + (double)j * j + (double)k * k);
    }
    return std::exp(s);
}

// Value of u at a node, with the optional on-load imposition of the Dirichlet data.
inline double u_at(const orc_problem& p, const Geo& g, const void* u, int b, int ix, int iy, int iz) {
    if (p.flags & ORC_IMPOSE_BC_ON_LOAD) {
        if (ix == 0) return p.bc_x0;
        if (ix == g.nx - 1) return p.bc_x1;
    }
    const size_t idx = (size_t)b * g.nodes + node_index(g, ix, iy, iz);
    return p.u_f64 ? ((const double*)u)[idx] : (double)((const float*)u)[idx];
}

// Shape function a (corner bits ax,ay,az) and its physical gradient at reference point (xi,eta,zeta).
inline void shape(const Geo& g, int a, const double ref[3], double& N, double dN[3]) {
    double fac[3], dfac[3];
    for (int ax = 0; ax < 3; ++ax) {
        if (ax >= g.dim) { fac[ax] = 1.0; dfac[ax] = 0.0; continue; }
        const double sgn = ((a >> ax) & 1) ? 1.0 : -1.0;
        fac[ax] = 0.5 * (1.0 + sgn * ref[ax]);
        dfac[ax] = 0.5 * sgn * (2.0 / g.h[ax]);   // d(ref)/d(phys) = 2/h
    }
    N = fac[0] * fac[1] * fac[2];
    dN[0] = dfac[0] * fac[1] * fac[2];
    dN[1] = fac[0] * dfac[1] * fac[2];
    dN[2] = fac[0] * fac[1] * dfac[2];
}

// One element: energy parts and the contribution to each corner's residual, and
// (optionally) the element stiffness matrix and load vector.
void element(const orc_problem& p, const Geo& g, const Rule& rule, int b, const void* u,
             int ex, int ey, int ez, double& Jdiff, double& Jload, double rc[8],
             double* Ke /*[8][8] or null*/, double* Fe /*[8] or null*/) {
    const int nc = g.nc;
    double uc[8], nuc[8], fc[8];
    for (int a = 0; a < nc; ++a) {
        const int ix = ex + (a & 1), iy = ey + ((a >> 1) & 1), iz = ez + ((a >> 2) & 1);
        const long idx = node_index(g, ix, iy, iz);
        uc[a] = u ? u_at(p, g, u, b, ix, iy, iz) : 0.0;
        nuc[a] = (p.nu_mode == ORC_NU_NODAL) ? (double)p.nu[(size_t)b * g.nodes + idx] : 0.0;
        if (p.nu_mode == ORC_NU_KL_NODAL)
            nuc[a] = kl_nu(p, b, ix * g.h[0], iy * g.h[1], (g.dim == 3) ? iz * g.h[2] : 0.0);
        fc[a] = p.f ? (double)p.f[(size_t)b * g.nodes + idx] : p.f_const;
    }
    Jdiff = 0.0; Jload = 0.0;
    for (int a = 0; a < nc; ++a) rc[a] = 0.0;
    if (Ke) std::memset(Ke, 0, sizeof(double) * 64);
    if (Fe) std::memset(Fe, 0, sizeof(double) * 8);

    const int nqz = (g.dim == 3) ? rule.n : 1;
    for (int qz = 0; qz < nqz; ++qz)
        for (int qy = 0; qy < rule.n; ++qy)
            for (int qx = 0; qx < rule.n; ++qx) {
                double ref[3] = {rule.xi[qx], rule.xi[qy], (g.dim == 3) ? rule.xi[qz] : 0.0};
                double W = rule.wt[qx] * rule.wt[qy] * (g.h[0] / 2.0) * (g.h[1] / 2.0);
                if (g.dim == 3) W *= rule.wt[qz] * (g.h[2] / 2.0);
                double N[8], dN[8][3];
                for (int a = 0; a < nc; ++a) shape(g, a, ref, N[a], dN[a]);
                double uq = 0.0, fq = 0.0, gu[3] = {0.0, 0.0, 0.0}, nuq = 0.0;
                for (int a = 0; a < nc; ++a) {
                    uq += N[a] * uc[a];
                    fq += N[a] * fc[a];
                    nuq += N[a] * nuc[a];
                    for (int c = 0; c < 3; ++c) gu[c] += dN[a][c] * uc[a];
                }
                if (p.nu_mode == ORC_NU_KL_GAUSS) {
                    const double x = (ex + 0.5 * (1.0 + ref[0])) * g.h[0];
                    const double y = (ey + 0.5 * (1.0 + ref[1])) * g.h[1];
                    const double z = (g.dim == 3) ? (ez + 0.5 * (1.0 + ref[2])) * g.h[2] : 0.0;
                    nuq = kl_nu(p, b, x, y, z);
                }
                Jdiff += W * 0.5 * nuq * (gu[0] * gu[0] + gu[1] * gu[1] + gu[2] * gu[2]);
                Jload += W * fq * uq;
                for (int a = 0; a < nc; ++a) {
                    rc[a] += W * (nuq * (gu[0] * dN[a][0] + gu[1] * dN[a][1] + gu[2] * dN[a][2]) - fq * N[a]);
                    if (Fe) Fe[a] += W * fq * N[a];
                    if (Ke)
                        for (int c = 0; c < nc; ++c)
                            Ke[a * 8 + c] += W * nuq * (dN[a][0] * dN[c][0] + dN[a][1] * dN[c][1] + dN[a][2] * dN[c][2]);
                }
            }
}

bool valid(const orc_problem& p) {
    if (p.dim != 2 && p.dim != 3) return false;
    if (p.nx < 2 || p.ny < 2 || (p.dim == 3 && p.nz < 2) || p.batch < 1) return false;
    if (p.nquad != 2 && p.nquad != 3) return false;
    if (p.nu_mode == ORC_NU_NODAL && !p.nu) return false;
    if ((p.nu_mode == ORC_NU_KL_GAUSS || p.nu_mode == ORC_NU_KL_NODAL) && (!p.kl_w || p.kl_modes < 1)) return false;
    if (p.nu_mode != ORC_NU_NODAL && p.nu_mode != ORC_NU_KL_GAUSS && p.nu_mode != ORC_NU_KL_NODAL) return false;
    return true;
}

}  // namespace

extern "C" {

int orc_num_threads() {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void orc_set_num_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

// nu at the nodes of the grid, from the KL formula.  nu_out is [B][nz][ny][nx] doubles.
int orc_kl_field(int dim, int nx, int ny, int nz, int batch, int kl_modes, const float* kl_w, double* nu_out) {
    orc_problem p{};
    p.dim = dim; p.nx = nx; p.ny = ny; p.nz = nz; p.batch = batch;
    p.nu_mode = ORC_NU_KL_GAUSS; p.kl_modes = kl_modes; p.kl_w = kl_w; p.nquad = 2;
    if (!valid(p) || !nu_out) return 1;
    const Geo g = make_geo(p);
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < batch; ++b)
        for (int iz = 0; iz < g.nz; ++iz)
            for (int iy = 0; iy < g.ny; ++iy)
                for (int ix = 0; ix < g.nx; ++ix)
                    nu_out[(size_t)b * g.nodes + node_index(g, ix, iy, iz)] =
                        kl_nu(p, b, ix * g.h[0], iy * g.h[1], (dim == 3) ? iz * g.h[2] : 0.0);
    return 0;
}

// Energy per sample (J = Jdiff - Jload) and, when r != NULL, the residual.
// gJ may be NULL.  r is [B][nz][ny][nx] doubles.
//
// Threads split the slabs of elements (rows in 2D, planes in 3D) of one sample in
// two sweeps, even slabs then odd slabs, so that no two threads add into the same
// node; each node still receives exactly the sum over its adjacent elements.  The
// energy is first summed per slab, then over slabs in index order.
int orc_energy_grad(const orc_problem* pp, const void* u, const double* gJ, double* J, double* Jdiff_out,
                    double* Jload_out, double* r) {
    if (!pp || !u) return 1;
    const orc_problem& p = *pp;
    if (!valid(p)) return 1;
    const Geo g = make_geo(p);
    const Rule rule = gauss_rule(p.nquad);
    const int nslab = (g.dim == 3) ? g.nz - 1 : g.ny - 1;
    const int nrow = (g.dim == 3) ? g.ny - 1 : 1;
    std::vector<double> sd(nslab), sl(nslab);
    for (int b = 0; b < p.batch; ++b) {
        double* rb = r ? r + (size_t)b * g.nodes : nullptr;
        if (rb) for (long i = 0; i < g.nodes; ++i) rb[i] = 0.0;
        for (int parity = 0; parity < 2; ++parity) {
#pragma omp parallel for schedule(dynamic, 1)
            for (int s = parity; s < nslab; s += 2) {
                double accd = 0.0, accl = 0.0;
                for (int row = 0; row < nrow; ++row)
                    for (int ex = 0; ex < g.nx - 1; ++ex) {
                        const int ey = (g.dim == 3) ? row : s;
                        const int ez = (g.dim == 3) ? s : 0;
                        double jd, jl, rc[8];
                        element(p, g, rule, b, u, ex, ey, ez, jd, jl, rc, nullptr, nullptr);
                        accd += jd; accl += jl;
                        if (rb)
                            for (int a = 0; a < g.nc; ++a)
                                rb[node_index(g, ex + (a & 1), ey + ((a >> 1) & 1), ez + ((a >> 2) & 1))] += rc[a];
                    }
                sd[s] = accd; sl[s] = accl;
            }
        }
        double jd = 0.0, jl = 0.0;
        for (int s = 0; s < nslab; ++s) { jd += sd[s]; jl += sl[s]; }
        if (J) J[b] = jd - jl;
        if (Jdiff_out) Jdiff_out[b] = jd;
        if (Jload_out) Jload_out[b] = jl;
        if (rb) {
            if (!(p.flags & ORC_NO_MASK))
                for (int iz = 0; iz < g.nz; ++iz)
                    for (int iy = 0; iy < g.ny; ++iy) {
                        rb[node_index(g, 0, iy, iz)] = 0.0;
                        rb[node_index(g, g.nx - 1, iy, iz)] = 0.0;
                    }
            if (gJ) for (long i = 0; i < g.nodes; ++i) rb[i] *= gJ[b];
        }
    }
    return 0;
}

// Residual at selected nodes only: idx[k] is a flat index into [B][nz][ny][nx].
// Each value is the plain sum over the (up to 2^d) elements that contain the node.
int orc_residual_at(const orc_problem* pp, const void* u, const double* gJ, long n, const int64_t* idx, double* out) {
    if (!pp || !u || !idx || !out) return 1;
    const orc_problem& p = *pp;
    if (!valid(p)) return 1;
    const Geo g = make_geo(p);
    const Rule rule = gauss_rule(p.nquad);
#pragma omp parallel for schedule(dynamic, 16)
    for (long k = 0; k < n; ++k) {
        const int b = (int)(idx[k] / g.nodes);
        long rem = idx[k] % g.nodes;
        const int ix = (int)(rem % g.nx); rem /= g.nx;
        const int iy = (int)(rem % g.ny);
        const int iz = (int)(rem / g.ny);
        double acc = 0.0;
        const int dz0 = (g.dim == 3) ? -1 : 0;
        for (int dz = dz0; dz <= 0; ++dz)
            for (int dy = -1; dy <= 0; ++dy)
                for (int dx = -1; dx <= 0; ++dx) {
                    const int ex = ix + dx, ey = iy + dy, ez = iz + dz;
                    if (ex < 0 || ex >= g.nx - 1 || ey < 0 || ey >= g.ny - 1) continue;
                    if (g.dim == 3 && (ez < 0 || ez >= g.nz - 1)) continue;
                    double jd, jl, rc[8];
                    element(p, g, rule, b, u, ex, ey, (g.dim == 3) ? ez : 0, jd, jl, rc, nullptr, nullptr);
                    const int a = (-dx) | ((-dy) << 1) | ((g.dim == 3 ? -dz : 0) << 2);
                    acc += rc[a];
                }
        if (!(p.flags & ORC_NO_MASK) && (ix == 0 || ix == g.nx - 1)) acc = 0.0;
        if (gJ) acc *= gJ[b];
        out[k] = acc;
    }
    return 0;
}

// Overwrite the two Dirichlet faces.  mode 0: set u = bc_x0 at ix = 0 and bc_x1 at
// ix = nx-1; mode 1: set both faces to zero.
int orc_apply_bc(int dim, int nx, int ny, int nz, int batch, double bc_x0, double bc_x1, int mode, float* field) {
    if ((dim != 2 && dim != 3) || nx < 2 || ny < 2 || (dim == 3 && nz < 2) || batch < 1 || !field) return 1;
    if (mode != 0 && mode != 1) return 1;
    const int nzz = (dim == 3) ? nz : 1;
    for (long line = 0; line < (long)batch * nzz * ny; ++line) {
        field[line * nx] = (mode == 0) ? (float)bc_x0 : 0.0f;
        field[line * nx + nx - 1] = (mode == 0) ? (float)bc_x1 : 0.0f;
    }
    return 0;
}

// Dense stiffness matrix K [n][n] and load vector F [n] of sample b (n = nodes per
// sample), by summing element matrices.  Tiny grids only.
int orc_assemble(const orc_problem* pp, int b, double* K, double* F) {
    if (!pp || !K || !F) return 1;
    const orc_problem& p = *pp;
    if (!valid(p) || b < 0 || b >= p.batch) return 1;
    const Geo g = make_geo(p);
    const Rule rule = gauss_rule(p.nquad);
    const long n = g.nodes;
    for (long i = 0; i < n * n; ++i) K[i] = 0.0;
    for (long i = 0; i < n; ++i) F[i] = 0.0;
    const int nez = (g.dim == 3) ? g.nz - 1 : 1;
    for (int ez = 0; ez < nez; ++ez)
        for (int ey = 0; ey < g.ny - 1; ++ey)
            for (int ex = 0; ex < g.nx - 1; ++ex) {
                double jd, jl, rc[8], Ke[64], Fe[8];
                element(p, g, rule, b, nullptr, ex, ey, ez, jd, jl, rc, Ke, Fe);
                long gi[8];
                for (int a = 0; a < g.nc; ++a)
                    gi[a] = node_index(g, ex + (a & 1), ey + ((a >> 1) & 1), ez + ((a >> 2) & 1));
                for (int a = 0; a < g.nc; ++a) {
                    F[gi[a]] += Fe[a];
                    for (int c = 0; c < g.nc; ++c) K[gi[a] * n + gi[c]] += Ke[a * 8 + c];
                }
            }
    return 0;
}

// Discrete solution of K u = F with u fixed to bc_x0 / bc_x1 on the two x faces:
// Gaussian elimination with partial pivoting on the free-node block.  u_out is [n] doubles.
int orc_solve_dirichlet(int dim, int nx, int ny, int nz, const double* K, const double* F, double bc_x0,
                        double bc_x1, double* u_out) {
    if (!K || !F || !u_out) return 1;
    const long n = (long)nx * ny * ((dim == 3) ? nz : 1);
    std::vector<long> freeidx;
    for (long i = 0; i < n; ++i) {
        const int ix = (int)(i % nx);
        if (ix == 0) u_out[i] = bc_x0;
        else if (ix == nx - 1) u_out[i] = bc_x1;
        else { u_out[i] = 0.0; freeidx.push_back(i); }
    }
    const long nf = (long)freeidx.size();
    std::vector<double> A((size_t)nf * nf), rhs(nf);
    for (long a = 0; a < nf; ++a) {
        const long i = freeidx[a];
        double s = F[i];
        for (long j = 0; j < n; ++j) {
            const int jx = (int)(j % nx);
            if (jx == 0 || jx == nx - 1) s -= K[i * n + j] * u_out[j];
        }
        rhs[a] = s;
        for (long c = 0; c < nf; ++c) A[a * nf + c] = K[i * n + freeidx[c]];
    }
    for (long k = 0; k < nf; ++k) {
        long piv = k;
        for (long i = k + 1; i < nf; ++i)
            if (std::fabs(A[i * nf + k]) > std::fabs(A[piv * nf + k])) piv = i;
        if (A[piv * nf + k] == 0.0) return 2;
        if (piv != k) {
            for (long j = 0; j < nf; ++j) std::swap(A[k * nf + j], A[piv * nf + j]);
            std::swap(rhs[k], rhs[piv]);
        }
        for (long i = k + 1; i < nf; ++i) {
            const double m = A[i * nf + k] / A[k * nf + k];
            if (m == 0.0) continue;
            for (long j = k; j < nf; ++j) A[i * nf + j] -= m * A[k * nf + j];
            rhs[i] -= m * rhs[k];
        }
    }
    for (long k = nf - 1; k >= 0; --k) {
        double s = rhs[k];
        for (long j = k + 1; j < nf; ++j) s -= A[k * nf + j] * u_out[freeidx[j]];
        u_out[freeidx[k]] = s / A[k * nf + k];
    }
    return 0;
}

}  // extern "C"
