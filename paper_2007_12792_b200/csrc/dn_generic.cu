// Any-size kernels: one thread per node gathers the contributions of its (up to) 4 / 8
// adjacent elements, recomputing each element; the thread at an element's low corner also
// adds that element's energy.  No atomics, fixed reduction order.  Handles every option
// (both nu modes, nodal forcing, unaligned pointers, any extents >= 2).  The tiled kernels
// are the fast path; these are the fall-back and their cross-check.
#include "dn_internal.cuh"

namespace dn {

namespace {

constexpr int GEN_THREADS = 128;

__device__ __forceinline__ float load_u(const Params& P, int b, const float* ub, int ix, long long idx) {
    if (P.flags & DN_IMPOSE_BC_ON_LOAD) {
        if (ix == 0) return P.bc0_b ? __ldg(P.bc0_b + b) : P.bc_x0;
        if (ix == P.nx - 1) return P.bc1_b ? __ldg(P.bc1_b + b) : P.bc_x1;
    }
    return __ldg(ub + idx);
}

// KL exponent (base 2) at the Gauss abscissae with per-axis indices (gx, gy, gz).
__device__ __forceinline__ float kl_exponent(const Params& P, const float* c, int gx, int gy, int gz) {
    const int m = P.m;
    float e = 0.0f;
    for (int i = 0; i < m; ++i) {
        float ei = 0.0f;
        for (int j = 0; j < m; ++j) {
            float ej;
            if (P.dim == 3) {
                ej = 0.0f;
                for (int k = 0; k < m; ++k) ej = fmaf(c[(i * m + j) * m + k], P.cg[2][k * P.gstride[2] + gz], ej);
            } else {
                ej = c[i * m + j];
            }
            ei = fmaf(ej, P.cg[1][j * P.gstride[1] + gy], ei);
        }
        e = fmaf(ei, P.cg[0][i * P.gstride[0] + gx], e);
    }
    return e;
}

// KL diffusivity at the node with per-axis indices (ix, iy, iz)  (DN_NU_KL_NODAL).
__device__ __forceinline__ float kl_node(const Params& P, const float* c, int ix, int iy, int iz) {
    const int m = P.m;
    float e = 0.0f;
    for (int i = 0; i < m; ++i) {
        float ei = 0.0f;
        for (int j = 0; j < m; ++j) {
            float ej;
            if (P.dim == 3) {
                ej = 0.0f;
                for (int k = 0; k < m; ++k) ej = fmaf(c[(i * m + j) * m + k], P.cn[2][k * P.nstride[2] + iz], ej);
            } else {
                ej = c[i * m + j];
            }
            ei = fmaf(ej, P.cn[1][j * P.nstride[1] + iy], ei);
        }
        e = fmaf(ei, P.cn[0][i * P.nstride[0] + ix], e);
    }
    return exp2f(e);
}

// ----- 2D element: contributions to its four corners and its energy parts -------------------
// Corner order (0,0), (1,0), (0,1), (1,1).  With e0 = u10-u00, s0 = u01-u00 and the twist
// t = u11-u10-u01+u00, the x-derivative at the Gauss row eta is (e0 + eta t)/hx and the
// y-derivative at the Gauss column xi is (s0 + xi t)/hy; the energy is a function of
// (e0, s0, t) and the chain rule distributes its three partial derivatives to the corners.
__device__ __forceinline__ void element2d(const Params& P, int b, int ex, int ey, const float* ub,
                                          const float* nub, const float* fb, const float* c,
                                          float rc[4], float& ed, float& el) {
    const int nx = P.nx;
    const long long i00 = (long long)ey * nx + ex;
    const float u00 = load_u(P, b, ub, ex, i00), u10 = load_u(P, b, ub, ex + 1, i00 + 1);
    const float u01 = load_u(P, b, ub, ex, i00 + nx), u11 = load_u(P, b, ub, ex + 1, i00 + nx + 1);
    const float ga[2] = {DN_GA, DN_GB};
    float nuq[2][2];                                   // [p: xi point][q: eta point]
    if (P.nu_mode != DN_NU_KL_GAUSS) {
        float n00, n10, n01, n11;
        if (P.nu_mode == DN_NU_NODAL) {
            n00 = __ldg(nub + i00); n10 = __ldg(nub + i00 + 1); n01 = __ldg(nub + i00 + nx); n11 = __ldg(nub + i00 + nx + 1);
        } else {
            n00 = kl_node(P, c, ex, ey, 0); n10 = kl_node(P, c, ex + 1, ey, 0);
            n01 = kl_node(P, c, ex, ey + 1, 0); n11 = kl_node(P, c, ex + 1, ey + 1, 0);
        }
        for (int p = 0; p < 2; ++p)
            for (int q = 0; q < 2; ++q) {
                const float lo = n00 + ga[p] * (n10 - n00), hi = n01 + ga[p] * (n11 - n01);
                nuq[p][q] = lo + ga[q] * (hi - lo);
            }
    } else {
        for (int p = 0; p < 2; ++p)
            for (int q = 0; q < 2; ++q) nuq[p][q] = exp2f(kl_exponent(P, c, 2 * ex + p, 2 * ey + q, 0));
    }
    const float kx = 0.25f * P.hy / P.hx, ky = 0.25f * P.hx / P.hy, W = 0.25f * P.hx * P.hy;
    const float e0 = u10 - u00, s0 = u01 - u00, t = (u11 - u01) - e0;
    float SX = 0.f, SY = 0.f, T = 0.f, en = 0.f;
    for (int q = 0; q < 2; ++q) {
        const float D = fmaf(ga[q], t, e0);
        const float G = kx * (nuq[0][q] + nuq[1][q]) * D;
        SX += G; T = fmaf(ga[q], G, T); en = fmaf(G, D, en);
    }
    for (int p = 0; p < 2; ++p) {
        const float D = fmaf(ga[p], t, s0);
        const float G = ky * (nuq[p][0] + nuq[p][1]) * D;
        SY += G; T = fmaf(ga[p], G, T); en = fmaf(G, D, en);
    }
    ed = 0.5f * en;
    rc[0] = T - SX - SY; rc[1] = SX - T; rc[2] = SY - T; rc[3] = T;
    if (fb) {
        const float f00 = __ldg(fb + i00), f10 = __ldg(fb + i00 + 1), f01 = __ldg(fb + i00 + nx), f11 = __ldg(fb + i00 + nx + 1);
        el = 0.f;
        for (int p = 0; p < 2; ++p)
            for (int q = 0; q < 2; ++q) {
                const float N[4] = {(1 - ga[p]) * (1 - ga[q]), ga[p] * (1 - ga[q]), (1 - ga[p]) * ga[q], ga[p] * ga[q]};
                const float fq = N[0] * f00 + N[1] * f10 + N[2] * f01 + N[3] * f11;
                const float uq = N[0] * u00 + N[1] * u10 + N[2] * u01 + N[3] * u11;
                el = fmaf(W * fq, uq, el);
                for (int a = 0; a < 4; ++a) rc[a] = fmaf(-W * fq, N[a], rc[a]);
            }
    } else {
        const float fw = P.f_const * W;
        el = fw * ((u00 + u10) + (u01 + u11));
        for (int a = 0; a < 4; ++a) rc[a] -= fw;
    }
}

// ----- 3D element -----------------------------------------------------------------------------
// Corner a = ax + 2 ay + 4 az.  d/dx at a Gauss point depends only on its (eta, zeta): it is
// the bilinear interpolation of the four x-edge differences; likewise for y and z.  Summing
// nu over the Gauss points along the derivative's own axis first leaves 4 weighted fluxes
// per direction, which are distributed back to the edges with the same bilinear weights.
__device__ __forceinline__ void element3d(const Params& P, int b, int ex, int ey, int ez, const float* ub,
                                          const float* nub, const float* fb, const float* c,
                                          float rc[8], float& ed, float& el) {
    const int nx = P.nx;
    const long long sy = nx, sz = (long long)nx * P.ny;
    const long long i0 = ((long long)ez * P.ny + ey) * nx + ex;
    float u[8];
    for (int a = 0; a < 8; ++a)
        u[a] = load_u(P, b, ub, ex + (a & 1), i0 + (a & 1) + ((a >> 1) & 1) * sy + ((a >> 2) & 1) * sz);
    const float L[2][2] = {{1.f - DN_GA, DN_GA}, {1.f - DN_GB, DN_GB}};   // L[point][corner bit]
    float nuq[2][2][2];                                                     // [p: xi][q: eta][s: zeta]
    if (P.nu_mode != DN_NU_KL_GAUSS) {
        float nn[8];
        for (int a = 0; a < 8; ++a)
            nn[a] = (P.nu_mode == DN_NU_NODAL) ? __ldg(nub + i0 + (a & 1) + ((a >> 1) & 1) * sy + ((a >> 2) & 1) * sz)
                                               : kl_node(P, c, ex + (a & 1), ey + ((a >> 1) & 1), ez + ((a >> 2) & 1));
        for (int p = 0; p < 2; ++p)
            for (int q = 0; q < 2; ++q)
                for (int s = 0; s < 2; ++s) {
                    float v = 0.f;
                    for (int a = 0; a < 8; ++a) v = fmaf(L[p][a & 1] * L[q][(a >> 1) & 1] * L[s][(a >> 2) & 1], nn[a], v);
                    nuq[p][q][s] = v;
                }
    } else {
        for (int p = 0; p < 2; ++p)
            for (int q = 0; q < 2; ++q)
                for (int s = 0; s < 2; ++s)
                    nuq[p][q][s] = exp2f(kl_exponent(P, c, 2 * ex + p, 2 * ey + q, 2 * ez + s));
    }
    const float W = 0.125f * P.hx * P.hy * P.hz;
    const float kdir[3] = {W / (P.hx * P.hx), W / (P.hy * P.hy), W / (P.hz * P.hz)};
    for (int a = 0; a < 8; ++a) rc[a] = 0.f;
    float en = 0.f;
    for (int dir = 0; dir < 3; ++dir) {
        const int bd = 1 << dir;                       // corner bit of the derivative axis
        const int o1 = (dir == 0) ? 1 : 0, o2 = (dir == 2) ? 1 : 2;   // the two other axes (as bit positions)
        float edge[2][2];                              // edge differences, indexed by the other two corner bits
        for (int j = 0; j < 2; ++j)
            for (int k = 0; k < 2; ++k) {
                const int lo = (j << o1) | (k << o2);
                edge[j][k] = u[lo | bd] - u[lo];
            }
        for (int q = 0; q < 2; ++q)                    // Gauss point along axis o1
            for (int s = 0; s < 2; ++s) {              // Gauss point along axis o2
                float D = 0.f;
                for (int j = 0; j < 2; ++j)
                    for (int k = 0; k < 2; ++k) D = fmaf(L[q][j] * L[s][k], edge[j][k], D);
                float nsum = 0.f;
                for (int p = 0; p < 2; ++p) {
                    int idx[3]; idx[dir] = p; idx[o1] = q; idx[o2] = s;
                    nsum += nuq[idx[0]][idx[1]][idx[2]];
                }
                const float G = kdir[dir] * nsum * D;
                en = fmaf(G, D, en);
                for (int j = 0; j < 2; ++j)
                    for (int k = 0; k < 2; ++k) {
                        const int lo = (j << o1) | (k << o2);
                        const float x = L[q][j] * L[s][k] * G;
                        rc[lo | bd] += x; rc[lo] -= x;
                    }
            }
    }
    ed = 0.5f * en;
    if (fb) {
        float f[8];
        for (int a = 0; a < 8; ++a) f[a] = __ldg(fb + i0 + (a & 1) + ((a >> 1) & 1) * sy + ((a >> 2) & 1) * sz);
        el = 0.f;
        for (int p = 0; p < 2; ++p)
            for (int q = 0; q < 2; ++q)
                for (int s = 0; s < 2; ++s) {
                    float fq = 0.f, uq = 0.f, N[8];
                    for (int a = 0; a < 8; ++a) {
                        N[a] = L[p][a & 1] * L[q][(a >> 1) & 1] * L[s][(a >> 2) & 1];
                        fq = fmaf(N[a], f[a], fq); uq = fmaf(N[a], u[a], uq);
                    }
                    el = fmaf(W * fq, uq, el);
                    for (int a = 0; a < 8; ++a) rc[a] = fmaf(-W * fq, N[a], rc[a]);
                }
    } else {
        const float fw = P.f_const * W;
        el = fw * (((u[0] + u[1]) + (u[2] + u[3])) + ((u[4] + u[5]) + (u[6] + u[7])));
        for (int a = 0; a < 8; ++a) rc[a] -= fw;
    }
}

template <int DIM>
__global__ void __launch_bounds__(GEN_THREADS) generic_kernel(const Params P) {
    const int b = blockIdx.y;
    const long long node = (long long)blockIdx.x * GEN_THREADS + threadIdx.x;
    const float* ub = P.u + (long long)b * P.nodes;
    const float* nub = P.nu ? P.nu + (long long)b * P.nodes : nullptr;
    const float* fb = P.f ? P.f + (long long)b * P.nodes : nullptr;
    long long mpow = 1;
    for (int a = 0; a < DIM; ++a) mpow *= P.m;
    const float* c = P.ckl + (long long)b * mpow;
    double ed_acc = 0.0, el_acc = 0.0;
    if (node < P.nodes) {
        const int ix = (int)(node % P.nx);
        const int iy = (int)((node / P.nx) % P.ny);
        const int iz = (int)(node / ((long long)P.nx * P.ny));
        float racc = 0.f;
        for (int dz = (DIM == 3 ? -1 : 0); dz <= 0; ++dz)
            for (int dy = -1; dy <= 0; ++dy)
                for (int dx = -1; dx <= 0; ++dx) {
                    const int ex = ix + dx, ey = iy + dy, ez = iz + dz;
                    if (ex < 0 || ex >= P.nx - 1 || ey < 0 || ey >= P.ny - 1) continue;
                    if (DIM == 3 && (ez < 0 || ez >= P.nz - 1)) continue;
                    float ed, el;
                    const int corner = (-dx) | ((-dy) << 1) | ((DIM == 3 ? -dz : 0) << 2);
                    if (DIM == 2) {
                        float rc[4];
                        element2d(P, b, ex, ey, ub, nub, fb, c, rc, ed, el);
                        racc += rc[corner];
                    } else {
                        float rc[8];
                        element3d(P, b, ex, ey, ez, ub, nub, fb, c, rc, ed, el);
                        racc += rc[corner];
                    }
                    if (corner == 0) { ed_acc = (double)ed; el_acc = (double)el; }
                }
        if (P.r) {
            if (!(P.flags & DN_NO_MASK) && (ix == 0 || ix == P.nx - 1)) racc = 0.f;
            if (P.gJ) racc *= __ldg(P.gJ + b);
            P.r[(long long)b * P.nodes + node] = racc;
        }
    }
    block_reduce_store(ed_acc, el_acc, P.partials + 2 * ((long long)b * P.nblk + blockIdx.x));
}

}  // namespace

int generic_blocks_per_sample(long long nodes) { return (int)((nodes + GEN_THREADS - 1) / GEN_THREADS); }

cudaError_t launch_generic(const Params& P, cudaStream_t s) {
    dim3 grid((unsigned)P.nblk, (unsigned)P.batch);
    if (P.dim == 2) generic_kernel<2><<<grid, GEN_THREADS, 0, s>>>(P);
    else generic_kernel<3><<<grid, GEN_THREADS, 0, s>>>(P);
    return cudaGetLastError();
}

}  // namespace dn
