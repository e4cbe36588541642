// Tiled 3D kernel: fused element quadrature, energy reduction, node gather, mask and store on
// hexahedra, for DN_NU_KL_GAUSS with constant forcing.
//
// Layout of the work.  A block owns a tile of TY node rows (y) across the whole x extent
// (WX warps of 128 nodes, 4 consecutive nodes per lane) and marches over a chunk of node planes
// in z.  A thread keeps, for its 4 node columns, the state of the last staged plane in registers
// (values, x- and y-edge differences, xy twists) and stages the next plane with one 128-bit load.
// Element (x, y, k) is computed once per block by the thread of node (x, y): everything it needs
// from row y+1 (values and x-edge differences of the new plane) comes through shared memory, the
// x+1 neighbour by shuffle.  Of its 8 corner contributions, those to column x+1 go to the next
// lane by shuffle (to the next warp through shared memory), those to row y+1 through shared
// memory, those to plane k+1 are carried to the next step.  One barrier per plane: the exchange
// of a step's row-(y+1) contributions rides on the barrier of the next step, so a node plane is
// finished two steps after it was staged.  The first row of a tile and the first plane of a
// chunk are recomputed by the neighbouring block (1/TY and 1/Z redundancy).
//
// Arithmetic of one element, with the corner values u_ijk (i, j, k the x, y, z bits):
//   e = u100-u000, s = u010-u000, w = u001-u000                      (edge differences at the low corner)
//   txy, txz, tyz  second differences on the three low faces, txyz the third difference
//   d/dx at Gauss (eta q, zeta s) = ((e + q txy) + s (txz + q txyz)) / hx, and cyclically for y, z.
// With N^x_qs = sum_p nu_pqs (nu summed along the derivative's own axis) the energy is
//   1/2 sum_dir k_dir sum N D^2,  k_x = hy hz / (8 hx), ...
// and its partial derivatives with respect to (e, s, w, txy, txz, tyz, txyz) are distributed to
// the corners by the chain rule (r111 = dtxyz, r110 = dtxy - dtxyz, ..., r000 = -sum of the rest).
//
// KL diffusivity: for a fixed Gauss line (y_q, z_s) the exponent is a polynomial of degree m in
// c = cos(pi x_p); its coefficients are prepared per block in double (shared memory).
#include "dn_internal.cuh"

namespace dn {

namespace {

constexpr int T3_THREADS = 512;

__device__ __forceinline__ float ex2_approx3(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int M> struct Gs3 { static constexpr int value = ((M + 1) + 3) / 4 * 4; };

template <int M>
__device__ __forceinline__ float horner3(const float* g, float c) {
    float e = g[M];
#pragma unroll
    for (int k = M - 1; k >= 0; --k) e = fmaf(e, c, g[k]);
    return e;
}

struct Contrib { float r000, r100, r010, r110, r001, r101, r011, r111; };

// One element.  nu[p][q][s]: p, q, s index the Gauss point along x, y, z.
__device__ __forceinline__ void element3(float e0, float s0, float w0, float txy, float txz, float tyz, float txyz,
                                         const float (&nu)[2][2][2], bool iso, float kx, float ky, float kz,
                                         Contrib& o, float& en) {
    const float a = DN_GA, b = DN_GB;
    // d/dx (times hx) at (q, s)
    const float Axa = fmaf(a, txy, e0), Axb = fmaf(b, txy, e0);
    const float Bxa = fmaf(a, txyz, txz), Bxb = fmaf(b, txyz, txz);
    const float Dx_aa = fmaf(a, Bxa, Axa), Dx_ab = fmaf(b, Bxa, Axa), Dx_ba = fmaf(a, Bxb, Axb), Dx_bb = fmaf(b, Bxb, Axb);
    // d/dy (times hy) at (p, s)
    const float Aya = fmaf(a, txy, s0), Ayb = fmaf(b, txy, s0);
    const float Bya = fmaf(a, txyz, tyz), Byb = fmaf(b, txyz, tyz);
    const float Dy_aa = fmaf(a, Bya, Aya), Dy_ab = fmaf(b, Bya, Aya), Dy_ba = fmaf(a, Byb, Ayb), Dy_bb = fmaf(b, Byb, Ayb);
    // d/dz (times hz) at (p, q): (w + p txz) + q (tyz + p txyz)
    const float Aza = fmaf(a, txz, w0), Azb = fmaf(b, txz, w0);
    const float Dz_aa = fmaf(a, Bya, Aza), Dz_ab = fmaf(b, Bya, Aza), Dz_ba = fmaf(a, Byb, Azb), Dz_bb = fmaf(b, Byb, Azb);
    // nu summed along the derivative's own axis
    float Nx_aa = nu[0][0][0] + nu[1][0][0], Nx_ab = nu[0][0][1] + nu[1][0][1];     // (q, s)
    float Nx_ba = nu[0][1][0] + nu[1][1][0], Nx_bb = nu[0][1][1] + nu[1][1][1];
    float Ny_aa = nu[0][0][0] + nu[0][1][0], Ny_ab = nu[0][0][1] + nu[0][1][1];     // (p, s)
    float Ny_ba = nu[1][0][0] + nu[1][1][0], Ny_bb = nu[1][0][1] + nu[1][1][1];
    float Nz_aa = nu[0][0][0] + nu[0][0][1], Nz_ab = nu[0][1][0] + nu[0][1][1];     // (p, q)
    float Nz_ba = nu[1][0][0] + nu[1][0][1], Nz_bb = nu[1][1][0] + nu[1][1][1];
    if (!iso) {
        Nx_aa *= kx; Nx_ab *= kx; Nx_ba *= kx; Nx_bb *= kx;
        Ny_aa *= ky; Ny_ab *= ky; Ny_ba *= ky; Ny_bb *= ky;
        Nz_aa *= kz; Nz_ab *= kz; Nz_ba *= kz; Nz_bb *= kz;
    }
    const float Gx_aa = Nx_aa * Dx_aa, Gx_ab = Nx_ab * Dx_ab, Gx_ba = Nx_ba * Dx_ba, Gx_bb = Nx_bb * Dx_bb;
    const float Gy_aa = Ny_aa * Dy_aa, Gy_ab = Ny_ab * Dy_ab, Gy_ba = Ny_ba * Dy_ba, Gy_bb = Ny_bb * Dy_bb;
    const float Gz_aa = Nz_aa * Dz_aa, Gz_ab = Nz_ab * Dz_ab, Gz_ba = Nz_ba * Dz_ba, Gz_bb = Nz_bb * Dz_bb;
    float acc = Gx_aa * Dx_aa;
    acc = fmaf(Gx_ab, Dx_ab, acc); acc = fmaf(Gx_ba, Dx_ba, acc); acc = fmaf(Gx_bb, Dx_bb, acc);
    acc = fmaf(Gy_aa, Dy_aa, acc); acc = fmaf(Gy_ab, Dy_ab, acc); acc = fmaf(Gy_ba, Dy_ba, acc); acc = fmaf(Gy_bb, Dy_bb, acc);
    acc = fmaf(Gz_aa, Dz_aa, acc); acc = fmaf(Gz_ab, Dz_ab, acc); acc = fmaf(Gz_ba, Dz_ba, acc); acc = fmaf(Gz_bb, Dz_bb, acc);
    en += acc;
    // adjoint of the three interpolations
    const float AXa = Gx_aa + Gx_ab, AXb = Gx_ba + Gx_bb;
    const float BXa = fmaf(b, Gx_ab, a * Gx_aa), BXb = fmaf(b, Gx_bb, a * Gx_ba);
    const float AYa = Gy_aa + Gy_ab, AYb = Gy_ba + Gy_bb;
    const float BYa = fmaf(b, Gy_ab, a * Gy_aa), BYb = fmaf(b, Gy_bb, a * Gy_ba);
    const float AZa = Gz_aa + Gz_ab, AZb = Gz_ba + Gz_bb;
    const float BZa = fmaf(b, Gz_ab, a * Gz_aa), BZb = fmaf(b, Gz_bb, a * Gz_ba);
    const float dE = AXa + AXb, dS = AYa + AYb, dW = AZa + AZb;
    float dXY = fmaf(b, AXb, a * AXa);
    dXY = fmaf(a, AYa, dXY); dXY = fmaf(b, AYb, dXY);
    float dXZ = BXa + BXb;
    dXZ = fmaf(a, AZa, dXZ); dXZ = fmaf(b, AZb, dXZ);
    float dYZ = (BYa + BYb) + (BZa + BZb);
    float dXYZ = fmaf(b, BXb, a * BXa);
    dXYZ = fmaf(a, BYa, dXYZ); dXYZ = fmaf(b, BYb, dXYZ);
    dXYZ = fmaf(a, BZa, dXYZ); dXYZ = fmaf(b, BZb, dXYZ);
    // chain rule to the corners
    o.r111 = dXYZ;
    o.r110 = dXY - dXYZ;
    o.r101 = dXZ - dXYZ;
    o.r011 = dYZ - dXYZ;
    o.r100 = (dE - o.r110) - dXZ;
    o.r010 = (dS - o.r110) - dYZ;
    o.r001 = (dW - o.r101) - dYZ;
    o.r000 = ((o.r011 - dW) + (dXY - dE)) + (dXZ - dS);
}

template <int M, bool WANT_R>
__global__ void __launch_bounds__(T3_THREADS, 1)
tiled3d_kernel(const Params P, const int WX, const int TY, const int Z, const int ntile_y) {
    extern __shared__ __align__(16) float smem[];
    constexpr int GS = Gs3<M>::value;
    const int lane = threadIdx.x & 31;
    const int wid = threadIdx.x >> 5;
    const int wx = wid % WX, ty = wid / WX;
    const int b = blockIdx.y;
    const int tile = blockIdx.x % ntile_y, zc = blockIdx.x / ntile_y;
    const int nx = P.nx, ny = P.ny, nz = P.nz;
    const int NXP = WX * 128;
    const int y0 = tile * (TY - 1);
    const int y = y0 + ty;                             // node row and element row of this thread
    const int x0 = wx * 128 + 4 * lane;
    const int p0 = zc * Z, p1 = min(p0 + Z, nz);
    const int kbeg = max(p0 - 1, 0), kend = min(p1 - 1, nz - 2);
    const bool col_ok = x0 < nx;
    const bool elem_row_ok = (y < ny - 1);
    const bool node_row_ok = (y < ny);
    const bool out_row = node_row_ok && (ty >= 1 || tile == 0);
    const bool top_row = (ty == TY - 1);

    // shared memory: two exchange buffers, then the KL coefficients of every Gauss line of the block
    const int XOFF = 4 * TY * NXP;                     // floats before the cross-warp slots
    const int BUF = XOFF + TY * WX * 4;
    float* gam = smem + 2 * BUF;

    // ---- prologue: KL polynomial coefficients for the Gauss lines (row q, plane s) of the block
    {
        const int nlines = (kend - kbeg + 1) * TY * 4;
        const float* c = P.ckl + (size_t)b * M * M * M;
        for (int t = threadIdx.x; t < nlines; t += blockDim.x) {
            const int s = t & 1, q = (t >> 1) & 1, row = (t >> 2) % TY, kk = (t >> 2) / TY;
            const int gy = min(2 * (y0 + row) + q, 2 * (ny - 1) - 1);
            const int gz = 2 * (kbeg + kk) + s;
            double g[M];
#pragma unroll
            for (int i = 0; i < M; ++i) {
                double acc = 0.0;
#pragma unroll
                for (int j = 0; j < M; ++j) {
                    double inner = 0.0;
#pragma unroll
                    for (int k = 0; k < M; ++k)
                        inner += (double)c[(i * M + j) * M + k] * (double)P.cg[2][k * P.gstride[2] + gz];
                    acc += inner * (double)P.cg[1][j * P.gstride[1] + gy];
                }
                g[i] = acc;
            }
            double acc[M + 1], tp[M + 1], tc[M + 1];
#pragma unroll
            for (int k = 0; k <= M; ++k) { acc[k] = 0.0; tp[k] = (k == 0) ? 1.0 : 0.0; tc[k] = (k == 1) ? 1.0 : 0.0; }
#pragma unroll
            for (int i = 1; i <= M; ++i) {
#pragma unroll
                for (int k = 0; k <= M; ++k) acc[k] += g[i - 1] * tc[k];
                double tn[M + 1];
#pragma unroll
                for (int k = 0; k <= M; ++k) tn[k] = ((k > 0) ? 2.0 * tc[k - 1] : 0.0) - tp[k];
#pragma unroll
                for (int k = 0; k <= M; ++k) { tp[k] = tc[k]; tc[k] = tn[k]; }
            }
#pragma unroll
            for (int k = 0; k < GS; ++k) gam[(size_t)t * GS + k] = (k <= M) ? (float)acc[k <= M ? k : 0] : 0.f;
        }
    }

    const bool iso = (P.hx == P.hy) && (P.hy == P.hz);
    const float W8 = 0.125f * P.hx * P.hy * P.hz;
    const float kx = W8 / (P.hx * P.hx), ky = W8 / (P.hy * P.hy), kz = W8 / (P.hz * P.hz);
    const float kap = iso ? kx : 1.f;                  // isotropic cells: one scale applied at the end
    const bool nomask = (P.flags & DN_NO_MASK) != 0;
    const bool impose = (P.flags & DN_IMPOSE_BC_ON_LOAD) != 0;
    const float gs = (WANT_R && P.gJ) ? __ldg(P.gJ + b) : 1.f;
    const float fw = P.f_const * P.hx * P.hy * P.hz;  // nodal load of an interior node
    const float wy = (y == 0 || y == ny - 1) ? 0.5f : 1.f;
    const bool first_col = (x0 == 0), last_col = (x0 + 3 == nx - 1);
    const bool last_elem_missing = (x0 + 3 >= nx - 1);  // element right of node x0+3 does not exist

    const int yl = min(y, ny - 1);                     // rows beyond the grid load a valid address; unused
    const int ya = min(y + 1, ny - 1);
    const float* ub = P.u + (size_t)b * P.nodes;
    float* rb = WANT_R ? P.r + (size_t)b * P.nodes : nullptr;
    const size_t plane = (size_t)nx * ny;

    float cpa[4], cpb[4];
    if (col_ok) {
        const float4 q0 = __ldg(reinterpret_cast<const float4*>(P.cg[0] + 2 * x0));
        const float4 q1 = __ldg(reinterpret_cast<const float4*>(P.cg[0] + 2 * x0 + 4));
        cpa[0] = q0.x; cpb[0] = q0.y; cpa[1] = q0.z; cpb[1] = q0.w;
        cpa[2] = q1.x; cpb[2] = q1.y; cpa[3] = q1.z; cpb[3] = q1.w;
    } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) { cpa[c] = 0.f; cpb[c] = 0.f; }
    }

    // ---- register state: plane kp = the last staged plane
    float uk[4], ek[4], sk[4], txyk[4];
    float L0p[4], U0p[4], carry[4], L1p[4], U1p[4], Xp[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        uk[c] = ek[c] = sk[c] = txyk[c] = 0.f;
        L0p[c] = U0p[c] = carry[c] = L1p[c] = U1p[c] = Xp[c] = 0.f;
    }
    float en = 0.f, enl = 0.f, ell = 0.f;

    auto load_own = [&](int p, float (&v)[4], float& halo) {
        if (col_ok) {
            const float4 q = __ldg(reinterpret_cast<const float4*>(ub + (size_t)p * plane + (size_t)yl * nx + x0));
            v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
        } else {
            v[0] = v[1] = v[2] = v[3] = 0.f;
        }
        halo = (lane == 31 && x0 + 4 < nx) ? __ldg(ub + (size_t)p * plane + (size_t)yl * nx + x0 + 4) : 0.f;
        if (impose) {
            if (first_col) v[0] = P.bc_x0;
            if (last_col) v[3] = P.bc_x1;
        }
    };
    auto load_above = [&](int p, float (&v)[4], float& halo) {   // row y+1, top warp row of the tile only
        if (col_ok) {
            const float4 q = __ldg(reinterpret_cast<const float4*>(ub + (size_t)p * plane + (size_t)ya * nx + x0));
            v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
        } else {
            v[0] = v[1] = v[2] = v[3] = 0.f;
        }
        halo = (lane == 31 && x0 + 4 < nx) ? __ldg(ub + (size_t)p * plane + (size_t)ya * nx + x0 + 4) : 0.f;
        if (impose) {
            if (first_col) v[0] = P.bc_x0;
            if (last_col) v[3] = P.bc_x1;
        }
    };
    auto xdiffs = [&](const float (&v)[4], float halo, float (&e)[4]) {
        float rn = __shfl_down_sync(0xffffffffu, v[0], 1);
        if (lane == 31) rn = halo;
        e[0] = v[1] - v[0]; e[1] = v[2] - v[1]; e[2] = v[3] - v[2]; e[3] = rn - v[3];
    };

    float un[4], unh, ua[4], uah;
    load_own(kbeg, un, unh);
    if (top_row) load_above(kbeg, ua, uah);

    // iteration p stages node plane p, computes element plane p-1, finishes node plane p-2
    for (int p = kbeg; p <= kend + 2; ++p) {
        const int par = p & 1;
        float* sb = smem + par * BUF;
        float* su = sb + (0 * TY + ty) * NXP + x0;
        float* se = sb + (1 * TY + ty) * NXP + x0;
        float* sL = sb + (2 * TY + ty) * NXP + x0;
        float* sU = sb + (3 * TY + ty) * NXP + x0;
        float* sX = sb + XOFF + (ty * WX + wx) * 4;
        const bool stage = (p <= kend + 1);
        float ep[4], vn[4], vnh, va[4], vah;
        if (stage) {
            xdiffs(un, unh, ep);
            if (col_ok) {
                *reinterpret_cast<float4*>(su) = make_float4(un[0], un[1], un[2], un[3]);
                *reinterpret_cast<float4*>(se) = make_float4(ep[0], ep[1], ep[2], ep[3]);
            }
            if (p + 1 <= kend + 1) {                   // prefetch the next plane
                load_own(p + 1, vn, vnh);
                if (top_row) load_above(p + 1, va, vah);
            }
            // load energy of the staged plane (owned planes and rows only)
            if (p >= p0 && p < p1 && out_row) {
                float rs = (un[0] + un[1]) + (un[2] + un[3]);
                if (first_col) rs -= 0.5f * un[0];
                if (last_col) rs -= 0.5f * un[3];
                const float wz = (p == 0 || p == nz - 1) ? 0.5f : 1.f;
                ell = fmaf(fw * wy * wz, rs, ell);
            }
        }
        if (WANT_R && col_ok) {                        // contributions of the previous element step to row y+1
            *reinterpret_cast<float4*>(sL) = make_float4(L1p[0], L1p[1], L1p[2], L1p[3]);
            *reinterpret_cast<float4*>(sU) = make_float4(U1p[0], U1p[1], U1p[2], U1p[3]);
            if (lane == 31) *reinterpret_cast<float4*>(sX) = make_float4(Xp[0], Xp[1], Xp[2], Xp[3]);
        }
        __syncthreads();

        // ---- finish node plane p-2 with what row y-1 (and the warp on the left) sent
        if (WANT_R && p - 2 >= kbeg) {
            float l1[4] = {0.f, 0.f, 0.f, 0.f}, u1[4] = {0.f, 0.f, 0.f, 0.f};
            if (ty > 0 && col_ok) {
                const float4 a = *reinterpret_cast<const float4*>(sL - NXP);
                const float4 c4 = *reinterpret_cast<const float4*>(sU - NXP);
                l1[0] = a.x; l1[1] = a.y; l1[2] = a.z; l1[3] = a.w;
                u1[0] = c4.x; u1[1] = c4.y; u1[2] = c4.z; u1[3] = c4.w;
            }
            if (lane == 0 && wx > 0) {                 // left warp's last element: (r100, r110, r101, r111)
                const float4 me = *reinterpret_cast<const float4*>(sX - 4);
                l1[0] += me.x; u1[0] += me.z;          // to this row: r100 (lower plane), r101 (upper plane)
                if (ty > 0) {
                    const float4 bl = *reinterpret_cast<const float4*>(sX - 4 - WX * 4);
                    l1[0] += bl.y; u1[0] += bl.w;      // from the row below: r110, r111
                }
            }
            const int pl = p - 2;                      // the plane being finished
            const bool own_plane = (pl >= p0);
            const float wz = (pl == 0 || pl == nz - 1) ? 0.5f : 1.f;
            const float lw = fw * wy * wz;
            const float sc = gs * kap, nl = -gs * lw;
            float o[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float raw = (L0p[c] + l1[c]) + carry[c];
                carry[c] = U0p[c] + u1[c];
                o[c] = fmaf(sc, raw, nl);
                if (c == 0 && first_col) o[c] = nomask ? fmaf(sc, raw, 0.5f * nl) : 0.f;
                if (c == 3 && last_col) o[c] = nomask ? fmaf(sc, raw, 0.5f * nl) : 0.f;
            }
            if (own_plane && out_row && col_ok && pl <= kend)
                *reinterpret_cast<float4*>(rb + (size_t)pl * plane + (size_t)y * nx + x0) = make_float4(o[0], o[1], o[2], o[3]);
        }

        // ---- finish staging plane p (needs row y+1) and compute element plane p-1
        if (stage) {
            float uab[4], eab[4];
            if (!top_row) {
                if (col_ok) {
                    const float4 a = *reinterpret_cast<const float4*>(su + NXP);
                    const float4 c4 = *reinterpret_cast<const float4*>(se + NXP);
                    uab[0] = a.x; uab[1] = a.y; uab[2] = a.z; uab[3] = a.w;
                    eab[0] = c4.x; eab[1] = c4.y; eab[2] = c4.z; eab[3] = c4.w;
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c) { uab[c] = 0.f; eab[c] = 0.f; }
                }
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c) uab[c] = ua[c];
                xdiffs(ua, uah, eab);
            }
            float sp[4], txyp[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) { sp[c] = uab[c] - un[c]; txyp[c] = eab[c] - ep[c]; }

            if (p > kbeg) {
                const int k = p - 1;
                const bool own_step = (k >= p0);      // the warm-up step only seeds the carried contributions
                Contrib prev;
                float l1n[4], u1n[4];
                prev.r100 = prev.r110 = prev.r101 = prev.r111 = 0.f;
                const float* gl = gam + ((size_t)((k - kbeg) * TY + ty) * 4) * GS;
                float g_aa[GS], g_ab[GS], g_ba[GS], g_bb[GS];      // (q, s) lines
#pragma unroll
                for (int i = 0; i < GS / 4; ++i) {
                    const float4 t0 = reinterpret_cast<const float4*>(gl)[i];
                    const float4 t1 = reinterpret_cast<const float4*>(gl + GS)[i];
                    const float4 t2 = reinterpret_cast<const float4*>(gl + 2 * GS)[i];
                    const float4 t3 = reinterpret_cast<const float4*>(gl + 3 * GS)[i];
                    g_aa[4 * i] = t0.x; g_aa[4 * i + 1] = t0.y; g_aa[4 * i + 2] = t0.z; g_aa[4 * i + 3] = t0.w;
                    g_ab[4 * i] = t1.x; g_ab[4 * i + 1] = t1.y; g_ab[4 * i + 2] = t1.z; g_ab[4 * i + 3] = t1.w;
                    g_ba[4 * i] = t2.x; g_ba[4 * i + 1] = t2.y; g_ba[4 * i + 2] = t2.z; g_ba[4 * i + 3] = t2.w;
                    g_bb[4 * i] = t3.x; g_bb[4 * i + 1] = t3.y; g_bb[4 * i + 2] = t3.z; g_bb[4 * i + 3] = t3.w;
                }
                float enrow = 0.f, enlast = 0.f;
                if (elem_row_ok) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        float nu[2][2][2];
                        nu[0][0][0] = ex2_approx3(horner3<M>(g_aa, cpa[c])); nu[1][0][0] = ex2_approx3(horner3<M>(g_aa, cpb[c]));
                        nu[0][0][1] = ex2_approx3(horner3<M>(g_ab, cpa[c])); nu[1][0][1] = ex2_approx3(horner3<M>(g_ab, cpb[c]));
                        nu[0][1][0] = ex2_approx3(horner3<M>(g_ba, cpa[c])); nu[1][1][0] = ex2_approx3(horner3<M>(g_ba, cpb[c]));
                        nu[0][1][1] = ex2_approx3(horner3<M>(g_bb, cpa[c])); nu[1][1][1] = ex2_approx3(horner3<M>(g_bb, cpb[c]));
                        Contrib o;
                        float e1 = 0.f;
                        element3(ek[c], sk[c], un[c] - uk[c], txyk[c], ep[c] - ek[c], sp[c] - sk[c], txyp[c] - txyk[c],
                                 nu, iso, kx, ky, kz, o, e1);
                        if (c == 3) enlast = e1; else enrow += e1;
                        if (WANT_R) {
                            if (c == 3 && last_elem_missing) {
                                o.r000 = o.r100 = o.r010 = o.r110 = o.r001 = o.r101 = o.r011 = o.r111 = 0.f;
                            }
                            if (c > 0) {
                                L0p[c] = o.r000 + prev.r100; l1n[c] = o.r010 + prev.r110;
                                U0p[c] = o.r001 + prev.r101; u1n[c] = o.r011 + prev.r111;
                            } else {
                                L0p[0] = o.r000; l1n[0] = o.r010; U0p[0] = o.r001; u1n[0] = o.r011;
                            }
                            prev = o;
                        }
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c) { L0p[c] = 0.f; l1n[c] = 0.f; U0p[c] = 0.f; u1n[c] = 0.f; }
                }
                if (WANT_R) {
                    // the left neighbour's last element feeds this thread's first node column
                    const float a100 = __shfl_up_sync(0xffffffffu, prev.r100, 1), a110 = __shfl_up_sync(0xffffffffu, prev.r110, 1);
                    const float a101 = __shfl_up_sync(0xffffffffu, prev.r101, 1), a111 = __shfl_up_sync(0xffffffffu, prev.r111, 1);
                    if (lane > 0) { L0p[0] += a100; l1n[0] += a110; U0p[0] += a101; u1n[0] += a111; }
                    Xp[0] = prev.r100; Xp[1] = prev.r110; Xp[2] = prev.r101; Xp[3] = prev.r111;
#pragma unroll
                    for (int c = 0; c < 4; ++c) { L1p[c] = l1n[c]; U1p[c] = u1n[c]; }
                }
                if (own_step && elem_row_ok) {
                    // energy of element row y belongs to the tile that computes it as a non-halo row
                    if (ty >= 1 || tile == 0) {
                        en += enrow;
                        if (!last_elem_missing) enl += enlast;
                    }
                }
            }
            // the staged plane becomes the state
#pragma unroll
            for (int c = 0; c < 4; ++c) { uk[c] = un[c]; ek[c] = ep[c]; sk[c] = sp[c]; txyk[c] = txyp[c]; }
            if (p + 1 <= kend + 1) {
#pragma unroll
                for (int c = 0; c < 4; ++c) un[c] = vn[c];
                unh = vnh;
                if (top_row) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) ua[c] = va[c];
                    uah = vah;
                }
            }
        } else if (WANT_R) {
#pragma unroll
            for (int c = 0; c < 4; ++c) { L0p[c] = 0.f; U0p[c] = 0.f; L1p[c] = 0.f; U1p[c] = 0.f; Xp[c] = 0.f; }
        }
    }

    // ---- the top node plane of the domain has no element plane above it: it is what was carried
    if (WANT_R && p1 == nz && out_row && col_ok) {
        const float lw = fw * wy * 0.5f;
        const float sc = gs * kap, nl = -gs * lw;
        float o[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            o[c] = fmaf(sc, carry[c], nl);
            if (c == 0 && first_col) o[c] = nomask ? fmaf(sc, carry[c], 0.5f * nl) : 0.f;
            if (c == 3 && last_col) o[c] = nomask ? fmaf(sc, carry[c], 0.5f * nl) : 0.f;
        }
        *reinterpret_cast<float4*>(rb + (size_t)(nz - 1) * plane + (size_t)y * nx + x0) = make_float4(o[0], o[1], o[2], o[3]);
    }
    const double etot = 0.5 * (double)kap * ((double)en + (double)enl);
    block_reduce_store(etot, (double)ell, P.partials + 2 * ((size_t)b * P.nblk + blockIdx.x));
}

struct Geo3 { int WX, TY, Z, ntile_y, nchunk_z, GS; size_t smem; };

int sm_count3() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
        (void)cudaGetLastError();
        n = 148;
    }
    return n;
}

Geo3 geometry3(const dn_problem& p) {
    Geo3 g{};
    const int nx = p.grid.nx, ny = p.grid.ny, nz = p.grid.nz;
    g.WX = (nx + 127) / 128;
    g.TY = (T3_THREADS / 32) / g.WX;
    if (g.TY > ny) g.TY = (ny < 2) ? 2 : ny;
    g.ntile_y = (ny - 1 + (g.TY - 1) - 1) / (g.TY - 1);
    const int m = p.kl_modes;
    g.GS = ((m + 1) + 3) / 4 * 4;
    const long long slots = sm_count3();
    const size_t fixed = sizeof(float) * 2 * ((size_t)4 * g.TY * g.WX * 128 + (size_t)g.TY * g.WX * 4);
    long long best = -1;
    int bestZ = 8;
    for (int Z = 4; Z <= 256; ++Z) {
        if (Z > nz && Z > 4) break;
        const size_t sm = fixed + sizeof(float) * (size_t)(Z + 1) * g.TY * 4 * g.GS;
        if (sm > 200 * 1024) break;
        const long long nch = (nz + Z - 1) / Z;
        const long long blocks = (long long)p.batch * g.ntile_y * nch;
        const long long waves = (blocks + slots - 1) / slots;
        const long long cost = waves * (Z + 3) * 1000 + 1000 / Z;
        if (best < 0 || cost < best) { best = cost; bestZ = Z; }
    }
    g.Z = bestZ;
    g.nchunk_z = (nz + g.Z - 1) / g.Z;
    g.smem = fixed + sizeof(float) * (size_t)(g.Z + 1) * g.TY * 4 * g.GS;
    return g;
}

template <int M>
cudaError_t launch_m(const Params& P, const Geo3& g, cudaStream_t s) {
    dim3 grid((unsigned)(g.ntile_y * g.nchunk_z), (unsigned)P.batch);
    const int threads = 32 * g.WX * g.TY;
    cudaError_t e;
    if (P.r) {
        e = cudaFuncSetAttribute(tiled3d_kernel<M, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g.smem);
        if (e != cudaSuccess) return e;
        tiled3d_kernel<M, true><<<grid, threads, g.smem, s>>>(P, g.WX, g.TY, g.Z, g.ntile_y);
    } else {
        e = cudaFuncSetAttribute(tiled3d_kernel<M, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g.smem);
        if (e != cudaSuccess) return e;
        tiled3d_kernel<M, false><<<grid, threads, g.smem, s>>>(P, g.WX, g.TY, g.Z, g.ntile_y);
    }
    return cudaGetLastError();
}

}  // namespace

bool tiled3d_applicable(const dn_problem& p) {
    return p.grid.dim == 3 && p.nu_mode == DN_NU_KL_GAUSS && p.grid.nx % 4 == 0 && p.grid.nx >= 8 && p.grid.nx <= 512 &&
           p.grid.ny >= 2 && p.grid.nz >= 2;
}

Launch tiled3d_geometry(const dn_problem& p) {
    const Geo3 g = geometry3(p);
    Launch l{};
    l.path = PATH_TILED3D;
    l.nblk = g.ntile_y * g.nchunk_z;
    l.chunk = g.Z;
    l.variant = g.TY;
    return l;
}

cudaError_t launch_tiled3d(const Params& P, const Launch& l, cudaStream_t s) {
    dn_problem p{};
    p.grid.dim = 3; p.grid.nx = P.nx; p.grid.ny = P.ny; p.grid.nz = P.nz; p.batch = P.batch;
    p.nu_mode = P.nu_mode; p.kl_modes = P.m;
    const Geo3 g = geometry3(p);
    (void)l;
    switch (P.m) {
        case 1: return launch_m<1>(P, g, s);
        case 2: return launch_m<2>(P, g, s);
        case 3: return launch_m<3>(P, g, s);
        case 4: return launch_m<4>(P, g, s);
        case 5: return launch_m<5>(P, g, s);
        case 6: return launch_m<6>(P, g, s);
        case 7: return launch_m<7>(P, g, s);
        case 8: return launch_m<8>(P, g, s);
    }
    return cudaErrorInvalidValue;
}

}  // namespace dn
