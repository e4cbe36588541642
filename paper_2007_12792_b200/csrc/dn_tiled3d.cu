// Tiled 3D kernel: fused element quadrature, energy reduction, node gather, mask and store on
// hexahedra, for both diffusivity modes, with constant forcing.
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
// finished two steps after it was staged.  Tiles do not overlap in y: the top element row of a
// tile writes what it contributes to the next tile's first node row into a global scratch array
// (seam), and a small second kernel adds those rows to r in a fixed order.  The first plane of a z
// chunk is recomputed by the chunk below (1/Z redundancy).
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

typedef unsigned long long u64;

__device__ __forceinline__ void unpack2_3(u64 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ u64 fma2_3(u64 a, u64 b, u64 c) {
    u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

// Register state of one staged node plane, for the 4 node columns of a thread.
struct PlaneState {
    float u[4], h, e[4], s[4], txy[4];     // h: node right of the strip (lane 31)
    float n[4], nh;                        // nodal mode: staged diffusivity of the own row (prefetch target)
    float v[4][4];                         // nodal mode: nu interpolated to the 4 (xi, eta) points of each element, on this plane
};

// Floats per Gauss row pair (q fixed, s = a and b interleaved) in the coefficient table.
template <int M> struct Gs3p { static constexpr int value = (2 * (M + 1) + 3) / 4 * 4; };

template <int M, bool WANT_R, bool FULL, bool NARROW>
__global__ void __launch_bounds__(T3_THREADS, 1)
tiled3d_kernel(const Params P, const int WX, const int TY, const int Z, const int ntile_y, const int LWarg) {
    extern __shared__ __align__(16) float smem[];
    constexpr bool KL = (M > 0);
    constexpr int MM = KL ? M : 1;
    constexpr int GS = Gs3p<MM>::value;                 // floats per (row q) line pair
    constexpr int NARR = KL ? 4 : 5;                    // exchange arrays: u, e, L1, U1 (, nu)
    const int lane = threadIdx.x & 31;
    const int wid = threadIdx.x >> 5;
    // A node row takes LW lanes: 32, or (NARROW) 16 / 8 on grids with nx <= 64 / 32, where a warp then holds 2 / 4 rows
    const int LW = NARROW ? LWarg : 32;
    const int lx = lane & (LW - 1), sub = lane / LW;
    const bool firstl = (lx == 0), lastl = (lx == LW - 1);
    const int wx = wid % WX, ty = (wid / WX) * (32 / LW) + sub;
    const int b = blockIdx.y;
    const int tile = blockIdx.x % ntile_y, zc = blockIdx.x / ntile_y;
    const int nx = P.nx, ny = P.ny, nz = P.nz;
    const int NXP = WX * 128;
    const int y0 = tile * TY;
    const int y = y0 + ty;                             // node row and element row of this thread
    const int x0 = wx * 128 + 4 * lx;
    const int p0 = zc * Z, p1 = min(p0 + Z, nz);
    const int kbeg = max(p0 - 1, 0), kend = min(p1 - 1, nz - 2);
    const bool col_ok = FULL || (x0 < nx);
    const bool elem_row_ok = (y < ny - 1);
    const bool out_row = (y < ny);
    const bool top_row = (ty == TY - 1);
    const bool warp_top = ((wid / WX + 1) * (32 / LW) == TY);       // this warp holds the tile's top row (uniform per warp)
    // the top element row of a tile also feeds the first node row of the next tile: through global scratch
    const bool seam_row = WANT_R && top_row && (tile + 1 < ntile_y) && (y + 1 < ny);

    // shared memory: two exchange buffers, then the KL coefficients of every Gauss line of the block
    const int TYNXP = TY * NXP;
    const int XOFF = NARR * TYNXP;                     // floats before the cross-warp slots
    const int BUF = XOFF + TY * WX * 4;
    float* gam = smem + 2 * BUF;

    // ---- prologue: KL polynomial coefficients; table index ((k - kbeg) * TY + row) * 2 + q, entries
    // interleave the two Gauss planes s = a, b of the element plane: [coef][s]
    if constexpr (KL) {
        const int nlines = (kend - kbeg + 1) * TY * 4;
        const float* c = P.ckl + (size_t)b * M * M * M;
        for (int t = threadIdx.x; t < nlines; t += blockDim.x) {
            const int s = t & 1, q = (t >> 1) & 1, row = (t >> 2) % TY, kk = (t >> 2) / TY;
            const int gy = min(2 * (y0 + row) + q, 2 * (ny - 1) - 1);
            const int gz = 2 * (kbeg + kk) + s;
            double g[MM];
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
            double acc[MM + 1], tp[MM + 1], tc[MM + 1];
#pragma unroll
            for (int k = 0; k <= M; ++k) { acc[k] = 0.0; tp[k] = (k == 0) ? 1.0 : 0.0; tc[k] = (k == 1) ? 1.0 : 0.0; }
#pragma unroll
            for (int i = 1; i <= M; ++i) {
#pragma unroll
                for (int k = 0; k <= M; ++k) acc[k] += g[i - 1] * tc[k];
                double tn[MM + 1];
#pragma unroll
                for (int k = 0; k <= M; ++k) tn[k] = ((k > 0) ? 2.0 * tc[k - 1] : 0.0) - tp[k];
#pragma unroll
                for (int k = 0; k <= M; ++k) { tp[k] = tc[k]; tc[k] = tn[k]; }
            }
            float* dst = gam + (size_t)(t >> 1) * GS + s;
#pragma unroll
            for (int k = 0; k <= M; ++k) dst[2 * k] = (float)acc[k];
        }
    }

    const bool iso = (P.hx == P.hy) && (P.hy == P.hz);
    const float W8 = 0.125f * P.hx * P.hy * P.hz;
    const float kx = W8 / (P.hx * P.hx), ky = W8 / (P.hy * P.hy), kz = W8 / (P.hz * P.hz);
    const float kap = iso ? kx : 1.f;                  // isotropic cells: one scale applied at the end
    const bool nomask = (P.flags & DN_NO_MASK) != 0;
    const bool impose = (P.flags & DN_IMPOSE_BC_ON_LOAD) != 0;
    const float bc0 = P.bc0_b ? __ldg(P.bc0_b + b) : P.bc_x0, bc1 = P.bc1_b ? __ldg(P.bc1_b + b) : P.bc_x1;
    const float gs = (WANT_R && P.gJ) ? __ldg(P.gJ + b) : 1.f;
    const float fw = P.f_const * P.hx * P.hy * P.hz;  // nodal load of an interior node
    const bool hasf = (P.f_const != 0.f);
    const float wy = (y == 0 || y == ny - 1) ? 0.5f : 1.f;
    const bool first_col = (x0 == 0), last_col = (x0 + 3 == nx - 1);
    const bool last_elem_missing = (x0 + 3 >= nx - 1);  // element right of node x0+3 does not exist
    const bool halo_ok = lastl && (x0 + 4 < nx);
    const float mfirst = first_col ? 0.f : 1.f, mlast = last_col ? 0.f : 1.f;

    const int yl = min(y, ny - 1);                     // rows beyond the grid load a valid address; unused
    const int ya = min(y + 1, ny - 1);
    const size_t plane = (size_t)nx * ny;
    const float* pu = P.u + (size_t)b * P.nodes + (size_t)yl * nx + x0;      // own row, plane 0
    const float* pa = P.u + (size_t)b * P.nodes + (size_t)ya * nx + x0;      // row above (top warp row only)
    const float* pn = KL ? nullptr : P.nu + (size_t)b * P.nodes + (size_t)yl * nx + x0;
    const float* pna = KL ? nullptr : P.nu + (size_t)b * P.nodes + (size_t)ya * nx + x0;
    float* pseam = seam_row ? P.seam + (((size_t)b * (ntile_y - 1) + tile) * nz) * nx + x0 : nullptr;
    float* pr = WANT_R ? P.r + (size_t)b * P.nodes + (size_t)yl * nx + x0 : nullptr;

    // cos(pi x) at the two Gauss columns of each element as duplicated pairs (ca, ca, cb, cb), kept in shared memory
    float4* cps = reinterpret_cast<float4*>(gam + (size_t)(Z + 1) * TY * 2 * GS) + threadIdx.x;
    const int cstr = blockDim.x;
    if constexpr (KL) {
        float4 q0 = make_float4(0.f, 0.f, 0.f, 0.f), q1 = q0;
        if (col_ok) {
            q0 = __ldg(reinterpret_cast<const float4*>(P.cg[0] + 2 * x0));
            q1 = __ldg(reinterpret_cast<const float4*>(P.cg[0] + 2 * x0 + 4));
        }
        cps[0] = make_float4(q0.x, q0.x, q0.y, q0.y); cps[cstr] = make_float4(q0.z, q0.z, q0.w, q0.w);
        cps[2 * cstr] = make_float4(q1.x, q1.x, q1.y, q1.y); cps[3 * cstr] = make_float4(q1.z, q1.z, q1.w, q1.w);
    }

    PlaneState S0, S1;
    float L0p[5], U0p[5], carry[4];                    // pending contributions to this row (5th: column of the next lane)
    float scarry[4] = {0.f, 0.f, 0.f, 0.f};            // seam rows: upper-plane contributions to the next tile's first row
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        S0.u[c] = S0.e[c] = S0.s[c] = S0.txy[c] = 0.f;
        S1.u[c] = S1.e[c] = S1.s[c] = S1.txy[c] = 0.f;
        S0.h = S1.h = 0.f;
        S0.n[c] = S1.n[c] = 0.f;
#pragma unroll
        for (int d = 0; d < 4; ++d) { S0.v[c][d] = 0.f; S1.v[c][d] = 0.f; }
        L0p[c] = U0p[c] = carry[c] = 0.f;
    }
    L0p[4] = U0p[4] = 0.f;
    S0.nh = S1.nh = 0.f;
    float en = 0.f, enl = 0.f, ell = 0.f;

    auto load4n = [&](const float* ptr, float (&v)[4], float& halo) {     // plain (diffusivity)
        v[0] = v[1] = v[2] = v[3] = 0.f;
        if (col_ok) {
            const float4 q = __ldg(reinterpret_cast<const float4*>(ptr));
            v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
        }
        halo = 0.f;
        if (halo_ok) halo = __ldg(ptr + 4);
    };
    auto load4 = [&](const float* ptr, float (&v)[4], float& halo) {
        if (col_ok) {
            const float4 q = __ldg(reinterpret_cast<const float4*>(ptr));
            v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
        } else {
            v[0] = v[1] = v[2] = v[3] = 0.f;
        }
        halo = 0.f;
        if (halo_ok) halo = __ldg(ptr + 4);
        if (impose) {
            if (first_col) v[0] = bc0;
            if (last_col) v[3] = bc1;
        }
    };
    auto xdiffs = [&](const float (&v)[4], float halo, float (&e)[4]) {
        float rn = __shfl_down_sync(0xffffffffu, v[0], 1, LW);
        if (lastl) rn = halo;
        e[0] = v[1] - v[0]; e[1] = v[2] - v[1]; e[2] = v[3] - v[2]; e[3] = rn - v[3];
    };

    float ua[4], uah = 0.f;                            // prefetched row above (top warp row of the tile only)
    ua[0] = ua[1] = ua[2] = ua[3] = 0.f;
    if (kbeg & 1) load4(pu + (size_t)kbeg * plane, S1.u, S1.h); else load4(pu + (size_t)kbeg * plane, S0.u, S0.h);
    if (top_row) load4(pa + (size_t)kbeg * plane, ua, uah);
    float na[4], nah = 0.f;                            // nodal mode: prefetched diffusivity of the row above (top warp row)
    na[0] = na[1] = na[2] = na[3] = 0.f;
    if constexpr (!KL) {
        if (kbeg & 1) load4n(pn + (size_t)kbeg * plane, S1.n, S1.nh); else load4n(pn + (size_t)kbeg * plane, S0.n, S0.nh);
        if (top_row) load4n(pna + (size_t)kbeg * plane, na, nah);
    }

    // Iteration p stages node plane p into `up`, computes element plane p-1 between `lo` and `up`,
    // and finishes node plane p-2.  PAR = p & 1 selects the exchange buffer.
    auto step = [&](PlaneState& lo, PlaneState& up, const int p, const int PAR) {
        float* sb = smem + PAR * BUF + ty * NXP + x0;
        float* sX = smem + PAR * BUF + XOFF + (ty * WX + wx) * 4;
        const bool stage = (p <= kend + 1);
        float w0[4];
        if (stage) {                                   // up.u / up.h were prefetched by the previous step
            xdiffs(up.u, up.h, up.e);
#pragma unroll
            for (int c = 0; c < 4; ++c) w0[c] = up.u[c] - lo.u[c];
            if (col_ok) {
                *reinterpret_cast<float4*>(sb) = make_float4(up.u[0], up.u[1], up.u[2], up.u[3]);
                *reinterpret_cast<float4*>(sb + TYNXP) = make_float4(up.e[0], up.e[1], up.e[2], up.e[3]);
            }
            if constexpr (!KL) {
                if (col_ok) *reinterpret_cast<float4*>(sb + 4 * TYNXP) = make_float4(up.n[0], up.n[1], up.n[2], up.n[3]);
            }
            if (p <= kend) {                           // prefetch the next plane (lo.u / lo.n are dead)
                load4(pu + (size_t)(p + 1) * plane, lo.u, lo.h);
                if constexpr (!KL) load4n(pn + (size_t)(p + 1) * plane, lo.n, lo.nh);
            }
            if (hasf && p >= p0 && p < p1 && out_row) { // load energy of the staged plane
                float rs = (up.u[0] + up.u[1]) + (up.u[2] + up.u[3]);
                if (first_col) rs -= 0.5f * up.u[0];
                if (last_col) rs -= 0.5f * up.u[3];
                const float wz = (p == 0 || p == nz - 1) ? 0.5f : 1.f;
                ell = fmaf(fw * wy * wz, rs, ell);
            }
        }
        __syncthreads();

        // ---- finish node plane p-2 with what row y-1 (and the warp on the left) sent
        if (WANT_R && p - 2 >= kbeg) {
            float l1[4] = {0.f, 0.f, 0.f, 0.f}, u1[4] = {0.f, 0.f, 0.f, 0.f};
            if (ty > 0 && col_ok) {
                const float4 a = *reinterpret_cast<const float4*>(sb + 2 * TYNXP - NXP);
                const float4 c4 = *reinterpret_cast<const float4*>(sb + 3 * TYNXP - NXP);
                l1[0] = a.x; l1[1] = a.y; l1[2] = a.z; l1[3] = a.w;
                u1[0] = c4.x; u1[1] = c4.y; u1[2] = c4.z; u1[3] = c4.w;
            }
            if (firstl && wx > 0) {                 // left warp's last element: (r100, r110, r101, r111)
                const float4 me = *reinterpret_cast<const float4*>(sX - 4);
                l1[0] += me.x; u1[0] += me.z;          // to this row: r100 (lower plane), r101 (upper plane)
                if (ty > 0) {
                    const float4 bl = *reinterpret_cast<const float4*>(sX - 4 - WX * 4);
                    l1[0] += bl.y; u1[0] += bl.w;      // from the row below: r110, r111
                }
            }
            const int pl = p - 2;                      // the plane being finished
            if (seam_row) {                            // same finish for the node row above, which the next tile owns
                float l1v[4] = {0.f, 0.f, 0.f, 0.f}, u1v[4] = {0.f, 0.f, 0.f, 0.f};
                if (col_ok) {
                    const float4 a = *reinterpret_cast<const float4*>(sb + 2 * TYNXP);
                    const float4 c4 = *reinterpret_cast<const float4*>(sb + 3 * TYNXP);
                    l1v[0] = a.x; l1v[1] = a.y; l1v[2] = a.z; l1v[3] = a.w;
                    u1v[0] = c4.x; u1v[1] = c4.y; u1v[2] = c4.z; u1v[3] = c4.w;
                }
                if (firstl && wx > 0) {
                    const float4 me = *reinterpret_cast<const float4*>(sX - 4);
                    l1v[0] += me.y; u1v[0] += me.w;
                }
                const float scs = gs * kap;
                float o[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) { o[c] = scs * (l1v[c] + scarry[c]); scarry[c] = u1v[c]; }
                if (!nomask) { o[0] *= mfirst; o[3] *= mlast; }
                if (pl >= p0 && col_ok)
                    *reinterpret_cast<float4*>(pseam + (size_t)pl * nx) = make_float4(o[0], o[1], o[2], o[3]);
            }
            const float wz = (pl == 0 || pl == nz - 1) ? 0.5f : 1.f;
            const float lw = fw * wy * wz;
            const float sc = gs * kap, nl = -gs * lw;
            float o[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float raw = (L0p[c] + l1[c]) + carry[c];
                carry[c] = U0p[c] + u1[c];
                o[c] = fmaf(sc, raw, nl);
            }
            if (!nomask) {
                o[0] *= mfirst; o[3] *= mlast;
            } else {
                if (first_col) o[0] -= 0.5f * nl;      // Dirichlet columns carry half the nodal load
                if (last_col) o[3] -= 0.5f * nl;
            }
            if (pl >= p0 && out_row && col_ok)
                *reinterpret_cast<float4*>(pr + (size_t)pl * plane) = make_float4(o[0], o[1], o[2], o[3]);
        }

        // ---- finish staging plane p (needs row y+1) and compute element plane p-1
        if (stage) {
            float uab[4], eab[4];
            // a warp that holds several rows has lanes on both sides of `top_row`: its shuffles run for the whole warp
            float eab_top[4] = {0.f, 0.f, 0.f, 0.f};
            if constexpr (NARROW) { if (warp_top) xdiffs(ua, uah, eab_top); }
            if (!top_row) {
                float4 a = make_float4(0.f, 0.f, 0.f, 0.f), c4 = a;
                if (col_ok) {
                    a = *reinterpret_cast<const float4*>(sb + NXP);
                    c4 = *reinterpret_cast<const float4*>(sb + TYNXP + NXP);
                }
                uab[0] = a.x; uab[1] = a.y; uab[2] = a.z; uab[3] = a.w;
                eab[0] = c4.x; eab[1] = c4.y; eab[2] = c4.z; eab[3] = c4.w;
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c) uab[c] = ua[c];
                if constexpr (NARROW) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) eab[c] = eab_top[c];
                } else {
                    xdiffs(ua, uah, eab);               // top_row is uniform in the warp
                }
                if (p <= kend) load4(pa + (size_t)(p + 1) * plane, ua, uah);
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) { up.s[c] = uab[c] - up.u[c]; up.txy[c] = eab[c] - up.e[c]; }
            if constexpr (!KL) {
                // nu of the staged plane at the 4 (xi, eta) points of each element: x lerp on rows y and y+1, then y lerp
                float nab[5];
                float rn_top = 0.f;
                if (NARROW ? warp_top : top_row) rn_top = __shfl_down_sync(0xffffffffu, na[0], 1, LW);
                if (!top_row) {
                    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
                    float a4 = 0.f;
                    if (col_ok) {
                        a = *reinterpret_cast<const float4*>(sb + 4 * TYNXP + NXP);
                        if (x0 + 4 < nx) a4 = sb[4 * TYNXP + NXP + 4];
                    }
                    nab[0] = a.x; nab[1] = a.y; nab[2] = a.z; nab[3] = a.w; nab[4] = a4;
                } else {
                    const float rn = lastl ? nah : rn_top;
                    nab[0] = na[0]; nab[1] = na[1]; nab[2] = na[2]; nab[3] = na[3]; nab[4] = rn;
                    if (p <= kend) load4n(pna + (size_t)(p + 1) * plane, na, nah);
                }
                float nrn = __shfl_down_sync(0xffffffffu, up.n[0], 1, LW);
                if (lastl) nrn = up.nh;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float n0 = up.n[c], n1 = (c < 3) ? up.n[c < 3 ? c + 1 : c] : nrn;
                    const float dl = n1 - n0, dh = nab[c + 1] - nab[c];
                    const float la = fmaf(DN_GA, dl, n0), lb = fmaf(DN_GB, dl, n0);          // row y at xi = a, b
                    const float ha = fmaf(DN_GA, dh, nab[c]), hb = fmaf(DN_GB, dh, nab[c]);  // row y+1
                    const float da = ha - la, db = hb - lb;
                    up.v[c][0] = fmaf(DN_GA, da, la); up.v[c][1] = fmaf(DN_GB, da, la);      // (p = a; q = a, b)
                    up.v[c][2] = fmaf(DN_GA, db, lb); up.v[c][3] = fmaf(DN_GB, db, lb);      // (p = b; q = a, b)
                }
            }

            if (p > kbeg) {
                const int k = p - 1;
                const bool own_energy = (k >= p0);
                float L1[5], U1[5];                    // contributions to row y+1 (lower / upper plane)
                float enrow = 0.f, enlast = 0.f;
                if (elem_row_ok) {
                    u64 gq_a[GS / 2], gq_b[GS / 2];       // Gauss row q = a / b; each entry holds (plane s = a, s = b)
                    if constexpr (KL) {
                        const ulonglong2* gl = reinterpret_cast<const ulonglong2*>(gam + (size_t)(((k - kbeg) * TY + ty) * 2) * GS);
#pragma unroll
                        for (int i = 0; i < GS / 4; ++i) {
                            const ulonglong2 t0 = gl[i], t1 = gl[GS / 4 + i];
                            gq_a[2 * i] = t0.x; gq_a[2 * i + 1] = t0.y; gq_b[2 * i] = t1.x; gq_b[2 * i + 1] = t1.y;
                        }
                    }
                    const float a = DN_GA, bq = DN_GB;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        float n000, n001, n010, n011, n100, n101, n110, n111;               // n p q s
                        if constexpr (KL) {
                            // nu[p][q][s] at the 8 Gauss points: 4 packed Horner chains (column p, row q) x (s = a, b)
                            u64 h_aa = gq_a[MM], h_ab = gq_b[MM], h_ba = gq_a[MM], h_bb = gq_b[MM];   // h_{p q}
                            const ulonglong2 cc = *reinterpret_cast<const ulonglong2*>(cps + c * cstr);
#pragma unroll
                            for (int i = MM - 1; i >= 0; --i) {
                                h_aa = fma2_3(h_aa, cc.x, gq_a[i]); h_ab = fma2_3(h_ab, cc.x, gq_b[i]);
                                h_ba = fma2_3(h_ba, cc.y, gq_a[i]); h_bb = fma2_3(h_bb, cc.y, gq_b[i]);
                            }
                            unpack2_3(h_aa, n000, n001); unpack2_3(h_ab, n010, n011);
                            unpack2_3(h_ba, n100, n101); unpack2_3(h_bb, n110, n111);
                            n000 = ex2_approx3(n000); n001 = ex2_approx3(n001); n010 = ex2_approx3(n010); n011 = ex2_approx3(n011);
                            n100 = ex2_approx3(n100); n101 = ex2_approx3(n101); n110 = ex2_approx3(n110); n111 = ex2_approx3(n111);
                        } else {
                            // nodal mode: z lerp between the (xi, eta)-interpolated values of planes k and k+1
                            const float d0 = up.v[c][0] - lo.v[c][0], d1 = up.v[c][1] - lo.v[c][1];
                            const float d2 = up.v[c][2] - lo.v[c][2], d3 = up.v[c][3] - lo.v[c][3];
                            n000 = fmaf(a, d0, lo.v[c][0]); n001 = fmaf(bq, d0, lo.v[c][0]);
                            n010 = fmaf(a, d1, lo.v[c][1]); n011 = fmaf(bq, d1, lo.v[c][1]);
                            n100 = fmaf(a, d2, lo.v[c][2]); n101 = fmaf(bq, d2, lo.v[c][2]);
                            n110 = fmaf(a, d3, lo.v[c][3]); n111 = fmaf(bq, d3, lo.v[c][3]);
                        }
                        float Nx_aa = n000 + n100, Nx_ab = n001 + n101, Nx_ba = n010 + n110, Nx_bb = n011 + n111;   // (q, s)
                        float Ny_aa = n000 + n010, Ny_ab = n001 + n011, Ny_ba = n100 + n110, Ny_bb = n101 + n111;   // (p, s)
                        float Nz_aa = n000 + n001, Nz_ab = n010 + n011, Nz_ba = n100 + n101, Nz_bb = n110 + n111;   // (p, q)
                        if (!iso) {
                            Nx_aa *= kx; Nx_ab *= kx; Nx_ba *= kx; Nx_bb *= kx;
                            Ny_aa *= ky; Ny_ab *= ky; Ny_ba *= ky; Ny_bb *= ky;
                            Nz_aa *= kz; Nz_ab *= kz; Nz_ba *= kz; Nz_bb *= kz;
                        }
                        // hierarchical coordinates of the element
                        const float e0 = lo.e[c], s0 = lo.s[c];
                        const float txy = lo.txy[c], txz = up.e[c] - e0, tyz = up.s[c] - s0, txyz = up.txy[c] - txy;
                        const float Axa = fmaf(a, txy, e0), Axb = fmaf(bq, txy, e0);
                        const float Bxa = fmaf(a, txyz, txz), Bxb = fmaf(bq, txyz, txz);
                        const float Dx_aa = fmaf(a, Bxa, Axa), Dx_ab = fmaf(bq, Bxa, Axa), Dx_ba = fmaf(a, Bxb, Axb), Dx_bb = fmaf(bq, Bxb, Axb);
                        const float Aya = fmaf(a, txy, s0), Ayb = fmaf(bq, txy, s0);
                        const float Bya = fmaf(a, txyz, tyz), Byb = fmaf(bq, txyz, tyz);
                        const float Dy_aa = fmaf(a, Bya, Aya), Dy_ab = fmaf(bq, Bya, Aya), Dy_ba = fmaf(a, Byb, Ayb), Dy_bb = fmaf(bq, Byb, Ayb);
                        const float Aza = fmaf(a, txz, w0[c]), Azb = fmaf(bq, txz, w0[c]);
                        const float Dz_aa = fmaf(a, Bya, Aza), Dz_ab = fmaf(bq, Bya, Aza), Dz_ba = fmaf(a, Byb, Azb), Dz_bb = fmaf(bq, Byb, Azb);
                        const float Gx_aa = Nx_aa * Dx_aa, Gx_ab = Nx_ab * Dx_ab, Gx_ba = Nx_ba * Dx_ba, Gx_bb = Nx_bb * Dx_bb;
                        const float Gy_aa = Ny_aa * Dy_aa, Gy_ab = Ny_ab * Dy_ab, Gy_ba = Ny_ba * Dy_ba, Gy_bb = Ny_bb * Dy_bb;
                        const float Gz_aa = Nz_aa * Dz_aa, Gz_ab = Nz_ab * Dz_ab, Gz_ba = Nz_ba * Dz_ba, Gz_bb = Nz_bb * Dz_bb;
                        // adjoint of the three interpolations
                        const float AXa = Gx_aa + Gx_ab, AXb = Gx_ba + Gx_bb;
                        const float BXa = fmaf(bq, Gx_ab, a * Gx_aa), BXb = fmaf(bq, Gx_bb, a * Gx_ba);
                        const float AYa = Gy_aa + Gy_ab, AYb = Gy_ba + Gy_bb;
                        const float BYa = fmaf(bq, Gy_ab, a * Gy_aa), BYb = fmaf(bq, Gy_bb, a * Gy_ba);
                        const float AZa = Gz_aa + Gz_ab, AZb = Gz_ba + Gz_bb;
                        const float BZa = fmaf(bq, Gz_ab, a * Gz_aa), BZb = fmaf(bq, Gz_bb, a * Gz_ba);
                        float dE = AXa + AXb, dS = AYa + AYb, dW = AZa + AZb;
                        float dXY = fmaf(bq, AXb, a * AXa);
                        dXY = fmaf(a, AYa, dXY); dXY = fmaf(bq, AYb, dXY);
                        float dXZ = BXa + BXb;
                        dXZ = fmaf(a, AZa, dXZ); dXZ = fmaf(bq, AZb, dXZ);
                        float dYZ = (BYa + BYb) + (BZa + BZb);
                        float dXYZ = fmaf(bq, BXb, a * BXa);
                        dXYZ = fmaf(a, BYa, dXYZ); dXYZ = fmaf(bq, BYb, dXYZ);
                        dXYZ = fmaf(a, BZa, dXYZ); dXYZ = fmaf(bq, BZb, dXYZ);
                        // the element energy is a quadratic form of its 7 coordinates: Euler's identity
                        float e1 = dE * e0;
                        e1 = fmaf(dS, s0, e1); e1 = fmaf(dW, w0[c], e1); e1 = fmaf(dXY, txy, e1);
                        e1 = fmaf(dXZ, txz, e1); e1 = fmaf(dYZ, tyz, e1); e1 = fmaf(dXYZ, txyz, e1);
                        if (c == 3) enlast = e1; else enrow += e1;
                        if (WANT_R) {
                            if (c == 3 && nomask && last_elem_missing) { dE = dS = dW = dXY = dXZ = dYZ = dXYZ = 0.f; }
                            // chain rule to the corners
                            const float r110 = dXY - dXYZ, r101 = dXZ - dXYZ, r011 = dYZ - dXYZ;
                            const float r100 = (dE - r110) - dXZ, r010 = (dS - r110) - dYZ, r001 = (dW - r101) - dYZ;
                            const float r000 = ((r011 - dW) + (dXY - dE)) + (dXZ - dS);
                            if (c == 0) { L0p[0] = r000; L1[0] = r010; U0p[0] = r001; U1[0] = r011; }
                            else { L0p[c] += r000; L1[c] += r010; U0p[c] += r001; U1[c] += r011; }
                            L0p[c + 1] = r100; L1[c + 1] = r110; U0p[c + 1] = r101; U1[c + 1] = dXYZ;
                        }
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 5; ++c) { L0p[c] = 0.f; L1[c] = 0.f; U0p[c] = 0.f; U1[c] = 0.f; }
                }
                if (WANT_R) {
                    // the left neighbour's last element feeds this thread's first node column
                    const float a100 = __shfl_up_sync(0xffffffffu, L0p[4], 1, LW), a110 = __shfl_up_sync(0xffffffffu, L1[4], 1, LW);
                    const float a101 = __shfl_up_sync(0xffffffffu, U0p[4], 1, LW), a111 = __shfl_up_sync(0xffffffffu, U1[4], 1, LW);
                    if (!firstl) { L0p[0] += a100; L1[0] += a110; U0p[0] += a101; U1[0] += a111; }
                    // what goes to row y+1 and to the warp on the right is published by the next step's
                    // barrier: write it into the other exchange buffer now (its readers finished before
                    // this step's barrier)
                    float* so = smem + (PAR ^ 1) * BUF + ty * NXP + x0;
                    if (col_ok) {
                        *reinterpret_cast<float4*>(so + 2 * TYNXP) = make_float4(L1[0], L1[1], L1[2], L1[3]);
                        *reinterpret_cast<float4*>(so + 3 * TYNXP) = make_float4(U1[0], U1[1], U1[2], U1[3]);
                    }
                    if (lastl)
                        *reinterpret_cast<float4*>(smem + (PAR ^ 1) * BUF + XOFF + (ty * WX + wx) * 4) =
                            make_float4(L0p[4], L1[4], U0p[4], U1[4]);
                }
                if (own_energy && elem_row_ok) {
                    en += enrow;
                    if (!last_elem_missing) enl += enlast;
                }
            }
        }
    };

    // ---- march; even planes are staged into S0, odd planes into S1
    {
        int p = kbeg;
        if (p & 1) { step(S0, S1, p, 1); ++p; }
        while (p <= kend + 2) {
            step(S1, S0, p, 0);
            if (++p > kend + 2) break;
            step(S0, S1, p, 1);
            ++p;
        }
    }

    // ---- the top node plane of the domain has no element plane above it: it is what was carried
    if (WANT_R && p1 == nz && out_row && col_ok) {
        const float lw = fw * wy * 0.5f;
        const float sc = gs * kap, nl = -gs * lw;
        float o[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) o[c] = fmaf(sc, carry[c], nl);
        if (!nomask) { o[0] *= mfirst; o[3] *= mlast; }
        else { if (first_col) o[0] -= 0.5f * nl; if (last_col) o[3] -= 0.5f * nl; }
        *reinterpret_cast<float4*>(pr + (size_t)(nz - 1) * plane) = make_float4(o[0], o[1], o[2], o[3]);
    }
    if (seam_row && p1 == nz && col_ok) {
        const float scs = gs * kap;
        float o[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) o[c] = scs * scarry[c];
        if (!nomask) { o[0] *= mfirst; o[3] *= mlast; }
        *reinterpret_cast<float4*>(pseam + (size_t)(nz - 1) * nx) = make_float4(o[0], o[1], o[2], o[3]);
    }
    const double etot = 0.5 * (double)kap * ((double)en + (double)enl);
    block_reduce_store(etot, (double)ell, P.partials + 2 * ((size_t)b * P.nblk + blockIdx.x));
}

// Adds the seam contributions to the first node row of every tile but the first (fixed order: deterministic).
__global__ void seam_fixup_kernel(float* __restrict__ r, const float* __restrict__ seam, int nx, int ny, int nz,
                                  int TY, int nseam, long long total4) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total4) return;
    const int nx4 = nx / 4;
    const int x4 = (int)(i % nx4);
    long long t = i / nx4;
    const int pl = (int)(t % nz); t /= nz;
    const int sm = (int)(t % nseam);
    const int b = (int)(t / nseam);
    const float4 a = __ldg(reinterpret_cast<const float4*>(seam) + i);
    float4* dst = reinterpret_cast<float4*>(r + (((size_t)b * nz + pl) * ny + (size_t)(sm + 1) * TY) * nx) + x4;
    float4 v = *dst;
    v.x += a.x; v.y += a.y; v.z += a.z; v.w += a.w;
    *dst = v;
}

struct Geo3 { int WX, TY, Z, ntile_y, nchunk_z, GS, bps, LW; size_t smem; };

int sm_count3() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
        (void)cudaGetLastError();
        n = 148;
    }
    return n;
}

Geo3 geometry3_search(const dn_problem& p) {
    Geo3 best{};
    const int nx = p.grid.nx, ny = p.grid.ny, nz = p.grid.nz;
    const int WX = (nx + 127) / 128;
    const int m = (p.nu_mode == DN_NU_KL_GAUSS) ? p.kl_modes : 0;
    const int GS = m ? (2 * (m + 1) + 3) / 4 * 4 : 0;               // floats per Gauss-row line pair
    const int sms = sm_count3();
    double best_cost = -1.0;
    const int LW = (nx <= 32) ? 8 : (nx <= 64) ? 16 : 32;          // lanes per node row
    const int RPW = 32 / LW;                                         // node rows per warp
    const int ty_max = (T3_THREADS / 32) / WX * RPW;
    // Tiles do not overlap, so any tile height works.  Pick (TY, Z) by a cost model fitted to sweeps on
    // B200: work grows with the warm-up plane of every z chunk, blocks should fill whole waves, an SM
    // wants 16 resident warps (128 registers each) in more than one block (barriers), and very flat tiles
    // pay more seam traffic.
    for (int TY = (RPW > 2 ? RPW : 2); TY <= ty_max; TY += (RPW > 1 ? RPW : 1)) {
        if (TY > ny && TY > 2 * RPW) break;
        const int TYW = TY / RPW;                                    // warp rows of a block
        int bps = 16 / (WX * TYW);                                   // blocks per SM by registers
        if (bps < 1) bps = 1;
        if (bps > 4) bps = 4;
        const int warps = bps * WX * TYW;
        const long long ntile = (ny + TY - 1) / TY;
        const size_t fixed = sizeof(float) * 2 * ((size_t)(m ? 4 : 5) * TY * WX * 128 + (size_t)TY * WX * 4);
        for (int Z = 4; Z <= 256; ++Z) {
            if (Z > nz && Z > 4) break;
            const size_t sm = fixed + sizeof(float) * (size_t)(Z + 1) * TY * 2 * GS + (m ? (size_t)16 * 4 * 32 * WX * TYW : 0);
            if (sm * bps > 200 * 1024) break;
            const long long nch = (nz + Z - 1) / Z;
            const long long blocks = (long long)p.batch * ntile * nch;
            const long long slots = (long long)sms * bps;
            const long long waves = (blocks + slots - 1) / slots;
            const double work = (double)blocks * (Z + 3) * TYW;
            const double imbalance = (double)waves * slots / (double)blocks;
            const double cost = work * imbalance * (16.0 / warps) * (1.0 + 0.1 / TY) * (1.0 + 0.05 / bps);
            if (best_cost < 0 || cost < best_cost) {
                best_cost = cost;
                best.WX = WX; best.TY = TY; best.Z = Z; best.ntile_y = (int)ntile; best.nchunk_z = (int)nch;
                best.GS = GS; best.bps = bps; best.smem = sm; best.LW = LW;
            }
        }
    }
    return best;
}

Geo3 geometry3(const dn_problem& p) {
    return memo_geometry<Geo3>(p, sm_count3(), [&]() { return geometry3_search(p); });
}

template <int M, bool FULL, bool NARROW>
cudaError_t launch_mf(const Params& P, const Geo3& g, cudaStream_t s) {
    dim3 grid((unsigned)(g.ntile_y * g.nchunk_z), (unsigned)P.batch);
    const int threads = 32 * g.WX * g.TY / (32 / g.LW);
    cudaError_t e;
    if (P.r) {
        e = cudaFuncSetAttribute(tiled3d_kernel<M, true, FULL, NARROW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g.smem);
        if (e != cudaSuccess) return e;
        tiled3d_kernel<M, true, FULL, NARROW><<<grid, threads, g.smem, s>>>(P, g.WX, g.TY, g.Z, g.ntile_y, g.LW);
        if (g.ntile_y > 1) {
            const long long total4 = (long long)P.batch * (g.ntile_y - 1) * P.nz * (P.nx / 4);
            seam_fixup_kernel<<<(unsigned)((total4 + 255) / 256), 256, 0, s>>>(P.r, P.seam, P.nx, P.ny, P.nz, g.TY,
                                                                              g.ntile_y - 1, total4);
        }
    } else {
        e = cudaFuncSetAttribute(tiled3d_kernel<M, false, FULL, NARROW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g.smem);
        if (e != cudaSuccess) return e;
        tiled3d_kernel<M, false, FULL, NARROW><<<grid, threads, g.smem, s>>>(P, g.WX, g.TY, g.Z, g.ntile_y, g.LW);
    }
    return cudaGetLastError();
}

template <int M>
cudaError_t launch_m(const Params& P, const Geo3& g, cudaStream_t s) {
    if (g.LW < 32) return launch_mf<M, false, true>(P, g, s);
    return (g.WX * 128 == P.nx) ? launch_mf<M, true, false>(P, g, s) : launch_mf<M, false, false>(P, g, s);
}

}  // namespace

bool tiled3d_applicable(const dn_problem& p) {
    return p.grid.dim == 3 && p.nu_mode != DN_NU_KL_NODAL && p.grid.nx % 4 == 0 && p.grid.nx >= 8 && p.grid.nx <= 512 &&
           p.grid.ny >= 2 && p.grid.nz >= 2;
}

size_t tiled3d_seam_floats(const dn_problem& p) {
    if (!tiled3d_applicable(p)) return 0;
    const Geo3 g = geometry3(p);
    return (size_t)p.batch * (g.ntile_y - 1) * p.grid.nz * p.grid.nx;
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

cudaError_t launch_seam_fixup(float* r, const float* seam, int nx, int ny, int nz, int rows_per_tile, int nseam, int batch,
                              cudaStream_t s) {
    const long long total4 = (long long)batch * nseam * nz * (nx / 4);
    seam_fixup_kernel<<<(unsigned)((total4 + 255) / 256), 256, 0, s>>>(r, seam, nx, ny, nz, rows_per_tile, nseam, total4);
    return cudaGetLastError();
}

cudaError_t launch_tiled3d(const Params& P, const Launch& l, cudaStream_t s) {
    dn_problem p{};
    p.grid.dim = 3; p.grid.nx = P.nx; p.grid.ny = P.ny; p.grid.nz = P.nz; p.batch = P.batch;
    p.nu_mode = P.nu_mode; p.kl_modes = P.m;
    const Geo3 g = geometry3(p);
    (void)l;
    switch (P.m) {
        case 0: return launch_m<0>(P, g, s);
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
