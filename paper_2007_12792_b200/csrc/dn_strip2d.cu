// Strip kernel for wide 2D grids, energy and residual fused, in all three diffusivity modes: KL evaluated in the
// kernel at the Gauss points, KL evaluated at the nodes and then interpolated, or a stored nodal field.
//
// Layout of the work.  A warp is a work unit of its own: one sample, one chunk of R node rows, one
// strip of 128 node columns (4 consecutive nodes per lane).  Strips overlap by one lane: lane 0 of
// every strip but the first recomputes the 4 elements left of the strip only to hand the
// contributions of the last of them to lane 1, and stores nothing.  So no warp ever waits for
// another one: there is no barrier and no exchange through shared memory, at the price of 1/31
// more elements.  A unit marches over its element rows from bottom to top.  The node row below
// lives in registers (values, horizontal differences, pending contributions); the row above and
// the polynomial of the KL exponent on that element row arrive through a per-warp ring in shared
// memory that the warp fills with asynchronous copies several rows ahead (each lane copies and
// reads back its own 16 bytes of the row; the 64-byte coefficient row is copied by four lanes and
// read by all after a warp-level sync).  Every element is computed once per unit; its
// contributions to its left nodes stay in the thread, those to its right nodes go to the next lane
// by shuffle, those to the upper row are carried to the next step.  The first element row of a
// chunk is recomputed by the chunk below (1/R).  No atomics.
//
// Arithmetic of one element: as in the tiled 2D kernel (differences e0, s0, t of the corner values;
// d/dx at Gauss row q is (e0 + q t)/hx, d/dy at Gauss column p is (s0 + p t)/hy; sums of nu along
// each derivative's own axis; chain rule to the four corners).  The diffusion energy is taken from
// the residual by Euler's identity for quadratic forms: 1/2 sum_i u_i (K u)_i.
//
// KL diffusivity: for a fixed Gauss row (or, with KN, node row) the exponent is a polynomial of degree m in c = cos(pi x).
// The table kernel prepares its coefficients in double once per call (they do not depend on u), for
// both Gauss rows of every element row, interleaved so that the two rows are evaluated together
// with packed two-wide FMAs.
#include "dn_internal.cuh"

namespace dn {

namespace {

constexpr int S2_WARPS = 8;                       // warps (work units) per block
constexpr int S2_NE = 4;                          // nodes per lane
constexpr int S2_COLS = 32 * S2_NE;               // node columns a warp holds
constexpr int S2_STRIDE = S2_COLS - S2_NE;        // distance of neighbouring strips
constexpr int S2_DEPTH0 = 8;                      // ring slots per warp (DEPTH - 1 rows in flight); a power of two
constexpr int S2_SLOT0 = 256;                     // floats per ring slot (node row, 4 nodes right of it, coefficient row); a power of two

typedef unsigned long long u64;

__device__ __forceinline__ float s2_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void s2_unpack(u64 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ u64 s2_pack(float lo, float hi) {
    u64 v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
    return v;
}
__device__ __forceinline__ u64 s2_fma2(u64 a, u64 b, u64 c) {
    u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ void s2_cp16(float* smem_dst, const float* gsrc) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void s2_cp16_if(float* smem_dst, const float* gsrc, int pred) {    // predicated, no branch
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.s32 p, %2, 0;\n\t@p cp.async.cg.shared.global [%0], [%1], 16;\n\t}"
                 ::"r"(d), "l"(gsrc), "r"(pred) : "memory");
}
__device__ __forceinline__ void s2_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void s2_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Floats per element row in the coefficient table: (row a, row b) pairs for k = 0..M, padded to a multiple of 4.
__host__ __device__ constexpr int s2_gs(int m) { return (2 * (m + 1) + 3) / 4 * 4; }

// NF: nodal forcing.  The f row rides in the ring next to the u row; the load vector is the consistent mass matrix
// applied to f, a 3 x 3 stencil that separates into a smoothing along x (neighbours by shuffle) and one along y (the row
// below carried, the row above arriving), with the one-sided weights on the boundary nodes.
// EO: energy only.  The same march, but every element adds its own energy and nothing is gathered or stored.
template <int M, int BPS, int MODE, bool NF, bool EO>
__global__ void __launch_bounds__(S2_WARPS * 32, BPS)
strip2d_kernel(const Params P, const float* __restrict__ rowpoly, const int R, const int nchunk, const int nstrip) {
    extern __shared__ __align__(16) float smem[];
    dep_wait();                                         // the tables of this call are complete
    dep_release();                                      // the finaliser may move in behind the last wave
    constexpr int NE = S2_NE;
    constexpr int GS = s2_gs(M);
    // MODE 0: KL at the Gauss points; 1 (KN): KL at the nodes, then Q1 interpolation; 2 (ND): stored nodal field
    constexpr bool KN = (MODE == 1), ND = (MODE == 2);
    // ring slot: node row of u, the 4 nodes right of it, then the coefficient row - or (ND) the same two pieces of nu;
    // with nodal forcing the f row and the 4 nodes right of it follow
    constexpr bool BIG = ND || NF;
    constexpr int S2_SLOT = BIG ? 2 * S2_SLOT0 : S2_SLOT0, S2_DEPTH = BIG ? S2_DEPTH0 / 2 : S2_DEPTH0;
    constexpr int NUOFF = S2_COLS + 4;                  // ND: where the nu row starts inside a slot
    constexpr int FOFF = ND ? 2 * (S2_COLS + 4) : S2_COLS + 4 + GS;      // NF: where the f row starts
    static_assert(S2_COLS + 4 + GS <= S2_SLOT0 && FOFF + S2_COLS + 4 <= 2 * S2_SLOT0, "ring slot too small");
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    float* ring = smem + (size_t)warp * S2_DEPTH * S2_SLOT;
    const long long unit = (long long)blockIdx.x * S2_WARPS + warp;
    const long long total = (long long)P.batch * nchunk * nstrip;
    if (unit >= total) return;                          // warps are independent: no block-wide barrier follows
    const int strip = (int)(unit % nstrip);
    const int chunk = (int)((unit / nstrip) % nchunk);
    const int b = (int)(unit / ((long long)nstrip * nchunk));

    const int nx = P.nx, ny = P.ny;
    const int xs = strip * S2_STRIDE;
    const int x0 = xs + NE * lane;
    const bool act = x0 < nx;                           // this lane holds nodes of the grid
    const int x0c = act ? x0 : nx - NE;                 // lanes beyond the grid load valid memory and store nothing
    const bool owner = act && (lane > 0 || strip == 0); // lane 0 of a later strip only feeds lane 1
    const bool has_first = (x0 == 0);                   // node 0 is this lane's first node
    const bool has_last = act && (x0 + NE == nx);       // node nx-1 is this lane's last node
    const bool has_halo = (xs + S2_COLS < nx);          // the nodes right of the strip exist
    const int n0 = chunk * R, n1 = min(n0 + R, ny);
    const int jbeg = max(n0 - 1, 0);
    const int jend = min(n1 - 1, ny - 2);               // last element row of this unit (inclusive)

    const float* ub = P.u + (size_t)b * P.nodes + x0c;
    float* rb = P.r + (size_t)b * P.nodes + x0c;
    const bool impose = (P.flags & DN_IMPOSE_BC_ON_LOAD) != 0;
    const bool nomask = (P.flags & DN_NO_MASK) != 0;
    float bc0 = P.bc_x0, bc1 = P.bc_x1;
    if (impose) {
        if (P.bc0_b) bc0 = __ldg(P.bc0_b + b);
        if (P.bc1_b) bc1 = __ldg(P.bc1_b + b);
    }
    const float kx = 0.25f * P.hy / P.hx, ky = 0.25f * P.hx / P.hy;
    const float kxa = kx * DN_GA, kxb = kx * DN_GB, kya = ky * DN_GA, kyb = ky * DN_GB;
    const float fw = NF ? 0.f : P.f_const * P.hx * P.hy;   // nodal load of an interior node (constant forcing)
    const bool hasf = !NF && (P.f_const != 0.f);
    const float gs = P.gJ ? __ldg(P.gJ + b) : 1.f;

    // Lane constants that make the march branch-free:
    //  lm        0 in lane 0 (nothing arrives from the left), else 1
    //  g3, ky3   0 in the lane whose last element lies right of node nx-1 (it does not exist), else 1 and ky
    //  gsf/gsl, nlf/nll   output scale and nodal load of the lane's first / last node (Dirichlet columns: masked
    //            to zero, or with DN_NO_MASK carrying half the nodal load); wf/wl their weights in the load energy
    const float lm = (lane == 0) ? 0.f : 1.f;
    const float g3 = has_last ? 0.f : 1.f, ky3 = ky * g3;
    const float nl = -gs * fw;
    const float gsf = (has_first && !nomask) ? 0.f : gs, gsl = (has_last && !nomask) ? 0.f : gs;
    const float nlf = has_first ? (nomask ? 0.5f * nl : 0.f) : nl, nll = has_last ? (nomask ? 0.5f * nl : 0.f) : nl;
    const float wf = has_first ? 0.5f : 1.f, wl = has_last ? 0.5f : 1.f;

    // cos(pi x) at the two Gauss columns of each element, duplicated into both halves of a pair
    u64 cda[NE], cdb[NE];
    u64 cnp[NE / 2];                                    // KN: cos(pi x) at this lane's nodes (pairs) and at the node right of them
    float cnh = 0.f;
    if constexpr (ND) {
    } else if constexpr (KN) {
        const float4 q = __ldg(reinterpret_cast<const float4*>(P.cn[0] + x0c));
        cnp[0] = s2_pack(q.x, q.y); cnp[1] = s2_pack(q.z, q.w);
        cnh = __ldg(P.cn[0] + x0c + NE);
    } else {
        const float4 q0 = __ldg(reinterpret_cast<const float4*>(P.cg[0] + 2 * x0c));
        const float4 q1 = __ldg(reinterpret_cast<const float4*>(P.cg[0] + 2 * x0c + 4));
        cda[0] = s2_pack(q0.x, q0.x); cdb[0] = s2_pack(q0.y, q0.y);
        cda[1] = s2_pack(q0.z, q0.z); cdb[1] = s2_pack(q0.w, q0.w);
        cda[2] = s2_pack(q1.x, q1.x); cdb[2] = s2_pack(q1.y, q1.y);
        cda[3] = s2_pack(q1.z, q1.z); cdb[3] = s2_pack(q1.w, q1.w);
    }

    // ---- the ring: step i = j - jbeg uses slot i % DEPTH, which holds node row j + 1 (every lane copies its own
    // 16 bytes), the 4 nodes right of the strip (lane 31) and the coefficients of element row j (lanes 0 .. GS/4-1)
    int fetch = jbeg;                                   // next element row to fetch
    const float* usrc = ub + (size_t)(jbeg + 1) * nx;
    const bool xcoef = !ND && (lane < GS / 4), xhalo = (lane == 31) && has_halo;
    const float* nsrc = ND ? P.nu + (size_t)b * P.nodes + x0c + (size_t)(jbeg + 1) * nx : nullptr;
    const float* fsrc = NF ? P.f + (size_t)b * P.nodes + x0c + (size_t)(jbeg + 1) * nx : nullptr;
    const int xp = (xcoef || xhalo) ? 1 : 0;            // this lane makes a second copy per row
    // coefficient rows: per element row (its two Gauss rows), or with KN per node row (the row that arrives with it)
    const float* polyb = rowpoly + (size_t)b * (KN ? ny : ny - 1) * GS;
    const float* xsrc = xcoef ? polyb + (size_t)(KN ? jbeg + 1 : jbeg) * GS + 4 * lane : usrc + NE;
    const int xstep = xcoef ? GS : nx;
    const int xdst = xcoef ? S2_COLS + 4 + 4 * lane : S2_COLS;
    auto issue = [&](float* slot) {
        if (fetch <= jend) {                            // uniform
            s2_cp16(slot + NE * lane, usrc);
            s2_cp16_if(slot + xdst, xsrc, xp);
            if constexpr (ND) {
                s2_cp16(slot + NUOFF + NE * lane, nsrc);
                s2_cp16_if(slot + NUOFF + S2_COLS, nsrc + NE, xp);
            }
            if constexpr (NF) {
                s2_cp16(slot + FOFF + NE * lane, fsrc);
                s2_cp16_if(slot + FOFF + S2_COLS, fsrc + NE, xhalo ? 1 : 0);
            }
        }
        s2_commit();                                    // one group per step, possibly empty
        ++fetch; usrc += nx; xsrc += xstep;
        if constexpr (ND) nsrc += nx;
        if constexpr (NF) fsrc += nx;
    };
#pragma unroll
    for (int d = 0; d < S2_DEPTH - 1; ++d) issue(ring + d * S2_SLOT);

    // ---- state of the node row below the current element row
    float lo[NE], cu[NE], ehor[NE], U[NE];
    {
        const float4 q = __ldg(reinterpret_cast<const float4*>(ub + (size_t)jbeg * nx));
        lo[0] = q.x; lo[1] = q.y; lo[2] = q.z; lo[3] = q.w;
        float halo = 0.f;
        if (xhalo) halo = __ldg(ub + (size_t)jbeg * nx + NE);
        if (impose) {
            if (has_first) lo[0] = bc0;
            if (has_last) lo[NE - 1] = bc1;
        }
        float rn = __shfl_down_sync(0xffffffffu, lo[0], 1);
        if (lane == 31) rn = halo;
        ehor[0] = lo[1] - lo[0]; ehor[1] = lo[2] - lo[1]; ehor[2] = lo[3] - lo[2]; ehor[3] = rn - lo[3];
#pragma unroll
        for (int k = 0; k < NE; ++k) U[k] = 0.f;
    }

    // KN: nu at this lane's 4 nodes and at the node right of them, from the polynomial of that node row
    auto nu_row = [&](const u64 (&gg)[GS / 2], float (&nn)[NE + 1]) {
#pragma unroll
        for (int h = 0; h < NE / 2; ++h) {
            u64 e = gg[M];
#pragma unroll
            for (int i = M - 1; i >= 0; --i) e = s2_fma2(e, cnp[h], gg[i]);
            float e0, e1;
            s2_unpack(e, e0, e1);
            nn[2 * h] = s2_ex2(e0); nn[2 * h + 1] = s2_ex2(e1);
        }
        float gh, dmy;
        s2_unpack(gg[M], gh, dmy);
#pragma unroll
        for (int i = M - 1; i >= 0; --i) { float gi; s2_unpack(gg[i], gi, dmy); gh = fmaf(gh, cnh, gi); }
        nn[NE] = s2_ex2(gh);
    };
    float nlo[NE + 1], hnu[NE];                         // KN, ND: nu on the node row below and its sums over x-neighbours
    if constexpr (ND) {
        const float* np = P.nu + (size_t)b * P.nodes + x0c + (size_t)jbeg * nx;
        const float4 q = __ldg(reinterpret_cast<const float4*>(np));
        nlo[0] = q.x; nlo[1] = q.y; nlo[2] = q.z; nlo[3] = q.w;
        float halo = 0.f;
        if (xhalo) halo = __ldg(np + NE);
        const float rn = __shfl_down_sync(0xffffffffu, nlo[0], 1);
        nlo[NE] = (lane == 31) ? halo : rn;
#pragma unroll
        for (int k = 0; k < NE; ++k) hnu[k] = nlo[k] + nlo[k + 1];
    }
    if constexpr (KN) {
        u64 gg[GS / 2];
        const ulonglong2* gp = reinterpret_cast<const ulonglong2*>(polyb + (size_t)jbeg * GS);
#pragma unroll
        for (int k = 0; k < GS / 4; ++k) { const ulonglong2 t = __ldg(gp + k); gg[2 * k] = t.x; gg[2 * k + 1] = t.y; }
        nu_row(gg, nlo);
#pragma unroll
        for (int k = 0; k < NE; ++k) hnu[k] = nlo[k] + nlo[k + 1];
    }

    // NF: x-smoothed forcing (hx/6) (f[k-1] + 4 f[k] + f[k+1]) of a node row, one-sided on the Dirichlet columns
    const float m6x = P.hx * (1.f / 6.f), m6y = P.hy * (1.f / 6.f);
    const float mxl = has_first ? 0.f : m6x, mxc0 = has_first ? 2.f * m6x : 4.f * m6x;     // node 0 of the lane
    const float mxr = has_last ? 0.f : m6x, mxc3 = has_last ? 2.f * m6x : 4.f * m6x;       // node 3 of the lane
    auto smooth_x = [&](const float (&f)[NE], const float fright, float (&g)[NE]) {
        const float fleft = __shfl_up_sync(0xffffffffu, f[NE - 1], 1);   // lane 0: its own value, unused (mxl = 0 or a lane that stores nothing)
        g[0] = fmaf(mxl, fleft, fmaf(mxc0, f[0], m6x * f[1]));
        g[1] = m6x * (fmaf(4.f, f[1], f[0]) + f[2]);
        g[2] = m6x * (fmaf(4.f, f[2], f[1]) + f[3]);
        g[3] = fmaf(mxr, fright, fmaf(mxc3, f[3], m6x * f[2]));
    };
    float gf_lo[NE], gf_mid[NE];                        // smoothed f of the row below the current node row, and of that row
#pragma unroll
    for (int k = 0; k < NE; ++k) { gf_lo[k] = 0.f; gf_mid[k] = 0.f; }
    if constexpr (NF) {
        const float* fp = P.f + (size_t)b * P.nodes + x0c + (size_t)jbeg * nx;
        const float4 q = __ldg(reinterpret_cast<const float4*>(fp));
        const float f0[NE] = {q.x, q.y, q.z, q.w};
        float halo = 0.f;
        if (xhalo) halo = __ldg(fp + NE);
        float fr = __shfl_down_sync(0xffffffffu, f0[0], 1);
        if (lane == 31) fr = halo;
        smooth_x(f0, fr, gf_mid);
        if (jbeg > 0) {                                 // the row below the unit's first row (uniform)
            const float4 q1 = __ldg(reinterpret_cast<const float4*>(fp - nx));
            const float f1[NE] = {q1.x, q1.y, q1.z, q1.w};
            float h1 = 0.f;
            if (xhalo) h1 = __ldg(fp - nx + NE);
            float fr1 = __shfl_down_sync(0xffffffffu, f1[0], 1);
            if (lane == 31) fr1 = h1;
            smooth_x(f1, fr1, gf_lo);
        }
    }
    float en = 0.f, ell = 0.f;                          // sum u (K u) and sum w u of the rows this lane went over
    float* rrow = rb + (size_t)jbeg * nx;
    int rd = 0;                                         // float offset of the slot to read; the one before it is refilled

    // One element row: a holds node row j, c receives node row j + 1.
    auto step = [&](float (&a)[NE], float (&c)[NE], const int j) {
        s2_wait<S2_DEPTH - 2>();                        // this step's slot has landed (for the lanes that copied it)
        __syncwarp();                                   // ... and is visible to the whole warp
        issue(ring + ((rd - S2_SLOT) & (S2_DEPTH * S2_SLOT - 1)));   // refill the slot the previous step consumed
        const float* slot = ring + rd;
        rd = (rd + S2_SLOT) & (S2_DEPTH * S2_SLOT - 1);
        {
            const float4 q = *reinterpret_cast<const float4*>(slot + NE * lane);
            c[0] = q.x; c[1] = q.y; c[2] = q.z; c[3] = q.w;
        }
        const float halo = slot[S2_COLS];
        u64 g2[GS / 2];
        if constexpr (!ND) {
            const ulonglong2* gp = reinterpret_cast<const ulonglong2*>(slot + S2_COLS + 4);
#pragma unroll
            for (int k = 0; k < GS / 4; ++k) { const ulonglong2 t = gp[k]; g2[2 * k] = t.x; g2[2 * k + 1] = t.y; }
        }
        if (impose) {
            if (has_first) c[0] = bc0;
            if (has_last) c[NE - 1] = bc1;
        }
        float ncur[NE + 1];
        if constexpr (KN) nu_row(g2, ncur);
        if constexpr (ND) {
            const float4 q = *reinterpret_cast<const float4*>(slot + NUOFF + NE * lane);
            ncur[0] = q.x; ncur[1] = q.y; ncur[2] = q.z; ncur[3] = q.w;
            const float nh = slot[NUOFF + S2_COLS];
            const float rn = __shfl_down_sync(0xffffffffu, ncur[0], 1);
            ncur[NE] = (lane == 31) ? (has_halo ? nh : 0.f) : rn;
        }
        float hir = __shfl_down_sync(0xffffffffu, c[0], 1);
        if (lane == 31) hir = has_halo ? halo : 0.f;

        float Q0 = 0.f, SY0 = 0.f, R0 = 0.f, Qp = 0.f, Tp = 0.f, rout[NE];
        float es = 0.f;                                 // EO: sum over this lane's elements of N D^2 (= u K u of the element row)
#pragma unroll
        for (int k = 0; k < NE; ++k) {
            const float uh = c[k];
            const float un = (k + 1 < NE) ? c[(k + 1 < NE) ? k + 1 : k] : hir;
            const float e1 = un - uh;
            const float s0 = uh - a[k];
            const float e0 = ehor[k];
            ehor[k] = e1;
            const float t = e1 - e0;
            const float Dxa = fmaf(DN_GA, t, e0), Dxb = fmaf(DN_GB, t, e0);
            const float Dya = fmaf(DN_GA, t, s0), Dyb = fmaf(DN_GB, t, s0);
            float Na, Nb, Ma, Mb;
            if constexpr (KN || ND) {
                // Q1 interpolation of the nodal values to the Gauss points, summed along each derivative's own axis
                const float h0 = hnu[k], h1 = ncur[k] + ncur[k + 1];
                hnu[k] = h1;
                const float v0 = nlo[k] + ncur[k], v1 = nlo[k + 1] + ncur[k + 1];
                const float dh = h1 - h0, dv = v1 - v0;
                Na = fmaf(DN_GA, dh, h0); Nb = fmaf(DN_GB, dh, h0);
                Ma = fmaf(DN_GA, dv, v0); Mb = fmaf(DN_GB, dv, v0);
            } else {
                u64 ea = g2[M], eb = g2[M];             // (row a, row b) pairs at column a / column b
#pragma unroll
                for (int i = M - 1; i >= 0; --i) { ea = s2_fma2(ea, cda[k], g2[i]); eb = s2_fma2(eb, cdb[k], g2[i]); }
                float xaa, xab, xba, xbb;
                s2_unpack(ea, xaa, xab);
                s2_unpack(eb, xba, xbb);
                const float naa = s2_ex2(xaa), nab = s2_ex2(xab), nba = s2_ex2(xba), nbb = s2_ex2(xbb);
                Na = naa + nba; Nb = nab + nbb; Ma = naa + nab; Mb = nba + nbb;
            }
            const float Gxa = Na * Dxa, Gxb = Nb * Dxb, Gya = Ma * Dya, Gyb = Mb * Dyb;
            if constexpr (EO) {
                const float e = fmaf(kx, fmaf(Gxa, Dxa, Gxb * Dxb), ky * fmaf(Gya, Dya, Gyb * Dyb));
                es += (k == NE - 1) ? g3 * e : e;       // the lane's last element may lie beyond the grid
                continue;
            }
            const float SXu = Gxa + Gxb, SYu = Gya + Gyb;
            float T = kxa * Gxa;
            T = fmaf(kxb, Gxb, T); T = fmaf(kya, Gya, T); T = fmaf(kyb, Gyb, T);
            const float Q = fmaf(kx, SXu, -T);
            const float Rr = fmaf(ky, SYu, -T);
            if (k == 0) {
                Q0 = Q; SY0 = SYu; R0 = Rr;
            } else if (k < NE - 1) {
                rout[k] = fmaf(-ky, SYu, Qp - Q) + U[k];
                U[k] = Rr + Tp;
            } else {                                    // the lane's last element may lie beyond the grid (g3 = 0)
                rout[k] = fmaf(-ky3, SYu, fmaf(-g3, Q, Qp)) + U[k];
                U[k] = fmaf(g3, Rr, Tp);
            }
            Qp = Q; Tp = T;
        }
        if constexpr (!EO) {
            // contributions of the element left of this lane's first node
            const float ql = __shfl_up_sync(0xffffffffu, Qp, 1);
            const float tl = __shfl_up_sync(0xffffffffu, Tp, 1);
            rout[0] = fmaf(-ky, SY0, fmaf(ql, lm, -Q0)) + U[0];
            U[0] = fmaf(tl, lm, R0);
        }
        float gf_up[NE];                                // NF: smoothed f of node row j + 1
        if constexpr (NF) {
            const float4 q = *reinterpret_cast<const float4*>(slot + FOFF + NE * lane);
            const float fu[NE] = {q.x, q.y, q.z, q.w};
            const float fh = slot[FOFF + S2_COLS];
            float fr = __shfl_down_sync(0xffffffffu, fu[0], 1);
            if (lane == 31) fr = has_halo ? fh : 0.f;
            smooth_x(fu, fr, gf_up);
        }
        if (j >= n0) {                                  // uniform: this unit owns node row j
            // rout is (K u) of node row j: Euler's identity gives the diffusion energy
            if constexpr (EO) {
                en += es;                               // element row j belongs to the chunk that owns node row j
#pragma unroll
                for (int k = 0; k < NE; ++k) rout[k] = 0.f;
            } else {
#pragma unroll
                for (int k = 0; k < NE; ++k) en = fmaf(a[k], rout[k], en);
            }
            float4 o;
            if constexpr (NF) {
                // load of node row j: the y-smoothing of the three smoothed rows (row 0 has no row below)
                const float wc = (j == 0) ? 2.f * m6y : 4.f * m6y;
                float F[NE];
#pragma unroll
                for (int k = 0; k < NE; ++k) {
                    F[k] = fmaf(m6y, gf_lo[k] + gf_up[k], wc * gf_mid[k]);
                    ell = fmaf(a[k], F[k], ell);
                }
                o.x = gsf * (rout[0] - F[0]); o.y = gs * (rout[1] - F[1]);
                o.z = gs * (rout[2] - F[2]); o.w = gsl * (rout[3] - F[3]);
            } else if (hasf) {
                const float wrow = (j == 0) ? 0.5f : 1.f;
                ell = fmaf(wrow, fmaf(a[0], wf, a[1]) + fmaf(a[NE - 1], wl, a[2]), ell);
                o.x = fmaf(gsf, rout[0], wrow * nlf); o.y = fmaf(gs, rout[1], wrow * nl);
                o.z = fmaf(gs, rout[2], wrow * nl); o.w = fmaf(gsl, rout[3], wrow * nll);
            } else {
                o.x = gsf * rout[0]; o.y = gs * rout[1]; o.z = gs * rout[2]; o.w = gsl * rout[3];
            }
            if constexpr (!EO) { if (owner) *reinterpret_cast<float4*>(rrow) = o; }
        }
        rrow += nx;
        if constexpr (NF) {
#pragma unroll
            for (int k = 0; k < NE; ++k) { gf_lo[k] = gf_mid[k]; gf_mid[k] = gf_up[k]; }
        }
        if constexpr (KN || ND) {
#pragma unroll
            for (int k = 0; k <= NE; ++k) nlo[k] = ncur[k];
        }
    };

    {
        int j = jbeg;
        while (true) {
            step(lo, cu, j);
            if (++j > jend) {
#pragma unroll
                for (int k = 0; k < NE; ++k) lo[k] = cu[k];
                break;
            }
            step(cu, lo, j);
            if (++j > jend) break;
        }
    }
    s2_wait<0>();

    // ---- the top node row of the grid has no element row above it (lo holds it, U what it received)
    if (n1 == ny) {
        if constexpr (!EO) {
#pragma unroll
            for (int k = 0; k < NE; ++k) en = fmaf(lo[k], U[k], en);
        }
        float4 o;
        if constexpr (NF) {
            float F[NE];
#pragma unroll
            for (int k = 0; k < NE; ++k) {              // the top row: one-sided in y
                F[k] = m6y * fmaf(2.f, gf_mid[k], gf_lo[k]);
                ell = fmaf(lo[k], F[k], ell);
            }
            o.x = gsf * (U[0] - F[0]); o.y = gs * (U[1] - F[1]); o.z = gs * (U[2] - F[2]); o.w = gsl * (U[3] - F[3]);
        } else {
            ell = fmaf(0.5f, fmaf(lo[0], wf, lo[1]) + fmaf(lo[NE - 1], wl, lo[2]), ell);
            o.x = fmaf(gsf, U[0], 0.5f * nlf); o.y = fmaf(gs, U[1], 0.5f * nl);
            o.z = fmaf(gs, U[2], 0.5f * nl); o.w = fmaf(gsl, U[3], 0.5f * nll);
        }
        if constexpr (!EO) { if (owner) *reinterpret_cast<float4*>(rb + (size_t)(ny - 1) * nx) = o; }
    }

    // ---- energy partial of this unit: owning lanes summed in a fixed order in double
    double d = owner ? 0.5 * (double)en : 0.0;
    double l = !owner ? 0.0 : NF ? (double)ell : hasf ? (double)fw * (double)ell : 0.0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        d += __shfl_down_sync(0xffffffffu, d, o);
        l += __shfl_down_sync(0xffffffffu, l, o);
    }
    if (lane == 0) {
        double* slot = P.partials + 2 * ((size_t)b * P.nblk + (size_t)chunk * nstrip + strip);
        slot[0] = d; slot[1] = l;
    }
}

struct GeoS { int R, nchunk, nstrip, bps; };

int s2_sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
        (void)cudaGetLastError();
        n = 148;
    }
    return n;
}

GeoS geometry_s_search(const dn_problem& p) {
    GeoS g{};
    const int nx = p.grid.nx, ny = p.grid.ny;
    g.nstrip = (nx <= S2_COLS) ? 1 : (nx - S2_COLS + S2_STRIDE - 1) / S2_STRIDE + 1;
    g.bps = 2;
    const long long slots = (long long)s2_sm_count() * g.bps * S2_WARPS;
    long long best = -1;
    int bestR = 16;
    for (int R = 16; R <= 1024; ++R) {
        if (R > ny && R > 16) break;
        const long long nch = (ny + R - 1) / R;
        const long long units = (long long)p.batch * g.nstrip * nch;
        const long long waves = (units + slots - 1) / slots;
        const long long cost = waves * (R + 4) * 1000 + (1000 / R);      // whole waves; prefer less redundancy on ties
        if (best < 0 || cost < best) { best = cost; bestR = R; }
    }
    g.R = bestR;
    g.nchunk = (ny + g.R - 1) / g.R;
    return g;
}

GeoS geometry_s(const dn_problem& p) {
    return memo_geometry<GeoS>(p, s2_sm_count(), [&]() { return geometry_s_search(p); });
}

template <int M, int MODE, bool NF, bool EO>
cudaError_t launch_mkfe(const Params& P, const float* rowpoly, const GeoS& g, cudaStream_t s) {
    const size_t smem = sizeof(float) * S2_WARPS * S2_DEPTH0 * S2_SLOT0;
    const long long units = (long long)P.batch * g.nchunk * g.nstrip;
    const unsigned blocks = (unsigned)((units + S2_WARPS - 1) / S2_WARPS);
    const cudaError_t e = cudaFuncSetAttribute(strip2d_kernel<M, 2, MODE, NF, EO>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return launch_dependent(strip2d_kernel<M, 2, MODE, NF, EO>, dim3(blocks), dim3(S2_WARPS * 32), smem, s, P, rowpoly, g.R,
                            g.nchunk, g.nstrip);
}

// no output array: the energy-only variant
template <int M, int MODE, bool NF>
cudaError_t launch_mkf(const Params& P, const float* rowpoly, const GeoS& g, cudaStream_t s) {
    return P.r ? launch_mkfe<M, MODE, NF, false>(P, rowpoly, g, s) : launch_mkfe<M, MODE, NF, true>(P, rowpoly, g, s);
}

template <int M, int MODE>
cudaError_t launch_mk(const Params& P, const float* rowpoly, const GeoS& g, cudaStream_t s) {
    return P.f ? launch_mkf<M, MODE, true>(P, rowpoly, g, s) : launch_mkf<M, MODE, false>(P, rowpoly, g, s);
}

template <int M>
cudaError_t launch_m(const Params& P, const float* rowpoly, const GeoS& g, cudaStream_t s) {
    return (P.nu_mode == DN_NU_KL_NODAL) ? launch_mk<M, 1>(P, rowpoly, g, s) : launch_mk<M, 0>(P, rowpoly, g, s);
}

}  // namespace

// The strips overlap by one lane and the last one may be mostly empty, so narrow grids waste lanes (a 256-wide
// row takes 3 strips of 128).  The tiled kernel is about 1.16 times slower per element in this mode: the strip
// kernel takes over where its lanes are at most 15 % more than the row, and wherever the tiled kernel cannot run.
bool strip2d_applicable(const dn_problem& p) {
    // with nodal forcing also narrow rows (one strip, part of its lanes idle): the other choice is the any-size kernel
    if (!(p.grid.dim == 2 && p.grid.nx % 4 == 0 &&
          p.grid.nx >= (p.f ? 8 : 2 * S2_COLS) && p.grid.ny >= 16))
        return false;
    const long long lanes = (long long)((p.grid.nx - S2_COLS + S2_STRIDE - 1) / S2_STRIDE + 1) * S2_COLS;
    return !tiled2d_applicable(p) || 100 * lanes <= 115ll * p.grid.nx || p.f != nullptr;   // nodal forcing: the only fast kernel
}

Launch strip2d_geometry(const dn_problem& p) {
    const GeoS g = geometry_s(p);
    Launch l{};
    l.path = PATH_STRIP2D;
    l.nblk = g.nchunk * g.nstrip;
    l.chunk = g.R;
    l.variant = g.nstrip;
    return l;
}

size_t strip2d_rowpoly_floats(const dn_problem& p) {
    if (p.nu_mode == DN_NU_NODAL) return 0;                      // the stored field needs no table
    return (size_t)p.batch * p.grid.ny * s2_gs(p.kl_modes);      // ny - 1 element rows, or ny node rows (KL at the nodes)
}

int strip2d_rowpoly_stride(int kl_modes) { return s2_gs(kl_modes); }

cudaError_t launch_strip2d(const Params& P, const float* rowpoly, cudaStream_t s) {
    dn_problem p{};
    p.grid.dim = 2; p.grid.nx = P.nx; p.grid.ny = P.ny; p.grid.nz = 1; p.batch = P.batch;
    p.nu_mode = P.nu_mode; p.kl_modes = P.m; p.f = P.f;
    const GeoS g = geometry_s(p);
    if (P.nu_mode == DN_NU_NODAL) return launch_mk<1, 2>(P, rowpoly, g, s);
    switch (P.m) {
        case 1: return launch_m<1>(P, rowpoly, g, s);
        case 2: return launch_m<2>(P, rowpoly, g, s);
        case 3: return launch_m<3>(P, rowpoly, g, s);
        case 4: return launch_m<4>(P, rowpoly, g, s);
        case 5: return launch_m<5>(P, rowpoly, g, s);
        case 6: return launch_m<6>(P, rowpoly, g, s);
        case 7: return launch_m<7>(P, rowpoly, g, s);
        case 8: return launch_m<8>(P, rowpoly, g, s);
    }
    return cudaErrorInvalidValue;
}

}  // namespace dn
