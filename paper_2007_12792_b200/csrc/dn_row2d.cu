// Row kernel for 2D grids whose rows fit one warp (nx <= 256): energy and residual fused, in all three diffusivity
// modes, constant forcing.  The 2D member of the strip family for narrow rows: where the strip 2D kernel cuts a wide
// row into overlapping 128-column strips, here a row belongs to one unit and nothing overlaps in x.
//
// Layout of the work.  A work unit is one sample and one chunk of R node rows across the whole x extent; it belongs
// to LW = 8, 16 or 32 lanes of one warp (a lane owns NX = 4 or 8 consecutive nodes, LW * NX >= nx); a warp with
// LW < 32 carries 32 / LW units that have nothing to do with one another.  No warp ever waits for another: no
// barrier after the start, no exchange through shared memory between units.  A unit marches over its element rows
// from bottom to top.  The node row below lives in registers (values, horizontal differences, pending contributions);
// the row above and the polynomial of the KL exponent on that element row (prepared once per call by the table kernel,
// as for the strip 2D kernel) arrive through a ring of DEPTH slots in shared memory that belongs to the unit alone,
// filled with cp.async (every lane its own 16-byte pieces, a few lanes the coefficient row).  The node right of a
// lane's last one is read from the ring (it is the next lane's first; behind the last lane sits a zero pad).  Every
// element is computed once per unit; its contributions to its left nodes stay in the lane, those to its right nodes go
// to the next element (to the next lane by shuffle), those to the upper row are carried to the next step.  The first
// element row of a chunk is recomputed by the chunk below (1 / R).  No atomics.
//
// Arithmetic of one element and the three diffusivity modes: as in the strip 2D kernel (differences e0, s0, t of the
// corner values; d/dx at Gauss row q is (e0 + q t) / hx, d/dy at Gauss column p is (s0 + p t) / hy; sums of nu along
// each derivative's own axis; chain rule to the four corners; the diffusion energy from the residual by Euler's
// identity for quadratic forms).
#include "dn_internal.cuh"

namespace dn {

namespace {

constexpr int R2_WARPS = 4;                       // warps per block (each warp is on its own)
// ring slots per unit (DEPTH - 1 rows in flight): the stored-field mode moves 12 bytes per node and computes least
__host__ __device__ constexpr int r2_depth(int mode) { return mode == 2 ? 6 : 4; }

typedef unsigned long long u64;

__device__ __forceinline__ float r2_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void r2_unpack(u64 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ u64 r2_pack(float lo, float hi) {
    u64 v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
    return v;
}
__device__ __forceinline__ u64 r2_fma2(u64 a, u64 b, u64 c) {
    u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ void r2_cp16(unsigned d, const float* gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void r2_cp16_if(unsigned d, const float* gsrc, int pred) {    // predicated, no branch
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.s32 p, %2, 0;\n\t@p cp.async.cg.shared.global [%0], [%1], 16;\n\t}"
                 ::"r"(d), "l"(gsrc), "r"(pred) : "memory");
}
__device__ __forceinline__ void r2_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void r2_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Floats per row of the coefficient table (the strip 2D kernel's layout): pairs for k = 0..M, padded to a multiple of 4.
__host__ __device__ constexpr int r2_gs(int m) { return (2 * (m + 1) + 3) / 4 * 4; }

struct R2Geo {
    int R, nchunk;        // node rows per unit, units per sample
    int LW, lwsh;         // lanes per unit and log2 of it
    int RS;               // floats per ring slot
    long long units;
};

// MODE 0: KL at the Gauss points; 1 (KN): KL at the nodes, then Q1 interpolation; 2 (ND): stored nodal field
// LWC: lanes per unit at compile time (16 or 32), or 0: taken from G (8 lanes)
template <int NX, int M, int MODE, int MINB, int LWC>
__global__ void __launch_bounds__(R2_WARPS * 32, MINB)
row2d_kernel(const Params P, const float* __restrict__ rowpoly, const R2Geo G) {
    extern __shared__ __align__(16) float smem[];
    dep_wait();                                         // the tables of this call are complete
    dep_release();                                      // the finaliser may move in behind the last units
    constexpr bool KG = (MODE == 0), KN = (MODE == 1), ND = (MODE == 2);
    constexpr int GS = r2_gs(M);
    constexpr int R2_DEPTH = r2_depth(MODE);
    constexpr int CFQ = ND ? 0 : GS / 4;                // 16-byte pieces of a coefficient row
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int LW = LWC ? LWC : G.LW, lwsh = (LWC == 32) ? 5 : (LWC == 16) ? 4 : G.lwsh, SUBS = 32 >> lwsh;
    const int sub = lane >> lwsh, lx = lane & (LW - 1);
    const unsigned submask = (LW == 32) ? 0xffffffffu : (((1u << LW) - 1u) << (sub * LW));
    const int nx = P.nx, ny = P.ny;
    const int x0 = NX * lx;
    const bool act = x0 < nx;                           // this lane holds nodes of the grid
    const int x0c = act ? x0 : nx - NX;                 // lanes beyond the grid load valid memory and store nothing

    // ---- shared by the block (KG): cos(pi x) at the two Gauss columns of each element of a lane, duplicated into both
    // halves of a pair, as float4 (ca, ca, cb, cb) at [element k][lane of the unit]
    float4* cps = reinterpret_cast<float4*>(smem);
    if constexpr (KG) {
        for (int i = threadIdx.x; i < NX * LW; i += blockDim.x) {
            const int k = i >> lwsh, l = i & (LW - 1);
            const int xe = min(NX * l, nx - NX) + k;    // element index = index of its left node
            const float ca = __ldg(P.cg[0] + 2 * xe), cb = __ldg(P.cg[0] + 2 * xe + 1);
            cps[i] = make_float4(ca, ca, cb, cb);
        }
        __syncthreads();                                // the only block-wide barrier: before the march starts
    }
    const float4* cpl = cps + lx;
    u64 cnp[NX / 2];                                    // KN: cos(pi x) at this lane's nodes, in pairs, and at the node right of them
    float cnh = 0.f;
    if constexpr (KN) {
#pragma unroll
        for (int h = 0; h < NX / 4; ++h) {
            const float4 q = __ldg(reinterpret_cast<const float4*>(P.cn[0] + x0c + 4 * h));
            cnp[2 * h] = r2_pack(q.x, q.y); cnp[2 * h + 1] = r2_pack(q.z, q.w);
        }
        cnh = __ldg(P.cn[0] + x0c + NX);
    }

    const long long su = ((long long)blockIdx.x * R2_WARPS + warp) * SUBS + sub;
    if (su >= G.units) return;                          // the other units of the warp synchronise among themselves only
    const int RS = G.RS;
    float* ring = smem + (KG ? 4 * NX * LW : 0) + (size_t)(warp * SUBS + sub) * R2_DEPTH * RS;
    const unsigned ring_s = (unsigned)__cvta_generic_to_shared(ring);
    const int UROW = NX * LW + 4;                       // floats of a node row in a slot (with the 4 floats of padding)
    const int COEF = ND ? 2 * UROW : UROW;              // offset of the coefficient row (ND: none; the nu row sits at UROW)
    const int H1 = 4 * LW + 4;                          // NX = 8: offset of the second 16 bytes of every lane

    const int b = (int)(su % P.batch);
    const int chunk = (int)(su / P.batch);
    const bool has_first = (x0 == 0), has_last = act && (x0 + NX == nx);
    const int n0 = chunk * G.R, n1 = min(n0 + G.R, ny);
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
    const float fw = P.f_const * P.hx * P.hy;           // nodal load of an interior node
    const bool hasf = (P.f_const != 0.f);
    const float gs = P.gJ ? __ldg(P.gJ + b) : 1.f;
    // Lane constants that make the march branch-free (as in the strip 2D kernel): lm = 0 in the first lane (nothing
    // arrives from the left); g3, ky3 = 0 in the lane whose last element lies right of node nx-1; output scale, nodal
    // load and load-energy weight of the lane's first / last node (Dirichlet columns).
    const float lm = (lx == 0) ? 0.f : 1.f;
    const float g3 = has_last ? 0.f : 1.f, ky3 = ky * g3;
    const float nl = -gs * fw;
    const float gsf = (has_first && !nomask) ? 0.f : gs, gsl = (has_last && !nomask) ? 0.f : gs;
    const float nlf = has_first ? (nomask ? 0.5f * nl : 0.f) : nl, nll = has_last ? (nomask ? 0.5f * nl : 0.f) : nl;
    const float wf = has_first ? 0.5f : 1.f, wl = has_last ? 0.5f : 1.f;

    // ---- the ring: step i = j - jbeg uses slot i % DEPTH, which holds node row j + 1, (ND) the nu row j + 1, and the
    // coefficients of element row j (KG) or of node row j + 1 (KN)
    for (int s = lx; s < R2_DEPTH; s += LW) {           // the 4 floats right of the last lane's nodes stay zero
        *reinterpret_cast<float4*>(ring + (size_t)s * RS + 4 * LW) = make_float4(0.f, 0.f, 0.f, 0.f);
        if constexpr (ND) *reinterpret_cast<float4*>(ring + (size_t)s * RS + UROW + 4 * LW) = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    int fetch = jbeg;                                   // next element row to fetch
    unsigned pfo = 0;                                   // byte offset of the slot it goes to
    const unsigned RSB = 4u * RS, RINGB = R2_DEPTH * RSB;
    const float* usrc = ub + (size_t)(jbeg + 1) * nx;
    const float* nsrc = ND ? P.nu + (size_t)b * P.nodes + x0c + (size_t)(jbeg + 1) * nx : nullptr;
    const int clx = (lx < CFQ) ? lx : 0;
    const float* polyb = rowpoly + (size_t)b * (KN ? ny : ny - 1) * GS;
    const float* csrc = polyb + (size_t)(KN ? jbeg + 1 : jbeg) * GS + 4 * clx;
    const unsigned d0 = ring_s + 16u * lx, d1 = ring_s + 4u * H1 + 16u * lx, dc = ring_s + 4u * COEF + 16u * clx;
    auto issue = [&]() {
        if (fetch <= jend) {                            // uniform in the unit
            r2_cp16(d0 + pfo, usrc);
            if constexpr (NX == 8) r2_cp16(d1 + pfo, usrc + 4);
            if constexpr (ND) {
                r2_cp16(d0 + 4u * UROW + pfo, nsrc);
                if constexpr (NX == 8) r2_cp16(d1 + 4u * UROW + pfo, nsrc + 4);
            } else {
                r2_cp16_if(dc + pfo, csrc, (lx < CFQ) ? 1 : 0);
                if constexpr (CFQ > 8) r2_cp16_if(dc + pfo + 16u * 8u, csrc + 32, (lx + 8 < CFQ && LW == 8) ? 1 : 0);
            }
        }
        r2_commit();                                    // one group per step, possibly empty
        ++fetch; usrc += nx; csrc += GS;
        if constexpr (ND) nsrc += nx;
        pfo += RSB;
        if (pfo == RINGB) pfo = 0;
    };
#pragma unroll
    for (int d = 0; d < R2_DEPTH - 1; ++d) issue();

    // a node row of u (or nu) from global memory / from a slot: the lane's NX nodes and the node right of them
    auto ldrow_g = [&](const float* p, float (&v)[NX + 1]) {
#pragma unroll
        for (int h = 0; h < NX / 4; ++h) {
            const float4 q = __ldg(reinterpret_cast<const float4*>(p + 4 * h));
            v[4 * h] = q.x; v[4 * h + 1] = q.y; v[4 * h + 2] = q.z; v[4 * h + 3] = q.w;
        }
        const float rn = __shfl_down_sync(submask, v[0], 1, LW);
        v[NX] = (lx == LW - 1 || has_last) ? 0.f : rn;
    };
    auto ldrow_s = [&](const float* slot, float (&v)[NX + 1]) {
        const float4 q = *reinterpret_cast<const float4*>(slot + 4 * lx);
        v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
        if constexpr (NX == 8) {
            const float4 q1 = *reinterpret_cast<const float4*>(slot + H1 + 4 * lx);
            v[4] = q1.x; v[5] = q1.y; v[6] = q1.z; v[7] = q1.w;
        }
        v[NX] = slot[4 * (lx + 1)];                     // first node of the next lane, or the zero pad
    };

    // ---- state of the node row below the current element row
    float lo[NX + 1], cu[NX + 1], ehor[NX], U[NX];
    ldrow_g(ub + (size_t)jbeg * nx, lo);
    if (impose) {
        if (has_first) lo[0] = bc0;
        if (has_last) lo[NX - 1] = bc1;
    }
#pragma unroll
    for (int k = 0; k < NX; ++k) { ehor[k] = lo[k + 1] - lo[k]; U[k] = 0.f; }

    // KN: nu at this lane's NX nodes and at the node right of them, from the polynomial of that node row
    auto nu_row = [&](const u64 (&gg)[GS / 2], float (&nn)[NX + 1]) {
#pragma unroll
        for (int h = 0; h < NX / 2; ++h) {
            u64 e = gg[M];
#pragma unroll
            for (int i = M - 1; i >= 0; --i) e = r2_fma2(e, cnp[h], gg[i]);
            float e0, e1;
            r2_unpack(e, e0, e1);
            nn[2 * h] = r2_ex2(e0); nn[2 * h + 1] = r2_ex2(e1);
        }
        float gh, dmy;
        r2_unpack(gg[M], gh, dmy);
#pragma unroll
        for (int i = M - 1; i >= 0; --i) { float gi; r2_unpack(gg[i], gi, dmy); gh = fmaf(gh, cnh, gi); }
        nn[NX] = r2_ex2(gh);
    };
    float nlo[NX + 1], hnu[NX];                         // KN, ND: nu on the node row below and its sums over x-neighbours
    if constexpr (ND) ldrow_g(P.nu + (size_t)b * P.nodes + x0c + (size_t)jbeg * nx, nlo);
    if constexpr (KN) {
        u64 gg[GS / 2];
        const ulonglong2* gp = reinterpret_cast<const ulonglong2*>(polyb + (size_t)jbeg * GS);
#pragma unroll
        for (int k = 0; k < GS / 4; ++k) { const ulonglong2 t = __ldg(gp + k); gg[2 * k] = t.x; gg[2 * k + 1] = t.y; }
        nu_row(gg, nlo);
    }
    if constexpr (KN || ND) {
#pragma unroll
        for (int k = 0; k < NX; ++k) hnu[k] = nlo[k] + nlo[k + 1];
    }

    float en = 0.f, ell = 0.f;                          // sum u (K u) and sum w u of the rows this lane went over
    float* rrow = rb + (size_t)jbeg * nx;
    unsigned rdo = 0;                                   // byte offset of the slot to read

    // One element row: a holds node row j, c receives node row j + 1.
    auto step = [&](float (&a)[NX + 1], float (&c)[NX + 1], const int j) {
        r2_wait<R2_DEPTH - 2>();                        // this step's slot has landed (for the lanes that copied it)
        __syncwarp(submask);                            // ... is visible to the unit, and the slot read last step is free
        issue();                                        // refill it
        const float* slot = reinterpret_cast<const float*>(reinterpret_cast<const char*>(ring) + rdo);
        rdo += RSB;
        if (rdo == RINGB) rdo = 0;
        ldrow_s(slot, c);
        if (impose) {
            if (has_first) c[0] = bc0;
            if (has_last) c[NX - 1] = bc1;
        }
        u64 g2[GS / 2];
        if constexpr (!ND) {
            const ulonglong2* gp = reinterpret_cast<const ulonglong2*>(slot + COEF);
#pragma unroll
            for (int k = 0; k < GS / 4; ++k) { const ulonglong2 t = gp[k]; g2[2 * k] = t.x; g2[2 * k + 1] = t.y; }
        }
        float ncur[NX + 1];
        if constexpr (KN) nu_row(g2, ncur);
        if constexpr (ND) ldrow_s(slot + UROW, ncur);

        float Q0 = 0.f, SY0 = 0.f, R0 = 0.f, Qp = 0.f, Tp = 0.f, rout[NX];
#pragma unroll
        for (int k = 0; k < NX; ++k) {
            const float e1 = c[k + 1] - c[k];
            const float s0 = c[k] - a[k];
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
                const ulonglong2 cc = *reinterpret_cast<const ulonglong2*>(cpl + k * LW);
                u64 ea = g2[M], eb = g2[M];             // (row a, row b) pairs at column a / column b
#pragma unroll
                for (int i = M - 1; i >= 0; --i) { ea = r2_fma2(ea, cc.x, g2[i]); eb = r2_fma2(eb, cc.y, g2[i]); }
                float xaa, xab, xba, xbb;
                r2_unpack(ea, xaa, xab);
                r2_unpack(eb, xba, xbb);
                const float naa = r2_ex2(xaa), nab = r2_ex2(xab), nba = r2_ex2(xba), nbb = r2_ex2(xbb);
                Na = naa + nba; Nb = nab + nbb; Ma = naa + nab; Mb = nba + nbb;
            }
            const float Gxa = Na * Dxa, Gxb = Nb * Dxb, Gya = Ma * Dya, Gyb = Mb * Dyb;
            const float SXu = Gxa + Gxb, SYu = Gya + Gyb;
            float T = kxa * Gxa;
            T = fmaf(kxb, Gxb, T); T = fmaf(kya, Gya, T); T = fmaf(kyb, Gyb, T);
            const float Q = fmaf(kx, SXu, -T);
            const float Rr = fmaf(ky, SYu, -T);
            if (k == 0) {
                Q0 = Q; SY0 = SYu; R0 = Rr;
            } else if (k < NX - 1) {
                rout[k] = fmaf(-ky, SYu, Qp - Q) + U[k];
                U[k] = Rr + Tp;
            } else {                                    // the lane's last element may lie beyond the grid (g3 = 0)
                rout[k] = fmaf(-ky3, SYu, fmaf(-g3, Q, Qp)) + U[k];
                U[k] = fmaf(g3, Rr, Tp);
            }
            Qp = Q; Tp = T;
        }
        // contributions of the element left of this lane's first node
        const float ql = __shfl_up_sync(submask, Qp, 1, LW);
        const float tl = __shfl_up_sync(submask, Tp, 1, LW);
        rout[0] = fmaf(-ky, SY0, fmaf(ql, lm, -Q0)) + U[0];
        U[0] = fmaf(tl, lm, R0);
        if (j >= n0) {                                  // uniform: this unit owns node row j
            // rout is (K u) of node row j: Euler's identity gives the diffusion energy
            const float wrow = (j == 0) ? 0.5f : 1.f;
            float o[NX];
#pragma unroll
            for (int k = 0; k < NX; ++k) {
                en = fmaf(a[k], rout[k], en);
                const float s = (k == 0) ? gsf : (k == NX - 1) ? gsl : gs;
                const float l = (k == 0) ? nlf : (k == NX - 1) ? nll : nl;
                o[k] = fmaf(s, rout[k], wrow * l);
            }
            if (hasf) {
                float w = wf * a[0];
#pragma unroll
                for (int k = 1; k < NX - 1; ++k) w += a[k];
                ell = fmaf(wrow, fmaf(wl, a[NX - 1], w), ell);
            }
            if (act) {
#pragma unroll
                for (int h = 0; h < NX / 4; ++h)
                    *reinterpret_cast<float4*>(rrow + 4 * h) = make_float4(o[4 * h], o[4 * h + 1], o[4 * h + 2], o[4 * h + 3]);
            }
        }
        rrow += nx;
        if constexpr (KN || ND) {
#pragma unroll
            for (int k = 0; k <= NX; ++k) nlo[k] = ncur[k];
        }
    };

    {
        int j = jbeg;
        while (true) {
            step(lo, cu, j);
            if (++j > jend) {
#pragma unroll
                for (int k = 0; k < NX; ++k) lo[k] = cu[k];
                break;
            }
            step(cu, lo, j);
            if (++j > jend) break;
        }
    }
    r2_wait<0>();

    // ---- the top node row of the grid has no element row above it (lo holds it, U what it received)
    if (n1 == ny) {
        float o[NX];
#pragma unroll
        for (int k = 0; k < NX; ++k) {
            en = fmaf(lo[k], U[k], en);
            const float s = (k == 0) ? gsf : (k == NX - 1) ? gsl : gs;
            const float l = (k == 0) ? nlf : (k == NX - 1) ? nll : nl;
            o[k] = fmaf(s, U[k], 0.5f * l);
        }
        float w = wf * lo[0];
#pragma unroll
        for (int k = 1; k < NX - 1; ++k) w += lo[k];
        ell = fmaf(0.5f, fmaf(wl, lo[NX - 1], w), ell);
        if (act) {
            float* rtop = rb + (size_t)(ny - 1) * nx;
#pragma unroll
            for (int h = 0; h < NX / 4; ++h)
                *reinterpret_cast<float4*>(rtop + 4 * h) = make_float4(o[4 * h], o[4 * h + 1], o[4 * h + 2], o[4 * h + 3]);
        }
    }

    // ---- energy partial of this unit: its lanes summed in a fixed order in double
    double d = act ? 0.5 * (double)en : 0.0, l = (act && hasf) ? (double)fw * (double)ell : 0.0;
    for (int off = LW >> 1; off > 0; off >>= 1) {
        d += __shfl_down_sync(submask, d, off, LW);
        l += __shfl_down_sync(submask, l, off, LW);
    }
    if (lx == 0) {
        double* slot = P.partials + 2 * ((size_t)b * P.nblk + chunk);
        slot[0] = d; slot[1] = l;
    }
}

int r2_sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
        (void)cudaGetLastError();
        n = 148;
    }
    return n;
}

int r2_nxl(int nx) { return (nx > 128) ? 8 : 4; }       // nodes per lane
int r2_minb(int nxl) { return (nxl == 8) ? 3 : 4; }     // resident blocks of 4 warps per SM the kernel is compiled for

R2Geo geometry_r_search(const dn_problem& p) {
    R2Geo g{};
    const int nx = p.grid.nx, ny = p.grid.ny;
    const int NX = r2_nxl(nx);
    g.LW = 8; g.lwsh = 3;
    while (g.LW * NX < nx) { g.LW *= 2; ++g.lwsh; }
    const int urow = NX * g.LW + 4;
    g.RS = (p.nu_mode == DN_NU_NODAL) ? 2 * urow : urow + r2_gs(p.kl_modes);
    const long long slots = (long long)r2_sm_count() * r2_minb(NX) * R2_WARPS * (32 / g.LW);
    // R from a cost search over whole waves of units; a unit pays the recomputed row and the filling of its ring
    long long best = -1;
    int bestR = 2;
    for (int R = 2; R <= 1024; ++R) {
        if (R > ny && R > 2) break;
        const long long nch = (ny + R - 1) / R;
        const long long units = (long long)p.batch * nch;
        const long long waves = (units + slots - 1) / slots;
        const long long cost = waves * (R + 5) * 1000 + (1000 / R);      // prefer less redundancy on ties
        if (best < 0 || cost < best) { best = cost; bestR = R; }
    }
    g.R = bestR;
    g.nchunk = (ny + g.R - 1) / g.R;
    g.units = (long long)p.batch * g.nchunk;
    return g;
}

R2Geo geometry_r(const dn_problem& p) {
    return memo_geometry<R2Geo>(p, r2_sm_count(), [&]() { return geometry_r_search(p); });
}

template <int NX, int M, int MODE, int MINB, int LWC>
cudaError_t launch_rl(const Params& P, const float* rowpoly, const R2Geo& g, cudaStream_t s) {
    const int subs = 32 / g.LW;
    const size_t smem = sizeof(float) * ((size_t)R2_WARPS * subs * r2_depth(MODE) * g.RS + (MODE == 0 ? 4 * NX * g.LW : 0));
    const long long per_block = (long long)R2_WARPS * subs;
    const unsigned blocks = (unsigned)((g.units + per_block - 1) / per_block);
    const cudaError_t e = cudaFuncSetAttribute(row2d_kernel<NX, M, MODE, MINB, LWC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return launch_dependent(row2d_kernel<NX, M, MODE, MINB, LWC>, dim3(blocks), dim3(R2_WARPS * 32), smem, s, P, rowpoly, g);
}

template <int NX, int M, int MODE, int MINB>
cudaError_t launch_r(const Params& P, const float* rowpoly, const R2Geo& g, cudaStream_t s) {
    if (g.LW == 32) return launch_rl<NX, M, MODE, MINB, 32>(P, rowpoly, g, s);
    if (g.LW == 16) return launch_rl<NX, M, MODE, MINB, 16>(P, rowpoly, g, s);
    return launch_rl<NX, M, MODE, MINB, 0>(P, rowpoly, g, s);
}

template <int M>
cudaError_t launch_rm(const Params& P, const float* rowpoly, const R2Geo& g, cudaStream_t s) {
    const bool wide = (r2_nxl(P.nx) == 8);
    if (P.nu_mode == DN_NU_KL_NODAL)
        return wide ? launch_r<8, M, 1, 3>(P, rowpoly, g, s) : launch_r<4, M, 1, 4>(P, rowpoly, g, s);
    return wide ? launch_r<8, M, 0, 3>(P, rowpoly, g, s) : launch_r<4, M, 0, 4>(P, rowpoly, g, s);
}

dn_problem r2_problem_of(const Params& P) {
    dn_problem p{};
    p.grid.dim = 2; p.grid.nx = P.nx; p.grid.ny = P.ny; p.grid.nz = 1; p.batch = P.batch;
    p.nu_mode = P.nu_mode; p.kl_modes = P.m;
    return p;
}

}  // namespace

// Rows of at most 128 nodes take 4 nodes per lane, rows of at most 256 nodes 8 (then nx must be a multiple of 8, so that
// only the last element of the last lane falls outside the grid).  Constant forcing only.  With a stored nodal field the
// 8-node layout is slower than the tiled kernel (measured on 256-wide rows: 213 against 151 us per 67 M nodes on tall
// grids, 24.2 against 22.3 us on 256^2 x 64), so that mode stops at 128 nodes.
bool row2d_applicable(const dn_problem& p) {
    if (!(p.grid.dim == 2 && p.f == nullptr && p.grid.nx % 4 == 0 && p.grid.nx >= 8 && p.grid.nx <= 256 && p.grid.ny >= 2))
        return false;
    if (p.grid.nx <= 128) return true;
    return p.grid.nx % 8 == 0 && p.nu_mode != DN_NU_NODAL;
}

Launch row2d_geometry(const dn_problem& p) {
    const R2Geo g = geometry_r(p);
    Launch l{};
    l.path = PATH_ROW2D;
    l.nblk = g.nchunk;
    l.chunk = g.R;
    l.variant = g.LW;
    return l;
}

size_t row2d_rowpoly_floats(const dn_problem& p) {
    if (p.nu_mode == DN_NU_NODAL) return 0;                      // the stored field needs no table
    return (size_t)p.batch * p.grid.ny * r2_gs(p.kl_modes);      // ny - 1 element rows, or ny node rows (KL at the nodes)
}

cudaError_t launch_row2d(const Params& P, const float* rowpoly, cudaStream_t s) {
    const R2Geo g = geometry_r(r2_problem_of(P));
    if (P.nu_mode == DN_NU_NODAL) return (r2_nxl(P.nx) == 4) ? launch_r<4, 1, 2, 4>(P, rowpoly, g, s) : cudaErrorInvalidValue;
    switch (P.m) {
        case 1: return launch_rm<1>(P, rowpoly, g, s);
        case 2: return launch_rm<2>(P, rowpoly, g, s);
        case 3: return launch_rm<3>(P, rowpoly, g, s);
        case 4: return launch_rm<4>(P, rowpoly, g, s);
        case 5: return launch_rm<5>(P, rowpoly, g, s);
        case 6: return launch_rm<6>(P, rowpoly, g, s);
        case 7: return launch_rm<7>(P, rowpoly, g, s);
        case 8: return launch_rm<8>(P, rowpoly, g, s);
    }
    return cudaErrorInvalidValue;
}

}  // namespace dn
