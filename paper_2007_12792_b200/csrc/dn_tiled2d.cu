// Tiled 2D kernel: fused element quadrature, energy reduction, node gather, mask and store.
//
// Layout of the work.  A warp owns a strip of 128*K consecutive nodes in x (K float4 per lane,
// K = 1 or 2) and marches over a chunk of node rows in y; W warps side by side cover the row
// (nx <= 128*K*W), WY such warp rows share a block.  Per element row the warp holds the node
// row below in registers (as the row itself, its horizontal differences and the pending
// contributions to it) and loads the row above once with 128-bit loads; the x+1 neighbour comes
// from the next lane by shuffle, across warps through shared memory.  Every element is computed
// exactly once per block: its contributions to the two nodes on its left stay in the thread,
// those to the two nodes on its right go to the owner of element k+1, those to the upper row are
// carried to the next step of the march.  The first element row of a chunk is recomputed by the
// chunk below (1/R redundancy).  No atomics; the energy is reduced per thread, warp, block.
//
// Arithmetic of one element (corners u00 u10 / u01 u11, e0 = u10-u00, s0 = u01-u00,
// t = u11-u10-u01+u00):  d/dx at Gauss row q is (e0 + q t)/hx, d/dy at Gauss column p is
// (s0 + p t)/hy.  With N_q = sum_p nu_pq, M_p = sum_q nu_pq, Gx_q = N_q Dx_q, Gy_p = M_p Dy_p:
//   energy   = 1/2 (kx sum_q Gx_q Dx_q + ky sum_p Gy_p Dy_p),   kx = hy/(4hx), ky = hx/(4hy)
//   dE/de0   = kx (Gx_a + Gx_b),  dE/ds0 = ky (Gy_a + Gy_b),
//   dE/dt    = T = kx (a Gx_a + b Gx_b) + ky (a Gy_a + b Gy_b)
// and the chain rule gives the corner contributions  (T - dE/de0 - dE/ds0, dE/de0 - T,
// dE/ds0 - T, T).
//
// KL diffusivity at the Gauss points: cos(i pi x) = T_i(cos pi x), so for a fixed Gauss row the
// exponent is a polynomial of degree m in c = cos(pi x_p) whose coefficients are uniform along
// the row.  They are prepared per block in double (shared memory); each point then costs m FMAs
// (Horner) and one ex2.
#include "dn_internal.cuh"

namespace dn {

namespace {

constexpr int T2_MAX_WARPS = 8;

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void named_barrier(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

template <int M> struct GamStride { static constexpr int value = ((M + 1) + 3) / 4 * 4; };

template <int M>
__device__ __forceinline__ float horner(const float (&g)[GamStride<M>::value], float c) {
    float e = g[M];
#pragma unroll
    for (int k = M - 1; k >= 0; --k) e = fmaf(e, c, g[k]);
    return e;
}

// One node row of a strip: K float4 per lane plus the node right of the strip (lane 0 holds it).
template <int K>
struct Row {
    float v[K][4];
    float halo;
};

template <int K>
__device__ __forceinline__ void load_row(Row<K>& r, const float* __restrict__ row, const int (&xs)[K], int nx,
                                         int xhalo, int lane) {
#pragma unroll
    for (int s = 0; s < K; ++s) {
        if (xs[s] < nx) {
            const float4 q = __ldg(reinterpret_cast<const float4*>(row + xs[s]));
            r.v[s][0] = q.x; r.v[s][1] = q.y; r.v[s][2] = q.z; r.v[s][3] = q.w;
        } else {
            r.v[s][0] = r.v[s][1] = r.v[s][2] = r.v[s][3] = 0.f;
        }
    }
    r.halo = (lane == 0 && xhalo < nx) ? __ldg(row + xhalo) : 0.f;
}

// Value at the node right of segment s of each lane: the next lane's first value; for lane 31 the
// first value of the next segment of lane 0, or the halo node.
template <int K>
__device__ __forceinline__ void right_neighbours(const Row<K>& r, float (&rn)[K], int lane) {
#pragma unroll
    for (int s = 0; s < K; ++s) {
        const float wrap = (s + 1 < K) ? r.v[(s + 1 < K) ? s + 1 : s][0] : r.halo;
        const float send = (lane == 0) ? wrap : r.v[s][0];
        rn[s] = __shfl_sync(0xffffffffu, send, (lane + 1) & 31);
    }
}

template <int K, int M, bool WANT_R>
__global__ void __launch_bounds__(256, 2)
tiled2d_kernel(const Params P, const int W, const int WY, const int R) {
    extern __shared__ __align__(16) float smem[];
    constexpr bool KL = (M > 0);
    constexpr int GS = GamStride<KL ? M : 1>::value;
    const int lane = threadIdx.x & 31;
    const int wid = threadIdx.x >> 5;
    const int wx = wid % W, wy = wid / W;
    const int b = blockIdx.y;
    const int nx = P.nx, ny = P.ny;
    const int chunk = blockIdx.x * WY + wy;
    const int n0 = chunk * R;
    const bool idle = (n0 >= ny);
    const int n1 = min(n0 + R, ny);
    const int jbeg = max(n0 - 1, 0);
    const int jend = min(n1 - 1, ny - 2);          // last element row of this chunk (inclusive)
    const int gam_rows = 2 * (R + 1);
    float* gam = smem + (size_t)wy * gam_rows * GS;
    float* xch = smem + (size_t)WY * gam_rows * (KL ? GS : 0) + (size_t)wy * 2 * T2_MAX_WARPS * 2;

    // ---- prologue: polynomial coefficients of the KL exponent for every Gauss row of the chunk
    if constexpr (KL) if (!idle) {
        const int count = 2 * (jend - jbeg + 1);
        const float* c = P.ckl + (size_t)b * M * M;
        for (int q = wx * 32 + lane; q < count; q += 32 * W) {
            const int gy = 2 * jbeg + q;
            double g[M > 0 ? M : 1];
#pragma unroll
            for (int i = 0; i < M; ++i) {
                double a = 0.0;
#pragma unroll
                for (int j = 0; j < M; ++j) a += (double)c[i * M + j] * (double)P.cg[1][j * P.gstride[1] + gy];
                g[i] = a;
            }
            // sum_i g_i T_i(c) in the monomial basis, T_{i+1} = 2 c T_i - T_{i-1}
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
            for (int k = 0; k < GS; ++k) gam[q * GS + k] = (k <= M) ? (float)acc[k <= M ? k : 0] : 0.f;
        }
    }
    __syncthreads();

    float enx = 0.f, eny = 0.f, enxl[K], enyl[K], ell = 0.f;
#pragma unroll
    for (int s = 0; s < K; ++s) { enxl[s] = 0.f; enyl[s] = 0.f; }

    if (!idle) {
        const int xw = wx * 128 * K;
        int xs[K];
#pragma unroll
        for (int s = 0; s < K; ++s) xs[s] = xw + 128 * s + 4 * lane;
        const int xhalo = xw + 128 * K;
        const float* ub = P.u + (size_t)b * P.nodes;
        const float* nub = KL ? nullptr : P.nu + (size_t)b * P.nodes;
        float* rb = WANT_R ? P.r + (size_t)b * P.nodes : nullptr;
        const bool impose = (P.flags & DN_IMPOSE_BC_ON_LOAD) != 0;
        const bool nomask = (P.flags & DN_NO_MASK) != 0;
        const float kx = 0.25f * P.hy / P.hx, ky = 0.25f * P.hx / P.hy;
        const float kxa = kx * DN_GA, kxb = kx * DN_GB, kya = ky * DN_GA, kyb = ky * DN_GB;
        const float fw = P.f_const * P.hx * P.hy;            // nodal load of an interior node
        const float gs = (WANT_R && P.gJ) ? __ldg(P.gJ + b) : 1.f;

        auto fix_bc = [&](Row<K>& r) {
            if (impose) {
#pragma unroll
                for (int s = 0; s < K; ++s) {
                    if (xs[s] == 0) r.v[s][0] = P.bc_x0;
                    if (xs[s] + 3 == nx - 1) r.v[s][3] = P.bc_x1;
                }
            }
        };

        // cos(pi x) at the two Gauss columns of each element
        float cpa[K][4], cpb[K][4];
        if constexpr (KL) {
#pragma unroll
            for (int s = 0; s < K; ++s) {
                if (xs[s] < nx) {
                    const float4 q0 = __ldg(reinterpret_cast<const float4*>(P.cg[0] + 2 * xs[s]));
                    const float4 q1 = __ldg(reinterpret_cast<const float4*>(P.cg[0] + 2 * xs[s] + 4));
                    cpa[s][0] = q0.x; cpb[s][0] = q0.y; cpa[s][1] = q0.z; cpb[s][1] = q0.w;
                    cpa[s][2] = q1.x; cpb[s][2] = q1.y; cpa[s][3] = q1.z; cpb[s][3] = q1.w;
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c) { cpa[s][c] = 0.f; cpb[s][c] = 0.f; }
                }
            }
        }

        // ---- state of the node row below the current element row
        Row<K> lo, nlo;
        float ehor[K][4], U[K][4], hnu[K][4], nlr[K];
        load_row<K>(lo, ub + (size_t)jbeg * nx, xs, nx, xhalo, lane);
        fix_bc(lo);
        {
            float rn[K];
            right_neighbours<K>(lo, rn, lane);
#pragma unroll
            for (int s = 0; s < K; ++s)
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    ehor[s][c] = ((c < 3) ? lo.v[s][c < 3 ? c + 1 : c] : rn[s]) - lo.v[s][c];
                    U[s][c] = 0.f;
                }
        }
        if (!KL) {
            load_row<K>(nlo, nub + (size_t)jbeg * nx, xs, nx, xhalo, lane);
            right_neighbours<K>(nlo, nlr, lane);
#pragma unroll
            for (int s = 0; s < K; ++s)
#pragma unroll
                for (int c = 0; c < 4; ++c) hnu[s][c] = nlo.v[s][c] + ((c < 3) ? nlo.v[s][c < 3 ? c + 1 : c] : nlr[s]);
        }
        Row<K> cur, ncur;
        load_row<K>(cur, ub + (size_t)(jbeg + 1) * nx, xs, nx, xhalo, lane);
        if (!KL) load_row<K>(ncur, nub + (size_t)(jbeg + 1) * nx, xs, nx, xhalo, lane);

        for (int j = jbeg; j <= jend; ++j) {
            // prefetch the row after next
            Row<K> nxt, nnxt;
            const bool more = (j < jend);
            if (more) {
                load_row<K>(nxt, ub + (size_t)(j + 2) * nx, xs, nx, xhalo, lane);
                if (!KL) load_row<K>(nnxt, nub + (size_t)(j + 2) * nx, xs, nx, xhalo, lane);
            }
            fix_bc(cur);
            const bool own = (j >= n0);
            float hir[K], nhr[K];
            right_neighbours<K>(cur, hir, lane);
            if (!KL) right_neighbours<K>(ncur, nhr, lane);

            float ga[GS], gb[GS];
            if constexpr (KL) {
                const float4* gp = reinterpret_cast<const float4*>(gam + (size_t)(2 * (j - jbeg)) * GS);
#pragma unroll
                for (int k = 0; k < GS / 4; ++k) {
                    const float4 a = gp[k], bq = gp[GS / 4 + k];
                    ga[4 * k] = a.x; ga[4 * k + 1] = a.y; ga[4 * k + 2] = a.z; ga[4 * k + 3] = a.w;
                    gb[4 * k] = bq.x; gb[4 * k + 1] = bq.y; gb[4 * k + 2] = bq.z; gb[4 * k + 3] = bq.w;
                }
            }

            // load energy of the node row below (owned rows only): f * hx hy * wy * sum_x wx u
            if (own) {
                float rs = 0.f;
#pragma unroll
                for (int s = 0; s < K; ++s) {
                    rs += (lo.v[s][0] + lo.v[s][1]) + (lo.v[s][2] + lo.v[s][3]);
                    if (xs[s] == 0) rs -= 0.5f * lo.v[s][0];
                    if (xs[s] + 3 == nx - 1) rs -= 0.5f * lo.v[s][3];
                }
                ell = fmaf((j == 0) ? 0.5f * fw : fw, rs, ell);
            }

            float Q0[K], SY0[K], R0[K], Q3[K], T3[K], rout[K][4];
#pragma unroll
            for (int s = 0; s < K; ++s) {
                float Qp = 0.f, Tp = 0.f;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float uh = cur.v[s][c];
                    const float un = (c < 3) ? cur.v[s][c < 3 ? c + 1 : c] : hir[s];
                    const float e1 = un - uh;
                    const float s0 = uh - lo.v[s][c];
                    const float e0 = ehor[s][c];
                    ehor[s][c] = e1;
                    const float t = e1 - e0;
                    const float Dxa = fmaf(DN_GA, t, e0), Dxb = fmaf(DN_GB, t, e0);
                    const float Dya = fmaf(DN_GA, t, s0), Dyb = fmaf(DN_GB, t, s0);
                    float Na, Nb, Ma, Mb;
                    if constexpr (KL) {
                        const float naa = ex2_approx(horner<M>(ga, cpa[s][c]));     // column a, row a
                        const float nab = ex2_approx(horner<M>(gb, cpa[s][c]));     // column a, row b
                        const float nba = ex2_approx(horner<M>(ga, cpb[s][c]));
                        const float nbb = ex2_approx(horner<M>(gb, cpb[s][c]));
                        Na = naa + nba; Nb = nab + nbb; Ma = naa + nab; Mb = nba + nbb;
                    } else {
                        const float n00 = nlo.v[s][c], n01 = ncur.v[s][c];
                        const float n10 = (c < 3) ? nlo.v[s][c < 3 ? c + 1 : c] : nlr[s];
                        const float n11 = (c < 3) ? ncur.v[s][c < 3 ? c + 1 : c] : nhr[s];
                        const float h0 = hnu[s][c], h1 = n01 + n11;
                        hnu[s][c] = h1;
                        const float v0 = n00 + n01, v1 = n10 + n11;
                        const float dh = h1 - h0, dv = v1 - v0;
                        Na = fmaf(DN_GA, dh, h0); Nb = fmaf(DN_GB, dh, h0);
                        Ma = fmaf(DN_GA, dv, v0); Mb = fmaf(DN_GB, dv, v0);
                    }
                    const float Gxa = Na * Dxa, Gxb = Nb * Dxb, Gya = Ma * Dya, Gyb = Mb * Dyb;
                    if (c < 3) {
                        enx = fmaf(Gxa, Dxa, enx); enx = fmaf(Gxb, Dxb, enx);
                        eny = fmaf(Gya, Dya, eny); eny = fmaf(Gyb, Dyb, eny);
                    } else {
                        enxl[s] = fmaf(Gxa, Dxa, enxl[s]); enxl[s] = fmaf(Gxb, Dxb, enxl[s]);
                        enyl[s] = fmaf(Gya, Dya, enyl[s]); enyl[s] = fmaf(Gyb, Dyb, enyl[s]);
                    }
                    if (WANT_R) {
                        const float SXu = Gxa + Gxb;
                        float SYu = Gya + Gyb;
                        float T = kxa * Gxa;
                        T = fmaf(kxb, Gxb, T); T = fmaf(kya, Gya, T); T = fmaf(kyb, Gyb, T);
                        float Q = fmaf(kx, SXu, -T);
                        float Rr = fmaf(ky, SYu, -T);
                        if (nomask && c == 3 && xs[s] + 3 == nx - 1) { T = 0.f; Q = 0.f; Rr = 0.f; SYu = 0.f; }
                        if (c == 0) {
                            Q0[s] = Q; SY0[s] = SYu; R0[s] = Rr;
                        } else {
                            const float rp = fmaf(-ky, SYu, Qp - Q);
                            rout[s][c] = rp + U[s][c];
                            U[s][c] = Rr + Tp;
                        }
                        Qp = Q; Tp = T;
                    }
                }
                if (WANT_R) { Q3[s] = Qp; T3[s] = Tp; }
            }

            if (WANT_R) {
                // contributions of the element left of each segment's first node
                float* slot = xch + (size_t)(j & 1) * T2_MAX_WARPS * 2;
                if (W > 1) {
                    if (lane == 31) { slot[2 * wx] = Q3[K - 1]; slot[2 * wx + 1] = T3[K - 1]; }
                    named_barrier(1 + wy, 32 * W);
                }
#pragma unroll
                for (int s = 0; s < K; ++s) {
                    const float sq = (lane == 31) ? ((s > 0) ? Q3[s > 0 ? s - 1 : 0] : 0.f) : Q3[s];
                    const float st = (lane == 31) ? ((s > 0) ? T3[s > 0 ? s - 1 : 0] : 0.f) : T3[s];
                    float ql = __shfl_sync(0xffffffffu, sq, (lane + 31) & 31);
                    float tl = __shfl_sync(0xffffffffu, st, (lane + 31) & 31);
                    if (s == 0 && lane == 0) {
                        if (W > 1 && wx > 0) { ql = slot[2 * (wx - 1)]; tl = slot[2 * (wx - 1) + 1]; }
                        else { ql = 0.f; tl = 0.f; }
                    }
                    const float rp = fmaf(-ky, SY0[s], ql - Q0[s]);
                    rout[s][0] = rp + U[s][0];
                    U[s][0] = R0[s] + tl;
                }
                if (own) {
                    const float lw = (j == 0) ? 0.5f * fw : fw;
                    const float nl = -gs * lw;
                    float* rrow = rb + (size_t)j * nx;
#pragma unroll
                    for (int s = 0; s < K; ++s) {
                        if (xs[s] < nx) {
                            float4 o;
                            o.x = fmaf(gs, rout[s][0], nl); o.y = fmaf(gs, rout[s][1], nl);
                            o.z = fmaf(gs, rout[s][2], nl); o.w = fmaf(gs, rout[s][3], nl);
                            if (xs[s] == 0) o.x = nomask ? gs * (rout[s][0] - 0.5f * lw) : 0.f;
                            if (xs[s] + 3 == nx - 1) o.w = nomask ? gs * (rout[s][3] - 0.5f * lw) : 0.f;
                            *reinterpret_cast<float4*>(rrow + xs[s]) = o;
                        }
                    }
                }
            }
            if (!own) {        // the warm-up row only seeds the carried contributions
                enx = 0.f; eny = 0.f;
#pragma unroll
                for (int s = 0; s < K; ++s) { enxl[s] = 0.f; enyl[s] = 0.f; }
            }
            // advance: the row above becomes the row below
            lo = cur;
            if (!KL) {
                nlo = ncur;
#pragma unroll
                for (int s = 0; s < K; ++s) nlr[s] = nhr[s];
            }
            if (more) { cur = nxt; if (!KL) ncur = nnxt; }
        }

        // ---- the top node row of the domain has no element row above it
        if (n1 == ny) {
            const float lw = 0.5f * fw;
            float rs = 0.f;
#pragma unroll
            for (int s = 0; s < K; ++s) {
                rs += (lo.v[s][0] + lo.v[s][1]) + (lo.v[s][2] + lo.v[s][3]);
                if (xs[s] == 0) rs -= 0.5f * lo.v[s][0];
                if (xs[s] + 3 == nx - 1) rs -= 0.5f * lo.v[s][3];
            }
            ell = fmaf(lw, rs, ell);
            if (WANT_R) {
                const float nl = -gs * lw;
                float* rrow = rb + (size_t)(ny - 1) * nx;
#pragma unroll
                for (int s = 0; s < K; ++s) {
                    if (xs[s] < nx) {
                        float4 o;
                        o.x = fmaf(gs, U[s][0], nl); o.y = fmaf(gs, U[s][1], nl);
                        o.z = fmaf(gs, U[s][2], nl); o.w = fmaf(gs, U[s][3], nl);
                        if (xs[s] == 0) o.x = nomask ? gs * (U[s][0] - 0.5f * lw) : 0.f;
                        if (xs[s] + 3 == nx - 1) o.w = nomask ? gs * (U[s][3] - 0.5f * lw) : 0.f;
                        *reinterpret_cast<float4*>(rrow + xs[s]) = o;
                    }
                }
            }
        }
        // the element right of the last node column does not exist: drop its energy
#pragma unroll
        for (int s = 0; s < K; ++s) {
            if (xs[s] + 3 < nx - 1) { enx += enxl[s]; eny += enyl[s]; }
        }
        enx *= kx; eny *= ky;
    }
    block_reduce_store(0.5 * ((double)enx + (double)eny), (double)ell,
                       P.partials + 2 * ((size_t)b * P.nblk + blockIdx.x));
}

struct Geo2 { int K, W, WY, R, nblkx, GS; size_t smem; };

int sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
        (void)cudaGetLastError();
        n = 148;
    }
    return n;
}

Geo2 geometry(const dn_problem& p) {
    Geo2 g{};
    const int nx = p.grid.nx, ny = p.grid.ny;
    g.K = (nx > 128) ? 2 : 1;
    g.W = (nx + 128 * g.K - 1) / (128 * g.K);
    g.WY = T2_MAX_WARPS / g.W;
    const int m = (p.nu_mode == DN_NU_KL_GAUSS) ? p.kl_modes : 0;
    g.GS = m ? ((m + 1) + 3) / 4 * 4 : 0;
    const long long slots = 2ll * sm_count();
    const int rmax_smem = g.GS ? (int)(40960 / ((size_t)g.WY * g.GS * 8)) - 1 : 4096;
    long long best = -1;
    int bestR = 16;
    for (int R = 8; R <= 512 && R <= rmax_smem; ++R) {
        if (R > ny && R > 8) break;
        const long long nch = (ny + R - 1) / R;
        const long long blocks = (long long)p.batch * ((nch + g.WY - 1) / g.WY);
        const long long waves = (blocks + slots - 1) / slots;
        const long long cost = waves * (R + 1) * 1000 + (1000 / R);      // prefer less redundancy on ties
        if (best < 0 || cost < best) { best = cost; bestR = R; }
    }
    g.R = bestR;
    const int nch = (ny + g.R - 1) / g.R;
    g.nblkx = (nch + g.WY - 1) / g.WY;
    g.smem = sizeof(float) * ((size_t)g.WY * 2 * (g.R + 1) * g.GS + (size_t)g.WY * 2 * T2_MAX_WARPS * 2);
    return g;
}

template <int K, int M>
cudaError_t launch_km(const Params& P, const Geo2& g, cudaStream_t s) {
    dim3 grid((unsigned)g.nblkx, (unsigned)P.batch);
    const int threads = 32 * g.W * g.WY;
    if (P.r) tiled2d_kernel<K, M, true><<<grid, threads, g.smem, s>>>(P, g.W, g.WY, g.R);
    else tiled2d_kernel<K, M, false><<<grid, threads, g.smem, s>>>(P, g.W, g.WY, g.R);
    return cudaGetLastError();
}

template <int K>
cudaError_t launch_k(const Params& P, const Geo2& g, cudaStream_t s) {
    switch (P.m) {
        case 0: return launch_km<K, 0>(P, g, s);
        case 1: return launch_km<K, 1>(P, g, s);
        case 2: return launch_km<K, 2>(P, g, s);
        case 3: return launch_km<K, 3>(P, g, s);
        case 4: return launch_km<K, 4>(P, g, s);
        case 5: return launch_km<K, 5>(P, g, s);
        case 6: return launch_km<K, 6>(P, g, s);
        case 7: return launch_km<K, 7>(P, g, s);
        case 8: return launch_km<K, 8>(P, g, s);
    }
    return cudaErrorInvalidValue;
}

}  // namespace

bool tiled2d_applicable(const dn_problem& p) {
    return p.grid.dim == 2 && p.grid.nx % 4 == 0 && p.grid.nx >= 8 && p.grid.nx <= 128 * 2 * T2_MAX_WARPS &&
           p.grid.ny >= 2;
}

Launch tiled2d_geometry(const dn_problem& p) {
    const Geo2 g = geometry(p);
    Launch l{};
    l.path = PATH_TILED2D;
    l.nblk = g.nblkx;
    l.chunk = g.R;
    l.variant = g.K;
    return l;
}

cudaError_t launch_tiled2d(const Params& P, const Launch& l, cudaStream_t s) {
    dn_problem p{};
    p.grid.dim = 2; p.grid.nx = P.nx; p.grid.ny = P.ny; p.grid.nz = 1; p.batch = P.batch;
    p.nu_mode = P.nu_mode; p.kl_modes = P.m;
    const Geo2 g = geometry(p);
    (void)l;
    return (g.K == 2) ? launch_k<2>(P, g, s) : launch_k<1>(P, g, s);
}

}  // namespace dn
