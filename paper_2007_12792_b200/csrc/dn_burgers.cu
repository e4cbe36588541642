// Finite-difference loss of the inviscid Burgers equation and its exact gradient
// ("Introduction", Eq. (Inviscid_Burgers); "DiffNets", Eq. (diffnetloss), Eq. (pde_loss),
// Eq. (boundaryloss); first derivatives by 3x3 Sobel stencils, "Implementing the forward model").
//
// With a = 2 hx ht res (zero outside the interior) and b = a u, the gradient of L_p separates:
//
//   g(j,i) = ct [ A(j-1,i) - A(j+1,i) ]                       A(j,i) = a(j,i-1) + 2 a(j,i) + a(j,i+1)
//          + cx [ D(j-1,i) + 2 D(j,i) + D(j+1,i) ]            D(j,i) = b(j,i-1) - b(j,i+1)
//          + a(j,i) u_x(j,i)                                  ct = 1/(8 ht), cx = 1/(8 hx)
//
// and the Sobel derivatives themselves are a central difference smoothed by (1,2,1) across the
// other axis.  The differences are taken first: neighbouring values of a smooth field are close, so
// their difference is (nearly) exact in fp32, which the sum-first order would not give.
//
// Marching kernel.  One warp owns 120 columns and a chunk of R rows of g.  Lane l holds the four
// columns x0 + 4 l .. + 3 of the rows in flight, x0 = 120 w - 4, so lanes 0 and 31 are halo lanes:
// they compute a and b for the column next to the warp's range and store nothing.  The warp walks up
// in t.  Row n of u arrives through a per-warp ring in shared memory (cp.async, 16 bytes per lane,
// RING-1 rows in flight; a lane reads back only what it copied, so the ring needs no barrier); with
// rows n-2, n-1, n in registers the residual of row n-1 is formed, and with it row n-2 of g is
// complete and stored.  Column neighbours come by shuffle.  Register state rotates by name (the loop
// body is unrolled over the six phases of the 3-row and 2-row rotations).  u is read once (plus
// 4/R of it again at chunk seams and 8/120 at warp seams, mostly from L2), g is written once.  No
// atomics: every warp writes its partial sums to a slot of its own and a second kernel adds them.
#include "dn_internal.cuh"

namespace dn {
namespace {

constexpr int BG_WARPS = 8;          // warps per block
constexpr int BG_RING = 6;           // ring slots per warp (BG_RING - 1 rows in flight), a multiple of 6: the step
                                     // phases (3-row and 2-row rotations of the register state) name the slots
static_assert(BG_RING % 6 == 0, "ring slots are named by the step phase");
constexpr int BG_COLS = 120;         // columns of g per warp
constexpr int BG_SMS = 148;
constexpr int BG_BLOCKS_PER_SM = 2;

struct BParams {
    int nx, nt, batch;
    int R, nchunk, wx, nslot;
    long long tasks;
    float ct, cx, w2;                // 1/(8 ht), 1/(8 hx), 2 hx ht
    float bx, bt;                    // lambda 2 hx, lambda 2 ht
    const float* u;
    const float* c;
    const float* gL;
    float* g;
    double* partials;                // [B][nslot][3]: sum res^2, sum (u - u0)^2 on row 0, sum u^2 on column 0
};

// 16-byte asynchronous copy into the ring slot at byte offset OFF of smem_base: n = 16 bytes are read from gsrc, or
// n = 0 and the slot is filled with zeros.
template <int OFF>
__device__ __forceinline__ void cp_async16_zfill(unsigned smem_base, const float* gsrc, int n) {
    asm volatile("cp.async.cg.shared.global [%0+%3], [%1], 16, %2;" ::"r"(smem_base), "l"(gsrc), "r"(n), "n"(OFF) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

struct MarchState {
    float u[3][6];                   // rows n-2, n-1, n (rotating), columns -1 .. 4 of this lane
    float Dx[2][4];                  // u(i+1) - u(i-1) of the two previous rows
    float Ax[2][4], Db[2][4], P[2][4];
};

struct MarchCtx {
    const float* ub;                 // this sample's field
    const float* psrc;               // this lane's four columns of the row that is copied next
    float* pg;                       // this lane's four columns of the row of g that is stored next
    unsigned ring_s;                 // this lane's entry of ring slot 0 (shared-space address)
    int nt_lane;                     // nt, or a negative number for lanes past the field (nothing to copy)
    int src_stride, src_bytes;       // nx and 16, or 0 and 0 for lanes past the field
    int j0, j1;
    bool store;                      // this lane's four columns exist and belong to this warp's range
    bool col0, colN;                 // this lane's first column is x = 0 / its last column is x = nx-1
    int nx;
    float ct, cx, s;                 // s = 2 hx ht gL
    float bts0, m0;                  // lambda 2 ht gL and 1 in the lane that holds column x = 0, else 0 and 0
    float ef, ebf;                   // running sums of res^2 and of u(0,t)^2 since the last flush
    double e, ebt;
};

// One step of the march: row n of u lands (ring slot PH), the residual of row n-1 is formed, row n-2 of g leaves.
// EDGE steps test every row index against the field and the chunk; the others are known to be clear of all edges.
template <int PH, bool EDGE, bool WANT_G>
__device__ __forceinline__ void march_step(MarchState& S, MarchCtx& C, int n) {
    constexpr int iu = PH % 3, ic = (PH + 2) % 3, im = (PH + 1) % 3;
    constexpr int p0 = PH % 2, p1 = 1 - p0;
    cp_wait<BG_RING - 2>();
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4+%5];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(C.ring_s), "n"(PH * 512) : "memory");
    {
        // row n + BG_RING - 1 goes to the slot that row n-1 has just left; away from the edges that row exists
        constexpr int off = ((PH + BG_RING - 1) % BG_RING) * 512;
        if (EDGE) {
            const int nn = n + BG_RING - 1;
            const bool ok = nn >= 0 && nn < C.nt_lane;
            cp_async16_zfill<off>(C.ring_s, ok ? C.psrc : C.ub, ok ? 16 : 0);
        } else {
            cp_async16_zfill<off>(C.ring_s, C.psrc, C.src_bytes);
        }
        cp_commit();
        C.psrc += C.src_stride;
    }
    S.u[iu][1] = v.x; S.u[iu][2] = v.y; S.u[iu][3] = v.z; S.u[iu][4] = v.w;
    S.u[iu][0] = __shfl_up_sync(0xffffffffu, v.w, 1);
    S.u[iu][5] = __shfl_down_sync(0xffffffffu, v.x, 1);

    float ux[4], a[6], b[6], res[4];
    const int q = n - 1;                                        // residual row
    const bool rowok = !EDGE || (q >= 1 && q <= C.nt_lane - 2 && q >= C.j0 - 1);
    const float s = rowok ? C.s : 0.0f;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const float dxn = S.u[iu][c + 2] - S.u[iu][c];
        ux[c] = C.cx * (S.Dx[p0][c] + dxn + 2.0f * S.Dx[p1][c]);
        S.Dx[p0][c] = dxn;
    }
    float dt[6];
#pragma unroll
    for (int c = 0; c < 6; ++c) dt[c] = S.u[iu][c] - S.u[im][c];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const float dts = dt[c] + dt[c + 2] + 2.0f * dt[c + 1];
        res[c] = C.ct * dts + S.u[ic][c + 1] * ux[c];
        if (c == 0 && C.col0) res[c] = 0.0f;                // the residual lives at interior columns only (lanes past
        if (c == 3 && C.colN) res[c] = 0.0f;                // the field carry s = 0)
        a[c + 1] = res[c] * s;
        b[c + 1] = a[c + 1] * S.u[ic][c + 1];
    }
    if (!EDGE || (rowok && q >= C.j0 && q < C.j1))              // lanes that store nothing drop their sum at the end
        C.ef += res[0] * res[0] + res[1] * res[1] + (res[2] * res[2] + res[3] * res[3]);
    a[0] = __shfl_up_sync(0xffffffffu, a[4], 1);
    a[5] = __shfl_down_sync(0xffffffffu, a[1], 1);
    b[0] = __shfl_up_sync(0xffffffffu, b[4], 1);
    b[5] = __shfl_down_sync(0xffffffffu, b[1], 1);

    float g[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const float axn = a[c] + a[c + 2] + 2.0f * a[c + 1];
        const float dbn = b[c] - b[c + 2];
        const float pn = a[c + 1] * ux[c];
        g[c] = C.ct * (S.Ax[p1][c] - axn) + C.cx * (S.Db[p1][c] + dbn + 2.0f * S.Db[p0][c]) + S.P[p0][c];
        S.Ax[p1][c] = axn; S.Db[p1][c] = dbn; S.P[p1][c] = pn;
    }
    const int jr = n - 2;                                       // row of g that is now complete
    if (!EDGE || (jr >= C.j0 && jr < C.j1)) {
        const float w = S.u[im][1];                             // inflow term of L_b: only the lane with x = 0 has m0, bts0 != 0
        g[0] = fmaf(C.bts0, w, g[0]);
        C.ebf = fmaf(w * C.m0, w, C.ebf);
        if (WANT_G && C.store) __stcs(reinterpret_cast<float4*>(C.pg), make_float4(g[0], g[1], g[2], g[3]));
    }
    C.pg += C.nx;
}

__device__ __forceinline__ void flush_sums(MarchCtx& C) {
    C.e += (double)C.ef; C.ef = 0.0f;
    C.ebt += (double)C.ebf; C.ebf = 0.0f;
}

// COUNT consecutive steps starting in phase K (mod BG_RING) at row n, unrolled at compile time.
template <int K, int COUNT, bool EDGE, bool WANT_G>
struct StepSeq {
    static __device__ __forceinline__ void run(MarchState& S, MarchCtx& C, int n) {
        march_step<K % BG_RING, EDGE, WANT_G>(S, C, n);
        StepSeq<K + 1, COUNT - 1, EDGE, WANT_G>::run(S, C, n + 1);
    }
    // the same, stopping in front of row nend; advances n; false once nend has been reached
    static __device__ __forceinline__ bool run_until(MarchState& S, MarchCtx& C, int& n, int nend) {
        if (n >= nend) return false;
        march_step<K % BG_RING, EDGE, WANT_G>(S, C, n);
        ++n;
        return StepSeq<K + 1, COUNT - 1, EDGE, WANT_G>::run_until(S, C, n, nend);
    }
};
template <int K, bool EDGE, bool WANT_G>
struct StepSeq<K, 0, EDGE, WANT_G> {
    static __device__ __forceinline__ void run(MarchState&, MarchCtx&, int) {}
    static __device__ __forceinline__ bool run_until(MarchState&, MarchCtx&, int&, int) { return true; }
};

template <bool WANT_G>
__global__ void __launch_bounds__(BG_WARPS * 32, BG_BLOCKS_PER_SM) burgers_march_kernel(BParams Q) {
    __shared__ float4 ring_all[BG_WARPS][BG_RING][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long task = (long long)blockIdx.x * BG_WARPS + warp;
    if (task >= Q.tasks) return;                                // whole warps leave; nothing below synchronises the block
    const int w = (int)(task % Q.wx);
    const int chunk = (int)((task / Q.wx) % Q.nchunk);
    const int bi = (int)(task / ((long long)Q.wx * Q.nchunk));

    MarchCtx C;
    C.nx = Q.nx;
    C.j0 = chunk * Q.R;
    C.j1 = min(C.j0 + Q.R, Q.nt);
    const int xl = BG_COLS * w - 4 + 4 * lane;
    const bool xvalid = xl >= 0 && xl < Q.nx;
    C.nt_lane = xvalid ? Q.nt : -(1 << 30);
    C.store = xvalid && lane >= 1 && lane <= 30;
    C.col0 = xl == 0;
    C.colN = xl + 4 == Q.nx;
    C.ub = Q.u + (size_t)bi * Q.nt * Q.nx;
    float* const gb = WANT_G ? Q.g + (size_t)bi * Q.nt * Q.nx : nullptr;
    C.ring_s = (unsigned)__cvta_generic_to_shared(&ring_all[warp][0][lane]);
    const float gl = Q.gL ? Q.gL[bi] : 1.0f;
    C.src_stride = xvalid ? Q.nx : 0;
    C.src_bytes = xvalid ? 16 : 0;
    C.ct = Q.ct; C.cx = Q.cx; C.s = xvalid ? Q.w2 * gl : 0.0f;
    C.bts0 = C.col0 ? Q.bt * gl : 0.0f;
    C.m0 = C.col0 ? 1.0f : 0.0f;
    C.e = 0.0; C.ebt = 0.0; C.ef = 0.0f; C.ebf = 0.0f;

    MarchState S;
#pragma unroll
    for (int r = 0; r < 3; ++r)
#pragma unroll
        for (int c = 0; c < 6; ++c) S.u[r][c] = 0.0f;
#pragma unroll
    for (int r = 0; r < 2; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) { S.Dx[r][c] = 0.0f; S.Ax[r][c] = 0.0f; S.Db[r][c] = 0.0f; S.P[r][c] = 0.0f; }

    // Rows n = nbeg .. nend-1 are walked.  Steps with  j0 + 2 <= n < min(j1 + 1, nt),  whose copy also stays at or
    // after row 0, touch no edge of the field or of the chunk.
    const int nbeg = C.j0 - 2, nend = C.j1 + 2;
    const int nfull1 = min(C.j1 + 1, Q.nt);
    {
        const float* p = C.ub + ((long long)nbeg * Q.nx + xl);  // not dereferenced unless the row exists
#pragma unroll
        for (int d = 0; d < BG_RING - 1; ++d) {
            const int nn = nbeg + d;
            const bool ok = nn >= 0 && nn < C.nt_lane;
            const unsigned dst = C.ring_s + d * 512;
            cp_async16_zfill<0>(dst, ok ? p : C.ub, ok ? 16 : 0);
            cp_commit();
            p += Q.nx;
        }
        C.psrc = xvalid ? p : C.ub;
        C.pg = gb + ((long long)(nbeg - 2) * Q.nx + xl);
    }
    // The first four steps (two rows to fill the registers, one residual row below the chunk, one row without a
    // complete g) and the last few take the EDGE variant; in between, groups of BG_RING edge-free steps run unchecked.
    int n = nbeg;
    StepSeq<0, 4, true, WANT_G>::run(S, C, n);
    n += 4;
    const int nmain1 = min(nfull1, Q.nt - (BG_RING - 1));       // ... and their copies stay inside the field
    while (n + BG_RING <= nmain1) {
        StepSeq<4, BG_RING, false, WANT_G>::run(S, C, n);
        n += BG_RING;
        flush_sums(C);
    }
    while (StepSeq<4, BG_RING, true, WANT_G>::run_until(S, C, n, nend)) flush_sums(C);
    flush_sums(C);
    if (!C.store) C.e = 0.0;
    cp_wait<0>();                                               // copies issued past the last row (zero-fill or unused rows)

    // Initial-condition term of L_b on row 0 (first chunk only): this lane adds it to the row it stored itself.
    double e0 = 0.0;
    if (C.j0 == 0 && C.store) {
        const float4 uv = *reinterpret_cast<const float4*>(C.ub + xl);
        const float uu[4] = {uv.x, uv.y, uv.z, uv.w};
        const double cc = (double)Q.c[bi];
        const float bxs = Q.bx * gl;
        float d[4], ee = 0.0f;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const float u0 = (float)(0.5 * (1.0 - cospi(2.0 * cc * ((double)(xl + c) / (double)(Q.nx - 1)))));
            d[c] = uu[c] - u0;
            ee += d[c] * d[c];
        }
        e0 = (double)ee;
        if (WANT_G) {
            float4* gp = reinterpret_cast<float4*>(gb + xl);
            float4 gv = *gp;
            gv.x += bxs * d[0]; gv.y += bxs * d[1]; gv.z += bxs * d[2]; gv.w += bxs * d[3];
            *gp = gv;
        }
    }
    double e = C.e, et = C.ebt;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        e += __shfl_xor_sync(0xffffffffu, e, o);
        e0 += __shfl_xor_sync(0xffffffffu, e0, o);
        et += __shfl_xor_sync(0xffffffffu, et, o);
    }
    if (lane == 0) {
        double* slot = Q.partials + ((size_t)bi * Q.nslot + (size_t)chunk * Q.wx + w) * 3;
        slot[0] = e; slot[1] = e0; slot[2] = et;
    }
}

// ---- any-size kernel: one thread per node, the residuals of the 3x3 neighbourhood recomputed ----------
__device__ __forceinline__ float residual_at(const float* ub, int nx, int j, int i, float ct, float cx, float& ux) {
    const float* r0 = ub + (size_t)(j - 1) * nx + i;
    const float* r1 = r0 + nx;
    const float* r2 = r1 + nx;
    ux = cx * ((r0[1] - r0[-1]) + (r2[1] - r2[-1]) + 2.0f * (r1[1] - r1[-1]));
    const float ut = ct * ((r2[-1] - r0[-1]) + (r2[1] - r0[1]) + 2.0f * (r2[0] - r0[0]));
    return ut + r1[0] * ux;
}

__global__ void __launch_bounds__(256) burgers_generic_kernel(BParams Q) {
    const int bi = blockIdx.y;
    const long long nodes = (long long)Q.nx * Q.nt;
    const long long id = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const float* ub = Q.u + (size_t)bi * nodes;
    const float gl = Q.gL ? Q.gL[bi] : 1.0f;
    double e = 0.0, e0 = 0.0, et = 0.0;
    if (id < nodes) {
        const int j = (int)(id / Q.nx), i = (int)(id % Q.nx);
        float g = 0.0f;
        for (int dj = -1; dj <= 1; ++dj)
            for (int di = -1; di <= 1; ++di) {
                const int jj = j - dj, ii = i - di;             // residual node whose stencil reaches (j,i) at offset (dj,di)
                if (jj < 1 || jj > Q.nt - 2 || ii < 1 || ii > Q.nx - 2) continue;
                float ux;
                const float res = residual_at(ub, Q.nx, jj, ii, Q.ct, Q.cx, ux);
                const float a = Q.w2 * res;
                const float wt = (float)(dj * (2 - di * di));  // Sobel t stencil: dj * (1,2,1)[di]
                const float wx = (float)(di * (2 - dj * dj));
                g += a * (wt * Q.ct + ub[(size_t)jj * Q.nx + ii] * wx * Q.cx);
                if (dj == 0 && di == 0) { g += a * ux; e = (double)(res * res); }
            }
        const float uv = ub[id];
        if (j == 0) {
            const double x = (double)i / (double)(Q.nx - 1);
            const float d = uv - (float)(0.5 * (1.0 - cospi(2.0 * (double)Q.c[bi] * x)));
            g += Q.bx * d;
            e0 = (double)(d * d);
        }
        if (i == 0) { g += Q.bt * uv; et = (double)(uv * uv); }
        if (Q.g) Q.g[(size_t)bi * nodes + id] = g * gl;
    }
    __shared__ double sh[3][8];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        e += __shfl_down_sync(0xffffffffu, e, o);
        e0 += __shfl_down_sync(0xffffffffu, e0, o);
        et += __shfl_down_sync(0xffffffffu, et, o);
    }
    const int wid = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) { sh[0][wid] = e; sh[1][wid] = e0; sh[2][wid] = et; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double s0 = 0.0, s1 = 0.0, s2 = 0.0;
        for (int k = 0; k < 8; ++k) { s0 += sh[0][k]; s1 += sh[1][k]; s2 += sh[2][k]; }
        double* slot = Q.partials + ((size_t)bi * Q.nslot + blockIdx.x) * 3;
        slot[0] = s0; slot[1] = s1; slot[2] = s2;
    }
}

__global__ void __launch_bounds__(256) burgers_finalize_kernel(const double* __restrict__ partials, int nslot, double hx,
                                                               double ht, double lambda, float* __restrict__ L,
                                                               float* __restrict__ parts) {
    const int b = blockIdx.x;
    const double* p = partials + (size_t)b * nslot * 3;
    double s[3] = {0.0, 0.0, 0.0};
    for (int i = threadIdx.x; i < nslot; i += blockDim.x)
        for (int k = 0; k < 3; ++k) s[k] += p[3 * i + k];
    __shared__ double sh[3][256];
    for (int k = 0; k < 3; ++k) sh[k][threadIdx.x] = s[k];
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o)
            for (int k = 0; k < 3; ++k) sh[k][threadIdx.x] += sh[k][threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const double lp = hx * ht * sh[0][0];
        const double lb = hx * sh[1][0] + ht * sh[2][0];
        if (L) L[b] = (float)(lp + lambda * lb);
        if (parts) { parts[2 * b] = (float)lp; parts[2 * b + 1] = (float)lb; }
    }
}

struct BGeom {
    bool march;
    int R, nchunk, wx, nslot;
    long long tasks;
};

dn_status validate_burgers(const dn_burgers* p) {
    if (!p) return DN_ERR_NULL;
    if (p->nx < 3 || p->nt < 3 || p->nx > DN_MAX_EXTENT || p->nt > DN_MAX_EXTENT) return DN_ERR_SIZE;
    if (p->batch < 1 || p->batch > 65535) return DN_ERR_SIZE;
    if (!(p->T > 0.0f) || !(p->lambda >= 0.0f)) return DN_ERR_MODE;
    if (!p->c) return DN_ERR_NULL;
    if (p->flags & ~DN_FORCE_GENERIC) return DN_ERR_MODE;
    return DN_OK;
}

int generic_slots(const dn_burgers& p) { return (int)(((long long)p.nx * p.nt + 255) / 256); }

// Rows per chunk: the warps of one launch should fill the resident warp slots of the GPU a whole
// number of times, and each chunk walks four extra rows.
BGeom march_geometry(const dn_burgers& p) {
    BGeom g{};
    g.march = true;
    g.wx = (p.nx + BG_COLS - 1) / BG_COLS;
    const long long resident = (long long)BG_SMS * BG_BLOCKS_PER_SM * BG_WARPS;
    double best = 1e300;
    for (int R = 8; R <= 512; ++R) {
        if (R > p.nt && R != 8) break;
        const int nchunk = (p.nt + R - 1) / R;
        const long long tasks = (long long)p.batch * nchunk * g.wx;
        const long long waves = (tasks + resident - 1) / resident;
        const double cost = (double)waves * (R + 4 + BG_RING);  // ring fill counted as rows of latency
        if (cost < best) { best = cost; g.R = R; g.nchunk = nchunk; g.tasks = tasks; }
    }
    g.nslot = g.nchunk * g.wx;
    return g;
}

bool march_applicable(const dn_burgers& p, const float* u, const float* g) {
    const bool al = ((reinterpret_cast<uintptr_t>(u) | reinterpret_cast<uintptr_t>(g)) & 15u) == 0;
    return !(p.flags & DN_FORCE_GENERIC) && (p.nx % 4 == 0) && al;
}

int max_slots(const dn_burgers& p) {
    int n = generic_slots(p);
    if (p.nx % 4 == 0) { const int m = march_geometry(p).nslot; if (m > n) n = m; }
    return n;
}

}  // namespace
}  // namespace dn

using namespace dn;

extern "C" {

size_t dn_burgers_workspace_bytes(const dn_burgers* p) {
    if (validate_burgers(p) != DN_OK) return 0;
    return align_up(sizeof(double) * 3 * (size_t)p->batch * max_slots(*p));
}

const char* dn_burgers_path_name(const dn_burgers* p, const float* u, const float* g) {
    if (validate_burgers(p) != DN_OK) return "invalid";
    return march_applicable(*p, u, g) ? "march" : "generic";
}

dn_status dn_burgers_loss_grad(const dn_burgers* p, const float* u, const float* gL, float* L, float* parts, float* g,
                               void* ws, size_t ws_bytes, void* stream, void* ev_before, void* ev_after) {
    dn_status st = validate_burgers(p);
    if (st != DN_OK) return st;
    if (!u || (!L && !parts && !g)) return DN_ERR_NULL;
    const size_t bytes = sizeof(float) * (size_t)p->batch * p->nx * p->nt;
    if (g) {
        const char* a = reinterpret_cast<const char*>(u);
        const char* b = reinterpret_cast<const char*>(g);
        if (a < b + bytes && b < a + bytes) return DN_ERR_ALIAS;
    }
    if (!ws || (reinterpret_cast<uintptr_t>(ws) % kAlign) != 0 || ws_bytes < dn_burgers_workspace_bytes(p))
        return DN_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const double hx = 1.0 / (p->nx - 1), ht = (double)p->T / (p->nt - 1);
    BParams Q{};
    Q.nx = p->nx; Q.nt = p->nt; Q.batch = p->batch;
    Q.ct = (float)(1.0 / (8.0 * ht)); Q.cx = (float)(1.0 / (8.0 * hx)); Q.w2 = (float)(2.0 * hx * ht);
    Q.bx = (float)(2.0 * hx * (double)p->lambda); Q.bt = (float)(2.0 * ht * (double)p->lambda);
    Q.u = u; Q.c = p->c; Q.gL = gL; Q.g = g;
    Q.partials = static_cast<double*>(ws);
    if (ev_before && cudaEventRecord(static_cast<cudaEvent_t>(ev_before), s) != cudaSuccess) return DN_ERR_CUDA;
    if (march_applicable(*p, u, g)) {
        const BGeom G = march_geometry(*p);
        Q.R = G.R; Q.nchunk = G.nchunk; Q.wx = G.wx; Q.nslot = G.nslot; Q.tasks = G.tasks;
        const unsigned blocks = (unsigned)((G.tasks + BG_WARPS - 1) / BG_WARPS);
        if (g) burgers_march_kernel<true><<<blocks, BG_WARPS * 32, 0, s>>>(Q);
        else burgers_march_kernel<false><<<blocks, BG_WARPS * 32, 0, s>>>(Q);
    } else {
        Q.nslot = generic_slots(*p);
        burgers_generic_kernel<<<dim3((unsigned)Q.nslot, (unsigned)p->batch), 256, 0, s>>>(Q);
    }
    if (cudaGetLastError() != cudaSuccess) return DN_ERR_CUDA;
    if (ev_after && cudaEventRecord(static_cast<cudaEvent_t>(ev_after), s) != cudaSuccess) return DN_ERR_CUDA;
    if (L || parts) {
        burgers_finalize_kernel<<<p->batch, 256, 0, s>>>(Q.partials, Q.nslot, hx, ht, (double)p->lambda, L, parts);
        if (cudaGetLastError() != cudaSuccess) return DN_ERR_CUDA;
    }
    return DN_OK;
}

size_t dn_burgers_host_staging_bytes(const dn_burgers* p) {
    if (validate_burgers(p) != DN_OK) return 0;
    const size_t field = align_up(sizeof(float) * (size_t)p->batch * p->nx * p->nt);
    const size_t small = align_up(sizeof(float) * 2 * (size_t)p->batch);
    return 2 * field + 4 * small + dn_burgers_workspace_bytes(p);
}

dn_status dn_burgers_loss_grad_host(const dn_burgers* p, const float* u_host, const float* gL_host, float* L_host,
                                    float* parts_host, float* g_host, void* staging, size_t staging_bytes, void* stream) {
    dn_status st = validate_burgers(p);
    if (st != DN_OK) return st;
    if (!u_host || !g_host) return DN_ERR_NULL;
    if (!staging || (reinterpret_cast<uintptr_t>(staging) % kAlign) != 0 || staging_bytes < dn_burgers_host_staging_bytes(p))
        return DN_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t nodes = (size_t)p->nx * p->nt;
    const size_t field = align_up(sizeof(float) * (size_t)p->batch * nodes);
    const size_t small = align_up(sizeof(float) * 2 * (size_t)p->batch);
    char* base = static_cast<char*>(staging);
    float* d_u = reinterpret_cast<float*>(base);
    float* d_g = reinterpret_cast<float*>(base + field);
    float* d_c = reinterpret_cast<float*>(base + 2 * field);
    float* d_gL = reinterpret_cast<float*>(base + 2 * field + small);
    float* d_L = reinterpret_cast<float*>(base + 2 * field + 2 * small);
    float* d_parts = reinterpret_cast<float*>(base + 2 * field + 3 * small);
    void* ws = base + 2 * field + 4 * small;
    const size_t ws_bytes = staging_bytes - (2 * field + 4 * small);   // a chunk never needs more than the whole batch

    const int csize = (p->batch + HostPipe::kMaxChunks - 1) / HostPipe::kMaxChunks;
    const int nchunks = (p->batch + csize - 1) / csize;
    HostPipe pipe;
    if (!pipe.create(nchunks)) return DN_ERR_CUDA;
#define DN_TRY(x) do { if ((x) != cudaSuccess) return DN_ERR_CUDA; } while (0)
    DN_TRY(cudaEventRecord(pipe.start, s));
    DN_TRY(cudaStreamWaitEvent(pipe.in, pipe.start, 0));
    DN_TRY(cudaStreamWaitEvent(pipe.out, pipe.start, 0));
    DN_TRY(cudaMemcpyAsync(d_c, p->c, sizeof(float) * p->batch, cudaMemcpyHostToDevice, pipe.in));
    if (gL_host) DN_TRY(cudaMemcpyAsync(d_gL, gL_host, sizeof(float) * p->batch, cudaMemcpyHostToDevice, pipe.in));
    for (int c = 0; c < nchunks; ++c) {
        const int b0 = c * csize;
        const int nb = (b0 + csize <= p->batch) ? csize : p->batch - b0;
        const size_t o = (size_t)b0 * nodes, n = (size_t)nb * nodes;
        DN_TRY(cudaMemcpyAsync(d_u + o, u_host + o, sizeof(float) * n, cudaMemcpyHostToDevice, pipe.in));
        DN_TRY(cudaEventRecord(pipe.copied[c], pipe.in));
        DN_TRY(cudaStreamWaitEvent(s, pipe.copied[c], 0));
        dn_burgers q = *p;
        q.batch = nb;
        q.c = d_c + b0;
        st = dn_burgers_loss_grad(&q, d_u + o, gL_host ? d_gL + b0 : nullptr, L_host ? d_L + b0 : nullptr,
                                  parts_host ? d_parts + 2 * (size_t)b0 : nullptr, d_g + o, ws, ws_bytes, s, nullptr, nullptr);
        if (st != DN_OK) { cudaStreamSynchronize(pipe.in); cudaStreamSynchronize(s); cudaStreamSynchronize(pipe.out); return st; }
        DN_TRY(cudaEventRecord(pipe.computed[c], s));
        DN_TRY(cudaStreamWaitEvent(pipe.out, pipe.computed[c], 0));
        DN_TRY(cudaMemcpyAsync(g_host + o, d_g + o, sizeof(float) * n, cudaMemcpyDeviceToHost, pipe.out));
    }
    DN_TRY(cudaStreamSynchronize(pipe.in));
    DN_TRY(cudaStreamSynchronize(s));
    if (L_host) DN_TRY(cudaMemcpyAsync(L_host, d_L, sizeof(float) * p->batch, cudaMemcpyDeviceToHost, pipe.out));
    if (parts_host) DN_TRY(cudaMemcpyAsync(parts_host, d_parts, sizeof(float) * 2 * p->batch, cudaMemcpyDeviceToHost, pipe.out));
    DN_TRY(cudaStreamSynchronize(pipe.out));
#undef DN_TRY
    return DN_OK;
}

}  // extern "C"
