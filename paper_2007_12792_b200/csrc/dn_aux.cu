// Small kernels around the fused loss kernel: cosine / coefficient tables for the KL
// expansion, the nodal KL field, the Dirichlet face overwrite, the energy finaliser.
#include "dn_internal.cuh"

namespace dn {

namespace {

constexpr double kLog2e = 1.4426950408889634074;

// ---------------------------------------------------------------------------------------
// Tables for the KL expansion evaluated at Gauss points (DN_NU_KL_GAUSS):
//   ckl[b][i][j]([k]) = w * log2(e) / (1 + i^2 + j^2 (+ k^2))      so that nu = 2^(sum ckl cos cos (cos))
//   cg[a][i-1][p]     = cos(i pi x_p),  x_p = (p/2 + (p odd ? GB : GA)) * h_a,  p < 2 (n_a - 1)
//   cn[a][i-1][n]     = cos(i pi n h_a) at the nodes (DN_NU_KL_NODAL)
// The cosines are evaluated in double (cospi) and rounded once.
// ---------------------------------------------------------------------------------------
struct TableArgs {
    int dim, m, batch;
    int n[3];
    int gstride[3];
    const float* kl_w;
    float* ckl;
    float* cg[3];
    int nstride[3];
    float* cn[3];
    float* rowpoly;       // 2D, optional: polynomial of the KL exponent along every Gauss row, [B][ny-1][rp_gs]
    int rp_gs;
    int rp_nodes;         // 0: the two Gauss rows of every element row, interleaved; 1: every node row, each coefficient twice
};

// exponent(x, y_q) = sum_k poly[k] c^k with c = cos(pi x), for the Gauss row q of element row j of sample b:
// g_i = sum_j ckl[i][j] cos(j pi y_q) are the coefficients in the Chebyshev basis (cos(i pi x) = T_i(c)), converted
// to monomials in double.  The scaled weights and the cosines are rounded to float first, exactly as the tables
// hold them, so every kernel family sees the same numbers.  Entry 2k + q of the row; the two Gauss rows of an
// element row interleave so that they can be evaluated together with two-wide FMAs.  MX >= m is the compiled loop
// bound (the kernel is instantiated for every m; compile-time bounds keep the small arrays in registers).
template <int MX>
__device__ void rowpoly_entry(const TableArgs& A, long long idx) {
    const int m = A.m, ny = A.n[1];
    const int q = (int)(idx & 1);
    const int rows = A.rp_nodes ? ny : ny - 1;
    const long long row = idx >> 1;                    // b * rows + j
    const int j = (int)(row % rows);
    const long long b = row / rows;
    const double ga = 0.5 * (1.0 - 0.57735026918962576451);
    const double gb = 0.5 * (1.0 + 0.57735026918962576451);
    const double y = ((double)j + (q ? gb : ga)) / (double)(ny - 1);
    // cos(jj pi y) from cos(pi y) by the Chebyshev recurrence in double, rounded to float as the cosine tables are
    double cy[MX], g[MX];
    {
        const double c1 = cospi(A.rp_nodes ? (double)j / (double)(ny - 1) : y);
        double tm = 1.0, tc = c1;
#pragma unroll
        for (int jj = 0; jj < MX; ++jj) {
            cy[jj] = (jj < m) ? (double)(float)tc : 0.0;
            const double tn = 2.0 * c1 * tc - tm;
            tm = tc; tc = tn;
        }
    }
    const float* w = A.kl_w + b * m * m;
#pragma unroll
    for (int i = 0; i < MX; ++i) {
        double a = 0.0;
#pragma unroll
        for (int jj = 0; jj < MX; ++jj) {
            if (i < m && jj < m) {
                const double den = 1.0 + (double)((i + 1) * (i + 1)) + (double)((jj + 1) * (jj + 1));
                a += (double)(float)((double)w[i * m + jj] * (kLog2e / den)) * cy[jj];     // the constant folds: no division
            }
        }
        g[i] = a;
    }
    // sum_i g_i T_i(c) in the monomial basis, T_{i+1} = 2 c T_i - T_{i-1}
    double acc[MX + 1], tp[MX + 1], tc[MX + 1];
#pragma unroll
    for (int k = 0; k <= MX; ++k) { acc[k] = 0.0; tp[k] = (k == 0) ? 1.0 : 0.0; tc[k] = (k == 1) ? 1.0 : 0.0; }
#pragma unroll
    for (int i = 1; i <= MX; ++i) {
        if (i > m) break;                              // uniform; the rest of the terms are zero
#pragma unroll
        for (int k = 0; k <= MX; ++k) acc[k] += g[i - 1] * tc[k];
        double tn[MX + 1];
#pragma unroll
        for (int k = 0; k <= MX; ++k) tn[k] = ((k > 0) ? 2.0 * tc[k - 1] : 0.0) - tp[k];
#pragma unroll
        for (int k = 0; k <= MX; ++k) { tp[k] = tc[k]; tc[k] = tn[k]; }
    }
    float* dst = A.rowpoly + row * A.rp_gs + q;
#pragma unroll
    for (int k = 0; k <= MX; ++k) dst[2 * k] = (float)acc[k];
    for (int k = MX + 1; 2 * k + q < A.rp_gs; ++k) dst[2 * k] = 0.f;      // the padding of the row
}

template <int MX>
__global__ void tables_kernel(TableArgs A) {
    dep_wait();                                        // whatever ran before in the stream may still read these tables
    dep_release();
    long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int m = A.m;
    long long mpow = 1;
    for (int a = 0; a < A.dim; ++a) mpow *= m;
    const long long ncoef = mpow * A.batch;
    if (idx < ncoef) {
        long long c = idx % mpow;
        int i, j, k = 0;
        if (A.dim == 3) { k = (int)(c % m) + 1; c /= m; }
        j = (int)(c % m) + 1;
        i = (int)(c / m) + 1;
        const double den = 1.0 + (double)i * i + (double)j * j + (double)k * k;
        A.ckl[idx] = (float)((double)A.kl_w[idx] * (kLog2e / den));      // the same product the row polynomials form
        return;
    }
    idx -= ncoef;
    const double ga = 0.5 * (1.0 - 0.57735026918962576451);
    const double gb = 0.5 * (1.0 + 0.57735026918962576451);
    for (int a = 0; a < A.dim; ++a) {
        const long long cnt = (long long)m * A.gstride[a];
        if (idx < cnt) {
            const int i = (int)(idx / A.gstride[a]) + 1;
            int p = (int)(idx % A.gstride[a]);
            const int ng = 2 * (A.n[a] - 1);
            if (p >= ng) p = ng - 1;                      // padding repeats the last abscissa
            const double x = ((double)(p >> 1) + ((p & 1) ? gb : ga)) / (double)(A.n[a] - 1);
            A.cg[a][idx] = (float)cospi((double)i * x);
            return;
        }
        idx -= cnt;
    }
    for (int a = 0; a < A.dim; ++a) {
        const long long cnt = (long long)m * A.nstride[a];
        if (idx < cnt) {
            const int i = (int)(idx / A.nstride[a]) + 1;
            int n = (int)(idx % A.nstride[a]);
            if (n >= A.n[a]) n = A.n[a] - 1;              // padding repeats the last node
            A.cn[a][idx] = (float)cospi((double)i * (double)n / (double)(A.n[a] - 1));
            return;
        }
        idx -= cnt;
    }
    if (A.rowpoly && idx < 2ll * A.batch * (A.n[1] - (A.rp_nodes ? 0 : 1))) rowpoly_entry<MX>(A, idx);
}

// ---------------------------------------------------------------------------------------
// Energy finaliser: J[b] = sum over block partials (diffusion part) - (load part), summed
// in a fixed order in double, rounded once to float.
// ---------------------------------------------------------------------------------------
__global__ void finalize_kernel(const double* __restrict__ partials, int nblk, float* __restrict__ J) {
    dep_wait();
    const int b = blockIdx.x;
    const double* p = partials + 2ll * b * nblk;
    double d = 0.0, l = 0.0;
    for (int i = threadIdx.x; i < nblk; i += blockDim.x) { d += p[2 * i]; l += p[2 * i + 1]; }
    __shared__ double sd[256], sl[256];
    sd[threadIdx.x] = d; sl[threadIdx.x] = l;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) { sd[threadIdx.x] += sd[threadIdx.x + o]; sl[threadIdx.x] += sl[threadIdx.x + o]; }
        __syncthreads();
    }
    if (threadIdx.x == 0) J[b] = (float)(sd[0] - sl[0]);
}

// ---------------------------------------------------------------------------------------
// Nodal KL field.  cos(i pi ix/(n-1)) is taken from cospif after an exact integer
// reduction of the angle to [0, pi/2], so the only rounding is that of k/(n-1).
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float cos_node(int i, int ix, int nm1) {
    int k = (int)(((long long)i * ix) % (2ll * nm1));     // angle = pi * k / nm1, k in [0, 2 nm1)
    if (k > nm1) k = 2 * nm1 - k;                        // cos(2 pi - t) = cos t
    float sgn = 1.0f;
    if (2 * k > nm1) { k = nm1 - k; sgn = -1.0f; }       // cos(pi - t) = -cos t
    return sgn * cospif((float)k / (float)nm1);
}

constexpr int KLF_THREADS = 128;
constexpr int KLF_LINES = 64;                           // grid lines (fixed y, z) per block

typedef unsigned long long klf_u64;
__device__ __forceinline__ klf_u64 klf_pack2(float lo, float hi) {
    klf_u64 v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
    return v;
}
__device__ __forceinline__ void klf_unpack2(klf_u64 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ klf_u64 klf_fma2(klf_u64 a, klf_u64 b, klf_u64 c) {
    klf_u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ float klf_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// A block owns up to KLF_LINES consecutive grid lines (y, z flattened) and a strip of 4 * KLF_THREADS
// nodes in x.  Along a line the exponent is a polynomial of degree m in c = cos(pi x) (cos(i pi x) =
// T_i(c)); its coefficients are prepared per line in double and stored, duplicated, in shared memory,
// so a pair of nodes costs m packed FMAs, two ex2 and half a 128-bit store: the kernel is write-bound.
template <int M, int VEC>
__global__ void __launch_bounds__(KLF_THREADS)
kl_field_kernel(int dim, int nx, int ny, int nz, const float* __restrict__ kl_w, float* __restrict__ nu) {
    constexpr int GS = (2 * (M + 1) + 3) / 4 * 4;       // floats per line: (g_k, g_k) pairs, padded
    __shared__ __align__(16) float gam[KLF_LINES][GS];
    const int b = blockIdx.z;
    const long long nlines = (long long)ny * nz;
    const long long l0 = (long long)blockIdx.x * KLF_LINES;
    const int tid = threadIdx.x;
    const float* w = kl_w + (long long)b * M * M * (dim == 3 ? M : 1);
    if (tid < KLF_LINES && l0 + tid < nlines) {
        const long long l = l0 + tid;
        const int iy = (int)(l % ny), iz = (int)(l / ny);
        double cy[M], cz[M], g[M];
#pragma unroll
        for (int j = 0; j < M; ++j) {
            cy[j] = (double)cos_node(j + 1, iy, ny - 1);
            cz[j] = (dim == 3) ? (double)cos_node(j + 1, iz, nz - 1) : 1.0;
        }
#pragma unroll
        for (int i = 0; i < M; ++i) {
            double acc = 0.0;
#pragma unroll
            for (int j = 0; j < M; ++j) {
                double inner;
                if (dim == 3) {
                    inner = 0.0;
#pragma unroll
                    for (int k = 0; k < M; ++k)
                        inner += (double)w[(i * M + j) * M + k] / (1.0 + (i + 1) * (i + 1) + (j + 1) * (j + 1) + (k + 1) * (k + 1)) * cz[k];
                } else {
                    inner = (double)w[i * M + j] / (1.0 + (i + 1) * (i + 1) + (j + 1) * (j + 1));
                }
                acc += inner * cy[j];
            }
            g[i] = acc * kLog2e;
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
        for (int k = 0; k <= M; ++k) { gam[tid][2 * k] = (float)acc[k]; gam[tid][2 * k + 1] = (float)acc[k]; }
    }
    __syncthreads();
    const int x0 = (blockIdx.y * KLF_THREADS + tid) * VEC;
    if (x0 >= nx) return;
    float c[4];
#pragma unroll
    for (int v = 0; v < 4; ++v) c[v] = cos_node(1, min(x0 + v, nx - 1), nx - 1);
    const klf_u64 c01 = klf_pack2(c[0], c[1]), c23 = klf_pack2(c[2], c[3]);
    float* out = nu + (long long)b * nlines * nx + l0 * nx + x0;
    const int lines = (int)min((long long)KLF_LINES, nlines - l0);
    for (int row = 0; row < lines; ++row) {
        klf_u64 g2[GS / 2];
        const ulonglong2* gp = reinterpret_cast<const ulonglong2*>(&gam[row][0]);
#pragma unroll
        for (int k = 0; k < GS / 4; ++k) { const ulonglong2 t = gp[k]; g2[2 * k] = t.x; g2[2 * k + 1] = t.y; }
        klf_u64 e01 = g2[M], e23 = g2[M];
#pragma unroll
        for (int k = M - 1; k >= 0; --k) { e01 = klf_fma2(e01, c01, g2[k]); if (VEC == 4) e23 = klf_fma2(e23, c23, g2[k]); }
        float e0, e1, e2, e3;
        klf_unpack2(e01, e0, e1);
        klf_unpack2(e23, e2, e3);
        if (VEC == 4) {
            *reinterpret_cast<float4*>(out) = make_float4(klf_ex2(e0), klf_ex2(e1), klf_ex2(e2), klf_ex2(e3));
        } else {
            out[0] = klf_ex2(e0);
        }
        out += nx;
    }
}

template <int VEC>
cudaError_t launch_kl_field_vec(const dn_grid& g, int nz, int batch, int m, const float* kl_w, float* nu, cudaStream_t s) {
    const int per_block = KLF_THREADS * VEC;
    const long long nlines = (long long)g.ny * nz;
    dim3 grid((unsigned)((nlines + KLF_LINES - 1) / KLF_LINES), (g.nx + per_block - 1) / per_block, batch);
    switch (m) {
        case 1: kl_field_kernel<1, VEC><<<grid, KLF_THREADS, 0, s>>>(g.dim, g.nx, g.ny, nz, kl_w, nu); break;
        case 2: kl_field_kernel<2, VEC><<<grid, KLF_THREADS, 0, s>>>(g.dim, g.nx, g.ny, nz, kl_w, nu); break;
        case 3: kl_field_kernel<3, VEC><<<grid, KLF_THREADS, 0, s>>>(g.dim, g.nx, g.ny, nz, kl_w, nu); break;
        case 4: kl_field_kernel<4, VEC><<<grid, KLF_THREADS, 0, s>>>(g.dim, g.nx, g.ny, nz, kl_w, nu); break;
        case 5: kl_field_kernel<5, VEC><<<grid, KLF_THREADS, 0, s>>>(g.dim, g.nx, g.ny, nz, kl_w, nu); break;
        case 6: kl_field_kernel<6, VEC><<<grid, KLF_THREADS, 0, s>>>(g.dim, g.nx, g.ny, nz, kl_w, nu); break;
        case 7: kl_field_kernel<7, VEC><<<grid, KLF_THREADS, 0, s>>>(g.dim, g.nx, g.ny, nz, kl_w, nu); break;
        case 8: kl_field_kernel<8, VEC><<<grid, KLF_THREADS, 0, s>>>(g.dim, g.nx, g.ny, nz, kl_w, nu); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

__global__ void apply_bc_kernel(long long lines, long long lines_per_sample, int nx, float v0, float v1,
                                const float* __restrict__ v0_b, const float* __restrict__ v1_b,
                                float* __restrict__ field) {
    const long long line = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (line >= lines) return;
    if (v0_b) v0 = v0_b[line / lines_per_sample];
    if (v1_b) v1 = v1_b[line / lines_per_sample];
    field[line * nx] = v0;
    field[line * nx + nx - 1] = v1;
}

}  // namespace

cudaError_t launch_tables(const Params& P, const float* kl_w, float* ckl, float* const cg[3], float* const cn[3],
                          cudaStream_t s, float* rowpoly, int rowpoly_stride, bool rowpoly_nodes) {
    TableArgs A{};
    A.dim = P.dim; A.m = P.m; A.batch = P.batch;
    A.n[0] = P.nx; A.n[1] = P.ny; A.n[2] = P.nz;
    long long total = (long long)P.batch;
    for (int a = 0; a < P.dim; ++a) total *= P.m;
    for (int a = 0; a < 3; ++a) {
        A.gstride[a] = P.gstride[a]; A.cg[a] = cg[a];
        A.nstride[a] = P.nstride[a]; A.cn[a] = cn[a];
        if (a < P.dim) total += (long long)P.m * (P.gstride[a] + P.nstride[a]);
    }
    A.kl_w = kl_w; A.ckl = ckl;
    A.rowpoly = (P.dim == 2) ? rowpoly : nullptr; A.rp_gs = rowpoly_stride; A.rp_nodes = rowpoly_nodes ? 1 : 0;
    if (A.rowpoly) total += 2ll * P.batch * (P.ny - (rowpoly_nodes ? 0 : 1));
    const int threads = 128;
    const dim3 grid((unsigned)((total + threads - 1) / threads));
    switch (A.rowpoly ? P.m : DN_MAX_KL_MODES) {       // the loop bound matters to the row polynomials only
        case 1: return launch_dependent(tables_kernel<1>, grid, dim3(threads), 0, s, A);
        case 2: return launch_dependent(tables_kernel<2>, grid, dim3(threads), 0, s, A);
        case 3: return launch_dependent(tables_kernel<3>, grid, dim3(threads), 0, s, A);
        case 4: return launch_dependent(tables_kernel<4>, grid, dim3(threads), 0, s, A);
        case 5: return launch_dependent(tables_kernel<5>, grid, dim3(threads), 0, s, A);
        case 6: return launch_dependent(tables_kernel<6>, grid, dim3(threads), 0, s, A);
        case 7: return launch_dependent(tables_kernel<7>, grid, dim3(threads), 0, s, A);
    }
    return launch_dependent(tables_kernel<DN_MAX_KL_MODES>, grid, dim3(threads), 0, s, A);
}

cudaError_t launch_finalize(const double* partials, int nblk, int batch, float* J, cudaStream_t s) {
    return launch_dependent(finalize_kernel, dim3((unsigned)batch), dim3(256), 0, s, partials, nblk, J);
}

cudaError_t launch_kl_field(const dn_grid& g, int batch, int m, const float* kl_w, float* nu, cudaStream_t s) {
    const int nz = (g.dim == 3) ? g.nz : 1;
    const bool vec = (g.nx % 4 == 0) && ((reinterpret_cast<uintptr_t>(nu) & 15u) == 0);
    return vec ? launch_kl_field_vec<4>(g, nz, batch, m, kl_w, nu, s) : launch_kl_field_vec<1>(g, nz, batch, m, kl_w, nu, s);
}

cudaError_t launch_apply_bc(const dn_grid& g, int batch, float b0, float b1, int mode, float* field, cudaStream_t s,
                            const float* b0_b, const float* b1_b) {
    const long long per_sample = (long long)g.ny * ((g.dim == 3) ? g.nz : 1);
    const long long lines = (long long)batch * per_sample;
    const int threads = 256;
    apply_bc_kernel<<<(unsigned)((lines + threads - 1) / threads), threads, 0, s>>>(
        lines, per_sample, g.nx, mode == 0 ? b0 : 0.0f, mode == 0 ? b1 : 0.0f, mode == 0 ? b0_b : nullptr,
        mode == 0 ? b1_b : nullptr, field);
    return cudaGetLastError();
}

}  // namespace dn
