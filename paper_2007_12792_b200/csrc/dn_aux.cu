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
// The cosines are evaluated in double (cospi) and rounded once.
// ---------------------------------------------------------------------------------------
struct TableArgs {
    int dim, m, batch;
    int n[3];
    int gstride[3];
    const float* kl_w;
    float* ckl;
    float* cg[3];
};

__global__ void tables_kernel(TableArgs A) {
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
        A.ckl[idx] = (float)((double)A.kl_w[idx] * kLog2e / den);
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
}

// ---------------------------------------------------------------------------------------
// Energy finaliser: J[b] = sum over block partials (diffusion part) - (load part), summed
// in a fixed order in double, rounded once to float.
// ---------------------------------------------------------------------------------------
__global__ void finalize_kernel(const double* __restrict__ partials, int nblk, float* __restrict__ J) {
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
constexpr int KLF_ROWS = 16;
constexpr int KLF_M = DN_MAX_KL_MODES;

template <int VEC>
__global__ void __launch_bounds__(KLF_THREADS)
kl_field_kernel(int dim, int nx, int ny, int nz, int m, const float* __restrict__ kl_w, float* __restrict__ nu) {
    __shared__ float cy[KLF_ROWS][KLF_M];
    __shared__ float cz[KLF_M];
    __shared__ float g[KLF_ROWS][KLF_M];
    const int b = blockIdx.z;
    const int rows_y = (ny + KLF_ROWS - 1) / KLF_ROWS;
    const int iz = blockIdx.x / rows_y;
    const int y0 = (blockIdx.x % rows_y) * KLF_ROWS;
    const int tid = threadIdx.x;
    long long mpow = (long long)m * m * (dim == 3 ? m : 1);
    const float* w = kl_w + (long long)b * mpow;
    if (tid < KLF_ROWS * m) {
        const int row = tid / m, j = tid % m + 1;
        const int iy = min(y0 + row, ny - 1);
        cy[row][j - 1] = cos_node(j, iy, ny - 1);
    }
    if (tid < m) cz[tid] = (dim == 3) ? cos_node(tid + 1, iz, nz - 1) : 1.0f;
    __syncthreads();
    if (tid < KLF_ROWS * m) {
        const int row = tid / m, i = tid % m + 1;
        float acc = 0.0f;
        for (int j = 1; j <= m; ++j) {
            float inner = 0.0f;
            if (dim == 3) {
                for (int k = 1; k <= m; ++k)
                    inner = fmaf(w[((i - 1) * m + (j - 1)) * m + (k - 1)] *
                                     (float)(kLog2e / (1.0 + i * i + j * j + k * k)), cz[k - 1], inner);
            } else {
                inner = w[(i - 1) * m + (j - 1)] * (float)(kLog2e / (1.0 + i * i + j * j));
            }
            acc = fmaf(inner, cy[row][j - 1], acc);
        }
        g[row][i - 1] = acc;
    }
    __syncthreads();
    const int x0 = (blockIdx.y * KLF_THREADS + tid) * VEC;
    if (x0 >= nx) return;
    float cx[KLF_M][VEC];
    for (int i = 0; i < m; ++i)
#pragma unroll
        for (int v = 0; v < VEC; ++v) cx[i][v] = cos_node(i + 1, min(x0 + v, nx - 1), nx - 1);
    for (int row = 0; row < KLF_ROWS; ++row) {
        const int iy = y0 + row;
        if (iy >= ny) break;
        float e[VEC];
#pragma unroll
        for (int v = 0; v < VEC; ++v) e[v] = 0.0f;
        for (int i = 0; i < m; ++i) {
            const float gi = g[row][i];
#pragma unroll
            for (int v = 0; v < VEC; ++v) e[v] = fmaf(cx[i][v], gi, e[v]);
        }
        float* out = nu + (((long long)b * nz + iz) * ny + iy) * nx + x0;
        if (VEC == 4) {
            float4 o = make_float4(exp2f(e[0]), exp2f(e[1]), exp2f(e[2]), exp2f(e[3]));
            *reinterpret_cast<float4*>(out) = o;
        } else {
            out[0] = exp2f(e[0]);
        }
    }
}

__global__ void apply_bc_kernel(long long lines, int nx, float v0, float v1, float* __restrict__ field) {
    const long long line = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (line >= lines) return;
    field[line * nx] = v0;
    field[line * nx + nx - 1] = v1;
}

}  // namespace

cudaError_t launch_tables(const Params& P, const float* kl_w, float* ckl, float* const cg[3], cudaStream_t s) {
    TableArgs A{};
    A.dim = P.dim; A.m = P.m; A.batch = P.batch;
    A.n[0] = P.nx; A.n[1] = P.ny; A.n[2] = P.nz;
    long long total = (long long)P.batch;
    for (int a = 0; a < P.dim; ++a) total *= P.m;
    for (int a = 0; a < 3; ++a) {
        A.gstride[a] = P.gstride[a]; A.cg[a] = cg[a];
        if (a < P.dim) total += (long long)P.m * P.gstride[a];
    }
    A.kl_w = kl_w; A.ckl = ckl;
    const int threads = 128;
    tables_kernel<<<(unsigned)((total + threads - 1) / threads), threads, 0, s>>>(A);
    return cudaGetLastError();
}

cudaError_t launch_finalize(const double* partials, int nblk, int batch, float* J, cudaStream_t s) {
    finalize_kernel<<<batch, 256, 0, s>>>(partials, nblk, J);
    return cudaGetLastError();
}

cudaError_t launch_kl_field(const dn_grid& g, int batch, int m, const float* kl_w, float* nu, cudaStream_t s) {
    const int nz = (g.dim == 3) ? g.nz : 1;
    const bool vec = (g.nx % 4 == 0) && ((reinterpret_cast<uintptr_t>(nu) & 15u) == 0);
    const int per_block = KLF_THREADS * (vec ? 4 : 1);
    dim3 grid(((g.ny + KLF_ROWS - 1) / KLF_ROWS) * nz, (g.nx + per_block - 1) / per_block, batch);
    if (vec) kl_field_kernel<4><<<grid, KLF_THREADS, 0, s>>>(g.dim, g.nx, g.ny, nz, m, kl_w, nu);
    else kl_field_kernel<1><<<grid, KLF_THREADS, 0, s>>>(g.dim, g.nx, g.ny, nz, m, kl_w, nu);
    return cudaGetLastError();
}

cudaError_t launch_apply_bc(const dn_grid& g, int batch, float b0, float b1, int mode, float* field, cudaStream_t s) {
    const long long lines = (long long)batch * g.ny * ((g.dim == 3) ? g.nz : 1);
    const int threads = 256;
    apply_bc_kernel<<<(unsigned)((lines + threads - 1) / threads), threads, 0, s>>>(
        lines, g.nx, mode == 0 ? b0 : 0.0f, mode == 0 ? b1 : 0.0f, field);
    return cudaGetLastError();
}

}  // namespace dn
