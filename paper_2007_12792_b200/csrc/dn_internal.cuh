// Internal declarations shared by the CUDA translation units of libdn.
#pragma once

#include <cstring>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "dn.h"

namespace dn {

// Gauss abscissae of the 2-point rule mapped to [0,1]: (1 -/+ 1/sqrt(3)) / 2.
#define DN_GA 0.21132486540518711775f
#define DN_GB 0.78867513459481288225f

constexpr int kAlign = 256;

inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }

// A launch geometry is a pure function of the problem's shape and mode and of the SM count of the current device.  Each
// kernel family remembers the last one it searched for, per host thread, so that a training loop pays the search once.
struct GeoKey { int v[10]; };
inline GeoKey geo_key(const dn_problem& p, int sms) {
    return GeoKey{{p.grid.dim, p.grid.nx, p.grid.ny, (p.grid.dim == 3) ? p.grid.nz : 1, p.batch, (int)p.nu_mode,
                   (p.nu_mode == DN_NU_NODAL) ? 0 : p.kl_modes,     // not read with a stored field
                   p.f != nullptr ? 1 : 0, sms, 1}};
}
template <class G, class F>
G memo_geometry(const dn_problem& p, int sms, F search) {
    thread_local GeoKey last{};                        // all zero: equal to no real key (the last entry of one is 1)
    thread_local G geo{};
    const GeoKey k = geo_key(p, sms);
    if (memcmp(k.v, last.v, sizeof k.v) != 0) { geo = search(); last = k; }
    return geo;
}

enum Path { PATH_GENERIC = 0, PATH_TILED2D = 1, PATH_TILED3D = 2, PATH_STRIP2D = 3, PATH_STRIP3D = 4, PATH_ROW2D = 5 };

// Where things live inside the caller's workspace (byte offsets, all 256-B aligned).
struct WsLayout {
    size_t partials;      // double [B][nblk][2]  (diffusion part, load part)
    size_t ckl;           // float  [B][m^dim]    KL weights * log2(e) / (1 + i^2 + j^2 (+ k^2))
    size_t cg[3];         // float  [m][gstride[a]] cos(i pi x) at the Gauss abscissae of axis a
    size_t seam;          // float  [B][nseam][nz][nx] contributions across tile seams (tiled 3D kernel)
    int gstride[3];       // padded row length of cg[a] (multiple of 4)
    size_t cn[3];         // float  [m][nstride[a]] cos(i pi x) at the nodes of axis a
    int nstride[3];
    size_t rowpoly;       // float  [B][ny-1][GS] polynomial of the KL exponent along every Gauss row (strip 2D and row 2D kernels)
    size_t zseam;         // float  contributions across the chunk seams of the strip 3D kernel
    size_t linepoly;      // float  [B][nz-1][ny-1][2 GS] the same along the four Gauss lines of every element row (strip 3D kernel)
    int nblk;             // energy partials per sample
    size_t total;
};

// Everything a kernel needs, passed by value.
struct Params {
    int dim, nx, ny, nz, batch;
    int nu_mode, m;
    unsigned flags;
    float f_const, bc_x0, bc_x1;
    float hx, hy, hz;
    const float* u;
    const float* nu;
    const float* f;
    const float* gJ;
    const float* bc0_b;   // per-sample boundary values or NULL (then bc_x0 / bc_x1 hold for every sample)
    const float* bc1_b;
    float* r;             // may be NULL (energy only)
    double* partials;
    const float* ckl;
    const float* cg[3];
    int gstride[3];
    const float* cn[3];   // cosines at the nodes (KL-at-nodes mode)
    int nstride[3];
    int nblk;
    long long nodes;      // per sample
    float* seam;          // tiled 3D: contributions of a tile's top element row to the next tile's first node row
    int nseam;
    float* zseam;         // strip 3D: contributions of a chunk's last element plane to the next chunk's first node plane
};

struct Launch {           // tiled-path launch geometry chosen on the host
    int path;
    int nblk;             // blocks (energy partials) per sample
    int chunk;            // rows (2D) or planes (3D) of elements per block
    int variant;          // kernel template variant
};

Launch choose_launch(const dn_problem& p, const float* u, const float* r);
WsLayout make_layout(const dn_problem& p, const Launch& l, bool tight = false);
// dn_energy_grad with the workspace sized for the chosen kernel family only (tight = true).
// What run_tight would answer for a scratch area of ws_bytes, without enqueuing anything or touching the device.
dn_status check_tight(const dn_problem* p, const float* u, const float* r, size_t ws_bytes);
dn_status run_tight(const dn_problem* p, const float* u, const float* gJ, float* J, float* r, void* ws,
                    size_t ws_bytes, void* stream);
// The fused kernel alone, for callers that apply the operator repeatedly: no energy finaliser; the KL tables are
// built only when build_tables is set (they depend on the problem, not on u); *partials / *nblk tell where the
// kernel left its per-block energy pairs (diffusion part, load part), [batch][*nblk][2] doubles.
dn_status run_operator(const dn_problem* p, const float* u, float* r, void* ws, size_t ws_bytes, cudaStream_t s,
                       bool build_tables, const double** partials, int* nblk);

// The KL tables alone, laid out as the kernel family chosen for (p, u, r) reads them.  For callers of run_operator
// that apply the operator to several problems sharing one diffusivity: build for the problem whose family needs
// the most (the cosine tables and scaled weights are common to all families).
dn_status build_tables(const dn_problem* p, const float* u, float* r, void* ws, size_t ws_bytes, cudaStream_t s);

// rowpoly (optional, 2D): also writes the per-Gauss-row polynomials the strip kernel reads, rows of rowpoly_stride floats
cudaError_t launch_tables(const Params& P, const float* kl_w, float* ckl, float* const cg[3], float* const cn[3],
                          cudaStream_t s, float* rowpoly = nullptr, int rowpoly_stride = 0,
                          bool rowpoly_nodes = false);   // rowpoly_nodes: one polynomial per node row (KL at the nodes)
cudaError_t launch_generic(const Params& P, cudaStream_t s);
cudaError_t launch_tiled2d(const Params& P, const Launch& l, cudaStream_t s);
cudaError_t launch_tiled3d(const Params& P, const Launch& l, cudaStream_t s);
cudaError_t launch_strip2d(const Params& P, const float* rowpoly, cudaStream_t s);
cudaError_t launch_row2d(const Params& P, const float* rowpoly, cudaStream_t s);   // same table as the strip 2D kernel
cudaError_t launch_finalize(const double* partials, int nblk, int batch, float* J, cudaStream_t s);
cudaError_t launch_kl_field(const dn_grid& g, int batch, int m, const float* kl_w, float* nu, cudaStream_t s);
cudaError_t launch_apply_bc(const dn_grid& g, int batch, float b0, float b1, int mode, float* field, cudaStream_t s,
                            const float* b0_b = nullptr, const float* b1_b = nullptr);

int generic_blocks_per_sample(long long nodes);
bool tiled2d_applicable(const dn_problem& p);
bool tiled3d_applicable(const dn_problem& p);
bool strip2d_applicable(const dn_problem& p);     // fused energy+residual, KL at the Gauss points, wide 2D grids
Launch strip2d_geometry(const dn_problem& p);
size_t strip2d_rowpoly_floats(const dn_problem& p);
int strip2d_rowpoly_stride(int kl_modes);          // floats per element row of that table
bool row2d_applicable(const dn_problem& p);       // fused energy+residual, 2D grids whose rows fit one warp (nx <= 256)
Launch row2d_geometry(const dn_problem& p);
size_t row2d_rowpoly_floats(const dn_problem& p);
Launch tiled2d_geometry(const dn_problem& p);
Launch tiled3d_geometry(const dn_problem& p);
size_t tiled3d_seam_floats(const dn_problem& p);   // scratch floats the tiled 3D kernel needs for its tile seams
// adds seam[b][s][plane][x] to node row (s + 1) * rows_per_tile of r, for every sample, seam and plane
cudaError_t launch_seam_fixup(float* r, const float* seam, int nx, int ny, int nz, int rows_per_tile, int nseam, int batch,
                              cudaStream_t s);
bool strip3d_applicable(const dn_problem& p);      // fused energy+residual, KL at the Gauss points, 3D rows of at most 256 nodes
Launch strip3d_geometry(const dn_problem& p);
size_t strip3d_seam_floats(const dn_problem& p);
size_t strip3d_zseam_floats(const dn_problem& p);
size_t strip3d_linepoly_floats(const dn_problem& p);
cudaError_t launch_linepoly3d(const Params& P, float* linepoly, cudaStream_t s);   // after launch_tables (reads ckl, cg)
cudaError_t launch_strip3d(const Params& P, const float* linepoly, cudaStream_t s);

// Streams and events of one *_host call (created and destroyed inside the call).
struct HostPipe {
    static constexpr int kMaxChunks = 32;
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, copied[kMaxChunks] = {}, computed[kMaxChunks] = {};
    bool create(int nchunks) {
        if (cudaStreamCreateWithFlags(&in, cudaStreamNonBlocking) != cudaSuccess) return false;
        if (cudaStreamCreateWithFlags(&out, cudaStreamNonBlocking) != cudaSuccess) return false;
        if (cudaEventCreateWithFlags(&start, cudaEventDisableTiming) != cudaSuccess) return false;
        for (int c = 0; c < nchunks; ++c) {
            if (cudaEventCreateWithFlags(&copied[c], cudaEventDisableTiming) != cudaSuccess) return false;
            if (cudaEventCreateWithFlags(&computed[c], cudaEventDisableTiming) != cudaSuccess) return false;
        }
        return true;
    }
    ~HostPipe() {
        for (int c = 0; c < kMaxChunks; ++c) {
            if (copied[c]) cudaEventDestroy(copied[c]);
            if (computed[c]) cudaEventDestroy(computed[c]);
        }
        if (start) cudaEventDestroy(start);
        if (in) cudaStreamDestroy(in);
        if (out) cudaStreamDestroy(out);
    }
};

// Launch of a kernel that may start before the kernel ahead of it in the stream has finished (programmatic
// dependent launch): its blocks become resident as the blocks of that kernel retire, and it must not touch anything
// that kernel writes, nor write anything it reads, before dep_wait() has returned.  Hides the launch latency and the
// tail of the kernel ahead.
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

#ifdef __CUDACC__
// dep_wait(): everything the kernels ahead in the stream wrote is complete and visible (a no-op in a kernel that was
// launched the ordinary way).  dep_release(): kernels launched behind this one with launch_dependent may become
// resident from now on (they still wait in dep_wait() for this kernel to finish).
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dep_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Sum (d, l) over the block in a fixed order and let thread 0 store the pair.
// Every thread of the block must call this.  blockDim.x * blockDim.y <= 1024.
__device__ __forceinline__ void block_reduce_store(double d, double l, double* slot) {
    __shared__ double sd[32], sl[32];
    const int tid = threadIdx.y * blockDim.x + threadIdx.x;
    const int nthreads = blockDim.x * blockDim.y;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        d += __shfl_down_sync(0xffffffffu, d, o);
        l += __shfl_down_sync(0xffffffffu, l, o);
    }
    if ((tid & 31) == 0) { sd[tid >> 5] = d; sl[tid >> 5] = l; }
    __syncthreads();
    if (tid == 0) {
        const int nw = (nthreads + 31) >> 5;
        double a = 0.0, b = 0.0;
        for (int w = 0; w < nw; ++w) { a += sd[w]; b += sl[w]; }
        slot[0] = a; slot[1] = b;
    }
}
#endif

}  // namespace dn
