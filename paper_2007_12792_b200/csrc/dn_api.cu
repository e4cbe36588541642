// C-ABI entry points: validation, workspace layout, choice of kernel family, launches.
// Host code only; the arithmetic lives in the kernels of the other translation units.
#include <cstdio>
#include <cstring>

#include "dn_internal.cuh"

namespace dn {

static bool valid_grid(const dn_grid& g, dn_status& st) {
    if (g.dim != 2 && g.dim != 3) { st = DN_ERR_DIM; return false; }
    const int nz = (g.dim == 3) ? g.nz : 2;
    if (g.nx < 2 || g.ny < 2 || nz < 2 || g.nx > DN_MAX_EXTENT || g.ny > DN_MAX_EXTENT || nz > DN_MAX_EXTENT) {
        st = DN_ERR_SIZE; return false;
    }
    return true;
}

static dn_status validate(const dn_problem* p) {
    if (!p) return DN_ERR_NULL;
    dn_status st = DN_OK;
    if (!valid_grid(p->grid, st)) return st;
    if (p->batch < 1 || p->batch > 65535) return DN_ERR_SIZE;
    if (p->nu_mode == DN_NU_NODAL) {
        if (!p->nu) return DN_ERR_NULL;
    } else if (p->nu_mode == DN_NU_KL_GAUSS || p->nu_mode == DN_NU_KL_NODAL) {
        if (p->kl_modes < 1 || p->kl_modes > DN_MAX_KL_MODES) return DN_ERR_MODE;
        if (!p->kl_w) return DN_ERR_NULL;
    } else {
        return DN_ERR_MODE;
    }
    return DN_OK;
}

static long long nodes_per_sample(const dn_grid& g) {
    return (long long)g.nx * g.ny * ((g.dim == 3) ? g.nz : 1);
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

Launch choose_launch(const dn_problem& p, const float* u, const float* r) {
    const bool vec_ok = aligned16(u) && aligned16(r) && (p.nu_mode != DN_NU_NODAL || aligned16(p.nu)) && aligned16(p.f);
    if (!(p.flags & DN_FORCE_GENERIC) && vec_ok) {
        if (r && row2d_applicable(p)) return row2d_geometry(p);          // narrow 2D rows, constant forcing
        // the strip kernels also take nodal forcing; without r they run their energy-only variant, which in 2D is
        // the choice where the tiled kernel cannot run (it is the faster of the two there: 153 against 171 us on 2048^2 x 16)
        if (strip2d_applicable(p) && (r || p.f != nullptr || !tiled2d_applicable(p))) return strip2d_geometry(p);
        if (strip3d_applicable(p)) return strip3d_geometry(p);           // ... and, without r, run their energy-only variant
        if (p.f == nullptr) {
            if (tiled2d_applicable(p)) return tiled2d_geometry(p);
            if (tiled3d_applicable(p)) return tiled3d_geometry(p);
        }
    }
    Launch l{};
    l.path = PATH_GENERIC;
    l.nblk = generic_blocks_per_sample(nodes_per_sample(p.grid));
    return l;
}

// The workspace is sized for the largest of the kernel families that could be chosen for
// this problem, so that the size does not depend on pointer alignment.
static int max_nblk(const dn_problem& p) {
    int n = generic_blocks_per_sample(nodes_per_sample(p.grid));
    if (tiled2d_applicable(p)) { int t = tiled2d_geometry(p).nblk; if (t > n) n = t; }
    if (strip2d_applicable(p)) { int t = strip2d_geometry(p).nblk; if (t > n) n = t; }
    if (row2d_applicable(p)) { int t = row2d_geometry(p).nblk; if (t > n) n = t; }
    if (tiled3d_applicable(p)) { int t = tiled3d_geometry(p).nblk; if (t > n) n = t; }
    if (strip3d_applicable(p)) { int t = strip3d_geometry(p).nblk; if (t > n) n = t; }
    return n;
}

WsLayout make_layout(const dn_problem& p, const Launch& l, bool tight) {
    WsLayout w{};
    const int dim = p.grid.dim;
    const int m = (p.nu_mode != DN_NU_NODAL) ? p.kl_modes : 0;
    w.nblk = l.nblk;
    size_t off = 0;
    w.partials = off; off += align_up(sizeof(double) * 2 * (size_t)p.batch * (tight ? l.nblk : max_nblk(p)));
    size_t mpow = 1;
    for (int a = 0; a < dim; ++a) mpow *= (size_t)m;
    w.ckl = off; off += align_up(sizeof(float) * (size_t)p.batch * (m ? mpow : 0) + 16);
    const int n[3] = {p.grid.nx, p.grid.ny, (dim == 3) ? p.grid.nz : 1};
    for (int a = 0; a < 3; ++a) {
        const int ng = (a < dim) ? 2 * (n[a] - 1) : 0;
        w.gstride[a] = (ng + 3) / 4 * 4 + 8;     // slack so that vector reads past the last point stay inside
        w.cg[a] = off;
        off += align_up(sizeof(float) * (size_t)m * w.gstride[a] + 16);
    }
    for (int a = 0; a < 3; ++a) {
        w.nstride[a] = (a < dim) ? (n[a] + 3) / 4 * 4 + 8 : 0;
        w.cn[a] = off;
        off += align_up(sizeof(float) * (size_t)m * w.nstride[a] + 16);
    }
    w.seam = off;
    {   // tile seams of the 3D kernel families: the family in use (tight), or the larger of the two that may be chosen
        size_t fl = 0;
        if (tight ? l.path == PATH_TILED3D : tiled3d_applicable(p)) fl = tiled3d_seam_floats(p);
        if (tight ? l.path == PATH_STRIP3D : strip3d_applicable(p)) { const size_t t = strip3d_seam_floats(p); if (t > fl) fl = t; }
        if (tight ? (l.path == PATH_TILED3D || l.path == PATH_STRIP3D) : (tiled3d_applicable(p) || strip3d_applicable(p)))
            off += align_up(sizeof(float) * fl + 16);
    }
    w.rowpoly = off;
    if ((tight ? l.path == PATH_STRIP2D : strip2d_applicable(p))) off += align_up(sizeof(float) * strip2d_rowpoly_floats(p) + 16);
    else if ((tight ? l.path == PATH_ROW2D : row2d_applicable(p))) off += align_up(sizeof(float) * row2d_rowpoly_floats(p) + 16);
    w.zseam = off;
    w.linepoly = off;
    if ((tight ? l.path == PATH_STRIP3D : strip3d_applicable(p))) {
        off += align_up(sizeof(float) * strip3d_zseam_floats(p) + 16);
        w.linepoly = off;
        off += align_up(sizeof(float) * strip3d_linepoly_floats(p) + 16);
    }
    w.total = off;
    return w;
}

static Params make_params(const dn_problem& p, const WsLayout& w, const float* u, const float* gJ, float* r, void* ws) {
    Params P{};
    P.dim = p.grid.dim; P.nx = p.grid.nx; P.ny = p.grid.ny; P.nz = (p.grid.dim == 3) ? p.grid.nz : 1;
    P.batch = p.batch; P.nu_mode = p.nu_mode; P.m = (p.nu_mode != DN_NU_NODAL) ? p.kl_modes : 0;
    P.flags = p.flags; P.f_const = p.f_const; P.bc_x0 = p.bc_x0; P.bc_x1 = p.bc_x1;
    P.hx = (float)(1.0 / (P.nx - 1)); P.hy = (float)(1.0 / (P.ny - 1));
    P.hz = (P.dim == 3) ? (float)(1.0 / (P.nz - 1)) : 1.0f;
    P.u = u; P.nu = p.nu; P.f = p.f; P.gJ = gJ; P.r = r;
    P.bc0_b = p.bc_x0_b; P.bc1_b = p.bc_x1_b;
    char* base = static_cast<char*>(ws);
    P.partials = reinterpret_cast<double*>(base + w.partials);
    P.ckl = reinterpret_cast<const float*>(base + w.ckl);
    for (int a = 0; a < 3; ++a) { P.cg[a] = reinterpret_cast<const float*>(base + w.cg[a]); P.gstride[a] = w.gstride[a]; }
    for (int a = 0; a < 3; ++a) { P.cn[a] = reinterpret_cast<const float*>(base + w.cn[a]); P.nstride[a] = w.nstride[a]; }
    P.nblk = w.nblk;
    P.seam = reinterpret_cast<float*>(base + w.seam);
    P.zseam = reinterpret_cast<float*>(base + w.zseam);
    P.nodes = nodes_per_sample(p.grid);
    return P;
}

// The KL tables of a problem, written into its workspace: scaled weights and cosines (the same for every kernel
// family) and, where the chosen family is the strip kernel, its per-row polynomials.
static cudaError_t tables_into(const dn_problem& p, const Params& P, const WsLayout& w, const Launch& l, void* ws,
                               cudaStream_t s) {
    char* base = static_cast<char*>(ws);
    float* cg[3] = {reinterpret_cast<float*>(base + w.cg[0]), reinterpret_cast<float*>(base + w.cg[1]),
                    reinterpret_cast<float*>(base + w.cg[2])};
    float* cn[3] = {reinterpret_cast<float*>(base + w.cn[0]), reinterpret_cast<float*>(base + w.cn[1]),
                    reinterpret_cast<float*>(base + w.cn[2])};
    const cudaError_t e = launch_tables(P, p.kl_w, reinterpret_cast<float*>(base + w.ckl), cg, cn, s,
                                        (l.path == PATH_STRIP2D || l.path == PATH_ROW2D) ? reinterpret_cast<float*>(base + w.rowpoly) : nullptr,
                                        strip2d_rowpoly_stride(p.kl_modes), p.nu_mode == DN_NU_KL_NODAL);
    if (e != cudaSuccess || l.path != PATH_STRIP3D) return e;
    return launch_linepoly3d(P, reinterpret_cast<float*>(base + w.linepoly), s);
}

// Everything that is decided before anything is enqueued: validation, the kernel family, the workspace layout and
// whether it fits ws_bytes.
static dn_status plan(const dn_problem* p, const float* u, const float* r, size_t ws_bytes, bool tight, Launch& l,
                      WsLayout& w) {
    dn_status st = validate(p);
    if (st != DN_OK) return st;
    if (!u) return DN_ERR_NULL;
    if (r) {
        const size_t bytes = sizeof(float) * (size_t)p->batch * nodes_per_sample(p->grid);
        const char* a = reinterpret_cast<const char*>(u);
        const char* b = reinterpret_cast<const char*>(r);
        if (a < b + bytes && b < a + bytes) return DN_ERR_ALIAS;
    }
    l = choose_launch(*p, u, r);
    w = make_layout(*p, l, tight);
    if (tight && (l.path == PATH_STRIP2D || l.path == PATH_ROW2D) && ws_bytes < w.total) {
        // the strip / row kernel's coefficient table does not fit: the tiled kernel where it can run (rows of at most
        // 2048 nodes, constant forcing), else the any-size kernel; if that does not fit either the call is refused
        if (p->f == nullptr && tiled2d_applicable(*p)) {
            l = tiled2d_geometry(*p);
        } else {
            l = Launch{};
            l.path = PATH_GENERIC;
            l.nblk = generic_blocks_per_sample(nodes_per_sample(p->grid));
        }
        w = make_layout(*p, l, tight);
    }
    if (tight && l.path == PATH_STRIP3D && ws_bytes < w.total) {
        // smaller scratch: the tiled kernel (no coefficient table, one kind of seam) where it can run (constant forcing,
        // KL at the Gauss points or a stored field), else the any-size kernel
        if (p->f == nullptr && tiled3d_applicable(*p)) {
            l = tiled3d_geometry(*p);
        } else {
            l = Launch{};
            l.path = PATH_GENERIC;
            l.nblk = generic_blocks_per_sample(nodes_per_sample(p->grid));
        }
        w = make_layout(*p, l, tight);
    }
    return (ws_bytes < w.total) ? DN_ERR_WORKSPACE : DN_OK;
}

dn_status check_tight(const dn_problem* p, const float* u, const float* r, size_t ws_bytes) {
    if (!r) return DN_ERR_NULL;
    Launch l{};
    WsLayout w{};
    return plan(p, u, r, ws_bytes, true, l, w);
}

static dn_status run(const dn_problem* p, const float* u, const float* gJ, float* J, float* r, void* ws,
                     size_t ws_bytes, void* stream, void* ev_before = nullptr, void* ev_after = nullptr,
                     bool tight = false) {
    Launch l{};
    WsLayout w{};
    const dn_status st = plan(p, u, r, ws_bytes, tight, l, w);
    if (st != DN_OK && st != DN_ERR_WORKSPACE) return st;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) % kAlign) != 0 || ws_bytes < w.total) return DN_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    Params P = make_params(*p, w, u, gJ, r, ws);
    cudaError_t e = cudaSuccess;
    if (p->nu_mode != DN_NU_NODAL && tables_into(*p, P, w, l, ws, s) != cudaSuccess) return DN_ERR_CUDA;
    if (ev_before && cudaEventRecord(static_cast<cudaEvent_t>(ev_before), s) != cudaSuccess) return DN_ERR_CUDA;
    if (l.path == PATH_STRIP2D) e = launch_strip2d(P, reinterpret_cast<const float*>(static_cast<char*>(ws) + w.rowpoly), s);
    else if (l.path == PATH_ROW2D) e = launch_row2d(P, reinterpret_cast<const float*>(static_cast<char*>(ws) + w.rowpoly), s);
    else if (l.path == PATH_TILED2D) e = launch_tiled2d(P, l, s);
    else if (l.path == PATH_TILED3D) e = launch_tiled3d(P, l, s);
    else if (l.path == PATH_STRIP3D) e = launch_strip3d(P, reinterpret_cast<const float*>(static_cast<char*>(ws) + w.linepoly), s);
    else e = launch_generic(P, s);
    if (e != cudaSuccess) return DN_ERR_CUDA;
    if (ev_after && cudaEventRecord(static_cast<cudaEvent_t>(ev_after), s) != cudaSuccess) return DN_ERR_CUDA;
    if (J) {
        e = launch_finalize(P.partials, w.nblk, p->batch, J, s);
        if (e != cudaSuccess) return DN_ERR_CUDA;
    }
    return DN_OK;
}

dn_status run_operator(const dn_problem* p, const float* u, float* r, void* ws, size_t ws_bytes, cudaStream_t s,
                       bool build_tables, const double** partials, int* nblk) {
    dn_status st = validate(p);
    if (st != DN_OK) return st;
    if (!u || !r) return DN_ERR_NULL;
    const Launch l = choose_launch(*p, u, r);
    const WsLayout w = make_layout(*p, l, false);
    if (!ws || (reinterpret_cast<uintptr_t>(ws) % kAlign) != 0 || ws_bytes < w.total) return DN_ERR_WORKSPACE;
    Params P = make_params(*p, w, u, nullptr, r, ws);
    cudaError_t e = cudaSuccess;
    if (build_tables && p->nu_mode != DN_NU_NODAL && tables_into(*p, P, w, l, ws, s) != cudaSuccess) return DN_ERR_CUDA;
    if (l.path == PATH_STRIP2D) e = launch_strip2d(P, reinterpret_cast<const float*>(static_cast<char*>(ws) + w.rowpoly), s);
    else if (l.path == PATH_ROW2D) e = launch_row2d(P, reinterpret_cast<const float*>(static_cast<char*>(ws) + w.rowpoly), s);
    else if (l.path == PATH_TILED2D) e = launch_tiled2d(P, l, s);
    else if (l.path == PATH_TILED3D) e = launch_tiled3d(P, l, s);
    else if (l.path == PATH_STRIP3D) e = launch_strip3d(P, reinterpret_cast<const float*>(static_cast<char*>(ws) + w.linepoly), s);
    else e = launch_generic(P, s);
    if (e != cudaSuccess) return DN_ERR_CUDA;
    if (partials) *partials = P.partials;
    if (nblk) *nblk = w.nblk;
    return DN_OK;
}

dn_status build_tables(const dn_problem* p, const float* u, float* r, void* ws, size_t ws_bytes, cudaStream_t s) {
    dn_status st = validate(p);
    if (st != DN_OK) return st;
    if (p->nu_mode == DN_NU_NODAL) return DN_OK;
    const Launch l = choose_launch(*p, u, r);
    const WsLayout w = make_layout(*p, l, false);
    if (!ws || (reinterpret_cast<uintptr_t>(ws) % kAlign) != 0 || ws_bytes < w.total) return DN_ERR_WORKSPACE;
    const Params P = make_params(*p, w, u, nullptr, r, ws);
    return tables_into(*p, P, w, l, ws, s) == cudaSuccess ? DN_OK : DN_ERR_CUDA;
}

dn_status run_tight(const dn_problem* p, const float* u, const float* gJ, float* J, float* r, void* ws,
                    size_t ws_bytes, void* stream) {
    if (!r) return DN_ERR_NULL;
    return run(p, u, gJ, J, r, ws, ws_bytes, stream, nullptr, nullptr, true);
}

}  // namespace dn

using namespace dn;

extern "C" {

size_t dn_workspace_bytes(const dn_problem* p) {
    if (validate(p) != DN_OK) return 0;
    Launch l{};
    l.nblk = 1;
    return make_layout(*p, l).total;
}

size_t dn_host_staging_bytes(const dn_problem* p) {
    if (validate(p) != DN_OK) return 0;
    const size_t field = align_up(sizeof(float) * (size_t)p->batch * nodes_per_sample(p->grid));
    size_t total = 2 * field;                                   // u, r
    total += 4 * align_up(sizeof(float) * (size_t)p->batch);    // J, gJ, per-sample boundary values
    if (p->nu_mode == DN_NU_NODAL) total += field;
    if (p->f) total += field;
    size_t mpow = 1;
    for (int a = 0; a < p->grid.dim; ++a) mpow *= (size_t)((p->nu_mode != DN_NU_NODAL) ? p->kl_modes : 0);
    total += align_up(sizeof(float) * (size_t)p->batch * mpow + 16);
    return total + dn_workspace_bytes(p);
}

dn_status dn_energy(const dn_problem* p, const float* u, float* J, void* ws, size_t ws_bytes, void* stream) {
    if (!J) return DN_ERR_NULL;
    return run(p, u, nullptr, J, nullptr, ws, ws_bytes, stream);
}

dn_status dn_energy_grad(const dn_problem* p, const float* u, const float* gJ, float* J, float* r, void* ws,
                         size_t ws_bytes, void* stream) {
    if (!r) return DN_ERR_NULL;
    return run(p, u, gJ, J, r, ws, ws_bytes, stream);
}

dn_status dn_energy_grad_traced(const dn_problem* p, const float* u, const float* gJ, float* J, float* r, void* ws,
                                size_t ws_bytes, void* stream, void* ev_before, void* ev_after) {
    if (!r) return DN_ERR_NULL;
    return run(p, u, gJ, J, r, ws, ws_bytes, stream, ev_before, ev_after);
}

dn_status dn_kl_field(const dn_grid* g, int32_t batch, int32_t m, const float* kl_w, float* nu, void* stream) {
    if (!g || !kl_w || !nu) return DN_ERR_NULL;
    dn_status st = DN_OK;
    if (!valid_grid(*g, st)) return st;
    if (batch < 1 || batch > 65535) return DN_ERR_SIZE;
    if (m < 1 || m > DN_MAX_KL_MODES) return DN_ERR_MODE;
    return launch_kl_field(*g, batch, m, kl_w, nu, static_cast<cudaStream_t>(stream)) == cudaSuccess ? DN_OK : DN_ERR_CUDA;
}

dn_status dn_apply_bc(const dn_grid* g, int32_t batch, float b0, float b1, int32_t mode, float* field, void* stream) {
    if (!g || !field) return DN_ERR_NULL;
    dn_status st = DN_OK;
    if (!valid_grid(*g, st)) return st;
    if (batch < 1 || batch > 65535) return DN_ERR_SIZE;
    if (mode != 0 && mode != 1) return DN_ERR_MODE;
    return launch_apply_bc(*g, batch, b0, b1, mode, field, static_cast<cudaStream_t>(stream)) == cudaSuccess ? DN_OK
                                                                                                            : DN_ERR_CUDA;
}

dn_status dn_apply_bc_per_sample(const dn_grid* g, int32_t batch, const float* b0, const float* b1, float* field,
                                 void* stream) {
    if (!g || !field || !b0 || !b1) return DN_ERR_NULL;
    dn_status st = DN_OK;
    if (!valid_grid(*g, st)) return st;
    if (batch < 1 || batch > 65535) return DN_ERR_SIZE;
    return launch_apply_bc(*g, batch, 0.f, 0.f, 0, field, static_cast<cudaStream_t>(stream), b0, b1) == cudaSuccess
               ? DN_OK : DN_ERR_CUDA;
}

// The batch is cut into chunks of whole samples that flow through three stages on three streams:
// host->device copy, kernels (on the caller's stream), device->host copy.  Chunk c+1 is copied in
// and chunk c-1 copied out while chunk c computes, so both directions of the host link stay busy.
dn_status dn_energy_grad_host(const dn_problem* p, const float* u_host, const float* gJ_host, float* J_host,
                              float* r_host, void* staging, size_t staging_bytes, void* stream) {
    dn_status st = validate(p);
    if (st != DN_OK) return st;
    if (!u_host || !r_host) return DN_ERR_NULL;
    if (!staging || (reinterpret_cast<uintptr_t>(staging) % kAlign) != 0 || staging_bytes < dn_host_staging_bytes(p))
        return DN_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t nodes = (size_t)nodes_per_sample(p->grid);
    const size_t nfield = (size_t)p->batch * nodes;
    const size_t field = align_up(sizeof(float) * nfield);
    const size_t small = align_up(sizeof(float) * (size_t)p->batch);
    size_t mpow = 1;
    for (int a = 0; a < p->grid.dim; ++a) mpow *= (size_t)((p->nu_mode != DN_NU_NODAL) ? p->kl_modes : 0);
    char* base = static_cast<char*>(staging);
    size_t off = 0;
    float* d_u = reinterpret_cast<float*>(base + off); off += field;
    float* d_r = reinterpret_cast<float*>(base + off); off += field;
    float* d_J = reinterpret_cast<float*>(base + off); off += small;
    float* d_g = reinterpret_cast<float*>(base + off); off += small;
    float* d_b0 = reinterpret_cast<float*>(base + off); off += small;
    float* d_b1 = reinterpret_cast<float*>(base + off); off += small;
    float* d_nu = nullptr; float* d_f = nullptr;
    if (p->nu_mode == DN_NU_NODAL) { d_nu = reinterpret_cast<float*>(base + off); off += field; }
    if (p->f) { d_f = reinterpret_cast<float*>(base + off); off += field; }
    float* d_w = reinterpret_cast<float*>(base + off); off += align_up(sizeof(float) * (size_t)p->batch * mpow + 16);
    void* ws = base + off;
    const size_t ws_bytes = staging_bytes - off;

    // chunks of whole samples; one chunk if a chunk's workspace would not fit (its kernels may tile differently)
    // ... of at least 8 MiB each, so that small problems are not cut into launches that cost more than they hide
    const size_t sample_bytes = sizeof(float) * nodes;
    int csize = (p->batch + HostPipe::kMaxChunks - 1) / HostPipe::kMaxChunks;
    const size_t min_chunk = (size_t)8 << 20;
    if ((size_t)csize * sample_bytes < min_chunk) csize = (int)((min_chunk + sample_bytes - 1) / sample_bytes);
    if (csize > p->batch) csize = p->batch;
    int nchunks = (p->batch + csize - 1) / csize;
    {   // both chunk sizes that will occur (full chunks and the shorter last one) must fit the workspace
        dn_problem q = *p;
        q.batch = csize;
        bool fits = dn_workspace_bytes(&q) <= ws_bytes;
        const int last = p->batch - (nchunks - 1) * csize;
        if (fits && last != csize) { q.batch = last; fits = dn_workspace_bytes(&q) <= ws_bytes; }
        if (!fits) { csize = p->batch; nchunks = 1; }
    }
    HostPipe pipe;
    if (!pipe.create(nchunks)) return DN_ERR_CUDA;
    // On any failure the copies and kernels already enqueued are waited for before the call returns (they read and
    // write the caller's host buffers, and the streams are destroyed on return).
    auto drain = [&]() { cudaStreamSynchronize(pipe.in); cudaStreamSynchronize(s); cudaStreamSynchronize(pipe.out); };
#define DN_TRY(x) do { if ((x) != cudaSuccess) { drain(); return DN_ERR_CUDA; } } while (0)
    DN_TRY(cudaEventRecord(pipe.start, s));                       // the call is ordered after earlier work on `stream`
    DN_TRY(cudaStreamWaitEvent(pipe.in, pipe.start, 0));
    DN_TRY(cudaStreamWaitEvent(pipe.out, pipe.start, 0));
    if (p->nu_mode != DN_NU_NODAL)
        DN_TRY(cudaMemcpyAsync(d_w, p->kl_w, sizeof(float) * (size_t)p->batch * mpow, cudaMemcpyHostToDevice, pipe.in));
    if (gJ_host) DN_TRY(cudaMemcpyAsync(d_g, gJ_host, sizeof(float) * p->batch, cudaMemcpyHostToDevice, pipe.in));
    if (p->bc_x0_b) DN_TRY(cudaMemcpyAsync(d_b0, p->bc_x0_b, sizeof(float) * p->batch, cudaMemcpyHostToDevice, pipe.in));
    if (p->bc_x1_b) DN_TRY(cudaMemcpyAsync(d_b1, p->bc_x1_b, sizeof(float) * p->batch, cudaMemcpyHostToDevice, pipe.in));
    for (int c = 0; c < nchunks; ++c) {
        const int b0 = c * csize;
        const int nb = (b0 + csize <= p->batch) ? csize : p->batch - b0;
        const size_t o = (size_t)b0 * nodes, n = (size_t)nb * nodes;
        DN_TRY(cudaMemcpyAsync(d_u + o, u_host + o, sizeof(float) * n, cudaMemcpyHostToDevice, pipe.in));
        if (d_nu) DN_TRY(cudaMemcpyAsync(d_nu + o, p->nu + o, sizeof(float) * n, cudaMemcpyHostToDevice, pipe.in));
        if (d_f) DN_TRY(cudaMemcpyAsync(d_f + o, p->f + o, sizeof(float) * n, cudaMemcpyHostToDevice, pipe.in));
        DN_TRY(cudaEventRecord(pipe.copied[c], pipe.in));
        DN_TRY(cudaStreamWaitEvent(s, pipe.copied[c], 0));
        dn_problem q = *p;
        q.batch = nb;
        q.nu = d_nu ? d_nu + o : nullptr;
        q.f = d_f ? d_f + o : nullptr;
        q.kl_w = (p->nu_mode != DN_NU_NODAL) ? d_w + (size_t)b0 * mpow : nullptr;
        q.bc_x0_b = p->bc_x0_b ? d_b0 + b0 : nullptr;
        q.bc_x1_b = p->bc_x1_b ? d_b1 + b0 : nullptr;
        st = run(&q, d_u + o, gJ_host ? d_g + b0 : nullptr, J_host ? d_J + b0 : nullptr, d_r + o, ws, ws_bytes, s);
        if (st != DN_OK) { drain(); return st; }
        DN_TRY(cudaEventRecord(pipe.computed[c], s));
        DN_TRY(cudaStreamWaitEvent(pipe.out, pipe.computed[c], 0));
        DN_TRY(cudaMemcpyAsync(r_host + o, d_r + o, sizeof(float) * n, cudaMemcpyDeviceToHost, pipe.out));
    }
    if (J_host) DN_TRY(cudaMemcpyAsync(J_host, d_J, sizeof(float) * p->batch, cudaMemcpyDeviceToHost, pipe.out));
    DN_TRY(cudaStreamSynchronize(pipe.in));
    DN_TRY(cudaStreamSynchronize(s));
    DN_TRY(cudaStreamSynchronize(pipe.out));
#undef DN_TRY
    return DN_OK;
}

int32_t dn_launches_per_call(const dn_problem* p) {
    if (validate(p) != DN_OK) return 0;
    const bool fast = !(p->flags & DN_FORCE_GENERIC) && p->f == nullptr;
    if (!(p->flags & DN_FORCE_GENERIC) && strip3d_applicable(*p))                 // (tables, line polynomials,) fused kernel, seam fix-up, finaliser
        return 2 + (p->nu_mode != DN_NU_NODAL ? 2 : 0) + ((strip3d_seam_floats(*p) + strip3d_zseam_floats(*p)) > 0 ? 1 : 0);
    const bool t3 = fast && !tiled2d_applicable(*p) && tiled3d_applicable(*p);
    return 2 + (p->nu_mode != DN_NU_NODAL ? 1 : 0) + ((t3 && tiled3d_seam_floats(*p) > 0) ? 1 : 0);
}

const char* dn_path_name(const dn_problem* p) {
    if (validate(p) != DN_OK) return "invalid";
    // the fused call (the strip kernels also with nodal forcing).  The energy-only call runs the same family in 3D; in
    // 2D the tiled kernel where it can run (constant forcing, rows of at most 2048 nodes), else the strip kernel
    if (!(p->flags & DN_FORCE_GENERIC) && row2d_applicable(*p)) return "row2d";
    if (!(p->flags & DN_FORCE_GENERIC) && strip2d_applicable(*p)) return "strip2d";
    if (!(p->flags & DN_FORCE_GENERIC) && p->f == nullptr && tiled2d_applicable(*p)) return "tiled2d";
    if (!(p->flags & DN_FORCE_GENERIC) && strip3d_applicable(*p)) return "strip3d";
    if (!(p->flags & DN_FORCE_GENERIC) && p->f == nullptr && tiled3d_applicable(*p)) return "tiled3d";
    return "generic";
}

const char* dn_status_string(dn_status s) {
    switch (s) {
        case DN_OK: return "ok";
        case DN_ERR_NULL: return "a required pointer is NULL";
        case DN_ERR_DIM: return "dim must be 2 or 3";
        case DN_ERR_SIZE: return "grid extent or batch out of range";
        case DN_ERR_MODE: return "unknown mode or kl_modes out of range";
        case DN_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case DN_ERR_CUDA: return "CUDA runtime error";
        case DN_ERR_ALIAS: return "r overlaps u";
    }
    return "unknown status";
}

}  // extern "C"
