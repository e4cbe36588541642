// Strip kernel for 3D grids whose rows fit one warp (nx <= 256): fused element quadrature, energy reduction,
// node gather, mask and store on hexahedra, without any barrier between warps.
//
// Layout of the work.  A work unit is one sample, one tile of Ry element rows (y) across the whole x extent, one
// chunk of Z element planes (z).  A unit belongs to LW = 8, 16 or 32 lanes of one warp (a lane owns NX = 4 or 8
// consecutive nodes of a row, so LW * NX >= nx); a warp with LW < 32 carries 32 / LW units that have nothing to do
// with one another.  No warp ever waits for another warp: there is no block-wide barrier and no exchange between
// warps through shared memory.
//
// A unit marches over its element planes from bottom to top, and inside a plane over its element rows.  The node
// rows it needs stream through a ring of rows in shared memory that belongs to the unit alone: row (plane k, row j)
// of the tile is entry k * T + j of a linear sequence (T node rows per plane), entry n lives in slot n mod C, and
// the ring always holds the two planes being worked on plus D rows in flight (cp.async, one group per row; every
// lane copies the 16-byte pieces of its own nodes, a few lanes also copy the coefficients described below).  Every
// node is read from global memory once per unit.
//
// Element (x, j, k) is computed once, by the lane that owns node x.  Of its 8 corner contributions those to column
// x + 1 pass to the next element of the lane (to the next lane by shuffle), those to row j + 1 are kept until the
// next row of the same plane, and those to plane k + 1 are parked in the output array itself: the lane stores the
// partial sums of node row (j, k + 1) into r, and one plane later reads them back, adds what element plane k + 1
// contributes, and stores the finished value (same thread, same address: program order makes the read see the
// write; the lines stay in L2 in between).  So the registers hold one row of pending values, not a plane.
//
// Tiles do not overlap in y: the top element row of a tile leaves what it contributes to the first node row of
// the next tile in a scratch array (seam, [B][ntile-1][nz][nx]), parked there between planes in the same way, and
// a small fix-up kernel adds those rows to r afterwards.  Chunks do not overlap in z either: what the last element
// plane of a chunk contributes to the first node plane of the next chunk goes to a second scratch array (zseam,
// [B][nchunk-1][ny][nx], plus [B][nchunk-1][ntile-1][nx] for the nodes that are on a tile seam as well), added by the
// same fix-up kernel.  Every element is computed exactly once.  No atomics; every sum has a fixed order.
//
// Arithmetic of one element: hierarchical coordinates of the trilinear field (edge differences e, s, w at the low
// corner, second differences txy, txz, tyz, third difference txyz), derivatives at the 4 Gauss lines of each
// direction, sums of nu along each derivative's own axis, the adjoint of the interpolation and the chain rule to
// the 8 corners -- the formulas of the tiled 3D kernel.  The diffusion energy is taken from the residual by
// Euler's identity for quadratic forms: 1/2 sum over (node, contribution) pairs of u_node times contribution, each
// pair counted by the unit that computes it.
//
// KL diffusivity at the Gauss points: along a Gauss line (y_q, z_s fixed) the exponent is a polynomial of degree m
// in c = cos(pi x).  A table kernel prepares the coefficients of all four lines of every element row of every
// element plane once per call in double ([B][nz-1][ny-1][2][GS] floats: Gauss row q, then coefficient i and Gauss
// plane s interleaved for packed two-wide FMAs); they travel through the ring with the node row that completes
// the element row.
#include "dn_internal.cuh"

namespace dn {

namespace {

constexpr int S3_WARPS = 4;                       // warps per block (each warp is on its own)
constexpr int S3_D = 3;                           // rows in flight beyond the two planes in use

typedef unsigned long long u64;

__device__ __forceinline__ float s3_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void s3_unpack(u64 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ u64 s3_pack(float lo, float hi) {
    u64 v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
    return v;
}
__device__ __forceinline__ u64 s3_fma2(u64 a, u64 b, u64 c) {
    u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ void s3_cp16(float* smem_dst, const float* gsrc) {
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void s3_cp16_if(float* smem_dst, const float* gsrc, int pred) {    // predicated, no branch
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.s32 p, %2, 0;\n\t@p cp.async.cg.shared.global [%0], [%1], 16;\n\t}"
                 ::"r"(d), "l"(gsrc), "r"(pred) : "memory");
}
// the same with the shared-memory address already converted
__device__ __forceinline__ void s3_cp16s(unsigned d, const float* gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void s3_cp16s_if(unsigned d, const float* gsrc, int pred) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.s32 p, %2, 0;\n\t@p cp.async.cg.shared.global [%0], [%1], 16;\n\t}"
                 ::"r"(d), "l"(gsrc), "r"(pred) : "memory");
}
__device__ __forceinline__ void s3_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void s3_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Floats per Gauss row (q fixed) of an element row in the coefficient table: (plane s = a, s = b) pairs for
// i = 0..M, padded to a multiple of 4.
__host__ __device__ constexpr int s3_gs(int m) { return (2 * (m + 1) + 3) / 4 * 4; }

}  // namespace

// The file is compiled twice to halve the build time: DN_S3_PART 0 (the default) holds everything and the kernels for
// m <= 4 and for the stored field; part 1 holds only the kernels for m = 5..8 and hands them out through
// launch_strip3d_hi.
#ifndef DN_S3_PART
#define DN_S3_PART 0
#endif

struct S3Geo {
    int Ry, Z;            // element rows per tile, element planes per chunk
    int ntile, nchunk;
    int LW, lwsh;         // lanes per unit and log2 of it
    int C, RS;            // ring slots (rows) per unit, floats per slot
    long long units;
};
cudaError_t launch_strip3d_hi(const Params& P, const float* linepoly, const S3Geo& g, cudaStream_t s);

namespace {

// nu at the 8 Gauss points of one element, index [p][q][s] -> n[4 p + 2 q + s]: four packed Horner chains
// (column p, row q), each over the planes s = a, b.
template <int M>
__device__ __forceinline__ void s3_nu_gauss(const u64 (&ga)[s3_gs(M) / 2], const u64 (&gb)[s3_gs(M) / 2], const u64 ca2,
                                            const u64 cb2, float (&n)[8]) {
    u64 h_aa = ga[M], h_ab = gb[M], h_ba = ga[M], h_bb = gb[M];          // h_{p q}
#pragma unroll
    for (int i = M - 1; i >= 0; --i) {
        h_aa = s3_fma2(h_aa, ca2, ga[i]); h_ab = s3_fma2(h_ab, ca2, gb[i]);
        h_ba = s3_fma2(h_ba, cb2, ga[i]); h_bb = s3_fma2(h_bb, cb2, gb[i]);
    }
    float x[8];
    s3_unpack(h_aa, x[0], x[1]); s3_unpack(h_ab, x[2], x[3]);
    s3_unpack(h_ba, x[4], x[5]); s3_unpack(h_bb, x[6], x[7]);
#pragma unroll
    for (int i = 0; i < 8; ++i) n[i] = s3_ex2(x[i]);
}

// Sums of nu along each derivative's own axis, from nu at the 8 Gauss points n[4p + 2q + s]:
// Nx[2q + s] = sum_p, Ny[2p + s] = sum_q, Nz[2p + q] = sum_s.
__device__ __forceinline__ void s3_sums_gauss(const float (&n)[8], float (&Nx)[4], float (&Ny)[4], float (&Nz)[4]) {
    Nx[0] = n[0] + n[4]; Nx[1] = n[1] + n[5]; Nx[2] = n[2] + n[6]; Nx[3] = n[3] + n[7];
    Ny[0] = n[0] + n[2]; Ny[1] = n[1] + n[3]; Ny[2] = n[4] + n[6]; Ny[3] = n[5] + n[7];
    Nz[0] = n[0] + n[1]; Nz[1] = n[2] + n[3]; Nz[2] = n[4] + n[5]; Nz[3] = n[6] + n[7];
}

// The same sums for a trilinear nu given at the corners.  Summing the interpolant over the two Gauss points of an axis
// leaves the sum of the two corner values along that axis (the weights a and b add up to 1), interpolated in the other
// two.  h00, h10, h01, h11: those edge sums at (first, second) other coordinate = low/high; out[2 i1 + i2] at the
// Gauss abscissae (i1, i2) of the two other axes.
__device__ __forceinline__ void s3_bilerp(const float h00, const float h10, const float h01, const float h11, float (&out)[4]) {
    const float d0 = h10 - h00, d1 = h11 - h01;
    const float ma0 = fmaf(DN_GA, d0, h00), mb0 = fmaf(DN_GB, d0, h00);     // first coordinate a / b, second low
    const float ma1 = fmaf(DN_GA, d1, h01), mb1 = fmaf(DN_GB, d1, h01);     // ... second high
    const float da = ma1 - ma0, db = mb1 - mb0;
    out[0] = fmaf(DN_GA, da, ma0); out[1] = fmaf(DN_GB, da, ma0);
    out[2] = fmaf(DN_GA, db, mb0); out[3] = fmaf(DN_GB, db, mb0);
}

// Nodal forcing: the element mass matrix applied to the 8 corner values of f, by sum factorisation (per axis the
// matrix [[2, 1], [1, 2]]; the factor hx hy hz / 216 is applied by the caller).  f and m are indexed i + 2j + 4k.
__device__ __forceinline__ void s3_mass(const float (&f)[8], float (&m)[8]) {
    float g[8], h[8];
#pragma unroll
    for (int t = 0; t < 8; t += 2) { g[t] = fmaf(2.f, f[t], f[t + 1]); g[t + 1] = fmaf(2.f, f[t + 1], f[t]); }          // x
#pragma unroll
    for (int t = 0; t < 8; ++t) { if (t & 2) continue; h[t] = fmaf(2.f, g[t], g[t + 2]); h[t + 2] = fmaf(2.f, g[t + 2], g[t]); }   // y
#pragma unroll
    for (int t = 0; t < 4; ++t) { m[t] = fmaf(2.f, h[t], h[t + 4]); m[t + 4] = fmaf(2.f, h[t + 4], h[t]); }               // z
}

// The element: from the 12 sums of nu and the 7 hierarchical coordinates of u to the 8 corner contributions
// r[i + 2j + 4k] (i, j, k the x, y, z bits of the corner), all in units of kap = hx hy hz / (8 h^2) on isotropic cells
// (iso), else scaled by kx, ky, kz here.
__device__ __forceinline__ void s3_element(const float (&Nx)[4], const float (&Ny)[4], const float (&Nz)[4],
                                           const float e0, const float s0, const float w0,
                                           const float txy, const float txz, const float tyz, const float txyz,
                                           const bool iso, const float kx, const float ky, const float kz,
                                           float (&r)[8]) {
    const float a = DN_GA, bq = DN_GB;
    float Nx_aa = Nx[0], Nx_ab = Nx[1], Nx_ba = Nx[2], Nx_bb = Nx[3];   // (q, s)
    float Ny_aa = Ny[0], Ny_ab = Ny[1], Ny_ba = Ny[2], Ny_bb = Ny[3];   // (p, s)
    float Nz_aa = Nz[0], Nz_ab = Nz[1], Nz_ba = Nz[2], Nz_bb = Nz[3];   // (p, q)
    if (!iso) {
        Nx_aa *= kx; Nx_ab *= kx; Nx_ba *= kx; Nx_bb *= kx;
        Ny_aa *= ky; Ny_ab *= ky; Ny_ba *= ky; Ny_bb *= ky;
        Nz_aa *= kz; Nz_ab *= kz; Nz_ba *= kz; Nz_bb *= kz;
    }
    // derivatives at the Gauss lines: d/dx at (eta q, zeta s) = (e + q txy) + s (txz + q txyz), and cyclically
    const float Axa = fmaf(a, txy, e0), Axb = fmaf(bq, txy, e0);
    const float Bxa = fmaf(a, txyz, txz), Bxb = fmaf(bq, txyz, txz);
    const float Dx_aa = fmaf(a, Bxa, Axa), Dx_ab = fmaf(bq, Bxa, Axa), Dx_ba = fmaf(a, Bxb, Axb), Dx_bb = fmaf(bq, Bxb, Axb);
    const float Aya = fmaf(a, txy, s0), Ayb = fmaf(bq, txy, s0);
    const float Bya = fmaf(a, txyz, tyz), Byb = fmaf(bq, txyz, tyz);
    const float Dy_aa = fmaf(a, Bya, Aya), Dy_ab = fmaf(bq, Bya, Aya), Dy_ba = fmaf(a, Byb, Ayb), Dy_bb = fmaf(bq, Byb, Ayb);
    const float Aza = fmaf(a, txz, w0), Azb = fmaf(bq, txz, w0);
    const float Dz_aa = fmaf(a, Bya, Aza), Dz_ab = fmaf(bq, Bya, Aza), Dz_ba = fmaf(a, Byb, Azb), Dz_bb = fmaf(bq, Byb, Azb);
    const float Gx_aa = Nx_aa * Dx_aa, Gx_ab = Nx_ab * Dx_ab, Gx_ba = Nx_ba * Dx_ba, Gx_bb = Nx_bb * Dx_bb;
    const float Gy_aa = Ny_aa * Dy_aa, Gy_ab = Ny_ab * Dy_ab, Gy_ba = Ny_ba * Dy_ba, Gy_bb = Ny_bb * Dy_bb;
    const float Gz_aa = Nz_aa * Dz_aa, Gz_ab = Nz_ab * Dz_ab, Gz_ba = Nz_ba * Dz_ba, Gz_bb = Nz_bb * Dz_bb;
    // Adjoint of the three interpolations: partial derivatives of the element energy.  With b = a + dl the weighted
    // sums over a 2 x 2 set of Gauss lines reduce to its total S, the sum R over the lines whose first index is b, the
    // sum C over those whose second index is b, and the (b, b) entry:
    //   sum i1 G = a S + dl R,   sum i2 G = a S + dl C,   sum i1 i2 G = a^2 S + a dl (R + C) + dl^2 G_bb.
    constexpr float dl = DN_GB - DN_GA;
    const float R1x = Gx_ba + Gx_bb, Cx = Gx_ab + Gx_bb, dE = (Gx_aa + Gx_ab) + R1x;     // Gx[q][s]
    const float R1y = Gy_ba + Gy_bb, Cy = Gy_ab + Gy_bb, dS = (Gy_aa + Gy_ab) + R1y;     // Gy[p][s]
    const float R1z = Gz_ba + Gz_bb, Cz = Gz_ab + Gz_bb, dW = (Gz_aa + Gz_ab) + R1z;     // Gz[p][q]
    const float Sxy = dE + dS, Sxz = dE + dW, Syz = dS + dW;
    const float P1 = R1x + R1y, P2 = Cx + R1z, P3 = Cy + Cz;
    const float dXY = fmaf(dl, P1, a * Sxy);           // txy enters d/dx through q and d/dy through p
    const float dXZ = fmaf(dl, P2, a * Sxz);           // txz enters d/dx through s and d/dz through p
    const float dYZ = fmaf(dl, P3, a * Syz);           // tyz enters d/dy through s and d/dz through q
    const float dXYZ = fmaf(dl * dl, (Gx_bb + Gy_bb) + Gz_bb, fmaf(a * dl, (P1 + P2) + P3, (a * a) * (Sxy + dW)));
    // chain rule to the corners
    const float r110 = dXY - dXYZ, r101 = dXZ - dXYZ, r011 = dYZ - dXYZ;
    const float r100 = (dE - r110) - dXZ, r010 = (dS - r110) - dYZ, r001 = (dW - r101) - dYZ;
    const float r000 = ((r011 - dW) + (dXY - dE)) + (dXZ - dS);
    r[0] = r000; r[1] = r100; r[2] = r010; r[3] = r110; r[4] = r001; r[5] = r101; r[6] = r011; r[7] = dXYZ;
}

// The element's diffusion energy, twice over and in the same units: sum over the 12 Gauss lines of N D^2 (the
// derivatives as in s3_element; the residual it returns is the gradient of half this sum).
__device__ __forceinline__ float s3_energy(const float (&Nx)[4], const float (&Ny)[4], const float (&Nz)[4],
                                           const float e0, const float s0, const float w0,
                                           const float txy, const float txz, const float tyz, const float txyz,
                                           const bool iso, const float kx, const float ky, const float kz) {
    const float a = DN_GA, bq = DN_GB;
    const float Axa = fmaf(a, txy, e0), Axb = fmaf(bq, txy, e0);
    const float Bxa = fmaf(a, txyz, txz), Bxb = fmaf(bq, txyz, txz);
    const float Dx_aa = fmaf(a, Bxa, Axa), Dx_ab = fmaf(bq, Bxa, Axa), Dx_ba = fmaf(a, Bxb, Axb), Dx_bb = fmaf(bq, Bxb, Axb);
    const float Aya = fmaf(a, txy, s0), Ayb = fmaf(bq, txy, s0);
    const float Bya = fmaf(a, txyz, tyz), Byb = fmaf(bq, txyz, tyz);
    const float Dy_aa = fmaf(a, Bya, Aya), Dy_ab = fmaf(bq, Bya, Aya), Dy_ba = fmaf(a, Byb, Ayb), Dy_bb = fmaf(bq, Byb, Ayb);
    const float Aza = fmaf(a, txz, w0), Azb = fmaf(bq, txz, w0);
    const float Dz_aa = fmaf(a, Bya, Aza), Dz_ab = fmaf(bq, Bya, Aza), Dz_ba = fmaf(a, Byb, Azb), Dz_bb = fmaf(bq, Byb, Azb);
    float ex = (Nx[0] * Dx_aa) * Dx_aa, ey = (Ny[0] * Dy_aa) * Dy_aa, ez = (Nz[0] * Dz_aa) * Dz_aa;
    ex = fmaf(Nx[1] * Dx_ab, Dx_ab, ex); ey = fmaf(Ny[1] * Dy_ab, Dy_ab, ey); ez = fmaf(Nz[1] * Dz_ab, Dz_ab, ez);
    ex = fmaf(Nx[2] * Dx_ba, Dx_ba, ex); ey = fmaf(Ny[2] * Dy_ba, Dy_ba, ey); ez = fmaf(Nz[2] * Dz_ba, Dz_ba, ez);
    ex = fmaf(Nx[3] * Dx_bb, Dx_bb, ex); ey = fmaf(Ny[3] * Dy_bb, Dy_bb, ey); ez = fmaf(Nz[3] * Dz_bb, Dz_bb, ez);
    return iso ? (ex + ey) + ez : fmaf(kx, ex, fmaf(ky, ey, kz * ez));
}

// MODE 0: KL at the Gauss points; 1 (KN): KL at the nodes, then Q1 interpolation; 2 (ND): stored nodal field.
// In the nodal modes a slot of the ring holds the nu row next to the u row: copied from the field (ND), or computed
// from the polynomial of that node line when the row is first used (KN: the table then holds one polynomial per node
// line, every coefficient twice, and travels with the row itself).
// NF: nodal forcing.  The f row sits in the slot as well; the load is taken element by element (mass matrix applied
// to the corner values of f) and joins the corner contributions before they are gathered, so it needs no other
// treatment at the boundary of the domain, a tile or a chunk than the stiffness part.
// EO: energy only.  The same march over the same units, but every element adds its own energy (s3_energy) and
// nothing is gathered, parked or stored: no residual, no seams.
// LWC: lanes per unit at compile time (32 or 16), or 0: taken from G (8 lanes, and every layout with nodal forcing).
// A lane count known to the compiler is worth 3 to 9 % on 256-wide rows and 3 to 4 % on 64-wide ones.
// ISO: the cells are known to be cubes when the kernel is compiled (the scaling of the sums of nu by kx, ky, kz and the
// branch around it go: 2 % on 256^3 x 4); false: decided from the spacings at run time.
template <int NX, int M, int MODE, bool NF, int MINB, bool EO, int LWC, bool ISO>
__global__ void __launch_bounds__(S3_WARPS * 32, MINB)
strip3d_kernel(const Params P, const float* __restrict__ linepoly, const S3Geo G) {
    extern __shared__ __align__(16) float smem[];
    dep_wait();                                         // the tables of this call are complete
    dep_release();                                      // the fix-up kernel may move in as units finish
    constexpr bool KG = (MODE == 0), KN = (MODE == 1), ND = (MODE == 2);
    constexpr int GS = s3_gs(M);
    constexpr int CF = KG ? 2 * GS : KN ? GS : 0;       // coefficient floats per slot (KG: Gauss rows q = a, b of an element row)
    constexpr int CFQ = CF / 4;                         // ... in 16-byte pieces
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int LW = LWC ? LWC : G.LW, lwsh = (LWC == 32) ? 5 : (LWC == 16) ? 4 : G.lwsh, SUBS = 32 >> lwsh;
    const int sub = lane >> lwsh, lx = lane & (LW - 1);
    const unsigned submask = (LW == 32) ? 0xffffffffu : (((1u << LW) - 1u) << (sub * LW));
    const int nx = P.nx, ny = P.ny, nz = P.nz;
    const int x0 = NX * lx;
    const bool act = x0 < nx;                           // this lane holds nodes of the grid
    const int x0c = act ? x0 : nx - NX;                 // lanes beyond the grid load valid memory and store nothing

    // ---- shared by the block: cos(pi x) at the two Gauss columns of each element of a lane, duplicated into both
    // halves of a pair, as float4 (ca, ca, cb, cb) at [element c][lane of the unit]
    float4* cps = reinterpret_cast<float4*>(smem);
    if constexpr (KG) {
        for (int i = threadIdx.x; i < NX * LW; i += blockDim.x) {
            const int c = i >> lwsh, l = i & (LW - 1);
            const int xe = min(NX * l, nx - NX) + c;    // element index = index of its left node
            const float ca = __ldg(P.cg[0] + 2 * xe), cb = __ldg(P.cg[0] + 2 * xe + 1);
            cps[i] = make_float4(ca, ca, cb, cb);
        }
        __syncthreads();                                // the only block-wide barrier: before the march starts
    }
    const float4* cpl = cps + lx;
    u64 cnp[NX / 2];                                    // KN: cos(pi x) at this lane's nodes, in pairs
    if constexpr (KN) {
#pragma unroll
        for (int h = 0; h < NX / 4; ++h) {
            const float4 q = __ldg(reinterpret_cast<const float4*>(P.cn[0] + x0c + 4 * h));
            cnp[2 * h] = s3_pack(q.x, q.y); cnp[2 * h + 1] = s3_pack(q.z, q.w);
        }
    }

    const long long su = ((long long)blockIdx.x * S3_WARPS + warp) * SUBS + sub;
    if (su >= G.units) return;                          // the other units of the warp synchronise among themselves only
    const int C = G.C, RS = G.RS;
    const unsigned RSB = (unsigned)RS * 4u, RINGB = (unsigned)C * RSB;
    // PREF (wide rows): the parked sums of a node row come back through shared memory, copied one step ahead of their
    // use; narrow rows load them directly (the copy cost more than it hid there: 83 against 77 us on 64^3 x 32)
    constexpr bool PREF = (NX == 8) && !EO;             // (the energy-only variant keeps the layout and leaves the row unused)
    float* ring = smem + (KG ? 4 * NX * LW : 0) + (size_t)(warp * SUBS + sub) * (C * RS + (NX == 8 ? NX * LW : 0));
    // behind the ring: one row of parked sums (each lane its own pieces)
    float* cbuf = ring + (size_t)C * RS + 4 * lx;
    const unsigned cbuf_s = (unsigned)__cvta_generic_to_shared(cbuf);
    const unsigned ring_s = (unsigned)__cvta_generic_to_shared(ring);
    const int UROW = NX * LW + 4;                       // floats of a node row in a slot (with the 4 floats of padding)
    const int FOFF = KG ? UROW : 2 * UROW;              // offset of the f row (nodal forcing)
    const int COEF = FOFF + (NF ? UROW : 0);            // offset of the coefficient row inside a slot
    const int H1 = 4 * LW + 4;                          // NX = 8: offset of the second 16 bytes of every lane

    const int b = (int)(su % P.batch);
    const int tile = (int)((su / P.batch) % G.ntile);
    const int chunk = (int)(su / ((long long)P.batch * G.ntile));
    const int y0 = tile * G.Ry, e1 = min(y0 + G.Ry, ny - 1);     // element rows y0 .. e1-1, node rows y0 .. e1
    const int T = e1 - y0 + 1;
    const bool lasttile = (e1 == ny - 1);               // then node row e1 = ny-1 is this tile's own, else the next tile's
    const int z0 = chunk * G.Z, ke = min(z0 + G.Z, nz - 1);
    const int kbeg = z0;                                // element planes z0 .. ke-1
    const int nplanes = ke - kbeg + 1;                  // node planes z0 .. ke
    const bool lastchunk = (ke == nz - 1);              // then node plane ke = nz-1 is this chunk's own, else the next chunk's

    const bool first_col = (x0 == 0), last_col = act && (x0 + NX == nx);
    const size_t plane = (size_t)nx * ny;
    const float* ub = P.u + (size_t)b * P.nodes + x0c;
    float* rb = P.r + (size_t)b * P.nodes + x0c;
    float* sb = lasttile ? nullptr : P.seam + (((size_t)b * (G.ntile - 1) + tile) * nz) * nx + x0c;
    // where the sums of node plane ke go: r, or for a chunk below another the z seam (row y0 of it; and the entry of
    // this tile's seam row among the nodes that lie on both seams)
    float* ztop = lastchunk ? rb + ((size_t)ke * ny + y0) * nx
                            : P.zseam + (((size_t)b * (G.nchunk - 1) + chunk) * ny + y0) * nx + x0c;
    float* zstop = lasttile ? nullptr
                 : lastchunk ? sb + (size_t)ke * nx
                             : P.zseam + (size_t)P.batch * (G.nchunk - 1) * ny * nx
                               + (((size_t)b * (G.nchunk - 1) + chunk) * (G.ntile - 1) + tile) * nx + x0c;

    const bool impose = (P.flags & DN_IMPOSE_BC_ON_LOAD) != 0;
    const bool nomask = (P.flags & DN_NO_MASK) != 0;
    float bc0 = P.bc_x0, bc1 = P.bc_x1;
    if (impose) {
        if (P.bc0_b) bc0 = __ldg(P.bc0_b + b);
        if (P.bc1_b) bc1 = __ldg(P.bc1_b + b);
    }
    const bool iso = ISO ? true : ((P.hx == P.hy) && (P.hy == P.hz));
    const float W8 = 0.125f * P.hx * P.hy * P.hz;
    const float kx = W8 / (P.hx * P.hx), ky = W8 / (P.hy * P.hy), kz = W8 / (P.hz * P.hz);
    const float kap = iso ? kx : 1.f;                   // isotropic cells: one scale applied at the end
    const float gs = P.gJ ? __ldg(P.gJ + b) : 1.f;
    const float fw = NF ? 0.f : P.f_const * P.hx * P.hy * P.hz;    // nodal load of an interior node (constant forcing)
    const bool hasf = !NF && (P.f_const != 0.f);
    const float fsabs = P.hx * P.hy * P.hz * (1.f / 216.f);        // NF: scale of the element mass matrix ...
    const float fs = fsabs / kap;                                   // ... in the units the corner contributions are kept in
    // Lane constants that keep the finish of a node row branch-free: output scale, share of the nodal load and
    // weight in the load energy of the lane's first / last node (Dirichlet columns: masked, or with DN_NO_MASK
    // carrying half a load); g3 = 0 in the lane whose last element lies right of node nx-1 (it does not exist).
    const float sc = gs * kap;
    const float sc0 = (first_col && !nomask) ? 0.f : sc, scL = (last_col && !nomask) ? 0.f : sc;
    const float lw0 = first_col ? (nomask ? 0.5f : 0.f) : 1.f, lwL = last_col ? (nomask ? 0.5f : 0.f) : 1.f;
    const float wx0 = first_col ? 0.5f : 1.f, wxL = last_col ? 0.5f : 1.f;
    const float g3 = last_col ? 0.f : 1.f;
    const float lm = (lx == 0) ? 0.f : 1.f;             // nothing arrives from the left in the first lane

    // ---- the ring.  Entry n = (plane index pk, row index pj) of the unit goes to slot n mod C: the node row
    // (every lane its own 16-byte pieces) and, for pk, pj >= 1, the coefficients of element row (pk-1, pj-1).
    for (int s = lx; s < C; s += LW) {                  // the 4 floats right of the last lane's nodes stay zero
        *reinterpret_cast<float4*>(ring + (size_t)s * RS + 4 * LW) = make_float4(0.f, 0.f, 0.f, 0.f);
        if constexpr (!KG) *reinterpret_cast<float4*>(ring + (size_t)s * RS + UROW + 4 * LW) = make_float4(0.f, 0.f, 0.f, 0.f);
        if constexpr (NF) *reinterpret_cast<float4*>(ring + (size_t)s * RS + FOFF + 4 * LW) = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    int pf = 0, pfj = 0, pfk = 0;
    unsigned pfo = 0;                                   // byte offset of the slot the next entry goes to
    const float* usrc = ub + (size_t)kbeg * plane + (size_t)y0 * nx;
    // coefficient piece of this lane.  KG: of element row (pfk-1, pfj-1), so the pointer starts one row and one plane
    // low; KN: of the node line of the entry itself
    const int clx = (lx < CFQ) ? lx : 0;
    const float* csrc = KG ? linepoly + (((size_t)b * (nz - 1) + kbeg) * (ny - 1) + y0) * CF - ((size_t)(ny - 1) + 1) * CF + 4 * clx
                           : linepoly + (((size_t)b * nz + kbeg) * ny + y0) * CF + 4 * clx;
    const float* nsrc = ND ? P.nu + (size_t)b * P.nodes + x0c + (size_t)kbeg * plane + (size_t)y0 * nx : nullptr;
    const float* fsrc = NF ? P.f + (size_t)b * P.nodes + x0c + (size_t)kbeg * plane + (size_t)y0 * nx : nullptr;
    const long long uwrap = (long long)plane - (long long)T * nx, cwrap = ((long long)(KG ? ny - 1 : ny) - T) * CF;
    const unsigned d0 = ring_s + 16u * lx, d1 = ring_s + 4u * H1 + 16u * lx, dc = ring_s + 4u * COEF + 16u * clx;
    auto issue = [&]() {
        if (pfk < nplanes) {                            // uniform in the unit
            s3_cp16s(d0 + pfo, usrc);
            if constexpr (NX == 8) s3_cp16s(d1 + pfo, usrc + 4);
            if constexpr (ND) {
                s3_cp16s(d0 + 4u * UROW + pfo, nsrc);
                if constexpr (NX == 8) s3_cp16s(d1 + 4u * UROW + pfo, nsrc + 4);
            }
            if constexpr (NF) {
                s3_cp16s(d0 + 4u * FOFF + pfo, fsrc);
                if constexpr (NX == 8) s3_cp16s(d1 + 4u * FOFF + pfo, fsrc + 4);
            }
            if constexpr (CF > 0) {
                const int cok = (KN || (pfk >= 1 && pfj >= 1)) ? 1 : 0;
                s3_cp16s_if(dc + pfo, csrc, (lx < CFQ) ? cok : 0);
                if constexpr (CFQ > 8) s3_cp16s_if(dc + pfo + 16u * 8u, csrc + 32, (lx + 8 < CFQ && LW == 8) ? cok : 0);
            }
        }
        s3_commit();                                    // one group per entry, possibly empty
        ++pf; ++pfj; usrc += nx; csrc += CF;
        if constexpr (ND) nsrc += nx;
        if constexpr (NF) fsrc += nx;
        if (pfj == T) {
            pfj = 0; ++pfk; usrc += uwrap; csrc += cwrap;
            if constexpr (ND) nsrc += uwrap;
            if constexpr (NF) fsrc += uwrap;
        }
        pfo += RSB;
        if (pfo == RINGB) pfo = 0;
    };
    for (int i = 0; i < C; ++i) issue();

    auto ldrow = [&](const unsigned off, float (&v)[NX + 1]) {
        const float* slot = reinterpret_cast<const float*>(reinterpret_cast<const char*>(ring) + off);
        const float4 q = *reinterpret_cast<const float4*>(slot + 4 * lx);
        v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
        if constexpr (NX == 8) {
            const float4 q1 = *reinterpret_cast<const float4*>(slot + H1 + 4 * lx);
            v[4] = q1.x; v[5] = q1.y; v[6] = q1.z; v[7] = q1.w;
        }
        v[NX] = slot[4 * (lx + 1)];                     // first node of the next lane, or the zero pad
        if (impose) {
            if (first_col) v[0] = bc0;
            if (last_col) v[NX - 1] = bc1;
        }
    };
    auto ldnu = [&](const unsigned off, float (&v)[NX + 1], const int rowoff) {      // the nu (or f) row of a slot
        const float* slot = reinterpret_cast<const float*>(reinterpret_cast<const char*>(ring) + off) + rowoff;
        const float4 q = *reinterpret_cast<const float4*>(slot + 4 * lx);
        v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
        if constexpr (NX == 8) {
            const float4 q1 = *reinterpret_cast<const float4*>(slot + H1 + 4 * lx);
            v[4] = q1.x; v[5] = q1.y; v[6] = q1.z; v[7] = q1.w;
        }
        v[NX] = slot[4 * (lx + 1)];
    };
    // KN: nu at this lane's nodes of the row in a slot, from the polynomial that came with the row, into the slot
    auto nurow = [&](const unsigned off) {
        float* slot = reinterpret_cast<float*>(reinterpret_cast<char*>(ring) + off);
        u64 gg[GS / 2];
        const ulonglong2* gp = reinterpret_cast<const ulonglong2*>(slot + COEF);
#pragma unroll
        for (int i = 0; i < GS / 4; ++i) { const ulonglong2 t = gp[i]; gg[2 * i] = t.x; gg[2 * i + 1] = t.y; }
        float nn[NX];
#pragma unroll
        for (int h = 0; h < NX / 2; ++h) {
            u64 e = gg[M];
#pragma unroll
            for (int i = M - 1; i >= 0; --i) e = s3_fma2(e, cnp[h], gg[i]);
            float e0, e1;
            s3_unpack(e, e0, e1);
            nn[2 * h] = s3_ex2(e0); nn[2 * h + 1] = s3_ex2(e1);
        }
        *reinterpret_cast<float4*>(slot + UROW + 4 * lx) = make_float4(nn[0], nn[1], nn[2], nn[3]);
        if constexpr (NX == 8) *reinterpret_cast<float4*>(slot + UROW + H1 + 4 * lx) = make_float4(nn[4], nn[5], nn[6], nn[7]);
    };
    // parked partial sums of one node row (plain loads: this thread wrote them one plane ago)
    auto ld4 = [&](const float* p, float (&v)[NX]) {
#pragma unroll
        for (int h = 0; h < NX / 4; ++h) {
            const float4 q = *reinterpret_cast<const float4*>(p + 4 * h);
            v[4 * h] = q.x; v[4 * h + 1] = q.y; v[4 * h + 2] = q.z; v[4 * h + 3] = q.w;
        }
    };
    auto st4 = [&](float* p, const float (&v)[NX]) {
#pragma unroll
        for (int h = 0; h < NX / 4; ++h)
            *reinterpret_cast<float4*>(p + 4 * h) = make_float4(v[4 * h], v[4 * h + 1], v[4 * h + 2], v[4 * h + 3]);
    };
    auto wrapb = [&](unsigned o) { return o >= RINGB ? o - RINGB : o; };

    float pendL1[NX], pendU1[NX];                       // what the element row below left for the current node row
    double end = 0.0, eld = 0.0;
    unsigned oA = 0;                                    // slot (byte offset) of the lower-plane, lower row of the current element row
    int n = 0;                                          // ... and its entry index
    const unsigned TB = (unsigned)T * RSB;
    for (int kk = 0; kk + 1 < nplanes; ++kk) {
        const int k = kbeg + kk;                        // element plane k lies between node planes k and k + 1: plane k is
        const bool hascarry = !EO && (kk > 0) && act;   // finished now, with the partial sums parked one step before;
        const bool last = (k + 1 == ke);                // the sums of plane k + 1 are parked (plane ke: finished after the march)
        const float wzlo = (k == 0) ? 0.5f : 1.f;
        const float nllo = -gs * fw * wzlo;
        float enlo = 0.f, ello = 0.f, elnf = 0.f;
#pragma unroll
        for (int c = 0; c < NX; ++c) { pendL1[c] = 0.f; pendU1[c] = 0.f; }
        float* rlo = rb + ((size_t)k * ny + y0) * nx;
        float* rup = last ? ztop : rlo + plane;
        float* ptoplo = lasttile ? rlo + (size_t)(T - 1) * nx : sb + (size_t)k * nx;   // where the tile's top row is finished
        // The sums parked for a node row one plane ago come back through shared memory, copied one step ahead (this
        // thread stored them long ago; the copy reads them from L2 while the elements of the row before are computed).
        auto fetch_parked = [&](const float* p) {
            s3_cp16s(cbuf_s, p);
            if constexpr (NX == 8) s3_cp16s(cbuf_s + 16u * LW, p + 4);
            s3_commit();
        };
        auto read_parked = [&](float (&v)[NX]) {
            const float4 q = *reinterpret_cast<const float4*>(cbuf);
            v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
            if constexpr (NX == 8) {
                const float4 q1 = *reinterpret_cast<const float4*>(cbuf + 4 * LW);
                v[4] = q1.x; v[5] = q1.y; v[6] = q1.z; v[7] = q1.w;
            }
        };
        if (PREF && hascarry) fetch_parked(rlo);
        for (int jj = 0; jj + 1 < T; ++jj) {
            s3_wait<0>();                               // everything issued up to the previous step has landed ...
            __syncwarp(submask);                        // ... is visible to the unit, and the rows it retired are free
            float cin[NX];
#pragma unroll
            for (int c = 0; c < NX; ++c) cin[c] = 0.f;
            if (hascarry) {
                if constexpr (PREF) {
                    read_parked(cin);
                    fetch_parked((jj + 2 < T) ? rlo + nx : ptoplo);
                } else {
                    ld4(rlo, cin);
                }
            }
            while (pf < n + C) issue();
            const unsigned oB = wrapb(oA + RSB), oC = wrapb(oA + TB), oD = wrapb(oC + RSB);
            const float wy = (y0 + jj == 0) ? 0.5f : 1.f;
            float uA[NX + 1], uB[NX + 1], uC[NX + 1], uD[NX + 1];
            ldrow(oA, uA); ldrow(oB, uB); ldrow(oC, uC); ldrow(oD, uD);
            u64 ga[GS / 2], gb[GS / 2];                 // Gauss row q = a / b; each entry holds (plane s = a, s = b)
            float nA[NX + 1], nB[NX + 1], nC[NX + 1], nD[NX + 1];      // nodal modes: nu on the four node rows
            float yA[NX + 1], yC[NX + 1], zA[NX + 1], zB[NX + 1];      // ... summed over the rows of a plane / the planes of a row
            if constexpr (KN) {
                // rows meet the march at its upper, far corner: a row is new when it is D, and also when it is B in the
                // unit's first plane, C in a plane's first row, A at the very start
                if (kk == 0 && jj == 0) nurow(oA);
                if (kk == 0) nurow(oB);
                if (jj == 0) nurow(oC);
                nurow(oD);
                __syncwarp(submask);                    // the node right of a lane's last is the next lane's
            }
            if constexpr (!KG) {
                ldnu(oA, nA, UROW); ldnu(oB, nB, UROW); ldnu(oC, nC, UROW); ldnu(oD, nD, UROW);
#pragma unroll
                for (int c = 0; c <= NX; ++c) {
                    yA[c] = nA[c] + nB[c]; yC[c] = nC[c] + nD[c];
                    zA[c] = nA[c] + nC[c]; zB[c] = nB[c] + nD[c];
                }
            }
            float fA[NX + 1], fB[NX + 1], fC[NX + 1], fD[NX + 1];      // nodal forcing on the four node rows
            if constexpr (NF) { ldnu(oA, fA, FOFF); ldnu(oB, fB, FOFF); ldnu(oC, fC, FOFF); ldnu(oD, fD, FOFF); }
            if constexpr (KG) {
                const ulonglong2* gp = reinterpret_cast<const ulonglong2*>(reinterpret_cast<const char*>(ring) + oD) + COEF / 4;
#pragma unroll
                for (int i = 0; i < GS / 4; ++i) {
                    const ulonglong2 t0 = gp[i], t1 = gp[GS / 4 + i];
                    ga[2 * i] = t0.x; ga[2 * i + 1] = t0.y; gb[2 * i] = t1.x; gb[2 * i + 1] = t1.y;
                }
            }
            const float nlrow = nllo * wy;
            float olo[NX], oup[NX];
            // Finish of node column c of this row on both planes: `lo` / `up` are everything the lane's elements of this
            // row contribute to node (c, j, k) / (c, j, k+1), `lo1` / `up1` what they leave for row j + 1.
            auto node = [&](const int c, const float lo, const float lo1, const float up, const float up1) {
                const float raw = (lo + pendL1[c]) + cin[c];
                oup[c] = up + pendU1[c];
                pendL1[c] = lo1; pendU1[c] = up1;
                enlo = fmaf(uA[c], raw, enlo);
                const float s = (c == 0) ? sc0 : (c == NX - 1) ? scL : sc;
                const float l = (c == 0) ? lw0 * nlrow : (c == NX - 1) ? lwL * nlrow : nlrow;
                olo[c] = fmaf(s, raw, l);
            };
            // ---- the NX elements of this lane, from right to left: element c completes node column c + 1
            float q000 = 0.f, q010 = 0.f, q001 = 0.f, q011 = 0.f;   // own-corner contributions of the element on the right
            float a100 = 0.f, a110 = 0.f, a101 = 0.f, a111 = 0.f;   // from the last element of the lane on the left
#pragma unroll
            for (int c = NX - 1; c >= 0; --c) {
                const float eA = uA[c + 1] - uA[c], eB = uB[c + 1] - uB[c];
                const float eC = uC[c + 1] - uC[c], eD = uD[c + 1] - uD[c];
                const float slo = uB[c] - uA[c], sup = uD[c] - uC[c], w0 = uC[c] - uA[c];
                const float txy = eB - eA, txyu = eD - eC, txz = eC - eA, tyz = sup - slo, txyz = txyu - txy;
                float Nx[4], Ny[4], Nz[4], r[8];
                (void)r;
                if constexpr (KG) {
                    float nu[8];
                    const ulonglong2 cc = *reinterpret_cast<const ulonglong2*>(cpl + c * LW);
                    s3_nu_gauss<M>(ga, gb, cc.x, cc.y, nu);
                    s3_sums_gauss(nu, Nx, Ny, Nz);
                } else {
                    s3_bilerp(nA[c] + nA[c + 1], nB[c] + nB[c + 1], nC[c] + nC[c + 1], nD[c] + nD[c + 1], Nx);   // (q, s)
                    s3_bilerp(yA[c], yA[c + 1], yC[c], yC[c + 1], Ny);                                           // (p, s)
                    s3_bilerp(zA[c], zA[c + 1], zB[c], zB[c + 1], Nz);                                           // (p, q)
                }
                if constexpr (EO) {
                    const float e = s3_energy(Nx, Ny, Nz, eA, slo, w0, txy, txz, tyz, txyz, iso, kx, ky, kz);
                    enlo += (c == NX - 1) ? e * g3 : e;
                    if constexpr (NF) {
                        const float fc[8] = {fA[c], fA[c + 1], fB[c], fB[c + 1], fC[c], fC[c + 1], fD[c], fD[c + 1]};
                        const float uc[8] = {uA[c], uA[c + 1], uB[c], uB[c + 1], uC[c], uC[c + 1], uD[c], uD[c + 1]};
                        float m[8], ef = 0.f;
                        s3_mass(fc, m);
#pragma unroll
                        for (int t = 0; t < 8; ++t) ef = fmaf(uc[t], m[t], ef);
                        elnf += (c == NX - 1) ? ef * g3 : ef;
                    }
                    continue;
                }
                s3_element(Nx, Ny, Nz, eA, slo, w0, txy, txz, tyz, txyz, iso, kx, ky, kz, r);
                if constexpr (NF) {
                    const float fc[8] = {fA[c], fA[c + 1], fB[c], fB[c + 1], fC[c], fC[c + 1], fD[c], fD[c + 1]};
                    const float uc[8] = {uA[c], uA[c + 1], uB[c], uB[c + 1], uC[c], uC[c + 1], uD[c], uD[c + 1]};
                    float m[8], e = 0.f;
                    s3_mass(fc, m);
#pragma unroll
                    for (int t = 0; t < 8; ++t) { r[t] = fmaf(-fs, m[t], r[t]); e = fmaf(uc[t], m[t], e); }
                    elnf += (c == NX - 1) ? e * g3 : e;
                }
                if (c == NX - 1) {
                    // the lane's last element: its right-hand corners belong to the next lane; in the lane that ends the
                    // row it does not exist (g3 = 0)
                    a100 = __shfl_up_sync(submask, r[1], 1, LW); a110 = __shfl_up_sync(submask, r[3], 1, LW);
                    a101 = __shfl_up_sync(submask, r[5], 1, LW); a111 = __shfl_up_sync(submask, r[7], 1, LW);
                    q000 = r[0] * g3; q010 = r[2] * g3; q001 = r[4] * g3; q011 = r[6] * g3;
                } else {
                    node(c + 1, q000 + r[1], q010 + r[3], q001 + r[5], q011 + r[7]);
                    q000 = r[0]; q010 = r[2]; q001 = r[4]; q011 = r[6];
                }
            }
            if constexpr (!EO) node(0, fmaf(a100, lm, q000), fmaf(a110, lm, q010), fmaf(a101, lm, q001), fmaf(a111, lm, q011));
            if (hasf) {
                float a = wx0 * uA[0];
#pragma unroll
                for (int c = 1; c < NX - 1; ++c) a += uA[c];
                ello = fmaf(wy, fmaf(wxL, uA[NX - 1], a), ello);
            }
            if constexpr (!EO) { if (act) { st4(rlo, olo); st4(rup, oup); } }
            rlo += nx; rup += nx;
            oA = oB; ++n;
        }
        // ---- the top node row e1 of the tile gets nothing more in this plane.  It is this tile's own if it is the
        // top of the domain; else it belongs to the next tile and its sums go to the seam array (no load term: the
        // owner adds it).
        {
            float uA[NX + 1];
            ldrow(oA, uA);
            float* plo = ptoplo;
            float* pup = lasttile ? rup : last ? zstop : plo + nx;
            const float wy = lasttile ? 0.5f : 0.f;
            const float nlrow = nllo * wy;
            float cin[NX], olo[NX];
#pragma unroll
            for (int c = 0; c < NX; ++c) cin[c] = 0.f;
            if (hascarry) {
                if constexpr (PREF) {
                    s3_wait<0>();
                    read_parked(cin);
                } else {
                    ld4(plo, cin);
                }
            }
            if constexpr (!EO) {
#pragma unroll
                for (int c = 0; c < NX; ++c) {
                    const float raw = pendL1[c] + cin[c];
                    enlo = fmaf(uA[c], raw, enlo);
                    const float s = (c == 0) ? sc0 : (c == NX - 1) ? scL : sc;
                    const float l = (c == 0) ? lw0 * nlrow : (c == NX - 1) ? lwL * nlrow : nlrow;
                    olo[c] = fmaf(s, raw, l);
                }
            }
            if (hasf) {
                float a = wx0 * uA[0];
#pragma unroll
                for (int c = 1; c < NX - 1; ++c) a += uA[c];
                ello = fmaf(wy, fmaf(wxL, uA[NX - 1], a), ello);
            }
            if constexpr (!EO) { if (act) { st4(plo, olo); st4(pup, pendU1); } }
            oA = wrapb(oA + RSB); ++n;
        }
        end += (double)enlo; eld += NF ? (double)elnf : (double)(wzlo * ello);   // per-plane sums go to double
    }
    s3_wait<0>();

    // ---- node plane ke gets nothing more from this chunk: what was parked for it is complete as far as this chunk
    // goes.  Top of the domain: finished into r with its load.  Else the plane is the next chunk's: the scaled, masked
    // sums stay in the z seam (no load term: the owner adds it).  Its rows are still in the ring (entry n is row 0).
    {
        float entop = 0.f, eltop = 0.f;
        const float lf = lastchunk ? 1.f : 0.f;
        float* ptop = ztop;
        for (int jj = 0; jj < T; ++jj) {
            const bool seamrow = (jj == T - 1) && !lasttile;
            float* p = seamrow ? zstop : ptop;
            const int j = y0 + jj;
            const float wy = seamrow ? 0.f : (j == 0 || j == ny - 1) ? 0.5f * lf : lf;
            const float nlrow = -gs * fw * 0.5f * wy;
            float part[NX], uT[NX + 1], o[NX];
#pragma unroll
            for (int c = 0; c < NX; ++c) part[c] = 0.f;
            if constexpr (!EO) { if (act) ld4(p, part); }
            ldrow(oA, uT);
#pragma unroll
            for (int c = 0; c < NX; ++c) {
                entop = fmaf(uT[c], part[c], entop);
                const float s = (c == 0) ? sc0 : (c == NX - 1) ? scL : sc;
                const float l = (c == 0) ? lw0 * nlrow : (c == NX - 1) ? lwL * nlrow : nlrow;
                o[c] = fmaf(s, part[c], l);
            }
            float a = wx0 * uT[0];
#pragma unroll
            for (int c = 1; c < NX - 1; ++c) a += uT[c];
            eltop = fmaf(wy, fmaf(wxL, uT[NX - 1], a), eltop);
            if constexpr (!EO) { if (act) st4(p, o); }
            ptop += nx;
            oA = wrapb(oA + RSB);
        }
        end += (double)entop;
        if constexpr (!NF) eld += (double)(0.5f * eltop);
    }

    // ---- energy partial of this unit: its lanes summed in a fixed order in double
    // NF: `end` holds sum u (K u - F) in units of kap and `eld` sum u_corner (M_e f_e)_corner, so that
    // the load part is fsabs * eld and the diffusion part half of (kap * end + load part)
    // (energy only: `end` is sum u K u itself, with or without nodal forcing)
    double l = !act ? 0.0 : NF ? (double)fsabs * eld : hasf ? (double)fw * eld : 0.0;
    double d = !act ? 0.0 : (NF && !EO) ? 0.5 * ((double)kap * end + l) : 0.5 * (double)kap * end;
    for (int off = LW >> 1; off > 0; off >>= 1) {
        d += __shfl_down_sync(submask, d, off, LW);
        l += __shfl_down_sync(submask, l, off, LW);
    }
    if (lx == 0) {
        double* slot = P.partials + 2 * ((size_t)b * P.nblk + (size_t)chunk * G.ntile + tile);
        slot[0] = d; slot[1] = l;
    }
}

// ---------------------------------------------------------------------------------------------------------
// Coefficient table: for element row ey of element plane ez of sample b, the polynomials (in c = cos(pi x)) of
// the KL exponent along the four Gauss lines (y_q, z_s):  sum_i g_i T_i(c)  with
// g_i = sum_{j,k} ckl[i][j][k] cos(j pi y_q) cos(k pi z_s), converted from the Chebyshev basis to monomials in
// double.  The scaled weights and the cosines are the float tables every kernel family reads.  One block per
// (sample, element plane, 128 element rows); a thread writes the four lines of its element row.
// ---------------------------------------------------------------------------------------------------------
template <int M>
__global__ void __launch_bounds__(128) linepoly3d_kernel(const Params P, float* __restrict__ out) {
    constexpr int GS = s3_gs(M);
    __shared__ double h[2][M][M];                       // h[s][i][j] = sum_k ckl[i][j][k] cos(k pi z_s)
    dep_wait();                                         // the scaled weights and cosine tables are complete
    dep_release();
    const int ez = blockIdx.y, b = blockIdx.z;
    const float* w = P.ckl + (size_t)b * M * M * M;
    for (int t = threadIdx.x; t < 2 * M * M; t += blockDim.x) {
        const int s = t / (M * M), ij = t % (M * M);
        const float* cz = P.cg[2] + 2 * ez + s;
        double acc = 0.0;
#pragma unroll
        for (int k = 0; k < M; ++k) acc += (double)w[ij * M + k] * (double)cz[(size_t)k * P.gstride[2]];
        h[s][ij / M][ij % M] = acc;
    }
    __syncthreads();
    const int ey = blockIdx.x * blockDim.x + threadIdx.x;
    if (ey >= P.ny - 1) return;
    float row[2 * GS];
#pragma unroll
    for (int i = 0; i < 2 * GS; ++i) row[i] = 0.f;      // the padding of a Gauss row stays zero
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        double cy[M];
#pragma unroll
        for (int j = 0; j < M; ++j) cy[j] = (double)P.cg[1][(size_t)j * P.gstride[1] + 2 * ey + q];
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            // sum_i g_i T_i(c) in the monomial basis, T_{i+1} = 2 c T_i - T_{i-1}
            double acc[M + 1], tp[M + 1], tc[M + 1];
#pragma unroll
            for (int k = 0; k <= M; ++k) { acc[k] = 0.0; tp[k] = (k == 0) ? 1.0 : 0.0; tc[k] = (k == 1) ? 1.0 : 0.0; }
#pragma unroll
            for (int i = 1; i <= M; ++i) {
                double g = 0.0;
#pragma unroll
                for (int j = 0; j < M; ++j) g += h[s][i - 1][j] * cy[j];
#pragma unroll
                for (int k = 0; k <= i; ++k) acc[k] += g * tc[k];
                double tn[M + 1];
#pragma unroll
                for (int k = 0; k <= M; ++k) tn[k] = ((k > 0) ? 2.0 * tc[k - 1] : 0.0) - tp[k];
#pragma unroll
                for (int k = 0; k <= M; ++k) { tp[k] = tc[k]; tc[k] = tn[k]; }
            }
#pragma unroll
            for (int k = 0; k <= M; ++k) row[q * GS + 2 * k + s] = (float)acc[k];
        }
    }
    float4* dst = reinterpret_cast<float4*>(out + (((size_t)b * (P.nz - 1) + ez) * (P.ny - 1) + ey) * (2 * GS));
#pragma unroll
    for (int i = 0; i < GS / 2; ++i) dst[i] = make_float4(row[4 * i], row[4 * i + 1], row[4 * i + 2], row[4 * i + 3]);
}

// KL at the nodes: the polynomial (in c = cos(pi x)) of the KL exponent along every node line (y_j, z_k), every
// coefficient twice so that two nodes share a packed FMA: [B][nz][ny][GS] floats.  One block per (sample, node plane,
// 128 node rows).
template <int M>
__global__ void __launch_bounds__(128) nodepoly3d_kernel(const Params P, float* __restrict__ out) {
    constexpr int GS = s3_gs(M);
    __shared__ double h[M][M];                          // h[i][j] = sum_k ckl[i][j][k] cos(k pi z)
    dep_wait();                                         // the scaled weights and cosine tables are complete
    dep_release();
    const int iz = blockIdx.y, b = blockIdx.z;
    const float* w = P.ckl + (size_t)b * M * M * M;
    for (int t = threadIdx.x; t < M * M; t += blockDim.x) {
        double acc = 0.0;
#pragma unroll
        for (int k = 0; k < M; ++k) acc += (double)w[t * M + k] * (double)P.cn[2][(size_t)k * P.nstride[2] + iz];
        h[t / M][t % M] = acc;
    }
    __syncthreads();
    const int iy = blockIdx.x * blockDim.x + threadIdx.x;
    if (iy >= P.ny) return;
    double cy[M];
#pragma unroll
    for (int j = 0; j < M; ++j) cy[j] = (double)P.cn[1][(size_t)j * P.nstride[1] + iy];
    double acc[M + 1], tp[M + 1], tc[M + 1];
#pragma unroll
    for (int k = 0; k <= M; ++k) { acc[k] = 0.0; tp[k] = (k == 0) ? 1.0 : 0.0; tc[k] = (k == 1) ? 1.0 : 0.0; }
#pragma unroll
    for (int i = 1; i <= M; ++i) {
        double g = 0.0;
#pragma unroll
        for (int j = 0; j < M; ++j) g += h[i - 1][j] * cy[j];
#pragma unroll
        for (int k = 0; k <= i; ++k) acc[k] += g * tc[k];
        double tn[M + 1];
#pragma unroll
        for (int k = 0; k <= M; ++k) tn[k] = ((k > 0) ? 2.0 * tc[k - 1] : 0.0) - tp[k];
#pragma unroll
        for (int k = 0; k <= M; ++k) { tp[k] = tc[k]; tc[k] = tn[k]; }
    }
    float row[GS];
#pragma unroll
    for (int i = 0; i < GS; ++i) row[i] = 0.f;
#pragma unroll
    for (int k = 0; k <= M; ++k) { row[2 * k] = (float)acc[k]; row[2 * k + 1] = (float)acc[k]; }
    float4* dst = reinterpret_cast<float4*>(out + (((size_t)b * P.nz + iz) * P.ny + iy) * GS);
#pragma unroll
    for (int i = 0; i < GS / 4; ++i) dst[i] = make_float4(row[4 * i], row[4 * i + 1], row[4 * i + 2], row[4 * i + 3]);
}

// Adds the seam contributions to r (fixed order per node: own sums, tile seam, chunk seam, the entry for nodes on both).
// First range of threads: the nodes of the tile seam rows (t + 1) Ry on every plane; second range: the nodes of the
// chunk seam planes (c + 1) Z that are not on a tile seam row.  The two ranges touch different nodes.
__global__ void seam_fixup3_kernel(float* __restrict__ r, const float* __restrict__ yseam, const float* __restrict__ zseam,
                                   int nx, int ny, int nz, int batch, int Ry, int ntile, int Z, int nchunk,
                                   long long nA, long long nB) {
    dep_wait();                                         // the fused kernel has finished
    dep_release();
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int nx4 = nx / 4;
    const float4* zy = reinterpret_cast<const float4*>(zseam + (size_t)batch * (nchunk - 1) * ny * nx);
    if (i < nA) {
        const int x4 = (int)(i % nx4);
        long long t = i / nx4;
        const int k = (int)(t % nz); t /= nz;
        const int sm = (int)(t % (ntile - 1));
        const int b = (int)(t / (ntile - 1));
        const int j = (sm + 1) * Ry;
        float4* dst = reinterpret_cast<float4*>(r + (((size_t)b * nz + k) * ny + j) * nx) + x4;
        float4 v = *dst;
        const float4 a = __ldg(reinterpret_cast<const float4*>(yseam) + i);
        v.x += a.x; v.y += a.y; v.z += a.z; v.w += a.w;
        if (k % Z == 0 && k > 0 && k < nz - 1) {        // also the first plane of a chunk
            const int c = k / Z - 1;
            const float4 z = __ldg(reinterpret_cast<const float4*>(zseam + (((size_t)b * (nchunk - 1) + c) * ny + j) * nx) + x4);
            v.x += z.x; v.y += z.y; v.z += z.z; v.w += z.w;
            const float4 w = __ldg(zy + (((size_t)b * (nchunk - 1) + c) * (ntile - 1) + sm) * nx4 + x4);
            v.x += w.x; v.y += w.y; v.z += w.z; v.w += w.w;
        }
        *dst = v;
    } else if (i < nA + nB) {
        const long long q = i - nA;
        const int x4 = (int)(q % nx4);
        long long t = q / nx4;
        const int j = (int)(t % ny); t /= ny;
        const int c = (int)(t % (nchunk - 1));
        const int b = (int)(t / (nchunk - 1));
        if (j % Ry == 0 && j > 0 && j < ny - 1) return;  // a tile seam row: done by the first range
        const int k = (c + 1) * Z;
        float4* dst = reinterpret_cast<float4*>(r + (((size_t)b * nz + k) * ny + j) * nx) + x4;
        float4 v = *dst;
        const float4 z = __ldg(reinterpret_cast<const float4*>(zseam) + q);
        v.x += z.x; v.y += z.y; v.z += z.z; v.w += z.w;
        *dst = v;
    }
}

int s3_sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
        (void)cudaGetLastError();
        n = 148;
    }
    return n;
}

constexpr size_t S3_SMEM_SM = 233472;              // shared memory of an SM; a block also reserves 1 KiB
constexpr size_t S3_SMEM_BLOCK = 232448;           // most a block can ask for

// Nodes per lane: 8 on rows of more than 128 nodes; also on rows of 65 to 128 nodes (two units per warp) with KL at the
// Gauss points and constant forcing, where it is 8 to 9 % faster than 4 (128^3 x 16: 263 against 290 us; with KL at the
// nodes or a stored field it is not: 314 against 306, 288 against 284 us); on narrower rows 4 (64^3 x 32: 79 against 89 us).
int s3_nxl(int nx, int mode, bool nf) {
    if (nx > 128) return 8;
    return (nx > 64 && nx % 8 == 0 && mode == DN_NU_KL_GAUSS && !nf) ? 8 : 4;
}
// resident blocks of 4 warps per SM the kernel is compiled for: the nodal modes keep two rows per slot and trade
// warps for taller tiles on wide rows
int s3_minb(int nxl, int mode, bool nf) { return (nxl == 8) ? ((mode == DN_NU_KL_GAUSS && !nf) ? 3 : 2) : 4; }
int s3_slot_floats(int nxl, int lw, int mode, int m, bool nf) {
    const int urow = nxl * lw + 4;
    const int rows = (mode == DN_NU_KL_GAUSS ? 1 : 2) + (nf ? 1 : 0);
    return rows * urow + (mode == DN_NU_KL_GAUSS ? 2 * s3_gs(m) : mode == DN_NU_KL_NODAL ? s3_gs(m) : 0);
}

S3Geo geometry3s_search(const dn_problem& p) {
    S3Geo g{};
    const int nx = p.grid.nx, ny = p.grid.ny, nz = p.grid.nz;
    const int NX = s3_nxl(nx, p.nu_mode, p.f != nullptr), minb = s3_minb(NX, p.nu_mode, p.f != nullptr);
    g.LW = 8; g.lwsh = 3;
    while (g.LW * NX < nx) { g.LW *= 2; ++g.lwsh; }
    const int subs = 32 / g.LW;
    g.RS = s3_slot_floats(NX, g.LW, p.nu_mode, p.kl_modes, p.f != nullptr);
    size_t per_block = (S3_SMEM_SM - (size_t)minb * 1024) / minb;
    if (per_block > S3_SMEM_BLOCK) per_block = S3_SMEM_BLOCK;
    if (p.nu_mode == DN_NU_KL_GAUSS) per_block -= sizeof(float) * 4 * NX * g.LW;      // the block's table of cosine pairs
    if (NX == 8) per_block -= sizeof(float) * S3_WARPS * subs * NX * g.LW;   // one row of parked sums per unit
    const int cmax = (int)(per_block / ((size_t)S3_WARPS * subs * g.RS * sizeof(float)));
    int ry_max = cmax - 2 - S3_D;
    if (ry_max > ny - 1) ry_max = ny - 1;
    if (ry_max > 64) ry_max = 64;
    if (ry_max < 1) ry_max = 1;
    const long long slots = (long long)s3_sm_count() * minb * S3_WARPS * subs;
    // (Ry, Z) by a cost model: whole waves of units; a unit pays, per plane, the finish of its top row, and once the
    // filling of its ring and the finish of its last plane; flat tiles and short chunks also pay seam traffic.
    double best = -1.0;
    for (int Ry = 1; Ry <= ry_max; ++Ry) {
        const long long ntile = (ny - 1 + Ry - 1) / Ry;
        for (int Z = 1; Z <= nz - 1; ++Z) {
            const long long nchunk = (nz - 1 + Z - 1) / Z;
            const long long units = (long long)p.batch * ntile * nchunk;
            const long long waves = (units + slots - 1) / slots;
            const double cost = (double)waves * (Z * (Ry + 0.5) + 0.4 * Ry + 3.0) * (1.0 + 0.15 / Ry + 0.15 / Z);
            if (best < 0 || cost < best * (1.0 - 1e-9)) {
                best = cost;
                g.Ry = Ry; g.Z = Z; g.ntile = (int)ntile; g.nchunk = (int)nchunk; g.units = units;
            }
        }
    }
    g.C = g.Ry + 2 + S3_D;
    return g;
}

S3Geo geometry3s(const dn_problem& p) {
    return memo_geometry<S3Geo>(p, s3_sm_count(), [&]() { return geometry3s_search(p); });
}

template <int NX, int M, int MODE, bool NF, int MINB, bool EO, int LWC, bool ISO>
cudaError_t launch_nmfei(const Params& P, const float* linepoly, const S3Geo& g, cudaStream_t s) {
    const int subs = 32 / g.LW;
    const size_t smem = sizeof(float) * ((size_t)S3_WARPS * subs * (g.C * g.RS + (NX == 8 ? NX * g.LW : 0)) + (MODE == 0 ? 4 * NX * g.LW : 0));
    const long long per_block = (long long)S3_WARPS * subs;
    const unsigned blocks = (unsigned)((g.units + per_block - 1) / per_block);
    const cudaError_t e = cudaFuncSetAttribute(strip3d_kernel<NX, M, MODE, NF, MINB, EO, LWC, ISO>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return launch_dependent(strip3d_kernel<NX, M, MODE, NF, MINB, EO, LWC, ISO>, dim3(blocks), dim3(S3_WARPS * 32), smem, s, P, linepoly, g);
}

// cubic cells on wide rows with constant forcing: the variant compiled for them
template <int NX, int M, int MODE, bool NF, int MINB, bool EO, int LWC>
cudaError_t launch_nmfe(const Params& P, const float* linepoly, const S3Geo& g, cudaStream_t s) {
    if constexpr (NX == 8 && LWC == 32 && !NF) {
        if (P.hx == P.hy && P.hy == P.hz) return launch_nmfei<NX, M, MODE, NF, MINB, EO, LWC, true>(P, linepoly, g, s);
    }
    return launch_nmfei<NX, M, MODE, NF, MINB, EO, LWC, false>(P, linepoly, g, s);
}

// no output array: the energy-only variant
template <int NX, int M, int MODE, bool NF, int MINB, int LWC = (NX == 8 ? 32 : 0)>
cudaError_t launch_nmf(const Params& P, const float* linepoly, const S3Geo& g, cudaStream_t s) {
    return P.r ? launch_nmfe<NX, M, MODE, NF, MINB, false, LWC>(P, linepoly, g, s)
               : launch_nmfe<NX, M, MODE, NF, MINB, true, LWC>(P, linepoly, g, s);
}

// MINB: blocks per SM without nodal forcing; with it, wide rows run two blocks per SM in every mode (s3_minb)
template <int NX, int M, int MODE, int MINB>
cudaError_t launch_nm(const Params& P, const float* linepoly, const S3Geo& g, cudaStream_t s) {
    if (P.f) return launch_nmf<NX, M, MODE, true, (NX == 8 ? 2 : 4)>(P, linepoly, g, s);
    if constexpr (NX == 4) {                            // 16 or 32 lanes per unit known to the compiler: 3 to 4 % (64^3 x 32: 78.8 -> 76.2 us)
        if (g.LW == 16) return launch_nmf<NX, M, MODE, false, MINB, 16>(P, linepoly, g, s);
        if (g.LW == 32) return launch_nmf<NX, M, MODE, false, MINB, 32>(P, linepoly, g, s);
    }
    return launch_nmf<NX, M, MODE, false, MINB>(P, linepoly, g, s);
}

template <int M>
cudaError_t launch_m3(const Params& P, const float* linepoly, const S3Geo& g, cudaStream_t s) {
    const bool wide = (s3_nxl(P.nx, P.nu_mode, P.f != nullptr) == 8);
    if (P.nu_mode == DN_NU_KL_NODAL)
        return wide ? launch_nm<8, M, 1, 2>(P, linepoly, g, s) : launch_nm<4, M, 1, 4>(P, linepoly, g, s);
    if (wide && P.nx <= 128) return launch_nmf<8, M, 0, false, 3, 16>(P, linepoly, g, s);      // two units per warp
    return wide ? launch_nm<8, M, 0, 3>(P, linepoly, g, s) : launch_nm<4, M, 0, 4>(P, linepoly, g, s);
}

dn_problem s3_problem_of(const Params& P) {
    dn_problem p{};
    p.grid.dim = 3; p.grid.nx = P.nx; p.grid.ny = P.ny; p.grid.nz = P.nz; p.batch = P.batch;
    p.nu_mode = P.nu_mode; p.kl_modes = P.m; p.f = P.f;
    return p;
}

}  // namespace

#if DN_S3_PART == 1
cudaError_t launch_strip3d_hi(const Params& P, const float* linepoly, const S3Geo& g, cudaStream_t s) {
    switch (P.m) {
        case 5: return launch_m3<5>(P, linepoly, g, s);
        case 6: return launch_m3<6>(P, linepoly, g, s);
        case 7: return launch_m3<7>(P, linepoly, g, s);
        case 8: return launch_m3<8>(P, linepoly, g, s);
    }
    return cudaErrorInvalidValue;
}
#else

// Rows of at most 128 nodes take 4 nodes per lane, rows of at most 256 nodes 8 (then nx must be a multiple of 8,
// so that only the last element of the last lane falls outside the grid).
bool strip3d_applicable(const dn_problem& p) {
    if (!(p.grid.dim == 3 && p.grid.nx % 4 == 0 && p.grid.nx >= 8 &&
          p.grid.nx <= 256 && p.grid.ny >= 2 && p.grid.nz >= 2))
        return false;
    return p.grid.nx <= 128 || p.grid.nx % 8 == 0;
}

Launch strip3d_geometry(const dn_problem& p) {
    const S3Geo g = geometry3s(p);
    Launch l{};
    l.path = PATH_STRIP3D;
    l.nblk = g.ntile * g.nchunk;
    l.chunk = g.Z;
    l.variant = g.Ry;
    return l;
}

size_t strip3d_seam_floats(const dn_problem& p) {
    if (!strip3d_applicable(p)) return 0;
    const S3Geo g = geometry3s(p);
    return (size_t)p.batch * (g.ntile - 1) * p.grid.nz * p.grid.nx;
}

// the chunk seams: [B][nchunk-1][ny][nx], then [B][nchunk-1][ntile-1][nx] for the nodes on a tile seam as well
size_t strip3d_zseam_floats(const dn_problem& p) {
    if (!strip3d_applicable(p)) return 0;
    const S3Geo g = geometry3s(p);
    return (size_t)p.batch * (g.nchunk - 1) * ((size_t)p.grid.ny + (g.ntile - 1)) * p.grid.nx;
}

// the coefficient table: per element row its four Gauss lines (KL at the Gauss points), or per node line (KL at the nodes)
size_t strip3d_linepoly_floats(const dn_problem& p) {
    if (!strip3d_applicable(p) || p.nu_mode == DN_NU_NODAL) return 0;
    if (p.nu_mode == DN_NU_KL_NODAL) return (size_t)p.batch * p.grid.nz * p.grid.ny * s3_gs(p.kl_modes);
    return (size_t)p.batch * (p.grid.nz - 1) * (p.grid.ny - 1) * 2 * s3_gs(p.kl_modes);
}

template <int M>
static cudaError_t launch_linepoly3d_m(const Params& P, float* linepoly, cudaStream_t s) {
    if (P.nu_mode == DN_NU_KL_NODAL) {
        const dim3 grid((unsigned)((P.ny + 127) / 128), (unsigned)P.nz, (unsigned)P.batch);
        return launch_dependent(nodepoly3d_kernel<M>, grid, dim3(128), 0, s, P, linepoly);
    } else {
        const dim3 grid((unsigned)((P.ny - 1 + 127) / 128), (unsigned)(P.nz - 1), (unsigned)P.batch);
        return launch_dependent(linepoly3d_kernel<M>, grid, dim3(128), 0, s, P, linepoly);
    }
}

cudaError_t launch_linepoly3d(const Params& P, float* linepoly, cudaStream_t s) {
    switch (P.m) {
        case 1: return launch_linepoly3d_m<1>(P, linepoly, s);
        case 2: return launch_linepoly3d_m<2>(P, linepoly, s);
        case 3: return launch_linepoly3d_m<3>(P, linepoly, s);
        case 4: return launch_linepoly3d_m<4>(P, linepoly, s);
        case 5: return launch_linepoly3d_m<5>(P, linepoly, s);
        case 6: return launch_linepoly3d_m<6>(P, linepoly, s);
        case 7: return launch_linepoly3d_m<7>(P, linepoly, s);
        case 8: return launch_linepoly3d_m<8>(P, linepoly, s);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_strip3d(const Params& P, const float* linepoly, cudaStream_t s) {
    const S3Geo g = geometry3s(s3_problem_of(P));
    cudaError_t e = cudaErrorInvalidValue;
    if (P.nu_mode == DN_NU_NODAL) {
        e = (s3_nxl(P.nx, P.nu_mode, P.f != nullptr) == 8) ? launch_nm<8, 1, 2, 2>(P, linepoly, g, s) : launch_nm<4, 1, 2, 4>(P, linepoly, g, s);
    } else switch (P.m) {
        case 1: e = launch_m3<1>(P, linepoly, g, s); break;
        case 2: e = launch_m3<2>(P, linepoly, g, s); break;
        case 3: e = launch_m3<3>(P, linepoly, g, s); break;
        case 4: e = launch_m3<4>(P, linepoly, g, s); break;
        default: e = launch_strip3d_hi(P, linepoly, g, s); break;      // m = 5..8: compiled in the second part
    }
    if (e != cudaSuccess || P.r == nullptr) return e;       // energy only: no seams
    const long long nA = (long long)P.batch * (g.ntile - 1) * P.nz * (P.nx / 4);
    const long long nB = (long long)P.batch * (g.nchunk - 1) * P.ny * (P.nx / 4);
    if (nA + nB > 0) {
        return launch_dependent(seam_fixup3_kernel, dim3((unsigned)((nA + nB + 255) / 256)), dim3(256), 0, s, P.r,
                                (const float*)P.seam, (const float*)P.zseam, P.nx, P.ny, P.nz, P.batch, g.Ry, g.ntile, g.Z,
                                g.nchunk, nA, nB);
    }
    return cudaSuccess;
}
#endif  // DN_S3_PART

}  // namespace dn
