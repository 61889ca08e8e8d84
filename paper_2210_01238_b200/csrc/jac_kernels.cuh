// Device code of libjac: Jacobi update (2D 5-point / 3D 7-point), halo pack / unpack,
// residual reduction, dense <-> block copies.  sm_100a, fp64, no tensor cores: the work is
// bound by HBM bandwidth, so the kernels are organised around coalesced 128-bit accesses,
// register reuse along the marching axis and single launches over all blocks.
//
// Arithmetic contract (same as the header): s = (W + E) + (S + N); 3D: s = s + (D + U);
// with f: s = s + f; u' = s * 0.25 or s * (1/6).  Every operation is an explicit
// round-to-nearest intrinsic, so the compiler cannot contract an FMA.
#pragma once
#include <cuda_runtime.h>

#include "jac_geom.h"

namespace jac {

enum : int { OP_UPDATE = 0, OP_UPDATE_PULL = 1, OP_RESIDUAL = 2, OP_UPDATE_RES = 3, OP_UPDATE_PULL_RES = 4,
             OP_UPDATE_EXT = 5 };
__host__ __device__ constexpr bool op_stores(int op) { return op != OP_RESIDUAL; }
__host__ __device__ constexpr bool op_pulls(int op) { return op == OP_UPDATE_PULL || op == OP_UPDATE_PULL_RES; }
__host__ __device__ constexpr bool op_sums(int op) { return op == OP_RESIDUAL || op == OP_UPDATE_RES || op == OP_UPDATE_PULL_RES; }
__host__ __device__ constexpr bool op_ext(int op) { return op == OP_UPDATE_EXT; }

// which state a run of sweeps also measures the residual of (host side)
enum : int { kResNone = 0,        // none
             kResBeforeLast = 1,  // the state before the last sweep
             kResOfInput = 2 };   // the state the run starts from
// A temporal kernel takes the level that measures as its RES template argument: level s (1..T) reads
// the state after s - 1 sweeps of the launch and accumulates that state's squared residual; 0: none.

__device__ __forceinline__ double add_rn(double a, double b) { return __dadd_rn(a, b); }
__device__ __forceinline__ double sub_rn(double a, double b) { return __dsub_rn(a, b); }
__device__ __forceinline__ double mul_rn(double a, double b) { return __dmul_rn(a, b); }

// has the solve this launch belongs to already met its tolerance?  (uniform over the grid: the flag
// only changes between launches)
__device__ __forceinline__ bool solve_stopped(const JacGeom& g) { return g.stop != nullptr && *g.stop != 0; }

// ask for a line to be brought into L2
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];\n" ::"l"(p)); }

// ---------------------------------------------------------------------------------------
// Checked build.  compute-sanitizer is not always at hand; compiled with -DJAC_CHECK_BOUNDS every
// global-memory access of the kernels first compares its address range with the array it belongs
// to (JacGeom::chk_lo / chk_hi).  An access outside is NOT made: the first one is recorded in
// *JacGeom::chk_rec -- kernel id in bits 56..63, array in bits 52..55, the byte offset from the
// array's start (two's complement, low 52 bits) below -- loads return 0, and the kernel carries
// on.  Nothing traps and nothing hangs; jac_debug_bounds reads the record.  In the ordinary build
// in_bounds() is the constant true and the checks compile to nothing.
// ---------------------------------------------------------------------------------------
enum : int { CHK_FIELD = 0, CHK_SEND = 1, CHK_SCRATCH = 2 };
enum : int { KID_SWEEP2D = 1, KID_SWEEP3D = 2, KID_REDUCE = 3, KID_HALO = 4, KID_CUT = 5, KID_HALO_WIDE = 6,
             KID_FILL_BOUNDARY = 7, KID_DENSE_COPY = 8, KID_TEMPORAL2D = 9, KID_TEMPORAL3D = 10, KID_RESIDENT = 11 };
#ifdef JAC_CHECK_BOUNDS
constexpr bool kChecksBounds = true;
__device__ __forceinline__ bool in_bounds(const JacGeom& g, const void* p, int bytes, int which, int kid) {
    const char* a = static_cast<const char*>(p);
    if (a >= g.chk_lo[which] && a + bytes <= g.chk_hi[which]) return true;
    const unsigned long long off = (unsigned long long)(a - g.chk_lo[which]) & ((1ULL << 52) - 1);
    atomicCAS(g.chk_rec, 0ULL, ((unsigned long long)kid << 56) | ((unsigned long long)which << 52) | off);
    return false;
}
#else
constexpr bool kChecksBounds = false;
__device__ __forceinline__ constexpr bool in_bounds(const JacGeom&, const void*, int, int, int) { return true; }
#endif
// global loads and stores that go through the check
__device__ __forceinline__ double g_ld(const JacGeom& g, const double* p, int which, int kid) {
    return in_bounds(g, p, 8, which, kid) ? *p : 0.0;
}
__device__ __forceinline__ void g_st(const JacGeom& g, double* p, double v, int which, int kid) {
    if (in_bounds(g, p, 8, which, kid)) *p = v;
}
__device__ __forceinline__ double2 g_ld2(const JacGeom& g, const double* p, int which, int kid) {
    return in_bounds(g, p, 16, which, kid) ? *reinterpret_cast<const double2*>(p) : make_double2(0.0, 0.0);
}
__device__ __forceinline__ void g_st2(const JacGeom& g, double* p, double2 v, int which, int kid) {
    if (in_bounds(g, p, 16, which, kid)) *reinterpret_cast<double2*>(p) = v;
}

// NV consecutive doubles held by one thread (NV = 1 or 2; NV = 2 uses one 128-bit access).
template <int NV> struct Vec { double v[NV]; };

template <int NV> __device__ __forceinline__ Vec<NV> load_vec(const double* p);
template <> __device__ __forceinline__ Vec<1> load_vec<1>(const double* p) {
    Vec<1> r; r.v[0] = *p; return r;
}
template <> __device__ __forceinline__ Vec<2> load_vec<2>(const double* p) {
    const double2 t = *reinterpret_cast<const double2*>(p);
    Vec<2> r; r.v[0] = t.x; r.v[1] = t.y; return r;
}
template <int NV> __device__ __forceinline__ void store_vec(double* p, const Vec<NV>& a);
template <> __device__ __forceinline__ void store_vec<1>(double* p, const Vec<1>& a) { *p = a.v[0]; }
template <> __device__ __forceinline__ void store_vec<2>(double* p, const Vec<2>& a) {
    *reinterpret_cast<double2*>(p) = make_double2(a.v[0], a.v[1]);
}

template <int NV> __device__ __forceinline__ Vec<NV> g_load_vec(const JacGeom& g, const double* p, int kid) {
    if (!in_bounds(g, p, 8 * NV, CHK_FIELD, kid)) { Vec<NV> z; for (int q = 0; q < NV; ++q) z.v[q] = 0.0; return z; }
    return load_vec<NV>(p);
}
template <int NV> __device__ __forceinline__ void g_store_vec(const JacGeom& g, double* p, const Vec<NV>& a, int kid) {
    if (in_bounds(g, p, 8 * NV, CHK_FIELD, kid)) store_vec<NV>(p, a);
}

// Sum of a per-thread value over the CTA in a fixed order: lanes by shuffle, then warps in
// index order by thread 0.  Returns the total in thread 0.
__device__ __forceinline__ double block_sum(double v) {
    __shared__ double warp_part[32];
    const int tid = threadIdx.x + blockDim.x * (threadIdx.y + blockDim.y * threadIdx.z);
    const int nthreads = blockDim.x * blockDim.y * blockDim.z;
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v = add_rn(v, __shfl_down_sync(0xffffffffu, v, off));
    if (lane == 0) warp_part[warp] = v;
    __syncthreads();
    double total = 0.0;
    if (tid == 0) {
        const int nwarps = (nthreads + 31) >> 5;
        for (int w = 0; w < nwarps; ++w) total = add_rn(total, warp_part[w]);
    }
    return total;
}

// interior extent of a block: the last block along an axis may be a remainder block
struct BlockExtent { int x, y, z; };
__device__ __forceinline__ BlockExtent block_extent(const JacGeom& g, long long blk)
{
    const int bxi = (int)(blk % g.gx);
    const int byi = (int)((blk / g.gx) % g.gy);
    const int bzi = (int)(blk / ((long long)g.gx * g.gy));
    BlockExtent e;
    e.x = bxi + 1 == g.gx ? g.rx : g.bx;
    e.y = byi + 1 == g.gy ? g.ry : g.by;
    e.z = bzi + 1 == g.gz ? g.rz : g.bz;
    return e;
}

// ---------------------------------------------------------------------------------------
// 2D: one CTA owns a strip of `rows` rows x (blockDim.x * NV) columns of one block and
// marches along y.  The rows j-1, j, j+1 of a thread's own columns live in registers; the
// west/east neighbours of the strip are read through L1 (those sectors were just fetched by
// the neighbouring lanes' vector loads).  DRAM sees each interior point once.
//
// OP_UPDATE       u' <- update(u), every out-of-block neighbour read from the block's ghosts
// OP_UPDATE_PULL  same arithmetic, but across a face that has a neighbour block the value is
//                 read from that block's interior (the cell its packed face would carry), so
//                 no exchange has to run before the sweep; Dirichlet ghosts are still read
// OP_RESIDUAL     per-CTA partial of sum r^2, r = s - 4u (ghost-reading)
// OP_UPDATE_RES, OP_UPDATE_PULL_RES  the update, and in the same pass the partial of sum r^2 of the
//                 state being read (s is in a register anyway): the residual at no extra traffic
// OP_UPDATE_EXT   the update over a block box that is the interior grown by g.ext layers on every
//                 side (the geometry passed in describes the grown box); positions outside the
//                 domain keep their value.  Used between wide exchanges.
// ---------------------------------------------------------------------------------------
template <int NV, bool HAS_F, int OP>
__global__ void __launch_bounds__(256)
sweep2d_kernel(const double* __restrict__ u, double* __restrict__ un, const double* __restrict__ f,
               double* __restrict__ partials, const JacGeom g, const long long blk0,
               const int tiles_x, const int tiles_y, const int rows)
{
    if (solve_stopped(g)) return;
    const long long t = blockIdx.x;
    const int xt = (int)(t % tiles_x);
    const int yt = (int)((t / tiles_x) % tiles_y);
    const long long blk = blk0 + t / ((long long)tiles_x * tiles_y);
    const int x = (xt * blockDim.x + threadIdx.x) * NV;
    const BlockExtent ext = block_extent(g, blk);
    const int j0 = yt * rows;
    const int j1 = min(ext.y, j0 + rows);
    const long long PX = g.PX;
    double acc = 0.0;

    if (x < ext.x && j0 < j1) {
        const long long base = blk * g.block_stride + g.origin + x;
        const double* ub = u + base;
        const double* fb = HAS_F ? f + base : nullptr;
        double* ob = op_stores(OP) ? un + base : nullptr;

        // where the neighbours outside the block are found, relative to the row's own address
        long long off_w = -1, off_e = NV;             // ghost columns
        long long off_s0 = -PX, off_n1 = PX;          // ghost rows below row 0 / above row by-1
        if (op_pulls(OP)) {
            const int bxi = (int)(blk % g.gx), byi = (int)(blk / g.gx);
            const long long bs = g.block_stride;
            if (x == 0 && bxi > 0) off_w = -bs + g.bx - 1;                     // left block, last column
            if (x + NV == g.bx && bxi + 1 < g.gx) off_e = bs - g.bx + NV;      // right block, column 0
            if (byi > 0) off_s0 = -bs * g.gx + (long long)(g.by - 1) * PX;     // block below, last row
            if (byi + 1 < g.gy) off_n1 = bs * g.gx - (long long)(g.by - 1) * PX;  // block above, row 0
        }

        // grown box: which of this thread's columns / which rows lie inside the domain
        bool xin[NV];
        long long gy0 = 0;
        if (op_ext(OP)) {
            const long long gx0 = (blk % g.gx) * (long long)(g.bx - 2 * g.ext) + x - g.ext;
#pragma unroll
            for (int q = 0; q < NV; ++q) xin[q] = gx0 + q >= 0 && gx0 + q < g.nx;
            gy0 = (blk / g.gx) * (long long)(g.by - 2 * g.ext) - g.ext;
        }

        // a thread at a block border reads its west / east neighbour from the next block: one
        // 32-byte sector per row that no other thread touches; asked for a few rows ahead, or the
        // whole warp waits for DRAM in every row
        const bool far_w = op_pulls(OP) && off_w != -1, far_e = op_pulls(OP) && off_e != NV;

        Vec<NV> S = g_load_vec<NV>(g, ub + (j0 == 0 ? off_s0 : (long long)(j0 - 1) * PX), KID_SWEEP2D);
        Vec<NV> Cc = g_load_vec<NV>(g, ub + (long long)j0 * PX, KID_SWEEP2D);
#pragma unroll 4
        for (int j = j0; j < j1; ++j) {
            const long long ro = (long long)j * PX;
            if (op_pulls(OP) && j + 8 < j1) {
                if (far_w) prefetch_l2(ub + ro + 8 * PX + off_w);
                if (far_e) prefetch_l2(ub + ro + 8 * PX + off_e);
            }
            const Vec<NV> N = g_load_vec<NV>(g, ub + ro + ((op_pulls(OP) && j + 1 == g.by) ? off_n1 : PX), KID_SWEEP2D);
            const double w = g_ld(g, ub + ro + off_w, CHK_FIELD, KID_SWEEP2D);
            const double e = g_ld(g, ub + ro + off_e, CHK_FIELD, KID_SWEEP2D);
            Vec<NV> ff;
            if (HAS_F) ff = g_load_vec<NV>(g, fb + ro, KID_SWEEP2D);
            Vec<NV> o;
#pragma unroll
            for (int q = 0; q < NV; ++q) {
                const double W = (q == 0) ? w : Cc.v[q - 1];
                const double E = (q == NV - 1) ? e : Cc.v[q + 1];
                double s = add_rn(add_rn(W, E), add_rn(S.v[q], N.v[q]));
                if (HAS_F) s = add_rn(s, ff.v[q]);
                if (op_sums(OP)) {
                    const double r = sub_rn(s, mul_rn(4.0, Cc.v[q]));
                    acc = add_rn(acc, mul_rn(r, r));
                }
                if (op_stores(OP)) o.v[q] = mul_rn(s, 0.25);
                if (op_ext(OP) && !(xin[q] && gy0 + j >= 0 && gy0 + j < g.ny)) o.v[q] = Cc.v[q];
            }
            if (op_stores(OP)) g_store_vec<NV>(g, ob + ro, o, KID_SWEEP2D);
            S = Cc;
            Cc = N;
        }
    }
    if (op_sums(OP)) {
        const double total = block_sum(acc);
        if (threadIdx.x == 0) g_st(g, partials + blockIdx.x, total, CHK_SCRATCH, KID_SWEEP2D);
    }
}

// ---------------------------------------------------------------------------------------
// 3D: one CTA owns (blockDim.x * NV) x blockDim.y columns of one block over a range of
// `planes` z-planes and marches along z.  Planes k-1, k, k+1 of a thread's own column are
// in registers (DRAM traffic: one load per point); the y and x neighbours of plane k come
// through L1, which holds the plane since it was fetched as "k+1" one step earlier.
// OP as for the 2D kernel.
// ---------------------------------------------------------------------------------------
template <int NV, bool HAS_F, int OP>
__global__ void __launch_bounds__(512)
sweep3d_kernel(const double* __restrict__ u, double* __restrict__ un, const double* __restrict__ f,
               double* __restrict__ partials, const JacGeom g, const long long blk0,
               const int tiles_x, const int tiles_y, const int tiles_z, const int planes)
{
    if (solve_stopped(g)) return;
    const long long t = blockIdx.x;
    const int xt = (int)(t % tiles_x);
    const int yt = (int)((t / tiles_x) % tiles_y);
    const int zt = (int)((t / ((long long)tiles_x * tiles_y)) % tiles_z);
    const long long blk = blk0 + t / ((long long)tiles_x * tiles_y * tiles_z);
    const int x = (xt * blockDim.x + threadIdx.x) * NV;
    const int y = yt * blockDim.y + threadIdx.y;
    const BlockExtent ext = block_extent(g, blk);
    const int k0 = zt * planes;
    const int k1 = min(ext.z, k0 + planes);
    const long long PX = g.PX, PXY = g.PXY;
    const double c6 = 1.0 / 6.0;
    double acc = 0.0;

    if (x < ext.x && y < ext.y && k0 < k1) {
        const long long base = blk * g.block_stride + g.origin + (long long)y * PX + x;
        const double* ub = u + base;
        const double* fb = HAS_F ? f + base : nullptr;
        double* ob = op_stores(OP) ? un + base : nullptr;

        long long off_w = -1, off_e = NV, off_s = -PX, off_n = PX;   // within the plane
        long long off_d0 = -PXY, off_u1 = PXY;                        // below plane 0 / above plane bz-1
        if (op_pulls(OP)) {
            const int bxi = (int)(blk % g.gx);
            const int byi = (int)((blk / g.gx) % g.gy);
            const int bzi = (int)(blk / ((long long)g.gx * g.gy));
            const long long bs = g.block_stride;
            const long long bsy = bs * g.gx, bsz = bs * g.gx * g.gy;
            if (x == 0 && bxi > 0) off_w = -bs + g.bx - 1;
            if (x + NV == g.bx && bxi + 1 < g.gx) off_e = bs - g.bx + NV;
            if (y == 0 && byi > 0) off_s = -bsy + (long long)(g.by - 1) * PX;
            if (y + 1 == g.by && byi + 1 < g.gy) off_n = bsy - (long long)(g.by - 1) * PX;
            if (bzi > 0) off_d0 = -bsz + (long long)(g.bz - 1) * PXY;
            if (bzi + 1 < g.gz) off_u1 = bsz - (long long)(g.bz - 1) * PXY;
        }

        // grown box (OP_UPDATE_EXT): is this thread's column inside the domain in x and y; first plane
        bool xyin[NV];
        long long gz0 = 0;
        if (op_ext(OP)) {
            const long long gx0 = (blk % g.gx) * (long long)(g.bx - 2 * g.ext) + x - g.ext;
            const long long gy = ((blk / g.gx) % g.gy) * (long long)(g.by - 2 * g.ext) + y - g.ext;
#pragma unroll
            for (int q = 0; q < NV; ++q) xyin[q] = gx0 + q >= 0 && gx0 + q < g.nx && gy >= 0 && gy < g.ny;
            gz0 = (blk / ((long long)g.gx * g.gy)) * (long long)(g.bz - 2 * g.ext) - g.ext;
        }

        // far west / east neighbours (the next block's column): asked for a few planes ahead, as in 2D
        const bool far_w = op_pulls(OP) && off_w != -1, far_e = op_pulls(OP) && off_e != NV;

        Vec<NV> D = g_load_vec<NV>(g, ub + (k0 == 0 ? off_d0 : (long long)(k0 - 1) * PXY), KID_SWEEP3D);
        Vec<NV> Cc = g_load_vec<NV>(g, ub + (long long)k0 * PXY, KID_SWEEP3D);
#pragma unroll 2
        for (int k = k0; k < k1; ++k) {
            const long long po = (long long)k * PXY;
            if (op_pulls(OP) && k + 4 < k1) {
                if (far_w) prefetch_l2(ub + po + 4 * PXY + off_w);
                if (far_e) prefetch_l2(ub + po + 4 * PXY + off_e);
            }
            const Vec<NV> U = g_load_vec<NV>(g, ub + po + ((op_pulls(OP) && k + 1 == g.bz) ? off_u1 : PXY), KID_SWEEP3D);
            const Vec<NV> S = g_load_vec<NV>(g, ub + po + off_s, KID_SWEEP3D);
            const Vec<NV> N = g_load_vec<NV>(g, ub + po + off_n, KID_SWEEP3D);
            const double w = g_ld(g, ub + po + off_w, CHK_FIELD, KID_SWEEP3D);
            const double e = g_ld(g, ub + po + off_e, CHK_FIELD, KID_SWEEP3D);
            Vec<NV> ff;
            if (HAS_F) ff = g_load_vec<NV>(g, fb + po, KID_SWEEP3D);
            Vec<NV> o;
#pragma unroll
            for (int q = 0; q < NV; ++q) {
                const double W = (q == 0) ? w : Cc.v[q - 1];
                const double E = (q == NV - 1) ? e : Cc.v[q + 1];
                double s = add_rn(add_rn(W, E), add_rn(S.v[q], N.v[q]));
                s = add_rn(s, add_rn(D.v[q], U.v[q]));
                if (HAS_F) s = add_rn(s, ff.v[q]);
                if (op_sums(OP)) {
                    const double r = sub_rn(s, mul_rn(6.0, Cc.v[q]));
                    acc = add_rn(acc, mul_rn(r, r));
                }
                if (op_stores(OP)) o.v[q] = mul_rn(s, c6);
                if (op_ext(OP) && !(xyin[q] && gz0 + k >= 0 && gz0 + k < g.nz)) o.v[q] = Cc.v[q];
            }
            if (op_stores(OP)) g_store_vec<NV>(g, ob + po, o, KID_SWEEP3D);
            D = Cc;
            Cc = U;
        }
    }
    if (op_sums(OP)) {
        const double total = block_sum(acc);
        if (threadIdx.x == 0 && threadIdx.y == 0) g_st(g, partials + blockIdx.x, total, CHK_SCRATCH, KID_SWEEP3D);
    }
}

// Second pass of the residual: one CTA adds the per-CTA partials in a fixed order and leaves the
// sum, or (root) its square root, the norm.
__global__ void __launch_bounds__(1024)
reduce_partials_kernel(const double* __restrict__ partials, const long long n, double* __restrict__ out, const bool root)
{
    double acc = 0.0;
    for (long long i = threadIdx.x; i < n; i += blockDim.x) acc = add_rn(acc, partials[i]);
    const double total = block_sum(acc);
    if (threadIdx.x == 0) *out = root ? sqrt(total) : total;
}

// ---------------------------------------------------------------------------------------
// Halo pack / unpack.  One launch covers `npairs` consecutive (block, face) pairs starting at
// pair0 (pair = block * nfaces + face).  Pairs whose face lies on the domain boundary, or is
// not in face_mask, do nothing.
//
// Element e of a packed face (source memory order):
//   x face: e = (k*by + j)*h + c      y face: e = (k*h + r)*bx + i      z face: e = (p*by + j)*bx + i
// Pack reads the interior strip next to the face; unpack writes the ghost strip of the same
// face from the neighbour's opposite-face buffer.
// ---------------------------------------------------------------------------------------
// Block coordinates, the neighbour across a face and the block's interior extent, from one
// decomposition of the block number.  IT is the integer type the arithmetic runs in: 32-bit
// whenever block, pair and thread counts fit (the host checks), since 64-bit divisions are what
// these short kernels would otherwise spend most of their instructions on.
template <typename IT>
struct BlockPlace {
    IT nb;            // neighbour across the face (valid if has_nb)
    bool has_nb;
    BlockExtent ext;
};
template <typename IT>
__device__ __forceinline__ BlockPlace<IT> block_place(const JacGeom& g, IT blk, int face)
{
    const IT gx = (IT)g.gx, gy = (IT)g.gy;
    const IT q = blk / gx;
    const int bxi = (int)(blk - q * gx);
    const IT bzi_ = q / gy;
    const int byi = (int)(q - bzi_ * gy);
    const int bzi = (int)bzi_;
    BlockPlace<IT> p;
    p.ext.x = bxi + 1 == g.gx ? g.rx : g.bx;
    p.ext.y = byi + 1 == g.gy ? g.ry : g.by;
    p.ext.z = bzi + 1 == g.gz ? g.rz : g.bz;
    switch (face) {
        case 0: p.has_nb = bxi > 0; p.nb = blk - 1; break;
        case 1: p.has_nb = bxi + 1 < g.gx; p.nb = blk + 1; break;
        case 2: p.has_nb = byi > 0; p.nb = blk - gx; break;
        case 3: p.has_nb = byi + 1 < g.gy; p.nb = blk + gx; break;
        case 4: p.has_nb = bzi > 0; p.nb = blk - gx * gy; break;
        default: p.has_nb = bzi + 1 < g.gz; p.nb = blk + gx * gy; break;
    }
    return p;
}

__device__ __forceinline__ long long neighbour_block(const JacGeom& g, long long blk, int face)
{
    const BlockPlace<long long> p = block_place<long long>(g, blk, face);
    return p.has_nb ? p.nb : -1;
}

// offset (relative to the block's interior origin) of element e of the strip on `face`;
// lo = first layer of the strip along the face's axis (interior-relative); ext = the block's
// interior extent, which the strip spans on the axes other than the face's.  e < 2^31.
__device__ __forceinline__ long long strip_offset(const JacGeom& g, const BlockExtent& ext, int face, unsigned e, int lo)
{
    const int axis = face >> 1;
    long long x, y, z;
    if (axis == 0) {
        const unsigned t = e / (unsigned)g.h; x = (int)(e - t * g.h) + lo;
        z = t / (unsigned)ext.y; y = t - (unsigned)z * ext.y;
    } else if (axis == 1) {
        const unsigned t = e / (unsigned)ext.x; x = e - t * ext.x;
        z = t / (unsigned)g.h; y = (int)(t - (unsigned)z * g.h) + lo;
    } else {
        const unsigned t = e / (unsigned)ext.x; x = e - t * ext.x;
        const unsigned p = t / (unsigned)ext.y; y = t - p * ext.y; z = (int)p + lo;
    }
    return z * g.PXY + y * g.PX + x;
}

// elements of the packed face of a block with interior extent `ext`
__device__ __forceinline__ long long face_elems_of(const JacGeom& g, const BlockExtent& ext, int face)
{
    const int axis = face >> 1;
    const long long h = g.h;
    return axis == 0 ? h * ext.y * ext.z : (axis == 1 ? h * ext.x * ext.z : h * ext.x * ext.y);
}

// Halo pack, unpack, or both at once.  `slots` threads (a multiple of 32, so a warp never straddles
// faces) are reserved per (block, face) pair and the grid is packed over threads, not faces: small
// faces do not leave CTAs mostly idle.  The work of a face is cut into units, up to four per thread,
// whose loads are all issued before the first store:
//   x face   a unit is one row (k, j) of the strip: h cells, strided by the row pitch in the block
//            and contiguous in the buffer; consecutive threads take consecutive rows, so a warp
//            touches 32 sectors of the block and 32 h contiguous doubles of the buffer.
//            Ghost columns are the innermost h cells of a four-cell margin that nothing else
//            uses; for h <= 2 the unpack writes the whole 32-byte sector (the ghost cells and
//            zeros beside them): a store of a full sector needs no read of the old one, a store
//            of 8 of its bytes does.
//   y, z     a unit is two cells of a line of the strip, contiguous on both sides (one 128-bit
//            access each when the line starts are 16-byte aligned); a thread keeps its column and
//            walks over lines, so the only division per unit is the line's split into (y, z).
// HALO_EXCHANGE does pack and unpack in one pass: the thread that fills ghost cells of (block,
// face) reads them from the neighbour's interior strip and also leaves them in the neighbour's
// send slot, so the buffers and the ghosts end up exactly as after pack followed by unpack: one
// read and two writes per face cell instead of two reads and two writes, and one launch.
enum : int { HALO_PACK = 0, HALO_UNPACK = 1, HALO_EXCHANGE = 2 };
constexpr int kHaloUnits = 4;     // units per thread

template <int OP, typename IT>
__global__ void __launch_bounds__(256)
halo_kernel(double* __restrict__ u, double* __restrict__ send, const JacGeom g,
            const long long pair0, const long long npairs, const int slots, const unsigned face_mask)
{
    if (solve_stopped(g)) return;
    const IT t = (IT)blockIdx.x * (IT)blockDim.x + (IT)threadIdx.x;
    const IT pr = t / (IT)slots;
    if (pr >= (IT)npairs) return;
    const unsigned local = (unsigned)(t - pr * (IT)slots);
    const IT pair = (IT)pair0 + pr;
    const IT blk = pair / (IT)g.nfaces;
    const int face = (int)(pair - blk * (IT)g.nfaces);
    if (!((face_mask >> face) & 1u)) return;
    const BlockPlace<IT> bp = block_place<IT>(g, blk, face);
    if (!bp.has_nb) return;
    const BlockExtent& be = bp.ext;          // the neighbour has the same extent on the axes the strip spans
    const int axis = face >> 1;
    const int h = g.h;
    const int ext = axis == 0 ? be.x : (axis == 1 ? be.y : be.z);
    const int full = axis == 0 ? g.bx : (axis == 1 ? g.by : g.bz);
    // first layer of the strip along the face's axis, interior-relative:
    //   where the data is read (pack: our interior strip; exchange: the neighbour's strip facing us --
    //   both blocks of such a pair are full along the axis, or the one at the high end is the remainder
    //   block, whose strip starts at 0)            and where ghost cells are written
    const int lo_src = OP == HALO_EXCHANGE ? ((face & 1) ? 0 : full - h) : ((face & 1) ? ext - h : 0);
    const int lo_dst = (face & 1) ? ext : -h;
    double* own = u + (long long)blk * g.block_stride + g.origin;
    const double* src_blk = OP == HALO_EXCHANGE ? u + (long long)bp.nb * g.block_stride + g.origin : own;
    // the send slot involved: ours (pack) or the neighbour's opposite one (unpack, exchange)
    double* buf = OP == HALO_PACK ? send + (long long)blk * g.send_stride + g.face_off[face]
                                  : send + (long long)bp.nb * g.send_stride + g.face_off[face ^ 1];
    const long long PX = g.PX, PXY = g.PXY;

    if (axis == 0) {
        const unsigned nrows = (unsigned)be.y * (unsigned)be.z;
        // whole-sector stores of the ghost columns: rows start on 32-byte boundaries
        const bool sector = OP != HALO_PACK && h <= 2 && g.xpad == 4 && (PX & 3) == 0 && ((face & 1) == 0 || (be.x & 3) == 0);
        double v[kHaloUnits][2];
        long long cell[kHaloUnits];
#pragma unroll
        for (int k = 0; k < kHaloUnits; ++k) {
            const unsigned R = local + (unsigned)k * (unsigned)slots;
            if (R >= nrows) continue;
            const unsigned z = be.z == 1 ? 0u : R / (unsigned)be.y;
            const unsigned y = R - z * (unsigned)be.y;
            cell[k] = (long long)z * PXY + (long long)y * PX;
            if (h <= 2) {
#pragma unroll
                for (int c = 0; c < 2; ++c)
                    if (c < h) v[k][c] = OP == HALO_UNPACK ? g_ld(g, buf + (long long)R * h + c, CHK_SEND, KID_HALO) : g_ld(g, src_blk + cell[k] + lo_src + c, CHK_FIELD, KID_HALO);
            }
        }
#pragma unroll
        for (int k = 0; k < kHaloUnits; ++k) {
            const unsigned R = local + (unsigned)k * (unsigned)slots;
            if (R >= nrows) continue;
            if (h <= 2) {
                if (OP != HALO_UNPACK) {
#pragma unroll
                    for (int c = 0; c < 2; ++c)
                        if (c < h) g_st(g, buf + (long long)R * h + c, v[k][c], CHK_SEND, KID_HALO);
                }
                if (OP != HALO_PACK) {
                    if (sector) {
                        double* sec = own + cell[k] + ((face & 1) ? ext : -4);
                        if (face & 1) {      // the ghosts are the first h cells of the sector
                            g_st2(g, sec, make_double2(v[k][0], h == 2 ? v[k][1] : 0.0), CHK_FIELD, KID_HALO);
                            g_st2(g, sec + 2, make_double2(0.0, 0.0), CHK_FIELD, KID_HALO);
                        } else {             // the last h
                            g_st2(g, sec, make_double2(0.0, 0.0), CHK_FIELD, KID_HALO);
                            g_st2(g, sec + 2, h == 2 ? make_double2(v[k][0], v[k][1]) : make_double2(0.0, v[k][0]), CHK_FIELD, KID_HALO);
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < 2; ++c)
                            if (c < h) g_st(g, own + cell[k] + lo_dst + c, v[k][c], CHK_FIELD, KID_HALO);
                    }
                }
            } else {                         // wider strips (h <= 8): the row's cells, loads before stores
                double w[8];
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    if (c < h) w[c] = OP == HALO_UNPACK ? g_ld(g, buf + (long long)R * h + c, CHK_SEND, KID_HALO) : g_ld(g, src_blk + cell[k] + lo_src + c, CHK_FIELD, KID_HALO);
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    if (c >= h) continue;
                    if (OP != HALO_UNPACK) g_st(g, buf + (long long)R * h + c, w[c], CHK_SEND, KID_HALO);
                    if (OP != HALO_PACK) g_st(g, own + cell[k] + lo_dst + c, w[c], CHK_FIELD, KID_HALO);
                }
            }
        }
        return;
    }

    // y and z faces: lines of be.x cells, contiguous in the block and in the buffer
    const unsigned ex = (unsigned)be.x;
    const bool vec = (ex & 1u) == 0 && (PX & 1) == 0;       // both sides 16-byte aligned
    const unsigned V = vec ? ex >> 1 : ex;                    // units per line
    const unsigned nlines = (unsigned)h * (unsigned)(axis == 1 ? be.z : be.y);
    const unsigned TL = (unsigned)slots / V;                  // lines the pair's threads cover side by side
    if (TL == 0) {
        // a line longer than the pair's threads (tiny slots): threads stride over the units of the face
        const unsigned nunits = V * nlines;
        for (unsigned q = local; q < nunits; q += (unsigned)slots) {
            const unsigned L = q / V, vi = q - L * V;
            const unsigned a = axis == 1 ? L / (unsigned)h : L / (unsigned)be.y;
            const unsigned r = axis == 1 ? L - a * h : L - a * be.y;
            const long long so = axis == 1 ? (long long)a * PXY + (long long)(lo_src + (int)r) * PX
                                           : (long long)r * PX + (long long)(lo_src + (int)a) * PXY;
            const long long dn = axis == 1 ? (long long)a * PXY + (long long)(lo_dst + (int)r) * PX
                                           : (long long)r * PX + (long long)(lo_dst + (int)a) * PXY;
            const unsigned x0 = vec ? 2 * vi : vi;
            for (unsigned c = 0; c < (vec ? 2u : 1u); ++c) {
                const long long bi = (long long)L * ex + x0 + c;
                const double w = OP == HALO_UNPACK ? g_ld(g, buf + bi, CHK_SEND, KID_HALO) : g_ld(g, src_blk + so + x0 + c, CHK_FIELD, KID_HALO);
                if (OP != HALO_UNPACK) g_st(g, buf + bi, w, CHK_SEND, KID_HALO);
                if (OP != HALO_PACK) g_st(g, own + dn + x0 + c, w, CHK_FIELD, KID_HALO);
            }
        }
        return;
    }
    const unsigned L0 = local / V;
    if (L0 >= TL) return;                                     // fewer than V threads left over
    const unsigned vi = local - L0 * V;
    const unsigned x0 = vec ? 2 * vi : vi;
    double2 w2[kHaloUnits];
    double w1[kHaloUnits];
    long long dst_off[kHaloUnits], buf_off[kHaloUnits];
    for (unsigned Lb = L0; Lb < nlines; Lb += kHaloUnits * TL) {
#pragma unroll
        for (int k = 0; k < kHaloUnits; ++k) {
            const unsigned L = Lb + (unsigned)k * TL;
            if (L >= nlines) continue;
            // line -> (layer along the axis, position along the other axis)
            unsigned a, r;
            if (axis == 1) { a = h == 1 ? L : L / (unsigned)h; r = L - a * (unsigned)h; }      // a = z, r = layer
            else { a = h == 1 ? 0u : L / (unsigned)be.y; r = L - a * (unsigned)be.y; }         // a = layer, r = y
            const long long so = axis == 1 ? (long long)a * PXY + (long long)(lo_src + (int)r) * PX
                                           : (long long)(lo_src + (int)a) * PXY + (long long)r * PX;
            dst_off[k] = (axis == 1 ? (long long)a * PXY + (long long)(lo_dst + (int)r) * PX
                                    : (long long)(lo_dst + (int)a) * PXY + (long long)r * PX) + x0;
            buf_off[k] = (long long)L * ex + x0;
            if (vec) w2[k] = OP == HALO_UNPACK ? g_ld2(g, buf + buf_off[k], CHK_SEND, KID_HALO)
                                               : g_ld2(g, src_blk + so + x0, CHK_FIELD, KID_HALO);
            else w1[k] = OP == HALO_UNPACK ? g_ld(g, buf + buf_off[k], CHK_SEND, KID_HALO) : g_ld(g, src_blk + so + x0, CHK_FIELD, KID_HALO);
        }
#pragma unroll
        for (int k = 0; k < kHaloUnits; ++k) {
            const unsigned L = Lb + (unsigned)k * TL;
            if (L >= nlines) continue;
            if (vec) {
                if (OP != HALO_UNPACK) g_st2(g, buf + buf_off[k], w2[k], CHK_SEND, KID_HALO);
                if (OP != HALO_PACK) g_st2(g, own + dst_off[k], w2[k], CHK_FIELD, KID_HALO);
            } else {
                if (OP != HALO_UNPACK) g_st(g, buf + buf_off[k], w1[k], CHK_SEND, KID_HALO);
                if (OP != HALO_PACK) g_st(g, own + dst_off[k], w1[k], CHK_FIELD, KID_HALO);
            }
        }
    }
}

// Cut faces of a slab context: the faces of the blocks on the slab's first or last plane along the
// slowest axis that look across the cut (they have no neighbour block inside the context).  Pack
// gathers their h interior layers into one contiguous plane buffer, unpack scatters such a buffer
// into their ghost layers.  Block m of the plane owns elements [m * slot, m * slot + its face
// elements) of the buffer, in the order of a packed face.  `slots` threads per block, two
// consecutive elements per thread (a cut face is a y face in 2D, a z face in 3D: contiguous rows).
template <bool UNPACK>
__global__ void __launch_bounds__(256)
cut_kernel(double* __restrict__ u, double* __restrict__ buf, const JacGeom g, const long long blk0,
           const long long nblk, const int slots, const int face, const long long slot)
{
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long m = t / slots;
    if (m >= nblk) return;
    const unsigned e = 2u * (unsigned)(t - m * slots);
    const long long blk = blk0 + m;
    const BlockExtent be = block_extent(g, blk);
    const long long n = face_elems_of(g, be, face);
    if (e >= n) return;
    const int axis = face >> 1;
    const int ext = axis == 1 ? be.y : be.z;
    const int lo = UNPACK ? ((face & 1) ? ext : -g.h) : ((face & 1) ? ext - g.h : 0);
    double* ub = u + blk * g.block_stride + g.origin;
    double* bp = buf + m * slot;
    // (the block side goes through the checked-build test; the plane may be another context's buffer)
    if ((be.x & 1) == 0 && (g.PX & 1) == 0) {
        double* cell = ub + strip_offset(g, be, face, e, lo);
        double2* sl = reinterpret_cast<double2*>(bp + e);
        if (UNPACK) g_st2(g, cell, *sl, CHK_FIELD, KID_CUT); else *sl = g_ld2(g, cell, CHK_FIELD, KID_CUT);
    } else {
        double* c0 = ub + strip_offset(g, be, face, e, lo);
        if (UNPACK) g_st(g, c0, bp[e], CHK_FIELD, KID_CUT); else bp[e] = g_ld(g, c0, CHK_FIELD, KID_CUT);
        if (e + 1 < n) {
            double* c1 = ub + strip_offset(g, be, face, e + 1, lo);
            if (UNPACK) g_st(g, c1, bp[e + 1], CHK_FIELD, KID_CUT); else bp[e + 1] = g_ld(g, c1, CHK_FIELD, KID_CUT);
        }
    }
}

// Wide exchange, one axis per launch: the strip of a face is h layers along `axis` (interior
// layers for pack, ghost layers for unpack) over the whole padded extent (-h .. extent + h) of the
// other axes, so edge and corner data delivered by the launches of earlier axes travels on.
// Element e of a wide face, source memory order (wx, wy, wz = the block's extent + 2h; wz = 1 in 2D):
//   x face: e = (k*wy + j)*h + c      y face: e = (k*h + r)*wx + i      z face: e = (p*wy + j)*wx + i
// One thread per element; `slots` threads (whole warps) per (block, side) pair.
template <bool UNPACK, typename IT>
__global__ void __launch_bounds__(256)
halo_wide_kernel(double* __restrict__ arr, double* __restrict__ send, const JacGeom g, const int axis,
                 const int slots)
{
    const IT t = (IT)blockIdx.x * (IT)blockDim.x + (IT)threadIdx.x;
    const IT pr = t / (IT)slots;
    if (pr >= (IT)(2 * g.nblocks)) return;
    const unsigned e = (unsigned)(t - pr * (IT)slots);
    const IT blk = pr >> 1;
    const int face = 2 * axis + (int)(pr & 1);
    const BlockPlace<IT> bp = block_place<IT>(g, blk, face);
    if (!bp.has_nb) return;
    const BlockExtent& be = bp.ext;
    const int h = g.h, hz = g.ndim == 3 ? g.h : 0;
    const unsigned wx = be.x + 2 * h, wy = be.y + 2 * h, wz = be.z + 2 * hz;
    const long long n = axis == 0 ? (long long)h * wy * wz : (axis == 1 ? (long long)h * wx * wz : (long long)h * wx * wy);
    if (e >= n) return;
    const int ext = axis == 0 ? be.x : (axis == 1 ? be.y : be.z);
    const int lo = UNPACK ? ((face & 1) ? ext : -h) : ((face & 1) ? ext - h : 0);
    long long x, y, z;
    if (axis == 0) {
        const unsigned q = e / (unsigned)h; x = (int)(e - q * h) + lo;
        const unsigned k = q / wy; y = (int)(q - k * wy) - h; z = (int)k - hz;
    } else if (axis == 1) {
        const unsigned q = e / wx; x = (int)(e - q * wx) - h;
        const unsigned k = q / (unsigned)h; y = (int)(q - k * h) + lo; z = (int)k - hz;
    } else {
        const unsigned q = e / wx; x = (int)(e - q * wx) - h;
        const unsigned k = q / wy; y = (int)(q - k * wy) - h; z = (int)k + lo;
    }
    double* cell = arr + (long long)blk * g.block_stride + g.origin + z * g.PXY + y * g.PX + x;
    if (UNPACK) g_st(g, cell, g_ld(g, send + (long long)bp.nb * g.send_stride + g.face_off[face ^ 1] + e, CHK_SEND, KID_HALO_WIDE),
                     CHK_FIELD, KID_HALO_WIDE);
    else g_st(g, send + (long long)blk * g.send_stride + g.face_off[face] + e, g_ld(g, cell, CHK_FIELD, KID_HALO_WIDE),
              CHK_SEND, KID_HALO_WIDE);
}

// Dirichlet value into the ghost strip of `face` of every block on that domain face, in both
// solution arrays.  grid = (chunks, blocks on the face).
__global__ void __launch_bounds__(256)
fill_boundary_kernel(double* __restrict__ u0, double* __restrict__ u1, const JacGeom g,
                     const int face, const double value, const int chunks)
{
    const int axis = face >> 1;
    const long long t = blockIdx.x;
    const long long m = t / chunks;  // index among the blocks on this face
    const int chunk = (int)(t % chunks);
    // enumerate blocks with the face's axis coordinate fixed at 0 or g-1
    long long c[3];
    const int ga[3] = {g.gx, g.gy, g.gz};
    long long rem = m;
    for (int a = 0; a < 3; ++a) {
        if (a == axis) { c[a] = (face & 1) ? ga[a] - 1 : 0; continue; }
        c[a] = rem % ga[a];
        rem /= ga[a];
    }
    const long long blk = (c[2] * g.gy + c[1]) * g.gx + c[0];
    const BlockExtent be = block_extent(g, blk);
    const int ext = axis == 0 ? be.x : (axis == 1 ? be.y : be.z);
    const int lo = (face & 1) ? ext : -g.h;
    const long long n = face_elems_of(g, be, face);
    const long long base = blk * g.block_stride + g.origin;
    for (long long e = (long long)chunk * blockDim.x + threadIdx.x; e < n;
         e += (long long)chunks * blockDim.x) {
        const long long off = base + strip_offset(g, be, face, e, lo);
        g_st(g, u0 + off, value, CHK_FIELD, KID_FILL_BOUNDARY);
        g_st(g, u1 + off, value, CHK_FIELD, KID_FILL_BOUNDARY);
    }
}

// Dense array (x fastest over the global interior) <-> block interiors.  One CTA copies a
// segment of one dense row: the row decomposition is done once per CTA, threads move NV
// consecutive doubles each (NV = 2 when bx is even: both sides are 16-byte aligned).
template <bool TO_BLOCKS, int NV>
__global__ void __launch_bounds__(256)
dense_copy_kernel(double* __restrict__ blocks, double* __restrict__ dense, const JacGeom g,
                  const int segs_per_row)
{
    const long long row = blockIdx.x / segs_per_row;          // gj + ny * gk
    const int seg = (int)(blockIdx.x % segs_per_row);
    const long long gj = row % g.ny, gk = row / g.ny;
    const long long byi = gj / g.by, bzi = gk / g.bz;
    const long long row_off = ((bzi * g.gy + byi) * g.gx) * g.block_stride + g.origin +
                              (gk - bzi * g.bz) * g.PXY + (gj - byi * g.by) * g.PX;
    const long long gi = ((long long)seg * blockDim.x + threadIdx.x) * NV;
    if (gi >= g.nx) return;
    const long long bxi = gi / g.bx;
    double* bp = blocks + row_off + bxi * g.block_stride + (gi - bxi * g.bx);
    double* dp = dense + row * g.nx + gi;
    if (TO_BLOCKS) g_store_vec<NV>(g, bp, load_vec<NV>(dp), KID_DENSE_COPY);
    else store_vec<NV>(dp, g_load_vec<NV>(g, bp, KID_DENSE_COPY));
}

// ---------------------------------------------------------------------------------------
// 2D temporal blocking: T sweeps per launch, in registers.
//
// A warp owns a strip 128 columns wide (4 consecutive points per lane) and streams it along
// y.  Input row r enters at level 0; in the same step level s (s = 1..T) produces its row r - s
// from rows r-s-1, r-s, r-s+1 of level s-1, the last of which level s-1 has produced a moment
// before.  Levels therefore run lowest first, and of each level only two rows are alive from one
// step to the next (2*4*T doubles per lane; a pipeline whose levels lag by two rows and are
// independent within a step keeps three, which at T = 8 leaves room for 8 warps per SM only).
// Across the points of a row and across the warps of an SM there is independent work to cover
// the latency of the chain of levels.  West/east neighbours come from the adjacent lanes by
// shuffle, so warps never synchronise with each other.  The two edge
// lanes of a warp lose one point of validity per level; lanes 1..30 (120 columns) are exact
// after T <= 4 levels and are the ones stored.  Strips read across block borders directly
// (the neighbour's interior is the halo), which is what an exchange before every sweep would
// deliver; Dirichlet values are injected for rows/columns outside the domain at every level.
// Steps that touch no domain boundary run a variant without any of those fix-ups.
//
// Input rows are fetched with cp.async into a per-warp shared-memory ring DEPTH rows deep, so
// the loads in flight cost no registers; each copy instruction of a warp covers 512
// contiguous bytes of the row.  Requires bx % 4 == 0 and ny < 2^30.
// ---------------------------------------------------------------------------------------
#ifndef JAC_TW
#define JAC_TW 4      // warps per CTA (independent strips)
#endif
#ifndef JAC_TD
#define JAC_TD 8      // input rows in flight per warp
#endif
#ifndef JAC_TOCC
#define JAC_TOCC 3    // CTAs per SM the register allocation aims for
#endif
// points per lane for T > 4.  2 was measured: 12 warps per SM instead of 8, but 1364 against
// 1702 GLUP/s at T = 8 (more halo lanes and more shuffles per point).
#ifndef JAC_TP_DEEP
#define JAC_TP_DEEP 4
#endif
constexpr int kTemporalWarps = JAC_TW;
constexpr int kTemporalDepth = JAC_TD;
// Right-hand side rows of the 2D temporal kernel travel through a second cp.async ring: a row is
// copied together with the u row of the same index and stays until the top level has used it,
// DEPTH + T steps later (at most 16).
constexpr int kTemporalFDepth = 16;
__host__ __device__ constexpr bool temporal_f_ring(int T, bool has_f) { return has_f && T + kTemporalDepth <= kTemporalFDepth; }
__host__ __device__ constexpr int temporal_stages_per_warp(int T, bool has_f) {
    return kTemporalDepth + (temporal_f_ring(T, has_f) ? kTemporalFDepth : 0);
}
// CTAs per SM the register allocation aims for
__host__ __device__ constexpr int temporal_ctas_per_sm(int T, bool has_f) {
#ifdef JAC_T2_FORCE_MINB
    return JAC_T2_FORCE_MINB;
#else
    return (T > 4 || has_f) ? 2 : JAC_TOCC;
#endif
}
// A lane holds P consecutive points (4; the code also runs with 2, which halves the window
// registers of deep pipelines but was measured slower).  A ring stage is one row of the strip: 16 P chunks of 16 bytes.
__host__ __device__ constexpr int temporal_points(int T) { return T > 4 ? JAC_TP_DEEP : 4; }
__host__ __device__ constexpr int temporal_stage_chunks(int P) { return 16 * P; }
__host__ __device__ constexpr size_t temporal_smem_bytes(int T, bool has_f) {
    return (size_t)kTemporalWarps * temporal_stages_per_warp(T, has_f) *
           temporal_stage_chunks(temporal_points(T)) * sizeof(double2);
}
// lanes at each end of a warp whose points are no longer exact after T levels
__host__ __device__ constexpr int temporal_halo_lanes(int T) {
    return (T + temporal_points(T) - 1) / temporal_points(T);
}
__host__ __device__ constexpr int temporal_strip_cols(int T) {
    return (32 - 2 * temporal_halo_lanes(T)) * temporal_points(T);
}

struct RowCursor {
    long long off;  // element offset of the row within the array, relative to a lane's column base
    int j;          // row index inside its block (negative while still below the domain)
    __device__ __forceinline__ void init(int gy, const JacGeom& g, long long block_row_stride) {
        if (gy < 0) { j = gy; off = (long long)gy * g.PX; }
        else {
            const int byi = gy / g.by;
            j = gy - byi * g.by;
            off = byi * block_row_stride + (long long)j * g.PX;
        }
    }
    __device__ __forceinline__ void advance(const JacGeom& g, long long block_row_stride) {
        ++j;
        off += g.PX;
        if (j == g.by) { j = 0; off += block_row_stride - (long long)g.by * g.PX; }
    }
};

template <int P> struct RowN { double v[P]; };

// P consecutive doubles as P/2 128-bit accesses (global or shared memory)
template <int P> __device__ __forceinline__ RowN<P> load_rown(const double* p) {
    RowN<P> r;
#pragma unroll
    for (int k = 0; k < P / 2; ++k) {
        const double2 a = reinterpret_cast<const double2*>(p)[k];
        r.v[2 * k] = a.x; r.v[2 * k + 1] = a.y;
    }
    return r;
}
template <int P> __device__ __forceinline__ void store_rown(double* p, const RowN<P>& r) {
#pragma unroll
    for (int k = 0; k < P / 2; ++k) reinterpret_cast<double2*>(p)[k] = make_double2(r.v[2 * k], r.v[2 * k + 1]);
}
template <int P> __device__ __forceinline__ RowN<P> fill_rown(double c) {
    RowN<P> r;
#pragma unroll
    for (int k = 0; k < P; ++k) r.v[k] = c;
    return r;
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
__device__ __forceinline__ void g_cp_async16(const JacGeom& g, void* smem_dst, const double* gmem_src, int kid) {
    if (in_bounds(g, gmem_src, 16, CHK_FIELD, kid)) cp_async16(smem_dst, gmem_src);
}
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}
// ask for a line to be brought into L2 (measured equal to an L1 prefetch here, and +9 % over none)
__device__ __forceinline__ void prefetch_line(const void* p) {
    asm volatile("prefetch.global.L2 [%0];\n" ::"l"(p));
}

// Per-lane constants of a strip.  A ring stage holds one row as 64 chunks of 16 bytes in
// natural order (chunk k = columns 2k, 2k+1 of the strip).  One copy instruction of the warp
// moves chunks `lane` (or `32 + lane`): 512 contiguous bytes on both sides, which the memory
// pipeline turns into four full-line requests (a permuted shared-memory destination was
// measured to split it into per-lane sector requests and to triple the L2 request count).
// A lane then reads its own 4 points from chunks 2*lane and 2*lane + 1.
struct TemporalCtx {
    const double* fb;     // f + this lane's column base (its 4 points)
    double* ob;           // u' + this lane's column base
    const double* src_a;  // u + column base of chunk `lane`
    const double* src_b;  // u + column base of chunk `32 + lane`
    double2* dst_a;       // ring positions (stage 0) of the two chunks this lane copies
    double2* dst_b;
    const double2* mine;  // ring position (stage 0) of this lane's first chunk
    long long fdelta;     // f - u in elements: the same copy sources serve the f ring
    long long brs;        // elements between vertically adjacent blocks
    int ny;
    int r0;               // first input row of the strip
    int in_end;           // one past the last input row that is needed
    int Y0, Y1;           // output rows of this strip
    double cx;            // Dirichlet value for this lane if it is outside the domain in x
    double c_my, c_py;    // Dirichlet values below / above the domain
    bool copy_a, copy_b;  // chunk lies inside the domain
    bool xout, edge_x, store_lane;
};

// start the copy of input row r into its ring stage (nothing to copy outside the domain).  With a
// right-hand side, f row r goes into the f ring (F_RING: stages follow the u stages of the warp),
// or is at least requested into L2 for the loads that follow DEPTH steps later.
template <int P, bool HAS_F, bool F_RING>
__device__ __forceinline__ void issue_row(const TemporalCtx& c, const JacGeom& g, int r, const RowCursor& cur) {
    constexpr int SC = temporal_stage_chunks(P);
    if (r >= 0 && r < c.ny && r < c.in_end) {
        const int st = ((r - c.r0) % kTemporalDepth) * SC;
        if (c.copy_a) g_cp_async16(g, c.dst_a + st, c.src_a + cur.off, KID_TEMPORAL2D);
        if (P == 4 && c.copy_b) g_cp_async16(g, c.dst_b + st, c.src_b + cur.off, KID_TEMPORAL2D);
        if (F_RING) {
            const int fs = (kTemporalDepth + ((r - c.r0) % kTemporalFDepth)) * SC;
            if (c.copy_a) g_cp_async16(g, c.dst_a + fs, c.src_a + c.fdelta + cur.off, KID_TEMPORAL2D);
            if (P == 4 && c.copy_b) g_cp_async16(g, c.dst_b + fs, c.src_b + c.fdelta + cur.off, KID_TEMPORAL2D);
        } else if (HAS_F && !c.xout) {
            prefetch_line(c.fb + cur.off);
        }
    }
    cp_async_commit();
}

// input row r for this lane once its copy has landed
template <int P, bool EDGE>
__device__ __forceinline__ RowN<P> take_row(const TemporalCtx& c, int r) {
    if (EDGE) {   // Dirichlet value outside the domain
        if (r < 0) return fill_rown<P>(c.xout ? c.cx : c.c_my);
        if (r >= c.ny) return fill_rown<P>(c.xout ? c.cx : c.c_py);
        if (c.xout) return fill_rown<P>(c.cx);
    }
    const double2* st = c.mine + ((r - c.r0) % kTemporalDepth) * temporal_stage_chunks(P);
    return load_rown<P>(reinterpret_cast<const double*>(st));
}

__host__ __device__ constexpr int slot3(int ph, int d) { return (((ph + d) % 3) + 3) % 3; }

// level s of one step: row r - s from the window of level s - 1 (input row r has phase PH = (r - r0) mod 3).
// EDGE = false is for steps in which no row and no column involved lies outside the domain: no
// Dirichlet fix-up is compiled in.
template <int T, bool HAS_F, int RES, int PH, bool EDGE, int s>
__device__ __forceinline__ void temporal_level(RowN<temporal_points(T)> (&win)[T][3], const TemporalCtx& c,
                                               const JacGeom& g, int r, const RowCursor& out_cur, double& acc)
{
    constexpr int P = temporal_points(T);
    using Row = RowN<P>;
    static_assert(!HAS_F || temporal_f_ring(T, HAS_F), "the right-hand side travels through its ring");
    constexpr int d = -s;                      // level s produces row r + d
    const int rs = r + d;
    const Row& S = win[s - 1][slot3(PH, d - 1)];
    const Row& M = win[s - 1][slot3(PH, d)];
    const Row& N = win[s - 1][slot3(PH, d + 1)];
    const double w = __shfl_up_sync(0xffffffffu, M.v[P - 1], 1);
    const double e = __shfl_down_sync(0xffffffffu, M.v[0], 1);
    Row ff;
    if (HAS_F) {
        const bool ok = EDGE ? (rs >= 0 && rs < c.ny && !c.xout) : true;
        if (ok) {
            // copied DEPTH + s steps ago; the warp-wide barriers of the steps in between made the
            // other lanes' chunks visible
            const double2* fr = c.mine + (kTemporalDepth + ((rs - c.r0) & (kTemporalFDepth - 1))) *
                                             temporal_stage_chunks(P);
            ff = load_rown<P>(reinterpret_cast<const double*>(fr));
        } else {
            ff = fill_rown<P>(0.0);
        }
    }
    constexpr bool MEASURES = RES == s;
    Row o, res;
#pragma unroll
    for (int q = 0; q < P; ++q) {
        const double W = (q == 0) ? w : M.v[q - 1];
        const double E = (q == P - 1) ? e : M.v[q + 1];
        double sum = add_rn(add_rn(W, E), add_rn(S.v[q], N.v[q]));
        if (HAS_F) sum = add_rn(sum, ff.v[q]);
        o.v[q] = mul_rn(sum, g.quarter);
        // residual of the state this level reads (M is that state at this point)
        if (MEASURES) res.v[q] = sub_rn(sum, mul_rn(4.0, M.v[q]));
    }
    if (EDGE) {
        if (rs < 0) o = fill_rown<P>(c.c_my);
        if (rs >= c.ny) o = fill_rown<P>(c.c_py);
        if (c.xout) o = fill_rown<P>(c.cx);
    }
    const bool in_strip = c.store_lane && rs >= c.Y0 && rs < c.Y1;
    if (s < T) {
        win[s][slot3(PH, d)] = o;
    } else if (in_strip) {
        if (in_bounds(g, c.ob + out_cur.off, 8 * P, CHK_FIELD, KID_TEMPORAL2D)) store_rown<P>(c.ob + out_cur.off, o);
    }
    // the points of the strip's output region: every interior point is in exactly one, and every
    // level is exact there
    if (MEASURES && in_strip) {
#pragma unroll
        for (int q = 0; q < P; ++q) acc = add_rn(acc, mul_rn(res.v[q], res.v[q]));
    }
}

template <int T, bool HAS_F, int RES, int PH, bool EDGE, int s>
struct TemporalLevels {   // levels s, s + 1, ..., T (lowest first: each reads the row the one below has just made)
    static __device__ __forceinline__ void run(RowN<temporal_points(T)> (&win)[T][3], const TemporalCtx& c, const JacGeom& g, int r,
                                               const RowCursor& out_cur, double& acc) {
        temporal_level<T, HAS_F, RES, PH, EDGE, s>(win, c, g, r, out_cur, acc);
        if constexpr (s < T) TemporalLevels<T, HAS_F, RES, PH, EDGE, s + 1>::run(win, c, g, r, out_cur, acc);
    }
};

// One pipeline step: input row r arrives (phase PH = (r - r0) mod 3) and every level advances one
// row, lowest first; then the ring stages that row r and f row r - T have left are refilled.
// EDGE = false is for steps in which no row and no column involved lies outside the domain: no
// Dirichlet fix-up is compiled in.
template <int T, bool HAS_F, int RES, int PH, bool EDGE>
__device__ __forceinline__ void temporal_step(RowN<temporal_points(T)> (&win)[T][3], const TemporalCtx& c, const JacGeom& g,
                                              int r, RowCursor& load_cur, RowCursor& out_cur, double& acc)
{
    constexpr bool F_RING = temporal_f_ring(T, HAS_F);
    cp_async_wait<kTemporalDepth - 1>();
    __syncwarp();                                    // the other lanes' chunks of row r have landed too
    win[0][PH] = take_row<temporal_points(T), EDGE>(c, r);
    TemporalLevels<T, HAS_F, RES, PH, EDGE, 1>::run(win, c, g, r, out_cur, acc);
    __syncwarp();                                    // everyone has read the stages before they are refilled
    issue_row<temporal_points(T), HAS_F, F_RING>(c, g, r + kTemporalDepth, load_cur);
    load_cur.advance(g, c.brs);
    out_cur.advance(g, c.brs);
}

// element offset of global column gx (row 0 of block row 0); gx must be inside the domain
__device__ __forceinline__ long long column_base(const JacGeom& g, long long gx) {
    const long long bxi = gx / g.bx;
    return bxi * g.block_stride + g.origin + (gx - bxi * g.bx);
}

template <int T, bool HAS_F, int RES, int PH>
__device__ __forceinline__ void temporal_step_any(RowN<temporal_points(T)> (&win)[T][3], const TemporalCtx& c, const JacGeom& g,
                                                  int r, RowCursor& load_cur, RowCursor& out_cur, double& acc)
{
    // warp-uniform: does this step see a row outside [0, ny) or a column outside [0, nx)?
    const bool edge = c.edge_x || (r - T - 1 < 0) || (r >= c.ny);
    if (edge) temporal_step<T, HAS_F, RES, PH, true>(win, c, g, r, load_cur, out_cur, acc);
    else temporal_step<T, HAS_F, RES, PH, false>(win, c, g, r, load_cur, out_cur, acc);
}

// RES: level RES (1..T; 0: none) also accumulates the squared residual of the state it reads, the one
// after RES - 1 sweeps of the launch; every warp writes its partial sum to partials[warp id].
template <int T, bool HAS_F, int RES>
__global__ void __launch_bounds__(kTemporalWarps * 32, temporal_ctas_per_sm(T, HAS_F))
temporal2d_kernel(const double* __restrict__ u, double* __restrict__ un, const double* __restrict__ f,
                  double* __restrict__ partials, const JacGeom g, const int strips_x, const int strips_y,
                  const int rows_per_strip)
{
    if (solve_stopped(g)) return;
    extern __shared__ __align__(16) double2 t2_ring_mem[];   // [warp][u stages, then f stages][64]
    constexpr bool F_RING = temporal_f_ring(T, HAS_F);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long wid = (long long)blockIdx.x * kTemporalWarps + warp;
    if (wid >= (long long)strips_x * strips_y) return;   // whole warps only; warps never meet at a barrier
    const int sx = (int)(wid % strips_x), sy = (int)(wid / strips_x);

    TemporalCtx c;
    constexpr int HL = temporal_halo_lanes(T);
    constexpr int P = temporal_points(T);
    constexpr int SC = temporal_stage_chunks(P);
    const long long X0 = (long long)sx * temporal_strip_cols(T) - P * HL;
    const long long gx = X0 + P * lane;
    c.xout = gx < 0 || gx >= g.nx;
    c.cx = gx < 0 ? g.bval[0] : g.bval[1];
    c.c_my = g.bval[2];
    c.c_py = g.bval[3];
    c.edge_x = (sx == 0) || (X0 + 32 * P > g.nx);
    c.store_lane = lane >= HL && lane <= 31 - HL && !c.xout;
    const long long col = c.xout ? g.origin : column_base(g, gx);
    c.fb = HAS_F ? f + col : nullptr;
    c.ob = un + col;
    // copy duty: chunk `lane` (and, with 4 points per lane, chunk `32 + lane`) of every row
    const long long xa = X0 + 2 * lane, xb = X0 + 64 + 2 * lane;
    c.copy_a = xa >= 0 && xa < g.nx;
    c.copy_b = P == 4 && xb >= 0 && xb < g.nx;
    c.src_a = u + (c.copy_a ? column_base(g, xa) : g.origin);
    c.src_b = u + (c.copy_b ? column_base(g, xb) : g.origin);
    double2* ring = t2_ring_mem + warp * temporal_stages_per_warp(T, HAS_F) * SC;
    c.fdelta = HAS_F ? (long long)(f - u) : 0;
    c.dst_a = ring + lane;        // chunk k = lane
    c.dst_b = ring + 32 + lane;   // chunk k = 32 + lane
    c.mine = ring + (P / 2) * lane;   // this lane's own P points: P/2 consecutive chunks
    c.brs = g.block_stride * g.gx;
    c.ny = (int)g.ny;
    c.Y0 = sy * rows_per_strip;
    c.Y1 = min(c.ny, c.Y0 + rows_per_strip);
    c.r0 = c.Y0 - T;
    c.in_end = c.Y1 + T;
    const int r_end = c.Y1 + T;           // the top level trails the input by T rows

    RowN<P> win[T][3];
#pragma unroll
    for (int s = 0; s < T; ++s)
#pragma unroll
        for (int k = 0; k < 3; ++k) win[s][k] = fill_rown<P>(0.0);

    RowCursor load_cur, out_cur;
    load_cur.init(c.r0, g, c.brs);
    out_cur.init(c.r0 - T, g, c.brs);           // row produced by the top level in the first step

    // fill the ring with the first DEPTH rows
#pragma unroll 1
    for (int k = 0; k < kTemporalDepth; ++k) {
        issue_row<P, HAS_F, F_RING>(c, g, c.r0 + k, load_cur);
        load_cur.advance(g, c.brs);
    }

    double acc = 0.0;
    for (int r = c.r0; r < r_end; r += 3) {
        temporal_step_any<T, HAS_F, RES, 0>(win, c, g, r, load_cur, out_cur, acc);
        if (r + 1 < r_end) temporal_step_any<T, HAS_F, RES, 1>(win, c, g, r + 1, load_cur, out_cur, acc);
        if (r + 2 < r_end) temporal_step_any<T, HAS_F, RES, 2>(win, c, g, r + 2, load_cur, out_cur, acc);
    }
    cp_async_wait<0>();
    if (RES != 0) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc = add_rn(acc, __shfl_down_sync(0xffffffffu, acc, off));
        if (lane == 0) g_st(g, partials + wid, acc, CHK_SCRATCH, KID_TEMPORAL2D);
    }
}

}  // namespace jac
