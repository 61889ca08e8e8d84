// 3D temporal blocking: T (1..4) sweeps per launch.
//
// A CTA of 16 warps owns a tile of 64 columns x 32 rows and streams it along z.  A lane holds 2
// consecutive points of each of its warp's 2 rows, so a warp covers 64 x 2 points of a plane and
// the CTA the whole tile.  Input plane p enters at level 0; level s (s = 1..T) produces plane p - s
// in the same step, one plane behind the level below, from planes p-s-1, p-s, p-s+1 of level s-1.
//
// Where the data lives:
//   level 0   only in shared memory: a cp.async ring of 5 planes (p-2, p-1, p are read, two more
//             are in flight).  A lane copies exactly the 16 bytes it later reads from its own rows,
//             so its own wait makes them visible to it; other warps' rows are read one step later,
//             after the step's barrier.  Cells outside the domain get their Dirichlet value
//             stored into the ring instead of a copy, so readers need no special cases.
//   level s   (0 < s < T) the lane's own column pair of the three live planes in registers
//             (3 x 2 x 2 doubles per level), and the whole middle plane once more in a
//             double-buffered shared-memory plane, for the north/south neighbours that belong to
//             other warps.  West/east neighbours come by shuffle.
//   f         a second cp.async ring, T + 2 planes deep: plane q is read by level s at step q + s.
//   level T   goes to global memory.
// One __syncthreads per step.  With 12 doubles of window state per level the kernel stays below 128
// registers, so the SM holds 16 warps; all planes of a step are independent per point, which is
// what covers the latencies.
//
// One column pair per level and side at the tile's x ends and one row per level at its y ends lose
// validity: whole lanes are stored, 60 columns (T <= 2) or 56 (T <= 4) x (32 - 2T) rows per plane.
// Tiles read across block borders directly (the neighbour block's interior is the halo), which is
// what an exchange before every sweep delivers.  Requires bx % 2 == 0 and nx % 2 == 0.
#pragma once
#include <cuda_runtime.h>

#include "jac_geom.h"
#include "jac_kernels.cuh"

namespace jac {

constexpr int kT3Warps = 16;                       // warps per CTA, stacked along y
constexpr int kT3Rows = 2;                         // rows per warp
constexpr int kT3TileRows = kT3Warps * kT3Rows;    // 32
constexpr int kT3Cols = 64;
constexpr int kT3Plane = kT3TileRows * kT3Cols;    // doubles per plane of the tile (16 KB)
constexpr int kT3Lead = 2;                         // input planes in flight ahead of the one consumed
constexpr int kT3Stages = kT3Lead + 3;             // u ring
constexpr int kT3MaxT = 4;
__host__ __device__ constexpr int t3_f_stages(int T) { return T + kT3Lead; }
__host__ __device__ constexpr int t3_halo_lanes(int T) { return (T + 1) / 2; }
__host__ __device__ constexpr int t3_out_cols(int T) { return kT3Cols - 4 * t3_halo_lanes(T); }
__host__ __device__ constexpr int t3_out_rows(int T) { return kT3TileRows - 2 * T; }
__host__ __device__ constexpr size_t t3_smem_bytes(int T, bool has_f) {
    return (size_t)(kT3Stages + (has_f ? t3_f_stages(T) : 0) + 2 * (T - 1)) * kT3Plane * sizeof(double);
}

struct Pair { double v[2]; };
__device__ __forceinline__ Pair pair_of(double c) { Pair r; r.v[0] = r.v[1] = c; return r; }
__device__ __forceinline__ Pair lds_pair(const double* p) {
    const double2 a = *reinterpret_cast<const double2*>(p);
    Pair r; r.v[0] = a.x; r.v[1] = a.y; return r;
}
__device__ __forceinline__ void sts_pair(double* p, const Pair& a) {
    *reinterpret_cast<double2*>(p) = make_double2(a.v[0], a.v[1]);
}

// the lane's column pair of its warp's rows in one plane
struct Rows2 { Pair row[kT3Rows]; };

// plane cursor: element offset of global plane gz, block-aware
struct ZCursor {
    long long off;
    int k;
    __device__ __forceinline__ void init(int gz, const JacGeom& g, long long bsz) {
        if (gz < 0) { k = gz; off = (long long)gz * g.PXY; }
        else {
            const int bzi = gz / g.bz;
            k = gz - bzi * g.bz;
            off = bzi * bsz + (long long)k * g.PXY;
        }
    }
    __device__ __forceinline__ void advance(const JacGeom& g, long long bsz) {
        ++k;
        off += g.PXY;
        if (k == g.bz) { k = 0; off += bsz - (long long)g.bz * g.PXY; }
    }
};

struct T3 {
    const double* ub;        // u + lane column base
    const double* fb;
    double* ob;
    long long row_off[kT3Rows];   // element offset of the warp's rows (rows inside the domain only)
    long long bsz;           // elements between blocks adjacent in z
    double* ring;            // shared: [stage][tile row][64]
    double* fring;           // shared: [stage][tile row][64]
    double* exch;            // shared: [level - 1][slot][tile row][64]
    int mine;                // offset of this lane's pair in its warp's first row inside a plane
    int below, above;        // offsets of the pairs one row below / above the warp's rows (clamped to the tile)
    int nz, p0, in_end, Z0, Z1;
    bool row_lo[kT3Rows], row_hi[kT3Rows];   // row lies below / above the domain
    bool row_store[kT3Rows];                 // row is an output row of the tile, inside the domain
    double cx, c_my, c_py, c_mz, c_pz;
    bool xout, store_lane;
};

// Dirichlet value of a cell outside the domain (plane, then row, then column decide)
__device__ __forceinline__ bool t3_outside(const T3& c, int plane, int r, double* val) {
    if (plane < 0) { *val = c.c_mz; return true; }
    if (plane >= c.nz) { *val = c.c_pz; return true; }
    if (c.row_lo[r]) { *val = c.c_my; return true; }
    if (c.row_hi[r]) { *val = c.c_py; return true; }
    if (c.xout) { *val = c.cx; return true; }
    return false;
}

// Start the copies of u plane p (and, with f, of f plane p - 1) into their ring stages: one group.
// Cells outside the domain receive their Dirichlet value by an ordinary store (f: nothing, the
// result there is replaced anyway).
template <int T, bool HAS_F, bool EDGE>
__device__ __forceinline__ void t3_issue(const T3& c, int p, int ustage, int fstage, const ZCursor& cur,
                                         const ZCursor& fcur) {
    if (p < c.in_end) {
        double* st = c.ring + ustage * kT3Plane + c.mine;
#pragma unroll
        for (int r = 0; r < kT3Rows; ++r) {
            double cval = 0.0;
            if (EDGE && t3_outside(c, p, r, &cval)) sts_pair(st + r * kT3Cols, pair_of(cval));
            else cp_async16(st + r * kT3Cols, c.ub + cur.off + c.row_off[r]);
        }
    }
    if (HAS_F) {
        const int q = p - 1;
        if (q < c.in_end && q >= c.p0) {
            double* st = c.fring + fstage * kT3Plane + c.mine;
#pragma unroll
            for (int r = 0; r < kT3Rows; ++r) {
                double cval = 0.0;
                if (!(EDGE && t3_outside(c, q, r, &cval))) cp_async16(st + r * kT3Cols, c.fb + fcur.off + c.row_off[r]);
            }
        }
    }
    cp_async_commit();
}

// One level: plane q of the level from planes D, M, U of the level below (the lane's own column
// pairs) and the pairs one row below / above the warp's rows in plane M.
// RES: the points flagged in `live` also add the squared residual of M (s - 6 M) to acc.
template <bool HAS_F, bool EDGE, bool RES>
__device__ __forceinline__ void t3_level(const T3& c, const Rows2& D, const Rows2& M, const Rows2& U,
                                         const Pair& below, const Pair& above, int q,
                                         const double* fplane /* this lane's pair in row 0 of the warp, f plane q */,
                                         Rows2& out, const bool (&live)[kT3Rows], double& acc)
{
    const double c6 = 1.0 / 6.0;
#pragma unroll
    for (int r = 0; r < kT3Rows; ++r) {
        const Pair& S = (r == 0) ? below : M.row[r - 1];
        const Pair& N = (r == kT3Rows - 1) ? above : M.row[r + 1];
        const double w = __shfl_up_sync(0xffffffffu, M.row[r].v[1], 1);
        const double e = __shfl_down_sync(0xffffffffu, M.row[r].v[0], 1);
        Pair ff = pair_of(0.0);
        if (HAS_F) ff = lds_pair(fplane + r * kT3Cols);
        Pair o;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const double W = (i == 0) ? w : M.row[r].v[0];
            const double E = (i == 1) ? e : M.row[r].v[1];
            double s = add_rn(add_rn(W, E), add_rn(S.v[i], N.v[i]));
            s = add_rn(s, add_rn(D.row[r].v[i], U.row[r].v[i]));
            if (HAS_F) s = add_rn(s, ff.v[i]);
            o.v[i] = mul_rn(s, c6);
            if (RES && live[r]) {
                const double rr = sub_rn(s, mul_rn(6.0, M.row[r].v[i]));
                acc = add_rn(acc, mul_rn(rr, rr));
            }
        }
        double cval = 0.0;
        if (EDGE && t3_outside(c, q, r, &cval)) o = pair_of(cval);
        out.row[r] = o;
    }
}

// Levels 2..T of one step, lowest first: level s computes plane p - s from the register window of
// level s - 1 (whose newest plane, p - s + 1, was produced a moment ago in this step) and the
// shared copy of that level's plane p - s, which its owners published in the previous step.
template <int T, bool HAS_F, bool RES, int PH, bool EDGE, int s>
__device__ __forceinline__ void t3_upper_levels(Rows2 (&win)[kT3MaxT - 1][3], const T3& c, int p, int par,
                                                const int (&fst)[kT3MaxT], const ZCursor& out_cur, double& acc)
{
    if constexpr (s <= T) {
        const int q = p - s;
        const Rows2& D = win[s - 2][slot3(PH, -s - 1)];
        const Rows2& M = win[s - 2][slot3(PH, -s)];
        const Rows2& U = win[s - 2][slot3(PH, -s + 1)];
        const double* ex = c.exch + ((s - 2) * 2 + (par ^ 1)) * kT3Plane;    // plane p - s of level s - 1
        const Pair below = lds_pair(ex + c.below);
        const Pair above = lds_pair(ex + c.above);
        const double* fp = HAS_F ? c.fring + fst[s - 1] * kT3Plane + c.mine : nullptr;
        if constexpr (s == T) {
            Rows2 o;
            const bool in_chunk = c.store_lane && q >= c.Z0 && q < c.Z1;
            const bool live[kT3Rows] = {in_chunk && c.row_store[0], in_chunk && c.row_store[1]};
            t3_level<HAS_F, EDGE, RES>(c, D, M, U, below, above, q, fp, o, live, acc);
#pragma unroll
            for (int r = 0; r < kT3Rows; ++r)
                if (live[r]) sts_pair(c.ob + out_cur.off + c.row_off[r], o.row[r]);
        } else {
            Rows2& o = win[s - 1][slot3(PH, -s)];
            const bool none[kT3Rows] = {false, false};
            t3_level<HAS_F, EDGE, false>(c, D, M, U, below, above, q, fp, o, none, acc);
            double* pub = c.exch + ((s - 1) * 2 + par) * kT3Plane + c.mine;
#pragma unroll
            for (int r = 0; r < kT3Rows; ++r) sts_pair(pub + r * kT3Cols, o.row[r]);
            t3_upper_levels<T, HAS_F, RES, PH, EDGE, s + 1>(win, c, p, par, fst, out_cur, acc);
        }
    }
}

// One step: input plane p has been requested LEAD steps ago; every level advances one plane.
// `ust` are the ring stages of planes p-2, p-1, p; `fst[s-1]` the f stage of plane p - s.
template <int T, bool HAS_F, bool RES, int PH, bool EDGE>
__device__ __forceinline__ void t3_step(Rows2 (&win)[kT3MaxT - 1][3], const T3& c, int p, int par,
                                        const int (&ust)[3], const int (&fst)[kT3MaxT], const ZCursor& out_cur,
                                        double& acc)
{
    // ---- level 1: plane p - 1 from level-0 planes p-2, p-1, p in the ring
    const int q = p - 1;
    Rows2 D, M, U;
    const double* sd = c.ring + ust[0] * kT3Plane + c.mine;
    const double* sm = c.ring + ust[1] * kT3Plane;
    const double* su = c.ring + ust[2] * kT3Plane + c.mine;
#pragma unroll
    for (int r = 0; r < kT3Rows; ++r) {
        D.row[r] = lds_pair(sd + r * kT3Cols);
        M.row[r] = lds_pair(sm + c.mine + r * kT3Cols);
        U.row[r] = lds_pair(su + r * kT3Cols);
    }
    const Pair below = lds_pair(sm + c.below);
    const Pair above = lds_pair(sm + c.above);
    const double* fp = HAS_F ? c.fring + fst[0] * kT3Plane + c.mine : nullptr;
    if constexpr (T == 1) {
        Rows2 o;
        const bool in_chunk = c.store_lane && q >= c.Z0 && q < c.Z1;
        const bool live[kT3Rows] = {in_chunk && c.row_store[0], in_chunk && c.row_store[1]};
        t3_level<HAS_F, EDGE, RES>(c, D, M, U, below, above, q, fp, o, live, acc);
#pragma unroll
        for (int r = 0; r < kT3Rows; ++r)
            if (live[r]) sts_pair(c.ob + out_cur.off + c.row_off[r], o.row[r]);
    } else {
        Rows2& o = win[0][slot3(PH, -1)];
        const bool none[kT3Rows] = {false, false};
        t3_level<HAS_F, EDGE, false>(c, D, M, U, below, above, q, fp, o, none, acc);
        double* pub = c.exch + par * kT3Plane + c.mine;
#pragma unroll
        for (int r = 0; r < kT3Rows; ++r) sts_pair(pub + r * kT3Cols, o.row[r]);
        t3_upper_levels<T, HAS_F, RES, PH, EDGE, 2>(win, c, p, par, fst, out_cur, acc);
    }
}

// RES: partials[CTA * 16 + warp] gets the warp's sum of squared residuals of the state before the
// last sweep of the launch, over exactly the points the warp stores.
template <int T, bool HAS_F, bool RES>
__global__ void __launch_bounds__(kT3Warps * 32, 1)
temporal3d_kernel(const double* __restrict__ u, double* __restrict__ un, const double* __restrict__ f,
                  double* __restrict__ partials, const JacGeom g, const int tiles_x, const int tiles_y,
                  const int tiles_z, const int zchunk)
{
    extern __shared__ __align__(16) double t3_smem[];
    constexpr int NFS = t3_f_stages(T);
    T3 c;
    c.ring = t3_smem;
    c.fring = t3_smem + kT3Stages * kT3Plane;
    c.exch = c.fring + (HAS_F ? NFS : 0) * kT3Plane;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long tix = blockIdx.x;
    const int sx = (int)(tix % tiles_x);
    const int sy = (int)((tix / tiles_x) % tiles_y);
    const int sz = (int)(tix / ((long long)tiles_x * tiles_y));
    (void)tiles_z;

    constexpr int HL = t3_halo_lanes(T);
    const long long X0 = (long long)sx * t3_out_cols(T) - 2 * HL;
    const long long gx = X0 + 2 * lane;
    c.xout = gx < 0 || gx >= g.nx;
    c.cx = gx < 0 ? g.bval[0] : g.bval[1];
    c.c_my = g.bval[2]; c.c_py = g.bval[3]; c.c_mz = g.bval[4]; c.c_pz = g.bval[5];
    c.store_lane = lane >= HL && lane <= 31 - HL && !c.xout;
    const long long col = c.xout ? g.origin : column_base(g, gx);
    c.ub = u + col;
    c.fb = HAS_F ? f + col : nullptr;
    c.ob = un + col;

    const int Yt0 = sy * t3_out_rows(T) - T;                 // global row of tile row 0
    const long long bsy = g.block_stride * g.gx;
    c.bsz = bsy * g.gy;
    const int trow0 = warp * kT3Rows;
#pragma unroll
    for (int r = 0; r < kT3Rows; ++r) {
        const int trow = trow0 + r;
        const long long gy = (long long)Yt0 + trow;
        c.row_lo[r] = gy < 0;
        c.row_hi[r] = gy >= g.ny;
        c.row_off[r] = 0;
        c.row_store[r] = false;
        if (!c.row_lo[r] && !c.row_hi[r]) {
            const long long byi = gy / g.by;
            c.row_off[r] = byi * bsy + (gy - byi * g.by) * g.PX;
            c.row_store[r] = trow >= T && trow < kT3TileRows - T;
        }
    }
    c.mine = trow0 * kT3Cols + 2 * lane;
    c.below = max(trow0 - 1, 0) * kT3Cols + 2 * lane;
    c.above = min(trow0 + kT3Rows, kT3TileRows - 1) * kT3Cols + 2 * lane;
    c.nz = (int)g.nz;
    c.Z0 = sz * zchunk;
    c.Z1 = min(c.nz, c.Z0 + zchunk);
    c.p0 = c.Z0 - T;                     // first input plane
    c.in_end = c.Z1 + T;                 // one past the last input plane
    const int p_end = c.Z1 + T;          // level T trails the input by T planes

    // does this tile ever see a cell outside the domain in x or y?  (z is checked per step)
    const bool edge_xy = (sx == 0) || (X0 + kT3Cols > g.nx) || (Yt0 < 0) || ((long long)Yt0 + kT3TileRows > g.ny);

    // defined contents everywhere: the first steps read planes nobody has written yet (their results
    // only reach cells that are never stored)
    {
        double2* z = reinterpret_cast<double2*>(t3_smem);
        const int n2 = (int)(t3_smem_bytes(T, HAS_F) / sizeof(double2));
        for (int i = threadIdx.x; i < n2; i += blockDim.x) z[i] = make_double2(0.0, 0.0);
    }
    __syncthreads();

    Rows2 win[kT3MaxT - 1][3];
#pragma unroll
    for (int s = 0; s < kT3MaxT - 1; ++s)
#pragma unroll
        for (int k = 0; k < 3; ++k)
#pragma unroll
            for (int r = 0; r < kT3Rows; ++r) win[s][k].row[r] = pair_of(0.0);

    ZCursor load_cur, fload_cur, out_cur;
    load_cur.init(c.p0, g, c.bsz);
    fload_cur.init(c.p0 - 1, g, c.bsz);    // the f plane that travels with u plane p is p - 1
    out_cur.init(c.p0 - T, g, c.bsz);      // output plane of level T in the first step
    // ring positions: plane p sits in u stage (p - p0) mod 5 and f stage (p - p0) mod NFS
    int us = 0;                             // u stage of the plane that is requested next
    int fs = NFS - 1;                       // f stage of plane p0 - 1 (never copied)
#pragma unroll 1
    for (int k = 0; k < kT3Lead; ++k) {
        const bool edge = edge_xy || (c.p0 + k - 1 < 0) || (c.p0 + k >= c.nz);
        if (edge) t3_issue<T, HAS_F, true>(c, c.p0 + k, us, fs, load_cur, fload_cur);
        else t3_issue<T, HAS_F, false>(c, c.p0 + k, us, fs, load_cur, fload_cur);
        load_cur.advance(g, c.bsz);
        if (HAS_F) fload_cur.advance(g, c.bsz);
        us = us + 1 == kT3Stages ? 0 : us + 1;
        fs = fs + 1 == NFS ? 0 : fs + 1;
    }

    double acc = 0.0;
    int cons = 0;        // u stage of plane p (the one consumed as U in this step)
    int fcons = NFS - 1; // f stage of plane p - 1
    int par = 0;

#define JAC_T3_STEP(PHASE, PL)                                                                          \
    do {                                                                                                \
        const int p_ = (PL);                                                                            \
        const bool edge = edge_xy || (p_ - T - 1 < 0) || (p_ + kT3Lead >= c.nz);                        \
        /* request plane p + LEAD into the stage plane p - 3 has left (last read one step ago) */       \
        if (edge) t3_issue<T, HAS_F, true>(c, p_ + kT3Lead, us, fs, load_cur, fload_cur);               \
        else t3_issue<T, HAS_F, false>(c, p_ + kT3Lead, us, fs, load_cur, fload_cur);                   \
        load_cur.advance(g, c.bsz);                                                                     \
        if (HAS_F) fload_cur.advance(g, c.bsz);                                                         \
        us = us + 1 == kT3Stages ? 0 : us + 1;                                                          \
        fs = fs + 1 == NFS ? 0 : fs + 1;                                                                \
        cp_async_wait<kT3Lead>();                       /* this lane's part of plane p has landed */    \
        const int ust[3] = {cons >= 2 ? cons - 2 : cons + kT3Stages - 2,                                \
                            cons >= 1 ? cons - 1 : cons + kT3Stages - 1, cons};                         \
        int fst[kT3MaxT];                                                                               \
        _Pragma("unroll") for (int s_ = 0; s_ < kT3MaxT; ++s_) {                                        \
            const int v = fcons - s_;                                                                   \
            fst[s_] = v < 0 ? v + NFS : v;                                                              \
        }                                                                                               \
        if (edge) t3_step<T, HAS_F, RES, PHASE, true>(win, c, p_, par, ust, fst, out_cur, acc);         \
        else t3_step<T, HAS_F, RES, PHASE, false>(win, c, p_, par, ust, fst, out_cur, acc);             \
        out_cur.advance(g, c.bsz);                                                                      \
        cons = cons + 1 == kT3Stages ? 0 : cons + 1;                                                    \
        fcons = fcons + 1 == NFS ? 0 : fcons + 1;                                                       \
        par ^= 1;                                                                                       \
        __syncthreads();                                                                                \
    } while (0)

    for (int p = c.p0; p < p_end; p += 3) {
        JAC_T3_STEP(0, p);
        if (p + 1 < p_end) JAC_T3_STEP(1, p + 1);
        if (p + 2 < p_end) JAC_T3_STEP(2, p + 2);
    }
#undef JAC_T3_STEP
    cp_async_wait<0>();
    if (RES) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc = add_rn(acc, __shfl_down_sync(0xffffffffu, acc, off));
        if (lane == 0) partials[(long long)blockIdx.x * kT3Warps + warp] = acc;
    }
}

}  // namespace jac
