// 3D temporal blocking: T (1..3) sweeps per launch.
//
// A CTA of 16 warps owns a tile of 64 columns x 32 rows and streams it along z.  A lane holds 2
// consecutive points of each of its warp's 2 rows, so a warp covers 64 x 2 points of a plane and
// the CTA the whole tile.  Input plane p enters at level 0; level s (s = 1..T) produces plane p - s
// in the same step, one plane behind the level below, from planes p-s-1, p-s, p-s+1 of level s-1.
//
// Where the data lives:
//   level 0   arrives through a cp.async ring of 4 planes in shared memory (p-1 and p are read, two
//             more are in flight; at T = 3, 5 planes, see t3_l0_in_registers).  A lane copies exactly the 16 bytes it later takes into
//             registers from its own rows, so its own wait makes them visible to it; other warps'
//             rows are read one step later, after the step's barrier.  Cells outside the domain get
//             their Dirichlet value stored into the ring instead of a copy, so readers need no
//             special cases.
//   level s   (0 <= s < T) the lane's own column pair of the three live planes in registers
//             (3 x 2 x 2 doubles per level); the whole middle plane is also in shared memory (level
//             0: the ring; above: a double-buffered plane each level publishes), for the north/south
//             neighbours that belong to other warps.  West/east neighbours come by shuffle.
//   f         a second cp.async ring, T + 2 planes deep: plane q is read by level s at step q + s.
//   level T   goes to global memory.
// One __syncthreads per step.  With 12 doubles of window state per level the kernel stays below 128
// registers, so the SM holds 16 warps; all planes of a step are independent per point, which is
// what covers the latencies.
//
// One column pair per level and side at the tile's x ends and one row per level at its y ends lose
// validity: whole lanes are stored, 60 columns (T <= 2) or 56 (T = 3) x (32 - 2T) rows per plane.
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
constexpr int kT3MaxT = 3;
// Level 0's own column pairs of planes p-2 and p-1 stay in registers up to T = 2; at T = 3 the
// register budget of 128 is spent on the windows of levels 1 and 2, and level 0 is read from the
// ring every time (which then has to keep plane p-2 as well).
__host__ __device__ constexpr bool t3_l0_in_registers(int T) { return T <= 2; }
__host__ __device__ constexpr int t3_u_stages(int T) { return kT3Lead + (t3_l0_in_registers(T) ? 2 : 3); }
__host__ __device__ constexpr int t3_f_stages(int T) { return T + kT3Lead; }
__host__ __device__ constexpr int t3_halo_lanes(int T) { return (T + 1) / 2; }
__host__ __device__ constexpr int t3_out_cols(int T) { return kT3Cols - 4 * t3_halo_lanes(T); }
__host__ __device__ constexpr int t3_out_rows(int T) { return kT3TileRows - 2 * T; }
__host__ __device__ constexpr size_t t3_smem_bytes(int T, bool has_f) {
    return (size_t)(t3_u_stages(T) + (has_f ? t3_f_stages(T) : 0) + 2 * (T - 1)) * kT3Plane * sizeof(double);
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

// plane cursor: element offset of the lane's column in global plane gz, block-aware
struct ZCursor {
    long long off;
    int k;
    __device__ __forceinline__ void init(int gz, const JacGeom& g, long long bsz, long long col) {
        if (gz < 0) { k = gz; off = col + (long long)gz * g.PXY; }
        else {
            const int bzi = gz / g.bz;
            k = gz - bzi * g.bz;
            off = col + bzi * bsz + (long long)k * g.PXY;
        }
    }
    __device__ __forceinline__ void advance(const JacGeom& g, long long bsz) {
        ++k;
        off += g.PXY;
        if (k == g.bz) { k = 0; off += bsz - (long long)g.bz * g.PXY; }
    }
};

// the kernel's dynamic shared memory: [u ring][f ring][published planes of levels 1 .. T-1, two each]
extern __shared__ __align__(16) double t3_smem[];

struct T3 {
    long long row_off[kT3Rows];   // element offset of the warp's rows (rows inside the domain only)
    long long bsz;           // elements between blocks adjacent in z
    int fring, exch;         // offsets of the f ring ([stage][tile row][64]) and of the published
                             // planes ([level - 1][slot][tile row][64]) in t3_smem; the u ring is at 0
    int mine;                // offset of this lane's pair in its warp's first row inside a plane
    int below, above;        // offsets of the pairs one row below / above the warp's rows (clamped to the tile)
    int nz, Z0, Z1;          // planes of the domain; output planes of this chunk
    // per row r of the warp: bit r = below the domain, bit 2 + r = above it, bit 4 + r = an output
    // row of the tile inside the domain; bit 6: the lane's columns lie outside the domain, bit 7:
    // below it (else above), bit 8: the lane's columns are output columns inside the domain
    unsigned bits;
    __device__ __forceinline__ bool row_lo(int r) const { return (bits >> r) & 1u; }
    __device__ __forceinline__ bool row_hi(int r) const { return (bits >> (2 + r)) & 1u; }
    __device__ __forceinline__ bool row_store(int r) const { return (bits >> (4 + r)) & 1u; }
    __device__ __forceinline__ bool xout() const { return (bits >> 6) & 1u; }
    __device__ __forceinline__ bool xlow() const { return (bits >> 7) & 1u; }
    __device__ __forceinline__ bool store_lane() const { return (bits >> 8) & 1u; }
};

// Dirichlet value of a cell outside the domain (plane, then row, then column decide)
__device__ __forceinline__ bool t3_outside(const T3& c, const JacGeom& g, int plane, int r, double* val) {
    if (plane < 0) { *val = g.bval[4]; return true; }
    if (plane >= c.nz) { *val = g.bval[5]; return true; }
    if (c.row_lo(r)) { *val = g.bval[2]; return true; }
    if (c.row_hi(r)) { *val = g.bval[3]; return true; }
    if (c.xout()) { *val = c.xlow() ? g.bval[0] : g.bval[1]; return true; }
    return false;
}

// Start the copies of u plane p (and, with f, of f plane p - 1) into their ring stages: one group.
// Cells outside the domain receive their Dirichlet value by an ordinary store (f: nothing, the
// result there is replaced anyway).
template <int T, bool HAS_F, bool EDGE>
__device__ __forceinline__ void t3_issue(const T3& c, const JacGeom& g, const double* __restrict__ u,
                                         const double* __restrict__ f, int p, int ustage, int fstage,
                                         const ZCursor& cur, long long f_off /* offset of plane p - 1 */) {
    const int in_end = c.Z1 + T, p0 = c.Z0 - T;     // input planes of the chunk
    if (p < in_end) {
        double* st = t3_smem + ustage * kT3Plane + c.mine;
#pragma unroll
        for (int r = 0; r < kT3Rows; ++r) {
            double cval = 0.0;
            if (EDGE && t3_outside(c, g, p, r, &cval)) sts_pair(st + r * kT3Cols, pair_of(cval));
            else g_cp_async16(g, st + r * kT3Cols, u + cur.off + c.row_off[r], KID_TEMPORAL3D);
        }
    }
    if (HAS_F) {
        const int q = p - 1;
        if (q < in_end && q >= p0) {
            double* st = t3_smem + c.fring + fstage * kT3Plane + c.mine;
#pragma unroll
            for (int r = 0; r < kT3Rows; ++r) {
                double cval = 0.0;
                if (!(EDGE && t3_outside(c, g, q, r, &cval))) g_cp_async16(g, st + r * kT3Cols, f + f_off + c.row_off[r], KID_TEMPORAL3D);
            }
        }
    }
    cp_async_commit();
}

// One level: plane q of the level from planes D, M, U of the level below (the lane's own column
// pairs) and the pairs one row below / above the warp's rows in plane M.
// RES: the points flagged in `live` also add the squared residual of M (s - 6 M) to acc.
template <bool HAS_F, bool EDGE, bool RES>
__device__ __forceinline__ void t3_level(const T3& c, const JacGeom& g, const Rows2& D, const Rows2& M, const Rows2& U,
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
        if (EDGE && t3_outside(c, g, q, r, &cval)) o = pair_of(cval);
        out.row[r] = o;
    }
}

// Levels 2..T of one step, lowest first: level s computes plane p - s from the register window of
// level s - 1 (whose newest plane, p - s + 1, was produced a moment ago in this step) and the
// shared copy of that level's plane p - s, which its owners published in the previous step.
template <int T, bool HAS_F, int RES, int PH, bool EDGE, int s>
__device__ __forceinline__ void t3_upper_levels(Rows2 (&win)[kT3MaxT][3], const T3& c, const JacGeom& g,
                                                double* __restrict__ un, int p, int par,
                                                const int (&fst)[kT3MaxT], const ZCursor& out_cur, double& acc)
{
    if constexpr (s <= T) {
        const int q = p - s;
        const Rows2& D = win[s - 1][slot3(PH, -s - 1)];
        const Rows2& M = win[s - 1][slot3(PH, -s)];
        const Rows2& U = win[s - 1][slot3(PH, -s + 1)];
        const double* ex = t3_smem + c.exch + ((s - 2) * 2 + (par ^ 1)) * kT3Plane;    // plane p - s of level s - 1
        const Pair below = lds_pair(ex + c.below);
        const Pair above = lds_pair(ex + c.above);
        const double* fp = HAS_F ? t3_smem + c.fring + fst[s - 1] * kT3Plane + c.mine : nullptr;
        if constexpr (s == T) {
            Rows2 o;
            const bool in_chunk = c.store_lane() && q >= c.Z0 && q < c.Z1;
            const bool live[kT3Rows] = {in_chunk && c.row_store(0), in_chunk && c.row_store(1)};
            t3_level<HAS_F, EDGE, RES == kResBeforeLast>(c, g, D, M, U, below, above, q, fp, o, live, acc);
#pragma unroll
            for (int r = 0; r < kT3Rows; ++r)
                if (live[r]) g_st2(g, un + out_cur.off + c.row_off[r], make_double2(o.row[r].v[0], o.row[r].v[1]), CHK_FIELD, KID_TEMPORAL3D);
        } else {
            Rows2& o = win[s][slot3(PH, -s)];
            const bool none[kT3Rows] = {false, false};
            t3_level<HAS_F, EDGE, false>(c, g, D, M, U, below, above, q, fp, o, none, acc);
            double* pub = t3_smem + c.exch + ((s - 1) * 2 + par) * kT3Plane + c.mine;
#pragma unroll
            for (int r = 0; r < kT3Rows; ++r) sts_pair(pub + r * kT3Cols, o.row[r]);
            t3_upper_levels<T, HAS_F, RES, PH, EDGE, s + 1>(win, c, g, un, p, par, fst, out_cur, acc);
        }
    }
}

// One step: input plane p has been requested LEAD steps ago; every level advances one plane.
// `ust` are the ring stages of planes p-1 and p; `fst[s-1]` the f stage of plane p - s.
template <int T, bool HAS_F, int RES, int PH, bool EDGE>
__device__ __forceinline__ void t3_step(Rows2 (&win)[kT3MaxT][3], const T3& c, const JacGeom& g,
                                        double* __restrict__ un, int p, int par, const int (&ust)[2],
                                        const int (&fst)[kT3MaxT], const ZCursor& out_cur, double& acc)
{
    // ---- level 0: this lane's pairs of plane p join the window (planes p-2 and p-1 are there
    // already, or are read from the ring again)
    constexpr bool L0REG = t3_l0_in_registers(T);
    constexpr int NUS = t3_u_stages(T);
    {
        const double* su = t3_smem + ust[1] * kT3Plane + c.mine;
#pragma unroll
        for (int r = 0; r < kT3Rows; ++r) win[0][PH].row[r] = lds_pair(su + r * kT3Cols);
        if constexpr (!L0REG) {
            const int sd_stage = ust[0] >= 1 ? ust[0] - 1 : ust[0] + NUS - 1;     // plane p - 2
            const double* sd = t3_smem + sd_stage * kT3Plane + c.mine;
            const double* s1 = t3_smem + ust[0] * kT3Plane + c.mine;
#pragma unroll
            for (int r = 0; r < kT3Rows; ++r) {
                win[0][slot3(PH, -2)].row[r] = lds_pair(sd + r * kT3Cols);
                win[0][slot3(PH, -1)].row[r] = lds_pair(s1 + r * kT3Cols);
            }
        }
    }
    // ---- level 1: plane p - 1 from level-0 planes p-2, p-1, p
    const int q = p - 1;
    const Rows2& D = win[0][slot3(PH, -2)];
    const Rows2& M = win[0][slot3(PH, -1)];
    const Rows2& U = win[0][PH];
    const double* sm = t3_smem + ust[0] * kT3Plane;
    const Pair below = lds_pair(sm + c.below);
    const Pair above = lds_pair(sm + c.above);
    const double* fp = HAS_F ? t3_smem + c.fring + fst[0] * kT3Plane + c.mine : nullptr;
    if constexpr (T == 1) {
        Rows2 o;
        const bool in_chunk = c.store_lane() && q >= c.Z0 && q < c.Z1;
        const bool live[kT3Rows] = {in_chunk && c.row_store(0), in_chunk && c.row_store(1)};
        t3_level<HAS_F, EDGE, RES != kResNone>(c, g, D, M, U, below, above, q, fp, o, live, acc);
#pragma unroll
        for (int r = 0; r < kT3Rows; ++r)
            if (live[r]) g_st2(g, un + out_cur.off + c.row_off[r], make_double2(o.row[r].v[0], o.row[r].v[1]), CHK_FIELD, KID_TEMPORAL3D);
    } else {
        Rows2& o = win[1][slot3(PH, -1)];
        // the residual of the state the launch reads: over the tile's output cells, which every
        // interior point is in exactly once, and where level 1 is exact
        const bool in_tile = RES == kResOfInput && c.store_lane() && q >= c.Z0 && q < c.Z1;
        const bool live[kT3Rows] = {in_tile && c.row_store(0), in_tile && c.row_store(1)};
        t3_level<HAS_F, EDGE, RES == kResOfInput>(c, g, D, M, U, below, above, q, fp, o, live, acc);
        double* pub = t3_smem + c.exch + par * kT3Plane + c.mine;
#pragma unroll
        for (int r = 0; r < kT3Rows; ++r) sts_pair(pub + r * kT3Cols, o.row[r]);
        t3_upper_levels<T, HAS_F, RES, PH, EDGE, 2>(win, c, g, un, p, par, fst, out_cur, acc);
    }
}

// RES: partials[CTA * 16 + warp] gets the warp's sum of squared residuals over exactly the points
// the warp stores -- of the state before the last sweep of the launch (kResBeforeLast) or of the
// state the launch reads (kResOfInput).
template <int T, bool HAS_F, int RES>
__global__ void __launch_bounds__(kT3Warps * 32, 1)
temporal3d_kernel(const double* __restrict__ u, double* __restrict__ un, const double* __restrict__ f,
                  double* __restrict__ partials, const JacGeom g, const int tiles_x, const int tiles_y,
                  const int tiles_z, const int zchunk)
{
    if (solve_stopped(g)) return;
    constexpr int NFS = t3_f_stages(T);
    constexpr int NUS = t3_u_stages(T);
    T3 c;
    c.fring = t3_u_stages(T) * kT3Plane;
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
    const bool xout = gx < 0 || gx >= g.nx;
    c.bits = (xout ? 1u << 6 : 0u) | (gx < 0 ? 1u << 7 : 0u) | ((lane >= HL && lane <= 31 - HL && !xout) ? 1u << 8 : 0u);
    const long long col = xout ? g.origin : column_base(g, gx);

    const int Yt0 = sy * t3_out_rows(T) - T;                 // global row of tile row 0
    const long long bsy = g.block_stride * g.gx;
    c.bsz = bsy * g.gy;
    const int trow0 = warp * kT3Rows;
#pragma unroll
    for (int r = 0; r < kT3Rows; ++r) {
        const int trow = trow0 + r;
        const long long gy = (long long)Yt0 + trow;
        c.row_off[r] = 0;
        if (gy < 0) c.bits |= 1u << r;
        else if (gy >= g.ny) c.bits |= 1u << (2 + r);
        else {
            const long long byi = gy / g.by;
            c.row_off[r] = byi * bsy + (gy - byi * g.by) * g.PX;
            if (trow >= T && trow < kT3TileRows - T) c.bits |= 1u << (4 + r);
        }
    }
    c.mine = trow0 * kT3Cols + 2 * lane;
    c.below = max(trow0 - 1, 0) * kT3Cols + 2 * lane;
    c.above = min(trow0 + kT3Rows, kT3TileRows - 1) * kT3Cols + 2 * lane;
    c.nz = (int)g.nz;
    c.Z0 = sz * zchunk;
    c.Z1 = min(c.nz, c.Z0 + zchunk);
    const int p0 = c.Z0 - T;             // first input plane; the last one is Z1 + T - 1, and
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

    Rows2 win[kT3MaxT][3];     // [level][plane mod 3]; only levels 0 .. T-1 are used
#pragma unroll
    for (int s = 0; s < kT3MaxT; ++s)
#pragma unroll
        for (int k = 0; k < 3; ++k)
#pragma unroll
            for (int r = 0; r < kT3Rows; ++r) win[s][k].row[r] = pair_of(0.0);

    ZCursor load_cur, out_cur;
    load_cur.init(p0, g, c.bsz, col);
    long long f_off = 0;                    // the f plane that travels with u plane p is p - 1: the
                                            // offset the load cursor had one step earlier
    out_cur.init(p0 - T, g, c.bsz, col);   // output plane of level T in the first step
    // ring positions: plane p sits in u stage (p - p0) mod 5 and f stage (p - p0) mod NFS
#pragma unroll 1
    for (int k = 0; k < kT3Lead; ++k) {
        const int us = k, fs = k == 0 ? NFS - 1 : k - 1;
        const bool edge = edge_xy || (p0 + k - 1 < 0) || (p0 + k >= c.nz);
        if (edge) t3_issue<T, HAS_F, true>(c, g, u, f, p0 + k, us, fs, load_cur, f_off);
        else t3_issue<T, HAS_F, false>(c, g, u, f, p0 + k, us, fs, load_cur, f_off);
        f_off = load_cur.off;
        load_cur.advance(g, c.bsz);
    }

    double acc = 0.0;
    int cons = 0;        // u stage of plane p (the one consumed as U in this step)
    int fcons = NFS - 1; // f stage of plane p - 1

#define JAC_T3_STEP(PHASE, PL)                                                                          \
    do {                                                                                                \
        const int p_ = (PL);                                                                            \
        const bool edge = edge_xy || (p_ - T - 1 < 0) || (p_ + kT3Lead >= c.nz);                        \
        /* request plane p + LEAD into the stage that the oldest plane has left (last read one step ago) */ \
        const int us = cons + kT3Lead >= NUS ? cons + kT3Lead - NUS : cons + kT3Lead;                   \
        const int fs = fcons + kT3Lead >= NFS ? fcons + kT3Lead - NFS : fcons + kT3Lead;                \
        const int par = (p_ - p0) & 1;                                                                  \
        if (edge) t3_issue<T, HAS_F, true>(c, g, u, f, p_ + kT3Lead, us, fs, load_cur, f_off);             \
        else t3_issue<T, HAS_F, false>(c, g, u, f, p_ + kT3Lead, us, fs, load_cur, f_off);                 \
        f_off = load_cur.off;                                                                           \
        load_cur.advance(g, c.bsz);                                                                     \
        cp_async_wait<kT3Lead>();                       /* this lane's part of plane p has landed */    \
        const int ust[2] = {cons >= 1 ? cons - 1 : cons + NUS - 1, cons};                               \
        int fst[kT3MaxT];                                                                               \
        _Pragma("unroll") for (int s_ = 0; s_ < kT3MaxT; ++s_) {                                        \
            const int v = fcons - s_;                                                                   \
            fst[s_] = v < 0 ? v + NFS : v;                                                              \
        }                                                                                               \
        if (edge) t3_step<T, HAS_F, RES, PHASE, true>(win, c, g, un, p_, par, ust, fst, out_cur, acc);     \
        else t3_step<T, HAS_F, RES, PHASE, false>(win, c, g, un, p_, par, ust, fst, out_cur, acc);         \
        out_cur.advance(g, c.bsz);                                                                      \
        cons = cons + 1 == NUS ? 0 : cons + 1;                                                          \
        fcons = fcons + 1 == NFS ? 0 : fcons + 1;                                                       \
        __syncthreads();                                                                                \
    } while (0)

    for (int p = p0; p < p_end; p += 3) {
        JAC_T3_STEP(0, p);
        if (p + 1 < p_end) JAC_T3_STEP(1, p + 1);
        if (p + 2 < p_end) JAC_T3_STEP(2, p + 2);
    }
#undef JAC_T3_STEP
    cp_async_wait<0>();
    if (RES != kResNone) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc = add_rn(acc, __shfl_down_sync(0xffffffffu, acc, off));
        if (lane == 0) g_st(g, partials + (long long)blockIdx.x * kT3Warps + warp, acc, CHK_SCRATCH, KID_TEMPORAL3D);
    }
}

}  // namespace jac
