// 3D temporal blocking: T (1..3) sweeps per launch.
//
// A CTA of 12 warps owns a tile of 64 columns x 24 rows and streams it along z.  A lane holds 2
// consecutive points of each of its warp's 2 rows, so a warp covers 64 x 2 points of a plane and
// the CTA the whole tile.  Input plane p enters at level 0; level s (s = 1..T) produces plane p - s
// in the same step, one plane behind the level below, from planes p-s-1, p-s, p-s+1 of level s-1.
//
// Where the data lives:
//   level 0   arrives through a cp.async ring of 6 planes in shared memory (p-1 and p are read,
//             three more are in flight).  A lane copies exactly the 16 bytes it later takes into
//             registers from its own rows, so its own wait makes them visible to it; other warps'
//             rows are read one step later, after the step's barrier.  Cells outside the domain get
//             their Dirichlet value stored into the ring instead of a copy, so readers need no
//             special cases.
//   level s   (0 <= s < T) the lane's own column pairs of the two planes that live on from step to
//             step, and of the one just made, in registers (3 x 2 x 2 doubles per level).  The
//             first and last row of every warp are also in shared memory for the warps next to it
//             (level 0: they are in the ring; above: a double-buffered array of 2 rows per warp that
//             the level publishes).  West/east neighbours come by shuffle.
//   f         a second cp.async ring of 6 planes: plane q is read by level s at step q + s.
//   level T   goes to global memory.
// One __syncthreads per step.
//
// Both rings have 6 stages and the loop over planes is unrolled 6 times, so every ring position,
// window slot (period 3) and buffer parity (period 2) is a compile-time constant: a step computes
// no ring index and forms every shared-memory address as one per-lane base plus an immediate.
// With 12 doubles of window state per level the kernel needs at most 168 registers, which is what
// 12 warps leave each thread; no variant spills.
//
// One column pair per level and side at the tile's x ends and one row per level at its y ends lose
// validity: whole lanes are stored, 60 columns (T <= 2) or 56 (T = 3) x (24 - 2T) rows per plane.
// Tiles read across block borders directly (the neighbour block's interior is the halo), which is
// what an exchange before every sweep delivers.  Requires bx % 2 == 0 and nx % 2 == 0.
//
// Shapes that were measured and lost (1024^3 with f, T = 3, ms per launch; this one: 7.78):
// 16 warps x 2 rows with ring positions computed per step and level 0 re-read from the ring, 7.97;
// 8 warps x 4 rows, 8.69 (two warps per scheduler cannot cover the shared-memory latencies, and the
// 6-fold unrolled code no longer fits the instruction cache); 14 warps x 2 rows, 12.1 (144
// registers: spills); fetching the next level's shared-memory inputs before computing a level, 7.95;
// per-warp mbarriers between neighbouring warps instead of the CTA barrier, 8.34.
#pragma once
#include <cuda_runtime.h>

#include "jac_geom.h"
#include "jac_kernels.cuh"

namespace jac {

constexpr int kT3Warps = 12;                       // warps per CTA, stacked along y
constexpr int kT3Rows = 2;                         // rows per warp
constexpr int kT3TileRows = kT3Warps * kT3Rows;    // 24
constexpr int kT3Cols = 64;
constexpr int kT3Plane = kT3TileRows * kT3Cols;    // doubles per plane of the tile (12 KB)
constexpr int kT3Lead = 3;                         // input planes in flight ahead of the one consumed
constexpr int kT3Ring = 6;                         // stages of the u ring and of the f ring
constexpr int kT3Pub = kT3Warps * 2 * kT3Cols;     // doubles of one published plane: the first and the last row of every warp
constexpr int kT3MaxT = 3;
static_assert(kT3Lead + 2 <= kT3Ring && kT3MaxT + kT3Lead <= kT3Ring, "ring depth");
__host__ __device__ constexpr int t3_halo_lanes(int T) { return (T + 1) / 2; }
__host__ __device__ constexpr int t3_out_cols(int T) { return kT3Cols - 4 * t3_halo_lanes(T); }
__host__ __device__ constexpr int t3_out_rows(int T) { return kT3TileRows - 2 * T; }
// shared memory: [u ring][f ring][published rows of levels 1 .. T-1, two buffers each]
__host__ __device__ constexpr int t3_fring_offset() { return kT3Ring * kT3Plane; }
__host__ __device__ constexpr int t3_pub_offset(bool has_f) { return (has_f ? 2 : 1) * kT3Ring * kT3Plane; }
__host__ __device__ constexpr size_t t3_smem_bytes(int T, bool has_f) {
    return (size_t)(t3_pub_offset(has_f) + 2 * (T - 1) * kT3Pub) * sizeof(double);
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
struct Rows { Pair row[kT3Rows]; };

// the kernel's dynamic shared memory
extern __shared__ __align__(16) double t3_smem[];

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

struct T3 {
    double* mine;            // shared: this lane's pair in its warp's first row of u ring stage 0
    const double* below;     // shared: the pair one row below the warp's rows in u ring stage 0 (clamped to the tile)
    const double* above;     // ... one row above
    double* pub_mine;        // shared: where this lane publishes its warp's first row (level 1, buffer 0);
                             //   the last row follows 64 doubles later
    const double* pub_below; // shared: the published last row of the warp below (clamped), same level and buffer
    const double* pub_above; // shared: the published first row of the warp above (clamped)
    long long bsz;           // elements between blocks adjacent in z
    int row_off[kT3Rows];    // element offset of the warp's rows from the lane's column in row 0 of
                             // the block row 0 (rows inside the domain only)
    int nz, Z0, Z1;          // planes of the domain; output planes of this chunk
    // per row r of the warp (R rows): bit r = below the domain, bit R + r = above it, bit 2R + r = an
    // output row of the tile inside the domain; bit 3R: the lane's columns lie outside the domain,
    // bit 3R + 1: below it (else above), bit 3R + 2: the lane's columns are output columns inside the domain
    unsigned bits;
    __device__ __forceinline__ bool row_lo(int r) const { return (bits >> r) & 1u; }
    __device__ __forceinline__ bool row_hi(int r) const { return (bits >> (kT3Rows + r)) & 1u; }
    __device__ __forceinline__ bool xout() const { return (bits >> (3 * kT3Rows)) & 1u; }
    __device__ __forceinline__ bool xlow() const { return (bits >> (3 * kT3Rows + 1)) & 1u; }
    __device__ __forceinline__ bool store_lane() const { return (bits >> (3 * kT3Rows + 2)) & 1u; }
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

// Start the copies of u plane p into ring stage US and of f plane p - 1 into f stage FS: one group.
// Cells outside the domain receive their Dirichlet value by an ordinary store (f: nothing, the
// result there is replaced anyway).
template <int T, bool HAS_F, bool EDGE, int US, int FS>
__device__ __forceinline__ void t3_issue(const T3& c, const JacGeom& g, const double* __restrict__ u,
                                         const double* __restrict__ f, int p, long long u_off,
                                         long long f_off /* offset of plane p - 1 */) {
    const int in_end = c.Z1 + T, p0 = c.Z0 - T;     // input planes of the chunk
    if (p < in_end) {
        double* st = c.mine + US * kT3Plane;
#pragma unroll
        for (int r = 0; r < kT3Rows; ++r) {
            double cval = 0.0;
            if (EDGE && t3_outside(c, g, p, r, &cval)) sts_pair(st + r * kT3Cols, pair_of(cval));
            else g_cp_async16(g, st + r * kT3Cols, u + u_off + c.row_off[r], KID_TEMPORAL3D);
        }
    }
    if (HAS_F) {
        const int q = p - 1;
        if (q < in_end && q >= p0) {
            double* st = c.mine + t3_fring_offset() + FS * kT3Plane;
#pragma unroll
            for (int r = 0; r < kT3Rows; ++r) {
                double cval = 0.0;
                if (!(EDGE && t3_outside(c, g, q, r, &cval)))
                    g_cp_async16(g, st + r * kT3Cols, f + f_off + c.row_off[r], KID_TEMPORAL3D);
            }
        }
    }
    cp_async_commit();
}

// One level: plane q of the level from planes D, M, U of the level below (the lane's own column
// pairs) and the pairs one row below / above the warp's rows in plane M.
// RES: the rows flagged in `live` also add the squared residual of M (s - 6 M) to acc.
template <bool HAS_F, bool EDGE, bool RES>
__device__ __forceinline__ void t3_level(const T3& c, const JacGeom& g, const Rows& D, const Rows& M, const Rows& U,
                                         const Pair& below, const Pair& above, int q,
                                         const double* fplane /* this lane's pair in row 0 of the warp, f plane q */,
                                         Rows& out, unsigned live, double& acc)
{
    const double c6 = g.sixth;
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
            if (RES && ((live >> r) & 1u)) {
                const double rr = sub_rn(s, mul_rn(6.0, M.row[r].v[i]));
                acc = add_rn(acc, mul_rn(rr, rr));
            }
        }
        double cval = 0.0;
        if (EDGE && t3_outside(c, g, q, r, &cval)) o = pair_of(cval);
        out.row[r] = o;
    }
}

// which of the warp's rows this lane stores in output plane q (bit r); 0 if none
__device__ __forceinline__ unsigned t3_live_rows(const T3& c, int q) {
    const bool in_chunk = c.store_lane() && q >= c.Z0 && q < c.Z1;
    return in_chunk ? (c.bits >> (2 * kT3Rows)) & ((1u << kT3Rows) - 1u) : 0u;
}

__device__ __forceinline__ void t3_store(const T3& c, const JacGeom& g, double* __restrict__ un, long long out_off,
                                         const Rows& o, unsigned live) {
#pragma unroll
    for (int r = 0; r < kT3Rows; ++r)
        if ((live >> r) & 1u)
            g_st2(g, un + out_off + c.row_off[r], make_double2(o.row[r].v[0], o.row[r].v[1]), CHK_FIELD, KID_TEMPORAL3D);
}

// Levels s..T of one step, lowest first: level s computes plane p - s from the register window of
// level s - 1 (whose newest plane, p - s + 1, was made a moment ago in this step) and, across warps,
// from the rows of that level's plane p - s which their owners put into shared memory in the
// previous step (level 0: the copy ring).
// PH: the step's position in the unrolled loop (0..5); window slots, buffer parity and ring stages follow from it.
template <int T, bool HAS_F, int RES, int PH, bool EDGE, int s>
__device__ __forceinline__ void t3_levels(Rows (&win)[kT3MaxT][3], const T3& c, const JacGeom& g,
                                          double* __restrict__ un, int p, long long out_off, double& acc)
{
    constexpr int PAR = PH & 1;
    constexpr int FS = (PH + 2 * kT3Ring - s) % kT3Ring;            // ring stage of f plane p - s (and of u plane p - s)
    const int q = p - s;
    const Rows& D = win[s - 1][slot3(PH, -s - 1)];
    const Rows& M = win[s - 1][slot3(PH, -s)];
    const Rows& U = win[s - 1][slot3(PH, -s + 1)];
    constexpr int pub_prev = ((s - 2) * 2 + (PAR ^ 1)) * kT3Pub;    // plane p - s of level s - 1 (s >= 2)
    const Pair below = lds_pair(s == 1 ? c.below + FS * kT3Plane : c.pub_below + pub_prev);
    const Pair above = lds_pair(s == 1 ? c.above + FS * kT3Plane : c.pub_above + pub_prev);
    const double* fp = HAS_F ? c.mine + t3_fring_offset() + FS * kT3Plane : nullptr;
    if constexpr (s == T) {
        Rows o;
        const unsigned live = t3_live_rows(c, q);
        t3_level<HAS_F, EDGE, RES == T>(c, g, D, M, U, below, above, q, fp, o, live, acc);
        t3_store(c, g, un, out_off, o, live);
    } else {
        Rows& o = win[s][slot3(PH, -s)];
        // a level below the top can also give the residual of the state it reads: over the tile's
        // output cells, which every interior point is in exactly once, and where every level is exact
        constexpr bool RES_HERE = s == RES;
        const unsigned live = RES_HERE ? t3_live_rows(c, q) : 0u;
        t3_level<HAS_F, EDGE, RES_HERE>(c, g, D, M, U, below, above, q, fp, o, live, acc);
        // the warp's first and last row are what other warps read
        constexpr int pub_here = ((s - 1) * 2 + PAR) * kT3Pub;
        sts_pair(c.pub_mine + pub_here, o.row[0]);
        sts_pair(c.pub_mine + pub_here + kT3Cols, o.row[kT3Rows - 1]);
        t3_levels<T, HAS_F, RES, PH, EDGE, s + 1>(win, c, g, un, p, out_off, acc);
    }
}

// One step: input plane p (ring stage PH) was requested LEAD steps ago; every level advances one plane.
template <int T, bool HAS_F, int RES, int PH, bool EDGE>
__device__ __forceinline__ void t3_step(Rows (&win)[kT3MaxT][3], const T3& c, const JacGeom& g,
                                        double* __restrict__ un, int p, long long out_off, double& acc)
{
    // level 0: this lane's pairs of plane p join the window (planes p-2 and p-1 are there)
#pragma unroll
    for (int r = 0; r < kT3Rows; ++r) win[0][slot3(PH, 0)].row[r] = lds_pair(c.mine + PH * kT3Plane + r * kT3Cols);
    t3_levels<T, HAS_F, RES, PH, EDGE, 1>(win, c, g, un, p, out_off, acc);
}

// RES (1..T; 0: none): partials[CTA * 12 + warp] gets the warp's sum of squared residuals over exactly
// the points the warp stores -- of the state level RES reads, the one after RES - 1 sweeps of the launch.
template <int T, bool HAS_F, int RES>
__global__ void __launch_bounds__(kT3Warps * 32, 1)
temporal3d_kernel(const double* __restrict__ u, double* __restrict__ un, const double* __restrict__ f,
                  double* __restrict__ partials, const JacGeom g, const int tiles_x, const int tiles_y,
                  const int tiles_z, const int zchunk)
{
    if (solve_stopped(g)) return;
    T3 c;
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
    c.bits = (xout ? 1u << (3 * kT3Rows) : 0u) | (gx < 0 ? 1u << (3 * kT3Rows + 1) : 0u) |
             ((lane >= HL && lane <= 31 - HL && !xout) ? 1u << (3 * kT3Rows + 2) : 0u);
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
        else if (gy >= g.ny) c.bits |= 1u << (kT3Rows + r);
        else {
            const long long byi = gy / g.by;
            c.row_off[r] = (int)(byi * bsy + (gy - byi * g.by) * g.PX);   // the host admits only grids where this fits
            if (trow >= T && trow < kT3TileRows - T) c.bits |= 1u << (2 * kT3Rows + r);
        }
    }
    c.mine = t3_smem + trow0 * kT3Cols + 2 * lane;
    c.below = t3_smem + max(trow0 - 1, 0) * kT3Cols + 2 * lane;
    c.above = t3_smem + min(trow0 + kT3Rows, kT3TileRows - 1) * kT3Cols + 2 * lane;
    double* pub = t3_smem + t3_pub_offset(HAS_F);
    c.pub_mine = pub + (warp * 2) * kT3Cols + 2 * lane;
    c.pub_below = pub + (max(warp - 1, 0) * 2 + 1) * kT3Cols + 2 * lane;
    c.pub_above = pub + (min(warp + 1, kT3Warps - 1) * 2) * kT3Cols + 2 * lane;
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

    Rows win[kT3MaxT][3];     // [level][plane mod 3]; only levels 0 .. T-1 are used
#pragma unroll
    for (int s = 0; s < kT3MaxT; ++s)
#pragma unroll
        for (int k = 0; k < 3; ++k)
#pragma unroll
            for (int r = 0; r < kT3Rows; ++r) win[s][k].row[r] = pair_of(0.0);

    ZCursor load_cur, out_cur;
    load_cur.init(p0, g, c.bsz, col);
    out_cur.init(p0 - T, g, c.bsz, col);   // output plane of level T in the first step
    long long f_off = 0;                    // the f plane that travels with u plane p is p - 1: the
                                            // offset the load cursor had one step earlier
    double acc = 0.0;

    // Request plane PL, which has position POS in the unrolled loop: u into stage POS mod 6, f plane
    // PL - 1 into the stage before it.
#define JAC_T3_ISSUE(POS, PL)                                                                            \
    do {                                                                                                 \
        const int pl_ = (PL);                                                                            \
        const bool edge_i = edge_xy || (pl_ - 1 < 0) || (pl_ >= c.nz);                                   \
        constexpr int US_ = (POS) % kT3Ring, FS_ = ((POS) + kT3Ring - 1) % kT3Ring;                      \
        if (edge_i) t3_issue<T, HAS_F, true, US_, FS_>(c, g, u, f, pl_, load_cur.off, f_off);            \
        else t3_issue<T, HAS_F, false, US_, FS_>(c, g, u, f, pl_, load_cur.off, f_off);                  \
        f_off = load_cur.off;                                                                            \
        load_cur.advance(g, c.bsz);                                                                      \
    } while (0)

    JAC_T3_ISSUE(0, p0);
    JAC_T3_ISSUE(1, p0 + 1);
    JAC_T3_ISSUE(2, p0 + 2);
    static_assert(kT3Lead == 3, "the three requests above");

#define JAC_T3_STEP(PHASE, PL)                                                                           \
    do {                                                                                                 \
        const int p_ = (PL);                                                                             \
        JAC_T3_ISSUE((PHASE) + kT3Lead, p_ + kT3Lead);   /* into the stage plane p - 3 has left */       \
        cp_async_wait<kT3Lead>();                        /* this lane's part of plane p has landed */    \
        const bool edge_s = edge_xy || (p_ - T - 1 < 0) || (p_ >= c.nz);                                 \
        if (edge_s) t3_step<T, HAS_F, RES, PHASE, true>(win, c, g, un, p_, out_cur.off, acc);            \
        else t3_step<T, HAS_F, RES, PHASE, false>(win, c, g, un, p_, out_cur.off, acc);                  \
        out_cur.advance(g, c.bsz);                                                                       \
        __syncthreads();                                                                                 \
    } while (0)

    for (int p = p0; p < p_end; p += kT3Ring) {
        JAC_T3_STEP(0, p);
        if (p + 1 < p_end) JAC_T3_STEP(1, p + 1);
        if (p + 2 < p_end) JAC_T3_STEP(2, p + 2);
        if (p + 3 < p_end) JAC_T3_STEP(3, p + 3);
        if (p + 4 < p_end) JAC_T3_STEP(4, p + 4);
        if (p + 5 < p_end) JAC_T3_STEP(5, p + 5);
    }
#undef JAC_T3_STEP
#undef JAC_T3_ISSUE
    cp_async_wait<0>();
    if (RES != 0) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc = add_rn(acc, __shfl_down_sync(0xffffffffu, acc, off));
        if (lane == 0) g_st(g, partials + (long long)blockIdx.x * kT3Warps + warp, acc, CHK_SCRATCH, KID_TEMPORAL3D);
    }
}

}  // namespace jac
