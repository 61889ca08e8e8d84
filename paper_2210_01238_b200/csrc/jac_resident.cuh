// Resident schedule for small 2D grids: the whole grid stays in the shared memory of one
// thread-block cluster for all sweeps of a launch.
//
// A grid of a few hundred KB is bound by launch and pipeline latency, not by bandwidth: every
// other schedule pays at least one launch per handful of sweeps and goes through L2 each time.
// Here CTA c of the cluster owns a slab of `rows` consecutive grid rows in two shared-memory
// buffers (plus the slab's right-hand side), sweeps from one buffer into the other, writes its
// first and last new row straight into the neighbouring CTAs' halo rows through distributed
// shared memory, and meets the other CTAs at one cluster barrier per sweep (arrive after the edge
// rows, wait after the inner rows, so the barrier's latency is covered by work).  Global memory is
// read once before the first sweep and written once after the last.
//
// Slab layout (doubles): row pitch RP = nx + 4; grid column i sits at index i + 2 (so pairs of
// columns are 16-byte aligned), the Dirichlet columns at 1 and nx + 2.  Local row 0 is the halo
// below the slab, rows 1..rows the slab, row rows + 1 the halo above.  Arithmetic and operation
// order are those of every other schedule, so results are bit-identical.
// Requires bx % 2 == 0 (pairs never straddle blocks).
#pragma once
#include <cooperative_groups.h>
#include <cuda_runtime.h>

#include "jac_geom.h"
#include "jac_kernels.cuh"

namespace jac {

constexpr int kResThreads = 512;

__host__ __device__ constexpr long long resident_pitch(long long nx) { return nx + 4; }
// shared-memory bytes of one CTA whose slab has `rows` rows
__host__ __device__ constexpr size_t resident_smem_bytes(long long nx, int rows, bool has_f) {
    return (size_t)((2 * (rows + 2) + (has_f ? rows : 0)) * resident_pitch(nx)) * sizeof(double);
}

// element offset of grid point (gx, gy) in the blocked arrays
__device__ __forceinline__ long long resident_offset(const JacGeom& g, long long gx, long long gy) {
    const long long bxi = gx / g.bx, byi = gy / g.by;
    return (byi * g.gx + bxi) * g.block_stride + g.origin + (gy - byi * g.by) * g.PX + (gx - bxi * g.bx);
}

template <bool HAS_F>
__global__ void __launch_bounds__(kResThreads, 1)
resident2d_kernel(const double* __restrict__ u, double* __restrict__ un, const double* __restrict__ f,
                  const JacGeom g, const int nsweeps, const int rows)
{
    if (solve_stopped(g)) return;      // every CTA of the cluster takes the same way out
    namespace cg = cooperative_groups;
    extern __shared__ __align__(16) double res_smem[];
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int nranks = (int)cluster.num_blocks();
    const int nx = (int)g.nx, ny = (int)g.ny;
    const int RP = (int)resident_pitch(nx);
    const int y0 = rank * rows;                              // first grid row of the slab
    const int mine = max(0, min(rows, ny - y0));             // rows this CTA really owns
    const bool has_lo = rank > 0 && mine > 0;                // a CTA below owns row y0 - 1
    const bool has_hi = rank + 1 < nranks && y0 + rows < ny; // a CTA above owns row y0 + rows
    double* const buf[2] = {res_smem, res_smem + (size_t)(rows + 2) * RP};
    double* fs = res_smem + (size_t)2 * (rows + 2) * RP;     // [rows][RP], same column placement
    const int tid = threadIdx.x;
    const int npairs = nx / 2;

    // ---- fill: Dirichlet frame in both buffers, then the slab, its halo rows and f from memory
    for (int i = tid; i < 2 * (rows + 2) * RP; i += kResThreads) res_smem[i] = 0.0;
    __syncthreads();
    for (int l = tid; l < rows + 2; l += kResThreads) {
        buf[0][l * RP + 1] = buf[1][l * RP + 1] = g.bval[0];
        buf[0][l * RP + nx + 2] = buf[1][l * RP + nx + 2] = g.bval[1];
    }
    for (int i = tid; i < nx; i += kResThreads) {
        if (y0 == 0) buf[0][2 + i] = buf[1][2 + i] = g.bval[2];
        if (mine > 0 && y0 + mine == ny) buf[0][(mine + 1) * RP + 2 + i] = buf[1][(mine + 1) * RP + 2 + i] = g.bval[3];
    }
    // rows y0 - 1 .. y0 + mine of u (the two outer ones only where another CTA owns them)
    for (int it = tid; it < (mine + 2) * npairs; it += kResThreads) {
        const int l = it / npairs, cp = it - l * npairs;
        const int gy = y0 + l - 1;
        if (mine == 0 || (l == 0 && !has_lo) || (l == mine + 1 && !has_hi)) continue;
        const long long off = resident_offset(g, 2 * cp, gy);
        *reinterpret_cast<double2*>(buf[0] + l * RP + 2 + 2 * cp) = *reinterpret_cast<const double2*>(u + off);
        if (HAS_F && l >= 1 && l <= mine)
            *reinterpret_cast<double2*>(fs + (l - 1) * RP + 2 + 2 * cp) = *reinterpret_cast<const double2*>(f + off);
    }
    // where the neighbours keep the halo row that mirrors this slab's first / last row
    // (A = the buffer being read, B = the one being written; they swap after every sweep)
    double *lo_A = nullptr, *lo_B = nullptr, *hi_A = nullptr, *hi_B = nullptr;
    if (has_lo) {
        // the CTA below is full (only the last owning CTA can be short): its upper halo is row rows + 1
        lo_A = cluster.map_shared_rank(buf[0], rank - 1) + (size_t)(rows + 1) * RP;
        lo_B = cluster.map_shared_rank(buf[1], rank - 1) + (size_t)(rows + 1) * RP;
    }
    if (has_hi) {
        hi_A = cluster.map_shared_rank(buf[0], rank + 1);
        hi_B = cluster.map_shared_rank(buf[1], rank + 1);
    }
    cluster.sync();

    // ---- sweeps: A -> B.  The slab's first and last row go first: they are what the neighbours
    // wait for, and the only rows that read this slab's halo rows.  Once they are written (here and
    // into the neighbours' halo rows) the CTA arrives at the cluster barrier, computes its inner
    // rows while the barrier completes, and waits before the next sweep.  The inner rows are
    // marched through in segments (rows below and above a thread's pair stay in registers).
    // The assignment of work to threads is the same in every sweep, so it is fixed here: a thread
    // owns the column pairs cp0, cp0 + pw, ... and row group `grp`; group 0 also computes edge row 1
    // and another group (the same one if there is only one) edge row `mine`.
    const int pw = min(npairs, kResThreads);                  // column pairs side by side
    const int groups = max(1, kResThreads / pw);              // row groups side by side
    const int cp0 = tid % pw, grp = tid / pw;
    const int inner = max(0, mine - 2);                       // rows 2 .. mine - 1
    const int segrows = (inner + groups - 1) / groups;
    const int l0 = 2 + grp * segrows;
    const int l1 = grp < groups ? min(mine, l0 + segrows) : l0;
    const bool does_lo = grp == 0 && mine >= 1;
    const bool does_hi = grp == min(groups, 2) - 1 && mine >= 2;
    double *A = buf[0], *B = buf[1];
    for (int s = 0; s < nsweeps; ++s) {
#pragma unroll 1
        for (int side = 0; side < 2; ++side) {
            if (side == 0 ? !does_lo : !does_hi) continue;
            const int l = side == 0 ? 1 : mine;
            for (int cp = cp0; cp < npairs; cp += pw) {
                const int at = l * RP + 2 + 2 * cp;
                const double2 S = *reinterpret_cast<const double2*>(A + at - RP);
                const double2 M = *reinterpret_cast<const double2*>(A + at);
                const double2 N = *reinterpret_cast<const double2*>(A + at + RP);
                const double w = A[at - 1];
                const double e = A[at + 2];
                double s0 = add_rn(add_rn(w, M.y), add_rn(S.x, N.x));
                double s1 = add_rn(add_rn(M.x, e), add_rn(S.y, N.y));
                if (HAS_F) {
                    const double2 ff = *reinterpret_cast<const double2*>(fs + at - RP);
                    s0 = add_rn(s0, ff.x);
                    s1 = add_rn(s1, ff.y);
                }
                const double2 o = make_double2(mul_rn(s0, 0.25), mul_rn(s1, 0.25));
                *reinterpret_cast<double2*>(B + at) = o;
                if (l == 1 && has_lo) *reinterpret_cast<double2*>(lo_B + 2 + 2 * cp) = o;
                if (l == mine && has_hi) *reinterpret_cast<double2*>(hi_B + 2 + 2 * cp) = o;
            }
        }
        cluster.barrier_arrive();   // release: this CTA's halo reads and edge-row writes are done
        if (l0 < l1) {
            for (int cp = cp0; cp < npairs; cp += pw) {
                int at = l0 * RP + 2 + 2 * cp;
                double2 S = *reinterpret_cast<const double2*>(A + at - RP);
                double2 M = *reinterpret_cast<const double2*>(A + at);
#pragma unroll 4
                for (int l = l0; l < l1; ++l, at += RP) {
                    const double2 N = *reinterpret_cast<const double2*>(A + at + RP);
                    const double w = A[at - 1];
                    const double e = A[at + 2];
                    double s0 = add_rn(add_rn(w, M.y), add_rn(S.x, N.x));
                    double s1 = add_rn(add_rn(M.x, e), add_rn(S.y, N.y));
                    if (HAS_F) {
                        const double2 ff = *reinterpret_cast<const double2*>(fs + at - RP);
                        s0 = add_rn(s0, ff.x);
                        s1 = add_rn(s1, ff.y);
                    }
                    *reinterpret_cast<double2*>(B + at) = make_double2(mul_rn(s0, 0.25), mul_rn(s1, 0.25));
                    S = M;
                    M = N;
                }
            }
        }
        __syncthreads();            // nobody in this CTA still reads A (the next sweep writes it)
        cluster.barrier_wait();     // acquire: the neighbours' rows have arrived in B's halo rows
        double* t = A; A = B; B = t;
        t = lo_A; lo_A = lo_B; lo_B = t;
        t = hi_A; hi_A = hi_B; hi_B = t;
    }

    // ---- write the final state back
    for (int it = tid; it < mine * npairs; it += kResThreads) {
        const int l = it / npairs + 1, cp = it - (l - 1) * npairs;
        *reinterpret_cast<double2*>(un + resident_offset(g, 2 * cp, y0 + l - 1)) =
            *reinterpret_cast<const double2*>(A + l * RP + 2 + 2 * cp);
    }
}

}  // namespace jac
