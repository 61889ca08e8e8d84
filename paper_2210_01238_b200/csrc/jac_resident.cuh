// Resident schedule for small 2D grids: the whole grid stays in the shared memory of one
// thread-block cluster for all sweeps of a launch.
//
// A grid of a few hundred KB is bound by launch and pipeline latency, not by bandwidth: every
// other schedule pays at least one launch per handful of sweeps and goes through L2 each time.
// Here CTA c of the cluster owns a slab of `rows` consecutive grid rows in two shared-memory
// buffers (plus the slab's right-hand side) and sweeps from one buffer into the other.  Global
// memory is read once before the first sweep and written once after the last.
//
// Neighbouring slabs only ever need each other's edge row, so they synchronise pairwise, not as a
// cluster: a CTA computes its first and last new row first and sends them straight into the
// neighbours' halo rows with st.async, which counts the bytes that have landed on an mbarrier in
// the RECEIVING CTA; one warp of the receiver waits on its two mbarriers (one per side) after it
// has computed its inner rows, and the CTA barrier that ends the sweep passes the rows on to the
// other warps.  No fence, no cluster-wide barrier per sweep: the cluster barrier is used once
// after the fill and once before the write-back.  Why a halo row can be overwritten safely: the
// row a neighbour sends for sweep s + 1 can only leave after that neighbour has received this
// CTA's row of sweep s, which each thread sends after it has read the halo cells it needs.
// Every wait is bounded: a CTA that has polled kResMaxPolls times sets the error word, stops
// waiting and runs to the end with whatever it has, so that all CTAs reach the final barrier.
// Measured with clock64 stamps in a copy of the kernel (256^2, 16 CTAs): a sweep took ~1850 cycles,
// ~740 of them for the edge row while thread 0 also announced the incoming rows to the mbarriers and
// every thread polled them; with the announcement made by a warp that has no edge row, one polling
// warp, and the two buffers alternating as compile-time constants, 100 sweeps take 94 us, not 113.
//
// Slab layout (doubles): row pitch RP = nx + 4; grid column i sits at index i + 2 (so pairs of
// columns are 16-byte aligned), the Dirichlet columns at 1 and nx + 2.  Local row 0 is the halo
// below the slab, rows 1..rows the slab, row rows + 1 the halo above.  Arithmetic and operation
// order are those of every other schedule, so results are bit-identical.
// Requires bx % 2 == 0 (pairs never straddle blocks).
#pragma once
#include <cooperative_groups.h>
#include <cuda_runtime.h>

#include <type_traits>

#include "jac_geom.h"
#include "jac_kernels.cuh"

namespace jac {

constexpr int kResThreads = 512;
constexpr int kResMaxPolls = 1 << 22;     // mbarrier polls before a CTA gives up waiting

// ---- mbarrier / distributed shared memory primitives (PTX) ---------------------------------
__device__ __forceinline__ unsigned smem_addr(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity) {
    unsigned ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// the address, in the cluster's shared window, of this CTA's shared address `local` in CTA `rank`
__device__ __forceinline__ unsigned map_to_rank(unsigned local, unsigned rank) {
    unsigned r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}
// 16 bytes into another CTA's shared memory; the bytes are counted on that CTA's mbarrier when they land
__device__ __forceinline__ void send_pair(unsigned remote, unsigned remote_bar, double2 v) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f64 [%0], {%1, %2}, [%3];\n"
                 ::"r"(remote), "d"(v.x), "d"(v.y), "r"(remote_bar) : "memory");
}

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
                  const JacGeom g, const int nsweeps, const int rows, int* __restrict__ timed_out)
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
    // arrival of the halo row below / above this slab in buffer 0 / 1: [side][buffer]
    __shared__ __align__(8) unsigned long long halo_bar[2][2];
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
        *reinterpret_cast<double2*>(buf[0] + l * RP + 2 + 2 * cp) = g_ld2(g, u + off, CHK_FIELD, KID_RESIDENT);
        if (HAS_F && l >= 1 && l <= mine)
            *reinterpret_cast<double2*>(fs + (l - 1) * RP + 2 + 2 * cp) = g_ld2(g, f + off, CHK_FIELD, KID_RESIDENT);
    }
    // where the neighbours keep the halo row that mirrors this slab's first / last row, and the
    // mbarrier that counts its arrival there, per buffer: this slab's first row goes to the upper
    // halo row (rows + 1) of the CTA below, which is full (only the last owning CTA can be short)
    unsigned lo_row[2] = {0, 0}, hi_row[2] = {0, 0}, lo_bar[2] = {0, 0}, hi_bar[2] = {0, 0};
    if (has_lo) {
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            lo_row[w] = map_to_rank(smem_addr(buf[w] + (size_t)(rows + 1) * RP), rank - 1);
            lo_bar[w] = map_to_rank(smem_addr(&halo_bar[1][w]), rank - 1);     // it arrives from above, there
        }
    }
    if (has_hi) {
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            hi_row[w] = map_to_rank(smem_addr(buf[w]), rank + 1);
            hi_bar[w] = map_to_rank(smem_addr(&halo_bar[0][w]), rank + 1);     // from below, there
        }
    }
    if (tid == 0) {
#pragma unroll
        for (int side = 0; side < 2; ++side)
#pragma unroll
            for (int w = 0; w < 2; ++w) mbar_init(smem_addr(&halo_bar[side][w]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    cluster.sync();

    // ---- sweeps: A -> B.  The slab's first and last row go first: they are what the neighbours
    // wait for, and the only rows that read this slab's halo rows.  They are written here and sent
    // into the neighbours' halo rows; then the inner rows are computed while those rows travel, and
    // only then does the CTA wait for the two rows it is owed.  The inner rows are marched through
    // in segments (rows below and above a thread's pair stay in registers).
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
    const unsigned row_bytes = (unsigned)nx * (unsigned)sizeof(double);
    bool gave_up = false;
    // One sweep into buffer WB, a compile-time constant: the loop below alternates the two, so no
    // sweep selects its buffers, halo rows or mbarriers at run time.
    auto sweep_once = [&](auto wbc, const int s) {
        constexpr int wb = decltype(wbc)::value;
        const double* const A = buf[wb ^ 1];
        double* const B = buf[wb];
        // this sweep's incoming rows: one arrival (this one) plus the row's bytes complete a phase.
        // Announced by a thread whose warp computes no edge row where there is one (four row
        // groups): the rows the neighbours wait for do not queue behind it.
        if (tid == kResThreads - 1) {
            if (has_lo) mbar_expect_tx(smem_addr(&halo_bar[0][wb]), row_bytes);
            if (has_hi) mbar_expect_tx(smem_addr(&halo_bar[1][wb]), row_bytes);
        }
        auto edge_row = [&](const int l) {
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
                const unsigned col = (unsigned)(2 + 2 * cp) * (unsigned)sizeof(double);
                if (l == 1 && has_lo) send_pair(lo_row[wb] + col, lo_bar[wb], o);
                if (l == mine && has_hi) send_pair(hi_row[wb] + col, hi_bar[wb], o);
            }
        };
        if (does_lo) edge_row(1);
        if (does_hi) edge_row(mine);
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
        // the neighbours' rows of this sweep (the k-th use of a buffer's mbarriers has parity k & 1).
        // One warp waits for them; the barrier below passes on what it has seen to the others.
        const unsigned parity = (unsigned)(s >> 1) & 1u;
        if (!gave_up && tid >= kResThreads - 32) {
#pragma unroll 1
            for (int side = 0; side < 2; ++side) {
                if (side == 0 ? !has_lo : !has_hi) continue;
                const unsigned bar = smem_addr(&halo_bar[side][wb]);
                int polls = 0;
                while (!mbar_try_wait(bar, parity)) {
                    if (++polls >= kResMaxPolls) {
                        gave_up = true;
                        *timed_out = 1;
                        break;
                    }
                }
            }
        }
        __syncthreads();            // this CTA's rows of B are complete, and nobody still reads A
    };
    {
        int s = 0;                  // sweep s writes buffer (s + 1) & 1
        for (; s + 1 < nsweeps; s += 2) {
            sweep_once(std::integral_constant<int, 1>{}, s);
            sweep_once(std::integral_constant<int, 0>{}, s + 1);
        }
        if (s < nsweeps) sweep_once(std::integral_constant<int, 1>{}, s);
    }
    cluster.sync();                 // no row is still on its way to a CTA that is about to leave
    double* const A = buf[nsweeps & 1];

    // ---- write the final state back
    for (int it = tid; it < mine * npairs; it += kResThreads) {
        const int l = it / npairs + 1, cp = it - (l - 1) * npairs;
        g_st2(g, un + resident_offset(g, 2 * cp, y0 + l - 1), *reinterpret_cast<const double2*>(A + l * RP + 2 + 2 * cp),
              CHK_FIELD, KID_RESIDENT);
    }
}

}  // namespace jac
