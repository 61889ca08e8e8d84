// Host side of libjac: descriptor validation, workspace layout, launch scheduling and the
// C ABI declared in include/jac.h.  No device memory is allocated here: every buffer lives
// in the caller's workspace.
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "jac.h"
#include "jac_geom.h"
#include "jac_kernels.cuh"
#include "jac_resident.cuh"
#include "jac_temporal3d.cuh"

namespace {

// SMs the launch planners assume when no device has been asked yet (the pure host queries: the
// workspace layout must not depend on the machine it is computed on).  A context asks its device
// once, at creation, and plans its launches with that count wherever the scratch sized for the
// nominal count allows it.
constexpr int kNominalSMs = 148;  // B200
constexpr long long kMaxGrid = 2147483647LL;

long long round_up(long long v, long long m) { return (v + m - 1) / m * m; }
long long ceil_div(long long a, long long b) { return (a + b - 1) / b; }
int pow2_ceil(long long v) { int p = 1; while (p < v) p <<= 1; return p; }

// How one launch of the sweep / residual kernels is cut into CTAs.
struct Tiling {
    int nv;        // points per thread along x (2 when bx is even: 128-bit accesses)
    dim3 block;
    int tiles_x, tiles_y, tiles_z;
    int march;     // rows (2D) or planes (3D) a CTA marches through
    long long ctas_per_block;
};

// force_nv = 1: one point per thread although the width is even (rows that do not start on a
// 16-byte boundary)
Tiling make_tiling(const JacGeom& g, int sms, int force_nv = 0)
{
    Tiling t{};
    t.nv = force_nv ? force_nv : ((g.bx % 2 == 0 && g.rx % 2 == 0) ? 2 : 1);
    const long long need = ceil_div(g.bx, t.nv);
    const long long want_ctas = (long long)sms * 16;
    if (g.ndim == 2) {
        const int tpb = (int)std::min<long long>(256, round_up(need, 32));
        t.block = dim3(tpb, 1, 1);
        t.tiles_x = (int)ceil_div(need, tpb);
        t.tiles_z = 1;
        int rows = std::min(g.by, 64);
        while (rows > 8 && g.nblocks * t.tiles_x * ceil_div(g.by, rows) < want_ctas) rows = (rows + 1) / 2;
        t.march = rows;
        t.tiles_y = (int)ceil_div(g.by, rows);
    } else {
        const int tx = std::min(64, pow2_ceil(need));
        // at least one whole warp: the CTA-wide sum shuffles over 32 lanes (threads beyond the block's
        // rows fail the extent test and contribute 0)
        const int ty = std::max(std::min(std::max(1, 512 / tx), std::min(8, pow2_ceil(g.by))), 32 / tx);
        t.block = dim3(tx, ty, 1);
        t.tiles_x = (int)ceil_div(need, tx);
        t.tiles_y = (int)ceil_div(g.by, ty);
        int planes = g.bz;
        while (planes > 16 && g.nblocks * t.tiles_x * t.tiles_y * ceil_div(g.bz, planes) < want_ctas)
            planes = (planes + 1) / 2;
        t.march = planes;
        t.tiles_z = (int)ceil_div(g.bz, planes);
    }
    t.ctas_per_block = (long long)t.tiles_x * t.tiles_y * t.tiles_z;
    return t;
}

// Geometry of the temporal launches (also bounds the reduction scratch they may fill).
struct TemporalGrid {
    int a, b, c, chunk;   // 2D: strips_x, strips_y, -, rows per strip; 3D: tiles x, y, z, planes per chunk
    long long warps;      // partial sums a residual-carrying launch writes
    long long ctas;
};

// Rows per strip of the 2D temporal kernel.  A strip of R rows costs R + 4T - 1 pipeline steps
// (2T rows of fill, 2T - 1 of drain); the GPU runs `capacity` strips at a time (148 SMs x CTAs per
// SM, as the kernel's launch bounds ask for, x warps per CTA); w = strips / capacity.  Strips are
// handed out dynamically, so a launch of many strips takes about
//     (R + 4T - 1) x (w + alpha):  all pipeline steps at full occupancy, plus a tail of part of one strip;
// alpha = 0.7 up to T = 4 and 0.45 beyond, fitted to launches of 2048^2 .. 16384^2 (deep pipelines
// are bound by issue and suffer less from an idle memory system in the tail).  With fewer than six
// rounds of strips the rounds count whole: a warp was measured to run no faster on a half-empty
// SM, so a round that is 3 % full costs as much as a full one.  R is the value in 8..256
// that minimises this estimate; longer strips were measured slower (512 rows lose 8 % at 16384^2,
// T = 8).  Measured against the earlier fixed rule (32 rows below 7104 strips): 4096^2 with f,
// T = 4: 0.107 ms per launch instead of 0.113; 8192^2, T = 4: 0.211 instead of 0.226; 2048^2,
// T = 8: 0.049 instead of 0.064; 16384^2 unchanged.
int temporal_rows_2d(const JacGeom& g, int T, bool has_f, int sms)
{
#ifdef JAC_FORCE_ROWS
    return JAC_FORCE_ROWS;
#endif
    const long long strips_x = ceil_div(g.nx, jac::temporal_strip_cols(T));
    const int ctas_per_sm = jac::temporal_ctas_per_sm(T, has_f);
    const double capacity = (double)sms * ctas_per_sm * jac::kTemporalWarps;
    const double alpha = T > 4 ? 0.45 : 0.7;
    int best = 8;
    double best_cost = 1e300;
    for (int rows = 8; rows <= 256; ++rows) {
        if (rows > g.ny && rows > 8) break;
        const double w = (double)(strips_x * ceil_div(g.ny, rows)) / capacity;
        const double rounds = w < 6.0 ? std::ceil(w - 1e-9) : w;
        const double cost = (rows + 2 * T) * (rounds + alpha);
        if (cost <= best_cost) {   // ties go to the longer strip (less redundant work)
            best_cost = cost;
            best = rows;
        }
    }
    return best;
}

TemporalGrid temporal_grid_2d(const JacGeom& g, int T, bool has_f, int sms)
{
    TemporalGrid t{};
    t.a = (int)ceil_div(g.nx, jac::temporal_strip_cols(T));
    const int rows = temporal_rows_2d(g, T, has_f, sms);
    t.chunk = rows;
    t.b = (int)ceil_div(g.ny, rows);
    t.c = 1;
    t.warps = (long long)t.a * t.b;
    t.ctas = ceil_div(t.warps, jac::kTemporalWarps);
    return t;
}

TemporalGrid temporal_grid_3d(const JacGeom& g, int T, int sms)
{
    TemporalGrid t{};
    t.a = (int)ceil_div(g.nx, jac::t3_out_cols(T));
    t.b = (int)ceil_div(g.ny, jac::t3_out_rows(T));
    // planes per chunk: a chunk of Z planes costs Z + 2T steps; long chunks waste the least, but the
    // launch should still be several rounds of CTAs (one CTA per SM)
    int zchunk = 256;
    while (zchunk > 16 && (long long)t.a * t.b * ceil_div(g.nz, zchunk) < (long long)sms * 6) zchunk /= 2;
    t.chunk = zchunk;
    t.c = (int)ceil_div(g.nz, zchunk);
    t.ctas = (long long)t.a * t.b * t.c;
    t.warps = t.ctas * jac::kT3Warps;
    return t;
}

// The resident schedule: the grid is cut into one slab of rows per CTA of a single cluster of 8 or
// 16 CTAs (pure host arithmetic).  A sweep is bound by the cluster barrier and the edge rows'
// trip through distributed shared memory, not by arithmetic, but halving the slabs still pays
// once they have a few rows each (256 rows: 1.17 us per sweep with 16 CTAs, 1.65 us with 8), so
// grids of 128 rows or more ask for 16 first.  jac_create falls back to the other size when the
// device cannot co-schedule the first choice.
struct ResidentPlan {
    int cluster, rows;
    size_t smem;
};
constexpr size_t kMaxSmemPerCta = 227 * 1024 - 64;   // dynamic shared memory beside the kernel's few static words

int plan_resident(const JacGeom& g, bool has_f, int want_cluster, ResidentPlan* p)
{
    if (g.ndim != 2 || g.bx % 2 != 0 || g.rx % 2 != 0 || g.nx >= (1LL << 24) || g.ny >= (1LL << 24)) return JAC_EINVAL;
    if (want_cluster != 0 && want_cluster != 8 && want_cluster != 16) return JAC_EINVAL;
    const int first = want_cluster ? want_cluster : (g.ny >= 128 ? 16 : 8);
    const int order[2] = {first, want_cluster ? first : 24 - first};
    for (int k = 0; k < 2; ++k) {
        const int cl = order[k];
        const int rows = (int)ceil_div(g.ny, cl);
        const size_t smem = jac::resident_smem_bytes(g.nx, rows, has_f);
        if (smem <= kMaxSmemPerCta) {
            p->cluster = cl;
            p->rows = rows;
            p->smem = smem;
            return JAC_OK;
        }
    }
    return JAC_EINVAL;
}

// largest number of partial sums any launch of this geometry can write
long long max_partials(const JacGeom& g, long long sweep_ctas, bool has_f, int sms)
{
    long long m = sweep_ctas;
    if (g.ndim == 2) for (int T = 1; T <= 8; ++T) m = std::max(m, temporal_grid_2d(g, T, has_f, sms).warps);
    else for (int T = 1; T <= jac::kT3MaxT; ++T) m = std::max(m, temporal_grid_3d(g, T, sms).warps);
    return m;
}

int build_geometry(const jac_desc* d, JacGeom* g, jac_layout* L)
{
    if (!d) return JAC_EINVAL;
    if (d->ndim != 2 && d->ndim != 3) return JAC_EINVAL;
    if (d->halo < 1 || d->halo > 8) return JAC_EINVAL;
    if (d->has_f != 0 && d->has_f != 1) return JAC_EINVAL;
    if (d->mode < JAC_MODE_FUSED || d->mode > JAC_MODE_RESIDENT) return JAC_EINVAL;
    if (d->tsteps < 0 || d->tsteps > (d->mode == JAC_MODE_RESIDENT ? 16 : 8)) return JAC_EINVAL;
    if (d->flags & ~(JAC_FLAG_HOST_STAGING | JAC_FLAG_CUT_LO | JAC_FLAG_CUT_HI)) return JAC_EINVAL;
    const bool has_cut = (d->flags & (JAC_FLAG_CUT_LO | JAC_FLAG_CUT_HI)) != 0;
    // a slab exchanges its cut faces once per sweep: only the one-sweep-per-exchange schedules
    if (has_cut && d->mode != JAC_MODE_FUSED && d->mode != JAC_MODE_EXCHANGE) return JAC_EINVAL;
    long long n[3] = {1, 1, 1}, b[3] = {1, 1, 1}, gr[3] = {1, 1, 1};
    for (int a = 0; a < d->ndim; ++a) {
        n[a] = d->n[a];
        b[a] = d->b[a];
        if (n[a] < 1 || b[a] < 1 || b[a] > n[a]) return JAC_EINVAL;
        if (d->halo > b[a]) return JAC_EINVAL;
        if (b[a] > (1LL << 30) || n[a] > (1LL << 40)) return JAC_EINVAL;
        gr[a] = ceil_div(n[a], b[a]);
        if (n[a] - (gr[a] - 1) * b[a] < d->halo) return JAC_EINVAL;   // a remainder block narrower than a face strip
        if (gr[a] > (1LL << 30)) return JAC_EINVAL;
    }
    // the blocks on a cut are whole: a remainder block exists only at the far end of the domain
    if ((d->flags & JAC_FLAG_CUT_HI) && n[d->ndim - 1] % b[d->ndim - 1] != 0) return JAC_EINVAL;
    std::memset(g, 0, sizeof(*g));
    g->ndim = d->ndim;
    g->h = d->halo;
    g->xpad = (int)round_up(d->halo, 4);
    g->nfaces = 2 * d->ndim;
    g->bx = (int)b[0]; g->by = (int)b[1]; g->bz = (int)b[2];
    g->gx = (int)gr[0]; g->gy = (int)gr[1]; g->gz = (int)gr[2];
    g->rx = (int)(n[0] - (gr[0] - 1) * b[0]);
    g->ry = (int)(n[1] - (gr[1] - 1) * b[1]);
    g->rz = (int)(n[2] - (gr[2] - 1) * b[2]);
    g->nx = n[0]; g->ny = n[1]; g->nz = n[2];
    const long long hz = (d->ndim == 3) ? d->halo : 0;
    const long long PY = b[1] + 2 * d->halo, PZ = b[2] + 2 * hz;
    g->PX = b[0] + 2 * g->xpad;
    g->PXY = g->PX * PY;
    g->block_stride = round_up(g->PXY * PZ, 16);
    g->origin = (hz * PY + d->halo) * g->PX + g->xpad;
    g->nblocks = gr[0] * gr[1] * gr[2];
    if (g->nblocks > (1LL << 40) / std::max<long long>(1, g->block_stride)) return JAC_EINVAL;
    const long long h = d->halo;
    g->face_elems[0] = g->face_elems[1] = h * b[1] * b[2];
    g->face_elems[2] = g->face_elems[3] = h * b[0] * b[2];
    g->face_elems[4] = g->face_elems[5] = (d->ndim == 3) ? h * b[0] * b[1] : 0;
    const long long wx = b[0] + 2 * h, wy = b[1] + 2 * h, wz = b[2] + 2 * hz;
    g->wface_elems[0] = g->wface_elems[1] = h * wy * wz;
    g->wface_elems[2] = g->wface_elems[3] = h * wx * wz;
    g->wface_elems[4] = g->wface_elems[5] = (d->ndim == 3) ? h * wx * wy : 0;
    // the send slots hold wide faces in the schedule that exchanges them, else the plain faces
    const bool wide = d->mode == JAC_MODE_WIDE;
    if (wide && d->tsteps > d->halo) return JAC_EINVAL;   // sweeps per exchange <= ghost layers
    long long off = 0;
    for (int fc = 0; fc < 6; ++fc) {
        g->face_off[fc] = off;
        off += round_up(wide ? g->wface_elems[fc] : g->face_elems[fc], 16);  // 128-byte lines
    }
    g->send_stride = off;

    if (d->mode == JAC_MODE_TEMPORAL) {
        // whole lanes lie inside or outside the domain: 4 points per lane in 2D, 2 in 3D
        if (n[1] >= (1LL << 30)) return JAC_EINVAL;
        if (d->ndim == 2 && (b[0] % 4 != 0 || n[0] % 4 != 0)) return JAC_EINVAL;
        if (d->ndim == 3 && (b[0] % 2 != 0 || n[0] % 2 != 0 || d->tsteps > jac::kT3MaxT || n[2] >= (1LL << 30)))
            return JAC_EINVAL;
        // the 3D kernel keeps row offsets inside one z-layer of blocks in 32 bits
        if (d->ndim == 3 && g->block_stride * g->gx * g->gy >= (1LL << 31)) return JAC_EINVAL;
    }
    if (d->mode == JAC_MODE_RESIDENT) {
        ResidentPlan rp;
        if (plan_resident(*g, d->has_f != 0, d->tsteps, &rp)) return JAC_EINVAL;   // 3D, odd bx, or too large
    }
    const Tiling t = make_tiling(*g, kNominalSMs);
    const long long ctas = g->nblocks * t.ctas_per_block;
    if (ctas > kMaxGrid) return JAC_EINVAL;
    long long max_face = 0;
    for (int fc = 0; fc < 6; ++fc) max_face = std::max(max_face, wide ? g->wface_elems[fc] : g->face_elems[fc]);
    if (max_face >= (1LL << 31)) return JAC_EINVAL;
    if (wide && 2 * g->nblocks * ceil_div(round_up(max_face, 32), 256) > kMaxGrid) return JAC_EINVAL;
    if (g->nblocks * g->nfaces * ceil_div(round_up(ceil_div(max_face, 2), 32), 256) > kMaxGrid) return JAC_EINVAL;

    if (L) {
        std::memset(L, 0, sizeof(*L));
        for (int a = 0; a < 3; ++a) L->g[a] = gr[a];
        L->nblocks = g->nblocks;
        L->pad[0] = g->PX; L->pad[1] = PY; L->pad[2] = PZ;
        L->xpad = g->xpad;
        L->origin = g->origin;
        L->block_stride = g->block_stride;
        for (int fc = 0; fc < 6; ++fc) {
            L->face_elems[fc] = g->face_elems[fc];
            L->face_offset[fc] = g->face_off[fc];
        }
        L->send_stride = g->send_stride;
        for (int fc = 0; fc < 6; ++fc) L->wide_face_elems[fc] = g->wface_elems[fc];
        L->partials = round_up(max_partials(*g, ctas, d->has_f != 0, kNominalSMs), 32);
        const long long arr_bytes = round_up(g->nblocks * g->block_stride * 8, 256);
        long long o = 0;
        L->off_u[0] = o; o += arr_bytes;
        L->off_u[1] = o; o += arr_bytes;
        if (d->has_f) { L->off_f = o; o += arr_bytes; } else L->off_f = -1;
        L->off_send = o; o += round_up(g->nblocks * g->send_stride * 8, 256);
        L->off_scratch = o; o += round_up((L->partials + 32) * 8, 256);
        L->cut_elems = 0;
        for (int sd = 0; sd < 2; ++sd) L->off_cut_send[sd][0] = L->off_cut_send[sd][1] = L->off_cut_recv[sd] = -1;
        if (has_cut) {
            const int sa = d->ndim - 1;
            L->cut_elems = (g->nblocks / gr[sa]) * round_up(g->face_elems[2 * sa], 16);
            const long long cut_bytes = round_up(L->cut_elems * 8, 256);
            for (int sd = 0; sd < 2; ++sd) {
                if (!(d->flags & (sd ? JAC_FLAG_CUT_HI : JAC_FLAG_CUT_LO))) continue;
                L->off_cut_send[sd][0] = o; o += cut_bytes;
                L->off_cut_send[sd][1] = o; o += cut_bytes;
                L->off_cut_recv[sd] = o; o += cut_bytes;
            }
        }
        L->off_stage_in = L->off_stage_out = -1;
        if (d->flags & JAC_FLAG_HOST_STAGING) {
            const long long dense_bytes = round_up(n[0] * n[1] * n[2] * 8, 256);
            L->off_stage_in = o; o += dense_bytes;
            L->off_stage_out = o; o += dense_bytes;
        }
        L->total_bytes = o;
    }
    return JAC_OK;
}

}  // namespace

struct jac_ctx {
    jac_desc desc;
    JacGeom g;
    jac_layout L;
    Tiling tile;
    char* ws;
    double* u[2];
    double* f;
    double* send;
    double* partials;
    double* result;
    int sms;            // SMs of the device, as the launch planners use it
    int cur;            // which of u[] holds the current state
    bool ghosts_fresh;  // inter-block ghosts of u[cur] equal the neighbours' current faces
    bool packed_current;  // the send buffers hold the faces of the current state
    bool f_ghosts_fresh;  // JAC_MODE_WIDE: the ghost layers of f hold the neighbours' f
    int res_cluster;      // JAC_MODE_RESIDENT: CTAs per cluster settled at creation
    // JAC_FLAG_HOST_STAGING: dense arrays between the host and the blocks, a copy stream per
    // direction, and the events that order them against the caller's stream
    double* stage_in;
    double* stage_out;
    cudaStream_t h2d;
    cudaEvent_t ev_in_ready, ev_in_free, ev_out_done;
    // JAC_FLAG_CUT_*: the slab's cut planes (side 0 = low, 1 = high end of the slowest axis)
    bool cut[2];
    double* cut_send[2][2];   // [side][parity]: packs alternate between two buffers
    double* cut_recv[2];
    int cut_parity;           // buffer the last pack wrote
    bool cut_fresh;           // the cut ghosts of u[cur] hold the neighbour slabs' current faces
    bool in_sweep;            // jac_sweep_begin without its jac_sweep_end
    cudaStream_t aux;         // the blocks away from the cuts run here while the cut faces travel
    cudaEvent_t ev_fork, ev_join, ev_cut_ready[2];
    const char* d2h_lo;   // host range the last copy out writes (until the stream has passed it)
    const char* d2h_hi;
    cudaStream_t stream;
    int device;
    int cuda_err;       // sticky
    bool timed_out;     // sticky: a resident launch gave up a wait
    long long launches;
};

namespace {

#define JAC_CK(ctx, call)                                  \
    do {                                                   \
        cudaError_t e_ = (call);                           \
        if (e_ != cudaSuccess) {                           \
            (ctx)->cuda_err = (int)e_;                     \
            return JAC_ECUDA;                              \
        }                                                  \
    } while (0)

void release_copy_objects(jac_ctx* c)
{
    if (c->ev_in_ready) cudaEventDestroy(c->ev_in_ready);
    if (c->ev_in_free) cudaEventDestroy(c->ev_in_free);
    if (c->ev_out_done) cudaEventDestroy(c->ev_out_done);
    if (c->h2d) cudaStreamDestroy(c->h2d);
    c->ev_in_ready = c->ev_in_free = c->ev_out_done = nullptr;
    c->h2d = nullptr;
    if (c->ev_fork) cudaEventDestroy(c->ev_fork);
    if (c->ev_join) cudaEventDestroy(c->ev_join);
    for (int side = 0; side < 2; ++side)
        if (c->ev_cut_ready[side]) cudaEventDestroy(c->ev_cut_ready[side]);
    if (c->aux) cudaStreamDestroy(c->aux);
    c->ev_fork = c->ev_join = c->ev_cut_ready[0] = c->ev_cut_ready[1] = nullptr;
    c->aux = nullptr;
}

int check_launch(jac_ctx* c)
{
    c->launches++;
    JAC_CK(c, cudaGetLastError());
    return JAC_OK;
}

// ---- kernel dispatch ---------------------------------------------------------------
template <int NV, bool HAS_F, int OP>
void launch_sweep_t(jac_ctx* c, const double* u, double* un, long long blk0, long long nblk)
{
    const Tiling& t = c->tile;
    const unsigned grid = (unsigned)(nblk * t.ctas_per_block);
    // a launch over a sub-range of blocks writes its partial sums where a full launch would
    double* parts = c->partials + blk0 * t.ctas_per_block;
    if (c->g.ndim == 2)
        jac::sweep2d_kernel<NV, HAS_F, OP><<<grid, t.block, 0, c->stream>>>(
            u, un, c->f, parts, c->g, blk0, t.tiles_x, t.tiles_y, t.march);
    else
        jac::sweep3d_kernel<NV, HAS_F, OP><<<grid, t.block, 0, c->stream>>>(
            u, un, c->f, parts, c->g, blk0, t.tiles_x, t.tiles_y, t.tiles_z, t.march);
}

template <int OP>
int launch_sweep(jac_ctx* c, const double* u, double* un, long long blk0, long long nblk)
{
    const bool f = c->desc.has_f != 0;
    if (c->tile.nv == 2) {
        if (f) launch_sweep_t<2, true, OP>(c, u, un, blk0, nblk);
        else launch_sweep_t<2, false, OP>(c, u, un, blk0, nblk);
    } else {
        if (f) launch_sweep_t<1, true, OP>(c, u, un, blk0, nblk);
        else launch_sweep_t<1, false, OP>(c, u, un, blk0, nblk);
    }
    return check_launch(c);
}

// threads reserved per (block, face) pair, whole warps: a thread takes up to kHaloUnits units (a row
// of an x face, two cells of a line of a y or z face), and there are at least as many threads as a
// line has units, so that threads keep their column and walk over lines
int halo_slots(const jac_ctx* c, unsigned face_mask)
{
    const JacGeom& g = c->g;
    const long long vec_per_line = (g.bx % 2 == 0 && g.PX % 2 == 0) ? g.bx / 2 : g.bx;
    long long units = 1, line = 1;
    for (int fc = 0; fc < g.nfaces; ++fc) {
        if (!((face_mask >> fc) & 1u)) continue;
        if (fc < 2) units = std::max(units, g.face_elems[fc] / g.h);                 // rows
        else {
            units = std::max(units, g.face_elems[fc] / g.bx * vec_per_line);
            line = vec_per_line;
        }
    }
    return (int)round_up(std::max(ceil_div(units, jac::kHaloUnits), std::min<long long>(line, 1 << 20)), 32);
}

template <int OP>
int launch_halo(jac_ctx* c, long long pair0, long long npairs, unsigned face_mask)
{
    const int slots = halo_slots(c, face_mask);
    const long long ctas = ceil_div(npairs * slots, 256);
    if (ctas > kMaxGrid) return JAC_EINVAL;
    // 32-bit index arithmetic when thread and pair numbers fit (they do for any grid that fits a GPU)
    if (ctas * 256 < (1LL << 32) && c->g.nblocks * c->g.nfaces < (1LL << 31))
        jac::halo_kernel<OP, unsigned><<<(unsigned)ctas, 256, 0, c->stream>>>(c->u[c->cur], c->send, c->g, pair0,
                                                                            npairs, slots, face_mask);
    else
        jac::halo_kernel<OP, long long><<<(unsigned)ctas, 256, 0, c->stream>>>(c->u[c->cur], c->send, c->g, pair0,
                                                                             npairs, slots, face_mask);
    return check_launch(c);
}

// pack or unpack the faces in face_mask of all blocks in one launch
template <int OP>
int launch_halo_all(jac_ctx* c, unsigned face_mask = 0x3fu)
{
    return launch_halo<OP>(c, 0, c->g.nblocks * c->g.nfaces, face_mask);
}

bool has_neighbour(const JacGeom& g, long long blk, int face)
{
    const long long co[3] = {blk % g.gx, (blk / g.gx) % g.gy, blk / ((long long)g.gx * g.gy)};
    const int ga[3] = {g.gx, g.gy, g.gz};
    const int a = face >> 1;
    return (face & 1) ? co[a] + 1 < ga[a] : co[a] > 0;
}

// one launch per (block, face) that has a neighbour: the task-per-block schedule
template <int OP>
int launch_halo_pertask(jac_ctx* c)
{
    for (long long blk = 0; blk < c->g.nblocks; ++blk)
        for (int face = 0; face < c->g.nfaces; ++face) {
            if (!has_neighbour(c->g, blk, face)) continue;
            const int rc = launch_halo<OP>(c, blk * c->g.nfaces + face, 1, 1u << face);
            if (rc) return rc;
        }
    return JAC_OK;
}

int do_pack(jac_ctx* c)
{
    return c->desc.mode == JAC_MODE_PERTASK ? launch_halo_pertask<jac::HALO_PACK>(c) : launch_halo_all<jac::HALO_PACK>(c);
}
int do_unpack(jac_ctx* c)
{
    return c->desc.mode == JAC_MODE_PERTASK ? launch_halo_pertask<jac::HALO_UNPACK>(c) : launch_halo_all<jac::HALO_UNPACK>(c);
}

// pack and unpack of all faces in one launch (same buffers and ghosts afterwards)
int do_exchange_fused(jac_ctx* c)
{
    const int rc = launch_halo_all<jac::HALO_EXCHANGE>(c);
    if (rc) return rc;
    c->packed_current = true;
    c->ghosts_fresh = true;
    return JAC_OK;
}

// the exchange before an update: pack and unpack as one launch (the task-per-block schedule keeps
// them apart, one launch per block face each)
int do_exchange(jac_ctx* c)
{
    if (c->desc.mode != JAC_MODE_PERTASK) return do_exchange_fused(c);
    int rc = do_pack(c);
    if (rc) return rc;
    c->packed_current = true;
    rc = do_unpack(c);
    if (rc) return rc;
    c->ghosts_fresh = true;
    return JAC_OK;
}

// ---- wide exchange and the updates between two of them ------------------------------
// all h ghost layers of `arr`, edges and corners included: per axis one pack and one unpack launch
int do_exchange_wide(jac_ctx* c, double* arr)
{
    for (int axis = 0; axis < c->g.ndim; ++axis) {
        const long long n = c->g.wface_elems[2 * axis];
        const int slots = (int)round_up(n, 32);
        const long long ctas = ceil_div(2 * c->g.nblocks * slots, 256);
        if (ctas > kMaxGrid) return JAC_EINVAL;
        const bool narrow = ctas * 256 < (1LL << 32) && 2 * c->g.nblocks < (1LL << 31);
        if (narrow) jac::halo_wide_kernel<false, unsigned><<<(unsigned)ctas, 256, 0, c->stream>>>(arr, c->send, c->g, axis, slots);
        else jac::halo_wide_kernel<false, long long><<<(unsigned)ctas, 256, 0, c->stream>>>(arr, c->send, c->g, axis, slots);
        int rc = check_launch(c);
        if (rc) return rc;
        if (narrow) jac::halo_wide_kernel<true, unsigned><<<(unsigned)ctas, 256, 0, c->stream>>>(arr, c->send, c->g, axis, slots);
        else jac::halo_wide_kernel<true, long long><<<(unsigned)ctas, 256, 0, c->stream>>>(arr, c->send, c->g, axis, slots);
        if ((rc = check_launch(c))) return rc;
    }
    return JAC_OK;
}

// the update over every block's interior grown by e >= 1 layers (positions outside the domain keep
// their value): the ordinary sweep kernels on a geometry whose block box is the grown one
template <int NV, bool HAS_F>
void launch_ext_t(jac_ctx* c, const JacGeom& ge, const Tiling& t, const double* u, double* un)
{
    const unsigned grid = (unsigned)(ge.nblocks * t.ctas_per_block);
    if (ge.ndim == 2)
        jac::sweep2d_kernel<NV, HAS_F, jac::OP_UPDATE_EXT><<<grid, t.block, 0, c->stream>>>(
            u, un, c->f, nullptr, ge, 0, t.tiles_x, t.tiles_y, t.march);
    else
        jac::sweep3d_kernel<NV, HAS_F, jac::OP_UPDATE_EXT><<<grid, t.block, 0, c->stream>>>(
            u, un, c->f, nullptr, ge, 0, t.tiles_x, t.tiles_y, t.tiles_z, t.march);
}

int launch_ext(jac_ctx* c, int e, const double* u, double* un)
{
    JacGeom ge = c->g;
    ge.ext = e;
    ge.bx += 2 * e; ge.rx += 2 * e;
    ge.by += 2 * e; ge.ry += 2 * e;
    ge.origin -= (long long)e * ge.PX + e;
    if (ge.ndim == 3) {
        ge.bz += 2 * e; ge.rz += 2 * e;
        ge.origin -= (long long)e * ge.PXY;
    }
    // 128-bit accesses need the first column of the grown box on a 16-byte boundary: e even
    const Tiling t = make_tiling(ge, c->sms, (e % 2 != 0) ? 1 : 0);
    if (ge.nblocks * t.ctas_per_block > kMaxGrid) return JAC_EINVAL;
    const bool f = c->desc.has_f != 0;
    if (t.nv == 2) {
        if (f) launch_ext_t<2, true>(c, ge, t, u, un);
        else launch_ext_t<2, false>(c, ge, t, u, un);
    } else {
        if (f) launch_ext_t<1, true>(c, ge, t, u, un);
        else launch_ext_t<1, false>(c, ge, t, u, un);
    }
    return check_launch(c);
}

// ---- strided box copies between a dense array and the padded blocks ------------------
cudaError_t copy_box(void* dst, size_t dpitch, size_t drows, const void* src, size_t spitch,
                     size_t srows, size_t width_bytes, size_t height, size_t depth,
                     cudaMemcpyKind kind, cudaStream_t st)
{
    cudaMemcpy3DParms p;
    std::memset(&p, 0, sizeof(p));
    p.srcPtr = make_cudaPitchedPtr(const_cast<void*>(src), spitch, width_bytes, srows);
    p.dstPtr = make_cudaPitchedPtr(dst, dpitch, width_bytes, drows);
    p.extent = make_cudaExtent(width_bytes, height, depth);
    p.kind = kind;
    return cudaMemcpy3DAsync(&p, st);
}

// host dense <-> interiors of all blocks of `arr`
int copy_dense_host(jac_ctx* c, double* arr, double* host, bool to_device, bool wait = true)
{
    const JacGeom& g = c->g;
    const size_t PY = (size_t)(g.PXY / g.PX);
    for (long long blk = 0; blk < g.nblocks; ++blk) {
        const long long bxi = blk % g.gx, byi = (blk / g.gx) % g.gy, bzi = blk / ((long long)g.gx * g.gy);
        double* dev = arr + blk * g.block_stride + g.origin;
        double* hp = host + ((bzi * g.bz) * g.ny + byi * g.by) * g.nx + bxi * g.bx;
        // interior extent of this block (the last one along an axis may be a remainder block)
        const size_t ex = bxi + 1 == g.gx ? g.rx : g.bx, ey = byi + 1 == g.gy ? g.ry : g.by,
                     ez = bzi + 1 == g.gz ? g.rz : g.bz;
        cudaError_t e;
        if (to_device)
            e = copy_box(dev, g.PX * 8, PY, hp, g.nx * 8, g.ny, ex * 8, ey, ez,
                         cudaMemcpyHostToDevice, c->stream);
        else
            e = copy_box(hp, g.nx * 8, g.ny, dev, g.PX * 8, PY, ex * 8, ey, ez,
                         cudaMemcpyDeviceToHost, c->stream);
        JAC_CK(c, e);
    }
    if (wait) JAC_CK(c, cudaStreamSynchronize(c->stream));
    return JAC_OK;
}

template <bool TO_BLOCKS>
int copy_dense_device(jac_ctx* c, double* arr, double* dense)
{
    const JacGeom& g = c->g;
    const int nv = ((g.bx % 2 == 0) && (g.nx % 2 == 0) && (((uintptr_t)dense & 15u) == 0)) ? 2 : 1;
    const int segs = (int)ceil_div(ceil_div(g.nx, nv), 256);
    const long long ctas = g.ny * g.nz * segs;
    if (ctas > kMaxGrid) return JAC_EINVAL;
    if (nv == 2)
        jac::dense_copy_kernel<TO_BLOCKS, 2><<<(unsigned)ctas, 256, 0, c->stream>>>(arr, dense, g, segs);
    else
        jac::dense_copy_kernel<TO_BLOCKS, 1><<<(unsigned)ctas, 256, 0, c->stream>>>(arr, dense, g, segs);
    return check_launch(c);
}

// ---- JAC_FLAG_HOST_STAGING: one contiguous copy per direction through a dense staging array ----
// Copy in: host -> staging array on the context's own host-to-device stream, then (on the caller's
// stream, after an event) the kernel that scatters the dense array into the blocks.  The copy does
// not queue behind the work already on the caller's stream -- the sweeps of the previous job, its
// copy out -- so it overlaps them (the two copy directions and the SMs are separate engines); it
// only waits until the staging array is free again and, if the host range is the target of a copy
// out that is still in flight, for that copy.
int staged_in(jac_ctx* c, double* arr, const double* host, bool wait)
{
    const size_t bytes = (size_t)(c->g.nx * c->g.ny * c->g.nz) * sizeof(double);
    JAC_CK(c, cudaStreamWaitEvent(c->h2d, c->ev_in_free, 0));
    const char* lo = reinterpret_cast<const char*>(host);
    if (c->d2h_lo && lo < c->d2h_hi && c->d2h_lo < lo + bytes) JAC_CK(c, cudaStreamWaitEvent(c->h2d, c->ev_out_done, 0));
    JAC_CK(c, cudaMemcpyAsync(c->stage_in, host, bytes, cudaMemcpyHostToDevice, c->h2d));
    JAC_CK(c, cudaEventRecord(c->ev_in_ready, c->h2d));
    JAC_CK(c, cudaStreamWaitEvent(c->stream, c->ev_in_ready, 0));
    const int rc = copy_dense_device<true>(c, arr, c->stage_in);
    if (rc) return rc;
    JAC_CK(c, cudaEventRecord(c->ev_in_free, c->stream));
    if (wait) JAC_CK(c, cudaStreamSynchronize(c->stream));
    return JAC_OK;
}

// Copy out: the kernel that gathers the blocks into the dense staging array, then one contiguous
// copy to the host, both on the caller's stream.
int staged_out(jac_ctx* c, double* arr, double* host, bool wait)
{
    const size_t bytes = (size_t)(c->g.nx * c->g.ny * c->g.nz) * sizeof(double);
    const int rc = copy_dense_device<false>(c, arr, c->stage_out);
    if (rc) return rc;
    JAC_CK(c, cudaMemcpyAsync(host, c->stage_out, bytes, cudaMemcpyDeviceToHost, c->stream));
    JAC_CK(c, cudaEventRecord(c->ev_out_done, c->stream));
    c->d2h_lo = reinterpret_cast<const char*>(host);
    c->d2h_hi = c->d2h_lo + bytes;
    if (wait) JAC_CK(c, cudaStreamSynchronize(c->stream));
    return JAC_OK;
}

// is this host memory page-locked (allocated or registered with CUDA)?  Only then is a copy on a
// stream of the library's own ordered by the events around it: the runtime moves pageable memory
// through a staging buffer of its own, on its own schedule.
bool is_pinned(const void* host)
{
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, host) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return at.type == cudaMemoryTypeHost;
}

// dense host array <-> blocks, by whichever route the context has (the staging arrays serve
// page-locked host memory; pageable memory takes the per-block copies on the caller's stream)
int host_to_blocks(jac_ctx* c, double* arr, const double* host, bool wait)
{
    return (c->stage_in && is_pinned(host)) ? staged_in(c, arr, host, wait)
                                            : copy_dense_host(c, arr, const_cast<double*>(host), true, wait);
}
int blocks_to_host(jac_ctx* c, double* arr, double* host, bool wait)
{
    return (c->stage_out && is_pinned(host)) ? staged_out(c, arr, host, wait) : copy_dense_host(c, arr, host, false, wait);
}

int usable(jac_ctx* c)
{
    if (!c) return JAC_EINVAL;
    if (c->cuda_err) return JAC_ECUDA;
    if (c->timed_out) return JAC_ETIMEOUT;
    return JAC_OK;
}

// Sweeps per launch when the caller leaves the choice to the library.  2D without a right-hand
// side: 8 on grids large enough to fill the GPU with long strips (measured: 16384^2 1817 vs 1356
// GLUP/s at 4), else 4 (4096^2: 1041 vs 1032).  2D with a right-hand side: 6 (4096^2: 702 GLUP/s
// against 671 at 4 and 577 at 8, whose windows plus the f row no longer fit the registers; 8192^2:
// 841 / 732 / 786).  3D: 3.
int default_tsteps(const jac_desc& d)
{
    if (d.tsteps > 0) return d.tsteps;
    if (d.ndim == 3) return 3;
    if (d.has_f) return 6;
    const bool large = d.n[0] * d.n[1] >= (1LL << 26);
    return large ? 8 : 4;
}

// The dynamic shared memory a kernel may use is an attribute of the kernel on a device: set it the
// first time the kernel is launched on that device, not on every launch (the call costs host time,
// which the launch-bound small grids feel).
template <auto Kern>
int ensure_dynamic_smem(jac_ctx* c, size_t smem)
{
    static std::atomic<unsigned long long> done{0};      // one bit per device ordinal
    const unsigned long long bit = 1ULL << (c->device & 63);
    if (c->device < 64 && (done.load(std::memory_order_acquire) & bit)) return JAC_OK;
    JAC_CK(c, cudaFuncSetAttribute(Kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    done.fetch_or(bit, std::memory_order_release);
    return JAC_OK;
}

// T sweeps in one launch (3D, tiles of 64 x 24 streamed along z).  RES = 1..T: level RES also leaves
// per-warp partial sums of the squared residual of the state it reads (the one after RES - 1 sweeps
// of the launch); 0: none.
template <int T, bool HAS_F, int RES>
int launch_temporal3d_t(jac_ctx* c, const double* u, double* un, long long* nparts)
{
    const TemporalGrid t = temporal_grid_3d(c->g, T, c->sms);
    if (t.ctas > kMaxGrid) return JAC_EINVAL;
    constexpr auto kern = jac::temporal3d_kernel<T, HAS_F, RES>;
    const size_t smem = jac::t3_smem_bytes(T, HAS_F);
    const int rc = ensure_dynamic_smem<kern>(c, smem);
    if (rc) return rc;
    kern<<<(unsigned)t.ctas, jac::kT3Warps * 32, smem, c->stream>>>(u, un, c->f, c->partials, c->g, t.a, t.b, t.c,
                                                                   t.chunk);
    if (RES != 0) *nparts = t.warps;
    return check_launch(c);
}

// T sweeps in one launch (2D, register-streaming temporal blocking); RES as above
template <int T, bool HAS_F, int RES>
int launch_temporal2d_t(jac_ctx* c, const double* u, double* un, long long* nparts)
{
    const TemporalGrid t = temporal_grid_2d(c->g, T, HAS_F, c->sms);
    constexpr auto kern = jac::temporal2d_kernel<T, HAS_F, RES>;
    const size_t smem = jac::temporal_smem_bytes(T, HAS_F);
    if (smem > 48 * 1024) {
        const int rc = ensure_dynamic_smem<kern>(c, smem);
        if (rc) return rc;
    }
    kern<<<(unsigned)t.ctas, jac::kTemporalWarps * 32, smem, c->stream>>>(u, un, c->f, c->partials, c->g, t.a, t.b,
                                                                         t.chunk);
    if (RES != 0) *nparts = t.warps;
    return check_launch(c);
}

// the run-time depth t and measuring level (0..t) picked out of the compiled ones
template <int NDIM, int T, int RES>
int launch_temporal_tr(jac_ctx* c, const double* u, double* un, long long* nparts)
{
    if constexpr (RES > T) {
        return JAC_EINVAL;
    } else if constexpr (NDIM == 2) {
        return c->desc.has_f ? launch_temporal2d_t<T, true, RES>(c, u, un, nparts)
                             : launch_temporal2d_t<T, false, RES>(c, u, un, nparts);
    } else {
        return c->desc.has_f ? launch_temporal3d_t<T, true, RES>(c, u, un, nparts)
                             : launch_temporal3d_t<T, false, RES>(c, u, un, nparts);
    }
}

template <int NDIM, int T>
int launch_temporal_level(jac_ctx* c, int level, const double* u, double* un, long long* nparts)
{
    switch (level) {
        case 0: return launch_temporal_tr<NDIM, T, 0>(c, u, un, nparts);
        case 1: return launch_temporal_tr<NDIM, T, 1>(c, u, un, nparts);
        case 2: return launch_temporal_tr<NDIM, T, 2>(c, u, un, nparts);
        case 3: return launch_temporal_tr<NDIM, T, 3>(c, u, un, nparts);
        case 4: return launch_temporal_tr<NDIM, T, 4>(c, u, un, nparts);
        case 5: return launch_temporal_tr<NDIM, T, 5>(c, u, un, nparts);
        case 6: return launch_temporal_tr<NDIM, T, 6>(c, u, un, nparts);
        case 7: return launch_temporal_tr<NDIM, T, 7>(c, u, un, nparts);
        case 8: return launch_temporal_tr<NDIM, T, 8>(c, u, un, nparts);
        default: return JAC_EINVAL;
    }
}

// one temporal launch of depth t whose level `level` (1..t; 0: none) measures the residual
int launch_temporal_n(jac_ctx* c, int t, const double* u, double* un, int level, long long* nparts)
{
    if (level < 0 || level > t) return JAC_EINVAL;
    if (c->g.ndim == 3) {
        switch (t) {
            case 1: return launch_temporal_level<3, 1>(c, level, u, un, nparts);
            case 2: return launch_temporal_level<3, 2>(c, level, u, un, nparts);
            case 3: return launch_temporal_level<3, 3>(c, level, u, un, nparts);
            default: return JAC_EINVAL;
        }
    }
    switch (t) {
        case 1: return launch_temporal_level<2, 1>(c, level, u, un, nparts);
        case 2: return launch_temporal_level<2, 2>(c, level, u, un, nparts);
        case 3: return launch_temporal_level<2, 3>(c, level, u, un, nparts);
        case 4: return launch_temporal_level<2, 4>(c, level, u, un, nparts);
        case 5: return launch_temporal_level<2, 5>(c, level, u, un, nparts);
        case 6: return launch_temporal_level<2, 6>(c, level, u, un, nparts);
        case 7: return launch_temporal_level<2, 7>(c, level, u, un, nparts);
        case 8: return launch_temporal_level<2, 8>(c, level, u, un, nparts);
        default: return JAC_EINVAL;
    }
}

// nsweeps sweeps in ONE launch of one thread-block cluster that keeps the grid in shared memory
template <bool HAS_F>
int launch_resident_t(jac_ctx* c, const ResidentPlan& rp, const double* u, double* un, int nsweeps)
{
    // the kernel's attributes (shared memory, cluster size) were set when the context was created
    auto kern = jac::resident2d_kernel<HAS_F>;
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)rp.cluster, 1, 1);
    cfg.blockDim = dim3(jac::kResThreads, 1, 1);
    cfg.dynamicSmemBytes = rp.smem;
    cfg.stream = c->stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)rp.cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    JAC_CK(c, cudaLaunchKernelEx(&cfg, kern, u, un, (const double*)c->f, c->g, nsweeps, rp.rows, reinterpret_cast<int*>(c->result + 4)));
    return check_launch(c);
}

int launch_resident(jac_ctx* c, const double* u, double* un, int nsweeps)
{
    ResidentPlan rp;
    if (plan_resident(c->g, c->desc.has_f != 0, c->res_cluster, &rp)) return JAC_EINVAL;
    return c->desc.has_f ? launch_resident_t<true>(c, rp, u, un, nsweeps)
                         : launch_resident_t<false>(c, rp, u, un, nsweeps);
}

// can a cluster of `cluster` CTAs be scheduled on this device at all? (16 CTAs with most of an
// SM's shared memory each need a GPC with 16 free SMs)
int resident_cluster_schedulable(jac_ctx* c, int cluster, bool* ok)
{
    ResidentPlan rp;
    *ok = false;
    if (plan_resident(c->g, c->desc.has_f != 0, cluster, &rp)) return JAC_OK;   // does not fit shared memory
    const void* kern = c->desc.has_f ? (const void*)jac::resident2d_kernel<true>
                                     : (const void*)jac::resident2d_kernel<false>;
    // once per context, and to the largest size any context may ask for, so that contexts of
    // different grids do not undo each other's setting
    JAC_CK(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxSmemPerCta));
    JAC_CK(c, cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)rp.cluster, 1, 1);
    cfg.blockDim = dim3(jac::kResThreads, 1, 1);
    cfg.dynamicSmemBytes = rp.smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)rp.cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int nclusters = 0;
    JAC_CK(c, cudaOccupancyMaxActiveClusters(&nclusters, kern, &cfg));
    *ok = nclusters >= 1;
    return JAC_OK;
}

// settles the cluster size of a resident context: the caller's, or the planner's first choice
// that the device can schedule
int choose_resident_cluster(jac_ctx* c)
{
    ResidentPlan rp;
    if (plan_resident(c->g, c->desc.has_f != 0, c->desc.tsteps, &rp)) return JAC_EINVAL;
    const int tries[2] = {rp.cluster, c->desc.tsteps ? rp.cluster : 24 - rp.cluster};
    for (int k = 0; k < 2; ++k) {
        bool ok = false;
        const int rc = resident_cluster_schedulable(c, tries[k], &ok);
        if (rc) return rc;
        if (ok) {
            c->res_cluster = tries[k];
            return JAC_OK;
        }
    }
    return JAC_EINVAL;
}

// Relative cost of one temporal launch of depth t: a pass over memory plus t levels, per output
// column (2D: a strip stores 120 of its 128 columns up to t = 4 and 112 beyond, so t = 5 pays for
// halo lanes that t = 8 would use too).  Fitted to launch times on 4096^2 with f (0.107 / 0.135 /
// 0.1425 ms at t = 4 / 5 / 6), 16384^2 without (0.750 / 1.141 ms at t = 4 / 8) and 1024^3 with f
// (5.11 / 6.13 / 7.65 ms at t = 1 / 2 / 3).
double temporal_launch_cost(int ndim, bool has_f, int t)
{
    if (ndim == 3) return t == 1 ? 5.11 : t == 2 ? 6.13 : 7.65;
    return ((has_f ? 2.0 : 3.7) + t) * 120.0 / jac::temporal_strip_cols(t);
}

// Depths of the launches that make up nsweeps sweeps at depth <= T: as few launches as the depth
// allows (a launch of one sweep costs most of what a launch of T does); all but the last few at
// full depth, and the last (up to four) share what is left in the cheapest way by the cost above
// -- ten sweeps at T = 6 run as 6 + 4, not 5 + 5; ten at T = 3 as 3 + 3 + 2 + 2.
void temporal_depths(int nsweeps, int T, int ndim, bool has_f, std::vector<int>* depths)
{
    depths->clear();
    const int launches = (nsweeps + T - 1) / T;
    const int m = std::min(launches, 4);
    for (int k = 0; k < launches - m; ++k) depths->push_back(T);
    const int tail = nsweeps - (launches - m) * T;
    int best[4] = {0, 0, 0, 0}, cur[4] = {0, 0, 0, 0};
    double best_cost = 1e300;
    // non-increasing depths cur[0] >= cur[1] >= ... summing to tail
    auto rec = [&](auto&& self, int k, int left, int cap, double cost) -> void {
        if (k == m) {
            if (left == 0 && cost < best_cost - 1e-12) {
                best_cost = cost;
                std::copy(cur, cur + 4, best);
            }
            return;
        }
        for (int t = std::min(cap, left - (m - k - 1)); t >= 1; --t) {
            if ((long long)t * (m - k) < left) break;   // the rest cannot be covered by depths <= t
            cur[k] = t;
            self(self, k + 1, left - t, t, cost + temporal_launch_cost(ndim, has_f, t));
        }
    };
    rec(rec, 0, tail, T, 0.0);
    for (int k = 0; k < m; ++k) depths->push_back(best[k]);
}

// nsweeps iterations in the context's schedule.  res (jac::kRes*): one launch also leaves partial
// sums of the squared residual in the scratch (*nparts of them) -- kResBeforeLast: the last sweep,
// of the state it reads; kResOfInput: the first sweep, of the state the call starts from.
int run_sweeps(jac_ctx* c, int nsweeps, int res, long long* nparts)
{
    int rc = JAC_OK;
    if (c->cut[0] || c->cut[1]) return JAC_EINVAL;   // a slab sweeps through jac_sweep_begin / jac_sweep_end
    const JacGeom& g = c->g;
    const long long sweep_parts = g.nblocks * c->tile.ctas_per_block;
    // does sweep number s (0-based) of the call carry the residual?
    auto carries = [&](int s) {
        return (res == jac::kResBeforeLast && s + 1 == nsweeps) || (res == jac::kResOfInput && s == 0);
    };
    switch (c->desc.mode) {
        case JAC_MODE_FUSED:
            for (int s = 0; s < nsweeps; ++s) {
                rc = carries(s) ? launch_sweep<jac::OP_UPDATE_PULL_RES>(c, c->u[c->cur], c->u[c->cur ^ 1], 0, g.nblocks)
                                : launch_sweep<jac::OP_UPDATE_PULL>(c, c->u[c->cur], c->u[c->cur ^ 1], 0, g.nblocks);
                if (rc) return rc;
                c->cur ^= 1;
            }
            if (res) *nparts = sweep_parts;
            c->ghosts_fresh = false;
            c->packed_current = false;
            break;
        case JAC_MODE_EXCHANGE:
            for (int s = 0; s < nsweeps; ++s) {
                if ((rc = do_exchange(c))) return rc;
                rc = carries(s) ? launch_sweep<jac::OP_UPDATE_RES>(c, c->u[c->cur], c->u[c->cur ^ 1], 0, g.nblocks)
                                : launch_sweep<jac::OP_UPDATE>(c, c->u[c->cur], c->u[c->cur ^ 1], 0, g.nblocks);
                if (rc) return rc;
                c->cur ^= 1;
                c->ghosts_fresh = false;
                c->packed_current = false;
            }
            if (res) *nparts = sweep_parts;
            break;
        case JAC_MODE_PERTASK:
            for (int s = 0; s < nsweeps; ++s) {
                if ((rc = do_exchange(c))) return rc;
                for (long long blk = 0; blk < g.nblocks; ++blk) {
                    rc = carries(s) ? launch_sweep<jac::OP_UPDATE_RES>(c, c->u[c->cur], c->u[c->cur ^ 1], blk, 1)
                                    : launch_sweep<jac::OP_UPDATE>(c, c->u[c->cur], c->u[c->cur ^ 1], blk, 1);
                    if (rc) return rc;
                }
                c->cur ^= 1;
                c->ghosts_fresh = false;
                c->packed_current = false;
            }
            if (res) *nparts = sweep_parts;
            break;
        case JAC_MODE_TEMPORAL: {
            const int T = default_tsteps(c->desc);
            std::vector<int> depths;
            temporal_depths(nsweeps, T, g.ndim, c->desc.has_f != 0, &depths);
            for (int k = 0, left = nsweeps; left > 0; ++k) {
                const int t = depths[(size_t)k];
                // the level that measures: the top one of the last launch, the first one of the first
                const int level = (res == jac::kResBeforeLast && left == t) ? t
                                  : (res == jac::kResOfInput && k == 0)     ? 1
                                                                            : 0;
                if ((rc = launch_temporal_n(c, t, c->u[c->cur], c->u[c->cur ^ 1], level, nparts))) return rc;
                c->cur ^= 1;
                left -= t;
            }
            c->ghosts_fresh = false;
            c->packed_current = false;
            break;
        }
        case JAC_MODE_RESIDENT: {
            // all sweeps in one launch; a residual-carrying first or last sweep runs as one ordinary launch
            const int n_res = res ? nsweeps - 1 : nsweeps;
            if (res == jac::kResOfInput) {
                if ((rc = launch_sweep<jac::OP_UPDATE_PULL_RES>(c, c->u[c->cur], c->u[c->cur ^ 1], 0, g.nblocks)))
                    return rc;
                c->cur ^= 1;
                *nparts = sweep_parts;
            }
            if (n_res > 0) {
                if ((rc = launch_resident(c, c->u[c->cur], c->u[c->cur ^ 1], n_res))) return rc;
                c->cur ^= 1;
            }
            if (res == jac::kResBeforeLast) {
                if ((rc = launch_sweep<jac::OP_UPDATE_PULL_RES>(c, c->u[c->cur], c->u[c->cur ^ 1], 0, g.nblocks)))
                    return rc;
                c->cur ^= 1;
                *nparts = sweep_parts;
            }
            c->ghosts_fresh = false;
            c->packed_current = false;
            break;
        }
        case JAC_MODE_WIDE: {
            // groups of up to K sweeps (K <= h): one wide exchange, then updates on boxes shrinking
            // from the interior grown by t - 1 layers down to the interior itself
            if (res == jac::kResOfInput) return JAC_EINVAL;   // the first update of a group runs on a grown box
            const int K = c->desc.tsteps > 0 ? c->desc.tsteps : g.h;
            if (c->f && !c->f_ghosts_fresh) {
                if ((rc = do_exchange_wide(c, c->f))) return rc;
                c->f_ghosts_fresh = true;
            }
            for (int left = nsweeps; left > 0;) {
                const int t = std::min(K, left);
                if ((rc = do_exchange_wide(c, c->u[c->cur]))) return rc;
                for (int m = 1; m <= t; ++m) {
                    const int e = t - m;
                    const bool last = res && left == t && e == 0;
                    if (e > 0) rc = launch_ext(c, e, c->u[c->cur], c->u[c->cur ^ 1]);
                    else rc = last ? launch_sweep<jac::OP_UPDATE_RES>(c, c->u[c->cur], c->u[c->cur ^ 1], 0, g.nblocks)
                                   : launch_sweep<jac::OP_UPDATE>(c, c->u[c->cur], c->u[c->cur ^ 1], 0, g.nblocks);
                    if (rc) return rc;
                    c->cur ^= 1;
                }
                left -= t;
            }
            if (res) *nparts = sweep_parts;
            c->ghosts_fresh = false;
            c->packed_current = false;
            break;
        }
        default:
            return JAC_EINVAL;
    }
    return JAC_OK;
}

// End of one group of jac_solve's sweeps, on the device: the group's partial sums are added in the
// usual fixed order, the norm and the sweeps done so far are recorded, and once the norm has met
// the tolerance a flag goes up that turns every later launch of the call into a no-op.
// result: [0] sum of squares, [1] its root; stop, done: the flag and the sweep count.
__global__ void __launch_bounds__(1024)
solve_check_kernel(const double* __restrict__ partials, const long long n, const double tol, const int group_sweeps,
                   double* __restrict__ result, int* __restrict__ stop, int* __restrict__ done)
{
    if (*stop != 0) return;
    double acc = 0.0;
    for (long long i = threadIdx.x; i < n; i += blockDim.x) acc = jac::add_rn(acc, partials[i]);
    const double total = jac::block_sum(acc);
    if (threadIdx.x == 0) {
        const double norm = sqrt(total);          // correctly rounded, as std::sqrt on the host
        result[0] = total;
        result[1] = norm;
        *done += group_sweeps;
        if (norm <= tol) *stop = 1;
    }
}

// fixed-order sum of the first nparts partial sums -> host, as a norm
// has a resident launch given up a wait?  (call after the stream has been waited for)
int check_timeout(jac_ctx* c)
{
    if (c->desc.mode != JAC_MODE_RESIDENT) return JAC_OK;
    int flag = 0;
    JAC_CK(c, cudaMemcpyAsync(&flag, c->result + 4, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
    JAC_CK(c, cudaStreamSynchronize(c->stream));
    if (flag) {
        c->timed_out = true;
        return JAC_ETIMEOUT;
    }
    return JAC_OK;
}

int finish_norm(jac_ctx* c, long long nparts, double* host_out_l2)
{
    jac::reduce_partials_kernel<<<1, 1024, 0, c->stream>>>(c->partials, nparts, c->result, false);
    int rc = check_launch(c);
    if (rc) return rc;
    double sum = 0.0;
    JAC_CK(c, cudaMemcpyAsync(&sum, c->result, sizeof(double), cudaMemcpyDeviceToHost, c->stream));
    JAC_CK(c, cudaStreamSynchronize(c->stream));
    if ((rc = check_timeout(c))) return rc;
    *host_out_l2 = std::sqrt(sum);
    return JAC_OK;
}

// ---- slab contexts (JAC_FLAG_CUT_*): the faces that cross a cut ------------------------------
bool has_cuts(const jac_ctx* c) { return c->cut[0] || c->cut[1]; }

struct PlaneRange { long long blk0, nblk; };

// the blocks of the slab's first (side 0) or last (side 1) plane along the slowest axis: blocks are
// numbered x fastest, so a plane is a contiguous range
PlaneRange cut_plane(const jac_ctx* c, int side)
{
    const int gs = c->g.ndim == 2 ? c->g.gy : c->g.gz;
    const long long per_plane = c->g.nblocks / gs;
    return PlaneRange{side ? (gs - 1) * per_plane : 0, per_plane};
}

template <bool UNPACK>
int launch_cut(jac_ctx* c, int side, double* arr, double* buf)
{
    const PlaneRange r = cut_plane(c, side);
    const int face = 2 * (c->g.ndim - 1) + side;
    const long long slot = round_up(c->g.face_elems[face], 16);
    const int slots = (int)round_up(ceil_div(c->g.face_elems[face], 2), 32);
    const long long ctas = ceil_div(r.nblk * slots, 256);
    if (ctas > kMaxGrid) return JAC_EINVAL;
    jac::cut_kernel<UNPACK><<<(unsigned)ctas, 256, 0, c->stream>>>(arr, buf, c->g, r.blk0, r.nblk, slots, face, slot);
    return check_launch(c);
}

// the cut faces of `arr` into the send buffers the previous pack did not use; an event per side
// tells a reader on another stream when its buffer is complete
int pack_cuts(jac_ctx* c, double* arr)
{
    c->cut_parity ^= 1;
    for (int side = 0; side < 2; ++side) {
        if (!c->cut[side]) continue;
        const int rc = launch_cut<false>(c, side, arr, c->cut_send[side][c->cut_parity]);
        if (rc) return rc;
        JAC_CK(c, cudaEventRecord(c->ev_cut_ready[side], c->stream));
    }
    return JAC_OK;
}

// the cut ghost layers of `arr` from packed planes: src[side] (a device pointer, e.g. the neighbour
// slab's send buffer; after `ready[side]` if given) or the context's own receive buffer
int unpack_cuts(jac_ctx* c, double* arr, const double* const src[2], void* const ready[2])
{
    for (int side = 0; side < 2; ++side) {
        if (!c->cut[side]) continue;
        if (ready[side]) JAC_CK(c, cudaStreamWaitEvent(c->stream, static_cast<cudaEvent_t>(ready[side]), 0));
        double* from = src[side] ? const_cast<double*>(src[side]) : c->cut_recv[side];
        const int rc = launch_cut<true>(c, side, arr, from);
        if (rc) return rc;
    }
    return JAC_OK;
}

// First half of a sweep of a slab: the planes of blocks next to a cut are updated first and their
// new cut faces packed, so that they can travel while the rest of the slab is updated on the
// context's second stream.
int slab_sweep_begin(jac_ctx* c)
{
    const JacGeom& g = c->g;
    const bool exch = c->desc.mode == JAC_MODE_EXCHANGE;
    int rc;
    if (exch && (rc = do_exchange(c))) return rc;       // the faces between the slab's own blocks
    const double* u = c->u[c->cur];
    double* un = c->u[c->cur ^ 1];
    const int gs = g.ndim == 2 ? g.gy : g.gz;
    const long long per_plane = g.nblocks / gs;
    JAC_CK(c, cudaEventRecord(c->ev_fork, c->stream));
    JAC_CK(c, cudaStreamWaitEvent(c->aux, c->ev_fork, 0));
    // planes next to a cut (one plane may be next to both)
    for (int side = 0; side < 2; ++side) {
        if (!c->cut[side] || (side == 1 && gs == 1 && c->cut[0])) continue;
        const PlaneRange r = cut_plane(c, side);
        rc = exch ? launch_sweep<jac::OP_UPDATE>(c, u, un, r.blk0, r.nblk)
                  : launch_sweep<jac::OP_UPDATE_PULL>(c, u, un, r.blk0, r.nblk);
        if (rc) return rc;
    }
    if ((rc = pack_cuts(c, un))) return rc;
    // the planes in between, meanwhile
    const long long p0 = c->cut[0] ? 1 : 0, p1 = c->cut[1] ? gs - 1 : gs;
    if (p1 > p0) {
        cudaStream_t keep = c->stream;
        c->stream = c->aux;
        rc = exch ? launch_sweep<jac::OP_UPDATE>(c, u, un, p0 * per_plane, (p1 - p0) * per_plane)
                  : launch_sweep<jac::OP_UPDATE_PULL>(c, u, un, p0 * per_plane, (p1 - p0) * per_plane);
        c->stream = keep;
        if (rc) return rc;
    }
    JAC_CK(c, cudaEventRecord(c->ev_join, c->aux));
    c->in_sweep = true;
    return JAC_OK;
}

// Second half: the neighbours' new cut faces go into the ghost layers of the new state, the
// second stream joins, and the new state becomes the current one.
int slab_sweep_end(jac_ctx* c, const double* const src[2], void* const ready[2])
{
    int rc;
    if ((rc = unpack_cuts(c, c->u[c->cur ^ 1], src, ready))) return rc;
    JAC_CK(c, cudaStreamWaitEvent(c->stream, c->ev_join, 0));
    c->cur ^= 1;
    c->in_sweep = false;
    c->cut_fresh = true;
    c->ghosts_fresh = false;
    c->packed_current = false;
    return JAC_OK;
}

}  // namespace

// =====================================================================================
// C ABI
// =====================================================================================
extern "C" {

int jac_workspace_bytes(const jac_desc* desc, size_t* bytes)
{
    if (!desc || !bytes) return JAC_EINVAL;
    JacGeom g;
    jac_layout L;
    const int rc = build_geometry(desc, &g, &L);
    if (rc) return rc;
    *bytes = (size_t)L.total_bytes;
    return JAC_OK;
}

int jac_get_layout(const jac_desc* desc, jac_layout* out)
{
    if (!desc || !out) return JAC_EINVAL;
    JacGeom g;
    jac_layout L;
    const int rc = build_geometry(desc, &g, &L);
    if (rc) return rc;
    *out = L;
    return JAC_OK;
}

int jac_create(const jac_desc* desc, void* dev_workspace, size_t bytes, jac_ctx** out)
{
    if (!desc || !out) return JAC_EINVAL;
    JacGeom g;
    jac_layout L;
    int rc = build_geometry(desc, &g, &L);
    if (rc) return rc;
    if (!dev_workspace || bytes < (size_t)L.total_bytes || ((uintptr_t)dev_workspace & 255u))
        return JAC_ENOMEM;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return JAC_ENODEV;
    }
    jac_ctx* c = new (std::nothrow) jac_ctx();
    if (!c) return JAC_ENOMEM;
    c->desc = *desc;
    c->g = g;
    c->L = L;
    // launch plans for the SM count of this device, if the scratch (sized for the nominal count) holds them
    c->sms = kNominalSMs;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0) {
        const Tiling t = make_tiling(g, sms);
        if (max_partials(g, g.nblocks * t.ctas_per_block, desc->has_f != 0, sms) <= L.partials &&
            g.nblocks * t.ctas_per_block <= kMaxGrid)
            c->sms = sms;
    } else {
        cudaGetLastError();
    }
    c->tile = make_tiling(g, c->sms);
    c->ws = static_cast<char*>(dev_workspace);
    c->u[0] = reinterpret_cast<double*>(c->ws + L.off_u[0]);
    c->u[1] = reinterpret_cast<double*>(c->ws + L.off_u[1]);
    c->f = desc->has_f ? reinterpret_cast<double*>(c->ws + L.off_f) : nullptr;
    c->send = reinterpret_cast<double*>(c->ws + L.off_send);
    c->partials = reinterpret_cast<double*>(c->ws + L.off_scratch);
    c->result = c->partials + L.partials;
    c->cur = 0;
    c->ghosts_fresh = false;
    c->packed_current = false;
    c->f_ghosts_fresh = false;
    c->res_cluster = 0;
    c->stage_in = c->stage_out = nullptr;
    c->h2d = nullptr;
    c->ev_in_ready = c->ev_in_free = c->ev_out_done = nullptr;
    c->d2h_lo = c->d2h_hi = nullptr;
    c->cut[0] = (desc->flags & JAC_FLAG_CUT_LO) != 0;
    c->cut[1] = (desc->flags & JAC_FLAG_CUT_HI) != 0;
    for (int side = 0; side < 2; ++side) {
        c->cut_send[side][0] = c->cut_send[side][1] = c->cut_recv[side] = nullptr;
        c->ev_cut_ready[side] = nullptr;
    }
    c->cut_parity = 0;
    c->cut_fresh = false;
    c->in_sweep = false;
    c->aux = nullptr;
    c->ev_fork = c->ev_join = nullptr;
    c->stream = static_cast<cudaStream_t>(desc->stream);
    c->device = dev;
    c->cuda_err = 0;
    c->timed_out = false;
    c->launches = 0;
    // the ranges a checked build holds every global access against, and its record word
    c->g.chk_lo[0] = c->ws + L.off_u[0];
    c->g.chk_hi[0] = c->ws + L.off_send;
    c->g.chk_lo[1] = c->ws + L.off_send;
    c->g.chk_hi[1] = c->ws + L.off_scratch;
    c->g.chk_lo[2] = c->ws + L.off_scratch;
    c->g.chk_hi[2] = c->ws + L.off_scratch + (L.partials + 32) * (long long)sizeof(double);
    c->g.chk_rec = reinterpret_cast<unsigned long long*>(c->result + 5);
    c->g.quarter = 0.25;
    c->g.sixth = 1.0 / 6.0;
    const cudaError_t e = cudaMemsetAsync(c->ws, 0, (size_t)L.total_bytes, c->stream);
    if (e != cudaSuccess) {
        delete c;
        return JAC_ECUDA;
    }
    if (desc->mode == JAC_MODE_RESIDENT && (rc = choose_resident_cluster(c))) {
        delete c;
        return rc;
    }
    if (desc->flags & JAC_FLAG_HOST_STAGING) {
        c->stage_in = reinterpret_cast<double*>(c->ws + L.off_stage_in);
        c->stage_out = reinterpret_cast<double*>(c->ws + L.off_stage_out);
        if (cudaStreamCreateWithFlags(&c->h2d, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_in_ready, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_in_free, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_out_done, cudaEventDisableTiming) != cudaSuccess) {
            cudaGetLastError();
            release_copy_objects(c);
            delete c;
            return JAC_ECUDA;
        }
        // the copy stream must not run ahead of the clearing of the workspace queued above on the
        // caller's stream: the staging array counts as free only once that has been done
        if (cudaEventRecord(c->ev_in_free, c->stream) != cudaSuccess) {
            cudaGetLastError();
            release_copy_objects(c);
            delete c;
            return JAC_ECUDA;
        }
    }
    if (has_cuts(c)) {
        bool ok = cudaStreamCreateWithFlags(&c->aux, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) == cudaSuccess;
        for (int side = 0; side < 2 && ok; ++side) {
            if (!c->cut[side]) continue;
            c->cut_send[side][0] = reinterpret_cast<double*>(c->ws + L.off_cut_send[side][0]);
            c->cut_send[side][1] = reinterpret_cast<double*>(c->ws + L.off_cut_send[side][1]);
            c->cut_recv[side] = reinterpret_cast<double*>(c->ws + L.off_cut_recv[side]);
            ok = cudaEventCreateWithFlags(&c->ev_cut_ready[side], cudaEventDisableTiming) == cudaSuccess;
        }
        if (!ok) {
            cudaGetLastError();
            release_copy_objects(c);
            delete c;
            return JAC_ECUDA;
        }
    }
    *out = c;
    return JAC_OK;
}

int jac_destroy(jac_ctx* ctx)
{
    if (!ctx) return JAC_EINVAL;
    if (ctx->h2d) cudaStreamSynchronize(ctx->h2d);
    if (ctx->aux) cudaStreamSynchronize(ctx->aux);
    cudaStreamSynchronize(ctx->stream);
    release_copy_objects(ctx);
    delete ctx;
    return JAC_OK;
}

int jac_set_u(jac_ctx* c, const double* host_dense)
{
    int rc = usable(c);
    if (rc) return rc;
    if (!host_dense) return JAC_EINVAL;
    c->ghosts_fresh = false;
    c->packed_current = false;
    c->cut_fresh = false;
    return host_to_blocks(c, c->u[c->cur], host_dense, true);
}

int jac_set_f(jac_ctx* c, const double* host_dense)
{
    int rc = usable(c);
    if (rc) return rc;
    if (!host_dense || !c->f) return JAC_EINVAL;
    c->f_ghosts_fresh = false;
    return host_to_blocks(c, c->f, host_dense, true);
}

int jac_get_u(jac_ctx* c, double* host_dense)
{
    int rc = usable(c);
    if (rc) return rc;
    if (!host_dense) return JAC_EINVAL;
    if ((rc = blocks_to_host(c, c->u[c->cur], host_dense, true))) return rc;
    return check_timeout(c);
}

int jac_set_u_device(jac_ctx* c, const double* dev_dense)
{
    int rc = usable(c);
    if (rc) return rc;
    if (!dev_dense) return JAC_EINVAL;
    c->ghosts_fresh = false;
    c->packed_current = false;
    c->cut_fresh = false;
    return copy_dense_device<true>(c, c->u[c->cur], const_cast<double*>(dev_dense));
}

int jac_set_f_device(jac_ctx* c, const double* dev_dense)
{
    int rc = usable(c);
    if (rc) return rc;
    if (!dev_dense || !c->f) return JAC_EINVAL;
    c->f_ghosts_fresh = false;
    return copy_dense_device<true>(c, c->f, const_cast<double*>(dev_dense));
}

int jac_get_u_device(jac_ctx* c, double* dev_dense)
{
    int rc = usable(c);
    if (rc) return rc;
    if (!dev_dense) return JAC_EINVAL;
    return copy_dense_device<false>(c, c->u[c->cur], dev_dense);
}

int jac_set_boundary(jac_ctx* c, int face, double value)
{
    int rc = usable(c);
    if (rc) return rc;
    if (face < 0 || face >= c->g.nfaces) return JAC_EINVAL;
    if ((face >> 1) == c->g.ndim - 1 && c->cut[face & 1]) return JAC_EINVAL;   // a cut is not a domain face
    c->g.bval[face] = value;
    const int axis = face >> 1;
    const long long on_face = c->g.nblocks / (axis == 0 ? c->g.gx : axis == 1 ? c->g.gy : c->g.gz);
    const int chunks = (int)std::min<long long>(ceil_div(c->g.face_elems[face], 256), 64);
    jac::fill_boundary_kernel<<<(unsigned)(on_face * chunks), 256, 0, c->stream>>>(
        c->u[0], c->u[1], c->g, face, value, chunks);
    return check_launch(c);
}

int jac_get_block_padded(jac_ctx* c, int64_t block, double* host)
{
    int rc = usable(c);
    if (rc) return rc;
    if (!host || block < 0 || block >= c->g.nblocks) return JAC_EINVAL;
    const JacGeom& g = c->g;
    const long long h = g.h, hz = (g.ndim == 3) ? g.h : 0;
    const size_t PY = (size_t)(g.PXY / g.PX);
    const double* src = c->u[c->cur] + block * g.block_stride + g.origin - (hz * g.PXY + h * g.PX + h);
    const size_t w = (size_t)(g.bx + 2 * h), ht = (size_t)(g.by + 2 * h), dp = (size_t)(g.bz + 2 * hz);
    JAC_CK(c, copy_box(host, w * 8, ht, src, g.PX * 8, PY, w * 8, ht, dp, cudaMemcpyDeviceToHost, c->stream));
    JAC_CK(c, cudaStreamSynchronize(c->stream));
    return JAC_OK;
}

int jac_get_halo_buffer(jac_ctx* c, int64_t block, int face, double* host)
{
    int rc = usable(c);
    if (rc) return rc;
    if (!host || block < 0 || block >= c->g.nblocks || face < 0 || face >= c->g.nfaces) return JAC_EINVAL;
    const double* src = c->send + block * c->g.send_stride + c->g.face_off[face];
    JAC_CK(c, cudaMemcpyAsync(host, src, (size_t)c->g.face_elems[face] * 8, cudaMemcpyDeviceToHost, c->stream));
    JAC_CK(c, cudaStreamSynchronize(c->stream));
    return JAC_OK;
}

int jac_pack_halos(jac_ctx* c)
{
    int rc = usable(c);
    if (rc) return rc;
    rc = do_pack(c);
    if (rc) return rc;
    c->packed_current = true;
    return JAC_OK;
}

int jac_unpack_halos(jac_ctx* c)
{
    int rc = usable(c);
    if (rc) return rc;
    rc = do_unpack(c);
    if (rc) return rc;
    // ghosts are current only if the buffers were packed from the current state
    c->ghosts_fresh = c->packed_current;
    return JAC_OK;
}

int jac_exchange_halos(jac_ctx* c)
{
    int rc = usable(c);
    if (rc) return rc;
    return do_exchange_fused(c);
}

int jac_pack_faces(jac_ctx* c, unsigned face_mask)
{
    int rc = usable(c);
    if (rc) return rc;
    const unsigned all = (1u << c->g.nfaces) - 1u;
    if (face_mask & ~all) return JAC_EINVAL;
    if (face_mask == all) return jac_pack_halos(c);
    if (!face_mask) return JAC_OK;
    return launch_halo_all<jac::HALO_PACK>(c, face_mask);
}

int jac_unpack_faces(jac_ctx* c, unsigned face_mask)
{
    int rc = usable(c);
    if (rc) return rc;
    const unsigned all = (1u << c->g.nfaces) - 1u;
    if (face_mask & ~all) return JAC_EINVAL;
    if (face_mask == all) return jac_unpack_halos(c);
    if (!face_mask) return JAC_OK;
    return launch_halo_all<jac::HALO_UNPACK>(c, face_mask);
}

int jac_sweep(jac_ctx* c, int nsweeps)
{
    int rc = usable(c);
    if (rc) return rc;
    if (nsweeps < 0) return JAC_EINVAL;
    if (nsweeps == 0) return JAC_OK;
    return run_sweeps(c, nsweeps, jac::kResNone, nullptr);
}

int jac_sweep_residual(jac_ctx* c, int nsweeps, double* host_out_l2)
{
    int rc = usable(c);
    if (rc) return rc;
    if (nsweeps < 1 || !host_out_l2) return JAC_EINVAL;
    long long nparts = 0;
    if ((rc = run_sweeps(c, nsweeps, jac::kResBeforeLast, &nparts))) return rc;
    return finish_norm(c, nparts, host_out_l2);
}

int jac_solve(jac_ctx* c, int max_sweeps, int check_every, double tol, int* host_sweeps_done,
              double* host_residual)
{
    int rc = usable(c);
    if (rc) return rc;
    if (max_sweeps < 1 || check_every < 1 || !(tol >= 0.0) || !host_sweeps_done || !host_residual)
        return JAC_EINVAL;
    if (c->desc.mode == JAC_MODE_WIDE) {
        // the wide exchange and the grown-box updates do not look at the flag: ask after every group
        int done = 0;
        double res = 0.0;
        while (done < max_sweeps) {
            const int n = std::min(check_every, max_sweeps - done);
            long long nparts = 0;
            if ((rc = run_sweeps(c, n, jac::kResBeforeLast, &nparts))) return rc;
            if ((rc = finish_norm(c, nparts, &res))) return rc;
            done += n;
            if (res <= tol) break;
        }
        *host_sweeps_done = done;
        *host_residual = res;
        return JAC_OK;
    }
    // The test against the tolerance runs on the device.  Groups are queued several at a time without
    // waiting; once a group's norm meets the tolerance the launches queued behind it return at once,
    // and the host only looks at the flag between batches.
    constexpr int kGroupsPerLook = 8;
    int* stop = reinterpret_cast<int*>(c->result + 2);
    int* done_dev = reinterpret_cast<int*>(c->result + 3);
    JAC_CK(c, cudaMemsetAsync(c->result, 0, 4 * sizeof(double), c->stream));
    const int cur0 = c->cur;
    std::vector<signed char> cur_after;      // which array is current after each queued group
    int queued = 0, done = 0;
    double norm = 0.0;
    bool stopped = false;
    c->g.stop = stop;
    while (queued < max_sweeps && !stopped && rc == JAC_OK) {
        for (int k = 0; k < kGroupsPerLook && queued < max_sweeps && rc == JAC_OK; ++k) {
            const int n = std::min(check_every, max_sweeps - queued);
            long long nparts = 0;
            if ((rc = run_sweeps(c, n, jac::kResBeforeLast, &nparts))) break;
            solve_check_kernel<<<1, 1024, 0, c->stream>>>(c->partials, nparts, tol, n, c->result, stop, done_dev);
            if ((rc = check_launch(c))) break;
            queued += n;
            cur_after.push_back((signed char)c->cur);
        }
        if (rc) break;
        double look[4];
        cudaError_t e = cudaMemcpyAsync(look, c->result, sizeof(look), cudaMemcpyDeviceToHost, c->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
        if (e != cudaSuccess) {
            c->cuda_err = (int)e;
            rc = JAC_ECUDA;
            break;
        }
        int flag = 0;
        std::memcpy(&flag, &look[2], sizeof(int));
        std::memcpy(&done, &look[3], sizeof(int));
        norm = look[1];
        stopped = flag != 0;
    }
    c->g.stop = nullptr;
    if (rc) return rc;
    // the launches queued behind the group that met the tolerance did nothing: the current array is
    // the one that was current after that group
    const int groups_done = (done + check_every - 1) / check_every;
    c->cur = groups_done > 0 ? cur_after[(size_t)groups_done - 1] : cur0;
    c->ghosts_fresh = false;
    c->packed_current = false;
    *host_sweeps_done = done;
    *host_residual = norm;
    return JAC_OK;
}

int jac_residual(jac_ctx* c, double* host_out_l2)
{
    int rc = usable(c);
    if (rc) return rc;
    if (!host_out_l2) return JAC_EINVAL;
    if (has_cuts(c) && (!c->cut_fresh || c->in_sweep)) return JAC_EINVAL;
    if (!c->ghosts_fresh && (rc = (c->desc.mode == JAC_MODE_PERTASK ? do_exchange(c) : do_exchange_fused(c)))) return rc;
    if ((rc = launch_sweep<jac::OP_RESIDUAL>(c, c->u[c->cur], nullptr, 0, c->g.nblocks))) return rc;
    return finish_norm(c, c->g.nblocks * c->tile.ctas_per_block, host_out_l2);
}

int jac_exchange_wide(jac_ctx* c)
{
    int rc = usable(c);
    if (rc) return rc;
    if (c->desc.mode != JAC_MODE_WIDE) return JAC_EINVAL;
    if ((rc = do_exchange_wide(c, c->u[c->cur]))) return rc;
    c->packed_current = false;   // the send slots now hold wide faces
    c->ghosts_fresh = true;      // the face ghosts are among the cells just filled
    return JAC_OK;
}

int jac_get_wide_buffer(jac_ctx* c, int64_t block, int face, double* host)
{
    int rc = usable(c);
    if (rc) return rc;
    if (c->desc.mode != JAC_MODE_WIDE) return JAC_EINVAL;
    if (!host || block < 0 || block >= c->g.nblocks || face < 0 || face >= c->g.nfaces) return JAC_EINVAL;
    const double* src = c->send + block * c->g.send_stride + c->g.face_off[face];
    JAC_CK(c, cudaMemcpyAsync(host, src, (size_t)c->g.wface_elems[face] * 8, cudaMemcpyDeviceToHost, c->stream));
    JAC_CK(c, cudaStreamSynchronize(c->stream));
    return JAC_OK;
}

int jac_set_u_async(jac_ctx* c, const double* host_dense)
{
    int rc = usable(c);
    if (rc) return rc;
    if (!host_dense) return JAC_EINVAL;
    c->ghosts_fresh = false;
    c->packed_current = false;
    c->cut_fresh = false;
    return host_to_blocks(c, c->u[c->cur], host_dense, false);
}

int jac_get_u_async(jac_ctx* c, double* host_dense)
{
    int rc = usable(c);
    if (rc) return rc;
    if (!host_dense) return JAC_EINVAL;
    return blocks_to_host(c, c->u[c->cur], host_dense, false);
}

namespace {
// the residual of the current state queued on the stream: its sum of squares, or the norm
int residual_queued(jac_ctx* c, double* host_out, bool norm)
{
    int rc = usable(c);
    if (rc) return rc;
    if (!host_out) return JAC_EINVAL;
    if (has_cuts(c) && (!c->cut_fresh || c->in_sweep)) return JAC_EINVAL;
    if (!c->ghosts_fresh && (rc = (c->desc.mode == JAC_MODE_PERTASK ? do_exchange(c) : do_exchange_fused(c)))) return rc;
    if ((rc = launch_sweep<jac::OP_RESIDUAL>(c, c->u[c->cur], nullptr, 0, c->g.nblocks))) return rc;
    jac::reduce_partials_kernel<<<1, 1024, 0, c->stream>>>(c->partials, c->g.nblocks * c->tile.ctas_per_block, c->result, norm);
    if ((rc = check_launch(c))) return rc;
    JAC_CK(c, cudaMemcpyAsync(host_out, c->result, sizeof(double), cudaMemcpyDeviceToHost, c->stream));
    return JAC_OK;
}
}  // namespace

int jac_residual_async(jac_ctx* c, double* host_out_l2) { return residual_queued(c, host_out_l2, true); }

int jac_residual_sumsq_async(jac_ctx* c, double* host_out_sumsq) { return residual_queued(c, host_out_sumsq, false); }

int jac_residual_sweep_async(jac_ctx* c, int nsweeps, double* host_out_l2)
{
    int rc = usable(c);
    if (rc) return rc;
    if (nsweeps < 1 || !host_out_l2 || has_cuts(c)) return JAC_EINVAL;
    // schedules whose first launch cannot carry the sum: the ordinary residual pass, then the sweeps
    if (c->desc.mode == JAC_MODE_WIDE) {
        if ((rc = residual_queued(c, host_out_l2, true))) return rc;
        return run_sweeps(c, nsweeps, jac::kResNone, nullptr);
    }
    long long nparts = 0;
    if ((rc = run_sweeps(c, nsweeps, jac::kResOfInput, &nparts))) return rc;
    jac::reduce_partials_kernel<<<1, 1024, 0, c->stream>>>(c->partials, nparts, c->result, true);
    if ((rc = check_launch(c))) return rc;
    JAC_CK(c, cudaMemcpyAsync(host_out_l2, c->result, sizeof(double), cudaMemcpyDeviceToHost, c->stream));
    return JAC_OK;
}

int jac_sweep_norms_async(jac_ctx* c, int nsweeps, int every, double* host_out_l2)
{
    int rc = usable(c);
    if (rc) return rc;
    if (nsweeps < 1 || every < 1 || has_cuts(c)) return JAC_EINVAL;
    const int nnorms = (nsweeps - 1) / every;
    if (nnorms > 0 && !host_out_l2) return JAC_EINVAL;
    const int T = default_tsteps(c->desc);
    if (c->desc.mode == JAC_MODE_TEMPORAL && nnorms > 0 && every >= T) {
        // The state after j sweeps is what sweep j + 1 reads: level j - a + 1 of the launch that starts
        // after a sweeps.  So the launches need not end where a norm is due; they keep the depths the
        // whole run would have, and at most one level of a launch measures (every >= T).
        std::vector<int> depths;
        temporal_depths(nsweeps, T, c->g.ndim, c->desc.has_f != 0, &depths);
        // The norms collect in the status words 8 .. 31 of the scratch and travel to the host 24 at a
        // time: a copy of 8 bytes after every measuring launch would put a gap into the stream each
        // time (a hundred of them in a job of 1000 sweeps with a norm every 10).
        constexpr int kNormRing = 24;
        double* const ring = c->result + 8;
        int pending = 0, copied = 0;
        int a = 0;
        for (const int t : depths) {
            int j = (a + every - 1) / every * every;     // the first multiple of `every` not below a
            if (j == 0) j = every;
            const int level = j < a + t ? j - a + 1 : 0;
            long long nparts = 0;
            if ((rc = launch_temporal_n(c, t, c->u[c->cur], c->u[c->cur ^ 1], level, &nparts))) return rc;
            c->cur ^= 1;
            c->ghosts_fresh = false;
            c->packed_current = false;
            if (level) {
                // norm number j / every - 1 = copied + pending: they are due in order
                jac::reduce_partials_kernel<<<1, 1024, 0, c->stream>>>(c->partials, nparts, ring + pending, true);
                if ((rc = check_launch(c))) return rc;
                if (++pending == kNormRing) {
                    JAC_CK(c, cudaMemcpyAsync(host_out_l2 + copied, ring, pending * sizeof(double),
                                              cudaMemcpyDeviceToHost, c->stream));
                    copied += pending;
                    pending = 0;
                }
            }
            a += t;
        }
        if (pending)
            JAC_CK(c, cudaMemcpyAsync(host_out_l2 + copied, ring, pending * sizeof(double), cudaMemcpyDeviceToHost,
                                      c->stream));
        return JAC_OK;
    }
    // every other case group by group: the norm of the state a group starts from comes out of the
    // group's first sweep
    int done = std::min(every, nsweeps);
    if ((rc = run_sweeps(c, done, jac::kResNone, nullptr))) return rc;
    for (int k = 0; done < nsweeps; ++k) {
        const int n = std::min(every, nsweeps - done);
        if ((rc = jac_residual_sweep_async(c, n, host_out_l2 + k))) return rc;
        done += n;
    }
    return JAC_OK;
}

int jac_pack_cut(jac_ctx* c)
{
    int rc = usable(c);
    if (rc) return rc;
    if (!has_cuts(c) || c->in_sweep) return JAC_EINVAL;
    return pack_cuts(c, c->u[c->cur]);
}

int jac_unpack_cut(jac_ctx* c, const double* dev_src_lo, void* ready_lo, const double* dev_src_hi, void* ready_hi)
{
    int rc = usable(c);
    if (rc) return rc;
    if (!has_cuts(c) || c->in_sweep) return JAC_EINVAL;
    const double* const src[2] = {dev_src_lo, dev_src_hi};
    void* const ready[2] = {ready_lo, ready_hi};
    if ((rc = unpack_cuts(c, c->u[c->cur], src, ready))) return rc;
    c->cut_fresh = true;
    return JAC_OK;
}

int jac_sweep_begin(jac_ctx* c)
{
    int rc = usable(c);
    if (rc) return rc;
    if (!has_cuts(c) || c->in_sweep || !c->cut_fresh) return JAC_EINVAL;
    return slab_sweep_begin(c);
}

int jac_sweep_end(jac_ctx* c, const double* dev_src_lo, void* ready_lo, const double* dev_src_hi, void* ready_hi)
{
    int rc = usable(c);
    if (rc) return rc;
    if (!has_cuts(c) || !c->in_sweep) return JAC_EINVAL;
    const double* const src[2] = {dev_src_lo, dev_src_hi};
    void* const ready[2] = {ready_lo, ready_hi};
    return slab_sweep_end(c, src, ready);
}

int jac_cut_info(const jac_ctx* c, int side, void** dev_send, void** dev_recv, size_t* bytes, void** ready_event)
{
    if (!c || side < 0 || side > 1 || !c->cut[side]) return JAC_EINVAL;
    if (dev_send) *dev_send = c->cut_send[side][c->cut_parity];
    if (dev_recv) *dev_recv = c->cut_recv[side];
    if (bytes) *bytes = (size_t)c->L.cut_elems * sizeof(double);
    if (ready_event) *ready_event = c->ev_cut_ready[side];
    return JAC_OK;
}

int jac_sweeps_per_launch(const jac_ctx* c, int* host_out)
{
    if (!c || !host_out) return JAC_EINVAL;
    *host_out = (c->desc.mode == JAC_MODE_TEMPORAL) ? default_tsteps(c->desc) : 1;
    return JAC_OK;
}

int jac_launch_count(const jac_ctx* c, int64_t* host_out)
{
    if (!c || !host_out) return JAC_EINVAL;
    *host_out = c->launches;
    return JAC_OK;
}

int jac_last_cuda_error(const jac_ctx* c) { return c ? c->cuda_err : 0; }

int jac_debug_shrink_bounds(jac_ctx* c, int array, int64_t bytes)
{
    if (!c || array < 0 || array > 2 || bytes < 0 || bytes > c->g.chk_hi[array] - c->g.chk_lo[array]) return JAC_EINVAL;
    c->g.chk_hi[array] -= bytes;
    return JAC_OK;
}

int jac_debug_bounds(jac_ctx* c, int* host_checked, uint64_t* host_record)
{
    if (!c || !host_checked || !host_record) return JAC_EINVAL;
    if (!jac::kChecksBounds) {
        *host_checked = 0;
        *host_record = 0;
        return JAC_OK;
    }
    unsigned long long rec = 0;
    JAC_CK(c, cudaMemcpyAsync(&rec, c->g.chk_rec, sizeof(rec), cudaMemcpyDeviceToHost, c->stream));
    JAC_CK(c, cudaStreamSynchronize(c->stream));
    *host_checked = jac::kChecksBounds ? 1 : 0;
    *host_record = rec;
    return JAC_OK;
}

const char* jac_strerror(int code)
{
    switch (code) {
        case JAC_OK: return "ok";
        case JAC_EINVAL: return "invalid argument";
        case JAC_ENOMEM: return "workspace missing, too small or misaligned";
        case JAC_ECUDA: return "CUDA runtime error";
        case JAC_ENODEV: return "no usable CUDA device";
        case JAC_ELIMIT: return "problem exceeds the fixed scratch of the no-allocation entry point";
        case JAC_ETIMEOUT: return "a bounded device-side wait ran out";
        default: return "unknown error code";
    }
}

}  // extern "C"
