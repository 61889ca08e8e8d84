/*
 * CPU oracle for block-decomposed Jacobi relaxation (2D 5-point / 3D 7-point, fp64).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * method computes; the GPU library is compared against it.  It shares no code
 * with the GPU library and must never be called from the product path.
 *
 * What the method is (paper, Section V-C "Proxy Application: Jacobi3d"): a fixed
 * number of Jacobi iterations on a domain decomposed into cuboid blocks; in each
 * iteration every block packs its faces, the faces travel to the neighbouring
 * blocks, are unpacked into their ghost cells, and then the Jacobi update runs.
 * The paper gives no coefficients, boundary rule, precision or residual; those
 * are fixed here as follows (the same readings the GPU library documents):
 *
 *   update   u'(p) = ( sum of the 2d face neighbours of u at p  [+ f(p)] ) * (1/c),
 *            c = 4 (2D) or 6 (3D); i.e. Jacobi for  -Laplace_h u = f  with h = 1.
 *   order    s = (W + E) + (S + N);  3D: s = s + (D + U);  with f: s = s + f;
 *            u' = s * 0.25  (2D)   or   u' = s * (1.0/6.0)  (3D).
 *            Every operation is one IEEE-754 round-to-nearest add or multiply
 *            (compile with -ffp-contract=off), so results are bit-reproducible.
 *   boundary Dirichlet values live in the ghost layer around the domain, one
 *            constant per domain face, default 0, never overwritten.
 *   residual r(p) = s(p) - c*u(p) with s as above; result sqrt(sum r^2) over all
 *            interior points, not normalised.  Accumulated in long double.
 *   faces    ids 0:-x 1:+x 2:-y 3:+y 4:-z 5:+z.  A face is the h interior layers
 *            next to that side, over the interior extent of the other axes only
 *            (no edges, no corners).  Packed order = source memory order
 *            restricted to the strip (x fastest, then y, then z).
 *            Faces on the domain boundary are neither packed nor unpacked.
 *   blocks   g = ceil(n / b) per axis.  When n is not a multiple of b the last block along that
 *            axis is a remainder block of n - (g-1)*b >= h points; it keeps a full-size padded
 *            array, its interior in the low corner, its +ghost layers right after its interior.
 *            (The paper's decomposition is into equal cuboids; remainder blocks are an extension.)
 *   exchange comes before the update in every sweep.
 *   wide     (last part of this file; not in the paper) one exchange of all h ghost layers with
 *            edges and corners, then up to h sweeps on shrinking extents: same bits.
 *
 * Index conventions: x is the fastest-varying axis, then y, then z.  In 2D, nz = bz = 1
 * and there is no padding along z.
 *
 * Pins (see tests/test_oracle_*.py): discrete sine eigenmodes decay by the known
 * factor per sweep; tiny grids against exact rational arithmetic on the textbook
 * matrix form; random-walk path enumeration for the heated-edge problem; blocked
 * run is bit-identical to the monolithic run; packed buffers equal numpy slices of
 * the dense array; residual identities (r = 4(u_{k+1}-u_k) in 2D, ||r|| = ||f|| at u = 0);
 * wide exchange: every ghost equals the padded global field, k sweeps per exchange are
 * bit-identical to the monolithic run for every k <= h.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK 0
#define ORC_EINVAL (-1)
#define ORC_ENOMEM (-2)

/* ------------------------------------------------------------------------- */
/* Monolithic form: one padded array (nx+2) x (ny+2) [x (nz+2)].             */
/* ------------------------------------------------------------------------- */

/* One Jacobi sweep over the whole domain.
 *   u    padded input,  dims (n[0]+2) x (n[1]+2) x (ndim==3 ? n[2]+2 : 1), x fastest
 *   f    dense right-hand side n[0] x n[1] x n[2], or NULL for f == 0
 *   out  padded output; only interior points are written
 */
int orc_sweep_mono(int ndim, const int64_t *n, const double *u, const double *f, double *out)
{
    if ((ndim != 2 && ndim != 3) || !n || !u || !out) return ORC_EINVAL;
    const int64_t nx = n[0], ny = n[1], nz = (ndim == 3) ? n[2] : 1;
    if (nx < 1 || ny < 1 || nz < 1) return ORC_EINVAL;
    const int64_t px = nx + 2, py = ny + 2;
    if (ndim == 2) {
#pragma omp parallel for schedule(static)
        for (int64_t j = 1; j <= ny; ++j) {
            for (int64_t i = 1; i <= nx; ++i) {
                const int64_t p = j * px + i;
                double s = (u[p - 1] + u[p + 1]) + (u[p - px] + u[p + px]);
                if (f) s = s + f[(j - 1) * nx + (i - 1)];
                out[p] = s * 0.25;
            }
        }
    } else {
        const double c6 = 1.0 / 6.0;
        const int64_t pxy = px * py;
#pragma omp parallel for schedule(static)
        for (int64_t k = 1; k <= nz; ++k) {
            for (int64_t j = 1; j <= ny; ++j) {
                for (int64_t i = 1; i <= nx; ++i) {
                    const int64_t p = (k * py + j) * px + i;
                    double s = (u[p - 1] + u[p + 1]) + (u[p - px] + u[p + px]);
                    s = s + (u[p - pxy] + u[p + pxy]);
                    if (f) s = s + f[((k - 1) * ny + (j - 1)) * nx + (i - 1)];
                    out[p] = s * c6;
                }
            }
        }
    }
    return ORC_OK;
}

/* L2 norm of the residual of the monolithic padded array. */
int orc_residual_mono(int ndim, const int64_t *n, const double *u, const double *f, double *out_l2)
{
    if ((ndim != 2 && ndim != 3) || !n || !u || !out_l2) return ORC_EINVAL;
    const int64_t nx = n[0], ny = n[1], nz = (ndim == 3) ? n[2] : 1;
    if (nx < 1 || ny < 1 || nz < 1) return ORC_EINVAL;
    const int64_t px = nx + 2, py = ny + 2, pxy = px * py;
    long double acc = 0.0L;
    for (int64_t k = 0; k < nz; ++k) {
        for (int64_t j = 1; j <= ny; ++j) {
            for (int64_t i = 1; i <= nx; ++i) {
                double s, t;
                if (ndim == 2) {
                    const int64_t p = j * px + i;
                    s = (u[p - 1] + u[p + 1]) + (u[p - px] + u[p + px]);
                    if (f) s = s + f[(j - 1) * nx + (i - 1)];
                    t = 4.0 * u[p];
                } else {
                    const int64_t p = ((k + 1) * py + j) * px + i;
                    s = (u[p - 1] + u[p + 1]) + (u[p - px] + u[p + px]);
                    s = s + (u[p - pxy] + u[p + pxy]);
                    if (f) s = s + f[(k * ny + (j - 1)) * nx + (i - 1)];
                    t = 6.0 * u[p];
                }
                const double r = s - t;
                acc += (long double)r * (long double)r;
            }
        }
    }
    *out_l2 = (double)sqrtl(acc);
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Blocked form: every block owns a padded array (b+2h)^d and send buffers.  */
/* ------------------------------------------------------------------------- */

typedef struct orc_blocked {
    int ndim;
    int64_t n[3], b[3], g[3]; /* global interior, block interior, block grid */
    int64_t h;                /* ghost width */
    int64_t p[3];             /* padded block dims: b + 2h (1 along z in 2D) */
    int64_t hz;               /* ghost width along z: h in 3D, 0 in 2D */
    int64_t nblocks;
    int64_t pad_elems;        /* elements of one padded block */
    int64_t blk_elems;        /* interior elements of one block */
    int64_t face_elems[6];    /* elements of one packed face */
    double *u[2];             /* two solution arrays, nblocks * pad_elems each */
    int cur;                  /* which of u[] holds the current state */
    double *f;                /* nblocks * blk_elems, or NULL */
    double *send;             /* nblocks * 6 * max_face */
    int64_t max_face;
    double bval[6];           /* Dirichlet value per domain face */
} orc_blocked;

static int64_t pad_index(const orc_blocked *s, int64_t i, int64_t j, int64_t k)
{
    /* i, j, k are interior-relative (0 .. b-1 interior, negative / >= b ghosts) */
    return ((k + s->hz) * s->p[1] + (j + s->h)) * s->p[0] + (i + s->h);
}

static double *blk_u(const orc_blocked *s, int which, int64_t blk)
{
    return s->u[which] + blk * s->pad_elems;
}

static double *blk_send(const orc_blocked *s, int64_t blk, int face)
{
    return s->send + (blk * 6 + face) * s->max_face;
}

static void blk_coords(const orc_blocked *s, int64_t blk, int64_t c[3])
{
    c[0] = blk % s->g[0];
    c[1] = (blk / s->g[0]) % s->g[1];
    c[2] = blk / (s->g[0] * s->g[1]);
}

/* interior extent of block `blk`: b, except for the last block along an axis when the grid is
 * not a multiple of the block size (then the remainder n - (g-1)*b; it still owns a full-size
 * padded array, its interior is the low corner and its +ghost layers follow the interior) */
static void blk_extent(const orc_blocked *s, int64_t blk, int64_t e[3])
{
    int64_t c[3];
    blk_coords(s, blk, c);
    for (int a = 0; a < 3; ++a) {
        const int64_t left = s->n[a] - c[a] * s->b[a];
        e[a] = left < s->b[a] ? left : s->b[a];
    }
}

/* neighbour block across `face`, or -1 if that side is the domain boundary */
static int64_t blk_neighbour(const orc_blocked *s, int64_t blk, int face)
{
    int64_t c[3];
    blk_coords(s, blk, c);
    const int axis = face / 2;
    if (axis >= s->ndim) return -1;
    c[axis] += (face & 1) ? 1 : -1;
    if (c[axis] < 0 || c[axis] >= s->g[axis]) return -1;
    return (c[2] * s->g[1] + c[1]) * s->g[0] + c[0];
}

/* Writes the Dirichlet value of every domain face into the ghost layers of the
 * blocks that touch it, in both solution arrays.  Ghost cells on edges/corners
 * are never read by the stencil; they are left as they are. */
static void fill_boundary_ghosts(orc_blocked *s)
{
    for (int64_t blk = 0; blk < s->nblocks; ++blk) {
        for (int face = 0; face < 2 * s->ndim; ++face) {
            if (blk_neighbour(s, blk, face) >= 0) continue;
            const int axis = face / 2;
            int64_t ext[3];
            blk_extent(s, blk, ext);
            int64_t lo[3] = {0, 0, 0}, hi[3] = {ext[0], ext[1], ext[2]};
            if (face & 1) { lo[axis] = ext[axis]; hi[axis] = ext[axis] + s->h; }
            else          { lo[axis] = -s->h;      hi[axis] = 0; }
            for (int w = 0; w < 2; ++w) {
                double *u = blk_u(s, w, blk);
                for (int64_t k = lo[2]; k < hi[2]; ++k)
                    for (int64_t j = lo[1]; j < hi[1]; ++j)
                        for (int64_t i = lo[0]; i < hi[0]; ++i)
                            u[pad_index(s, i, j, k)] = s->bval[face];
            }
        }
    }
}

int orc_blocked_destroy(orc_blocked *s)
{
    if (!s) return ORC_EINVAL;
    free(s->u[0]); free(s->u[1]); free(s->f); free(s->send); free(s);
    return ORC_OK;
}

int orc_blocked_create(int ndim, const int64_t *n, const int64_t *b, int64_t h, int has_f,
                       orc_blocked **out)
{
    if ((ndim != 2 && ndim != 3) || !n || !b || !out || h < 1) return ORC_EINVAL;
    orc_blocked *s = (orc_blocked *)calloc(1, sizeof(*s));
    if (!s) return ORC_ENOMEM;
    s->ndim = ndim;
    s->h = h;
    s->hz = (ndim == 3) ? h : 0;
    s->nblocks = 1;
    for (int a = 0; a < 3; ++a) {
        s->n[a] = (a < ndim) ? n[a] : 1;
        s->b[a] = (a < ndim) ? b[a] : 1;
        if (s->n[a] < 1 || s->b[a] < 1 || s->b[a] > s->n[a] || (a < ndim && h > s->b[a])) {
            free(s);
            return ORC_EINVAL;
        }
        s->g[a] = (s->n[a] + s->b[a] - 1) / s->b[a];
        /* a remainder block must still be at least h wide: its face strips are h layers */
        if (a < ndim && s->n[a] - (s->g[a] - 1) * s->b[a] < h) {
            free(s);
            return ORC_EINVAL;
        }
        s->p[a] = (a < ndim) ? s->b[a] + 2 * h : 1;
        s->nblocks *= s->g[a];
    }
    s->pad_elems = s->p[0] * s->p[1] * s->p[2];
    s->blk_elems = s->b[0] * s->b[1] * s->b[2];
    s->face_elems[0] = s->face_elems[1] = h * s->b[1] * s->b[2];
    s->face_elems[2] = s->face_elems[3] = h * s->b[0] * s->b[2];
    s->face_elems[4] = s->face_elems[5] = (ndim == 3) ? h * s->b[0] * s->b[1] : 0;
    s->max_face = 0;
    for (int fc = 0; fc < 6; ++fc)
        if (s->face_elems[fc] > s->max_face) s->max_face = s->face_elems[fc];
    s->u[0] = (double *)calloc((size_t)(s->nblocks * s->pad_elems), sizeof(double));
    s->u[1] = (double *)calloc((size_t)(s->nblocks * s->pad_elems), sizeof(double));
    s->send = (double *)calloc((size_t)(s->nblocks * 6 * s->max_face), sizeof(double));
    if (has_f) s->f = (double *)calloc((size_t)(s->nblocks * s->blk_elems), sizeof(double));
    if (!s->u[0] || !s->u[1] || !s->send || (has_f && !s->f)) {
        orc_blocked_destroy(s);
        return ORC_ENOMEM;
    }
    *out = s;
    return ORC_OK;
}

int orc_blocked_set_boundary(orc_blocked *s, int face, double value)
{
    if (!s || face < 0 || face >= 2 * s->ndim) return ORC_EINVAL;
    s->bval[face] = value;
    fill_boundary_ghosts(s);
    return ORC_OK;
}

/* dense <-> blocks; dense is n[0] x n[1] x n[2], x fastest */
static void scatter_dense(const orc_blocked *s, const double *dense, double *dst, int padded)
{
#pragma omp parallel for schedule(static)
    for (int64_t blk = 0; blk < s->nblocks; ++blk) {
        int64_t c[3], ext[3];
        blk_coords(s, blk, c);
        blk_extent(s, blk, ext);
        for (int64_t k = 0; k < ext[2]; ++k)
            for (int64_t j = 0; j < ext[1]; ++j)
                for (int64_t i = 0; i < ext[0]; ++i) {
                    const int64_t gi = c[0] * s->b[0] + i, gj = c[1] * s->b[1] + j,
                                  gk = c[2] * s->b[2] + k;
                    const double v = dense[(gk * s->n[1] + gj) * s->n[0] + gi];
                    if (padded) dst[blk * s->pad_elems + pad_index(s, i, j, k)] = v;
                    else dst[blk * s->blk_elems + (k * s->b[1] + j) * s->b[0] + i] = v;
                }
    }
}

int orc_blocked_set_u(orc_blocked *s, const double *dense)
{
    if (!s || !dense) return ORC_EINVAL;
    scatter_dense(s, dense, s->u[s->cur], 1);
    return ORC_OK;
}

int orc_blocked_set_f(orc_blocked *s, const double *dense)
{
    if (!s || !dense || !s->f) return ORC_EINVAL;
    scatter_dense(s, dense, s->f, 0);
    return ORC_OK;
}

int orc_blocked_get_u(const orc_blocked *s, double *dense)
{
    if (!s || !dense) return ORC_EINVAL;
#pragma omp parallel for schedule(static)
    for (int64_t blk = 0; blk < s->nblocks; ++blk) {
        int64_t c[3], ext[3];
        blk_coords(s, blk, c);
        blk_extent(s, blk, ext);
        const double *u = blk_u(s, s->cur, blk);
        for (int64_t k = 0; k < ext[2]; ++k)
            for (int64_t j = 0; j < ext[1]; ++j)
                for (int64_t i = 0; i < ext[0]; ++i) {
                    const int64_t gi = c[0] * s->b[0] + i, gj = c[1] * s->b[1] + j,
                                  gk = c[2] * s->b[2] + k;
                    dense[(gk * s->n[1] + gj) * s->n[0] + gi] = u[pad_index(s, i, j, k)];
                }
    }
    return ORC_OK;
}

/* the whole padded block (b+2h)^d of the current state, x fastest */
int orc_blocked_get_block_padded(const orc_blocked *s, int64_t blk, double *out)
{
    if (!s || !out || blk < 0 || blk >= s->nblocks) return ORC_EINVAL;
    memcpy(out, blk_u(s, s->cur, blk), (size_t)s->pad_elems * sizeof(double));
    return ORC_OK;
}

/* elements of the packed face of (block, face): h layers times the block's extent on the other axes */
int64_t orc_blocked_face_elems(const orc_blocked *s, int64_t blk, int face)
{
    if (!s || blk < 0 || blk >= s->nblocks || face < 0 || face >= 2 * s->ndim) return ORC_EINVAL;
    int64_t e[3];
    blk_extent(s, blk, e);
    e[face / 2] = s->h;
    return e[0] * e[1] * e[2];
}

/* the packed send buffer of (block, face) as left by the last pack */
int orc_blocked_get_halo_buffer(const orc_blocked *s, int64_t blk, int face, double *out)
{
    if (!s || !out || blk < 0 || blk >= s->nblocks || face < 0 || face >= 2 * s->ndim)
        return ORC_EINVAL;
    memcpy(out, blk_send(s, blk, face), (size_t)orc_blocked_face_elems(s, blk, face) * sizeof(double));
    return ORC_OK;
}

/* interior-relative index range of the h-wide strip on `face`:
 * ghost == 0: the interior layers next to the face; ghost == 1: the ghost layers */
static void strip_range(const orc_blocked *s, int64_t blk, int face, int ghost, int64_t lo[3], int64_t hi[3])
{
    const int axis = face / 2;
    int64_t ext[3];
    blk_extent(s, blk, ext);
    for (int a = 0; a < 3; ++a) { lo[a] = 0; hi[a] = ext[a]; }
    if (face & 1) {
        lo[axis] = ghost ? ext[axis] : ext[axis] - s->h;
        hi[axis] = lo[axis] + s->h;
    } else {
        lo[axis] = ghost ? -s->h : 0;
        hi[axis] = lo[axis] + s->h;
    }
}

/* Pack: every face that has a neighbour block -> its contiguous send buffer. */
int orc_blocked_pack(orc_blocked *s)
{
    if (!s) return ORC_EINVAL;
#pragma omp parallel for schedule(static)
    for (int64_t blk = 0; blk < s->nblocks; ++blk) {
        const double *u = blk_u(s, s->cur, blk);
        for (int face = 0; face < 2 * s->ndim; ++face) {
            if (blk_neighbour(s, blk, face) < 0) continue;
            int64_t lo[3], hi[3];
            strip_range(s, blk, face, 0, lo, hi);
            double *buf = blk_send(s, blk, face);
            int64_t q = 0;
            for (int64_t k = lo[2]; k < hi[2]; ++k)
                for (int64_t j = lo[1]; j < hi[1]; ++j)
                    for (int64_t i = lo[0]; i < hi[0]; ++i)
                        buf[q++] = u[pad_index(s, i, j, k)];
        }
    }
    return ORC_OK;
}

/* Unpack: ghost layers on face F of block B <- send buffer (neighbour(B,F), F^1),
 * same element order. */
int orc_blocked_unpack(orc_blocked *s)
{
    if (!s) return ORC_EINVAL;
#pragma omp parallel for schedule(static)
    for (int64_t blk = 0; blk < s->nblocks; ++blk) {
        double *u = blk_u(s, s->cur, blk);
        for (int face = 0; face < 2 * s->ndim; ++face) {
            const int64_t nb = blk_neighbour(s, blk, face);
            if (nb < 0) continue;
            int64_t lo[3], hi[3];
            strip_range(s, blk, face, 1, lo, hi);
            const double *buf = blk_send(s, nb, face ^ 1);
            int64_t q = 0;
            for (int64_t k = lo[2]; k < hi[2]; ++k)
                for (int64_t j = lo[1]; j < hi[1]; ++j)
                    for (int64_t i = lo[0]; i < hi[0]; ++i)
                        u[pad_index(s, i, j, k)] = buf[q++];
        }
    }
    return ORC_OK;
}

/* The Jacobi update inside every block, reading ghosts as they are. No exchange. */
int orc_blocked_update(orc_blocked *s)
{
    if (!s) return ORC_EINVAL;
    const int64_t px = s->p[0], pxy = s->p[0] * s->p[1];
    const double c6 = 1.0 / 6.0;
#pragma omp parallel for schedule(static)
    for (int64_t blk = 0; blk < s->nblocks; ++blk) {
        const double *u = blk_u(s, s->cur, blk);
        double *o = blk_u(s, s->cur ^ 1, blk);
        const double *f = s->f ? s->f + blk * s->blk_elems : NULL;
        int64_t ext[3];
        blk_extent(s, blk, ext);
        for (int64_t k = 0; k < ext[2]; ++k)
            for (int64_t j = 0; j < ext[1]; ++j)
                for (int64_t i = 0; i < ext[0]; ++i) {
                    const int64_t p = pad_index(s, i, j, k);
                    double sum = (u[p - 1] + u[p + 1]) + (u[p - px] + u[p + px]);
                    if (s->ndim == 3) sum = sum + (u[p - pxy] + u[p + pxy]);
                    if (f) sum = sum + f[(k * s->b[1] + j) * s->b[0] + i];
                    o[p] = (s->ndim == 3) ? sum * c6 : sum * 0.25;
                }
    }
    s->cur ^= 1;
    return ORC_OK;
}

/* nsweeps x ( pack ; unpack ; update ) */
int orc_blocked_sweep(orc_blocked *s, int64_t nsweeps)
{
    if (!s || nsweeps < 0) return ORC_EINVAL;
    for (int64_t it = 0; it < nsweeps; ++it) {
        orc_blocked_pack(s);
        orc_blocked_unpack(s);
        orc_blocked_update(s);
    }
    return ORC_OK;
}

/* exchange, then || s - c*u ||_2 over all interior points of all blocks */
int orc_blocked_residual(orc_blocked *s, double *out_l2)
{
    if (!s || !out_l2) return ORC_EINVAL;
    orc_blocked_pack(s);
    orc_blocked_unpack(s);
    const int64_t px = s->p[0], pxy = s->p[0] * s->p[1];
    long double total = 0.0L;
    for (int64_t blk = 0; blk < s->nblocks; ++blk) {
        const double *u = blk_u(s, s->cur, blk);
        const double *f = s->f ? s->f + blk * s->blk_elems : NULL;
        long double acc = 0.0L;
        int64_t ext[3];
        blk_extent(s, blk, ext);
        for (int64_t k = 0; k < ext[2]; ++k)
            for (int64_t j = 0; j < ext[1]; ++j)
                for (int64_t i = 0; i < ext[0]; ++i) {
                    const int64_t p = pad_index(s, i, j, k);
                    double sum = (u[p - 1] + u[p + 1]) + (u[p - px] + u[p + px]);
                    if (s->ndim == 3) sum = sum + (u[p - pxy] + u[p + pxy]);
                    if (f) sum = sum + f[(k * s->b[1] + j) * s->b[0] + i];
                    const double t = (s->ndim == 3 ? 6.0 : 4.0) * u[p];
                    const double r = sum - t;
                    acc += (long double)r * (long double)r;
                }
        total += acc;
    }
    *out_l2 = (double)sqrtl(total);
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Wide exchange: h ghost layers license up to h sweeps per exchange.        */
/*                                                                           */
/* Not in the paper, which exchanges before every update (Section V-C); this */
/* is the same pack -> transfer -> unpack step made once per group of sweeps.*/
/* A radius-1 stencil applied t times reaches t cells in every axis at once, */
/* so the ghost layers must also hold edge and corner data.  They are filled */
/* axis by axis: phase x, then y, then z.  In phase a the strip of a face is */
/* the h layers next to it along a, over the WHOLE padded extent (-h .. b+h) */
/* of every other axis, so what an earlier phase delivered travels on.       */
/* After the last phase every ghost cell whose position lies inside the      */
/* domain holds the owner's current value, and every ghost cell outside the  */
/* domain in exactly one axis holds that face's Dirichlet value (cells       */
/* outside in two or more axes are never read).                              */
/*                                                                           */
/* A group of t <= h sweeps then runs with no further exchange: sweep number */
/* m (m = 1..t) updates every block's interior extended by e = t - m layers  */
/* on every side; positions outside the domain keep their value.  The last   */
/* sweep of a group (e = 0) is the ordinary update.  Interiors end up bit    */
/* for bit as with an exchange before every sweep.                           */
/* ------------------------------------------------------------------------- */

/* index range of the wide strip on `face`: h layers along the face's axis (interior layers if
 * ghost == 0, ghost layers if ghost == 1), the whole padded extent along the other axes */
static void wide_strip_range(const orc_blocked *s, int64_t blk, int face, int ghost, int64_t lo[3], int64_t hi[3])
{
    strip_range(s, blk, face, ghost, lo, hi);
    const int axis = face / 2;
    for (int a = 0; a < s->ndim; ++a)
        if (a != axis) { lo[a] = -s->h; hi[a] = hi[a] + s->h; }
}

int64_t orc_blocked_wide_face_elems(const orc_blocked *s, int64_t blk, int face)
{
    if (!s || blk < 0 || blk >= s->nblocks || face < 0 || face >= 2 * s->ndim) return ORC_EINVAL;
    int64_t lo[3], hi[3];
    wide_strip_range(s, blk, face, 0, lo, hi);
    return (hi[0] - lo[0]) * (hi[1] - lo[1]) * (hi[2] - lo[2]);
}

static int64_t wide_max_face(const orc_blocked *s)
{
    int64_t m = 0;
    for (int fc = 0; fc < 2 * s->ndim; ++fc) {
        const int64_t e = orc_blocked_wide_face_elems(s, 0, fc);   /* block 0 is never a remainder block unless it is the only one */
        if (e > m) m = e;
    }
    return m;
}

/* One phase (one axis) of the wide exchange on the padded arrays `arr` (nblocks * pad_elems):
 * pack both faces of every block that have a neighbour, then unpack. `wsend` holds
 * nblocks * 6 * wmax doubles. */
static void wide_phase(const orc_blocked *s, double *arr, double *wsend, int64_t wmax, int axis)
{
    for (int64_t blk = 0; blk < s->nblocks; ++blk) {
        const double *u = arr + blk * s->pad_elems;
        for (int face = 2 * axis; face < 2 * axis + 2; ++face) {
            if (blk_neighbour(s, blk, face) < 0) continue;
            int64_t lo[3], hi[3];
            wide_strip_range(s, blk, face, 0, lo, hi);
            double *buf = wsend + (blk * 6 + face) * wmax;
            int64_t q = 0;
            for (int64_t k = lo[2]; k < hi[2]; ++k)
                for (int64_t j = lo[1]; j < hi[1]; ++j)
                    for (int64_t i = lo[0]; i < hi[0]; ++i)
                        buf[q++] = u[pad_index(s, i, j, k)];
        }
    }
    for (int64_t blk = 0; blk < s->nblocks; ++blk) {
        double *u = arr + blk * s->pad_elems;
        for (int face = 2 * axis; face < 2 * axis + 2; ++face) {
            const int64_t nb = blk_neighbour(s, blk, face);
            if (nb < 0) continue;
            int64_t lo[3], hi[3];
            wide_strip_range(s, blk, face, 1, lo, hi);
            const double *buf = wsend + (nb * 6 + (face ^ 1)) * wmax;
            int64_t q = 0;
            for (int64_t k = lo[2]; k < hi[2]; ++k)
                for (int64_t j = lo[1]; j < hi[1]; ++j)
                    for (int64_t i = lo[0]; i < hi[0]; ++i)
                        u[pad_index(s, i, j, k)] = buf[q++];
        }
    }
}

/* Wide exchange of the current state.  If wide_bufs is not NULL it receives the packed wide
 * faces as each phase left them: nblocks * 6 slots of orc_blocked_wide_max_face() doubles. */
int orc_blocked_exchange_wide(orc_blocked *s, double *wide_bufs)
{
    if (!s) return ORC_EINVAL;
    const int64_t wmax = wide_max_face(s);
    double *wsend = wide_bufs ? wide_bufs
                              : (double *)calloc((size_t)(s->nblocks * 6 * wmax), sizeof(double));
    if (!wsend) return ORC_ENOMEM;
    for (int axis = 0; axis < s->ndim; ++axis)
        wide_phase(s, s->u[s->cur], wsend, wmax, axis);
    if (!wide_bufs) free(wsend);
    return ORC_OK;
}

int64_t orc_blocked_wide_max_face(const orc_blocked *s)
{
    return s ? wide_max_face(s) : ORC_EINVAL;
}

/* f at block-relative position (i, j, k) of block `blk`, which may lie in a neighbouring
 * block: f is one global field, looked up by global coordinates */
static double f_global(const orc_blocked *s, const int64_t c[3], int64_t i, int64_t j, int64_t k)
{
    const int64_t rel[3] = {i, j, k};
    int64_t bc[3], in[3];
    for (int a = 0; a < 3; ++a) {
        const int64_t gpos = c[a] * s->b[a] + rel[a];
        bc[a] = gpos / s->b[a];
        in[a] = gpos - bc[a] * s->b[a];
    }
    int64_t owner = (bc[2] * s->g[1] + bc[1]) * s->g[0] + bc[0];
    return s->f[owner * s->blk_elems + (in[2] * s->b[1] + in[1]) * s->b[0] + in[0]];
}

/* The update over every block's interior extended by e layers on every side (0 <= e < h),
 * reading the padded array as it is.  Positions outside the domain keep their value. */
int orc_blocked_update_ext(orc_blocked *s, int64_t e)
{
    if (!s || e < 0 || e >= s->h) return ORC_EINVAL;
    const int64_t px = s->p[0], pxy = s->p[0] * s->p[1];
    const int64_t ez = (s->ndim == 3) ? e : 0;
    const double c6 = 1.0 / 6.0;
#pragma omp parallel for schedule(static)
    for (int64_t blk = 0; blk < s->nblocks; ++blk) {
        const double *u = blk_u(s, s->cur, blk);
        double *o = blk_u(s, s->cur ^ 1, blk);
        int64_t c[3], ext[3];
        blk_coords(s, blk, c);
        blk_extent(s, blk, ext);
        for (int64_t k = -ez; k < ext[2] + ez; ++k)
            for (int64_t j = -e; j < ext[1] + e; ++j)
                for (int64_t i = -e; i < ext[0] + e; ++i) {
                    const int64_t p = pad_index(s, i, j, k);
                    const int64_t gi = c[0] * s->b[0] + i, gj = c[1] * s->b[1] + j,
                                  gk = c[2] * s->b[2] + k;
                    if (gi < 0 || gi >= s->n[0] || gj < 0 || gj >= s->n[1] || gk < 0 || gk >= s->n[2]) {
                        o[p] = u[p];
                        continue;
                    }
                    double sum = (u[p - 1] + u[p + 1]) + (u[p - px] + u[p + px]);
                    if (s->ndim == 3) sum = sum + (u[p - pxy] + u[p + pxy]);
                    if (s->f) sum = sum + f_global(s, c, i, j, k);
                    o[p] = (s->ndim == 3) ? sum * c6 : sum * 0.25;
                }
    }
    s->cur ^= 1;
    return ORC_OK;
}

/* nsweeps sweeps in groups of at most k (1 <= k <= h): wide exchange, then the group's
 * updates on extents shrinking to the interior. */
int orc_blocked_sweep_wide(orc_blocked *s, int64_t nsweeps, int64_t k)
{
    if (!s || nsweeps < 0 || k < 1 || k > s->h) return ORC_EINVAL;
    for (int64_t left = nsweeps; left > 0;) {
        const int64_t t = left < k ? left : k;
        const int rc = orc_blocked_exchange_wide(s, NULL);
        if (rc) return rc;
        for (int64_t m = 1; m <= t; ++m) orc_blocked_update_ext(s, t - m);
        left -= t;
    }
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Slabs: one domain held as several blocked states, cut along the slowest   */
/* axis into runs of whole block planes (the paper's proxy spreads its       */
/* blocks over many GPUs, Section V-C; each slab stands for one GPU's part). */
/*                                                                           */
/* A slab is an ordinary blocked state over its own extent.  Where its low   */
/* or high end along the slowest axis is a cut and not a domain face, the    */
/* ghost layers there hold the neighbouring slab's face instead of a         */
/* Dirichlet value: before every update the h interior layers next to the    */
/* cut are packed (all blocks of that plane, block order, each block's face  */
/* in the order of a packed face, one slot of face_elems[] per block),       */
/* carried to the neighbour, and unpacked into its ghost layers.  Exactly    */
/* the pack -> transfer -> unpack of the faces between blocks, for the faces */
/* that cross a cut.  A run over slabs is bit-identical to the run over the  */
/* whole domain.                                                             */
/* ------------------------------------------------------------------------- */

/* blocks of the first (side 0) or last (side 1) plane along the slowest axis */
static void slab_plane(const orc_blocked *s, int side, int64_t *blk0, int64_t *count)
{
    const int sa = s->ndim - 1;
    *count = s->nblocks / s->g[sa];
    *blk0 = side ? (s->g[sa] - 1) * *count : 0;
}

/* doubles of one packed cut plane */
int64_t orc_blocked_cut_elems(const orc_blocked *s)
{
    if (!s) return ORC_EINVAL;
    int64_t blk0, count;
    slab_plane(s, 0, &blk0, &count);
    return count * s->face_elems[2 * (s->ndim - 1)];
}

/* the h interior layers next to the low / high end of the slowest axis -> out */
int orc_blocked_pack_cut(const orc_blocked *s, int side, double *out)
{
    if (!s || !out || side < 0 || side > 1) return ORC_EINVAL;
    const int face = 2 * (s->ndim - 1) + side;
    int64_t blk0, count;
    slab_plane(s, side, &blk0, &count);
    for (int64_t m = 0; m < count; ++m) {
        const double *u = blk_u(s, s->cur, blk0 + m);
        int64_t lo[3], hi[3];
        strip_range(s, blk0 + m, face, 0, lo, hi);
        double *buf = out + m * s->face_elems[face];
        int64_t q = 0;
        for (int64_t k = lo[2]; k < hi[2]; ++k)
            for (int64_t j = lo[1]; j < hi[1]; ++j)
                for (int64_t i = lo[0]; i < hi[0]; ++i)
                    buf[q++] = u[pad_index(s, i, j, k)];
    }
    return ORC_OK;
}

/* in (a plane packed by the neighbouring slab from its face towards this one) -> the ghost
 * layers at the low / high end of the slowest axis */
int orc_blocked_unpack_cut(orc_blocked *s, int side, const double *in)
{
    if (!s || !in || side < 0 || side > 1) return ORC_EINVAL;
    const int face = 2 * (s->ndim - 1) + side;
    int64_t blk0, count;
    slab_plane(s, side, &blk0, &count);
    for (int64_t m = 0; m < count; ++m) {
        double *u = blk_u(s, s->cur, blk0 + m);
        int64_t lo[3], hi[3];
        strip_range(s, blk0 + m, face, 1, lo, hi);
        const double *buf = in + m * s->face_elems[face];
        int64_t q = 0;
        for (int64_t k = lo[2]; k < hi[2]; ++k)
            for (int64_t j = lo[1]; j < hi[1]; ++j)
                for (int64_t i = lo[0]; i < hi[0]; ++i)
                    u[pad_index(s, i, j, k)] = buf[q++];
    }
    return ORC_OK;
}
