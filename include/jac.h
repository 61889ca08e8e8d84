/*
 * jac.h -- C ABI of libjac: block-decomposed Jacobi relaxation on one NVIDIA B200 (sm_100a).
 *
 * The method (paper, Section V-C "Proxy Application: Jacobi3d"): a fixed number of Jacobi
 * iterations over a domain decomposed into cuboid blocks.  In every iteration each block
 * packs its boundary faces into contiguous buffers, the buffers reach the neighbouring
 * blocks, are unpacked into their ghost cells, and once all halos are in place the Jacobi
 * update runs on the GPU.  The paper fixes neither the stencil nor the boundary rule; this
 * library uses
 *
 *     u'(p) = ( sum of the 2d face neighbours of u at p  [+ f(p)] ) * (1/c),   c = 2d,
 *
 * evaluated as  s = (W + E) + (S + N);  3D: s = s + (D + U);  with f: s = s + f;
 * u' = s * 0.25 (2D) or s * (1.0/6.0) (3D), every operation one IEEE-754 round-to-nearest
 * fp64 add or multiply (no fused multiply-add), Dirichlet values in the ghost layer around
 * the domain (one constant per domain face, default 0).
 *
 * Conventions
 *   - x is the fastest-varying axis, then y, then z.  "Dense" arrays are n[0]*n[1]*n[2]
 *     doubles in that order (in 2D n[2] = 1).
 *   - Blocks are numbered x-fastest over the block grid g[a] = ceil(n[a] / b[a]).  When n[a] is
 *     not a multiple of b[a] the last block along that axis is a remainder block of
 *     n[a] - (g[a]-1)*b[a] points (at least `halo`, else JAC_EINVAL).  It keeps the full-size
 *     placement of every block; its interior is the low corner of it and its +ghost layers come
 *     right after its interior; its packed faces are correspondingly smaller.  (The paper's
 *     decomposition is into equal cuboids; remainder blocks are an extension of this library.)
 *   - Faces: 0:-x 1:+x 2:-y 3:+y 4:-z 5:+z.  A face is the `halo` interior layers next to
 *     that side over the interior extent of the other axes (no edges, no corners).  A packed
 *     face holds those elements in source memory order: an x face is [bz][by][halo], a y face
 *     [bz][halo][bx], a z face [halo][by][bx] (last index fastest).  Faces on the domain
 *     boundary are neither packed nor unpacked.
 *   - All device work is issued on the caller's stream and is asynchronous unless stated.
 *   - The library never allocates or frees device memory: the caller passes one workspace
 *     (see jac_workspace_bytes) and keeps it, and the stream, alive until jac_destroy.
 *   - Every function returns JAC_OK (0) or a negative error code and never aborts; on error
 *     out-parameters are left untouched.  A CUDA failure is sticky: later calls on the same
 *     context return JAC_ECUDA until it is destroyed.
 *   - A context is not thread-safe; different contexts are independent.
 */
#ifndef JAC_H_
#define JAC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define JAC_OK        0
#define JAC_EINVAL   (-1)  /* null pointer, bad dimension, size, face, block or count            */
#define JAC_ENOMEM   (-2)  /* workspace null, too small or not 256-byte aligned                  */
#define JAC_ECUDA    (-3)  /* a CUDA runtime call failed (sticky); see jac_last_cuda_error       */
#define JAC_ENODEV   (-4)  /* no usable CUDA device                                              */
#define JAC_ELIMIT   (-5)  /* problem larger than the fixed scratch of jac_residual_dense_static */
#define JAC_ETIMEOUT (-6)  /* JAC_MODE_RESIDENT: a CTA gave up waiting for a neighbour's row (every
                              device-side wait is bounded); the state is not to be trusted.  Reported
                              by the next call that waits for the stream (sticky)                  */

/* How jac_sweep schedules one iteration.  All modes leave bit-identical interiors. */
#define JAC_MODE_FUSED    0 /* one launch per sweep over all blocks; across a face with a neighbour
                               block the update reads the neighbour's interior cell directly (the
                               value its packed face would carry): the exchange is fused into
                               the sweep and the inter-block ghost cells are not touched         */
#define JAC_MODE_PERTASK  1 /* the task-per-block schedule: per sweep one pack launch per
                               (block, face), one unpack launch per (block, face), one update
                               launch per block                                                  */
#define JAC_MODE_TEMPORAL 2 /* `tsteps` sweeps per launch; tiles read across block borders
                               directly (equivalent to an exchange before every sweep).
                               2D: b[0] % 4 == 0 and n[0] % 4 == 0, tsteps <= 8;
                               3D: b[0] % 2 == 0 and n[0] % 2 == 0, tsteps <= 3;
                               jac_create returns JAC_EINVAL otherwise                           */
#define JAC_MODE_EXCHANGE 3 /* the paper's order made explicit: per sweep every face is packed into
                               its send buffer and unpacked into the neighbour's ghost cells (both
                               by one launch over all blocks, as jac_exchange_halos), then one
                               update launch over all blocks reads the ghosts                    */
#define JAC_MODE_WIDE     4 /* one wide exchange (jac_exchange_wide: all h ghost layers, edges and
                               corners included) per group of `tsteps` <= h sweeps (0 = h); the
                               group's sweeps update boxes shrinking from the interior grown by
                               tsteps - 1 layers down to the interior, so neighbours are computed
                               redundantly instead of being exchanged.  2 * ndim + tsteps launches
                               per group                                                         */
#define JAC_MODE_RESIDENT 5 /* small 2D grids: all sweeps of a jac_sweep call in ONE launch of one
                               thread-block cluster (8 or 16 CTAs) that keeps the whole grid in
                               shared memory, slabs of rows per CTA, neighbouring slabs exchanging
                               their edge rows through distributed shared memory, one
                               row exchange per sweep (pairwise, through mbarriers).  Needs ndim == 2, b[0] and n[0] even and
                               (2*(r+2) + (has_f ? r : 0)) * (n[0]+4) * 8 bytes <= 227 KB for
                               r = ceil(n[1]/8) or ceil(n[1]/16) (e.g. 256 x 256 with f);
                               JAC_EINVAL otherwise, also when the device cannot co-schedule a
                               cluster of that size.  desc.tsteps = 8 or 16 fixes the cluster
                               size (0: 16 for grids of 128 rows or more, else 8; the other
                               size if that one does not fit or cannot be scheduled)             */

/* Descriptor flags. */
#define JAC_FLAG_HOST_STAGING 1 /* the workspace also holds two dense staging arrays (n[0]*n[1]*n[2]
                                   doubles each, accounted for by jac_workspace_bytes), and jac_set_u,
                                   jac_set_f, jac_get_u and their *_async forms move the grid as ONE
                                   contiguous copy per direction between the host and a staging
                                   array plus one kernel between the staging array and the blocks,
                                   instead of one strided copy per block.  The copy in runs on a
                                   stream of the context's own: it starts as soon as the staging
                                   array is free and overlaps whatever is queued on the caller's
                                   stream (the previous job's sweeps and copy out); the caller's
                                   stream waits for it before it touches the blocks.  For callers
                                   that stream jobs through a context from page-locked (pinned or
                                   registered) host memory; pageable host arrays are still accepted
                                   and take the per-block copies on the caller's stream            */

#define JAC_FLAG_CUT_LO 2       /* the context is one SLAB of a larger domain that is cut into slabs of  */
#define JAC_FLAG_CUT_HI 4       /* whole block planes along the slowest axis (y in 2D, z in 3D), one slab
                                   per GPU: the low / high end of that axis is a cut towards a
                                   neighbouring slab, not a domain face.  n[] is the slab's own extent.
                                   The ghost layers on a cut hold the neighbouring slab's face, which
                                   arrives through jac_unpack_cut / jac_sweep_end; the workspace also
                                   holds the packed cut planes (two send buffers and one receive buffer
                                   per cut).  Modes JAC_MODE_FUSED and JAC_MODE_EXCHANGE only; a slab
                                   sweeps through jac_sweep_begin / jac_sweep_end, jac_sweep is
                                   JAC_EINVAL.  With JAC_FLAG_CUT_HI n[slowest] must be a multiple of
                                   b[slowest]                                                      */

typedef struct jac_ctx jac_ctx; /* opaque, host memory, owned by the library */

typedef struct jac_desc {
    int32_t ndim;    /* 2 or 3                                                                   */
    int32_t halo;    /* ghost width h, 1 <= h <= min(b[a]) and h <= 8                            */
    int32_t has_f;   /* 0: f == 0 and is never read (16 B/point/sweep); 1: f present (24 B)      */
    int32_t mode;    /* JAC_MODE_*                                                               */
    int32_t tsteps;  /* JAC_MODE_TEMPORAL: sweeps per launch; JAC_MODE_WIDE: sweeps per exchange
                        (<= halo); JAC_MODE_RESIDENT: CTAs in the cluster (8 or 16); 0 = the
                        library chooses                                                          */
    int32_t flags;   /* JAC_FLAG_* bits, 0 for none                                              */
    int64_t n[3];    /* global interior points; n[2] ignored (taken as 1) when ndim == 2         */
    int64_t b[3];    /* block interior points, 1 <= b[a] <= n[a]                                 */
    void   *stream;  /* cudaStream_t of the caller (NULL = the legacy default stream)            */
} jac_desc;

/* Physical placement chosen for a descriptor (pure host query; element = one double). */
typedef struct jac_layout {
    int64_t g[3];          /* block grid                                                         */
    int64_t nblocks;
    int64_t pad[3];        /* padded block dims: pad[0] = b[0] + 2*xpad, pad[1] = b[1] + 2h,
                              pad[2] = b[2] + 2h (3D) or 1                                       */
    int64_t xpad;          /* ghost columns are the innermost h of an xpad-wide margin           */
    int64_t origin;        /* element offset of interior point (0,0,0) inside a padded block     */
    int64_t block_stride;  /* elements between consecutive blocks of one array                   */
    int64_t face_elems[6]; /* elements of one packed face of a full-size block                   */
    int64_t face_offset[6];/* element offset of each face inside a block's send region           */
    int64_t send_stride;   /* elements of one block's send region                                */
    int64_t partials;      /* doubles of reduction scratch                                       */
    int64_t off_u[2];      /* byte offsets inside the workspace: the two solution arrays,        */
    int64_t off_f;         /*   f (same padded layout as u; -1 if has_f == 0),                   */
    int64_t off_send;      /*   send buffers,                                                    */
    int64_t off_scratch;   /*   reduction scratch + result word                                  */
    int64_t total_bytes;
    int64_t wide_face_elems[6]; /* elements of one packed wide face (jac_exchange_wide); in
                                   JAC_MODE_WIDE the send slots are sized for these              */
    int64_t off_stage_in;  /* byte offsets of the dense staging arrays (JAC_FLAG_HOST_STAGING),  */
    int64_t off_stage_out; /*   -1 without the flag                                              */
    int64_t cut_elems;     /* doubles of one packed cut plane (JAC_FLAG_CUT_*; else 0): blocks of
                              the plane in block order, 128-byte aligned slots of face_elems     */
    int64_t off_cut_send[2][2]; /* [side][buffer] byte offsets of the send buffers of a cut,     */
    int64_t off_cut_recv[2];    /*   and of its receive buffer; -1 where the side is no cut      */
} jac_layout;

/* Workspace size in bytes for `desc` (pure host computation, no CUDA call).
 * Errors: JAC_EINVAL for a null pointer or an invalid descriptor. */
int jac_workspace_bytes(const jac_desc *desc, size_t *bytes);

/* The placement behind jac_workspace_bytes (pure host computation). */
int jac_get_layout(const jac_desc *desc, jac_layout *out);

/* Create a context over `dev_workspace` (DEVICE pointer, 256-byte aligned, >= the size from
 * jac_workspace_bytes).  Zero-fills both solution arrays, f and the send buffers on the
 * stream (so u = 0, f = 0, all Dirichlet values 0).  The device current at this call is the
 * one every later call on the context must be issued under.
 * Errors: JAC_EINVAL, JAC_ENOMEM, JAC_ENODEV, JAC_ECUDA. */
int jac_create(const jac_desc *desc, void *dev_workspace, size_t bytes, jac_ctx **out);

/* Frees the host-side context only (after synchronising the stream). */
int jac_destroy(jac_ctx *ctx);

/* Set / read the current solution or the right-hand side from a dense array.
 * jac_set_u, jac_set_f, jac_get_u take HOST pointers (pageable or pinned) and return after
 * the copy has completed; the *_device variants take DEVICE pointers to dense arrays and
 * are asynchronous on the stream.  jac_set_f* returns JAC_EINVAL when has_f == 0.
 * Setting u leaves inter-block ghost cells stale until the next exchange. */
int jac_set_u(jac_ctx *ctx, const double *host_dense);
int jac_set_f(jac_ctx *ctx, const double *host_dense);
int jac_get_u(jac_ctx *ctx, double *host_dense);
int jac_set_u_device(jac_ctx *ctx, const double *dev_dense);
int jac_set_f_device(jac_ctx *ctx, const double *dev_dense);
int jac_get_u_device(jac_ctx *ctx, double *dev_dense);

/* The same copies and the same residual without waiting for them: the work is queued on the
 * stream and the call returns.  For callers that keep several contexts busy at once, e.g. two
 * contexts on two streams so that the input copy of one job, the sweeps of another and the output
 * copy of a third overlap (the two copy directions and the SMs are separate engines).  The host
 * array must stay alive and untouched until the stream has passed the call, and should be pinned:
 * pageable memory makes the copies synchronous again.  jac_residual_async writes the norm to
 * *host_out_l2 when the stream gets there (pinned memory; synchronise the stream before reading);
 * its value has the bits jac_residual would return.  (No counterpart in the paper, whose proxy
 * keeps its data on the GPUs between iterations.) */
int jac_set_u_async(jac_ctx *ctx, const double *host_dense);
int jac_get_u_async(jac_ctx *ctx, double *host_dense);
int jac_residual_async(jac_ctx *ctx, double *host_out_l2);

/* Dirichlet value of one domain face: written into the ghost layers (all h of them, interior
 * extent) of every block touching that face, in both solution arrays.  Asynchronous. */
int jac_set_boundary(jac_ctx *ctx, int face, double value);

/* Inspection (synchronous, HOST output).
 * jac_get_block_padded: the canonical padded block (b+2h)^d of the current state, x fastest,
 *   ghost cells as they currently are (edge/corner ghosts are never written: they stay 0).
 * jac_get_halo_buffer: the packed face of (block, face) as the last pack left it; always
 *   face_elems[face] doubles are copied, of which a remainder block's face fills only the first
 *   h * (its extents on the other two axes). */
int jac_get_block_padded(jac_ctx *ctx, int64_t block, double *host);
int jac_get_halo_buffer(jac_ctx *ctx, int64_t block, int face, double *host);

/* Halo pack: for every block and every face with a neighbour block, gather the h interior
 * layers next to that face of the current state into the face's contiguous send buffer
 * (the packing step of paper Section V-C).  One launch over all blocks and faces
 * (JAC_MODE_PERTASK: one launch per block face). */
int jac_pack_halos(jac_ctx *ctx);

/* Halo unpack: for every block and every face with a neighbour, copy the neighbour's
 * opposite-face send buffer into this block's h ghost layers on that face (the unpacking step
 * of paper Section V-C).  On one GPU the transfer between pack and
 * unpack is the neighbour reading the send buffer in place. */
int jac_unpack_halos(jac_ctx *ctx);

/* jac_pack_halos followed by jac_unpack_halos as ONE launch: the thread that fills a ghost cell
 * reads the neighbour's interior cell and also leaves it in the neighbour's send slot, so the send
 * buffers and the ghosts are afterwards exactly what the two calls leave (one read and two writes
 * per face cell instead of two and two).  On one GPU, where the "transfer" between pack and unpack
 * (paper Section V-C) is a read in place, nothing is lost by not stopping in between; jac_residual
 * uses it when the ghosts are stale. */
int jac_exchange_halos(jac_ctx *ctx);

/* Pack / unpack only the faces whose bit is set in face_mask (bit i = face i).  Same kernels
 * and buffers as jac_pack_halos / jac_unpack_halos, one launch over all blocks; a mask with all
 * 2*ndim bits set is exactly those calls.  A partial exchange never marks the ghosts as current.
 * Lets a caller exchange one axis at a time, and lets the strided (x) and contiguous (y, z) faces
 * be timed apart.  Errors: JAC_EINVAL for bits beyond 2*ndim. */
int jac_pack_faces(jac_ctx *ctx, unsigned face_mask);
int jac_unpack_faces(jac_ctx *ctx, unsigned face_mask);

/* Wide exchange (JAC_MODE_WIDE contexts only, else JAC_EINVAL): fills ALL h ghost layers of the
 * current state, edges and corners included, so that up to h sweeps can follow without another
 * exchange (a radius-1 stencil applied t times reaches t cells along every axis at once).  The
 * paper exchanges before every update (Section V-C); this is the same pack -> transfer -> unpack
 * step made once per group of sweeps, the usual way to trade redundant computation for fewer,
 * larger messages.  It runs axis by axis, x then y then z, one pack and one unpack launch each:
 * the strip of a face is the h layers next to it along its axis over the WHOLE padded extent
 * (b + 2h) of the other axes, so data delivered for an earlier axis travels on into the edges
 * and corners.  A packed wide face is in source memory order: an x face is [bz+2h][by+2h][h], a y
 * face [bz+2h][h][bx+2h], a z face [h][by+2h][bx+2h] (2D: no z extent).  Afterwards every ghost
 * cell whose position lies inside the domain holds its owner's current value, and every ghost cell
 * outside the domain in exactly one axis holds that face's Dirichlet value.  Asynchronous.
 * jac_get_wide_buffer: the packed wide face of (block, face) as the exchange left it (HOST output,
 * synchronous; wide_face_elems[face] doubles). */
int jac_exchange_wide(jac_ctx *ctx);
int jac_get_wide_buffer(jac_ctx *ctx, int64_t block, int face, double *host);

/* nsweeps Jacobi iterations, each "exchange halos, then update every block" (paper Section
 * V-C), scheduled as desc.mode says.  Afterwards the interiors hold the new state; the
 * inter-block ghost cells are only guaranteed current after the next jac_pack_halos +
 * jac_unpack_halos (jac_residual does that itself when needed).  nsweeps == 0 is a no-op;
 * nsweeps < 0 is JAC_EINVAL. */
int jac_sweep(jac_ctx *ctx, int nsweeps);

/* jac_sweep(nsweeps) and, from the same pass over memory, the L2 residual norm of the state
 * BEFORE the last of those sweeps: the last sweep has s(p) of that state in a register anyway and
 * also accumulates ( s(p) - c*u(p) )^2, so the norm costs no extra memory traffic (jac_residual
 * reads u, and f, once more).  The value equals what jac_residual would return after
 * nsweeps - 1 sweeps, up to summation order (<= 1e-10 relative).  nsweeps >= 1.  Synchronises the
 * stream and writes one HOST double.  (The paper runs a fixed iteration count; this is the usual
 * one-iteration-lagged convergence monitor of a Jacobi solver.) */
int jac_sweep_residual(jac_ctx *ctx, int nsweeps, double *host_out_l2);

/* The residual norm of the CURRENT state, and then nsweeps sweeps, with the norm coming out of the
 * first sweep's pass over memory: that sweep reads the current state and forms s(p) anyway, so
 * it also accumulates ( s(p) - c*u(p) )^2.  The value is what jac_residual would return now (up to
 * summation order, <= 1e-10 relative), at no extra memory traffic and without the halo exchange a
 * separate residual pass needs.  For jobs that monitor the residual every k sweeps: a call per
 * group of k, and one jac_residual at the very end.  Nothing waits: the norm is written to
 * *host_out_l2 (pinned memory) when the stream gets there.  nsweeps >= 1.  In JAC_MODE_WIDE the
 * norm comes from an ordinary residual pass before the sweeps.  (Not in the paper, which runs a
 * fixed iteration count.) */
int jac_residual_sweep_async(jac_ctx *ctx, int nsweeps, double *host_out_l2);

/* nsweeps sweeps of a job that monitors the residual every `every` sweeps: host_out_l2[m - 1]
 * receives the L2 residual norm of the state after m * every sweeps, for every m >= 1 with
 * m * every < nsweeps (the state after the last sweep is read by no sweep of the call: jac_residual
 * or jac_residual_async gives its norm).  Each norm is what jac_residual would return at that
 * point, up to summation order (<= 1e-10 relative), and comes out of the sweep that reads the
 * state, as in jac_residual_sweep_async.  In JAC_MODE_TEMPORAL with every >= the sweeps per launch
 * the launches are not cut where a norm is due: a launch of T sweeps holds the states after
 * 0 .. T - 1 of its sweeps in its levels, and the level that reads the wanted state measures it,
 * so 50 sweeps at T = 3 with a norm every 10 run as 16 launches of depth 3 and one of 2, not as
 * 5 x (3 + 3 + 2 + 2).  Other schedules, and every < T, run group by group.  Nothing waits: the
 * norms are written (pinned memory: (nsweeps - 1) / every doubles) as the stream gets there.
 * nsweeps >= 1, every >= 1; host_out_l2 may be NULL when no norm falls inside the call.  Not for
 * slab contexts.  (Not in the paper, which runs a fixed iteration count.) */
int jac_sweep_norms_async(jac_ctx *ctx, int nsweeps, int every, double *host_out_l2);

/* Iterate until converged: runs sweeps in groups of check_every (each group as
 * jac_sweep_residual does) until the lagged residual norm is <= tol or max_sweeps sweeps have run.
 * The comparison with tol is made on the device: several groups are queued at a time without
 * waiting, a group whose norm meets tol raises a flag in the workspace, the launches queued behind
 * it see the flag and return at once, and the host looks at the flag only between batches of
 * groups (JAC_MODE_WIDE: after every group).  The result is that of stopping exactly after the
 * group that met tol.  HOST outputs: the sweeps actually done and the last norm measured (the
 * residual of the state one sweep before the final one).  Errors: JAC_EINVAL for max_sweeps < 1,
 * check_every < 1, tol < 0 or NaN, null outputs. */
int jac_solve(jac_ctx *ctx, int max_sweeps, int check_every, double tol, int *host_sweeps_done,
              double *host_residual);

/* L2 norm of the residual of the current state, sqrt( sum_p ( s(p) - c*u(p) )^2 ) with s as in
 * the update (including + f), over all interior points, not normalised.  (The paper runs a
 * fixed iteration count and has no residual; this is the convergence measure of the same
 * Jacobi method.)  Exchanges halos first if the ghosts are stale (jac_exchange_halos; pack and
 * unpack per block face in JAC_MODE_PERTASK), reduces on the device in a
 * fixed order (repeatable bit for bit), synchronises the stream and writes one HOST double. */
int jac_residual(jac_ctx *ctx, double *host_out_l2);

/* ---- Slab contexts: one domain sharded over several GPUs (JAC_FLAG_CUT_LO / JAC_FLAG_CUT_HI) ----
 *
 * The paper's proxy (Section V-C) spreads the blocks over many GPUs and credits its gains to
 * overlapping the halo messages with kernel work.  Here each GPU owns a slab of whole block planes
 * along the slowest axis as a context of its own; between slabs only the faces on the cut planes
 * travel, once per sweep, and the residual needs one 8-byte sum.  The library packs, unpacks and
 * orders its own streams; MOVING a packed plane to the neighbour is the caller's part -- an NCCL
 * send/recv between the buffers jac_cut_info names, or nothing at all when the neighbour slab's
 * send buffer can be read in place (same device, or a peer device mapped into this one: the unpack
 * kernel reads it with ordinary loads, every CTA its own part).
 *
 * jac_pack_cut: packs the cut faces of the CURRENT state into the send buffers (alternating between
 *   two buffers per cut, so a neighbour may still be reading the previous one).  Asynchronous.
 * jac_unpack_cut: fills the cut ghost layers of the current state from packed planes: dev_src_lo /
 *   dev_src_hi are DEVICE pointers to the plane the lower / upper neighbour packed from its face
 *   towards this slab (NULL: this context's own receive buffer of that side; ignored where the
 *   side is no cut); ready_lo / ready_hi are cudaEvent_t values the stream waits for before it
 *   reads (NULL: none; pass the neighbour's event from jac_cut_info when reading its buffer in
 *   place).  Marks the cut ghosts current.  jac_pack_cut + transfer + jac_unpack_cut is the cut
 *   exchange of the initial state; after that jac_sweep_begin / jac_sweep_end keep them current.
 * jac_sweep_begin: first half of one sweep.  Updates the block planes next to a cut first, packs
 *   their NEW cut faces (as jac_pack_cut does, recording the ready events), and starts the update
 *   of all other planes on a second stream of the context, so that the faces travel while the bulk
 *   of the slab is computed.  Needs current cut ghosts (JAC_EINVAL otherwise).
 * jac_sweep_end: second half.  Unpacks the neighbours' new faces (arguments as jac_unpack_cut) into
 *   the ghost layers of the new state, joins the second stream and makes the new state current.
 * jac_cut_info: for cut `side` (0 low, 1 high): the send buffer the LAST pack wrote, the receive
 *   buffer, their size in bytes and the event recorded after that pack (cudaEvent_t).  Host query;
 *   any output pointer may be NULL.
 * jac_residual_sumsq_async: as jac_residual_async, but the SUM OF SQUARES of the slab's residual
 *   (no square root), so that the sums of all slabs can be added and rooted once.  Works on any
 *   context.  jac_residual* on a slab need current cut ghosts.
 * Errors: JAC_EINVAL on a context without cuts, for a call out of order, a side that is no cut. */
int jac_pack_cut(jac_ctx *ctx);
int jac_unpack_cut(jac_ctx *ctx, const double *dev_src_lo, void *ready_lo, const double *dev_src_hi,
                   void *ready_hi);
int jac_sweep_begin(jac_ctx *ctx);
int jac_sweep_end(jac_ctx *ctx, const double *dev_src_lo, void *ready_lo, const double *dev_src_hi,
                  void *ready_hi);
int jac_cut_info(const jac_ctx *ctx, int side, void **dev_send, void **dev_recv, size_t *bytes,
                 void **ready_event);
int jac_residual_sumsq_async(jac_ctx *ctx, double *host_out_sumsq);

/* Residual norm of a DENSE grid without a context, a workspace or any allocation.
 * (The paper has no counterpart: this is a convenience of this library.)
 *
 * For callers that cannot allocate device memory -- code living inside another framework's
 * memory pool, a monitoring hook that must not stall the solver it watches (cudaMalloc
 * synchronises the device), a process whose device memory is already full -- and that hold
 * nothing but the solver's dense arrays.  Computes sqrt( sum_p ( s(p) - c*u(p) )^2 ), s as in the
 * update, over the n[0]*n[1](*n[2]) points of `dev_u` (DEVICE pointer, dense, x fastest; n[2] is
 * ignored when ndim == 2).  `dev_f` is a DEVICE pointer of the same shape or NULL for f == 0.
 * `host_bvals` is a HOST array of 2*ndim Dirichlet values in face order, or NULL for all zero.
 * `stream` is a cudaStream_t (NULL = legacy default stream).  Writes one HOST double after
 * synchronising the stream.  Inputs are only read; nothing is retained after the call.
 *
 * The only scratch is a fixed ~0.5 MB array inside the library image, held by every GPU that
 * loads the library until the process exits.  Hence:
 *   - at most 2^29 points (a 4 GiB fp64 grid); more returns JAC_ELIMIT and does nothing;
 *   - the array is shared by all calls on a device and keeps the previous call's contents; the
 *     part a call uses is cleared first.  Calls whose GPU work overlaps (other streams or
 *     threads) race on it: serialise them;
 *   - the first call on each device looks up the array's device address; make that first call
 *     before any stream capture begins.  (Every call, the first included, ends by synchronising
 *     `stream` to hand back the host double.)
 * Calls no cudaMalloc/cudaFree or other allocating routine.
 * Errors: JAC_EINVAL (null u or out, ndim not 2 or 3, a size < 1), JAC_ELIMIT, JAC_ECUDA. */
int jac_residual_dense_static(int ndim, const int64_t *n, const double *dev_u,
                              const double *dev_f, const double *host_bvals, void *stream,
                              double *host_out_l2);

/* Sweeps one launch of jac_sweep performs for this context (HOST output): desc.tsteps, or the
 * library's choice when that was 0, in JAC_MODE_TEMPORAL; 1 in every other mode. */
int jac_sweeps_per_launch(const jac_ctx *ctx, int *host_out);

/* Number of kernel launches this context has issued so far (HOST output). */
int jac_launch_count(const jac_ctx *ctx, int64_t *host_out);

/* cudaError_t value of the failure that made the context sticky (0 if none). */
int jac_last_cuda_error(const jac_ctx *ctx);

/* Out-of-bounds evidence of a CHECKED BUILD of the library (compiled with -DJAC_CHECK_BOUNDS: every
 * global-memory access of the kernels is first compared with the array it belongs to; an access
 * outside is skipped and the first one recorded; nothing traps).  Waits for the stream, then HOST
 * outputs: *host_checked = 1 if this build makes the checks, else 0; *host_record = 0 if no access
 * has left its array since the context was created, else kernel id << 56 | array << 52 | byte
 * offset from the array's start (low 52 bits, two's complement) of the first one (arrays: 0 the
 * solution arrays and f, 1 the send buffers, 2 the reduction scratch).  For tests; the ordinary
 * build always reports 0, 0. */
int jac_debug_bounds(jac_ctx *ctx, int *host_checked, uint64_t *host_record);

/* Test aid for the checked build: from now on the kernels of this context hold their accesses to
 * `array` (0, 1, 2 as above) against a range that ends `bytes` before the array's real end, so
 * that accesses which are in fact legitimate get flagged and skipped -- the way to see the check,
 * the record and the skipping at work without a single access outside the workspace.  No effect on
 * the ordinary build.  Errors: JAC_EINVAL for a bad array or more bytes than the array has. */
int jac_debug_shrink_bounds(jac_ctx *ctx, int array, int64_t bytes);

/* Static, NUL-terminated description of an error code. */
const char *jac_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* JAC_H_ */
