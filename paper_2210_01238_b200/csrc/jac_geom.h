// Geometry shared by the host code and the kernels of libjac (plain data, passed by value).
//
// Physical placement of one block (element = one double):
//
//   row    = [ xpad margin | bx interior | xpad margin ]      PX  = bx + 2*xpad
//   plane  = (h + by + h) rows                                PXY = PX * (by + 2h)
//   block  = (h + bz + h) planes in 3D, 1 plane in 2D         block_stride (multiple of 16)
//
// xpad is h rounded up to a multiple of 4, so the first interior point of every row sits on
// a 32-byte sector boundary and the ghost columns are the innermost h cells of the margin.
// `origin` is the offset of interior point (0,0,0).  u, u' and f all use this placement, so
// one offset addresses all three.
#pragma once
#include <stdint.h>

struct JacGeom {
    int ndim, h, xpad, nfaces;
    int bx, by, bz;  // block interior
    int rx, ry, rz;  // interior of the last block along each axis: b, or the remainder n - (g-1)*b when
                     // the grid is not a multiple of the block size (the block keeps full-size storage,
                     // its interior in the low corner, its +ghost layers right after its interior)
    int gx, gy, gz;  // block grid
    long long nx, ny, nz;
    long long PX, PXY, block_stride, origin;
    long long nblocks;
    long long face_elems[6];
    long long face_off[6];
    long long send_stride;
    double bval[6];
    // 1/4 and 1/6 (correctly rounded), for kernels that want the stencil's factor as an operand
    // from the constant bank instead of a literal they would have to build in registers
    double quarter, sixth;
    // wide exchange: a wide face is h layers along its axis and the whole padded extent
    // (b + 2h) along the other axes
    long long wface_elems[6];
    // extended update: the kernel is handed a geometry whose block box is the interior grown by
    // `ext` layers on every side (bx, by, bz and origin adjusted; 0 in the context's own geometry)
    int ext;
    // jac_solve: where a call that has met its tolerance raises a flag; the sweep and halo kernels of
    // the call's later groups look at it first and return at once (null outside jac_solve)
    const int* stop;
    // Checked build (JAC_CHECK_BOUNDS): the byte ranges a kernel's global accesses must stay inside --
    // [0] the solution arrays and f, [1] the send buffers, [2] the reduction scratch -- and the word
    // that records the first access outside them (which is then skipped).  Unused otherwise.
    const char* chk_lo[3];
    const char* chk_hi[3];
    unsigned long long* chk_rec;
};
