// jac_residual_dense_static: residual norm of a dense grid with no workspace at all.
//
// Who needs this.  Every other entry point of the library works on a context, and a context
// needs a device workspace of two to three times the grid -- which the caller must allocate.
// Some callers cannot allocate: code that runs inside another framework's memory pool and is
// not allowed to call cudaMalloc behind its back, a monitoring hook that fires in the middle of
// someone else's time step (cudaMalloc synchronises the whole device and would stall that
// step), or a process whose device memory is already filled by the solver it is watching.
// Such a caller usually holds just the solver's dense u (and f) arrays and wants one number:
// how far from converged they are.  This entry point computes that number from the dense
// arrays directly.  Its only scratch -- one partial sum per chunk of the grid, and the final
// sum -- lives in a fixed array that is part of the loaded library image.
//
// Consequences of the fixed array, all of them part of the contract:
//   * every GPU that loads the library carries the array (about 0.5 MB) until the process exits;
//   * the grid may have at most kMaxPoints points; larger ones are refused with JAC_ELIMIT;
//   * all calls on one device share the array, and it keeps whatever the previous call left in
//     it.  The part a call uses is cleared first, on the caller's stream.  Two calls whose GPU
//     work overlaps (different streams, or different host threads) race on it and give garbage:
//     serialise them.
//   * the address of the array is looked up the first time the entry point is called on a
//     device.  That lookup is not stream work; make the first call on each device outside any
//     stream capture.
//
// This file shares nothing with the rest of the library except the header: it has its own
// kernels and calls no allocating routine (no cudaMalloc, cudaFree, cudaMallocAsync, ...).
#include <cuda_runtime.h>

#include <cmath>
#include <mutex>

#include "jac.h"

namespace {

constexpr int kChunk = 8192;                         // points reduced by one CTA
constexpr long long kMaxPartials = 65536;            // one double per chunk
constexpr long long kMaxPoints = kMaxPartials * kChunk;  // 2^29 points (a 4 GiB fp64 grid)
constexpr int kMaxDevices = 64;

// [0, kMaxPartials): per-chunk partial sums; [kMaxPartials]: the total.
static __device__ __align__(256) double g_static_scratch[kMaxPartials + 32];

// In host code `g_static_scratch` is only a handle for the runtime, not a device address;
// the address a kernel can use has to be asked for, once per device.
double* g_scratch_addr[kMaxDevices] = {nullptr};
std::mutex g_scratch_mutex;

cudaError_t scratch_for_current_device(double** out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        double* p = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

struct DenseGrid {
    int ndim;
    long long nx, ny, nz;
    double bval[6];
};

// Fixed-order sum over the CTA; total valid in thread 0.
__device__ double cta_sum(double v)
{
    __shared__ double part[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v = __dadd_rn(v, __shfl_down_sync(0xffffffffu, v, off));
    if (lane == 0) part[warp] = v;
    __syncthreads();
    double total = 0.0;
    if (threadIdx.x == 0)
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) total = __dadd_rn(total, part[w]);
    return total;
}

// One CTA per chunk of kChunk consecutive points of the dense array (x fastest).  A neighbour
// outside the grid is the Dirichlet value of that face.  Same operation order as the library's
// update: s = (W + E) + (S + N) [+ (D + U)] [+ f]; r = s - c*u.
template <bool HAS_F>
__global__ void __launch_bounds__(256)
dense_residual_kernel(const double* __restrict__ u, const double* __restrict__ f, const DenseGrid g,
                      double* __restrict__ partials)
{
    const long long total = g.nx * g.ny * g.nz;
    const long long p0 = (long long)blockIdx.x * kChunk;
    const long long nxy = g.nx * g.ny;
    double acc = 0.0;
    for (int q = threadIdx.x; q < kChunk; q += blockDim.x) {
        const long long p = p0 + q;
        if (p >= total) break;
        const long long i = p % g.nx;
        const long long t = p / g.nx;
        const long long j = t % g.ny;
        const long long k = t / g.ny;
        const double W = i > 0 ? u[p - 1] : g.bval[0];
        const double E = i + 1 < g.nx ? u[p + 1] : g.bval[1];
        const double S = j > 0 ? u[p - g.nx] : g.bval[2];
        const double N = j + 1 < g.ny ? u[p + g.nx] : g.bval[3];
        double s = __dadd_rn(__dadd_rn(W, E), __dadd_rn(S, N));
        double c = 4.0;
        if (g.ndim == 3) {
            const double D = k > 0 ? u[p - nxy] : g.bval[4];
            const double U = k + 1 < g.nz ? u[p + nxy] : g.bval[5];
            s = __dadd_rn(s, __dadd_rn(D, U));
            c = 6.0;
        }
        if (HAS_F) s = __dadd_rn(s, f[p]);
        const double r = __dsub_rn(s, __dmul_rn(c, u[p]));
        acc = __dadd_rn(acc, __dmul_rn(r, r));
    }
    const double sum = cta_sum(acc);
    if (threadIdx.x == 0) partials[blockIdx.x] = sum;
}

__global__ void __launch_bounds__(1024)
dense_residual_total_kernel(const double* __restrict__ partials, const long long n, double* __restrict__ out)
{
    double acc = 0.0;
    for (long long i = threadIdx.x; i < n; i += blockDim.x) acc = __dadd_rn(acc, partials[i]);
    const double sum = cta_sum(acc);
    if (threadIdx.x == 0) *out = sum;
}

}  // namespace

extern "C" int jac_residual_dense_static(int ndim, const int64_t* n, const double* dev_u,
                                         const double* dev_f, const double* host_bvals,
                                         void* stream, double* host_out_l2)
{
    if ((ndim != 2 && ndim != 3) || !n || !dev_u || !host_out_l2) return JAC_EINVAL;
    DenseGrid g;
    g.ndim = ndim;
    g.nx = n[0];
    g.ny = n[1];
    g.nz = ndim == 3 ? n[2] : 1;
    if (g.nx < 1 || g.ny < 1 || g.nz < 1) return JAC_EINVAL;
    if (g.nx > kMaxPoints || g.ny > kMaxPoints || g.nz > kMaxPoints) return JAC_ELIMIT;
    if (g.nx * g.ny > kMaxPoints || g.nx * g.ny * g.nz > kMaxPoints) return JAC_ELIMIT;
    for (int fc = 0; fc < 6; ++fc) g.bval[fc] = (host_bvals && fc < 2 * ndim) ? host_bvals[fc] : 0.0;

    double* scratch = nullptr;
    if (scratch_for_current_device(&scratch) != cudaSuccess) {
        cudaGetLastError();
        return JAC_ECUDA;
    }
    const cudaStream_t st = static_cast<cudaStream_t>(stream);
    const long long total = g.nx * g.ny * g.nz;
    const long long nparts = (total + kChunk - 1) / kChunk;
    double* result = scratch + kMaxPartials;

    // the array still holds the previous call's numbers: clear the part this call uses
    if (cudaMemsetAsync(scratch, 0, (size_t)nparts * sizeof(double), st) != cudaSuccess ||
        cudaMemsetAsync(result, 0, sizeof(double), st) != cudaSuccess) {
        cudaGetLastError();
        return JAC_ECUDA;
    }
    if (dev_f)
        dense_residual_kernel<true><<<(unsigned)nparts, 256, 0, st>>>(dev_u, dev_f, g, scratch);
    else
        dense_residual_kernel<false><<<(unsigned)nparts, 256, 0, st>>>(dev_u, dev_f, g, scratch);
    dense_residual_total_kernel<<<1, 1024, 0, st>>>(scratch, nparts, result);
    if (cudaGetLastError() != cudaSuccess) return JAC_ECUDA;
    double sum = 0.0;
    if (cudaMemcpyAsync(&sum, result, sizeof(double), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return JAC_ECUDA;
    }
    *host_out_l2 = std::sqrt(sum);
    return JAC_OK;
}
