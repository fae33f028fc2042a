// Generic sweep: gathers every tap from global memory.  Covers every request the plan
// accepts (2D/3D, star/box, any radius up to the plan limit, zero or periodic boundary,
// any grid size including grids smaller than the stencil, fp32 or FP64).  It is the
// safety net behind the tiled kernels, not the fast path.
//
// out[p] = sum_t w_t * in[p + o_t]   (cross-correlation, stride 1; taps that leave the
// grid contribute 0 under the zero boundary and wrap under the periodic one).
//
// A CTA works on one segment of one grid row at a time, so y and z are the same for all of
// its threads.  For every segment the threads first resolve each tap once for the whole
// CTA: which input row it reads (after the bounds test or the wrap in y and z) as a flat
// offset, kept in shared memory.  The per-point loop is then one shared-memory read, the
// x test or wrap, one coalesced global read and one FMA per tap.
#pragma once
#include "common.cuh"

namespace stencil {

constexpr int kGenericThreads = 256;
constexpr int kGenericSmemTaps = 1024;   // taps resolved per round (more taps: several rounds)

__device__ __forceinline__ int wrap_index(int q, int n) {
    q %= n;
    return q < 0 ? q + n : q;
}

template <typename T>
struct ResolvedTap {
    long long row;      // flat offset of the input row this tap reads; -1: the row is outside the grid
    int dx;
    T w;
};

// T = float, or double for FP64 plans (the precision of the paper's case study).
template <bool kPeriodic, typename T = float>
__global__ void __launch_bounds__(kGenericThreads)
stencil_generic_kernel(const T* __restrict__ in, T* __restrict__ out, Grid g,
                       const TapT<T>* __restrict__ taps, int ntaps) {
    constexpr int kRound = sizeof(T) == 8 ? kGenericSmemTaps / 2 : kGenericSmemTaps;   // taps per round
    __shared__ TapT<T> s_raw[kRound];            // the taps as given (staged once when they fit)
    __shared__ ResolvedTap<T> s_tap[kRound];     // ... resolved for the current row

    const bool staged = ntaps <= kRound;
    if (staged) {
        for (int t = threadIdx.x; t < ntaps; t += kGenericThreads) s_raw[t] = taps[t];
    }
    const int xblocks = (g.nx + kGenericThreads - 1) / kGenericThreads;
    const long long nsegments = (long long)xblocks * g.ny * g.nz;
    // every CTA takes a contiguous run of segments (x fastest, then y): the rows above and below
    // a row are then read by the same CTA one step earlier or later and hit in L1
    const long long per_cta = (nsegments + gridDim.x - 1) / gridDim.x;
    const long long seg_end = min(nsegments, (long long)(blockIdx.x + 1) * per_cta);
    for (long long seg = (long long)blockIdx.x * per_cta; seg < seg_end; ++seg) {
        const int xb = (int)(seg % xblocks);
        const long long row = seg / xblocks;                 // = z * ny + y
        const int y = (int)(row % g.ny);
        const int z = (int)(row / g.ny);
        const int x = min(xb * kGenericThreads + (int)threadIdx.x, g.nx - 1);   // idle lanes shadow the last point
        const long long self = row * g.nx + x;
        T acc = T(0);
        for (int t0 = 0; t0 < ntaps; t0 += kRound) {
            const int nt = min(kRound, ntaps - t0);
            __syncthreads();                                 // taps staged / previous round no longer read
            for (int t = threadIdx.x; t < nt; t += kGenericThreads) {
                const TapT<T> tap = staged ? s_raw[t] : taps[t0 + t];
                int qz = z + tap.dz, qy = y + tap.dy;
                bool inside = true;
                if (kPeriodic) {
                    qz = wrap_index(qz, g.nz);
                    qy = wrap_index(qy, g.ny);
                } else {
                    inside = (unsigned)qz < (unsigned)g.nz && (unsigned)qy < (unsigned)g.ny;
                }
                ResolvedTap<T> r;
                r.row = inside ? ((long long)qz * g.ny + qy) * g.nx : -1;
                r.dx = tap.dx;
                r.w = tap.w;
                s_tap[t] = r;
            }
            __syncthreads();
            // Branch-free inner loop so that several loads are in flight per thread: a tap that
            // leaves the grid loads the thread's own point (a safe address) and contributes an exact
            // zero, value and weight both, so that a non-finite own point cannot leak into the sum
            // (the tiled kernels read zero-filled halos there and give the same result).
#pragma unroll 4
            for (int t = 0; t < nt; ++t) {
                const ResolvedTap<T> r = s_tap[t];
                int qx = x + r.dx;
                bool ok = r.row >= 0;
                if (kPeriodic) {
                    if (qx < 0 || qx >= g.nx) qx = wrap_index(qx, g.nx);
                } else {
                    ok = ok && (unsigned)qx < (unsigned)g.nx;
                }
                const T v = __ldg(in + (ok ? r.row + qx : self));
                acc = fma_t(ok ? r.w : T(0), ok ? v : T(0), acc);
            }
        }
        if (xb * kGenericThreads + (int)threadIdx.x < g.nx) out[self] = acc;
    }
}

// Grid size for a launch of the kernel above: a few resident waves of CTAs that loop over the
// row segments.
inline int generic_grid_size(const Grid& g, int sm_count) {
    const long long xblocks = (g.nx + kGenericThreads - 1) / kGenericThreads;
    const long long nsegments = xblocks * g.ny * g.nz;
    const long long cap = (long long)sm_count * 8 * 4;
    return (int)(nsegments < cap ? nsegments : cap);
}

}  // namespace stencil
