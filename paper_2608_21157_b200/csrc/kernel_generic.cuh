// Generic sweep: gathers every tap from global memory.  Covers every request the plan
// accepts (2D/3D, star/box, any radius up to the plan limit, zero or periodic boundary,
// any grid size including grids smaller than the stencil, fp32 or FP64).  It is the
// safety net behind the tiled kernels, not the fast path.
//
// out[p] = sum_t w_t * in[p + o_t]   (cross-correlation, stride 1; taps that leave the
// grid contribute 0 under the zero boundary and wrap under the periodic one).
//
// A CTA owns a segment of one grid row, so y and z (and with them the row a tap reads, and
// whether that row exists or where it wraps to) are the same for the whole CTA: the only
// per-thread boundary work is in x.  Reads along x are coalesced; the (2R+1) rows a CTA
// touches are shared with its neighbours through L1/L2.
#pragma once
#include "common.cuh"

namespace stencil {

constexpr int kGenericThreads = 256;
constexpr int kGenericSmemTaps = 1024;   // taps staged in shared memory when they fit

__device__ __forceinline__ int wrap_index(int q, int n) {
    q %= n;
    return q < 0 ? q + n : q;
}

// T = float, or double for FP64 plans (the precision of the paper's case study).
template <bool kPeriodic, typename T = float>
__global__ void __launch_bounds__(kGenericThreads)
stencil_generic_kernel(const T* __restrict__ in, T* __restrict__ out, Grid g,
                       const TapT<T>* __restrict__ taps, int ntaps) {
    __shared__ TapT<T> s_taps[kGenericSmemTaps];
    const bool staged = ntaps <= kGenericSmemTaps;
    if (staged) {
        for (int t = threadIdx.x; t < ntaps; t += blockDim.x) s_taps[t] = taps[t];
        __syncthreads();
    }
    const TapT<T>* tp = staged ? s_taps : taps;

    const int xblocks = (g.nx + kGenericThreads - 1) / kGenericThreads;
    const int64_t nsegments = (int64_t)xblocks * g.ny * g.nz;
    for (int64_t seg = blockIdx.x; seg < nsegments; seg += gridDim.x) {
        const int xb = (int)(seg % xblocks);
        const int64_t row = seg / xblocks;                 // = z * ny + y
        const int y = (int)(row % g.ny);
        const int z = (int)(row / g.ny);
        const int x = xb * kGenericThreads + threadIdx.x;
        if (x < g.nx) {
            T acc = T(0);
            for (int t = 0; t < ntaps; ++t) {
                const TapT<T> tap = tp[t];
                int qz = z + tap.dz, qy = y + tap.dy, qx = x + tap.dx;
                if (kPeriodic) {
                    qz = wrap_index(qz, g.nz);             // the same for the whole CTA
                    qy = wrap_index(qy, g.ny);
                    if (qx < 0 || qx >= g.nx) qx = wrap_index(qx, g.nx);
                } else {
                    if ((unsigned)qz >= (unsigned)g.nz || (unsigned)qy >= (unsigned)g.ny) continue;
                    if ((unsigned)qx >= (unsigned)g.nx) continue;
                }
                acc = fma_t(tap.w, __ldg(in + ((int64_t)qz * g.ny + qy) * g.nx + qx), acc);
            }
            out[row * g.nx + x] = acc;
        }
    }
}

// Grid size for a launch of the kernel above: a few resident waves of CTAs that loop over the
// row segments (one CTA per segment would spend its time on CTA turnover and tap staging).
inline int generic_grid_size(const Grid& g, int sm_count) {
    const int64_t xblocks = (g.nx + kGenericThreads - 1) / kGenericThreads;
    const int64_t nsegments = xblocks * g.ny * g.nz;
    const int64_t cap = (int64_t)sm_count * 8 * 4;
    return (int)(nsegments < cap ? nsegments : cap);
}

}  // namespace stencil
