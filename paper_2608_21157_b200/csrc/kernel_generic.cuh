// Generic sweep: one thread per grid point, gathers its taps from global
// memory.  Covers every request the plan accepts (2D/3D, star/box, any radius
// up to the plan limit, zero or periodic boundary, any grid size including
// grids smaller than the stencil).  It is the safety net behind the tiled
// kernels, not the fast path.
//
// out[p] = sum_t w_t * in[p + o_t]   (cross-correlation, stride 1; taps that
// leave the grid contribute 0 under the zero boundary and wrap under the
// periodic one).
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

    const int64_t plane = (int64_t)g.ny * g.nx;
    const int64_t N = plane * g.nz;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < N; i += stride) {
        const int x = (int)(i % g.nx);
        const int64_t r = i / g.nx;
        const int y = (int)(r % g.ny);
        const int z = (int)(r / g.ny);
        T acc = T(0);
        for (int t = 0; t < ntaps; ++t) {
            const TapT<T> tap = tp[t];
            int qz = z + tap.dz, qy = y + tap.dy, qx = x + tap.dx;
            if (kPeriodic) {
                qz = wrap_index(qz, g.nz);
                qy = wrap_index(qy, g.ny);
                qx = wrap_index(qx, g.nx);
            } else if ((unsigned)qz >= (unsigned)g.nz || (unsigned)qy >= (unsigned)g.ny ||
                       (unsigned)qx >= (unsigned)g.nx) {
                continue;
            }
            acc = fma_t(tap.w, __ldg(in + (int64_t)qz * plane + (int64_t)qy * g.nx + qx), acc);
        }
        out[i] = acc;
    }
}

}  // namespace stencil
