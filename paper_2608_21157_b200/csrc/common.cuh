// Shared device-side definitions of the stencil library (CUDA path only).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace stencil {

// One non-zero tap: in[p + (dz,dy,dx)] * w.
template <typename T>
struct TapT {
    int dz, dy, dx;
    T w;
};
using Tap = TapT<float>;

__device__ __forceinline__ float fma_t(float a, float b, float c) { return fmaf(a, b, c); }
__device__ __forceinline__ double fma_t(double a, double b, double c) { return fma(a, b, c); }

// Grid extents as the kernels see them; 2D grids have nz == 1.
struct Grid {
    int nz, ny, nx;
};

// Value of the plan's device status word once a bounded wait has given up.
constexpr int kStatusTimeout = -5;

}  // namespace stencil
