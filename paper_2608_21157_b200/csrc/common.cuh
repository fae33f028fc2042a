// Shared device-side definitions of the stencil library (CUDA path only).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace stencil {

// One non-zero tap: in[p + (dz,dy,dx)] * w.
struct Tap {
    int dz, dy, dx;
    float w;
};

// Grid extents as the kernels see them; 2D grids have nz == 1.
struct Grid {
    int nz, ny, nx;
};

// Value of the plan's device status word once a bounded wait has given up.
constexpr int kStatusTimeout = -5;

}  // namespace stencil
