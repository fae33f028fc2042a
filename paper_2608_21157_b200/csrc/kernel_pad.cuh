// Periodic boundary for the tiled kernels: the grid is first copied into a padded grid
// whose halo cells hold the wrapped values (R planes and rows on either side, 4 columns on
// either side so that rows stay 16-byte multiples); the zero-boundary kernels then read
// that copy with shifted TMA coordinates and never leave it.  Costs one extra read and
// write of the grid per sweep, which still beats gathering wrapped taps one by one.
#pragma once
#include "common.cuh"

namespace stencil {

constexpr int kPadX = 4;            // halo columns per side of the padded copy

// pad[z'][y'][x'] = in[(z' - rz) mod nz][(y' - ry) mod ny][(x' - 4) mod nx], one float4 per thread.
// rz = 0 for 2D grids (nz = 1).  nx is a multiple of 4, so every float4 wraps as a whole.
__global__ void __launch_bounds__(256)
stencil_pad_periodic_kernel(const float* __restrict__ in, float* __restrict__ pad, Grid g, int ry, int rz) {
    const int px4 = (g.nx + 2 * kPadX) / 4;
    const int nx4 = g.nx / 4;
    const int py = g.ny + 2 * ry, pz = g.nz + 2 * rz;
    const int64_t total = (int64_t)px4 * py * pz;          // float4 cells of the padded grid
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const float4* src = reinterpret_cast<const float4*>(in);
    float4* dst = reinterpret_cast<float4*>(pad);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int x4 = (int)(i % px4);
        const int64_t row = i / px4;
        const int yp = (int)(row % py), zp = (int)(row / py);
        int y = (yp - ry) % g.ny; if (y < 0) y += g.ny;
        int z = (zp - rz) % g.nz; if (z < 0) z += g.nz;
        int s4 = (x4 - kPadX / 4) % nx4; if (s4 < 0) s4 += nx4;
        dst[i] = src[((int64_t)z * g.ny + y) * nx4 + s4];
    }
}

}  // namespace stencil
