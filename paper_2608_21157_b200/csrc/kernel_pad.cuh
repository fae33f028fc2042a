// Periodic boundary for the tiled kernels: the grid is first copied into a padded grid
// whose halo cells hold the wrapped values (R planes and rows on either side, 4 columns on
// either side so that rows stay 16-byte multiples); the zero-boundary kernels then read
// that copy with shifted TMA coordinates and never leave it.  Costs one extra read and
// write of the grid per sweep, which still beats gathering wrapped taps one by one.
#pragma once
#include "common.cuh"

namespace stencil {

constexpr int kPadX = 4;            // halo columns per side of the padded copy

template <typename T> struct Vec16;                          // the 16-byte vector of a grid's value type
template <> struct Vec16<float>  { using type = float4;  static constexpr int n = 4; };
template <> struct Vec16<double> { using type = double2; static constexpr int n = 2; };

// pad[z'][y'][x'] = in[(z' - rz) mod nz][(y' - ry) mod ny][(x' - 4) mod nx], one 16-byte vector per
// thread.  rz = 0 for 2D grids (nz = 1).  A row is a whole number of vectors (nx a multiple of 4 for
// fp32, of 2 for FP64), so every vector wraps as a whole.
template <typename T>
__global__ void __launch_bounds__(256)
stencil_pad_periodic_kernel(const T* __restrict__ in, T* __restrict__ pad, Grid g, int ry, int rz) {
    using V = typename Vec16<T>::type;
    constexpr int n = Vec16<T>::n;
    const int pxv = (g.nx + 2 * kPadX) / n;
    const int nxv = g.nx / n;
    const int py = g.ny + 2 * ry, pz = g.nz + 2 * rz;
    const int64_t total = (int64_t)pxv * py * pz;          // vectors of the padded grid
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const V* src = reinterpret_cast<const V*>(in);
    V* dst = reinterpret_cast<V*>(pad);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int xv = (int)(i % pxv);
        const int64_t row = i / pxv;
        const int yp = (int)(row % py), zp = (int)(row / py);
        int y = (yp - ry) % g.ny; if (y < 0) y += g.ny;
        int z = (zp - rz) % g.nz; if (z < 0) z += g.nz;
        int sv = (xv - kPadX / n) % nxv; if (sv < 0) sv += nxv;
        dst[i] = src[((int64_t)z * g.ny + y) * nxv + sv];
    }
}

// Iterated periodic sweeps stay in the padded layout: a sweep over the whole padded grid
// (as if it were a zero-boundary grid) leaves correct values in the interior and rubbish in
// the halo cells, and this kernel rewrites the halo cells from the interior cells they
// wrap to.  It reads interior cells only and writes halo cells only.  The shell is walked
// in three parts: whole halo planes, halo rows of the interior planes, halo vectors of the
// interior rows.
template <typename T>
__global__ void __launch_bounds__(256)
stencil_refresh_halo_kernel(T* __restrict__ pad, Grid g, int ry, int rz) {
    using V = typename Vec16<T>::type;
    constexpr int n = Vec16<T>::n;
    constexpr int hx = kPadX / n;                          // halo vectors per side of a row
    const int pxv = (g.nx + 2 * kPadX) / n;
    const int nxv = g.nx / n;
    const int py = g.ny + 2 * ry;
    const int64_t part1 = (int64_t)2 * rz * py * pxv;
    const int64_t part2 = (int64_t)g.nz * 2 * ry * pxv;
    const int64_t part3 = (int64_t)g.nz * g.ny * 2 * hx;
    const int64_t total = part1 + part2 + part3;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    V* cells = reinterpret_cast<V*>(pad);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        int zp, yp, xv;                                    // the halo cell, in padded coordinates
        if (i < part1) {
            const int64_t plane = (int64_t)py * pxv;
            const int zi = (int)(i / plane);
            const int r = (int)(i % plane);
            zp = zi < rz ? zi : g.nz + zi;
            yp = r / pxv;
            xv = r % pxv;
        } else if (i < part1 + part2) {
            const int64_t j = i - part1;
            const int per_z = 2 * ry * pxv;
            const int r = (int)(j % per_z);
            const int yi = r / pxv;
            zp = (int)(j / per_z) + rz;
            yp = yi < ry ? yi : g.ny + yi;
            xv = r % pxv;
        } else {
            const int64_t j = i - part1 - part2;
            const int per_z = g.ny * 2 * hx;
            const int r = (int)(j % per_z);
            const int c = r % (2 * hx);
            zp = (int)(j / per_z) + rz;
            yp = r / (2 * hx) + ry;
            xv = c < hx ? c : nxv + c;
        }
        int z = (zp - rz) % g.nz; if (z < 0) z += g.nz;
        int y = (yp - ry) % g.ny; if (y < 0) y += g.ny;
        int sv = (xv - hx) % nxv; if (sv < 0) sv += nxv;
        cells[((int64_t)zp * py + yp) * pxv + xv] = cells[((int64_t)(z + rz) * py + (y + ry)) * pxv + sv + hx];
    }
}

// Periodic boundary without a padded copy: a zero-boundary sweep already holds, at every
// point, the taps that stay inside the grid.  What is missing are the taps that leave it,
// and only points within R of a face have any.  This kernel walks that shell (whole planes
// near the z faces, whole rows near the y faces of the other planes, the first and last R
// points of the other rows) and adds, to each point, its wrapped taps.  Needs every extent
// of the grid to be at least 2R, so that the three parts are disjoint.
constexpr int kWrapSmemTaps = 128;

template <typename T>
__global__ void __launch_bounds__(256)
stencil_wrap_correction_kernel(const T* __restrict__ in, T* __restrict__ out, Grid g, int R, int rz,
                               const TapT<T>* __restrict__ taps, int ntaps) {
    __shared__ TapT<T> s_taps[kWrapSmemTaps];
    const bool staged = ntaps <= kWrapSmemTaps;
    if (staged)
        for (int t = threadIdx.x; t < ntaps; t += blockDim.x) s_taps[t] = taps[t];
    __syncthreads();
    const int inner_z = g.nz - 2 * rz, inner_y = g.ny - 2 * R;
    const int64_t part1 = (int64_t)2 * rz * g.ny * g.nx;
    const int64_t part2 = (int64_t)inner_z * 2 * R * g.nx;
    const int64_t part3 = (int64_t)inner_z * inner_y * 2 * R;
    const int64_t total = part1 + part2 + part3;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        int z, y, x;
        if (i < part1) {
            const int64_t plane = (int64_t)g.ny * g.nx;
            const int zi = (int)(i / plane);
            const int r = (int)(i % plane);
            z = zi < rz ? zi : g.nz - 2 * rz + zi;
            y = r / g.nx;
            x = r % g.nx;
        } else if (i < part1 + part2) {
            const int64_t j = i - part1;
            const int per_z = 2 * R * g.nx;
            const int r = (int)(j % per_z);
            const int yi = r / g.nx;
            z = (int)(j / per_z) + rz;
            y = yi < R ? yi : g.ny - 2 * R + yi;
            x = r % g.nx;
        } else {
            const int64_t j = i - part1 - part2;
            const int64_t per_z = (int64_t)inner_y * 2 * R;
            const int r = (int)(j % per_z);
            const int c = r % (2 * R);
            z = (int)(j / per_z) + rz;
            y = r / (2 * R) + R;
            x = c < R ? c : g.nx - 2 * R + c;
        }
        T acc = T(0);
        for (int t = 0; t < ntaps; ++t) {
            const TapT<T> tap = staged ? s_taps[t] : taps[t];
            int qz = z + tap.dz, qy = y + tap.dy, qx = x + tap.dx;
            const bool inside = (unsigned)qz < (unsigned)g.nz && (unsigned)qy < (unsigned)g.ny &&
                                (unsigned)qx < (unsigned)g.nx;
            if (inside) continue;                          // the sweep has this tap already
            // every extent is at least 2R >= |offset|: one step brings the index back
            qz = qz < 0 ? qz + g.nz : (qz >= g.nz ? qz - g.nz : qz);
            qy = qy < 0 ? qy + g.ny : (qy >= g.ny ? qy - g.ny : qy);
            qx = qx < 0 ? qx + g.nx : (qx >= g.nx ? qx - g.nx : qx);
            acc = fma_t(tap.w, in[((int64_t)qz * g.ny + qy) * g.nx + qx], acc);
        }
        const int64_t self = ((int64_t)z * g.ny + y) * g.nx + x;
        out[self] += acc;
    }
}

// Rows whose length is not a multiple of 16 bytes (4 floats, 2 doubles): the tiled kernels need a 16-byte row pitch
// (a TMA stride rule, and their 128-bit stores), so such a grid is swept between two grids
// with padded rows.  This kernel copies into and out of that layout (rows of `nx` values from
// one pitch to another); `lanes` (a power of two, at most the CTA size) threads share a row, the CTA's other threads take further rows.
// The tail columns of a padded row are never read as grid cells (the tensor map ends at nx),
// so they are left as they are.
template <typename T>
__global__ void __launch_bounds__(256)
stencil_repitch_rows_kernel(const T* __restrict__ src, T* __restrict__ dst, int64_t rows, int nx,
                            int src_pitch, int dst_pitch, int lanes_log2) {
    const int lanes = 1 << lanes_log2;
    const int lx = threadIdx.x & (lanes - 1);
    const int sub = threadIdx.x >> lanes_log2;
    const int rows_per_cta = blockDim.x >> lanes_log2;
    const int64_t group = (int64_t)gridDim.x * rows_per_cta;       // rows the grid takes per round
    constexpr int kRows = 4;                                       // rows per thread and round: loads in flight
    for (int64_t row = (int64_t)blockIdx.x * rows_per_cta + sub; row < rows; row += kRows * group) {
#pragma unroll 2
        for (int x = lx; x < nx; x += lanes) {
            T v[kRows];
#pragma unroll
            for (int j = 0; j < kRows; ++j) {
                const int64_t r = row + j * group;
                v[j] = r < rows ? src[r * src_pitch + x] : T(0);
            }
#pragma unroll
            for (int j = 0; j < kRows; ++j) {
                const int64_t r = row + j * group;
                if (r < rows) dst[r * dst_pitch + x] = v[j];
            }
        }
    }
}

}  // namespace stencil
