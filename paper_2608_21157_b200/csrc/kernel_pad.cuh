// Periodic boundary for the tiled kernels: the grid is first copied into a padded grid
// whose halo cells hold the wrapped values (R planes and rows on either side, 4 columns on
// either side so that rows stay 16-byte multiples); the zero-boundary kernels then read
// that copy with shifted TMA coordinates and never leave it.  Costs one extra read and
// write of the grid per sweep, which still beats gathering wrapped taps one by one.
#pragma once
#include "common.cuh"
#include "geom.cuh"
#include "ptx.cuh"

namespace stencil {


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

// Point number i of the shell of depth R (rz along z): first the 2*rz whole planes next to the
// z faces, then the 2R whole rows next to the y faces of the other planes, then the first and
// last R points of the other rows.
__device__ __forceinline__ void shell_point(int64_t i, const Grid& g, int R, int rz, int64_t part1, int64_t part2,
                                            int inner_y, int& z, int& y, int& x) {
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
}

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
        shell_point(i, g, R, rz, part1, part2, inner_y, z, y, x);
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

// Periodic boundary under temporal blocking.  A fused pass of L time steps with a zero boundary
// is right wherever the L-step cone of dependence stays inside the grid: at every point at
// least H = L*R cells from every face.  The sweep is linear and, on the torus, invariant under
// shifts, so L periodic steps equal ONE sweep with the operator's L-fold self-convolution (radius
// H).  This kernel walks the shell of depth H and overwrites each of its points with that
// composite sweep of the pass's input, indices wrapped.  The composite taps are doubles and the
// sum runs in double, rounded once: the shell points skip the rounding to T after every
// intermediate step, a difference far below the rounding error of the steps themselves.
// Needs every extent of the grid to be at least 2H.
// The kernel is bound by integer instructions (decoding the point, wrapping and indexing each
// tap), so the index type I is 32 bits wide where the grid has fewer than 2^31 points, an axis
// is only wrapped for points within H of its faces, and the point decode divides 32-bit numbers.
template <typename T, typename I>
__global__ void __launch_bounds__(256)
stencil_shell_compose_kernel(const T* __restrict__ in, T* __restrict__ out, Grid g, int H, int hz,
                             const TapT<double>* __restrict__ taps, int ntaps) {
    __shared__ TapT<double> s_taps[kWrapSmemTaps];
    __shared__ I s_off[kWrapSmemTaps];
    const bool staged = ntaps <= kWrapSmemTaps;
    const I row = (I)g.nx, plane = (I)g.ny * (I)g.nx;
    if (staged)
        for (int t = threadIdx.x; t < ntaps; t += blockDim.x) {
            s_taps[t] = taps[t];
            s_off[t] = (I)taps[t].dz * plane + (I)taps[t].dy * row + (I)taps[t].dx;
        }
    __syncthreads();
    const int inner_z = g.nz - 2 * hz, inner_y = g.ny - 2 * H;
    const I part1 = (I)2 * hz * plane;
    const I per_z2 = (I)2 * H * row, part2 = (I)inner_z * per_z2;
    const I per_z3 = (I)inner_y * 2 * H, part3 = (I)inner_z * per_z3;
    const I total = part1 + part2 + part3;
    const I stride = (I)gridDim.x * blockDim.x;
    for (I i = (I)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        int z, y, x;
        if (i < part1) {                            // whole planes next to the z faces
            const int zi = (int)(i / plane);
            const I r = i - (I)zi * plane;
            z = zi < hz ? zi : g.nz - 2 * hz + zi;
            y = (int)(r / row);
            x = (int)(r - (I)y * row);
        } else if (i < part1 + part2) {             // whole rows next to the y faces of the other planes
            const I j = i - part1;
            const int zi = (int)(j / per_z2);
            const I r = j - (I)zi * per_z2;
            const int yi = (int)(r / row);
            z = zi + hz;
            y = yi < H ? yi : g.ny - 2 * H + yi;
            x = (int)(r - (I)yi * row);
        } else {                                    // the first and last H points of the other rows
            const I j = i - part1 - part2;
            const int zi = (int)(j / per_z3);
            const int r = (int)(j - (I)zi * per_z3);
            const int yi = r / (2 * H);
            const int c = r - yi * 2 * H;
            z = zi + hz;
            y = yi + H;
            x = c < H ? c : g.nx - 2 * H + c;
        }
        const I self = (I)z * plane + (I)y * row + (I)x;
        // An axis wraps only for points within H of its faces, and then in one direction only: a
        // point near the low face wraps taps with d < -coordinate, one near the high face taps with
        // d >= extent - coordinate.  (Every extent is at least 2H, so a point is near one face at most.)
        const bool zlo = z < hz, zhi = z >= g.nz - hz;
        const bool ylo = y < H, yhi = y >= g.ny - H;
        const bool xlo = x < H, xhi = x >= g.nx - H;
        const I zfix = zlo ? (I)g.nz * plane : -(I)g.nz * plane;
        const I yfix = ylo ? plane : -plane;
        const I xfix = xlo ? row : -row;
        double acc = 0.0;
#pragma unroll 4
        for (int t = 0; t < ntaps; ++t) {
            TapT<double> tap;
            I idx;
            if (staged) { tap = s_taps[t]; idx = self + s_off[t]; }
            else { tap = taps[t]; idx = self + (I)tap.dz * plane + (I)tap.dy * row + (I)tap.dx; }
            if (zlo || zhi) { if (zlo ? z + tap.dz < 0 : z + tap.dz >= g.nz) idx += zfix; }
            if (ylo || yhi) { if (ylo ? y + tap.dy < 0 : y + tap.dy >= g.ny) idx += yfix; }
            if (xlo || xhi) { if (xlo ? x + tap.dx < 0 : x + tap.dx >= g.nx) idx += xfix; }
            acc = fma(tap.w, (double)in[idx], acc);
        }
        out[self] = (T)acc;
    }
}

// The same job split in two for speed (the point-by-point walk above spends some 30 instructions
// per tap on wrapping and indexing, and stays as the fallback for operators with more than
// kShellTaps composite taps).  The sums run in T with the composite weights rounded to T.
//
// Whole rows (the planes next to the z faces, the rows next to the y faces of the other planes):
// one CTA per kShellRowChunk points of a row.  The row's z and y are the CTA's, so the wrapped row every tap reads from is
// resolved once per CTA into shared memory; a point between the row's ends then spends a shared
// load, an add, a global load and an FMA per tap, and only the first and last H points wrap in x.
constexpr int kShellTaps = 160;
constexpr int kShellRowChunk = 512;

template <typename T, typename I>
struct ShellRowTap {
    I base;                // index of the cell the tap reads for x = 0 (dx included)
    T w;
};

// I: int where every index of the grid fits (a tap then costs a shared load, one address and a load and an FMA per
// point), int64_t beyond.
template <typename T, typename I>
__global__ void __launch_bounds__(256)
stencil_shell_rows_kernel(const T* __restrict__ in, T* __restrict__ out, Grid g, int H, int hz,
                          const TapT<double>* __restrict__ taps, int ntaps, int xchunks) {
    __shared__ ShellRowTap<T, I> s_tap[kShellTaps];
    __shared__ int s_dx[kShellTaps];
    const int r = blockIdx.x / xchunks;
    const int xbegin = (int)(blockIdx.x % xchunks) * kShellRowChunk;
    const int xend = min(xbegin + kShellRowChunk, g.nx);
    int z, y;
    if (r < 2 * hz * g.ny) {
        const int zi = r / g.ny;
        z = zi < hz ? zi : g.nz - 2 * hz + zi;
        y = r - zi * g.ny;
    } else {
        const int q = r - 2 * hz * g.ny;
        const int yi = q % (2 * H);
        z = q / (2 * H) + hz;
        y = yi < H ? yi : g.ny - 2 * H + yi;
    }
    for (int t = threadIdx.x; t < ntaps; t += blockDim.x) {
        const TapT<double> tap = taps[t];
        int qz = z + tap.dz, qy = y + tap.dy;
        // every extent is at least 2H >= |offset|: one step brings the index back
        qz = qz < 0 ? qz + g.nz : (qz >= g.nz ? qz - g.nz : qz);
        qy = qy < 0 ? qy + g.ny : (qy >= g.ny ? qy - g.ny : qy);
        s_tap[t].base = (I)(((int64_t)qz * g.ny + qy) * g.nx + tap.dx);
        s_tap[t].w = (T)tap.w;
        s_dx[t] = tap.dx;
    }
    __syncthreads();
    // launched as a programmatic dependent of the pass whose shell it rewrites (and the next pass as
    // a dependent of this kernel): everything above overlaps with the predecessor's tail
    allow_dependents();
    dependency_wait();
    T* orow = out + ((int64_t)z * g.ny + y) * g.nx;
    int x = xbegin + threadIdx.x;
    // two points of the row per trip where both lie between the row's ends: they share the tap's shared load
    for (; x >= H && x + (int)blockDim.x < min(xend, g.nx - H); x += 2 * blockDim.x) {
        const T* px = in + x;
        const T* py = px + blockDim.x;
        T a0 = T(0), a1 = T(0);
#pragma unroll 4
        for (int t = 0; t < ntaps; ++t) {
            const ShellRowTap<T, I> tap = s_tap[t];
            a0 = fma_t(tap.w, px[tap.base], a0);
            a1 = fma_t(tap.w, py[tap.base], a1);
        }
        orow[x] = a0;
        orow[x + blockDim.x] = a1;
    }
    for (; x < xend; x += blockDim.x) {
        T acc = T(0);
        if (x >= H && x < g.nx - H) {
            const T* px = in + x;
#pragma unroll 4
            for (int t = 0; t < ntaps; ++t) acc = fma_t(s_tap[t].w, px[s_tap[t].base], acc);
        } else {
            for (int t = 0; t < ntaps; ++t) {
                const int qx = x + s_dx[t];
                const int fix = qx < 0 ? g.nx : (qx >= g.nx ? -g.nx : 0);
                acc = fma_t(s_tap[t].w, in[s_tap[t].base + x + fix], acc);
            }
        }
        orow[x] = acc;
    }
}

// The first and last H points of all other rows.  Walked point by point, every tap of every
// point costs a 32-byte sector of its own; here a CTA takes a tile of TZ planes x TY rows, first
// gathers the two ends of every row the tile's taps reach into shared memory as one circular
// segment of 4H cells ([nx - 2H, nx) followed by [0, 2H)), and sums from there: the tile's rows lie
// at least H rows and planes inside the grid, so nothing wraps in y or z, and the x wrap is the
// segment's own order.  seg is (TZ + 2hz) x (TY + 2H) x 4H cells of dynamic shared memory.
constexpr int kShellTY = 32;
__host__ __device__ constexpr int shell_tz(int H, int hz) { return hz == 0 ? 1 : (H <= 2 ? 8 : 4); }   // planes per tile

template <typename T>
struct ShellSegTap {
    int off;               // offset of the tap's cell from the output's own cell inside seg
    T w;
};

template <typename T>
__global__ void __launch_bounds__(256)
stencil_shell_xfaces_kernel(const T* __restrict__ in, T* __restrict__ out, Grid g, int H, int hz,
                            const TapT<double>* __restrict__ taps, int ntaps) {
    extern __shared__ __align__(16) unsigned char shell_smem[];
    __shared__ ShellSegTap<T> s_tap[kShellTaps];
    T* seg = reinterpret_cast<T*>(shell_smem);
    const int tz = shell_tz(H, hz);
    const int tiles_y = (g.ny - 2 * H + kShellTY - 1) / kShellTY;
    const int y0 = H + (int)(blockIdx.x % tiles_y) * kShellTY;          // first output row and plane of the tile
    const int z0 = hz + (int)(blockIdx.x / tiles_y) * tz;
    const int sw = 4 * H, sy = kShellTY + 2 * H, sz = tz + 2 * hz;
    for (int t = threadIdx.x; t < ntaps; t += blockDim.x) {
        s_tap[t].off = (taps[t].dz * sy + taps[t].dy) * sw + taps[t].dx;
        s_tap[t].w = (T)taps[t].w;
    }
    const int64_t plane = (int64_t)g.ny * g.nx;
    // one thread per (row of the tile, cell of its segment); consecutive threads read consecutive cells
    const int rows_per_round = blockDim.x / sw, k = threadIdx.x % sw;
    for (int row = threadIdx.x / sw; row < sz * sy && (int)threadIdx.x < rows_per_round * sw; row += rows_per_round) {
        const int lz = row / sy, ly = row - lz * sy;
        const int gz = z0 - hz + lz, gy = y0 - H + ly;
        const int gx = k < 2 * H ? g.nx - 2 * H + k : k - 2 * H;
        seg[row * sw + k] = (gz < g.nz && gy < g.ny) ? in[(int64_t)gz * plane + (int64_t)gy * g.nx + gx] : T(0);
    }
    __syncthreads();
    for (int e = threadIdx.x; e < tz * kShellTY * 2 * H; e += blockDim.x) {
        const int c = e % (2 * H), ly = (e / (2 * H)) % kShellTY, lz = e / (2 * H * kShellTY);
        const int z = z0 + lz, y = y0 + ly;
        if (z >= g.nz - hz || y >= g.ny - H) continue;
        const T* ctr = seg + ((lz + hz) * sy + (ly + H)) * sw + H + c;          // this output's own cell
        T acc = T(0);
#pragma unroll 4
        for (int t = 0; t < ntaps; ++t) acc = fma_t(s_tap[t].w, ctr[s_tap[t].off], acc);
        const int x = c < H ? g.nx - H + c : c - H;                             // the cell at segment position H + c
        out[(int64_t)z * plane + (int64_t)y * g.nx + x] = acc;
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
