// ROWS2D kernel for FP64 grids: the precision of the paper's own case study (2D box
// stencil, radius 3, 49 points).  Same structure as the fp32 row-streaming kernel: one
// warp owns a strip of columns and a chunk of rows and streams it through a private TMA
// ring; partial sums of the 2R+1 output rows an input row reaches sit in registers and
// slide down one slot inside the FMA that updates them.
//
// Differences: a lane owns one double2 (two points), so a strip is 64 columns wide; the
// x neighbourhood of a lane (R values on each side) is read straight from shared
// memory as aligned double2 loads.  The sweep is bound by the FP64 pipe (49 DFMA per
// point at 64 DFMA per clock per SM) about as much as by HBM (16 B per point).
#pragma once
#include "common.cuh"
#include "kernel_rows2d.cuh"
#include "ptx.cuh"

namespace stencil {

constexpr int kStrip64 = 64;                 // columns per warp
constexpr int kPX64 = kStrip64 + 8;          // + 4 doubles of halo on both sides (TMA x stays 16-byte aligned)

template <int R>
struct Weights2D64 {                         // dense, [dy+R][dx+R]
    double w[2 * R + 1][2 * R + 1];
};

template <int YB, int PXV = kPX64>
struct Rows2D64Shape {
    static constexpr int BATCH_DOUBLES = YB * PXV;
    static constexpr int BATCH_BYTES = BATCH_DOUBLES * 8;        // 576 * YB (640 * YB for the wide stars): a multiple of 128 for even YB
};

template <int R, bool BOX, int YB, int NW>
__global__ void __launch_bounds__(NW * 32)
stencil_rows2d_f64_kernel(const __grid_constant__ CUtensorMap tmap_in, double* __restrict__ out,
                          const Rows2DGeom g, const __grid_constant__ Weights2D64<R> wt,
                          int* __restrict__ status) {
    constexpr int PX = StreamHalo64<R>::PX;
    constexpr int HX = StreamHalo64<R>::HX;
    using S = Rows2D64Shape<YB, PX>;
    constexpr int M = 2 * R + 1;
    constexpr int HW = (R + 1) / 2 * 2;          // halo doubles read per side, rounded up to a double2
    constexpr int NV = 2 * HW + 2;               // window of a lane: columns -HW .. 1+HW around its pair
    extern __shared__ __align__(128) unsigned char smem_raw[];
    unsigned char* base = smem_raw + ((128u - (smem_addr(smem_raw) & 127u)) & 127u);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nstage = g.stages;
    double* ring = reinterpret_cast<double*>(base) + (size_t)warp * nstage * S::BATCH_DOUBLES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + (size_t)NW * nstage * S::BATCH_BYTES) + warp * kMaxStages;
    const uint32_t full0 = smem_addr(bars);

    if (lane == 0) {
        for (int s = 0; s < nstage; ++s) mbar_init(full0 + 8 * s, 1);
        fence_barrier_init();
    }
    __syncwarp();
    allow_dependents();
    dependency_wait();           // the input may be the output of the previous launch of an iteration

    const int unit = blockIdx.x * NW + warp;
    if (unit >= g.strips * g.nchunks) return;
    const int strip = unit % g.strips;
    const int chunk = unit / g.strips;
    const int x0 = strip * kStrip64;
    const int y0 = g.y_begin + chunk * g.chunk_y;
    const int y1 = min(y0 + g.chunk_y, g.y_end);
    const int nrows = (y1 - y0) + 2 * R;
    const int nbatches = (nrows + YB - 1) / YB;
    const int ystart = y0 - R;

    int issued = 0;
    if (lane == 0) {
        prefetch_tensormap(&tmap_in);
        const int pre = min(nstage, nbatches);
        issued = pre;
        for (int b = 0; b < pre; ++b) {
            if (b == g.drop_batch) continue;
            mbar_arrive_expect_tx(full0 + 8 * b, S::BATCH_BYTES);
            tma_load_3d(smem_addr(ring + (size_t)b * S::BATCH_DOUBLES), &tmap_in, full0 + 8 * b,
                        x0 - HX + g.in_off_x, ystart + b * YB + g.in_off_y, 0);
        }
    }

    const int xg = x0 + 2 * lane;
    const bool x_in = xg < g.nx;                 // nx is even: the pair is inside or outside as a whole
    double* op = out + (size_t)y0 * g.nx + xg;

    double2 A[2 * R];
#pragma unroll
    for (int j = 0; j < 2 * R; ++j) A[j] = make_double2(0.0, 0.0);

    int s = 0;
    uint32_t ph = 0;
    for (int b = 0; b < nbatches; ++b) {
        if (!mbar_wait_bounded(full0 + 8 * s, ph, g.wait_polls)) {
            atomicExch(status, kStatusTimeout);
            if (lane == 0)
                for (int q = max(b + 1, issued - nstage); q < issued; ++q)
                    mbar_wait_bounded(full0 + 8 * (q % nstage), (q / nstage) & 1, g.wait_polls);
            return;
        }
        const double* bp = ring + (size_t)s * S::BATCH_DOUBLES;
#pragma unroll
        for (int r = 0; r < YB; ++r) {
            const int i = b * YB + r;
            if (i < nrows) {
                // v[HW + m + dx] is the input at column (pair column m) + dx
                const double* wp = bp + r * PX + HX + 2 * lane - HW;
                double v[NV];
#pragma unroll
                for (int t = 0; t < NV / 2; ++t) {
                    const double2 d = *reinterpret_cast<const double2*>(wp + 2 * t);
                    v[2 * t] = d.x;
                    v[2 * t + 1] = d.y;
                }
                const double c[2] = {v[HW], v[HW + 1]};
                double2 done;
                if constexpr (BOX) {
                    double e[2] = {A[0].x, A[0].y};
#pragma unroll
                    for (int dx = 0; dx < M; ++dx)
#pragma unroll
                        for (int m = 0; m < 2; ++m) e[m] = fma(wt.w[2 * R][dx], v[HW - R + m + dx], e[m]);
                    done = make_double2(e[0], e[1]);
#pragma unroll
                    for (int j = 0; j < 2 * R - 1; ++j) {
                        double a[2] = {A[j + 1].x, A[j + 1].y};
#pragma unroll
                        for (int dx = 0; dx < M; ++dx)
#pragma unroll
                            for (int m = 0; m < 2; ++m)
                                a[m] = fma(wt.w[2 * R - 1 - j][dx], v[HW - R + m + dx], a[m]);
                        A[j] = make_double2(a[0], a[1]);
                    }
                    {
                        double a[2];
#pragma unroll
                        for (int m = 0; m < 2; ++m) a[m] = wt.w[0][0] * v[HW - R + m];
#pragma unroll
                        for (int dx = 1; dx < M; ++dx)
#pragma unroll
                            for (int m = 0; m < 2; ++m) a[m] = fma(wt.w[0][dx], v[HW - R + m + dx], a[m]);
                        A[2 * R - 1] = make_double2(a[0], a[1]);
                    }
                } else {
                    done.x = fma(wt.w[2 * R][R], c[0], A[0].x);
                    done.y = fma(wt.w[2 * R][R], c[1], A[0].y);
                    double acc[2] = {A[R].x, A[R].y};
#pragma unroll
                    for (int dx = 0; dx < M; ++dx)
#pragma unroll
                        for (int m = 0; m < 2; ++m) acc[m] = fma(wt.w[R][dx], v[HW - R + m + dx], acc[m]);
#pragma unroll
                    for (int j = 0; j < 2 * R - 1; ++j) {
                        if (j == R - 1) continue;
                        const double wy = wt.w[2 * R - 1 - j][R];
                        A[j].x = fma(wy, c[0], A[j + 1].x);
                        A[j].y = fma(wy, c[1], A[j + 1].y);
                    }
                    A[2 * R - 1] = make_double2(wt.w[0][R] * c[0], wt.w[0][R] * c[1]);
                    A[R - 1] = make_double2(acc[0], acc[1]);
                }
                if (i >= 2 * R) {
                    if (x_in && store_in_grid(op, 2, out, g, status)) *reinterpret_cast<double2*>(op) = done;
                    op += g.nx;
                }
            }
        }
        __syncwarp();
        if (lane == 0 && b + nstage < nbatches && b + nstage != g.drop_batch) {
            mbar_arrive_expect_tx(full0 + 8 * s, S::BATCH_BYTES);
            tma_load_3d(smem_addr(ring + (size_t)s * S::BATCH_DOUBLES), &tmap_in, full0 + 8 * s,
                        x0 - HX + g.in_off_x, ystart + (b + nstage) * YB + g.in_off_y, 0);
            issued = b + nstage + 1;
        }
        if (++s == nstage) { s = 0; ph ^= 1; }
    }
}

}  // namespace stencil
