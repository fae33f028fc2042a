// ROWS2D kernel: single sweep of a 2D grid with a zero boundary (the shape of the
// paper's case study: a box stencil of radius R on a large 2D grid).
//
// The grid is cut into strips of 128 columns and chunks of rows; one WARP owns one
// (strip, chunk) and streams it top to bottom on its own: no CTA-wide barrier exists.
// Lane 0 of the warp drives a private TMA ring (batches of YB rows, 4-float halo on both
// sides, zero fill outside the grid).  Every lane owns one float4 of the strip.  An
// arriving row is a tap of the 2R+1 output rows it reaches; their partial sums sit in
// registers, oldest first, and slide down one slot inside the FMAs that update them.
// The oldest is complete after the update and goes to global memory as one 128-bit
// store per lane (512 contiguous bytes per warp).
//
// box  : (2R+1)^2 FMAs per point;  star: 4R+1.
#pragma once
#include "common.cuh"
#include "kernel_stream.cuh"
#include "ptx.cuh"

namespace stencil {

template <int R>
struct Weights2D {              // dense, [dy+R][dx+R]; a star has zeros off the axes
    float w[2 * R + 1][2 * R + 1];
};


template <int YB, int PXV = kStreamPX>     // PXV: row pitch of a batch (the strip plus its halo columns)
struct Rows2DShape {
    static constexpr int BATCH_FLOATS = YB * PXV;
    static constexpr int BATCH_BYTES = BATCH_FLOATS * 4;          // multiple of 128 for even YB
    static size_t smem_bytes(int nwarps, int stages) {
        return (size_t)nwarps * stages * BATCH_BYTES + 128 + (size_t)nwarps * kMaxStages * 8;
    }
};

template <int R, bool BOX, int YB, int NW>
__global__ void __launch_bounds__(NW * 32)
stencil_rows2d_kernel(const __grid_constant__ CUtensorMap tmap_in, float* __restrict__ out,
                      const Rows2DGeom g, const __grid_constant__ Weights2D<R> wt,
                      int* __restrict__ status) {
    constexpr int PX = StreamHalo<R>::PX;          // 4 halo columns per side up to radius 4, 8 beyond
    constexpr int HX = StreamHalo<R>::HX;
    using S = Rows2DShape<YB, PX>;
    constexpr int M = 2 * R + 1;
    constexpr int kRowCopies = (BOX && R >= 3) ? 1 : YB;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    unsigned char* base = smem_raw + ((128u - (smem_addr(smem_raw) & 127u)) & 127u);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nstage = g.stages;
    float* ring = reinterpret_cast<float*>(base) + (size_t)warp * nstage * S::BATCH_FLOATS;
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
    if (unit >= g.strips * g.nchunks) return;           // warps are independent: no barrier follows
    const int strip = unit % g.strips;                   // neighbouring strips run side by side (shared halo in L2)
    const int chunk = unit / g.strips;
    const int x0 = strip * kStreamTX;
    const int y0 = g.y_begin + chunk * g.chunk_y;
    const int y1 = min(y0 + g.chunk_y, g.y_end);
    const int nrows = (y1 - y0) + 2 * R;                 // input rows y0-R .. y1-1+R
    const int nbatches = (nrows + YB - 1) / YB;
    const int ystart = y0 - R;

    int issued = 0;                                      // batches requested so far (lane 0 only)
    if (lane == 0) {
        prefetch_tensormap(&tmap_in);
        const int pre = min(nstage, nbatches);
        issued = pre;
        for (int b = 0; b < pre; ++b) {
            if (b == g.drop_batch) continue;
            mbar_arrive_expect_tx(full0 + 8 * b, S::BATCH_BYTES);
            tma_load_3d(smem_addr(ring + (size_t)b * S::BATCH_FLOATS), &tmap_in, full0 + 8 * b,
                        x0 - HX + g.in_off_x, ystart + b * YB + g.in_off_y, 0);
        }
    }

    const int xg = x0 + 4 * lane;
    const bool x_in = xg < g.nx;
    float* op = out + (size_t)y0 * g.nx + xg;            // next output row of this lane

    float4 A[2 * R];                                     // partial sums, oldest output row first
#pragma unroll
    for (int j = 0; j < 2 * R; ++j) A[j] = make_float4(0.f, 0.f, 0.f, 0.f);

    int s = 0;
    uint32_t ph = 0;
    for (int b = 0; b < nbatches; ++b) {
        if (!mbar_wait_bounded(full0 + 8 * s, ph, g.wait_polls)) {
            atomicExch(status, kStatusTimeout);
            // let copies that may still be in flight land before the warp leaves
            if (lane == 0)
                for (int q = max(b + 1, issued - nstage); q < issued; ++q)
                    mbar_wait_bounded(full0 + 8 * (q % nstage), (q / nstage) & 1, g.wait_polls);
            return;
        }
        const float* bp = ring + (size_t)s * S::BATCH_FLOATS;
        // the big boxes keep one copy of the row body: YB copies of (2R+1)^2 FMAs per point would
        // not fit the instruction cache
#pragma unroll(kRowCopies)
        for (int r = 0; r < YB; ++r) {
            const int i = b * YB + r;                    // input row index inside the chunk
            if (i < nrows) {
                const float* rowbase = bp + r * PX;
                const float* rowp = rowbase + HX + 4 * lane;
                const float4 c = *reinterpret_cast<const float4*>(rowp);
                float v[4 + 2 * R];
                gather_row<R>(rowp, rowbase, lane, c, v);
                float4 done;
                if constexpr (BOX) {
                    // this row is tap dy = +R of the oldest output (complete after this), dy = R-1-j
                    // of the output moving into slot j, dy = -R of the one that starts now
                    float e[4] = {A[0].x, A[0].y, A[0].z, A[0].w};
#pragma unroll
                    for (int dx = 0; dx < M; ++dx)
#pragma unroll
                        for (int m = 0; m < 4; ++m) e[m] = fmaf(wt.w[2 * R][dx], v[m + dx], e[m]);
                    done = make_float4(e[0], e[1], e[2], e[3]);
#pragma unroll
                    for (int j = 0; j < 2 * R - 1; ++j) {
                        float a[4] = {A[j + 1].x, A[j + 1].y, A[j + 1].z, A[j + 1].w};
#pragma unroll
                        for (int dx = 0; dx < M; ++dx)
#pragma unroll
                            for (int m = 0; m < 4; ++m) a[m] = fmaf(wt.w[2 * R - 1 - j][dx], v[m + dx], a[m]);
                        A[j] = make_float4(a[0], a[1], a[2], a[3]);
                    }
                    {
                        float a[4];
#pragma unroll
                        for (int m = 0; m < 4; ++m) a[m] = wt.w[0][0] * v[m];
#pragma unroll
                        for (int dx = 1; dx < M; ++dx)
#pragma unroll
                            for (int m = 0; m < 4; ++m) a[m] = fmaf(wt.w[0][dx], v[m + dx], a[m]);
                        A[2 * R - 1] = make_float4(a[0], a[1], a[2], a[3]);
                    }
                } else {
                    // star: only the output whose own row this is takes the x taps.  The y taps and the
                    // centre tap work on the two halves of the lane's float4 (packed FMAs).
                    done = fma4r(wt.w[2 * R][R], c, A[0]);
                    const float4 ctr = fma4r(wt.w[R][R], c, A[R]);
                    float acc[4] = {ctr.x, ctr.y, ctr.z, ctr.w};
#pragma unroll
                    for (int dx = 0; dx < M; ++dx) {
                        if (dx == R) continue;         // the centre tap is in `ctr` already (v[m + R] is c)
#pragma unroll
                        for (int m = 0; m < 4; ++m) acc[m] = fmaf(wt.w[R][dx], v[m + dx], acc[m]);
                    }
#pragma unroll
                    for (int j = 0; j < 2 * R - 1; ++j) {
                        if (j == R - 1) continue;
                        A[j] = fma4r(wt.w[2 * R - 1 - j][R], c, A[j + 1]);
                    }
                    A[2 * R - 1] = mul4(wt.w[0][R], c);
                    A[R - 1] = make_float4(acc[0], acc[1], acc[2], acc[3]);
                }
                if (i >= 2 * R) {
                    if (x_in && store_in_grid(op, 4, out, g, status)) *reinterpret_cast<float4*>(op) = done;
                    op += g.nx;
                }
            }
        }
        // every lane is done with the batch: refill its slot with the batch nstage ahead
        __syncwarp();
        if (lane == 0 && b + nstage < nbatches && b + nstage != g.drop_batch) {
            mbar_arrive_expect_tx(full0 + 8 * s, S::BATCH_BYTES);
            tma_load_3d(smem_addr(ring + (size_t)s * S::BATCH_FLOATS), &tmap_in, full0 + 8 * s,
                        x0 - HX + g.in_off_x, ystart + (b + nstage) * YB + g.in_off_y, 0);
            issued = b + nstage + 1;
        }
        if (++s == nstage) { s = 0; ph ^= 1; }
    }
}

}  // namespace stencil
