// ROWS2D FUSED kernel for FP64 grids: temporal blocking for iterated 2D sweeps with a zero
// boundary, the double-precision twin of the fp32 register cascade (kernel_rows2d_fused.cuh).
//
// One warp owns a strip of 64 columns (a double2 per lane) and a chunk of rows; every
// arriving input row completes one row of level 1, which completes one row of level 2, ...
// and the row of level T is stored.  Level 0 takes its x neighbourhood from the input batch
// in shared memory, the levels above it from the neighbour lanes by shuffles (radius <= 2:
// one lane to either side is enough).  The two lanes at either end of a strip are not
// stored: whatever the missing neighbours spoil, (T-1)*R <= 4 columns per side, stays inside
// them; a strip stores its inner 56 columns and strips overlap by 8.  Cells outside the grid
// are forced to zero at every level.
#pragma once
#include "common.cuh"
#include "kernel_rows2d.cuh"
#include "kernel_rows2d_f64.cuh"
#include "kernel_rows2d_fused.cuh"
#include "ptx.cuh"

namespace stencil {

constexpr int kFused2D64Tile = kStrip64 - 2 * kFused2DHalo;      // 56 columns stored per strip

// x neighbourhood of a row held in registers: v[R + m + d] is the value d columns from
// column m of the lane's pair; zero where the warp ends.
template <int R>
__device__ __forceinline__ void gather_regs64(const double2& c, int lane, double (&v)[2 + 2 * R]) {
    static_assert(R <= 2, "one neighbour lane per side");
    v[R] = c.x; v[R + 1] = c.y;
    const double lx = __shfl_up_sync(0xffffffffu, c.x, 1);
    const double ly = __shfl_up_sync(0xffffffffu, c.y, 1);
    const double rx = __shfl_down_sync(0xffffffffu, c.x, 1);
    const double ry = __shfl_down_sync(0xffffffffu, c.y, 1);
    const bool first = lane == 0, last = lane == 31;
    v[R - 1] = first ? 0.0 : ly;
    v[R + 2] = last ? 0.0 : rx;
    if constexpr (R == 2) {
        v[0] = first ? 0.0 : lx;
        v[R + 3] = last ? 0.0 : ry;
    }
}

// Folds one row of a level into the 2R partial sums of the next level, oldest output row
// first, and returns the row it completes.
template <int R, bool BOX>
__device__ __forceinline__ double2 fold_row64(double2 (&A)[2 * R], const Weights2D64<R>& wt, const double2& c,
                                              const double (&v)[2 + 2 * R]) {
    constexpr int M = 2 * R + 1;
    double2 done;
    if constexpr (BOX) {
        double e[2] = {A[0].x, A[0].y};
#pragma unroll
        for (int dx = 0; dx < M; ++dx)
#pragma unroll
            for (int m = 0; m < 2; ++m) e[m] = fma(wt.w[2 * R][dx], v[m + dx], e[m]);
        done = make_double2(e[0], e[1]);
#pragma unroll
        for (int j = 0; j < 2 * R - 1; ++j) {
            double a[2] = {A[j + 1].x, A[j + 1].y};
#pragma unroll
            for (int dx = 0; dx < M; ++dx)
#pragma unroll
                for (int m = 0; m < 2; ++m) a[m] = fma(wt.w[2 * R - 1 - j][dx], v[m + dx], a[m]);
            A[j] = make_double2(a[0], a[1]);
        }
        double a[2];
#pragma unroll
        for (int m = 0; m < 2; ++m) a[m] = wt.w[0][0] * v[m];
#pragma unroll
        for (int dx = 1; dx < M; ++dx)
#pragma unroll
            for (int m = 0; m < 2; ++m) a[m] = fma(wt.w[0][dx], v[m + dx], a[m]);
        A[2 * R - 1] = make_double2(a[0], a[1]);
    } else {
        done.x = fma(wt.w[2 * R][R], c.x, A[0].x);
        done.y = fma(wt.w[2 * R][R], c.y, A[0].y);
        double acc[2] = {A[R].x, A[R].y};
#pragma unroll
        for (int dx = 0; dx < M; ++dx)
#pragma unroll
            for (int m = 0; m < 2; ++m) acc[m] = fma(wt.w[R][dx], v[m + dx], acc[m]);
#pragma unroll
        for (int j = 0; j < 2 * R - 1; ++j) {
            if (j == R - 1) continue;
            const double wy = wt.w[2 * R - 1 - j][R];
            A[j].x = fma(wy, c.x, A[j + 1].x);
            A[j].y = fma(wy, c.y, A[j + 1].y);
        }
        A[2 * R - 1] = make_double2(wt.w[0][R] * c.x, wt.w[0][R] * c.y);
        A[R - 1] = make_double2(acc[0], acc[1]);
    }
    return done;
}

template <int R, bool BOX, int T, int YB, int NW>
__global__ void __launch_bounds__(NW * 32)
stencil_rows2d_fused_f64_kernel(const __grid_constant__ CUtensorMap tmap_in, double* __restrict__ out,
                                const Rows2DFusedGeom g, const __grid_constant__ Weights2D64<R> wt,
                                int* __restrict__ status) {
    static_assert((T - 1) * R <= kFused2DHalo, "the spoiled columns must stay inside the end lanes");
    using S = Rows2D64Shape<YB>;
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
    dependency_wait();           // the input is the output of the previous pass

    const int unit = blockIdx.x * NW + warp;
    if (unit >= g.strips * g.nchunks) return;           // warps are independent: no barrier follows
    const int strip = unit % g.strips;
    const int chunk = unit / g.strips;
    const int nlev = g.nlev;
    const int H = nlev * R;                              // rows a chunk reads beyond its output rows, per side
    const int x0 = strip * kFused2D64Tile - kFused2DHalo;   // first column of the strip's 64 (may be -4)
    const int y0 = chunk * g.chunk_y;
    const int y1 = min(y0 + g.chunk_y, g.ny);
    const int nrows = (y1 - y0) + 2 * H;                 // input rows y0-H .. y1-1+H
    const int nbatches = (nrows + YB - 1) / YB;
    const int ystart = y0 - H;

    int issued = 0;                                      // batches requested so far (lane 0 only)
    if (lane == 0) {
        prefetch_tensormap(&tmap_in);
        const int pre = min(nstage, nbatches);
        issued = pre;
        for (int b = 0; b < pre; ++b) {
            if (b == g.drop_batch) continue;
            mbar_arrive_expect_tx(full0 + 8 * b, S::BATCH_BYTES);
            tma_load_3d(smem_addr(ring + (size_t)b * S::BATCH_DOUBLES), &tmap_in, full0 + 8 * b, x0 - 4,
                        ystart + b * YB, 0);
        }
    }

    const int xg = x0 + 2 * lane;
    const bool x_in = xg >= 0 && xg < g.nx;              // nx is even: a pair is in or out as a whole
    const bool x_store = x_in && lane >= 2 && lane <= 29;
    double* op = out + (size_t)y0 * g.nx + xg;           // next output row of this lane

    double2 A[T][2 * R];                                 // A[l]: partial sums of level l+1, oldest row first
#pragma unroll
    for (int l = 0; l < T; ++l)
#pragma unroll
        for (int j = 0; j < 2 * R; ++j) A[l][j] = make_double2(0.0, 0.0);

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
        const double* bp = ring + (size_t)s * S::BATCH_DOUBLES;
#pragma unroll 1
        for (int r = 0; r < YB; ++r) {
            const int i = b * YB + r;                    // input row index inside the chunk
            if (i >= nrows) break;
            // level 0: the lane's pair and one double2 to either side, straight from the batch
            const double* wp = bp + r * kPX64 + 4 + 2 * lane;
            const double2 lft = *reinterpret_cast<const double2*>(wp - 2);
            double2 c = *reinterpret_cast<const double2*>(wp);
            const double2 rgt = *reinterpret_cast<const double2*>(wp + 2);
            double v[2 + 2 * R];
            v[R] = c.x; v[R + 1] = c.y;
            v[R - 1] = lft.y; v[R + 2] = rgt.x;
            if constexpr (R == 2) { v[0] = lft.x; v[R + 3] = rgt.y; }
#pragma unroll
            for (int l = 1; l <= T; ++l) {
                if (l <= nlev) {
                    double2 done = fold_row64<R, BOX>(A[l - 1], wt, c, v);
                    const int yl = ystart + i - l * R;   // the row of level l that is complete now
                    // the zero boundary holds at every time level
                    if (!(x_in && yl >= 0 && yl < g.ny)) done = make_double2(0.0, 0.0);
                    if (l == nlev) {
                        if (yl >= y0 && yl < y1) {
                            if (x_store && store_in_grid(op, 2, out, g, status)) *reinterpret_cast<double2*>(op) = done;
                            op += g.nx;
                        }
                    } else {
                        c = done;
                        gather_regs64<R>(c, lane, v);
                    }
                }
            }
        }
        // every lane is done with the batch: refill its slot with the batch nstage ahead
        __syncwarp();
        if (lane == 0 && b + nstage < nbatches && b + nstage != g.drop_batch) {
            mbar_arrive_expect_tx(full0 + 8 * s, S::BATCH_BYTES);
            tma_load_3d(smem_addr(ring + (size_t)s * S::BATCH_DOUBLES), &tmap_in, full0 + 8 * s, x0 - 4,
                        ystart + (b + nstage) * YB, 0);
            issued = b + nstage + 1;
        }
        if (++s == nstage) { s = 0; ph ^= 1; }
    }
}

}  // namespace stencil
