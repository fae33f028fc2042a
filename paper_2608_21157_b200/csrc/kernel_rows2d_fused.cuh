// ROWS2D FUSED kernel: temporal blocking for iterated sweeps of a 2D grid with a zero
// boundary.  One pass advances the field by up to T time steps while reading the input
// once and writing the result once.
//
// Same decomposition as the single-step 2D kernel: one WARP owns a strip of 128 columns and
// a chunk of rows and streams it top to bottom on its own private TMA ring; no CTA-wide
// barrier, and here no shared memory for the intermediate levels either: a row of level l
// is complete, in the registers of the warp that needs it, the moment the row of level l-1
// that closes its window has been folded in.  So every arriving input row runs down a
// cascade: it completes one row of level 1, which completes one row of level 2, ... and the
// row of level T goes to global memory.  Level l lags the input by l*R rows.
//
// Neighbours in x come from shuffles at every level.  The two end lanes of a strip have no
// neighbour lane on one side: at level 0 they read the halo columns of the input batch in
// shared memory; above it the missing neighbour counts as zero, which is wrong for an
// interior strip and spoils (T-1)*R columns per side by level T.  With (T-1)*R <= 4 that
// stays inside the end lanes, whose float4 is never stored: a strip stores its inner 120
// columns and strips overlap by 8.  Where the missing neighbour lies outside the grid, zero
// is the right value.  Cells outside the grid are forced back to zero at every level, and
// every level is an fp32 value, so the result equals T separate sweeps up to summation
// order.  A chunk starts T*R rows above its first output row and ends T*R below its last.
#pragma once
#include "common.cuh"
#include "kernel_rows2d.cuh"
#include "kernel_stream.cuh"
#include "ptx.cuh"

namespace stencil {

constexpr int kFused2DHalo = 4;                         // columns per side of a strip that are not stored
constexpr int kFused2DTile = kStreamTX - 2 * kFused2DHalo;


// x neighbourhood of a row held in registers: the lane's float4 plus R values on either
// side from the neighbour lanes; zero where the warp ends.
template <int R>
__device__ __forceinline__ void gather_regs(const float4& c, int lane, float (&v)[4 + 2 * R]) {
    const float c4[4] = {c.x, c.y, c.z, c.w};
    v[R + 0] = c.x; v[R + 1] = c.y; v[R + 2] = c.z; v[R + 3] = c.w;
#pragma unroll
    for (int t = 0; t < R; ++t) {
        const float l = __shfl_up_sync(0xffffffffu, c4[4 - R + t], 1);
        const float r = __shfl_down_sync(0xffffffffu, c4[t], 1);
        v[t] = lane == 0 ? 0.0f : l;
        v[R + 4 + t] = lane == 31 ? 0.0f : r;
    }
}

// Folds one row of a level (`c`, with its x neighbourhood `v`) into the 2R partial sums of
// the next level, oldest output row first, and returns the row it completes.
template <int R, bool BOX>
__device__ __forceinline__ float4 fold_row(float4 (&A)[2 * R], const Weights2D<R>& wt, const float4& c,
                                           const float (&v)[4 + 2 * R]) {
    constexpr int M = 2 * R + 1;
    float4 done;
    if constexpr (BOX) {
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
        float a[4];
#pragma unroll
        for (int m = 0; m < 4; ++m) a[m] = wt.w[0][0] * v[m];
#pragma unroll
        for (int dx = 1; dx < M; ++dx)
#pragma unroll
            for (int m = 0; m < 4; ++m) a[m] = fmaf(wt.w[0][dx], v[m + dx], a[m]);
        A[2 * R - 1] = make_float4(a[0], a[1], a[2], a[3]);
    } else {
        // star: only the output whose own row this is takes the x taps.  The y taps and the centre tap
        // work on the two halves of the lane's float4 (packed FMAs), the x taps on single lanes.
        done = fma4r(wt.w[2 * R][R], c, A[0]);
        const float4 ctr = fma4r(wt.w[R][R], c, A[R]);
        float acc[4] = {ctr.x, ctr.y, ctr.z, ctr.w};
#pragma unroll
        for (int dx = 0; dx < M; ++dx) {
            if (dx == R) continue;                     // the centre tap is in `ctr` already (v[m + R] is c)
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
    return done;
}

template <int R, bool BOX, int T, int YB, int NW>
__global__ void __launch_bounds__(NW * 32)
stencil_rows2d_fused_kernel(const __grid_constant__ CUtensorMap tmap_in, float* __restrict__ out,
                            const Rows2DFusedGeom g, const __grid_constant__ Weights2D<R> wt,
                            int* __restrict__ status) {
    static_assert((T - 1) * R <= kFused2DHalo, "the spoiled columns must stay inside the end lanes");
    using S = Rows2DShape<YB>;
    constexpr int PX = kStreamPX;
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
    dependency_wait();           // the input is the output of the previous pass

    const int unit = blockIdx.x * NW + warp;
    if (unit >= g.strips * g.nchunks) return;           // warps are independent: no barrier follows
    const int strip = unit % g.strips;
    const int chunk = unit / g.strips;
    const int nlev = g.nlev;
    const int H = nlev * R;                              // rows a chunk reads beyond its output rows, per side
    const int x0 = strip * kFused2DTile - kFused2DHalo;  // first column of the strip's 128 (may be -4)
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
            tma_load_3d(smem_addr(ring + (size_t)b * S::BATCH_FLOATS), &tmap_in, full0 + 8 * b, x0 - 4,
                        ystart + b * YB, 0);
        }
    }

    const int xg = x0 + 4 * lane;
    const bool x_in = xg >= 0 && xg < g.nx;              // nx is a multiple of 4: a float4 is in or out as a whole
    const bool x_store = x_in && lane >= 1 && lane <= 30;
    float* op = out + (size_t)y0 * g.nx + xg;            // next output row of this lane

    float4 A[T][2 * R];                                  // A[l]: partial sums of level l+1, oldest row first
#pragma unroll
    for (int l = 0; l < T; ++l)
#pragma unroll
        for (int j = 0; j < 2 * R; ++j) A[l][j] = make_float4(0.f, 0.f, 0.f, 0.f);

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
#pragma unroll 1
        for (int r = 0; r < YB; ++r) {
            const int i = b * YB + r;                    // input row index inside the chunk
            if (i >= nrows) break;
            const float* rowbase = bp + r * PX;
            const float* rowp = rowbase + 4 + 4 * lane;
            float4 c = *reinterpret_cast<const float4*>(rowp);
            float v[4 + 2 * R];
            gather_row<R>(rowp, rowbase, lane, c, v);
#pragma unroll
            for (int l = 1; l <= T; ++l) {
                if (l <= nlev) {
                    float4 done = fold_row<R, BOX>(A[l - 1], wt, c, v);
                    const int yl = ystart + i - l * R;   // the row of level l that is complete now
                    // the zero boundary holds at every time level
                    if (!(x_in && yl >= 0 && yl < g.ny)) done = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (l == nlev) {
                        if (yl >= y0 && yl < y1) {
                            if (x_store && store_in_grid(op, 4, out, g, status)) *reinterpret_cast<float4*>(op) = done;
                            op += g.nx;
                        }
                    } else {
                        c = done;
                        gather_regs<R>(c, lane, v);
                    }
                }
            }
        }
        // every lane is done with the batch: refill its slot with the batch nstage ahead
        __syncwarp();
        if (lane == 0 && b + nstage < nbatches && b + nstage != g.drop_batch) {
            mbar_arrive_expect_tx(full0 + 8 * s, S::BATCH_BYTES);
            tma_load_3d(smem_addr(ring + (size_t)s * S::BATCH_FLOATS), &tmap_in, full0 + 8 * s, x0 - 4,
                        ystart + (b + nstage) * YB, 0);
            issued = b + nstage + 1;
        }
        if (++s == nstage) { s = 0; ph ^= 1; }
    }
}

}  // namespace stencil
