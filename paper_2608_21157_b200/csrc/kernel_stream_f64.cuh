// STREAM kernel for FP64 grids: 3D sweep with a zero boundary, the double-precision twin
// of the fp32 plane-streaming kernel (same CTA layout, same TMA ring with a producer warp,
// same in-place register accumulators along z).
//
// Differences: a lane owns one double2 (two points), so a tile is 64 columns wide; the x
// neighbourhood of a lane is read from shared memory as aligned double2 loads instead of
// being exchanged by shuffles.  At 16 B per point the sweep is bound by HBM for the stars
// (25 DFMA per point at radius 4) and the 27-point box, since the FP64 pipe
// sustains 64 DFMA per clock per SM; the 125-point box is bound by that pipe.
#pragma once
#include "common.cuh"
#include "kernel_stream.cuh"
#include "ptx.cuh"

namespace stencil {

constexpr int kStream64TX = 64;                  // tile width in points
constexpr int kStream64PX = kStream64TX + 8;     // + 4 doubles of halo on both sides (radius <= 4; see StreamHalo64)

template <int R>
struct StarWeights64 {
    double c;
    double x[2 * R + 1], y[2 * R + 1], z[2 * R + 1];   // entry [R] unused
};

template <int R>
struct BoxWeights64 {
    double w[2 * R + 1][2 * R + 1][2 * R + 1];         // [dz+R][dy+R][dx+R]
};

template <int R, int K, int NW>
struct Stream64Shape {
    static constexpr int TY = NW * K;
    static constexpr int ROWS = TY + 2 * R;             // even, so a plane is a multiple of 128 bytes
    static constexpr int PLANE_DOUBLES = ROWS * StreamHalo64<R>::PX;   // 576 or 640 bytes per row

    static constexpr int PLANE_BYTES = PLANE_DOUBLES * 8;
    static constexpr int THREADS = (NW + 1) * 32;
    // periodic sweeps (WRAP): beside every plane the cells its halo would hold on a torus, as in the
    // fp32 kernel: 4 columns x ROWS rows beyond either end of the rows, R rows x PX columns above and below
    static constexpr int XS_BYTES = (ROWS * 32 + 127) / 128 * 128;
    static constexpr int YS_BYTES = (R * StreamHalo64<R>::PX * 8 + 127) / 128 * 128;
    static constexpr int CS_BYTES = (R * 32 + 127) / 128 * 128;      // boxes: a corner of the halo, 4 columns x R rows
    static constexpr int STAGE_BYTES = 2 * XS_BYTES + 2 * YS_BYTES + 4 * CS_BYTES;
};

__device__ __forceinline__ double d2get(const double2& v, int m) { return m == 0 ? v.x : v.y; }

// WRAP: the sweep of a periodic grid, as in the fp32 kernel (stars of radius <= 4, rows a whole number
// of 64-column tiles): z wraps in the plane coordinate of the TMA loads; a tile at an x face reads the
// halo columns of its centre rows from blocks loaded beside the plane; a tile at a y face copies its
// own columns of the halo rows over the zeros TMA filled in.
template <int R, bool BOX, int K, int NW, bool WRAP>
__device__ __forceinline__ void
stream_f64_body(const CUtensorMap& tmap_in, const CUtensorMap& tmap_xs, const CUtensorMap& tmap_ys,
                const CUtensorMap& tmap_cs, double* __restrict__ out, const StreamGeom& g, const StarWeights64<R>& sw,
                const BoxWeights64<BOX ? R : 0>& bw, int* __restrict__ status) {
    static_assert(!WRAP || R <= 4, "WRAP: 4-column halos");
    using S = Stream64Shape<R, K, NW>;
    constexpr int SLOT_DOUBLES = (S::PLANE_BYTES + (WRAP ? S::STAGE_BYTES : 0)) / 8;
    constexpr int PX = StreamHalo64<R>::PX;
    constexpr int HX = StreamHalo64<R>::HX;
    constexpr int HW = (R + 1) / 2 * 2;              // halo doubles read per side (a whole double2)
    constexpr int NV = 2 * HW + 2;                   // x window of a lane
    extern __shared__ __align__(128) unsigned char smem_raw[];
    unsigned char* base = smem_raw + ((128u - (smem_addr(smem_raw) & 127u)) & 127u);
    double* ring = reinterpret_cast<double*>(base);
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + (size_t)g.stages * SLOT_DOUBLES * 8);
    const uint32_t full0 = smem_addr(bars);
    const uint32_t empty0 = smem_addr(bars + kMaxStages);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int nstage = g.stages;

    if (threadIdx.x == 0) {
        for (int s = 0; s < nstage; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, NW);
        }
        fence_barrier_init();
    }
    __syncthreads();
    allow_dependents();
    dependency_wait();

    const int bid = blockIdx.x;
    const int tile_x = bid % g.tiles_x;
    const int tile_y = (bid / g.tiles_x) % g.tiles_y;
    const int chunk = bid / (g.tiles_x * g.tiles_y);
    const int x0 = tile_x * kStream64TX;
    const int y0 = tile_y * S::TY;
    const int z0 = g.z_begin + chunk * g.chunk_z;
    const int z1 = min(z0 + g.chunk_z, g.z_end);
    const int nplanes = (z1 - z0) + 2 * R;
    const int pstart = z0 - R;
    // WRAP: which faces the tile's halo reaches across, and the plane row where the halo below the grid begins
    const bool edge_l = WRAP && tile_x == 0, edge_r = WRAP && tile_x == g.tiles_x - 1;
    const bool edge_t = WRAP && tile_y == 0, edge_b = WRAP && y0 + S::TY + R > g.ny;
    const int row_b = R + g.ny - y0;

    if (warp == NW) {
        if (lane == 0) {
            prefetch_tensormap(&tmap_in);
            bool ok = true;
            int issued = 0;
            int s = 0;
            uint32_t ph = 1;
            for (int i = 0; i < nplanes; ++i) {
                if (i >= nstage && !mbar_wait_bounded(empty0 + 8 * s, ph, g.wait_polls)) { ok = false; break; }
                if (i == g.drop_plane) {
                    // test hook: this plane is never requested, so the consumers' wait for it runs out
                } else if constexpr (WRAP) {
                    int zc = pstart + i;                           // nz >= 2R: one step brings it back
                    zc = zc < 0 ? zc + g.nz : (zc >= g.nz ? zc - g.nz : zc);
                    const uint32_t bar = full0 + 8 * s;
                    double* slot = ring + (size_t)s * SLOT_DOUBLES;
                    const int ncorner = BOX ? ((int)edge_l + (int)edge_r) * ((int)edge_t + (int)edge_b) : 0;
                    mbar_arrive_expect_tx(bar, S::PLANE_BYTES + ((int)edge_l + (int)edge_r) * S::ROWS * 32 +
                                                   ((int)edge_t + (int)edge_b) * R * PX * 8 + ncorner * R * 32);
                    tma_load_3d(smem_addr(slot), &tmap_in, bar, x0 - HX, y0 - R, zc);
                    double* stage = slot + S::PLANE_DOUBLES;
                    if (edge_l) tma_load_3d(smem_addr(stage), &tmap_xs, bar, g.nx - 4, y0 - R, zc);
                    if (edge_r) tma_load_3d(smem_addr(stage + S::XS_BYTES / 8), &tmap_xs, bar, 0, y0 - R, zc);
                    if (edge_t) tma_load_3d(smem_addr(stage + 2 * S::XS_BYTES / 8), &tmap_ys, bar, x0 - HX, g.ny - R, zc);
                    if (edge_b)
                        tma_load_3d(smem_addr(stage + (2 * S::XS_BYTES + S::YS_BYTES) / 8), &tmap_ys, bar, x0 - HX, 0, zc);
                    if constexpr (BOX) {                           // corners: (left, right) x (top, bottom)
                        double* cs = stage + (2 * S::XS_BYTES + 2 * S::YS_BYTES) / 8;
                        if (edge_l && edge_t) tma_load_3d(smem_addr(cs), &tmap_cs, bar, g.nx - 4, g.ny - R, zc);
                        if (edge_r && edge_t) tma_load_3d(smem_addr(cs + S::CS_BYTES / 8), &tmap_cs, bar, 0, g.ny - R, zc);
                        if (edge_l && edge_b) tma_load_3d(smem_addr(cs + 2 * S::CS_BYTES / 8), &tmap_cs, bar, g.nx - 4, 0, zc);
                        if (edge_r && edge_b) tma_load_3d(smem_addr(cs + 3 * S::CS_BYTES / 8), &tmap_cs, bar, 0, 0, zc);
                    }
                } else {
                    mbar_arrive_expect_tx(full0 + 8 * s, S::PLANE_BYTES);
                    tma_load_3d(smem_addr(ring + (size_t)s * S::PLANE_DOUBLES), &tmap_in, full0 + 8 * s,
                                x0 - HX + g.in_off_x, y0 - R + g.in_off_y, pstart + i + g.in_off_z);
                }
                issued = i + 1;
                if (++s == nstage) { s = 0; ph ^= 1; }
            }
            if (!ok) {
                atomicExch(status, kStatusTimeout);
                for (int i = max(0, issued - nstage); i < issued; ++i)
                    mbar_wait_bounded(full0 + 8 * (i % nstage), (i / nstage) & 1, g.wait_polls);
            }
        }
        return;
    }

    const int row0 = warp * K;
    const int xg = x0 + 2 * lane;
    const bool x_in = xg < g.nx;                     // nx is even
    const size_t plane_stride = (size_t)g.ny * g.nx;
    bool row_ok[K];
#pragma unroll
    for (int k = 0; k < K; ++k) row_ok[k] = x_in && (y0 + row0 + k) < g.ny;
    double* op = out + (size_t)z0 * plane_stride + (size_t)(y0 + row0) * g.nx + xg;
    int s = 0;
    uint32_t ph = 0;

    if constexpr (!BOX) {
        double2 A[K][2 * R];                         // partial sums, oldest incomplete output plane first
#pragma unroll
        for (int k = 0; k < K; ++k)
#pragma unroll
            for (int j = 0; j < 2 * R; ++j) A[k][j] = make_double2(0.0, 0.0);

        for (int i = 0; i < nplanes; ++i) {
            if (!mbar_wait_bounded(full0 + 8 * s, ph, g.wait_polls)) {
                atomicExch(status, kStatusTimeout);
                return;
            }
            const double* pl = ring + (size_t)s * SLOT_DOUBLES;
            if constexpr (WRAP) {
                if (edge_t || edge_b) {                                // uniform over the CTA
                    double* plw = ring + (size_t)s * SLOT_DOUBLES;
                    const double* stage = pl + S::PLANE_DOUBLES;
#pragma unroll
                    for (int rr = 0; rr < R; ++rr) {
                        // the halo rows inside this warp's window of rows, the lane's own columns
                        if (edge_t && rr >= row0 && rr < row0 + K + 2 * R)
                            *reinterpret_cast<double2*>(plw + rr * PX + HX + 2 * lane) =
                                *reinterpret_cast<const double2*>(stage + 2 * S::XS_BYTES / 8 + rr * PX + HX + 2 * lane);
                        const int rb = row_b + rr;
                        if (edge_b && rb < S::ROWS && rb >= row0 && rb < row0 + K + 2 * R)
                            *reinterpret_cast<double2*>(plw + rb * PX + HX + 2 * lane) =
                                *reinterpret_cast<const double2*>(stage + (2 * S::XS_BYTES + S::YS_BYTES) / 8 + rr * PX +
                                                                  HX + 2 * lane);
                    }
                    // later TMA copies into this slot must not overtake these stores
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                }
            }
            const double* colp = pl + row0 * PX + HX + 2 * lane;
            double acc[K][2];
#pragma unroll
            for (int k = 0; k < K; ++k) { acc[k][0] = A[k][R].x; acc[k][1] = A[k][R].y; }
            double2 done[K];
#pragma unroll
            for (int kk = 0; kk < K + 2 * R; ++kk) {
                const double2 c = *reinterpret_cast<const double2*>(colp + kk * PX);
#pragma unroll
                for (int k = 0; k < K; ++k) {
                    const int d = kk - k - R;
                    if (d != 0 && d >= -R && d <= R) {
                        acc[k][0] = fma(sw.y[d + R], c.x, acc[k][0]);
                        acc[k][1] = fma(sw.y[d + R], c.y, acc[k][1]);
                    }
                }
                if (kk >= R && kk < K + R) {
                    const int k = kk - R;
                    double v[NV];                     // v[HW + m + dx]: the input at column m + dx of the pair
#pragma unroll
                    for (int t = 0; t < NV / 2; ++t) {
                        double2 dd;
                        if constexpr (WRAP) {
                            // the double2 that holds tile columns c, c+1.  The windows of the first (last) HW/2
                            // lanes reach into the row's halo, c < 0 (c >= 64): at an x face that halo is the
                            // staged block (4 columns per row), else the plane's own halo columns.
                            const int c = 2 * lane - HW + 2 * t;
                            int o = (row0 + kk) * PX + HX + c;
                            const int o_xs = S::PLANE_DOUBLES + (row0 + kk) * 4;
                            if (2 * t < HW && edge_l && c < 0) o = o_xs + 4 + c;
                            if (2 * t >= HW + 2 && edge_r && c >= kStream64TX) o = o_xs + S::XS_BYTES / 8 + c - kStream64TX;
                            dd = *reinterpret_cast<const double2*>(pl + o);
                        } else {
                            dd = *reinterpret_cast<const double2*>(colp + kk * PX - HW + 2 * t);
                        }
                        v[2 * t] = dd.x;
                        v[2 * t + 1] = dd.y;
                    }
#pragma unroll
                    for (int m = 0; m < 2; ++m) {
                        double a = fma(sw.c, v[HW + m], acc[k][m]);
#pragma unroll
                        for (int d = 1; d <= R; ++d) {
                            a = fma(sw.x[R - d], v[HW + m - d], a);
                            a = fma(sw.x[R + d], v[HW + m + d], a);
                        }
                        acc[k][m] = a;
                    }
                    done[k].x = fma(sw.z[2 * R], c.x, A[k][0].x);
                    done[k].y = fma(sw.z[2 * R], c.y, A[k][0].y);
#pragma unroll
                    for (int j = 0; j < 2 * R - 1; ++j) {
                        if (j == R - 1) continue;
                        const double wz = sw.z[2 * R - 1 - j];
                        A[k][j].x = fma(wz, c.x, A[k][j + 1].x);
                        A[k][j].y = fma(wz, c.y, A[k][j + 1].y);
                    }
                    A[k][2 * R - 1] = make_double2(sw.z[0] * c.x, sw.z[0] * c.y);
                }
            }
#pragma unroll
            for (int k = 0; k < K; ++k) A[k][R - 1] = make_double2(acc[k][0], acc[k][1]);
            __syncwarp();
            mbar_arrive_if(lane == 0, empty0 + 8 * s);
            if (++s == nstage) { s = 0; ph ^= 1; }

            if (i >= 2 * R) {
#pragma unroll
                for (int k = 0; k < K; ++k)
                    if (row_ok[k] && store_in_grid(op + (size_t)k * g.nx, 2, out, g, status))
                        *reinterpret_cast<double2*>(op + (size_t)k * g.nx) = done[k];
                op += plane_stride;
            }
        }
    } else {
        constexpr int M = 2 * R + 1;
        double2 T[K][M];                              // accumulator of output plane z lives in slot z mod M
#pragma unroll
        for (int k = 0; k < K; ++k)
#pragma unroll
            for (int d = 0; d < M; ++d) T[k][d] = make_double2(0.0, 0.0);

        for (int i0 = 0; i0 < nplanes; i0 += M) {
            const bool ok = static_for<M>([&](auto uc) -> bool {
                constexpr int u = decltype(uc)::value;
                const int i = i0 + u;
                if (i >= nplanes) return true;
                if (!mbar_wait_bounded(full0 + 8 * s, ph, g.wait_polls)) return false;
                const double* pl = ring + (size_t)s * SLOT_DOUBLES;
                if constexpr (WRAP) {
                    if (edge_t || edge_b) {                            // uniform over the CTA
                        // the halo rows inside this warp's window of rows: the lane's own columns, the rows' own
                        // halo columns (first and last two lanes) and, at an x face, the corner cells, which go
                        // into the halo rows of the column blocks
                        double* plw = ring + (size_t)s * SLOT_DOUBLES;
                        double* stw = plw + S::PLANE_DOUBLES;
                        const double* ys = stw + 2 * S::XS_BYTES / 8;
                        const double* cs = ys + 2 * S::YS_BYTES / 8;
#pragma unroll
                        for (int rr = 0; rr < R; ++rr) {
#pragma unroll
                            for (int side = 0; side < 2; ++side) {     // 0: rows above the grid, 1: rows below it
                                const int r = side == 0 ? rr : row_b + rr;
                                const bool mine = (side == 0 ? edge_t : edge_b) && r < S::ROWS && r >= row0 &&
                                                  r < row0 + K + 2 * R;
                                if (!mine) continue;
                                const double* yrow = ys + side * (S::YS_BYTES / 8) + rr * PX;
                                *reinterpret_cast<double2*>(plw + r * PX + HX + 2 * lane) =
                                    *reinterpret_cast<const double2*>(yrow + HX + 2 * lane);
                                if (lane < 2)                          // the 4 halo columns left of the tile
                                    *reinterpret_cast<double2*>(plw + r * PX + 2 * lane) =
                                        *reinterpret_cast<const double2*>(yrow + 2 * lane);
                                if (lane >= 30)                        // ... and right of it
                                    *reinterpret_cast<double2*>(plw + r * PX + HX + kStream64TX + 2 * (lane - 30)) =
                                        *reinterpret_cast<const double2*>(yrow + HX + kStream64TX + 2 * (lane - 30));
                                if (edge_l && (lane == 2 || lane == 3))
                                    *reinterpret_cast<double2*>(stw + r * 4 + 2 * (lane - 2)) =
                                        *reinterpret_cast<const double2*>(cs + (2 * side) * (S::CS_BYTES / 8) + rr * 4 +
                                                                          2 * (lane - 2));
                                if (edge_r && (lane == 4 || lane == 5))
                                    *reinterpret_cast<double2*>(stw + S::XS_BYTES / 8 + r * 4 + 2 * (lane - 4)) =
                                        *reinterpret_cast<const double2*>(cs + (2 * side + 1) * (S::CS_BYTES / 8) + rr * 4 +
                                                                          2 * (lane - 4));
                            }
                        }
                        // later TMA copies into this slot must not overtake these stores
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                    }
                }
                const double* colp = pl + row0 * PX + HX + 2 * lane;
                (void)colp;                                        // the WRAP instantiation indexes from pl
                double v[K + 2 * R][NV];
#pragma unroll
                for (int kk = 0; kk < K + 2 * R; ++kk)
#pragma unroll
                    for (int t = 0; t < NV / 2; ++t) {
                        double2 dd;
                        if constexpr (WRAP) {
                            const int c = 2 * lane - HW + 2 * t;       // first tile column of this double2
                            int o = (row0 + kk) * PX + HX + c;
                            const int o_xs = S::PLANE_DOUBLES + (row0 + kk) * 4;
                            if (2 * t < HW && edge_l && c < 0) o = o_xs + 4 + c;
                            if (2 * t >= HW + 2 && edge_r && c >= kStream64TX) o = o_xs + S::XS_BYTES / 8 + c - kStream64TX;
                            dd = *reinterpret_cast<const double2*>(pl + o);
                        } else {
                            dd = *reinterpret_cast<const double2*>(colp + kk * PX - HW + 2 * t);
                        }
                        v[kk][2 * t] = dd.x;
                        v[kk][2 * t + 1] = dd.y;
                    }
                __syncwarp();
                mbar_arrive_if(lane == 0, empty0 + 8 * s);
                if (++s == nstage) { s = 0; ph ^= 1; }

#pragma unroll
                for (int k = 0; k < K; ++k) {
#pragma unroll
                    for (int d = 0; d < M; ++d) {     // this plane is tap dz = d - R of output i-(d-R)
                        double2& t = T[k][(u - d + R + 2 * M) % M];
                        double a[2];
                        if (d == 0) {
                            a[0] = bw.w[0][0][0] * v[k][HW - R];
                            a[1] = bw.w[0][0][0] * v[k][HW - R + 1];
                        } else {
                            a[0] = t.x; a[1] = t.y;
                        }
#pragma unroll
                        for (int dy = 0; dy < M; ++dy)
#pragma unroll
                            for (int dx = 0; dx < M; ++dx) {
                                if (d == 0 && dy == 0 && dx == 0) continue;
                                const double wv = bw.w[d][dy][dx];
                                a[0] = fma(wv, v[k + dy][HW - R + dx], a[0]);
                                a[1] = fma(wv, v[k + dy][HW - R + 1 + dx], a[1]);
                            }
                        t = make_double2(a[0], a[1]);
                    }
                }
                if (i >= 2 * R) {
#pragma unroll
                    for (int k = 0; k < K; ++k)
                        if (row_ok[k] && store_in_grid(op + (size_t)k * g.nx, 2, out, g, status))
                            *reinterpret_cast<double2*>(op + (size_t)k * g.nx) = T[k][(u + R + 1) % M];
                    op += plane_stride;
                }
                return true;
            });
            if (!ok) {
                atomicExch(status, kStatusTimeout);
                return;
            }
        }
    }
}

template <int R, bool BOX, int K, int NW, int MINB>
__global__ void __launch_bounds__((NW + 1) * 32, MINB)
stencil_stream_f64_kernel(const __grid_constant__ CUtensorMap tmap_in, double* __restrict__ out,
                          const StreamGeom g,
                          const __grid_constant__ StarWeights64<R> sw,
                          const __grid_constant__ BoxWeights64<BOX ? R : 0> bw,
                          int* __restrict__ status) {
    stream_f64_body<R, BOX, K, NW, false>(tmap_in, tmap_in, tmap_in, tmap_in, out, g, sw, bw, status);
}

// The sweep of a periodic grid: tmap_xs has boxes of 4 columns x ROWS rows, tmap_ys of PX columns x R rows.
// (the 27-point box is held to two CTAs per SM like its zero-boundary kernel: left alone it takes 120 registers;
// the 125-point box takes 84 instead of 68 and spills when it is held to the three CTAs those 68 allow)
template <int R, bool BOX, int K, int NW, int MINB>
__global__ void __launch_bounds__((NW + 1) * 32, (BOX && R == 1) ? 2 : MINB)
stencil_stream_f64_wrap_kernel(const __grid_constant__ CUtensorMap tmap_in,
                               const __grid_constant__ CUtensorMap tmap_xs,
                               const __grid_constant__ CUtensorMap tmap_ys,
                               const __grid_constant__ CUtensorMap tmap_cs, double* __restrict__ out,
                               const StreamGeom g, const __grid_constant__ StarWeights64<R> sw,
                               const __grid_constant__ BoxWeights64<BOX ? R : 0> bw, int* __restrict__ status) {
    stream_f64_body<R, BOX, K, NW, true>(tmap_in, tmap_xs, tmap_ys, tmap_cs, out, g, sw, bw, status);
}

}  // namespace stencil
