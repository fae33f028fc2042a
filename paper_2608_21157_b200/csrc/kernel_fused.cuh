// FUSED kernel: temporal blocking for the iterated 3D star sweep with a zero
// boundary, on fp32 or FP64 grids (element type E; a lane holds one 16-byte
// vector of a row, four floats or two doubles).  One pass over the grid advances it by up to T time steps while
// reading the input once and writing the result once.
//
// A CTA owns a TXE x TYE region of the x-y plane (its output tile plus a halo
// of T*R cells that is recomputed redundantly) and a range of z.  Input planes
// arrive through a TMA ring exactly as in the single-step kernel.  Time level
// l (1..T) is computed from level l-1 one plane at a time:
//
//   - each thread owns the same K rows x one 16-byte column at every level, so
//     the centre values of level l-1 are already in its registers;
//   - the rows above/below its block and the cells left/right of a warp come
//     from the level's plane in shared memory (double-buffered; one CTA
//     barrier per level per plane);
//   - the +-z taps never touch shared memory: forward accumulation with a
//     register queue, as in the single-step kernel.
//
// Level l lags level l-1 by R planes.  Cells outside the grid are forced back
// to zero at every level (the zero boundary holds at every time step), and
// every intermediate level is a value of the grid's own type, so the result equals
// T separate sweeps up to summation order.  The last level goes straight to global
// memory; only the tile interior is stored.
#pragma once
#include "common.cuh"
#include "kernel_stream.cuh"
#include "ptx.cuh"

namespace stencil {


// The 16-byte vector of a row that one lane holds, and the taps of a star in the grid's type.
template <typename E> struct FusedVec;
template <> struct FusedVec<float>  { using V = float4;  static constexpr int N = 4; };
template <> struct FusedVec<double> { using V = double2; static constexpr int N = 2; };

template <typename E, int R>
struct StarTaps {               // index d + R along each axis, entry [R] unused
    E c;
    E x[2 * R + 1], y[2 * R + 1], z[2 * R + 1];
};

template <int R, int K, int XW, int NWY, typename E = float>
struct FusedShape {
    static constexpr int NV = FusedVec<E>::N;                   // points of a row per lane
    static constexpr int WX = 32 * NV;                          // columns one warp spans
    static constexpr int TXE = WX * XW;
    static constexpr int TYE = NWY * K;
    static constexpr int THREADS = XW * NWY * 32;
    // A TMA box is at most 256 elements wide, so a wider plane lies in shared memory as NP parts
    // of PW columns (two of 256 for a 512-wide region, three of 128 for a 384-wide one), each loaded by its own copy and each with its own pad rows:
    // cell (row r, column x) of a plane is at  (x / PW) * PART_FLOATS + r * PW + x % PW.
    static constexpr int PW = TXE <= 256 ? TXE : (TXE % 256 == 0 ? 256 : 128);
    static constexpr int NP = TXE / PW;
    static constexpr int PART_FLOATS = (TYE + 2 * R) * PW;      // R pad rows above and below
    static constexpr int SLOT_FLOATS = NP * PART_FLOATS;
    static constexpr int SLOT_BYTES = SLOT_FLOATS * (int)sizeof(E);   // multiple of 512
    static constexpr int BOX_BYTES = TYE * TXE * (int)sizeof(E);      // bytes of all parts of one plane
    static size_t smem_bytes(int stages, int T) {
        return (size_t)(stages + 2 * (T - 1)) * SLOT_BYTES + 128 + kMaxStages * 8;
    }
};

__device__ __forceinline__ void consumer_barrier(int nthreads) {
    asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
}

// MODE 1 (SPEC): the launch advances exactly T levels and one region spans a whole row of exactly
// 128*XW points (64*XW in FP64).  The level count, the row pitch and the x bounds are then compile-time
// constants (the common case of the iterated apply on a 256-wide grid).
// MODE 2 (SPEC and WRAP): the same, on a grid that is periodic along x and z (the pass of a
// periodic grid; its y faces are put right afterwards).  z wraps in the plane coordinate of the
// TMA loads, since every plane is a load of its own, and no plane counts as outside the grid;
// x wraps where the first and last warp of a row fetch the cells beyond the row's ends, at every
// level, from the other end of the same row of the level's plane in shared memory.
template <typename E, int R, int T, int K, int XW, int NWY, int MODE = 0>
__global__ void __launch_bounds__(XW * NWY * 32, (XW * NWY * 32 <= 256 ? 2 : 1))
stencil_fused_kernel(const __grid_constant__ CUtensorMap tmap_in, E* __restrict__ out,
                     const FusedGeom g, const __grid_constant__ StarTaps<E, R> sw,
                     int* __restrict__ status) {
    constexpr bool SPEC = MODE >= 1, WRAP = MODE == 2;
    using S = FusedShape<R, K, XW, NWY, E>;
    using V = typename FusedVec<E>::V;
    constexpr int NV = S::NV;
    constexpr int TXE = S::TXE;
    constexpr int PW = S::PW;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    // indexing the shared array keeps every derived pointer in the shared address space
    unsigned char* base = smem_raw + ((128u - (smem_addr(smem_raw) & 127u)) & 127u);
    const int nstage = g.stages;
    E* ring = reinterpret_cast<E*>(base);                                           // nstage slots
    E* lvl = ring + (size_t)nstage * S::SLOT_FLOATS;                                // (T-1) x 2 slots
    uint64_t* bars = reinterpret_cast<uint64_t*>(lvl + (size_t)2 * (T - 1) * S::SLOT_FLOATS);
    const uint32_t full0 = smem_addr(bars);

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int wx = warp % XW, wy = warp / XW;
    const int col = NV * (wx * 32 + lane);         // x offset inside the region
    const int row0 = wy * K;                       // first region row of this thread

    // zero the pad rows of every slot once; TMA and the level stores never touch them
    {
        const int nslots = nstage + 2 * (T - 1);
        for (int s = 0; s < nslots; ++s) {
            E* slot = ring + (size_t)s * S::SLOT_FLOATS;
            for (int e = tid; e < R * TXE; e += S::THREADS) {
                E* part = slot + (e / (R * PW)) * S::PART_FLOATS;
                part[e % (R * PW)] = E(0);
                part[(S::TYE + R) * PW + e % (R * PW)] = E(0);
            }
        }
    }
    if (tid == 0) {
        for (int s = 0; s < nstage; ++s) mbar_init(full0 + 8 * s, 1);
        fence_barrier_init();
    }
    __syncthreads();
    allow_dependents();
    dependency_wait();           // the input is the output of the previous pass

    // CTAs are numbered region-fastest.  The first g.main_ctas of them cut planes [0, nz - rest_z) of every
    // region into chunks of chunk_z planes.  The launcher may add more: those cut the last rest_z planes into
    // chunks of rest_chunk planes; they are short and come last in the grid, so that they fill the SMs which
    // the long chunks leave idle in their last wave.
    const bool tail = (int)blockIdx.x >= g.main_ctas;
    const int bid = tail ? blockIdx.x - g.main_ctas : blockIdx.x;
    const int tix = bid % g.tiles_x;
    const int tiy = (bid / g.tiles_x) % g.tiles_y;
    const int chunk = bid / (g.tiles_x * g.tiles_y);
    const int x0e = SPEC ? 0 : tix * g.tile_x - g.halo_x;     // region origin (may be negative)
    const int y0e = tiy * g.tile_y - g.halo_y;
    const int main_z = g.nz - g.rest_z;
    const int z0 = tail ? main_z + chunk * g.rest_chunk : chunk * g.chunk_z;
    const int z1 = tail ? min(z0 + g.rest_chunk, g.nz) : min(z0 + g.chunk_z, main_z);
    const int nlev = SPEC ? T : g.nlev;
    const int nx = SPEC ? TXE : g.nx;
    const int pstart = z0 - nlev * R;
    const int nsteps = (z1 - z0) + 2 * nlev * R;

    const int xg = x0e + col;
    const bool x_in = SPEC || (xg >= 0 && xg < nx);
    const bool x_store = SPEC || (x_in && col >= g.halo_x && col < g.halo_x + g.tile_x);
    // per-row flags packed into bit masks; the common case (every row inside the grid,
    // every row stored) is tested once per plane instead of once per row
    uint32_t in_mask = 0, store_mask = 0;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        const int yg = y0e + row0 + k;
        const bool y_in = yg >= 0 && yg < g.ny;
        if (y_in && x_in) in_mask |= 1u << k;
        if (y_in && x_store && (row0 + k) >= g.halo_y && (row0 + k) < g.halo_y + g.tile_y) store_mask |= 1u << k;
    }
    constexpr uint32_t kAllRows = (1u << K) - 1u;
    // the same flags for the whole warp, so that the common case is a uniform branch
    const bool warp_all_in = __all_sync(0xffffffffu, in_mask == kAllRows);
    const bool warp_all_store = __all_sync(0xffffffffu, store_mask == kAllRows);
    const size_t plane_stride = (size_t)g.ny * nx;
    E* const out_col = out + (size_t)(y0e + row0) * nx + xg;           // this thread's column of rows
    const int toff = (col / PW) * S::PART_FLOATS + row0 * PW + col % PW;   // its offset inside a plane
    // the cells just left and right of the warp's columns (they may lie in another part)
    constexpr int WX = S::WX;
    const int hl_off = wx > 0 ? ((wx * WX - 1) / PW) * S::PART_FLOATS + (wx * WX - R) - ((wx * WX - 1) / PW) * PW : 0;
    const int hr_off = wx < XW - 1 ? (((wx + 1) * WX) / PW) * S::PART_FLOATS + (wx + 1) * WX - (((wx + 1) * WX) / PW) * PW : 0;

    // the plane a load fetches: wrapped into the grid under WRAP (nz >= 2*T*R, so one step is enough)
    auto plane_coord = [&](int zc) { return !WRAP ? zc : (zc < 0 ? zc + g.nz : (zc >= g.nz ? zc - g.nz : zc)); };
    // the cells beyond the two ends of a row under WRAP: the last R cells of the last part, the first R of the first
    constexpr int wrap_l_off = (S::NP - 1) * S::PART_FLOATS + PW - R;
    constexpr int wrap_r_off = 0;

    int issued = 0;                                // planes requested so far (thread 0 only)
    if (tid == 0) {
        prefetch_tensormap(&tmap_in);
        const int pre = min(nstage, nsteps);
        issued = pre;
        for (int i = 0; i < pre; ++i) {
            if (i == g.drop_plane) continue;
            mbar_arrive_expect_tx(full0 + 8 * i, S::BOX_BYTES);
#pragma unroll
            for (int part = 0; part < S::NP; ++part)
                tma_load_3d(smem_addr(ring + (size_t)i * S::SLOT_FLOATS + part * S::PART_FLOATS + R * PW), &tmap_in,
                            full0 + 8 * i, x0e + part * PW, y0e, plane_coord(pstart + i));
        }
    }

    // A[l][k][j]: level l+1's partial sums, oldest incomplete output plane first (see the
    // single-step kernel: arriving planes update them in place, nothing is copied)
    V A[T][K][2 * R];
#pragma unroll
    for (int l = 0; l < T; ++l)
#pragma unroll
        for (int k = 0; k < K; ++k)
#pragma unroll
            for (int j = 0; j < 2 * R; ++j) A[l][k][j] = vzero<V>();

    bool dead = false;
    int s = 0;                                     // input ring slot and its phase parity
    uint32_t ph = 0;
    // One plane step.  `par` is the parity of the level buffers; FAST marks a step in the steady
    // state whose planes lie inside the grid along z at every level: nothing needs its z range
    // checked and the last level always stores.
    auto step = [&](auto par_c, auto fast_c, const int i) {
            constexpr int par = decltype(par_c)::value & 1;
            constexpr bool FAST = decltype(fast_c)::value != 0;
            if (!dead && !mbar_wait_bounded(full0 + 8 * s, ph, g.wait_polls)) {
                dead = true;
                atomicExch(status, kStatusTimeout);
            }
            const E* src = ring + (size_t)s * S::SLOT_FLOATS + R * PW;          // region row 0 (of part 0)
            V cin[K + 2 * R];
#pragma unroll
            for (int kk = 0; kk < K + 2 * R; ++kk)
                cin[kk] = *reinterpret_cast<const V*>(src + toff + (kk - R) * PW);

#pragma unroll
            for (int l = 1; l <= T; ++l) {
                if (l <= nlev) {
                    const int zl = pstart + i - l * R;          // plane this level completes now
                    V e[K];
                    {
#pragma unroll
                        for (int k = 0; k < K; ++k) {
                            const V ctr = cin[k + R];
                            E v[NV + 2 * R];
                            E c4[NV];
                            vunpack(ctr, c4);
#pragma unroll
                            for (int m = 0; m < NV; ++m) v[R + m] = c4[m];
                            {
                                const E* rowb = src + (row0 + k) * PW;        // first cell of the region row (part 0)
#pragma unroll
                                for (int t = 0; t < R; ++t) {
                                    // cells across the warp boundary: one broadcast read per side from the
                                    // level's plane (wx is warp-uniform); zero at the region's edge
                                    E xl = E(0), xr = E(0);
                                    if (XW > 1) {
                                        if (wx > 0) xl = rowb[hl_off + t];
                                        if (wx < XW - 1) xr = rowb[hr_off + t];
                                    }
                                    if (WRAP) {
                                        if (wx == 0) xl = rowb[wrap_l_off + t];
                                        if (wx == XW - 1) xr = rowb[wrap_r_off + t];
                                    }
                                    const E lft = __shfl_up_sync(0xffffffffu, c4[NV - R + t], 1);
                                    const E rgt = __shfl_down_sync(0xffffffffu, c4[t], 1);
                                    v[t] = lane == 0 ? xl : lft;
                                    v[R + NV + t] = lane == 31 ? xr : rgt;
                                }
                            }
                            V (&Al)[2 * R] = A[l - 1][k];
                            // the output whose centre plane this is continues from Al[R]; the centre and
                            // y taps work on aligned pairs (packed FMAs), the x taps on single lanes
                            V a4 = fma4r(sw.c, ctr, Al[R]);
#pragma unroll
                            for (int d = 1; d <= R; ++d) {
                                fma4(a4, sw.y[R - d], cin[k + R - d]);
                                fma4(a4, sw.y[R + d], cin[k + R + d]);
                            }
                            E acc[NV];
                            vunpack(a4, acc);
#pragma unroll
                            for (int m = 0; m < NV; ++m) {
                                E a = acc[m];
#pragma unroll
                                for (int d = 1; d <= R; ++d) {
                                    a = fma_t(sw.x[R - d], v[R + m - d], a);
                                    a = fma_t(sw.x[R + d], v[R + m + d], a);
                                }
                                acc[m] = a;
                            }
                            // z taps: oldest output complete; the others slide down inside their FMA
                            e[k] = fma4r(sw.z[2 * R], ctr, Al[0]);
#pragma unroll
                            for (int j = 0; j < 2 * R - 1; ++j) {
                                if (j == R - 1) continue;
                                Al[j] = fma4r(sw.z[2 * R - 1 - j], ctr, Al[j + 1]);
                            }
                            Al[2 * R - 1] = mul4(sw.z[0], ctr);
                            Al[R - 1] = vpack<V>(acc);
                        }
                        // the zero boundary holds at every time level: cells outside the grid go
                        // back to zero (nothing to do for regions and planes inside the grid)
                        if (!warp_all_in || (!WRAP && !FAST && (zl < 0 || zl >= g.nz))) {
                            const bool z_in = WRAP || FAST || (zl >= 0 && zl < g.nz);
#pragma unroll
                            for (int k = 0; k < K; ++k)
                                if (!(z_in && ((in_mask >> k) & 1u))) e[k] = vzero<V>();
                        }

                        if (l == nlev) {
                            // last level of this pass: interior of the tile goes to global memory
                            if (!dead && (FAST || (zl >= z0 && zl < z1))) {
                                E* op = out_col + (size_t)zl * plane_stride;
                                if (warp_all_store) {
#pragma unroll
                                    for (int k = 0; k < K; ++k)
                                        if (store_in_grid(op + (size_t)k * nx, NV, out, g, status))
                                            *reinterpret_cast<V*>(op + (size_t)k * nx) = e[k];
                                } else {
#pragma unroll
                                    for (int k = 0; k < K; ++k)
                                        if (((store_mask >> k) & 1u) && store_in_grid(op + (size_t)k * nx, NV, out, g, status))
                                            *reinterpret_cast<V*>(op + (size_t)k * nx) = e[k];
                                }
                            }
                        } else {
                            E* buf = lvl + (size_t)(2 * (l - 1) + par) * S::SLOT_FLOATS + R * PW;
#pragma unroll
                            for (int k = 0; k < K; ++k)
                                *reinterpret_cast<V*>(buf + toff + k * PW) = e[k];
                        }
                    }
                    if (l < nlev || l == 1) {
                        // everyone has finished with level l-1's plane and has published level l
                        consumer_barrier(S::THREADS);
                        if (l == 1 && tid == 0 && i + nstage < nsteps && i + nstage != g.drop_plane) {
                            // the input slot is free: refill it with the plane nstage steps ahead
                            mbar_arrive_expect_tx(full0 + 8 * s, S::BOX_BYTES);
#pragma unroll
                            for (int part = 0; part < S::NP; ++part)
                                tma_load_3d(smem_addr(ring + (size_t)s * S::SLOT_FLOATS + part * S::PART_FLOATS + R * PW),
                                            &tmap_in, full0 + 8 * s, x0e + part * PW, y0e,
                                            plane_coord(pstart + i + nstage));
                            issued = i + nstage + 1;
                        }
                    }
                    if (l < nlev) {
                        const E* buf = lvl + (size_t)(2 * (l - 1) + par) * S::SLOT_FLOATS + R * PW;
                        src = buf;
#pragma unroll
                        for (int k = 0; k < K; ++k) cin[k + R] = e[k];
#pragma unroll
                        for (int kk = 0; kk < R; ++kk) {
                            cin[kk] = *reinterpret_cast<const V*>(buf + toff + (kk - R) * PW);
                            cin[K + R + kk] = *reinterpret_cast<const V*>(buf + toff + (K + kk) * PW);
                        }
                    }
                }
            }
            if (++s == nstage) { s = 0; ph ^= 1; }
    };
    // two planes per trip, so that the parity of the level buffers is a compile-time constant in
    // each copy of the step; the first 2*nlev*R steps fill the pipeline and store nothing
    using std::integral_constant;
    for (int i0 = 0; i0 < nsteps; i0 += 2) {
        const bool fast = SPEC && i0 >= 2 * nlev * R && i0 + 1 < nsteps &&
                          (WRAP || (pstart + i0 - nlev * R >= 0 && pstart + i0 + 1 - R < g.nz));
        if (fast) {
            step(integral_constant<int, 0>{}, integral_constant<int, 1>{}, i0);
            step(integral_constant<int, 1>{}, integral_constant<int, 1>{}, i0 + 1);
        } else {
            step(integral_constant<int, 0>{}, integral_constant<int, 0>{}, i0);
            if (i0 + 1 < nsteps) step(integral_constant<int, 1>{}, integral_constant<int, 0>{}, i0 + 1);
        }
    }
    if (dead && tid == 0) {
        // let copies that may still be in flight land before shared memory is released
        for (int i = max(0, issued - nstage); i < issued; ++i)
            mbar_wait_bounded(full0 + 8 * (i % nstage), (i / nstage) & 1, g.wait_polls);
    }
}

}  // namespace stencil
