// STREAM kernels: 3D sweep with a zero boundary, x-y tiles staged by TMA into a
// shared-memory ring and streamed along the slowest axis (z).
//
// One CTA owns a TX x TY tile of the x-y plane and a contiguous range of z.
// A producer warp issues one TMA tile load per input plane (tile plus halo;
// everything outside the grid arrives as zero, so the zero boundary costs no
// branches).  NW consumer warps each own K rows of the tile, one float4 of x
// per lane.  Every arriving plane is used once, at arrival:
//
//   star  - the in-plane taps (x through warp shuffles / the smem halo, y from
//           smem rows) start the output of that plane; the +-z taps are
//           applied by forward accumulation: the plane's own-column values
//           are added into the R outputs still pending, and the last R
//           own-column values (a register queue) feed the new output.
//   box   - the plane's (2R+1)^2 in-plane sums for each dz are added into the
//           2R+1 outputs it touches; the oldest is complete and is stored.
//
// Finished outputs go to global memory as 128-bit coalesced stores straight
// from registers.  Every intermediate stays in registers; shared memory only
// holds the ring of input planes.
#pragma once
#include <type_traits>
#include <utility>

#include "common.cuh"
#include "geom.cuh"
#include "ptx.cuh"

namespace stencil {

constexpr int kStreamPX = kStreamTX + 8;  // smem row pitch: 4-float halo each side keeps
                                          // TMA x-coordinates and LDS.128 16-byte aligned

// Halo columns on either side of a tile row in shared memory: 4 floats reach radius 4; the
// wider stars (radius 5..8) take 8.  Multiples of 4 keep TMA x-coordinates and LDS.128 aligned.
template <int R>
struct StreamHalo {
    static_assert(R >= 1 && R <= 8, "radius 1..8");
    static constexpr int HX = R <= 4 ? 4 : 8;
    static constexpr int PX = kStreamTX + 2 * HX;      // smem row pitch
};

// The same for the FP64 kernels, whose tile rows are 64 doubles wide.
template <int R>
struct StreamHalo64 {
    static_assert(R >= 1 && R <= 8, "radius 1..8");
    static constexpr int HX = R <= 4 ? 4 : 8;
    static constexpr int PX = 64 + 2 * HX;
};

template <int R>
struct StarWeights {            // taps of a star stencil, index d + R along each axis
    float c;
    float x[2 * R + 1], y[2 * R + 1], z[2 * R + 1];   // entry [R] unused
};

template <int R>
struct BoxWeights {             // dense cube, [dz+R][dy+R][dx+R]
    float w[2 * R + 1][2 * R + 1][2 * R + 1];
};


template <int R, int K, int NW>
struct StreamShape {
    static constexpr int TY = NW * K;
    static constexpr int ROWS = TY + 2 * R;
    static constexpr int PLANE_FLOATS = ROWS * StreamHalo<R>::PX;
    static constexpr int BOX_BYTES = PLANE_FLOATS * 4;
    static constexpr int PLANE_BYTES = (BOX_BYTES + 127) / 128 * 128;
    static constexpr int THREADS = (NW + 1) * 32;
    static size_t smem_bytes(int stages) { return (size_t)stages * PLANE_BYTES + 128 + 128; }
    // Periodic sweeps (WRAP): beside every plane of the ring, the cells the plane's halo would hold on a
    // torus, each block loaded by a TMA copy of its own: the 4 columns beyond the left and the right end of
    // the tile's rows (ROWS x 4 cells each) and the R rows above and below it (R x PX cells each).
    static constexpr int XS_BYTES = (ROWS * 16 + 127) / 128 * 128;
    static constexpr int YS_BYTES = (R * StreamHalo<R>::PX * 4 + 127) / 128 * 128;
    // ... and, for boxes, the four corners of the halo (4 columns x R rows each)
    static constexpr int CS_BYTES = (R * 16 + 127) / 128 * 128;
    static constexpr int STAGE_BYTES = 2 * XS_BYTES + 2 * YS_BYTES + 4 * CS_BYTES;
};

// Calls f(integral_constant<int, 0>) ... f(integral_constant<int, N-1>) in order and
// stops at the first call that returns false.  The index is a compile-time constant
// inside f, which keeps register arrays indexed by it in registers.
template <class F, int... Is>
__device__ __forceinline__ bool static_for_impl(F&& f, std::integer_sequence<int, Is...>) {
    return (f(std::integral_constant<int, Is>{}) && ...);
}
template <int N, class F>
__device__ __forceinline__ bool static_for(F&& f) {
    return static_for_impl(f, std::make_integer_sequence<int, N>{});
}

__device__ __forceinline__ float f4get(const float4& v, int m) {
    return m == 0 ? v.x : (m == 1 ? v.y : (m == 2 ? v.z : v.w));
}

__device__ __forceinline__ void store_f4(float* p, const float4& v, int streaming) {
    if (streaming) __stcs(reinterpret_cast<float4*>(p), v);
    else *reinterpret_cast<float4*>(p) = v;
}

// Predicated shared-memory load: returns *p where `take` holds, `keep` elsewhere,
// without a divergent branch.
__device__ __forceinline__ float lds_if(bool take, const float* p, float keep) {
    asm volatile(
        "{\n\t.reg .pred q;\n\t"
        "setp.ne.u32 q, %2, 0;\n\t"
        "@q ld.shared.f32 %0, [%1];\n\t}"
        : "+f"(keep)
        : "r"(smem_addr(p)), "r"((uint32_t)take)
        : "memory");
    return keep;
}

// Fills v[0 .. 4+2R) with the R values left of the lane's float4, the float4
// itself, and the R values right of it, for one smem row.  `rowp` points at the
// lane's float4 inside the row; `rowbase` at the row's first float (x = -4; the
// R <= 2 path, the only one that uses it, always has a 4-float halo).  FROM_SMEM
// makes radius 1 and 2 read their neighbours from the row as well, like the wider radii.
template <int R, bool FROM_SMEM = false>
__device__ __forceinline__ void gather_row(const float* rowp, const float* rowbase, int lane,
                                           const float4& ctr, float (&v)[4 + 2 * R]) {
    v[R + 0] = ctr.x; v[R + 1] = ctr.y; v[R + 2] = ctr.z; v[R + 3] = ctr.w;
    if constexpr (R <= 2 && !FROM_SMEM) {
        // neighbours' registers through shuffles; the row's two end lanes read the smem halo
        const float c4[4] = {ctr.x, ctr.y, ctr.z, ctr.w};
#pragma unroll
        for (int t = 0; t < R; ++t) {
            // every lane reads the two halo words (a broadcast, one wavefront each, no
            // branch); only the end lanes keep them
            const float hl = rowbase[4 - R + t];
            const float hr = rowbase[4 + kStreamTX + t];
            const float l = __shfl_up_sync(0xffffffffu, c4[4 - R + t], 1);
            const float r = __shfl_down_sync(0xffffffffu, c4[t], 1);
            v[t] = lane == 0 ? hl : l;
            v[R + 4 + t] = lane == 31 ? hr : r;
        }
    } else if constexpr (R <= 4) {
        const float4 l = *reinterpret_cast<const float4*>(rowp - 4);
        const float4 r = *reinterpret_cast<const float4*>(rowp + 4);
        const float l4[4] = {l.x, l.y, l.z, l.w};
        const float r4[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int t = 0; t < R; ++t) {
            v[t] = l4[4 - R + t];
            v[R + 4 + t] = r4[t];
        }
    } else {
        // radius 5..8: two float4 on either side (the row has an 8-float halo)
        const float4 la = *reinterpret_cast<const float4*>(rowp - 8);
        const float4 lb = *reinterpret_cast<const float4*>(rowp - 4);
        const float4 ra = *reinterpret_cast<const float4*>(rowp + 4);
        const float4 rb = *reinterpret_cast<const float4*>(rowp + 8);
        const float l8[8] = {la.x, la.y, la.z, la.w, lb.x, lb.y, lb.z, lb.w};
        const float r8[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
#pragma unroll
        for (int t = 0; t < R; ++t) {
            v[t] = l8[8 - R + t];
            v[R + 4 + t] = r8[t];
        }
    }
}

// gather_row for a row whose halo columns may live elsewhere (radius <= 4).  Everything is an offset
// from one pointer into shared memory, so that the loads stay shared-space loads whichever way the
// selects go: `o_rowp` is the lane's float4, `o_lh` the 4 cells left of the row's first tile column,
// `o_rh` the 4 cells right of its last one.
template <int R>
__device__ __forceinline__ void gather_row_split(const float* base, int o_rowp, int o_lh, int o_rh, int lane,
                                                 const float4& ctr, float (&v)[4 + 2 * R]) {
    static_assert(R <= 4, "4-column halos");
    v[R + 0] = ctr.x; v[R + 1] = ctr.y; v[R + 2] = ctr.z; v[R + 3] = ctr.w;
    if constexpr (R <= 2) {
        const float c4[4] = {ctr.x, ctr.y, ctr.z, ctr.w};
#pragma unroll
        for (int t = 0; t < R; ++t) {
            const float hl = base[o_lh + 4 - R + t];
            const float hr = base[o_rh + t];
            const float l = __shfl_up_sync(0xffffffffu, c4[4 - R + t], 1);
            const float r = __shfl_down_sync(0xffffffffu, c4[t], 1);
            v[t] = lane == 0 ? hl : l;
            v[R + 4 + t] = lane == 31 ? hr : r;
        }
    } else {
        const float4 l = *reinterpret_cast<const float4*>(base + (lane == 0 ? o_lh : o_rowp - 4));
        const float4 r = *reinterpret_cast<const float4*>(base + (lane == 31 ? o_rh : o_rowp + 4));
        const float l4[4] = {l.x, l.y, l.z, l.w};
        const float r4[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int t = 0; t < R; ++t) {
            v[t] = l4[4 - R + t];
            v[R + 4 + t] = r4[t];
        }
    }
}

// WRAP: the sweep of a periodic grid (stars of radius <= 4, boxes of radius <= 2, rows a whole number of tiles).  z wraps
// in the plane coordinate of the TMA loads (every plane is a load of its own).  A tile at an x or y
// face gets, beside each plane, the cells its halo would hold on a torus (see StreamShape), and
// its consumer warps read the halo columns of their centre rows straight from there (a tile in the
// middle of a row reads them from the plane, as ever: one pointer select per row); the halo rows,
// which only the few tiles at a y face need, are copied over the zeros TMA filled in, every warp
// copying its own columns of the rows it is about to read.  A star does not read the corners of
// the halo; a box does, so its tiles at an x and a y face get them as four more small blocks, which
// go into the halo rows of the staged column blocks in the same step.
template <int R, bool BOX, int K, int NW, bool WRAP>
__device__ __forceinline__ void
stream_body(const CUtensorMap& tmap_in, const CUtensorMap& tmap_xs, const CUtensorMap& tmap_ys,
            const CUtensorMap& tmap_cs, float* __restrict__ out, const StreamGeom& g, const StarWeights<R>& sw,
            const BoxWeights<BOX ? R : 0>& bw, int* __restrict__ status) {
    static_assert(!WRAP || R <= 4, "WRAP: 4-column halos");
    using S = StreamShape<R, K, NW>;
    constexpr int PX = StreamHalo<R>::PX;
    constexpr int HX = StreamHalo<R>::HX;
    constexpr int SLOT_BYTES = S::PLANE_BYTES + (WRAP ? S::STAGE_BYTES : 0);
    extern __shared__ __align__(128) unsigned char smem_raw[];
    // ring of planes first (128-byte aligned slots), then the barriers.  The pointer is
    // formed by indexing the shared array (no integer round trip), so the compiler
    // keeps it in the shared address space and emits ld.shared for the plane reads.
    unsigned char* ring = smem_raw + ((128u - (smem_addr(smem_raw) & 127u)) & 127u);
    uint64_t* bars = reinterpret_cast<uint64_t*>(ring + (size_t)g.stages * SLOT_BYTES);
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
    dependency_wait();           // the input may be the output of the previous launch of an iteration

    // tile and z range of this CTA; x-y tiles vary fastest so that neighbours
    // (which share halo rows) are resident together and hit in L2
    const int bid = blockIdx.x;
    const int tile_x = bid % g.tiles_x;
    const int tile_y = (bid / g.tiles_x) % g.tiles_y;
    const int chunk = bid / (g.tiles_x * g.tiles_y);
    const int x0 = tile_x * kStreamTX;
    const int y0 = tile_y * S::TY;
    const int z0 = g.z_begin + chunk * g.chunk_z;
    const int z1 = min(z0 + g.chunk_z, g.z_end);
    const int nplanes = (z1 - z0) + 2 * R;      // input planes z0-R .. z1-1+R
    const int pstart = z0 - R;
    // WRAP: which faces the tile touches, and the plane row where the halo below the grid begins
    const bool edge_l = WRAP && tile_x == 0, edge_r = WRAP && tile_x == g.tiles_x - 1;
    // (a short last tile leaves the halo of the tile before it reaching below the grid as well)
    const bool edge_t = WRAP && tile_y == 0, edge_b = WRAP && y0 + S::TY + R > g.ny;
    const int row_b = R + g.ny - y0;

    if (warp == NW) {
        // ---------------- producer: one lane drives the TMA ring ----------------
        if (lane == 0) {
            prefetch_tensormap(&tmap_in);
            bool ok = true;
            int issued = 0;
            int s = 0;
            uint32_t ph = 1;                       // parity of the previous use of the slot
            for (int i = 0; i < nplanes; ++i) {
                if (i >= nstage && !mbar_wait_bounded(empty0 + 8 * s, ph, g.wait_polls)) { ok = false; break; }
                if (i != g.drop_plane) {
                    if constexpr (WRAP) {
                        int zc = pstart + i;                       // nz >= 2R: one step brings it back
                        zc = zc < 0 ? zc + g.nz : (zc >= g.nz ? zc - g.nz : zc);
                        const uint32_t bar = full0 + 8 * s;
                        unsigned char* slot = ring + (size_t)s * SLOT_BYTES;
                        const int ncorner = BOX ? ((int)edge_l + (int)edge_r) * ((int)edge_t + (int)edge_b) : 0;
                        mbar_arrive_expect_tx(bar, S::BOX_BYTES + ((int)edge_l + (int)edge_r) * S::ROWS * 16 +
                                                       ((int)edge_t + (int)edge_b) * R * PX * 4 + ncorner * R * 16);
                        tma_load_3d(smem_addr(slot), &tmap_in, bar, x0 - HX, y0 - R, zc);
                        unsigned char* stage = slot + S::PLANE_BYTES;
                        if (edge_l) tma_load_3d(smem_addr(stage), &tmap_xs, bar, g.nx - 4, y0 - R, zc);
                        if (edge_r) tma_load_3d(smem_addr(stage + S::XS_BYTES), &tmap_xs, bar, 0, y0 - R, zc);
                        if (edge_t) tma_load_3d(smem_addr(stage + 2 * S::XS_BYTES), &tmap_ys, bar, x0 - HX, g.ny - R, zc);
                        if (edge_b)
                            tma_load_3d(smem_addr(stage + 2 * S::XS_BYTES + S::YS_BYTES), &tmap_ys, bar, x0 - HX, 0, zc);
                        if constexpr (BOX) {                       // corners: (left, right) x (top, bottom)
                            unsigned char* cs = stage + 2 * S::XS_BYTES + 2 * S::YS_BYTES;
                            if (edge_l && edge_t) tma_load_3d(smem_addr(cs), &tmap_cs, bar, g.nx - 4, g.ny - R, zc);
                            if (edge_r && edge_t) tma_load_3d(smem_addr(cs + S::CS_BYTES), &tmap_cs, bar, 0, g.ny - R, zc);
                            if (edge_l && edge_b) tma_load_3d(smem_addr(cs + 2 * S::CS_BYTES), &tmap_cs, bar, g.nx - 4, 0, zc);
                            if (edge_r && edge_b) tma_load_3d(smem_addr(cs + 3 * S::CS_BYTES), &tmap_cs, bar, 0, 0, zc);
                        }
                    } else {
                        mbar_arrive_expect_tx(full0 + 8 * s, S::BOX_BYTES);
                        tma_load_3d(smem_addr(ring + (size_t)s * S::PLANE_BYTES), &tmap_in, full0 + 8 * s,
                                    x0 - HX + g.in_off_x, y0 - R + g.in_off_y, pstart + i + g.in_off_z);
                    }
                }
                issued = i + 1;
                if (++s == nstage) { s = 0; ph ^= 1; }
            }
            if (!ok) {
                atomicExch(status, kStatusTimeout);
                // let copies already in flight land before the CTA's smem goes away
                for (int i = max(0, issued - nstage); i < issued; ++i)
                    mbar_wait_bounded(full0 + 8 * (i % nstage), (i / nstage) & 1, g.wait_polls);
            }
        }
        return;
    }

    // ------------------------------- consumers --------------------------------
    const int row0 = warp * K;                         // first tile row of this warp
    const int xg = x0 + 4 * lane;                      // global x of the lane's float4
    const bool x_in = xg < g.nx;
    const size_t plane_stride = (size_t)g.ny * g.nx;
    bool row_ok[K];
#pragma unroll
    for (int k = 0; k < K; ++k) row_ok[k] = x_in && (y0 + row0 + k) < g.ny;
    // Interior warps (every lane stores every row) can take a branch-free store path.  It pays
    // for the sweeps that are bound by instruction issue (+3 % measured on the 27-point box and
    // the radius-4 star) and costs 3 % on the bandwidth-bound 7-point star, hence the switch.
    constexpr bool kUniformStores = BOX || R >= 3;
    bool mine_ok = kUniformStores;
#pragma unroll
    for (int k = 0; k < K; ++k) mine_ok = mine_ok && row_ok[k];
    const bool all_ok = kUniformStores && __all_sync(0xffffffffu, mine_ok);
    // next output plane of this thread (advanced after every stored plane)
    float* op = out + (size_t)z0 * plane_stride + (size_t)(y0 + row0) * g.nx + xg;
    const int streaming = g.streaming_store;
    int s = 0;                                      // ring slot and its phase parity
    uint32_t ph = 0;

    if constexpr (!BOX) {
        // A[k][j]: partial sum of the output 1+j planes above the oldest incomplete one.
        // An arriving plane adds its tap to each of the 2R+1 outputs it reaches: the oldest
        // is then complete, the others move down one slot as part of the FMA that updates
        // them (no register copies), and a new one starts at the top.
        float4 A[K][2 * R];
#pragma unroll
        for (int k = 0; k < K; ++k)
#pragma unroll
            for (int j = 0; j < 2 * R; ++j) A[k][j] = make_float4(0.f, 0.f, 0.f, 0.f);

        for (int i = 0; i < nplanes; ++i) {
            if (!mbar_wait_bounded(full0 + 8 * s, ph, g.wait_polls)) {
                atomicExch(status, kStatusTimeout);
                return;
            }
            const float* pl = reinterpret_cast<const float*>(ring + (size_t)s * SLOT_BYTES);
            if constexpr (WRAP) {
                if (edge_t || edge_b) {                                // uniform over the CTA
                    float* plw = reinterpret_cast<float*>(ring + (size_t)s * SLOT_BYTES);
                    const float* stage = pl + S::PLANE_BYTES / 4;
#pragma unroll
                    for (int rr = 0; rr < R; ++rr) {
                        // the halo rows inside this warp's window of rows, the lane's own columns
                        if (edge_t && rr >= row0 && rr < row0 + K + 2 * R)
                            *reinterpret_cast<float4*>(plw + rr * PX + HX + 4 * lane) =
                                *reinterpret_cast<const float4*>(stage + 2 * S::XS_BYTES / 4 + rr * PX + HX + 4 * lane);
                        const int rb = row_b + rr;
                        if (edge_b && rb < S::ROWS && rb >= row0 && rb < row0 + K + 2 * R)
                            *reinterpret_cast<float4*>(plw + rb * PX + HX + 4 * lane) =
                                *reinterpret_cast<const float4*>(stage + (2 * S::XS_BYTES + S::YS_BYTES) / 4 + rr * PX +
                                                                 HX + 4 * lane);
                    }
                    // later TMA copies into this slot must not overtake these stores
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                }
            }
            const float* colp = pl + row0 * PX + HX + 4 * lane;
            // Rows are visited once, top to bottom.  A row is a y-neighbour of up to 2R output
            // rows and the centre row of at most one; it is consumed at once, so only one
            // loaded row is live at a time.  acc[k] is the output whose centre plane this is:
            // it continues from the partial sum A[k][R] that the planes below have built.
            // The y, centre and z taps work on aligned pairs of the lane's float4 (packed FMAs), and so
            // do the x taps at even distances; the x taps at odd distances straddle the pairs and stay
            // single FMAs.
            float4 acc[K];
#pragma unroll
            for (int k = 0; k < K; ++k) acc[k] = A[k][R];
            float4 done[K];
#pragma unroll
            for (int kk = 0; kk < K + 2 * R; ++kk) {
                const float4 c = *reinterpret_cast<const float4*>(colp + kk * PX);
#pragma unroll
                for (int k = 0; k < K; ++k) {
                    const int d = kk - k - R;              // row kk is tap dy = d of output row k
                    if (d != 0 && d >= -R && d <= R) fma4(acc[k], sw.y[d + R], c);
                }
                if (kk >= R && kk < K + R) {
                    const int k = kk - R;                  // centre row of output row k
                    float v[4 + 2 * R];
                    if constexpr (WRAP) {
                        const int o_row = (row0 + kk) * PX;
                        const int o_xs = S::PLANE_BYTES / 4 + (row0 + kk) * 4;
                        gather_row_split<R>(pl, o_row + HX + 4 * lane, edge_l ? o_xs : o_row,
                                            edge_r ? o_xs + S::XS_BYTES / 4 : o_row + HX + kStreamTX, lane, c, v);
                    } else {
                        gather_row<R>(colp + kk * PX, pl + (row0 + kk) * PX, lane, c, v);
                    }
                    float4 a4 = fma4r(sw.c, c, acc[k]);
                    // v[R + m + d] is tap dx = d of the lane's point m: for even d the operands of points
                    // (0, 1) and (2, 3) are the register pairs the row was loaded as (R >= 3: the row's
                    // left and right float4; the shuffled neighbours of R <= 2 have no such pairs)
                    float2 alo = lo2(a4), ahi = hi2(a4);
#pragma unroll
                    for (int d = 2; d <= R; d += 2) {
                        if constexpr (R >= 3) {
                            alo = fma2(sw.x[R - d], make_float2(v[R - d], v[R + 1 - d]), alo);
                            ahi = fma2(sw.x[R - d], make_float2(v[R + 2 - d], v[R + 3 - d]), ahi);
                            alo = fma2(sw.x[R + d], make_float2(v[R + d], v[R + 1 + d]), alo);
                            ahi = fma2(sw.x[R + d], make_float2(v[R + 2 + d], v[R + 3 + d]), ahi);
                        }
                    }
                    float a[4] = {alo.x, alo.y, ahi.x, ahi.y};
#pragma unroll
                    for (int m = 0; m < 4; ++m) {
#pragma unroll
                        for (int d = 1; d <= R; ++d) {
                            if (R >= 3 && d % 2 == 0) continue;     // done above
                            a[m] = fmaf(sw.x[R - d], v[R + m - d], a[m]);
                            a[m] = fmaf(sw.x[R + d], v[R + m + d], a[m]);
                        }
                    }
                    acc[k] = make_float4(a[0], a[1], a[2], a[3]);
                    // z taps: this plane is tap dz = +R of the oldest output (now complete),
                    // dz = R-1-j of the one moving into slot j, dz = -R of the new one
                    done[k] = fma4r(sw.z[2 * R], c, A[k][0]);
#pragma unroll
                    for (int j = 0; j < 2 * R - 1; ++j) {
                        if (j == R - 1) continue;          // that slot receives acc[k] below
                        A[k][j] = fma4r(sw.z[2 * R - 1 - j], c, A[k][j + 1]);
                    }
                    A[k][2 * R - 1] = mul4(sw.z[0], c);
                }
            }
#pragma unroll
            for (int k = 0; k < K; ++k) A[k][R - 1] = acc[k];
            __syncwarp();
            mbar_arrive_if(lane == 0, empty0 + 8 * s);
            if (++s == nstage) { s = 0; ph ^= 1; }

            if (i >= 2 * R) {
                if (all_ok) {
#pragma unroll
                    for (int k = 0; k < K; ++k)
                        if (store_in_grid(op + (size_t)k * g.nx, 4, out, g, status)) store_f4(op + (size_t)k * g.nx, done[k], streaming);
                } else {
#pragma unroll
                    for (int k = 0; k < K; ++k)
                        if (row_ok[k] && store_in_grid(op + (size_t)k * g.nx, 4, out, g, status))
                            store_f4(op + (size_t)k * g.nx, done[k], streaming);
                }
                op += plane_stride;
            }
        }
    } else {
        // M = 2R+1 accumulators per row; the accumulator of output plane z lives in slot
        // z mod M, so nothing is shifted: M planes per trip, slots known at compile time.
        // From 125 taps on, M copies of the plane body (M x 500 FFMA per row) no longer fit the
        // instruction cache (measured: 4 fetch stalls per issued instruction); there the body
        // exists once and the M accumulators rotate by register moves after every plane
        // (M moves against (2R+1)^3 FMAs).
        constexpr int M = 2 * R + 1;
        constexpr int UNR = R >= 2 ? 1 : M;              // copies of the plane body
        // The 125-point box takes a row's x neighbours as two more 128-bit loads from the plane instead
        // of shuffles plus halo words (fewer instructions and registers: 512^3 218 against 201 GPoints/s);
        // the 27-point box keeps the shuffles (769 against 752 in a short run; in a seconds-long run
        // under the power cap the loads are ahead, 676 against 654).
        constexpr bool kBoxRowsFromSmem = R >= 2;
        float4 T[K][M];
#pragma unroll
        for (int k = 0; k < K; ++k)
#pragma unroll
            for (int d = 0; d < M; ++d) T[k][d] = make_float4(0.f, 0.f, 0.f, 0.f);

        for (int i0 = 0; i0 < nplanes; i0 += UNR) {
            const bool ok = static_for<UNR>([&](auto uc) -> bool {
                constexpr int u = decltype(uc)::value;
                const int i = i0 + u;
                if (i >= nplanes) return true;
                if (!mbar_wait_bounded(full0 + 8 * s, ph, g.wait_polls)) return false;
                const float* pl = reinterpret_cast<const float*>(ring + (size_t)s * SLOT_BYTES);
                if constexpr (WRAP) {
                    if (edge_t || edge_b) {                            // uniform over the CTA
                        // The halo rows inside this warp's window of rows: the lane's own columns, the row's own
                        // halo columns (first and last lane; a tile in the middle of a row reads them) and,
                        // at an x face, the corner cells, which go into the halo rows of the column blocks.
                        float* plw = reinterpret_cast<float*>(ring + (size_t)s * SLOT_BYTES);
                        float* stw = plw + S::PLANE_BYTES / 4;
                        const float* ys = stw + 2 * S::XS_BYTES / 4;
                        const float* cs = ys + 2 * S::YS_BYTES / 4;
#pragma unroll
                        for (int rr = 0; rr < R; ++rr) {
#pragma unroll
                            for (int side = 0; side < 2; ++side) {     // 0: rows above the grid, 1: rows below it
                                const int r = side == 0 ? rr : row_b + rr;
                                const bool mine = (side == 0 ? edge_t : edge_b) && r < S::ROWS && r >= row0 &&
                                                  r < row0 + K + 2 * R;
                                if (!mine) continue;
                                const float* yrow = ys + side * (S::YS_BYTES / 4) + rr * PX;
                                *reinterpret_cast<float4*>(plw + r * PX + HX + 4 * lane) =
                                    *reinterpret_cast<const float4*>(yrow + HX + 4 * lane);
                                if (lane == 0) *reinterpret_cast<float4*>(plw + r * PX) = *reinterpret_cast<const float4*>(yrow);
                                if (lane == 31)
                                    *reinterpret_cast<float4*>(plw + r * PX + HX + kStreamTX) =
                                        *reinterpret_cast<const float4*>(yrow + HX + kStreamTX);
                                if (edge_l && lane == 1)
                                    *reinterpret_cast<float4*>(stw + r * 4) =
                                        *reinterpret_cast<const float4*>(cs + (2 * side) * (S::CS_BYTES / 4) + rr * 4);
                                if (edge_r && lane == 2)
                                    *reinterpret_cast<float4*>(stw + S::XS_BYTES / 4 + r * 4) =
                                        *reinterpret_cast<const float4*>(cs + (2 * side + 1) * (S::CS_BYTES / 4) + rr * 4);
                            }
                        }
                        // later TMA copies into this slot must not overtake these stores
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                    }
                }
                const float* colp = pl + row0 * PX + HX + 4 * lane;
                float v[K + 2 * R][4 + 2 * R];
#pragma unroll
                for (int kk = 0; kk < K + 2 * R; ++kk) {
                    const float4 ctr = *reinterpret_cast<const float4*>(colp + kk * PX);
                    if constexpr (WRAP) {
                        const int o_row = (row0 + kk) * PX;
                        const int o_xs = S::PLANE_BYTES / 4 + (row0 + kk) * 4;
                        gather_row_split<R>(pl, o_row + HX + 4 * lane, edge_l ? o_xs : o_row,
                                            edge_r ? o_xs + S::XS_BYTES / 4 : o_row + HX + kStreamTX, lane, ctr, v[kk]);
                    } else {
                        gather_row<R, kBoxRowsFromSmem>(colp + kk * PX, pl + (row0 + kk) * PX, lane, ctr, v[kk]);
                    }
                }
                __syncwarp();
                mbar_arrive_if(lane == 0, empty0 + 8 * s);
                if (++s == nstage) { s = 0; ph ^= 1; }

                // (Packed FMAs do not pay here: their three operands are register pairs, so each of the
                // (2R+1)^3 weights would have to sit in two registers or be moved there before use; measured
                // on 512^3, 27 taps: 703 against 755 GPoints/s.)
#pragma unroll
                for (int k = 0; k < K; ++k) {
#pragma unroll
                    for (int d = 0; d < M; ++d) {         // this plane is tap dz = d - R of output i-(d-R)
                        float4& t = T[k][(u - d + R + 2 * M) % M];
                        float a[4];
                        if (d == 0) {                     // first contribution: starts the accumulator
#pragma unroll
                            for (int m = 0; m < 4; ++m) a[m] = bw.w[0][0][0] * v[k][m];
                        } else {
                            a[0] = t.x; a[1] = t.y; a[2] = t.z; a[3] = t.w;
                        }
#pragma unroll
                        for (int dy = 0; dy < M; ++dy)
#pragma unroll
                            for (int dx = 0; dx < M; ++dx) {
                                if (d == 0 && dy == 0 && dx == 0) continue;
                                const float wv = bw.w[d][dy][dx];
#pragma unroll
                                for (int m = 0; m < 4; ++m) a[m] = fmaf(wv, v[k + dy][m + dx], a[m]);
                            }
                        t = make_float4(a[0], a[1], a[2], a[3]);
                    }
                }
                if (i >= 2 * R) {                         // tap dz = +R was the last one of plane i-R
                    if (all_ok) {
#pragma unroll
                        for (int k = 0; k < K; ++k)
                            if (store_in_grid(op + (size_t)k * g.nx, 4, out, g, status))
                                store_f4(op + (size_t)k * g.nx, T[k][(u + R + 1) % M], streaming);
                    } else {
#pragma unroll
                        for (int k = 0; k < K; ++k)
                            if (row_ok[k] && store_in_grid(op + (size_t)k * g.nx, 4, out, g, status))
                                store_f4(op + (size_t)k * g.nx, T[k][(u + R + 1) % M], streaming);
                    }
                    op += plane_stride;
                }
                if constexpr (UNR == 1) {                 // next plane finds every accumulator one slot down
#pragma unroll
                    for (int k = 0; k < K; ++k) {
                        const float4 first = T[k][0];
#pragma unroll
                        for (int j = 0; j + 1 < M; ++j) T[k][j] = T[k][j + 1];
                        T[k][M - 1] = first;
                    }
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
stencil_stream_kernel(const __grid_constant__ CUtensorMap tmap_in, float* __restrict__ out,
                      const StreamGeom g,
                      const __grid_constant__ StarWeights<R> sw,
                      const __grid_constant__ BoxWeights<BOX ? R : 0> bw,
                      int* __restrict__ status) {
    stream_body<R, BOX, K, NW, false>(tmap_in, tmap_in, tmap_in, tmap_in, out, g, sw, bw, status);
}

// The sweep of a periodic grid: tmap_xs has boxes of 4 columns x ROWS rows, tmap_ys of PX columns x R rows,
// tmap_cs (boxes only) of 4 columns x R rows.
// The boxes need their register count capped to keep the CTAs per SM of the zero-boundary kernels
// (left alone the 27-point box takes 80 registers instead of 64 and the 125-point box 108 instead of 56).
template <int R, bool BOX, int K, int NW, int MINB>
constexpr int wrap_min_ctas() {
    if (!BOX) return MINB;
    const int threads = (NW + 1) * 32;
    const int regs = R == 1 ? (K == 1 ? 48 : K == 2 ? 64 : 96) : (K == 1 ? 56 : 96);   // of the zero-boundary kernels
    const int n = 65536 / (threads * regs);
    return n < 1 ? 1 : (n > 4 ? 4 : n);
}

template <int R, bool BOX, int K, int NW, int MINB>
__global__ void __launch_bounds__((NW + 1) * 32, wrap_min_ctas<R, BOX, K, NW, MINB>())
stencil_stream_wrap_kernel(const __grid_constant__ CUtensorMap tmap_in, const __grid_constant__ CUtensorMap tmap_xs,
                           const __grid_constant__ CUtensorMap tmap_ys, const __grid_constant__ CUtensorMap tmap_cs,
                           float* __restrict__ out, const StreamGeom g,
                           const __grid_constant__ StarWeights<R> sw,
                           const __grid_constant__ BoxWeights<BOX ? R : 0> bw, int* __restrict__ status) {
    stream_body<R, BOX, K, NW, true>(tmap_in, tmap_xs, tmap_ys, tmap_cs, out, g, sw, bw, status);
}

}  // namespace stencil
