// Launch geometry of the tiled kernels: plain structs the host fills in and passes by value, and
// the few constants both sides need.
#pragma once

namespace stencil {

constexpr int kStreamTX = 128;            // tile width (points) of the fp32 kernels; one warp spans a row
constexpr int kMaxStages = 8;             // deepest shared-memory ring
constexpr int kPadX = 4;                  // halo columns per side of the padded copy of a periodic grid

struct StreamGeom {
    int nz, ny, nx;
    int tiles_x, tiles_y;
    int z_begin, z_end;         // output planes of this launch: [z_begin, z_end), normally [0, nz)
    int chunk_z;                // planes of output per CTA
    int stages;                 // depth of the plane ring
    int streaming_store;        // 1: st.global.cs
    int in_off_x, in_off_y, in_off_z;   // added to every TMA coordinate: non-zero when the input is a
                                // padded copy of the grid (periodic boundary), else 0
    unsigned wait_polls;        // cap of every bounded wait
    int drop_plane;             // test hook: the producer never loads this plane of a CTA (-1: none)
#ifdef STENCIL_DEBUG
    long long out_points;       // debug build: the extent of the output grid that every store is checked against
#endif
};

// (a multiple of 16 bytes, so that the kernel parameters behind it keep their 16-byte alignment: without it the
// fused kernels take four more registers)
struct alignas(16) FusedGeom {
    int nz, ny, nx;
    int tiles_x, tiles_y;
    int tile_x, tile_y;        // output tile (interior) size
    int halo_x, halo_y;        // region = tile + 2*halo; halo_x is a multiple of 4
    int chunk_z;               // planes per CTA over planes [0, nz - rest_z) of every region: main_ctas CTAs
    int stages;
    int nlev;                  // time steps advanced by this pass, 1..T
    unsigned wait_polls;       // cap of every bounded wait
    int drop_plane;            // test hook: a CTA never loads its input plane of this index (-1: none)
    int rest_z, rest_chunk;    // the last rest_z planes of every region go to further CTAs, rest_chunk planes each
    int main_ctas;
#ifdef STENCIL_DEBUG
    long long out_points;       // debug build: the extent of the output grid that every store is checked against
#endif
};

struct Rows2DGeom {
    int ny, nx;
    int strips;                 // ceil(nx / 128)
    int chunk_y;                // output rows per warp
    int nchunks;
    int stages;                 // batches in a warp's ring
    int in_off_x, in_off_y;     // added to the TMA coordinates (padded input of a periodic grid), else 0
    int y_begin, y_end;         // output rows of this launch (the whole grid: 0, ny)
    unsigned wait_polls;        // cap of every bounded wait
    int drop_batch;             // test hook: a warp never loads its input batch of this index (-1: none)
#ifdef STENCIL_DEBUG
    long long out_points;       // debug build: the extent of the output grid that every store is checked against
#endif
};

struct Rows2DFusedGeom {
    int ny, nx;
    int strips;                 // ceil(nx / kFused2DTile)
    int chunk_y;                // output rows per warp
    int nchunks;
    int stages;                 // batches in a warp's ring
    int nlev;                   // time steps advanced by this pass, 1..T
    unsigned wait_polls;        // cap of every bounded wait
    int drop_batch;             // test hook: a warp never loads its input batch of this index (-1: none)
#ifdef STENCIL_DEBUG
    long long out_points;       // debug build: the extent of the output grid that every store is checked against
#endif
};

}  // namespace stencil
