// Host side of the 3D single-sweep kernels (fp32): configurations, chunking, launches.
#include "host.h"
#include "kernel_stream.cuh"

namespace stencil_host {

template <int R, bool BOX, int K, int NW, int MINB>
cudaError_t launch_stream_t(const stencil_plan_s* p, const StreamConfig&, const CUtensorMap& map,
                            float* out, const StreamGeom& g, int grid, size_t smem, cudaStream_t st) {
    StarWeights<R> sw;
    BoxWeights<BOX ? R : 0> bw;
    pack_taps3d<float, R, BOX>(p, sw, bw);
    return launch_kernel(&stencil_stream_kernel<R, BOX, K, NW, MINB>, grid, StreamShape<R, K, NW>::THREADS, smem,
                         st, p->chained, map, out, g, sw, bw, p->d_status);
}

template <int R, bool BOX, int K, int NW, int MINB>
cudaError_t launch_stream_wrap_t(const stencil_plan_s* p, const CUtensorMap& map, const CUtensorMap& map_xs,
                                 const CUtensorMap& map_ys, const CUtensorMap& map_cs, float* out,
                                 const StreamGeom& g, int grid, size_t smem, cudaStream_t st) {
    StarWeights<R> sw;
    BoxWeights<BOX ? R : 0> bw;
    pack_taps3d<float, R, BOX>(p, sw, bw);
    return launch_kernel(&stencil_stream_wrap_kernel<R, BOX, K, NW, MINB>, grid, StreamShape<R, K, NW>::THREADS, smem,
                         st, p->chained, map, map_xs, map_ys, map_cs, out, g, sw, bw, p->d_status);
}

template <int R, bool BOX, int K, int NW, int MINB>
StreamConfig make_cfg() {
    using S = StreamShape<R, K, NW>;
    StreamConfig c;
    c.radius = R; c.box = BOX; c.K = K; c.NW = NW; c.tile_y = S::TY;
    c.plane_bytes = S::PLANE_BYTES; c.box_rows = S::ROWS; c.threads = S::THREADS;
    c.px = StreamHalo<R>::PX;
    c.kernel = reinterpret_cast<const void*>(&stencil_stream_kernel<R, BOX, K, NW, MINB>);
    c.launch = &launch_stream_t<R, BOX, K, NW, MINB>;
    c.kernel_wrap = nullptr; c.launch_wrap = nullptr; c.stage_bytes = 0;
    if constexpr (R <= 4) {
        c.kernel_wrap = reinterpret_cast<const void*>(&stencil_stream_wrap_kernel<R, BOX, K, NW, MINB>);
        c.launch_wrap = &launch_stream_wrap_t<R, BOX, K, NW, MINB>;
        c.stage_bytes = S::STAGE_BYTES;
    }
    return c;
}

// First entry of a (radius, box) group is the default; the others are reachable
// through STENCIL_KEY_TILE_Y / STENCIL_KEY_ROWS_PER_THREAD.
const std::vector<StreamConfig>& stream_configs() {
    // tile heights 14 and 28 (7 consumer warps + the producer = 256 threads) exist
    // because 4 x 37 tiles of 128 x 14 cover a 512 x 512 plane with one tile per SM
    static const std::vector<StreamConfig> v = {
        make_cfg<1, false, 2, 8, 1>(),  make_cfg<1, false, 2, 7, 4>(),  make_cfg<1, false, 4, 8, 1>(),
        make_cfg<1, false, 4, 7, 1>(),  make_cfg<1, false, 1, 8, 1>(),
        make_cfg<2, false, 2, 8, 1>(),  make_cfg<2, false, 2, 7, 1>(),  make_cfg<2, false, 4, 8, 1>(),
        // radius 3: four rows per thread (32-row tiles: the 6 halo rows are 19 % of a plane instead
        // of 43 % with 14-row tiles) measured 799 against 667 GPoints/s on 512^3
        make_cfg<3, false, 4, 8, 1>(),  make_cfg<3, false, 2, 8, 2>(),  make_cfg<3, false, 2, 7, 2>(),
        make_cfg<4, false, 2, 8, 2>(),  make_cfg<4, false, 2, 7, 2>(),  make_cfg<4, false, 4, 8, 1>(),
        make_cfg<4, false, 2, 16, 1>(),
        // radius 5..8 (8-float halo columns): one row per thread, the 2R accumulators per row leave no
        // registers for more; 16-row tiles halve the share of the 2R halo rows
        make_cfg<5, false, 1, 16, 1>(), make_cfg<5, false, 1, 8, 2>(),
        make_cfg<6, false, 1, 16, 1>(), make_cfg<6, false, 1, 8, 2>(),
        make_cfg<7, false, 1, 16, 1>(), make_cfg<7, false, 1, 8, 2>(),
        make_cfg<8, false, 1, 16, 1>(), make_cfg<8, false, 1, 8, 2>(),
        make_cfg<1, true, 2, 8, 1>(),   make_cfg<1, true, 2, 7, 4>(),   make_cfg<1, true, 4, 8, 1>(),
        make_cfg<1, true, 4, 7, 1>(),   make_cfg<1, true, 1, 8, 1>(),
        // 125 taps: one row per thread (56 registers, twice the warps of two rows per thread)
        // keeps the FMA pipe busier: 165 against 122 GPoints/s on 512^3
        // (a 7-row variant, whole waves on 512^2 planes, measured 153: not kept)
        make_cfg<2, true, 1, 8, 1>(),   make_cfg<2, true, 1, 16, 1>(),
        make_cfg<2, true, 2, 8, 1>(),   make_cfg<2, true, 2, 7, 1>(),
    };
    return v;
}

const StreamConfig* find_stream_cfg(int radius, bool box, int tile_y, int rows_per_thread) {
    for (const StreamConfig& c : stream_configs())
        if (c.radius == radius && c.box == box && (tile_y == 0 || c.tile_y == tile_y) &&
            (rows_per_thread == 0 || c.K == rows_per_thread))
            return &c;
    return nullptr;
}

size_t stream_smem_bytes(const StreamConfig* cfg, int stages) {
    return (size_t)stages * cfg->plane_bytes + 128 + 2 * kMaxStages * sizeof(uint64_t);
}

// Resident CTAs per SM of a configuration at a given ring depth on the plan's device (asked once per size),
// -1 if the ring does not fit shared memory.
int stream_occupancy(const stencil_plan_s* p, const StreamConfig* cfg, int stages) {
    const size_t smem = stream_smem_bytes(cfg, stages);
    if (smem > kMaxSmemBytes) return -1;
    return kernel_limits(cfg->kernel, cfg->threads, smem, p->device, cfg->lim, true);
}

// The sweeps with few FMAs per point are bound by HBM: there many short CTAs work
// best (the hardware scheduler balances them, and CTAs that outlive the others
// simply get more bandwidth).  The others are bound by instruction issue: there
// every SM must get the same amount of work, so the grid is cut into whole waves.
bool issue_bound(const stencil_plan_s* p) {
    return (p->shape == STENCIL_STAR && p->radius >= 3) || (p->shape == STENCIL_BOX && p->radius >= 2);
}

// The 7-point star runs best in very short chunks: the CTAs in flight then span only a few dozen
// planes, whose input stays in L2 until the neighbouring chunks have read their two halo planes
// from it (with 32-plane chunks the in-flight planes exceed L2 and the halo planes are fetched
// from DRAM twice).  512^3: 8 planes 820 GPoints/s, 16: 788, 32: 763; FP64 417 / 408 / 396.
// Grids whose planes hold more tiles than the machine has CTA slots run one layer of chunks at
// a time, so the halo planes miss L2 anyway: there 16 planes, which lose less to them.  Small
// grids pick, among 8..12 planes, the length whose CTAs fill whole waves best.
int short_chunk_star1(int nz, int64_t tiles, int64_t slots) {
    if (tiles > slots) return 16;
    if (tiles * ((nz + 7) / 8) >= 4 * slots) return 8;
    int best_chunk = 8;
    double best = 1e300;
    for (int c = 8; c <= 12; ++c) {
        const int64_t ctas = tiles * ((nz + c - 1) / c);
        const double cost = (double)((ctas + slots - 1) / slots) * (c + 4);
        if (cost < best * 0.999) { best = cost; best_chunk = c; }
    }
    return best_chunk;
}

// Planes of output per CTA, and the relative cost of the launch, for one configuration.
int choose_chunk(const stencil_plan_s* p, const StreamConfig* cfg, int stages, double* cost_out,
                 int span = 0) {
    const int R = p->radius;
    const int nz = span > 0 ? span : p->nz;      // planes this launch covers
    const int tiles = ((p->nx + kStreamTX - 1) / kStreamTX) * ((p->ny + cfg->tile_y - 1) / cfg->tile_y);
    const int occ = std::max(1, stream_occupancy(p, cfg, stages));
    const int slots = occ * plan_sms(p);
    if (!issue_bound(p)) {
        // measured on 512^3: 32-plane chunks (several thousand short CTAs) beat every longer chunk
        int chunk = nz >= 64 ? 32 : nz;
        if (p->shape == STENCIL_STAR && R == 1 && nz >= 16) {
            chunk = short_chunk_star1(nz, tiles, slots);
        } else if (nz >= 16 && (int64_t)tiles * ((nz + 31) / 32) < 4 * (int64_t)slots) {
            // A grid that does not cut into several machines' worth of 32-plane CTAs: the CTAs no longer
            // balance themselves, so z is cut into the number of chunks (of 8 to 32 planes) whose CTAs
            // fill whole waves of the resident slots at the least cost, a chunk costing its planes, its
            // 2R halo planes and the start-up of its pipeline.  GPoints/s, this rule against 32 planes,
            // 27-point box / 13-point star: 256^3 632 vs 456 / 727 vs 478, 128 x 256 x 256 556 vs 338 /
            // 635 vs 400, 64 x 512 x 512 624 vs 436 / 712 vs 705.  (Chunks longer than 32 planes lose even
            // where they fill one wave exactly: 384^3 box 655 against 742.)
            double best = 1e300;
            for (int nch = (nz + 31) / 32; nch <= std::max(1, nz / 8); ++nch) {
                const int c = (nz + nch - 1) / nch;
                const int64_t ctas = (int64_t)tiles * ((nz + c - 1) / c);
                const double cost = (double)((ctas + slots - 1) / slots) * (c + 2 * R + 4.0);
                if (cost < best * 0.999) { best = cost; chunk = c; }
            }
        }
        if (cost_out) {
            const int64_t ctas = (int64_t)tiles * ((nz + chunk - 1) / chunk);
            *cost_out = ((double)ctas / slots + 0.5) * occ * (chunk + 2 * R) * cfg->tile_y;
        }
        return chunk;
    }
    const double fill = 4.0;                       // pipeline start-up, in planes
    int best_chunk = nz;
    double best = 1e300;
    const int max_chunks = std::max(1, nz / std::max(8 * R, 16));
    for (int nch = 1; nch <= max_chunks; ++nch) {
        const int chunk = (nz + nch - 1) / nch;
        const int real_nch = (nz + chunk - 1) / chunk;
        const int64_t ctas = (int64_t)tiles * real_nch;
        const double waves = (double)((ctas + slots - 1) / slots);
        // CTAs resident together share the SM, so a wave of `occ` CTAs per SM costs occ units
        const double cost = waves * occ * (chunk + 2 * R + fill) * cfg->tile_y;
        if (cost < best * 0.999) { best = cost; best_chunk = chunk; }
    }
    if (cost_out) *cost_out = best;
    return best_chunk;
}

// One sweep of a periodic grid with the kernel that wraps all three axes itself (see stream_body).
// Called under a zero-boundary view of the plan; the tensor maps are copied out of the plan's cache
// at once, since a later entry may move the earlier ones.
int launch_stream_wrap(stencil_plan_s* p, const StreamConfig* cfg, int stages, const float* src, float* dst,
                       cudaStream_t st) {
    if (!cfg->launch_wrap) return STENCIL_ERR_UNSUPPORTED;
    const char* key = reinterpret_cast<const char*>(cfg);
    const CUtensorMap* m = nullptr;
    CUtensorMap map, map_xs, map_ys, map_cs;
    int rc;
    if ((rc = get_tensor_map(p, key, cfg->px, cfg->box_rows, src, &m)) != STENCIL_OK) return rc;
    map = *m;
    if ((rc = get_tensor_map(p, key + 1, 4, cfg->box_rows, src, &m)) != STENCIL_OK) return rc;
    map_xs = *m;
    if ((rc = get_tensor_map(p, key + 2, cfg->px, p->radius, src, &m)) != STENCIL_OK) return rc;
    map_ys = *m;
    map_cs = map;                                   // the corner blocks: boxes only
    if (cfg->box) {
        if ((rc = get_tensor_map(p, key + 3, 4, p->radius, src, &m)) != STENCIL_OK) return rc;
        map_cs = *m;
    }
    const size_t smem = (size_t)stages * (cfg->plane_bytes + cfg->stage_bytes) + 128 + 2 * kMaxStages * sizeof(uint64_t);
    if (smem > kMaxSmemBytes) return STENCIL_ERR_UNSUPPORTED;
    if (kernel_limits(cfg->kernel_wrap, cfg->threads, smem, p->device, cfg->lim_wrap, false) < 0) return STENCIL_ERR_CUDA;
    StreamGeom g;
    g.in_off_x = g.in_off_y = g.in_off_z = 0;
    g.nz = p->nz; g.ny = p->ny; g.nx = p->nx;
    g.tiles_x = (p->nx + kStreamTX - 1) / kStreamTX;
    g.tiles_y = (p->ny + cfg->tile_y - 1) / cfg->tile_y;
    g.stages = stages;
    g.streaming_store = p->streaming_store;
    if (stream_occupancy(p, cfg, stages) <= 0) return STENCIL_ERR_UNSUPPORTED;
    int chunk = p->chunk_z > 0 ? p->chunk_z : choose_chunk(p, cfg, stages, nullptr, p->nz);
    chunk = std::max(1, std::min(chunk, p->nz));
    g.chunk_z = chunk;
    g.z_begin = 0; g.z_end = p->nz;
    g.wait_polls = p->wait_polls; g.drop_plane = p->drop_plane;
    STENCIL_SET_OUT_POINTS(g, p);
    const int64_t grid64 = (int64_t)g.tiles_x * g.tiles_y * ((p->nz + chunk - 1) / chunk);
    if (grid64 > 0x7fffffffLL) return STENCIL_ERR_UNSUPPORTED;
    if (cfg->launch_wrap(p, map, map_xs, map_ys, map_cs, dst, g, (int)grid64, smem, st) != cudaSuccess)
        return STENCIL_ERR_CUDA;
    p->launches++;
    return STENCIL_OK;
}

// dst[z_begin, z_end) = one sweep of src; the whole grid when z_end <= z_begin.
int launch_stream(stencil_plan_s* p, const float* src, float* dst, cudaStream_t st, int z_begin,
                  int z_end) {
    if (z_end <= z_begin) { z_begin = 0; z_end = p->nz; }
    const int span = z_end - z_begin;
    // ring depth: 5 for the issue-bound sweeps and the radius-2 star (750 against 732 GPoints/s), else 4
    const int stages = p->stages > 0 ? std::min(p->stages, kMaxStages)
                                     : (issue_bound(p) || (p->shape == STENCIL_STAR && p->radius == 2) ? 5 : 4);
    if (!p->stream_cfg_fixed && !p->stream_cfg_tuned && p->rows_per_thread == 0 && p->shape == STENCIL_STAR &&
        p->radius == 3) {
        // Radius 3: four rows per thread (128 x 32 tiles, little halo) win where the grid cuts into a
        // machine's worth of such tiles with chunks of 64 planes or more; smaller grids balance better on
        // two rows per thread (GPoints/s, four rows vs two: 512^3 797 vs 667; 300^3 440 vs 511; 128^3 91 vs
        // 140; 64 x 1024^2 697 vs 716).
        const int64_t big_tiles = (int64_t)((p->nx + kStreamTX - 1) / kStreamTX) * ((p->ny + 31) / 32);
        const bool plentiful = big_tiles * (span / 64) >= 2 * (int64_t)plan_sms(p);
        if (const StreamConfig* c = find_stream_cfg(3, false, 0, plentiful ? 4 : 2)) p->stream_cfg = c;
    }
    if (!p->stream_cfg_fixed && !p->stream_cfg_tuned) {
        // pick the tile height that balances this grid best (same rows per thread)
        const StreamConfig* best_cfg = p->stream_cfg;
        double best = 1e300;
        for (const StreamConfig& c : stream_configs()) {
            if (c.radius != p->radius || c.box != (p->shape == STENCIL_BOX) || c.K != p->stream_cfg->K) continue;
            if (stream_occupancy(p, &c, stages) <= 0) continue;
            double cost = 0;
            choose_chunk(p, &c, stages, &cost);
            if (cost < best * 0.98) { best = cost; best_cfg = &c; }
        }
        p->stream_cfg = best_cfg;
        p->stream_cfg_tuned = true;
    }
    const StreamConfig* cfg = p->stream_cfg;
    if (p->stream_wrap) return launch_stream_wrap(p, cfg, stages, src, dst, st);
    const CUtensorMap* map = nullptr;
    const bool periodic = p->boundary == STENCIL_PERIODIC;
    int rc;
    if (periodic) {
        int pnx, pny, pnz;
        const float* padded = nullptr;
        if ((rc = pad_periodic(p, src, st, &padded, &pnx, &pny, &pnz)) != STENCIL_OK) return rc;
        rc = get_tensor_map(p, cfg, cfg->px, cfg->box_rows, padded, &map, pnx, pny, pnz);
    } else {
        rc = get_tensor_map(p, cfg, cfg->px, cfg->box_rows, src, &map);
    }
    if (rc != STENCIL_OK) return rc;

    StreamGeom g;
    g.in_off_x = periodic ? kPadX : 0;
    g.in_off_y = periodic ? p->radius : 0;
    g.in_off_z = periodic ? p->radius : 0;
    g.nz = p->nz; g.ny = p->ny; g.nx = p->nx;
    g.tiles_x = (p->nx + kStreamTX - 1) / kStreamTX;
    g.tiles_y = (p->ny + cfg->tile_y - 1) / cfg->tile_y;
    g.stages = stages;
    g.streaming_store = p->streaming_store;
    const int tiles = g.tiles_x * g.tiles_y;
    if (stream_occupancy(p, cfg, stages) <= 0) return STENCIL_ERR_UNSUPPORTED;
    int chunk = p->chunk_z > 0 ? p->chunk_z : choose_chunk(p, cfg, stages, nullptr, span);
    chunk = std::max(1, std::min(chunk, span));
    g.chunk_z = chunk;
    g.z_begin = z_begin; g.z_end = z_end;
    g.wait_polls = p->wait_polls; g.drop_plane = p->drop_plane;
    STENCIL_SET_OUT_POINTS(g, p);
    const int nchunks = (span + chunk - 1) / chunk;
    const int64_t grid64 = (int64_t)tiles * nchunks;
    if (grid64 > 0x7fffffffLL) return STENCIL_ERR_UNSUPPORTED;
    const size_t smem = stream_smem_bytes(cfg, stages);
    if (cfg->launch(p, *cfg, *map, dst, g, (int)grid64, smem, st) != cudaSuccess) return STENCIL_ERR_CUDA;
    p->launches++;
    return STENCIL_OK;
}

}  // namespace stencil_host
