// Host side of the FP64 kernels: configurations and launches of the 2D and 3D sweeps and of 2D
// temporal blocking.
#include "host.h"
#include "kernel_rows2d_f64.cuh"
#include "kernel_rows2d_fused_f64.cuh"
#include "kernel_stream_f64.cuh"

namespace stencil_host {

template <int R, bool BOX, int YB, int NW>
cudaError_t launch_rows2d64_t(const stencil_plan_s* p, const CUtensorMap& map, double* out, const Rows2DGeom& g,
                              int grid, size_t smem, cudaStream_t st) {
    Weights2D64<R> wt;
    pack_taps2d<double, R>(p, wt);
    return launch_kernel(&stencil_rows2d_f64_kernel<R, BOX, YB, NW>, grid, NW * 32, smem, st, p->chained, map, out,
                         g, wt, p->d_status);
}

template <int R, bool BOX, int YB, int NW>
Rows2D64Config make_rows2d64() {
    Rows2D64Config c;
    c.radius = R; c.box = BOX; c.YB = YB; c.NW = NW; c.px = StreamHalo64<R>::PX;
    c.batch_bytes = Rows2D64Shape<YB, StreamHalo64<R>::PX>::BATCH_BYTES;
    c.kernel = reinterpret_cast<const void*>(&stencil_rows2d_f64_kernel<R, BOX, YB, NW>);
    c.launch = &launch_rows2d64_t<R, BOX, YB, NW>;
    return c;
}

const std::vector<Rows2D64Config>& rows2d64_configs() {
    static const std::vector<Rows2D64Config> v = {
        make_rows2d64<1, false, 8, 8>(), make_rows2d64<2, false, 8, 8>(), make_rows2d64<3, false, 8, 8>(),
        make_rows2d64<4, false, 8, 8>(), make_rows2d64<5, false, 8, 8>(), make_rows2d64<6, false, 8, 8>(),
        make_rows2d64<7, false, 8, 8>(), make_rows2d64<8, false, 8, 8>(),
        // the FP64 boxes from 25 taps on are bound by the FP64 pipe and run better with twice the warps
        // per SM (batches of 4 rows, 16 warps per CTA): 10240^2, 49 taps 291 against 265 GPoints/s, 25
        // taps 337 against 318
        make_rows2d64<1, true, 8, 8>(),  make_rows2d64<2, true, 4, 16>(),  make_rows2d64<3, true, 4, 16>(),
        make_rows2d64<4, true, 4, 8>(),
    };
    return v;
}

const Rows2D64Config* find_rows2d64_cfg(const stencil_plan_s* p) {
    if (p->ndim != 2 || (p->boundary != STENCIL_ZERO && p->nx % 2 != 0)) return nullptr;   // odd rows: apply_row_padded_f64
    if (p->radius > 4 && p->boundary == STENCIL_PERIODIC && !wrap_correction_fits(p)) return nullptr;
    for (const Rows2D64Config& c : rows2d64_configs())
        if (c.radius == p->radius && c.box == (p->shape == STENCIL_BOX)) return &c;
    return nullptr;
}

template <int R, bool BOX, int K, int NW, int MINB>
cudaError_t launch_stream64_t(const stencil_plan_s* p, const CUtensorMap& map, double* out, const StreamGeom& g,
                              int grid, size_t smem, cudaStream_t st) {
    StarWeights64<R> sw;
    BoxWeights64<BOX ? R : 0> bw;
    pack_taps3d<double, R, BOX>(p, sw, bw);
    return launch_kernel(&stencil_stream_f64_kernel<R, BOX, K, NW, MINB>, grid, Stream64Shape<R, K, NW>::THREADS,
                         smem, st, p->chained, map, out, g, sw, bw, p->d_status);
}

template <int R, bool BOX, int K, int NW, int MINB>
cudaError_t launch_stream64_wrap_t(const stencil_plan_s* p, const CUtensorMap& map, const CUtensorMap& map_xs,
                                   const CUtensorMap& map_ys, const CUtensorMap& map_cs, double* out,
                                   const StreamGeom& g, int grid, size_t smem, cudaStream_t st) {
    StarWeights64<R> sw;
    BoxWeights64<BOX ? R : 0> bw;
    pack_taps3d<double, R, BOX>(p, sw, bw);
    return launch_kernel(&stencil_stream_f64_wrap_kernel<R, BOX, K, NW, MINB>, grid, Stream64Shape<R, K, NW>::THREADS,
                         smem, st, p->chained, map, map_xs, map_ys, map_cs, out, g, sw, bw, p->d_status);
}

template <int R, bool BOX, int K, int NW, int MINB>
Stream64Config make_stream64() {
    using S = Stream64Shape<R, K, NW>;
    Stream64Config c;
    c.radius = R; c.box = BOX; c.tile_y = S::TY; c.plane_bytes = S::PLANE_BYTES; c.box_rows = S::ROWS;
    c.threads = S::THREADS; c.px = StreamHalo64<R>::PX;
    c.kernel = reinterpret_cast<const void*>(&stencil_stream_f64_kernel<R, BOX, K, NW, MINB>);
    c.launch = &launch_stream64_t<R, BOX, K, NW, MINB>;
    c.kernel_wrap = nullptr; c.launch_wrap = nullptr; c.stage_bytes = 0;
    if constexpr (R <= 4) {
        c.kernel_wrap = reinterpret_cast<const void*>(&stencil_stream_f64_wrap_kernel<R, BOX, K, NW, MINB>);
        c.launch_wrap = &launch_stream64_wrap_t<R, BOX, K, NW, MINB>;
        c.stage_bytes = S::STAGE_BYTES;
    }
    return c;
}

const std::vector<Stream64Config>& stream64_configs() {
    static const std::vector<Stream64Config> v = {
        // The wide stars need their register count capped at two CTAs per SM (the last template
        // argument): left alone the compiler takes 104 (R = 3) and 124 (R = 4) registers and a single
        // 288-thread CTA fits.  Measured on 512^3 (GPoints/s), rows per thread x consumer warps:
        // R = 3: 2 x 8 uncapped 285, capped 366, 4 x 4 capped 379; R = 4: 2 x 8 uncapped 273,
        // capped 313, 2 x 7 capped 323.
        make_stream64<1, false, 2, 8, 1>(), make_stream64<2, false, 2, 8, 1>(), make_stream64<3, false, 4, 4, 2>(),
        make_stream64<4, false, 2, 7, 2>(), make_stream64<1, true, 2, 8, 1>(), make_stream64<2, true, 1, 8, 1>(),
        make_stream64<5, false, 1, 8, 2>(), make_stream64<6, false, 1, 8, 2>(), make_stream64<7, false, 1, 8, 2>(),
        make_stream64<8, false, 1, 8, 2>(),
    };
    return v;
}

const Stream64Config* find_stream64_cfg(const stencil_plan_s* p) {
    if (p->ndim != 3 || (p->boundary != STENCIL_ZERO && p->nx % 2 != 0)) return nullptr;   // odd rows: apply_row_padded_f64
    if (p->radius > 4 && p->boundary == STENCIL_PERIODIC && !wrap_correction_fits(p)) return nullptr;
    for (const Stream64Config& c : stream64_configs())
        if (c.radius == p->radius && c.box == (p->shape == STENCIL_BOX)) return &c;
    return nullptr;
}

template <int R, bool BOX, int T, int YB, int NW>
cudaError_t launch_rows2d_fused64_t(const stencil_plan_s* p, const CUtensorMap& map, double* out,
                                    const Rows2DFusedGeom& g, int grid, size_t smem, cudaStream_t st) {
    Weights2D64<R> wt;
    pack_taps2d<double, R>(p, wt);
    return launch_kernel(&stencil_rows2d_fused_f64_kernel<R, BOX, T, YB, NW>, grid, NW * 32, smem, st, p->chained,
                         map, out, g, wt, p->d_status);
}

template <int R, bool BOX, int T, int YB, int NW>
Rows2DFused64Config make_rows2d_fused64() {
    Rows2DFused64Config c;
    c.radius = R; c.box = BOX; c.T = T; c.YB = YB; c.NW = NW; c.batch_bytes = Rows2D64Shape<YB>::BATCH_BYTES;
    c.kernel = reinterpret_cast<const void*>(&stencil_rows2d_fused_f64_kernel<R, BOX, T, YB, NW>);
    c.launch = &launch_rows2d_fused64_t<R, BOX, T, YB, NW>;
    return c;
}

// FP64 twin of rows2d_fused_configs(): radius <= 2 (one neighbour lane per side in the register exchange).
const std::vector<Rows2DFused64Config>& rows2d_fused64_configs() {
    static const std::vector<Rows2DFused64Config> v = {
        make_rows2d_fused64<1, false, 4, 8, 8>(), make_rows2d_fused64<1, true, 4, 8, 8>(),
        make_rows2d_fused64<2, false, 3, 8, 8>(), make_rows2d_fused64<2, true, 2, 8, 8>(),
    };
    return v;
}

const Rows2DFused64Config* pick_fused2d64(const stencil_plan_s* p) {
    if (p->ndim != 2 || p->nx % 2 != 0 || p->fuse_steps == 1) return nullptr;
    for (const Rows2DFused64Config& c : rows2d_fused64_configs())
        if (c.radius == p->radius && c.box == (p->shape == STENCIL_BOX) && (p->fuse_steps == 0 || p->fuse_steps == c.T))
            return (p->boundary == STENCIL_PERIODIC && !shell_fits(p, c.T * p->radius)) ? nullptr : &c;
    return nullptr;
}

int resolve_variant_f64(stencil_plan_s* p, int want) {
    const Rows2D64Config* c2 = find_rows2d64_cfg(p);
    const Stream64Config* c3 = find_stream64_cfg(p);
    if (want == STENCIL_VARIANT_AUTO) want = (c2 || c3) ? STENCIL_VARIANT_STREAM : STENCIL_VARIANT_GENERIC;
    if (want == STENCIL_VARIANT_GENERIC) {
        p->variant = want; p->rows2d64_cfg = nullptr; p->stream64_cfg = nullptr; p->fused2d64_cfg = nullptr;
        p->fused64_cfg = nullptr;
        return STENCIL_OK;
    }
    if (want == STENCIL_VARIANT_STREAM && (c2 || c3)) {
        p->variant = want; p->rows2d64_cfg = c2; p->stream64_cfg = c3;
        p->fused2d64_cfg = c2 ? pick_fused2d64(p) : nullptr;
        p->fused64_cfg = c3 ? pick_fused64(p) : nullptr;
        return STENCIL_OK;
    }
    return STENCIL_ERR_UNSUPPORTED;
}

// One fused pass of a 2D FP64 grid: nlev time steps (1..T) from src to dst.
int launch_rows2d_fused64(stencil_plan_s* p, const double* src, double* dst, int nlev, cudaStream_t st) {
    const Rows2DFused64Config* cfg = p->fused2d64_cfg;
    const CUtensorMap* map = nullptr;
    int rc = get_tensor_map_f64(p, cfg, kPX64, cfg->YB, src, &map);
    if (rc != STENCIL_OK) return rc;
    int stages = p->stages > 0 ? std::min(p->stages, kMaxStages) : 2;
    auto smem_for = [&](int s_) { return (size_t)cfg->NW * s_ * cfg->batch_bytes + 128 + (size_t)cfg->NW * kMaxStages * 8; };
    while (stages > 2 && smem_for(stages) > kMaxSmemBytes) --stages;      // a ring deeper than shared memory holds is cut back
    const size_t smem = smem_for(stages);
    if (smem > kMaxSmemBytes) return STENCIL_ERR_UNSUPPORTED;
    const int occ = kernel_limits(cfg->kernel, cfg->NW * 32, smem, p->device, cfg->lim, true);
    if (occ < 0) return STENCIL_ERR_CUDA;
    Rows2DFusedGeom g;
    g.ny = p->ny; g.nx = p->nx;
    g.strips = (p->nx + kFused2D64Tile - 1) / kFused2D64Tile;
    g.stages = stages;
    g.nlev = nlev;
    g.wait_polls = p->wait_polls; g.drop_batch = p->drop_plane;
    STENCIL_SET_OUT_POINTS(g, p);
    int chunk = p->chunk_z;
    if (chunk <= 0) {                                 // same sizing rule as the fp32 kernel
        const int H = nlev * p->radius;
        const int slots = occ * plan_sms(p) * cfg->NW;
        const int nch_max = std::max(1, slots / g.strips);
        const int chunk_min = (p->ny + nch_max - 1) / nch_max;
        int nbatch = std::max(1, (chunk_min + 2 * H + cfg->YB - 1) / cfg->YB);
        while (nbatch * cfg->YB - 2 * H < 1) ++nbatch;
        chunk = nbatch * cfg->YB - 2 * H;
    }
    chunk = std::max(1, std::min(chunk, p->ny));
    g.chunk_y = chunk;
    g.nchunks = (p->ny + chunk - 1) / chunk;
    const int64_t units = (int64_t)g.strips * g.nchunks;
    const int64_t grid64 = (units + cfg->NW - 1) / cfg->NW;
    if (grid64 > 0x7fffffffLL) return STENCIL_ERR_UNSUPPORTED;
    if (cfg->launch(p, *map, dst, g, (int)grid64, smem, st) != cudaSuccess) return STENCIL_ERR_CUDA;
    p->launches++;
    return STENCIL_OK;
}

// dst = one sweep of src; with begin < end only the output planes (3D) or rows (2D) [begin, end) on the tiled kernels.
int launch_sweep_f64(stencil_plan_s* p, const double* src, double* dst, cudaStream_t st, int begin, int end) {
    const int slow = p->ndim == 3 ? p->nz : p->ny;              // extent of the streamed axis
    if (end <= begin) { begin = 0; end = slow; }
    const int span = end - begin;
    if (p->variant == STENCIL_VARIANT_STREAM && p->stream64_cfg) {
        const Stream64Config* cfg = p->stream64_cfg;
        const CUtensorMap* map = nullptr;
        const bool periodic = p->boundary == STENCIL_PERIODIC;      // swept from a padded copy, as in fp32
        int rc;
        if (periodic) {
            int pnx, pny, pnz;
            const double* padded = nullptr;
            if ((rc = pad_periodic(p, src, st, &padded, &pnx, &pny, &pnz)) != STENCIL_OK) return rc;
            rc = get_tensor_map_f64(p, cfg, cfg->px, cfg->box_rows, padded, &map, pnx, pny, pnz);
        } else {
            rc = get_tensor_map_f64(p, cfg, cfg->px, cfg->box_rows, src, &map);
        }
        if (rc != STENCIL_OK) return rc;
        // the sweep that wraps a periodic grid itself: three tensor maps, copied out of the plan's cache at
        // once (a later entry may move the earlier ones), and the staged halo blocks beside every plane
        const bool wrap = p->stream_wrap && cfg->launch_wrap;
        if (p->stream_wrap && !wrap) return STENCIL_ERR_UNSUPPORTED;
        CUtensorMap map0, map_xs, map_ys, map_cs;
        if (wrap) {
            const char* key = reinterpret_cast<const char*>(cfg);
            map0 = *map;
            if ((rc = get_tensor_map_f64(p, key + 1, 4, cfg->box_rows, src, &map)) != STENCIL_OK) return rc;
            map_xs = *map;
            if ((rc = get_tensor_map_f64(p, key + 2, cfg->px, p->radius, src, &map)) != STENCIL_OK) return rc;
            map_ys = *map;
            map_cs = map0;                                // the corner blocks: boxes only
            if (cfg->box) {
                if ((rc = get_tensor_map_f64(p, key + 3, 4, p->radius, src, &map)) != STENCIL_OK) return rc;
                map_cs = *map;
            }
        }
        int stages = p->stages > 0 ? std::min(p->stages, kMaxStages) : (p->radius >= 3 ? 5 : 4);
        auto smem_for = [&](int s_) {
            return (size_t)s_ * (cfg->plane_bytes + (wrap ? cfg->stage_bytes : 0)) + 128 + 2 * kMaxStages * sizeof(uint64_t);
        };
        while (stages > 2 && smem_for(stages) > kMaxSmemBytes) --stages;      // a ring deeper than shared memory holds is cut back
        const size_t smem = smem_for(stages);
        if (smem > kMaxSmemBytes) return STENCIL_ERR_UNSUPPORTED;
        // resident CTAs per SM of the kernel this launch runs, asked once per device and size
        const int occ64 = wrap ? kernel_limits(cfg->kernel_wrap, cfg->threads, smem, p->device, cfg->lim_wrap, true)
                               : kernel_limits(cfg->kernel, cfg->threads, smem, p->device, cfg->lim, true);
        if (occ64 < 0) return STENCIL_ERR_CUDA;
        StreamGeom g;
        g.nz = p->nz; g.ny = p->ny; g.nx = p->nx;
        g.tiles_x = (p->nx + kStream64TX - 1) / kStream64TX;
        g.tiles_y = (p->ny + cfg->tile_y - 1) / cfg->tile_y;
        g.stages = stages;
        g.streaming_store = 0;
        g.z_begin = begin; g.z_end = end;
        g.in_off_x = periodic ? kPadX : 0;
        g.in_off_y = periodic ? p->radius : 0;
        g.in_off_z = periodic ? p->radius : 0;
        g.wait_polls = p->wait_polls; g.drop_plane = p->drop_plane;
        STENCIL_SET_OUT_POINTS(g, p);
        // many short CTAs, as for the bandwidth-bound fp32 sweeps; the wide stars re-read 2R halo
        // planes per chunk, so they get longer chunks (measured on 512^3)
        const int want_chunk = p->radius >= 3 ? 64 : 32;
        int chunk = p->chunk_z > 0 ? p->chunk_z : (span >= 2 * want_chunk ? want_chunk : span);
        const int64_t tiles64 = (int64_t)g.tiles_x * g.tiles_y, slots64 = (int64_t)occ64 * plan_sms(p);
        if (p->chunk_z <= 0 && p->shape == STENCIL_STAR && p->radius == 1 && span >= 16) {
            chunk = short_chunk_star1(span, tiles64, slots64);      // the 7-point star: very short chunks, as in fp32
        } else if (p->chunk_z <= 0 && span >= 16 && tiles64 * ((span + want_chunk - 1) / want_chunk) < 4 * slots64) {
            // a grid that does not cut into several machines' worth of CTAs: whole waves of chunks of 8 planes
            // or more, none longer than the usual length (the same rule as the fp32 sweeps)
            double best = 1e300;
            for (int n = (span + want_chunk - 1) / want_chunk; n <= std::max(1, span / 8); ++n) {
                const int c = (span + n - 1) / n;
                const int64_t ctas = tiles64 * ((span + c - 1) / c);
                const double cost = (double)((ctas + slots64 - 1) / slots64) * (c + 2 * p->radius + 4.0);
                if (cost < best * 0.999) { best = cost; chunk = c; }
            }
        }
        if (p->chunk_z <= 0 && (p->radius >= 4 || (p->shape == STENCIL_BOX && p->radius >= 2))) {
            // The radius-4 star is no longer bound by memory alone (25 DFMA and 15 shared-memory
            // loads per pair of points) and the 125-point box is bound by the FP64 pipe: every SM
            // should get the same number of planes and as
            // few re-read halo planes as possible, so z is cut into the number of chunks whose
            // CTAs fill whole waves of the two-per-SM slots at the least cost (512^3: one chunk,
            // 296 CTAs, 356 against 313 GPoints/s with 64-plane chunks).
            const int64_t tiles = (int64_t)g.tiles_x * g.tiles_y;
            const int64_t slots = 2 * (int64_t)plan_sms(p);
            double best = 1e300;
            for (int n = 1; n <= std::max(1, span / (4 * p->radius)); ++n) {
                const int c = (span + n - 1) / n;
                const int64_t ctas = tiles * ((span + c - 1) / c);
                const double cost = (double)((ctas + slots - 1) / slots) * (c + 2 * p->radius + 4.0);
                if (cost < best * 0.999) { best = cost; chunk = c; }
            }
        }
        chunk = std::max(1, std::min(chunk, span));
        g.chunk_z = chunk;
        const int64_t grid64 = (int64_t)g.tiles_x * g.tiles_y * ((span + chunk - 1) / chunk);
        if (grid64 > 0x7fffffffLL) return STENCIL_ERR_UNSUPPORTED;
        const cudaError_t err = wrap ? cfg->launch_wrap(p, map0, map_xs, map_ys, map_cs, dst, g, (int)grid64, smem, st)
                                     : cfg->launch(p, *map, dst, g, (int)grid64, smem, st);
        if (err != cudaSuccess) return STENCIL_ERR_CUDA;
        p->launches++;
        return STENCIL_OK;
    }
    if (p->variant == STENCIL_VARIANT_STREAM && p->rows2d64_cfg) {
        const Rows2D64Config* cfg = p->rows2d64_cfg;
        const CUtensorMap* map = nullptr;
        const bool periodic = p->boundary == STENCIL_PERIODIC;
        int rc;
        if (periodic) {
            int pnx, pny, pnz;
            const double* padded = nullptr;
            if ((rc = pad_periodic(p, src, st, &padded, &pnx, &pny, &pnz)) != STENCIL_OK) return rc;
            rc = get_tensor_map_f64(p, cfg, cfg->px, cfg->YB, padded, &map, pnx, pny, pnz);
        } else {
            rc = get_tensor_map_f64(p, cfg, cfg->px, cfg->YB, src, &map);
        }
        if (rc != STENCIL_OK) return rc;
        int stages = p->stages > 0 ? std::min(p->stages, kMaxStages) : 3;
        auto smem_for = [&](int s_) { return (size_t)cfg->NW * s_ * cfg->batch_bytes + 128 + (size_t)cfg->NW * kMaxStages * 8; };
        while (stages > 2 && smem_for(stages) > kMaxSmemBytes) --stages;      // a ring deeper than shared memory holds is cut back
        const size_t smem = smem_for(stages);
        if (smem > kMaxSmemBytes) return STENCIL_ERR_UNSUPPORTED;
        if (kernel_limits(cfg->kernel, cfg->NW * 32, smem, p->device, cfg->lim, false) < 0) return STENCIL_ERR_CUDA;
        Rows2DGeom g;
        g.ny = p->ny; g.nx = p->nx;
        g.strips = (p->nx + kStrip64 - 1) / kStrip64;
        g.stages = stages;
        g.in_off_x = periodic ? kPadX : 0;
        g.in_off_y = periodic ? p->radius : 0;
        int chunk = p->chunk_z;
        if (chunk <= 0) {                             // same sizing rule as the fp32 kernel
            const int R = p->radius;
            const int slots = 2 * plan_sms(p) * cfg->NW;
            const int nch_max = std::max(1, slots / g.strips);
            const int chunk_min = (span + nch_max - 1) / nch_max;
            int nbatch = std::max(1, (chunk_min + 2 * R + cfg->YB - 1) / cfg->YB);
            while (nbatch * cfg->YB - 2 * R < 1) ++nbatch;
            chunk = nbatch * cfg->YB - 2 * R;
            chunk = std::min(chunk, short_chunk_2d(p, cfg->YB));
        }
        chunk = std::max(1, std::min(chunk, span));
        g.chunk_y = chunk;
        g.nchunks = (span + chunk - 1) / chunk;
        g.y_begin = begin; g.y_end = end;
        g.wait_polls = p->wait_polls; g.drop_batch = p->drop_plane;
        STENCIL_SET_OUT_POINTS(g, p);
        const int64_t units = (int64_t)g.strips * g.nchunks;
        const int64_t grid64 = (units + cfg->NW - 1) / cfg->NW;
        if (grid64 > 0x7fffffffLL) return STENCIL_ERR_UNSUPPORTED;
        if (cfg->launch(p, *map, dst, g, (int)grid64, smem, st) != cudaSuccess) return STENCIL_ERR_CUDA;
        p->launches++;
        return STENCIL_OK;
    }
    return launch_generic_f64(p, src, dst, st);
}

int fp64_stream_tile_x() { return kStream64TX; }

}  // namespace stencil_host
