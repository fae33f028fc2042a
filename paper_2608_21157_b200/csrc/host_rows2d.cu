// Host side of the 2D kernels (fp32): single sweeps and temporal blocking.
#include "host.h"
#include "kernel_rows2d.cuh"
#include "kernel_rows2d_fused.cuh"

namespace stencil_host {

template <int R, bool BOX, int YB, int NW>
cudaError_t launch_rows2d_t(const stencil_plan_s* p, const CUtensorMap& map, float* out, const Rows2DGeom& g,
                            int grid, size_t smem, cudaStream_t st) {
    Weights2D<R> wt;
    pack_taps2d<float, R>(p, wt);
    return launch_kernel(&stencil_rows2d_kernel<R, BOX, YB, NW>, grid, NW * 32, smem, st, p->chained, map, out, g,
                         wt, p->d_status);
}

template <int R, bool BOX, int YB, int NW>
Rows2DConfig make_rows2d() {
    Rows2DConfig c;
    c.radius = R; c.box = BOX; c.YB = YB; c.NW = NW;
    c.px = StreamHalo<R>::PX;
    c.batch_bytes = Rows2DShape<YB, StreamHalo<R>::PX>::BATCH_BYTES;
    c.kernel = reinterpret_cast<const void*>(&stencil_rows2d_kernel<R, BOX, YB, NW>);
    c.launch = &launch_rows2d_t<R, BOX, YB, NW>;
    return c;
}

const std::vector<Rows2DConfig>& rows2d_configs() {
    static const std::vector<Rows2DConfig> v = {
        make_rows2d<1, false, 8, 8>(), make_rows2d<2, false, 8, 8>(), make_rows2d<3, false, 8, 8>(),
        // the radius-4 star runs better in CTAs of 4 warps (725 against 668 GPoints/s on 10240^2)
        make_rows2d<4, false, 8, 4>(),
        make_rows2d<1, true, 8, 8>(),  make_rows2d<2, true, 8, 8>(),  make_rows2d<3, true, 8, 8>(),
        // 81 taps: batches of 4 rows and 16 warps per CTA (twice the warps per SM) measured 329
        // against 286 GPoints/s on 10240^2; the smaller boxes gain nothing from it
        make_rows2d<4, true, 4, 16>(),
        // stars of radius 5..8: batches with 8 halo columns per side
        make_rows2d<5, false, 8, 8>(), make_rows2d<6, false, 8, 8>(), make_rows2d<7, false, 8, 8>(),
        make_rows2d<8, false, 8, 8>(),
    };
    return v;
}

const Rows2DConfig* find_rows2d_cfg(int radius, bool box) {
    for (const Rows2DConfig& c : rows2d_configs())
        if (c.radius == radius && c.box == box) return &c;
    return nullptr;
}

template <int R, bool BOX, int T, int YB, int NW>
cudaError_t launch_rows2d_fused_t(const stencil_plan_s* p, const CUtensorMap& map, float* out,
                                  const Rows2DFusedGeom& g, int grid, size_t smem, cudaStream_t st) {
    Weights2D<R> wt;
    pack_taps2d<float, R>(p, wt);
    return launch_kernel(&stencil_rows2d_fused_kernel<R, BOX, T, YB, NW>, grid, NW * 32, smem, st, p->chained, map,
                         out, g, wt, p->d_status);
}

template <int R, bool BOX, int T, int YB, int NW>
Rows2DFusedConfig make_rows2d_fused() {
    Rows2DFusedConfig c;
    c.radius = R; c.box = BOX; c.T = T; c.YB = YB; c.NW = NW; c.batch_bytes = Rows2DShape<YB>::BATCH_BYTES;
    c.kernel = reinterpret_cast<const void*>(&stencil_rows2d_fused_kernel<R, BOX, T, YB, NW>);
    c.launch = &launch_rows2d_fused_t<R, BOX, T, YB, NW>;
    return c;
}

// One depth per operator: the deepest with (T - 1) * R <= 4 (the columns a strip spoils must stay inside
// its end lanes) that the operator's arithmetic leaves room for.
const std::vector<Rows2DFusedConfig>& rows2d_fused_configs() {
    static const std::vector<Rows2DFusedConfig> v = {
        make_rows2d_fused<1, false, 4, 8, 8>(), make_rows2d_fused<1, true, 4, 8, 8>(),
        make_rows2d_fused<2, false, 3, 8, 8>(), make_rows2d_fused<2, true, 2, 8, 8>(),
        make_rows2d_fused<3, false, 2, 8, 8>(), make_rows2d_fused<4, false, 2, 8, 8>(),
    };
    return v;
}

const Rows2DFusedConfig* pick_fused2d(const stencil_plan_s* p) {
    if (p->ndim != 2 || p->nx % 4 != 0 || p->fuse_steps == 1) return nullptr;
    for (const Rows2DFusedConfig& c : rows2d_fused_configs())
        if (c.radius == p->radius && c.box == (p->shape == STENCIL_BOX) && (p->fuse_steps == 0 || p->fuse_steps == c.T))
            return (p->boundary == STENCIL_PERIODIC && !shell_fits(p, c.T * p->radius)) ? nullptr : &c;
    return nullptr;
}

// Upper limit of the rows per (strip, chunk) unit of a 2D sweep.  The sweeps that are bound by
// memory (stars, the 9-point box) run best as many short units that the hardware scheduler
// balances, like the 3D ones: about 32 rows, more for wide stars whose 2R halo rows are re-read
// by every unit (10240^2, GPoints/s, short vs one wave of long units: 5-point 791 vs 700,
// 17-point star 667 vs 545, FP64 5-point 410 vs 361).  The boxes from 25 taps on are bound by
// the FMA pipe and keep the one-wave rule (49-point: 526 vs 488).
int short_chunk_2d(const stencil_plan_s* p, int YB) {
    const int R = p->radius;
    if (p->shape == STENCIL_BOX && R >= 2) return 0x7fffffff;
    const int target = std::max(32, 16 * R);
    const int nbatch = std::max(1, (target + 2 * R + YB / 2) / YB);
    return std::max(1, nbatch * YB - 2 * R);
}

// 2D grids: one warp per (128-column strip, chunk of rows).  dst[y_begin, y_end) = one sweep of
// src; the whole grid when y_end <= y_begin.
int launch_rows2d(stencil_plan_s* p, const float* src, float* dst, cudaStream_t st, int y_begin, int y_end) {
    if (y_end <= y_begin) { y_begin = 0; y_end = p->ny; }
    const int span = y_end - y_begin;
    const Rows2DConfig* cfg = p->rows2d_cfg;
    const CUtensorMap* map = nullptr;
    const bool periodic = p->boundary == STENCIL_PERIODIC;
    int rc;
    if (periodic) {
        int pnx, pny, pnz;
        const float* padded = nullptr;
        if ((rc = pad_periodic(p, src, st, &padded, &pnx, &pny, &pnz)) != STENCIL_OK) return rc;
        rc = get_tensor_map(p, cfg, cfg->px, cfg->YB, padded, &map, pnx, pny, pnz);
    } else {
        rc = get_tensor_map(p, cfg, cfg->px, cfg->YB, src, &map);
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
    g.strips = (p->nx + kStreamTX - 1) / kStreamTX;
    g.stages = stages;
    g.in_off_x = periodic ? kPadX : 0;
    g.in_off_y = periodic ? p->radius : 0;
    int chunk = p->chunk_z;                          // the streamed axis of a 2D grid is y
    if (chunk <= 0) {
        // As many (strip, chunk) units as fill the machine's warp slots once (two CTAs per SM),
        // never more: a second, partial wave of long units would double the run time.  A unit
        // reads chunk + 2R rows in batches of YB, so chunk + 2R is made a whole number of
        // batches; small grids end up with one batch per warp and as many warps as rows allow.
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
    g.y_begin = y_begin; g.y_end = y_end;
    g.wait_polls = p->wait_polls; g.drop_batch = p->drop_plane;
    STENCIL_SET_OUT_POINTS(g, p);
    const int64_t units = (int64_t)g.strips * g.nchunks;
    const int64_t grid64 = (units + cfg->NW - 1) / cfg->NW;
    if (grid64 > 0x7fffffffLL) return STENCIL_ERR_UNSUPPORTED;
    if (cfg->launch(p, *map, dst, g, (int)grid64, smem, st) != cudaSuccess) return STENCIL_ERR_CUDA;
    p->launches++;
    return STENCIL_OK;
}

// One fused pass: dst = S^nlev(src), nlev <= cfg->T.
// One fused pass of a 2D grid: nlev time steps (1..T) from src to dst.
int launch_rows2d_fused(stencil_plan_s* p, const float* src, float* dst, int nlev, cudaStream_t st) {
    const Rows2DFusedConfig* cfg = p->fused2d_cfg;
    const CUtensorMap* map = nullptr;
    int rc = get_tensor_map(p, cfg, kStreamPX, cfg->YB, src, &map);
    if (rc != STENCIL_OK) return rc;
    // two batches per warp: the small ring lets three CTAs share an SM (measured on 10240^2: 2082 G
    // updates/s against 1671 with three batches and 1214 with four)
    int stages = p->stages > 0 ? std::min(p->stages, kMaxStages) : 2;
    auto smem_for = [&](int s_) { return (size_t)cfg->NW * s_ * cfg->batch_bytes + 128 + (size_t)cfg->NW * kMaxStages * 8; };
    while (stages > 2 && smem_for(stages) > kMaxSmemBytes) --stages;      // a ring deeper than shared memory holds is cut back
    const size_t smem = smem_for(stages);
    if (smem > kMaxSmemBytes) return STENCIL_ERR_UNSUPPORTED;
    const int occ = kernel_limits(cfg->kernel, cfg->NW * 32, smem, p->device, cfg->lim, true);
    if (occ < 0) return STENCIL_ERR_CUDA;
    Rows2DFusedGeom g;
    g.ny = p->ny; g.nx = p->nx;
    g.strips = (p->nx + kFused2DTile - 1) / kFused2DTile;
    g.stages = stages;
    g.nlev = nlev;
    g.wait_polls = p->wait_polls; g.drop_batch = p->drop_plane;
    STENCIL_SET_OUT_POINTS(g, p);
    int chunk = p->chunk_z;                          // the streamed axis of a 2D grid is y
    if (chunk <= 0) {
        // A unit reads chunk + 2*nlev*R rows in batches of YB and recomputes the 2*nlev*R extra ones at
        // every level, so chunks should be long; as many (strip, chunk) units as fill the machine's
        // resident warp slots once, never more (10240^2: 248-row chunks 2082 G updates/s, 504-row
        // chunks, half a wave, 1479; 120-row chunks 1843).
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

}  // namespace stencil_host
