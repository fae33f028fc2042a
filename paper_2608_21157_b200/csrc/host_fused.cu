// Host side of 3D temporal blocking (fp32 and FP64): configurations, the default fusion rule, launches.
#include "host.h"
#include "kernel_fused.cuh"

namespace stencil_host {

template <typename E, int R, int T, int K, int XW, int NWY, int MODE>
cudaError_t launch_fused_t(const stencil_plan_s* p, const CUtensorMap& map, void* out, const FusedGeom& g,
                           int grid, size_t smem, cudaStream_t st) {
    StarTaps<E, R> sw;
    pack_star3d<E, R>(p, sw);
    return launch_kernel(&stencil_fused_kernel<E, R, T, K, XW, NWY, MODE>, grid,
                         FusedShape<R, K, XW, NWY, E>::THREADS, smem, st, p->chained, map, static_cast<E*>(out), g,
                         sw, p->d_status);
}

template <typename E, int R, int T, int K, int XW, int NWY>
FusedConfig make_fused_e() {
    using S = FusedShape<R, K, XW, NWY, E>;
    FusedConfig c;
    c.radius = R; c.T = T; c.K = K; c.XW = XW; c.NWY = NWY; c.box = false; c.f64 = sizeof(E) == 8;
    c.txe = S::TXE; c.tye = S::TYE; c.threads = S::THREADS; c.slot_bytes = S::SLOT_BYTES; c.pw = S::PW;
    c.kernel = reinterpret_cast<const void*>(&stencil_fused_kernel<E, R, T, K, XW, NWY, 0>);
    c.kernel_spec = reinterpret_cast<const void*>(&stencil_fused_kernel<E, R, T, K, XW, NWY, 1>);
    c.launch = &launch_fused_t<E, R, T, K, XW, NWY, 0>;
    c.launch_spec = &launch_fused_t<E, R, T, K, XW, NWY, 1>;
    c.kernel_wrap = nullptr; c.launch_wrap = nullptr;
    if constexpr (sizeof(E) == 4) {            // the pass of a periodic grid that wraps x and z itself: fp32 only
        c.kernel_wrap = reinterpret_cast<const void*>(&stencil_fused_kernel<E, R, T, K, XW, NWY, 2>);
        c.launch_wrap = &launch_fused_t<E, R, T, K, XW, NWY, 2>;
    }
    return c;
}

template <int R, int T, int K, int XW, int NWY>
FusedConfig make_fused() { return make_fused_e<float, R, T, K, XW, NWY>(); }

// First match of (radius, T, region width) wins; T == 0 / width == 0 match anything.
const std::vector<FusedConfig>& fused_configs() {
    static const std::vector<FusedConfig> v = {
        make_fused<1, 2, 4, 2, 8>(),  make_fused<1, 3, 4, 2, 8>(),  make_fused<1, 2, 4, 2, 4>(),
        make_fused<1, 2, 2, 2, 8>(),  make_fused<1, 2, 4, 4, 4>(),  make_fused<1, 2, 4, 3, 5>(),
        make_fused<1, 4, 2, 1, 16>(), make_fused<1, 2, 2, 1, 16>(), make_fused<1, 3, 2, 1, 16>(),
        make_fused<2, 2, 2, 1, 16>(),
    };
    return v;
}

const FusedConfig* find_fused_cfg(int radius, int T, int txe, int tye = 0) {
    for (const FusedConfig& c : fused_configs())
        if (c.radius == radius && (T == 0 || c.T == T) && (txe == 0 || c.txe == txe) && (tye == 0 || c.tye == tye))
            return &c;
    return nullptr;
}

// FP64: a lane holds two doubles, so a warp spans 64 columns and the regions are 128 (two CTAs per SM, or one of
// twice the height) or 256
// columns wide (XW = 4: 512 threads, one CTA per SM); 512 columns would take 1024 threads of 64 registers, which
// the two accumulators per row and level do not fit.
const std::vector<FusedConfig>& fused64_configs() {
    static const std::vector<FusedConfig> v = {
        make_fused_e<double, 1, 2, 4, 4, 4>(), make_fused_e<double, 1, 2, 4, 2, 4>(),
        make_fused_e<double, 1, 2, 2, 2, 8>(), make_fused_e<double, 1, 3, 2, 2, 8>(),
        make_fused_e<double, 1, 2, 4, 2, 8>(),
    };
    return v;
}

// Temporal blocking of an FP64 3D grid: the 7-point-like stars (radius 1), zero boundary, even rows.  Default:
// two steps per pass where the rows fill 80 % of the lanes of their regions: one 128- or 256-wide region per row,
// or, on wider rows, several 128-wide regions with 4 halo columns per side (two CTAs per SM, which the
// 256-wide regions do not allow).  Measured, G updates/s, fused against one launch per step: 256^3 461 / 381,
// 512 x 512 x 256 516 / 421, 512 x 512 x 128 620 / 408, 512^3 484 / 422 (five 128-wide regions per row; three
// 256-wide ones: 275); three steps per pass on 128-wide regions lose to two (445 against 620).
const FusedConfig* pick_fused64(const stencil_plan_s* p) {
    if (!p->f64 || p->ndim != 3 || p->shape != STENCIL_STAR || p->boundary != STENCIL_ZERO) return nullptr;
    if (p->nx % 2 != 0 || p->fuse_steps == 1) return nullptr;
    const bool forced = p->fuse_steps > 2 || p->tile_x != 0 || p->fused_tile_y != 0;
    const int width = p->nx <= 128 ? 128 : p->nx <= 256 ? 256 : 128;
    const int64_t regions = p->nx <= width ? 1 : (p->nx + (width - 8) - 1) / (width - 8);
    const double lanes_used = (double)p->nx / (double)(regions * width);
    // as in fp32, the 128-wide regions are 32 rows high (one CTA per SM) from 448 rows on: G updates/s, 16 / 32 rows,
    // nz x ny x nx: 512 x 512 x 128 619 / 666, 256 x 1024 x 128 622 / 708, 256 x 448 x 128 565 / 615, 256 x 384 x 128
    // 598 / 580, 256 x 256 x 128 530 / 491, 128 x 640 x 640 469 / 501, 512^3 488 / 490
    const int height = (width == 128 && p->ny >= 448) ? 32 : 16;
    for (const FusedConfig& c : fused64_configs()) {
        if (c.radius != p->radius) continue;
        if (forced) {
            if ((p->fuse_steps <= 1 || c.T == p->fuse_steps) && (p->tile_x == 0 || c.txe == p->tile_x) &&
                (p->fused_tile_y == 0 || c.tye == p->fused_tile_y))
                return &c;
            continue;
        }
        // (a caller that asks for two steps per pass gets them on the default width whatever the rows fill)
        if (c.T == 2 && c.txe == width && c.tye == height && (lanes_used >= 0.8 || p->fuse_steps == 2)) return &c;
    }
    return nullptr;
}

// Temporal blocking covers what the STREAM kernels cover, restricted to star stencils.
const FusedConfig* pick_fused_region(const stencil_plan_s* p);

const FusedConfig* pick_fused(const stencil_plan_s* p) {
    const FusedConfig* c = pick_fused_region(p);
    if (c && p->boundary == STENCIL_PERIODIC && !shell_fits(p, c->T * p->radius)) c = nullptr;
    return c;
}

const FusedConfig* pick_fused_region(const stencil_plan_s* p) {
    if (!stream_supported(p) || p->shape != STENCIL_STAR || p->ndim != 3) return nullptr;
    if (p->nx % 4 != 0) return nullptr;                   // ... over the row pitch, which padded rows exceed
    if (p->fuse_steps == 1) return nullptr;
    int txe = p->tile_x;
    // no preference for the region: the default below, also when the caller asks for its step count
    if ((p->fuse_steps == 0 || p->fuse_steps == 2) && txe == 0 && p->fused_tile_y == 0) {
        // Default: fuse two steps per pass when one region spans a whole row (no redundant
        // columns) and the row fills at least 80 % of the region's lanes.  Regions are 128, 256
        // (16 rows high with two CTAs per SM, which cover each other's barrier stalls, or 32 rows
        // high: see `height` below) or 512 columns wide (one CTA per SM, each plane
        // loaded as two TMA boxes).  With several regions per row the halo recomputation costs
        // more than the saved traffic, and idle lanes cost what they would compute, so other
        // grids stay unfused unless the caller asks for fusion.  Measured (G updates/s, fused
        // vs unfused, 512 x 512 x nx): nx = 128: 1083 vs 644 (256-wide region: 499); 192: 744 vs
        // 709; 400: 761 vs 776; 448: 851 vs 788; 512: 1257 vs 781.
        // 384-wide regions are 20 rows high (15 warps, one CTA per SM; their planes are loaded as
        // three boxes of 128 columns): 512 x 512 x 384 1359 vs 827, nx = 320: 1027 vs 773.
        // Rows wider than 512 points take several 384- or 512-wide regions, each with 4 halo
        // columns per side for every 2 levels of radius 1, under the same 80 % rule; per lane the
        // 384-wide regions are a quarter faster there (256 x 512 x nx, 384-wide / 512-wide / unfused:
        // nx = 1128: 1217 / 693 / 836; 1500: 1128 / 954 / 830; 256 x 1024 x 1024: 1126 / 687 / 808;
        // nx = 768 fills neither to 80 %: 788 / 753 / 828).
        const FusedConfig* c = nullptr;
        const int halo = (2 * p->radius + 3) / 4 * 4;                         // per side, when a row takes several regions
        auto lanes_used = [&](int w) {
            const int64_t regions = p->nx <= w ? 1 : (p->nx + (w - 2 * halo) - 1) / (w - 2 * halo);
            return (double)p->nx / (double)(regions * w);
        };
        int width = p->nx <= 128 ? 128 : p->nx <= 256 ? 256 : p->nx <= 384 ? 384 : 512;
        if (p->nx > 512 && 1.25 * lanes_used(384) >= lanes_used(512)) width = 384;
        // 256-wide regions are 16 rows high (two CTAs per SM) on grids of fewer than 448 rows and 32 rows high (one
        // CTA per SM, 28 of 32 rows stored instead of 12 of 16) from there on, where the taller regions' fewer
        // CTAs still cut evenly (G updates/s, 16 / 32 rows, nz x ny x 256: 256 x 256: 1163 / 1093, 256 x 384:
        // 1270 / 1245, 256 x 448: 1224 / 1302, 256 x 512: 1235 / 1300, 256 x 1024: 1330 / 1477, 512 x 512: 1329 /
        // 1413, 512 x 256: 1300 / 1258)
        const int height = width == 128 ? 0 : width == 384 ? 20 : (width == 256 && p->ny >= 448) ? 32 : 16;
        // the 384-wide regions pay off from fewer used lanes: any row of 257..384 points (nx = 260:
        // 838 vs 676), three quarters of the lanes with several regions per row (896: 983 vs 843)
        const double need = width != 384 ? 0.8 : p->nx <= 384 ? 0.0 : 0.75;
        if (lanes_used(width) >= need) {
            // 128-wide regions leave registers for a third level (512 x 512 x 128: 1224 G updates/s
            // with three steps per pass, 1083 with two, 1108 with four); at 256 columns three
            // levels spill (256^3: 820 against 1056)
            // ... provided the grid still cuts into a machine's worth of CTAs (a B200 has 148
            // SMs; 128^3 x 64 steps: 302 with three levels, 393 with two)
            if (width == 128 && p->fuse_steps == 0) {
                const FusedConfig* c3 = find_fused_cfg(p->radius, 3, 128);
                if (c3) {
                    const int tile_y = c3->tye - 2 * 3 * p->radius;
                    const int64_t ctas = tile_y < 1 ? 0 : (int64_t)((p->ny + tile_y - 1) / tile_y) *
                                                              std::max(1, p->nz / (4 * 3 * p->radius));
                    if (ctas >= 148) c = c3;
                }
            }
            if (!c) c = find_fused_cfg(p->radius, 2, width, height);
            if (!c && width == 256) c = find_fused_cfg(p->radius, 2, 256);
        }
        if (c || p->fuse_steps == 0) return c;
    }
    return find_fused_cfg(p->radius, p->fuse_steps, txe, p->fused_tile_y);
}

// The z cut of a fused pass: every region (a strip of rows) is cut along z into chunks, one CTA each, handed to
// the machine's `slots` resident-CTA slots in index order.  The kernel is bound by instruction issue, so every SM
// should be busy to the end: a chunk costs its planes plus the `halo` (2*T*R) extra input planes and the start-up
// of its pipeline, and the cut with the least makespan wins.  Equal chunks fill whole waves of the slots only where
// the regions divide them (512^3 in 43 regions of 512 x 16: three chunks per region occupy 129 of 148 SMs).  So
// the search also tries cuts whose last `rest` planes per region go to shorter chunks that come last in the grid:
// the hardware hands those to the SMs that the long chunks leave idle, and to the others as they finish.  Such a
// cut is taken where it models 3 % ahead of the best equal chunks.  (With two CTAs per SM the slots are not
// independent, since a CTA alone on its SM runs faster, and the model rarely finds such a cut 3 % ahead: 256^3
// keeps equal chunks, whose hand-picked alternatives all measured slower; FP64 256 x 320 x 512 takes one, 446
// against 423 G updates/s.)
void fused_z_cut(int nz, int tiles, int slots, int halo, int* chunk_out, int* rest_out, int* rest_chunk_out) {
    const double ovh = halo + 4.0;
    const int max_chunks = std::max(1, nz / (2 * halo));
    std::vector<double> free_at;
    // makespan of n_main CTAs of cost a followed by n_tail CTAs of cost b, each going to the slot that frees first
    auto makespan = [&](int64_t n_main, double a, int64_t n_tail, double b) {
        const int64_t w = n_main / slots, q = n_main % slots;
        if (n_tail == 0) return (double)(w + (q ? 1 : 0)) * a;
        free_at.assign((size_t)slots, (double)w * a);
        for (int64_t i = 0; i < q; ++i) free_at[(size_t)i] += a;
        std::make_heap(free_at.begin(), free_at.end(), std::greater<double>());
        for (int64_t i = 0; i < n_tail; ++i) {
            std::pop_heap(free_at.begin(), free_at.end(), std::greater<double>());
            free_at.back() += b;
            std::push_heap(free_at.begin(), free_at.end(), std::greater<double>());
        }
        return *std::max_element(free_at.begin(), free_at.end());
    };
    double best = 1e300;
    int best_n = 1;
    for (int n = 1; n <= max_chunks; ++n) {
        const int c = (nz + n - 1) / n;
        const int real_n = (nz + c - 1) / c;
        const double cost = makespan((int64_t)tiles * real_n, c + ovh, 0, 0);
        if (cost < best * 0.999) { best = cost; best_n = real_n; }
    }
    int chunk = (nz + best_n - 1) / best_n, rest = 0, rest_chunk = 1;
    // (grids of many waves are balanced already, and a candidate costs time linear in its CTAs: the search stays
    // within about a thousand candidates of a few thousand CTAs)
    if ((int64_t)tiles * best_n <= 8 * (int64_t)slots) {
        double best_tail = 1e300;
        int t_chunk = 0, t_rest = 0, t_rc = 1;
        const int step = std::max(2, nz / 256);
        for (int k = 1; k <= 4; ++k) {
            const int n = (int)std::min<int64_t>((int64_t)k * slots / tiles, max_chunks);    // long chunks per region
            if (n < 1) continue;
            for (int r = 8; r <= nz / 2 && nz - r >= n * 2 * halo; r += step)
                for (int m = 1; m <= 2; ++m) {
                    const int c = (nz - r + n - 1) / n, rc = (r + m - 1) / m;
                    const int64_t n_main = (int64_t)tiles * ((nz - r + c - 1) / c);
                    const int64_t n_tail = (int64_t)tiles * ((r + rc - 1) / rc);
                    const double cost = makespan(n_main, c + ovh, n_tail, rc + ovh);
                    if (cost < best_tail) { best_tail = cost; t_chunk = c; t_rest = r; t_rc = rc; }
                }
        }
        if (best_tail < best * 0.97) { chunk = t_chunk; rest = t_rest; rest_chunk = t_rc; }
    }
    *chunk_out = chunk; *rest_out = rest; *rest_chunk_out = rest_chunk;
}

int launch_fused(stencil_plan_s* p, const void* src, void* dst, int nlev, cudaStream_t st) {
    const FusedConfig* cfg = p->f64 ? p->fused64_cfg : p->fused_cfg;
    const CUtensorMap* map = nullptr;
    int rc = p->f64 ? get_tensor_map_f64(p, cfg, cfg->pw, cfg->tye, static_cast<const double*>(src), &map)
                    : get_tensor_map(p, cfg, cfg->pw, cfg->tye, static_cast<const float*>(src), &map);   // a box is at most 256 wide
    if (rc != STENCIL_OK) return rc;
    const int R = p->radius, T = cfg->T;
    FusedGeom g;
    g.nz = p->nz; g.ny = p->ny; g.nx = p->nx;
    g.nlev = nlev;
    g.wait_polls = p->wait_polls; g.drop_plane = p->drop_plane;
    STENCIL_SET_OUT_POINTS(g, p);
    if (p->nx <= cfg->txe) {                     // one region spans the row: the x halo is the zero boundary
        g.halo_x = 0; g.tile_x = cfg->txe; g.tiles_x = 1;
    } else {
        g.halo_x = (T * R + 3) / 4 * 4;
        g.tile_x = cfg->txe - 2 * g.halo_x;
        g.tiles_x = (p->nx + g.tile_x - 1) / g.tile_x;
    }
    g.halo_y = T * R;
    g.tile_y = cfg->tye - 2 * g.halo_y;
    if (g.tile_x < 4 || g.tile_y < 1) return STENCIL_ERR_UNSUPPORTED;
    g.tiles_y = (p->ny + g.tile_y - 1) / g.tile_y;
    // shared memory: input ring + two planes per intermediate level
    int stages = p->stages > 0 ? std::min(p->stages, kMaxStages) : 2;   // measured: 2 beats 3 and 4
    auto smem_for = [&](int s) { return (size_t)(s + 2 * (T - 1)) * cfg->slot_bytes + 128 + kMaxStages * sizeof(uint64_t); };
    while (stages > 2 && smem_for(stages) > kMaxSmemBytes) --stages;
    const size_t smem = smem_for(stages);
    if (smem > kMaxSmemBytes) return STENCIL_ERR_UNSUPPORTED;
    g.stages = stages;
    const int tiles = g.tiles_x * g.tiles_y;
    // shared-memory limit of the three instantiations and occupancy of the general one, asked once per device and size
    const int occ = kernel_limits(cfg->kernel, cfg->threads, smem, p->device, cfg->lim, true);
    if (occ < 0 || kernel_limits(cfg->kernel_spec, cfg->threads, smem, p->device, cfg->lim_spec, false) < 0 ||
        (cfg->kernel_wrap && kernel_limits(cfg->kernel_wrap, cfg->threads, smem, p->device, cfg->lim_wrap, false) < 0))
        return STENCIL_ERR_CUDA;
    int chunk = p->chunk_z, rest = 0, rest_chunk = 1;
    const int slots = occ * plan_sms(p);
    stencil_plan_s::FusedSchedule& memo = p->fused_schedule;
    if (chunk <= 0) {
        if (!(memo.cfg == cfg && memo.nz == p->nz && memo.tiles == tiles && memo.slots == slots)) {
            memo.cfg = cfg; memo.nz = p->nz; memo.tiles = tiles; memo.slots = slots;
            fused_z_cut(p->nz, tiles, slots, 2 * T * R, &memo.chunk, &memo.rest, &memo.rest_chunk);
        }
        chunk = memo.chunk; rest = memo.rest; rest_chunk = memo.rest_chunk;
    }
    chunk = std::max(1, std::min(chunk, p->nz - rest));
    g.chunk_z = chunk;
    g.rest_z = rest;
    g.rest_chunk = rest_chunk;
    const int64_t main_ctas = (int64_t)tiles * ((p->nz - rest + chunk - 1) / chunk);
    const int64_t grid64 = main_ctas + (int64_t)tiles * ((rest + rest_chunk - 1) / rest_chunk);
    g.main_ctas = (int)std::min<int64_t>(main_ctas, 0x7fffffffLL);
    if (grid64 > 0x7fffffffLL) return STENCIL_ERR_UNSUPPORTED;
    // full passes over rows of exactly one region take the instantiation with those facts compiled in
    // ... and the one that also wraps x and z when the pass belongs to a periodic apply (fused_wrap_ok tells
    // the caller beforehand that it will)
    const bool spec = nlev == T && p->nx == cfg->txe;
    auto launch = !spec ? cfg->launch : (p->fused_wrap ? cfg->launch_wrap : cfg->launch_spec);
    if (p->fused_wrap && (!spec || !cfg->launch_wrap)) return STENCIL_ERR_UNSUPPORTED;
    if (launch(p, *map, dst, g, (int)grid64, smem, st) != cudaSuccess) return STENCIL_ERR_CUDA;
    p->launches++;
    return STENCIL_OK;
}

}  // namespace stencil_host
