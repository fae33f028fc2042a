// Host side of the stencil library: plan validation, kernel selection, tensor
// maps, launches, and the extern "C" boundary declared in include/stencil.h.
// No CPU compute path exists here: every sweep runs in the CUDA kernels.
#include "../../include/stencil.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "common.cuh"
#include "kernel_generic.cuh"
#include "kernel_pad.cuh"
#include "kernel_stream.cuh"
#include "kernel_fused.cuh"
#include "kernel_rows2d.cuh"
#include "kernel_rows2d_fused.cuh"
#include "kernel_rows2d_f64.cuh"
#include "kernel_rows2d_fused_f64.cuh"
#include "kernel_stream_f64.cuh"

using namespace stencil;

namespace {

constexpr uint32_t kPlanMagic = 0x5354434cu;   // "STCL"
constexpr int kMaxRadius = 8;

// ---------------------------------------------------------------------------
// driver entry point for tensor-map encoding, fetched at run time so that the
// library loads on machines without a driver
// ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

// Kernel launch; `chained` marks a launch that follows another launch of this library on
// the same stream inside one iterated apply: it may then begin its preamble while the
// previous kernel drains (programmatic dependent launch; the kernels wait for their
// predecessor before they touch global memory).
template <typename... KArgs, typename... Args>
cudaError_t launch_kernel(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t st,
                          bool chained, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    if (chained) {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    const cudaError_t err = cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
    if (err != cudaSuccess) cudaGetLastError();      // leave no stale error behind for the caller
    return err;
}

// The configuration tables below are shared by all plans and cache per-device facts
// (occupancy, the shared-memory limit already granted to a kernel); this lock makes those
// caches safe when several host threads drive their own plans.
std::mutex g_config_mutex;

// ---------------------------------------------------------------------------
// STREAM kernel configurations
// ---------------------------------------------------------------------------
struct StreamConfig {
    int radius;
    bool box;
    int K, NW;            // rows per thread, consumer warps
    int tile_y;           // K * NW
    int plane_bytes, box_rows, threads;
    int px;               // columns of the TMA box: the tile plus its halo on both sides
    mutable int occupancy[kMaxStages + 1];   // resident CTAs per SM by ring depth; 0 = not asked yet
    mutable size_t smem_allowed;             // dynamic shared memory the kernel is currently allowed
    mutable int cache_device;                // device the two caches above were filled on
    const void* kernel;
    cudaError_t (*launch)(const struct stencil_plan_s*, const StreamConfig&, const CUtensorMap&,
                          float*, const StreamGeom&, int grid, size_t smem, cudaStream_t);
    // the sweep of a periodic grid inside the kernel (stars of radius <= 4 and the boxes; null otherwise)
    const void* kernel_wrap;
    int stage_bytes;                         // per ring slot, beside the plane
    mutable size_t smem_allowed_wrap;
    cudaError_t (*launch_wrap)(const struct stencil_plan_s*, const CUtensorMap&, const CUtensorMap&,
                               const CUtensorMap&, const CUtensorMap&, float*, const StreamGeom&, int grid,
                               size_t smem, cudaStream_t);
};

// ---------------------------------------------------------------------------
// FUSED kernel configurations (temporal blocking, 3D star)
// ---------------------------------------------------------------------------
struct FusedConfig {
    int radius, T, K, XW, NWY;
    int txe, tye, threads, slot_bytes;
    int pw;                                  // width of the TMA boxes a plane is loaded as
    const void* kernel;
    const void* kernel_spec;                 // the instantiation for full passes over rows of exactly txe points
    const void* kernel_wrap;                 // ... and the one of those that wraps x and z (passes of a periodic grid)
    mutable size_t smem_allowed;             // dynamic shared memory already granted to both kernels
    mutable size_t occ_smem;                 // ... and the occupancy measured at this size
    mutable int occ;
    mutable int cache_device;
    cudaError_t (*launch)(const struct stencil_plan_s*, const CUtensorMap&, float*, const FusedGeom&,
                          int grid, size_t smem, cudaStream_t);
    cudaError_t (*launch_spec)(const struct stencil_plan_s*, const CUtensorMap&, float*, const FusedGeom&,
                               int grid, size_t smem, cudaStream_t);
    cudaError_t (*launch_wrap)(const struct stencil_plan_s*, const CUtensorMap&, float*, const FusedGeom&,
                               int grid, size_t smem, cudaStream_t);
};

// ---------------------------------------------------------------------------
// ROWS2D kernel configurations (2D grids)
// ---------------------------------------------------------------------------
struct Rows2DConfig {
    int radius;
    bool box;
    int YB, NW, batch_bytes;
    int px;                     // columns of the TMA box: the strip plus its halo on both sides
    const void* kernel;
    mutable size_t smem_allowed;
    mutable int cache_device;
    cudaError_t (*launch)(const struct stencil_plan_s*, const CUtensorMap&, float*, const Rows2DGeom&,
                          int grid, size_t smem, cudaStream_t);
};

// ---------------------------------------------------------------------------
// ROWS2D FUSED kernel configurations (iterated 2D sweeps, T time steps per pass)
// ---------------------------------------------------------------------------
struct Rows2DFusedConfig {
    int radius;
    bool box;
    int T, YB, NW, batch_bytes;
    const void* kernel;
    mutable size_t smem_allowed;
    mutable size_t occ_smem;                 // shared-memory size the occupancy below was measured at
    mutable int occ;                         // resident CTAs per SM
    mutable int cache_device;
    cudaError_t (*launch)(const struct stencil_plan_s*, const CUtensorMap&, float*, const Rows2DFusedGeom&,
                          int grid, size_t smem, cudaStream_t);
};

}  // namespace

struct Rows2DFused64Config {
    int radius;
    bool box;
    int T, YB, NW, batch_bytes;
    const void* kernel;
    mutable size_t smem_allowed;
    mutable size_t occ_smem;
    mutable int occ;
    mutable int cache_device;
    cudaError_t (*launch)(const struct stencil_plan_s*, const CUtensorMap&, double*, const stencil::Rows2DFusedGeom&,
                          int grid, size_t smem, cudaStream_t);
};

struct Rows2D64Config {
    int radius;
    bool box;
    int YB, NW, batch_bytes, px;
    const void* kernel;
    mutable size_t smem_allowed;
    mutable int cache_device;
    cudaError_t (*launch)(const struct stencil_plan_s*, const CUtensorMap&, double*, const Rows2DGeom&,
                          int grid, size_t smem, cudaStream_t);
};

struct Stream64Config {
    int radius;
    bool box;
    int tile_y, plane_bytes, box_rows, threads, px;
    const void* kernel;
    mutable size_t smem_allowed;
    mutable size_t occ_smem;                 // shared-memory size the occupancy below was asked for
    mutable int occ;                         // resident CTAs per SM
    mutable int cache_device;
    cudaError_t (*launch)(const struct stencil_plan_s*, const CUtensorMap&, double*, const StreamGeom&,
                          int grid, size_t smem, cudaStream_t);
    // the sweep of a periodic grid inside the kernel (stars of radius <= 4; null otherwise)
    const void* kernel_wrap;
    int stage_bytes;                         // per ring slot, beside the plane
    mutable size_t smem_allowed_wrap;
    cudaError_t (*launch_wrap)(const struct stencil_plan_s*, const CUtensorMap&, const CUtensorMap&,
                               const CUtensorMap&, const CUtensorMap&, double*, const StreamGeom&, int grid,
                               size_t smem, cudaStream_t);
};

constexpr int kMaxFuseLevels = 4;          // deepest temporal blocking of any fused kernel

struct stencil_plan_s {
    uint32_t magic;
    int ndim;
    int nz, ny, nx;
    int64_t npoints;
    int radius, shape, boundary;
    bool f64;                      // FP64 plan (stencil_plan_f64): only the *_f64 calls accept it
    std::vector<float> w;          // dense (2R+1)^ndim, as given
    std::vector<Tap> taps;         // non-zero taps, dense C order
    std::vector<double> w64;       // the same for FP64 plans
    std::vector<TapT<double>> taps64;
    TapT<double>* d_taps64;
    // taps of the operator's L-fold self-convolution, L = 1..kMaxFuseLevels (periodic boundary under
    // temporal blocking); built and uploaded at first need
    std::vector<TapT<double>> ctaps[kMaxFuseLevels + 1];
    TapT<double>* d_ctaps[kMaxFuseLevels + 1];
    double* scratch64;             // N doubles, iteration ping-pong of FP64 plans
    const struct Rows2D64Config* rows2d64_cfg;
    const struct Rows2DFused64Config* fused2d64_cfg;   // non-null: iterated applies of a 2D FP64 grid run fused passes
    const struct Stream64Config* stream64_cfg;
    // device state (created lazily, on the device current at first apply)
    int device;
    Tap* d_taps;
    int* d_status;
    float* scratch;                // N floats, iteration ping-pong
    float* pad;                    // padded copy of the input (periodic boundary on the tiled kernels;
                                   // first of the two padded-row grids when nx is not a multiple of 4)
    float* pad2;                   // second padded-row grid
    int tmap_nx;                   // non-zero while a padded-row sweep runs: the true row length
    int periodic_route;            // knob: 0 = by measured cost, 1 = padded copy, 2 = wrap correction where it fits
    bool fused_wrap;               // set for one launch_fused call: the pass wraps x and z in the kernel
    bool stream_wrap;              // set while a periodic apply sweeps with the kernel that wraps all three axes
    bool src_padded;               // set while an iterated periodic apply runs: the source of a sweep is
                                   // a padded grid with current halos
    float* host_in;                // N floats each, apply_host staging
    float* host_out;
    cudaStream_t copy_in, copy_out; // apply_host: upload / download streams (created on first use)
    std::vector<cudaEvent_t> events; // apply_host: slab hand-over events
    // selection and tuning
    int variant;                   // resolved STENCIL_VARIANT_*
    int tile_y, rows_per_thread, chunk_z, stages, fuse_steps, streaming_store;
    bool chain_launches;           // knob: launches 2..n of an iterated apply start early (see launch_kernel)
    bool chained;                  // set by the apply loop for those launches
    unsigned wait_polls;           // cap of the bounded device waits (single-step 3D kernel)
    int drop_plane;                // test hook, -1 = off
    const StreamConfig* stream_cfg;
    bool stream_cfg_fixed;         // the caller chose the tile shape
    bool stream_cfg_tuned;         // the library has chosen it for this grid
    const FusedConfig* fused_cfg;  // non-null: iterated applies run fused passes
    const Rows2DConfig* rows2d_cfg; // non-null: 2D grid on the row-streaming kernel
    const Rows2DFusedConfig* fused2d_cfg;  // non-null: iterated applies of a 2D grid run fused passes
    int tile_x;                    // requested region width for fused passes (0 = auto)
    int fused_tile_y;              // requested region height for fused passes (0 = any)
    // bookkeeping
    int64_t launches;
    cudaStream_t last_stream;
    bool used;
    // tensor-map cache: one entry per source pointer
    struct MapEntry { const void* ptr; const void* cfg; CUtensorMap map; };
    std::vector<MapEntry> maps;
};

namespace {

// ---------------------------------------------------------------------------
// weight packing for the tiled kernels
// ---------------------------------------------------------------------------
inline float dense_w(const stencil_plan_s* p, int dz, int dy, int dx) {
    const int R = p->radius, side = 2 * R + 1;
    if (p->ndim == 3) return p->w[((size_t)(dz + R) * side + (dy + R)) * side + (dx + R)];
    return dz == 0 ? p->w[(size_t)(dy + R) * side + (dx + R)] : 0.0f;
}

template <int R, bool BOX, int K, int NW, int MINB>
cudaError_t launch_stream_t(const stencil_plan_s* p, const StreamConfig&, const CUtensorMap& map,
                            float* out, const StreamGeom& g, int grid, size_t smem, cudaStream_t st) {
    StarWeights<R> sw;
    BoxWeights<BOX ? R : 0> bw;
    std::memset(&sw, 0, sizeof(sw));
    std::memset(&bw, 0, sizeof(bw));
    if (!BOX) {
        sw.c = dense_w(p, 0, 0, 0);
        for (int d = -R; d <= R; ++d) {
            if (d == 0) continue;
            sw.x[d + R] = dense_w(p, 0, 0, d);
            sw.y[d + R] = dense_w(p, 0, d, 0);
            sw.z[d + R] = dense_w(p, d, 0, 0);
        }
    } else {
        constexpr int RB = BOX ? R : 0;
        for (int a = -RB; a <= RB; ++a)
            for (int b = -RB; b <= RB; ++b)
                for (int c = -RB; c <= RB; ++c) bw.w[a + RB][b + RB][c + RB] = dense_w(p, a, b, c);
    }
    return launch_kernel(&stencil_stream_kernel<R, BOX, K, NW, MINB>, grid, StreamShape<R, K, NW>::THREADS, smem,
                         st, p->chained, map, out, g, sw, bw, p->d_status);
}

template <int R, bool BOX, int K, int NW, int MINB>
cudaError_t launch_stream_wrap_t(const stencil_plan_s* p, const CUtensorMap& map, const CUtensorMap& map_xs,
                                 const CUtensorMap& map_ys, const CUtensorMap& map_cs, float* out,
                                 const StreamGeom& g, int grid, size_t smem, cudaStream_t st) {
    StarWeights<R> sw;
    BoxWeights<BOX ? R : 0> bw;
    std::memset(&sw, 0, sizeof(sw));
    std::memset(&bw, 0, sizeof(bw));
    if (!BOX) {
        sw.c = dense_w(p, 0, 0, 0);
        for (int d = -R; d <= R; ++d) {
            if (d == 0) continue;
            sw.x[d + R] = dense_w(p, 0, 0, d);
            sw.y[d + R] = dense_w(p, 0, d, 0);
            sw.z[d + R] = dense_w(p, d, 0, 0);
        }
    } else {
        constexpr int RB = BOX ? R : 0;
        for (int a = -RB; a <= RB; ++a)
            for (int b = -RB; b <= RB; ++b)
                for (int c = -RB; c <= RB; ++c) bw.w[a + RB][b + RB][c + RB] = dense_w(p, a, b, c);
    }
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
    for (int& o : c.occupancy) o = 0;
    c.smem_allowed = 0;
    c.cache_device = -1;
    c.kernel = reinterpret_cast<const void*>(&stencil_stream_kernel<R, BOX, K, NW, MINB>);
    c.launch = &launch_stream_t<R, BOX, K, NW, MINB>;
    c.kernel_wrap = nullptr; c.launch_wrap = nullptr; c.stage_bytes = 0; c.smem_allowed_wrap = 0;
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

template <int R>
void pack_star(const stencil_plan_s* p, StarWeights<R>& sw) {
    std::memset(&sw, 0, sizeof(sw));
    sw.c = dense_w(p, 0, 0, 0);
    for (int d = -R; d <= R; ++d) {
        if (d == 0) continue;
        sw.x[d + R] = dense_w(p, 0, 0, d);
        sw.y[d + R] = dense_w(p, 0, d, 0);
        sw.z[d + R] = dense_w(p, d, 0, 0);
    }
}

template <int R, int T, int K, int XW, int NWY, int MODE>
cudaError_t launch_fused_t(const stencil_plan_s* p, const CUtensorMap& map, float* out, const FusedGeom& g,
                           int grid, size_t smem, cudaStream_t st) {
    StarWeights<R> sw;
    pack_star<R>(p, sw);
    return launch_kernel(&stencil_fused_kernel<R, T, K, XW, NWY, MODE>, grid, FusedShape<R, K, XW, NWY>::THREADS,
                         smem, st, p->chained, map, out, g, sw, p->d_status);
}

template <int R, int T, int K, int XW, int NWY>
FusedConfig make_fused() {
    using S = FusedShape<R, K, XW, NWY>;
    FusedConfig c;
    c.radius = R; c.T = T; c.K = K; c.XW = XW; c.NWY = NWY;
    c.txe = S::TXE; c.tye = S::TYE; c.threads = S::THREADS; c.slot_bytes = S::SLOT_BYTES; c.pw = S::PW;
    c.kernel = reinterpret_cast<const void*>(&stencil_fused_kernel<R, T, K, XW, NWY, 0>);
    c.kernel_spec = reinterpret_cast<const void*>(&stencil_fused_kernel<R, T, K, XW, NWY, 1>);
    c.kernel_wrap = reinterpret_cast<const void*>(&stencil_fused_kernel<R, T, K, XW, NWY, 2>);
    c.smem_allowed = 0; c.occ_smem = 0; c.occ = 0; c.cache_device = -1;
    c.launch = &launch_fused_t<R, T, K, XW, NWY, 0>;
    c.launch_spec = &launch_fused_t<R, T, K, XW, NWY, 1>;
    c.launch_wrap = &launch_fused_t<R, T, K, XW, NWY, 2>;
    return c;
}

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

template <int R, bool BOX, int YB, int NW>
cudaError_t launch_rows2d_t(const stencil_plan_s* p, const CUtensorMap& map, float* out, const Rows2DGeom& g,
                            int grid, size_t smem, cudaStream_t st) {
    Weights2D<R> wt;
    for (int a = -R; a <= R; ++a)
        for (int b = -R; b <= R; ++b) wt.w[a + R][b + R] = dense_w(p, 0, a, b);
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
    c.smem_allowed = 0; c.cache_device = -1;
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
    for (int a = -R; a <= R; ++a)
        for (int b = -R; b <= R; ++b) wt.w[a + R][b + R] = dense_w(p, 0, a, b);
    return launch_kernel(&stencil_rows2d_fused_kernel<R, BOX, T, YB, NW>, grid, NW * 32, smem, st, p->chained, map,
                         out, g, wt, p->d_status);
}

template <int R, bool BOX, int T, int YB, int NW>
Rows2DFusedConfig make_rows2d_fused() {
    Rows2DFusedConfig c;
    c.radius = R; c.box = BOX; c.T = T; c.YB = YB; c.NW = NW; c.batch_bytes = Rows2DShape<YB>::BATCH_BYTES;
    c.kernel = reinterpret_cast<const void*>(&stencil_rows2d_fused_kernel<R, BOX, T, YB, NW>);
    c.smem_allowed = 0; c.occ_smem = 0; c.occ = 0; c.cache_device = -1;
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

// Temporal blocking of a 2D grid: 16-byte rows, the operators in the table above (a periodic grid must hold
// the two shells of depth T * R along either axis).
inline bool shell_fits(const stencil_plan_s* p, int H);
const Rows2DFusedConfig* pick_fused2d(const stencil_plan_s* p) {
    if (p->ndim != 2 || p->nx % 4 != 0 || p->fuse_steps == 1) return nullptr;
    for (const Rows2DFusedConfig& c : rows2d_fused_configs())
        if (c.radius == p->radius && c.box == (p->shape == STENCIL_BOX) && (p->fuse_steps == 0 || p->fuse_steps == c.T))
            return (p->boundary == STENCIL_PERIODIC && !shell_fits(p, c.T * p->radius)) ? nullptr : &c;
    return nullptr;
}

// The tiled kernels need rows whose byte length is a multiple of 16 (a TMA stride rule).
// The zero boundary comes from TMA's zero fill of out-of-grid cells; a periodic grid is first
// copied into a padded grid with wrapped halos (kernel_pad.cuh) and swept from there.  A
// zero-boundary grid with other row lengths is swept between two grids with padded rows
// (apply_row_padded).
bool wrap_correction_fits(const stencil_plan_s* p);

bool stream_supported(const stencil_plan_s* p) {
    if (p->nx % 4 != 0 && p->boundary != STENCIL_ZERO) return false;
    // radius > 4: the padded periodic copy has only 4 halo columns, so the wrap correction must fit
    if (p->radius > 4 && p->boundary == STENCIL_PERIODIC && !wrap_correction_fits(p)) return false;
    const bool box = p->shape == STENCIL_BOX;
    if (p->ndim == 2) return find_rows2d_cfg(p->radius, box) != nullptr;
    return find_stream_cfg(p->radius, box, 0, 0) != nullptr;
}

// A periodic grid takes fused passes of L steps as zero-boundary passes whose shell of depth
// H = L * R is then rewritten (stencil_shell_compose_kernel): every extent must hold both shells.
inline bool shell_fits(const stencil_plan_s* p, int H) {
    return p->nx >= 2 * H && p->ny >= 2 * H && (p->ndim == 2 || p->nz >= 2 * H);
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
        // (two CTAs per SM, which cover each other's barrier stalls: 16-row regions beat 32-row
        // ones, 922 vs 846 G updates/s on 256^3) or 512 columns wide (one CTA per SM, each plane
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
        const int height = width == 128 ? 0 : width == 384 ? 20 : 16;
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

int resolve_variant(stencil_plan_s* p, int want) {
    if (want == STENCIL_VARIANT_AUTO) want = stream_supported(p) ? STENCIL_VARIANT_STREAM : STENCIL_VARIANT_GENERIC;
    if (want == STENCIL_VARIANT_GENERIC) {
        p->variant = want; p->fused_cfg = nullptr; p->fused2d_cfg = nullptr;
        return STENCIL_OK;
    }
    if (want == STENCIL_VARIANT_STREAM || want == STENCIL_VARIANT_FUSED) {
        if (!stream_supported(p)) return STENCIL_ERR_UNSUPPORTED;
        if (p->ndim == 2) {
            const Rows2DFusedConfig* f2 = pick_fused2d(p);
            if (want == STENCIL_VARIANT_FUSED && !f2) return STENCIL_ERR_UNSUPPORTED;
            p->rows2d_cfg = find_rows2d_cfg(p->radius, p->shape == STENCIL_BOX);
            p->fused2d_cfg = f2;
            p->stream_cfg = nullptr; p->fused_cfg = nullptr;
            p->variant = STENCIL_VARIANT_STREAM;
            return STENCIL_OK;
        }
        const StreamConfig* c = find_stream_cfg(p->radius, p->shape == STENCIL_BOX, p->tile_y, p->rows_per_thread);
        if (!c) return STENCIL_ERR_UNSUPPORTED;
        const FusedConfig* f = pick_fused(p);
        if (want == STENCIL_VARIANT_FUSED && !f) return STENCIL_ERR_UNSUPPORTED;
        p->stream_cfg = c;
        p->fused_cfg = f;
        p->variant = STENCIL_VARIANT_STREAM;
        return STENCIL_OK;
    }
    return STENCIL_ERR_UNSUPPORTED;
}

// ---------------------------------------------------------------------------
// device state
// ---------------------------------------------------------------------------
int ensure_device_state(stencil_plan_s* p) {
    if (p->d_status) return STENCIL_OK;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return STENCIL_ERR_CUDA; }
    int* status = nullptr;
    Tap* taps = nullptr;
    TapT<double>* taps64 = nullptr;
    const size_t bytes = p->taps.size() * sizeof(Tap);
    const size_t bytes64 = p->taps64.size() * sizeof(TapT<double>);
    int rc = STENCIL_OK;
    if (cudaMalloc(&status, sizeof(int)) != cudaSuccess) rc = STENCIL_ERR_ALLOC;
    if (rc == STENCIL_OK && cudaMemset(status, 0, sizeof(int)) != cudaSuccess) rc = STENCIL_ERR_CUDA;
    if (rc == STENCIL_OK && bytes && cudaMalloc(&taps, bytes) != cudaSuccess) rc = STENCIL_ERR_ALLOC;
    if (rc == STENCIL_OK && bytes &&
        cudaMemcpy(taps, p->taps.data(), bytes, cudaMemcpyHostToDevice) != cudaSuccess)
        rc = STENCIL_ERR_CUDA;
    if (rc == STENCIL_OK && bytes64 && cudaMalloc(&taps64, bytes64) != cudaSuccess) rc = STENCIL_ERR_ALLOC;
    if (rc == STENCIL_OK && bytes64 &&
        cudaMemcpy(taps64, p->taps64.data(), bytes64, cudaMemcpyHostToDevice) != cudaSuccess)
        rc = STENCIL_ERR_CUDA;
    if (rc != STENCIL_OK) {                         // all or nothing: a later call starts afresh
        cudaGetLastError();
        if (status) cudaFree(status);
        if (taps) cudaFree(taps);
        if (taps64) cudaFree(taps64);
        cudaGetLastError();
        return rc;
    }
    p->device = dev;
    p->d_status = status;
    p->d_taps = taps;
    p->d_taps64 = taps64;
    return STENCIL_OK;
}

int ensure_grid(float** slot, int64_t npoints) {
    if (*slot) return STENCIL_OK;
    if (cudaMalloc(slot, (size_t)npoints * sizeof(float)) != cudaSuccess) {
        cudaGetLastError();
        *slot = nullptr;
        return STENCIL_ERR_ALLOC;
    }
    return STENCIL_OK;
}

// ---------------------------------------------------------------------------
// launches
// ---------------------------------------------------------------------------
int sm_count();

int launch_generic(stencil_plan_s* p, const float* src, float* dst, cudaStream_t st) {
    Grid g{p->nz, p->ny, p->nx};
    const int grid = generic_grid_size(g, sm_count());
    const int ntaps = (int)p->taps.size();
    if (p->boundary == STENCIL_PERIODIC)
        stencil_generic_kernel<true><<<grid, kGenericThreads, 0, st>>>(src, dst, g, p->d_taps, ntaps);
    else
        stencil_generic_kernel<false><<<grid, kGenericThreads, 0, st>>>(src, dst, g, p->d_taps, ntaps);
    if (cudaGetLastError() != cudaSuccess) return STENCIL_ERR_CUDA;
    p->launches++;
    return STENCIL_OK;
}

int get_tensor_map(stencil_plan_s* p, const void* cfg, int box_x, int box_y, const float* src,
                   const CUtensorMap** out, int tnx = 0, int tny = 0, int tnz = 0) {
    if (tnx == 0) { tnx = p->nx; tny = p->ny; tnz = p->nz; }     // extents of the tensor `src` points at
    // padded rows: the pitch is tnx, the cells past the true row length read as out of grid (zero)
    const int row_cells = p->tmap_nx > 0 ? p->tmap_nx : tnx;
    for (auto& e : p->maps)
        if (e.ptr == src && e.cfg == cfg) { *out = &e.map; return STENCIL_OK; }
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return STENCIL_ERR_CUDA;
    stencil_plan_s::MapEntry e;
    e.ptr = src; e.cfg = cfg;
    const cuuint64_t dims[3] = {(cuuint64_t)row_cells, (cuuint64_t)tny, (cuuint64_t)tnz};
    const cuuint64_t strides[2] = {(cuuint64_t)tnx * 4, (cuuint64_t)tnx * (cuuint64_t)tny * 4};
    const cuuint32_t box[3] = {(cuuint32_t)box_x, (cuuint32_t)box_y, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(&e.map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(src), dims, strides,
                     box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return STENCIL_ERR_CUDA;
    if (p->maps.size() >= 16) p->maps.erase(p->maps.begin());
    p->maps.push_back(e);
    *out = &p->maps.back().map;
    return STENCIL_OK;
}

int sm_count() {
    static int n = 0;
    if (n == 0) {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
            n = v;
        else { cudaGetLastError(); n = 148; }
    }
    return n;
}

size_t stream_smem_bytes(const StreamConfig* cfg, int stages) {
    return (size_t)stages * cfg->plane_bytes + 128 + 2 * kMaxStages * sizeof(uint64_t);
}

// Resident CTAs per SM of a configuration at a given ring depth (asked once).
int stream_occupancy(const StreamConfig* cfg, int stages) {
    const size_t smem = stream_smem_bytes(cfg, stages);
    if (smem > 227 * 1024) return -1;
    std::lock_guard<std::mutex> lock(g_config_mutex);
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return -1; }
    if (dev != cfg->cache_device) {                // function attributes are per device
        for (int& o : cfg->occupancy) o = 0;
        cfg->smem_allowed = 0;
        cfg->smem_allowed_wrap = 0;
        cfg->cache_device = dev;
    }
    if (smem > cfg->smem_allowed) {                // the limit only ever grows
        if (cudaFuncSetAttribute(cfg->kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
            cudaGetLastError();
            return -1;
        }
        cfg->smem_allowed = smem;
    }
    if (cfg->occupancy[stages] != 0) return cfg->occupancy[stages];
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, cfg->kernel, cfg->threads, smem) != cudaSuccess) {
        cudaGetLastError();
        occ = 0;
    }
    cfg->occupancy[stages] = occ > 0 ? occ : -1;
    return cfg->occupancy[stages];
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
    const int occ = std::max(1, stream_occupancy(cfg, stages));
    const int slots = occ * sm_count();
    if (!issue_bound(p)) {
        // measured on 512^3: 32-plane chunks (several thousand short CTAs) beat every longer chunk
        int chunk = nz >= 64 ? 32 : nz;
        if (p->shape == STENCIL_STAR && R == 1 && nz >= 16) chunk = short_chunk_star1(nz, tiles, slots);
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

// Periodic boundary: copy `src` into the plan's padded grid (wrapped halos) on `st`.
// The padded grid and its extents come back through padded and pnx/pny/pnz.  Inside an
// iterated apply `src` already is a padded grid with current halos (apply_periodic) and
// comes back as it is.
template <typename T>
int pad_periodic(stencil_plan_s* p, const T* src, cudaStream_t st, const T** padded, int* pnx, int* pny,
                 int* pnz) {
    const int R = p->radius;
    const int rz = p->ndim == 3 ? R : 0;
    *pnx = p->nx + 2 * kPadX; *pny = p->ny + 2 * R; *pnz = p->nz + 2 * rz;
    if (p->src_padded) { *padded = src; return STENCIL_OK; }
    if (!p->pad) {
        const size_t bytes = (size_t)*pnx * *pny * *pnz * sizeof(T);
        if (cudaMalloc(&p->pad, bytes) != cudaSuccess) {
            cudaGetLastError();
            p->pad = nullptr;
            return STENCIL_ERR_ALLOC;
        }
    }
    Grid g{p->nz, p->ny, p->nx};
    const int64_t cells = (int64_t)(*pnx / Vec16<T>::n) * *pny * *pnz;
    const int grid = (int)std::min<int64_t>((cells + 255) / 256, (int64_t)sm_count() * 32);
    stencil_pad_periodic_kernel<T><<<grid, 256, 0, st>>>(src, reinterpret_cast<T*>(p->pad), g, R, rz);
    if (cudaGetLastError() != cudaSuccess) return STENCIL_ERR_CUDA;
    p->launches++;
    *padded = reinterpret_cast<const T*>(p->pad);
    return STENCIL_OK;
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
    if (smem > 227 * 1024) return STENCIL_ERR_UNSUPPORTED;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return STENCIL_ERR_CUDA; }
    {
        std::lock_guard<std::mutex> lock(g_config_mutex);
        if (dev != cfg->cache_device) {
            cfg->smem_allowed = 0; cfg->smem_allowed_wrap = 0; cfg->cache_device = dev;
            for (int& o : cfg->occupancy) o = 0;
        }
        if (smem > cfg->smem_allowed_wrap) {
            if (cudaFuncSetAttribute(cfg->kernel_wrap, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
                cudaSuccess) {
                cudaGetLastError();
                return STENCIL_ERR_CUDA;
            }
            cfg->smem_allowed_wrap = smem;
        }
    }
    StreamGeom g;
    g.in_off_x = g.in_off_y = g.in_off_z = 0;
    g.nz = p->nz; g.ny = p->ny; g.nx = p->nx;
    g.tiles_x = (p->nx + kStreamTX - 1) / kStreamTX;
    g.tiles_y = (p->ny + cfg->tile_y - 1) / cfg->tile_y;
    g.stages = stages;
    g.streaming_store = p->streaming_store;
    if (stream_occupancy(cfg, stages) <= 0) return STENCIL_ERR_UNSUPPORTED;
    int chunk = p->chunk_z > 0 ? p->chunk_z : choose_chunk(p, cfg, stages, nullptr, p->nz);
    chunk = std::max(1, std::min(chunk, p->nz));
    g.chunk_z = chunk;
    g.z_begin = 0; g.z_end = p->nz;
    g.wait_polls = p->wait_polls; g.drop_plane = -1;
    const int64_t grid64 = (int64_t)g.tiles_x * g.tiles_y * ((p->nz + chunk - 1) / chunk);
    if (grid64 > 0x7fffffffLL) return STENCIL_ERR_UNSUPPORTED;
    if (cfg->launch_wrap(p, map, map_xs, map_ys, map_cs, dst, g, (int)grid64, smem, st) != cudaSuccess)
        return STENCIL_ERR_CUDA;
    p->launches++;
    return STENCIL_OK;
}

// dst[z_begin, z_end) = one sweep of src; the whole grid when z_end <= z_begin.
int launch_stream(stencil_plan_s* p, const float* src, float* dst, cudaStream_t st, int z_begin = 0,
                  int z_end = 0) {
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
        const bool plentiful = big_tiles * (span / 64) >= 2 * (int64_t)sm_count();
        if (const StreamConfig* c = find_stream_cfg(3, false, 0, plentiful ? 4 : 2)) p->stream_cfg = c;
    }
    if (!p->stream_cfg_fixed && !p->stream_cfg_tuned) {
        // pick the tile height that balances this grid best (same rows per thread)
        const StreamConfig* best_cfg = p->stream_cfg;
        double best = 1e300;
        for (const StreamConfig& c : stream_configs()) {
            if (c.radius != p->radius || c.box != (p->shape == STENCIL_BOX) || c.K != p->stream_cfg->K) continue;
            if (stream_occupancy(&c, stages) <= 0) continue;
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
    if (stream_occupancy(cfg, stages) <= 0) return STENCIL_ERR_UNSUPPORTED;
    int chunk = p->chunk_z > 0 ? p->chunk_z : choose_chunk(p, cfg, stages, nullptr, span);
    chunk = std::max(1, std::min(chunk, span));
    g.chunk_z = chunk;
    g.z_begin = z_begin; g.z_end = z_end;
    g.wait_polls = p->wait_polls; g.drop_plane = p->drop_plane;
    const int nchunks = (span + chunk - 1) / chunk;
    const int64_t grid64 = (int64_t)tiles * nchunks;
    if (grid64 > 0x7fffffffLL) return STENCIL_ERR_UNSUPPORTED;
    const size_t smem = stream_smem_bytes(cfg, stages);
    if (cfg->launch(p, *cfg, *map, dst, g, (int)grid64, smem, st) != cudaSuccess) return STENCIL_ERR_CUDA;
    p->launches++;
    return STENCIL_OK;
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
int launch_rows2d(stencil_plan_s* p, const float* src, float* dst, cudaStream_t st, int y_begin = 0, int y_end = 0) {
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
    while (stages > 2 && smem_for(stages) > 227 * 1024) --stages;      // a ring deeper than shared memory holds is cut back
    const size_t smem = smem_for(stages);
    if (smem > 227 * 1024) return STENCIL_ERR_UNSUPPORTED;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return STENCIL_ERR_CUDA; }
    {
        std::lock_guard<std::mutex> lock(g_config_mutex);
        if (dev != cfg->cache_device) { cfg->smem_allowed = 0; cfg->cache_device = dev; }
        if (smem > cfg->smem_allowed) {
            if (cudaFuncSetAttribute(cfg->kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
                cudaSuccess) {
                cudaGetLastError();
                return STENCIL_ERR_CUDA;
            }
            cfg->smem_allowed = smem;
        }
    }
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
        const int slots = 2 * sm_count() * cfg->NW;
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
    while (stages > 2 && smem_for(stages) > 227 * 1024) --stages;      // a ring deeper than shared memory holds is cut back
    const size_t smem = smem_for(stages);
    if (smem > 227 * 1024) return STENCIL_ERR_UNSUPPORTED;
    int dev = -1, occ = 1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return STENCIL_ERR_CUDA; }
    {
        std::lock_guard<std::mutex> lock(g_config_mutex);
        if (dev != cfg->cache_device) { cfg->smem_allowed = 0; cfg->occ_smem = 0; cfg->cache_device = dev; }
        if (smem > cfg->smem_allowed) {
            if (cudaFuncSetAttribute(cfg->kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
                cudaSuccess) {
                cudaGetLastError();
                return STENCIL_ERR_CUDA;
            }
            cfg->smem_allowed = smem;
        }
        if (cfg->occ_smem != smem) {
            int o = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, cfg->kernel, cfg->NW * 32, smem) != cudaSuccess) {
                cudaGetLastError();
                o = 0;
            }
            cfg->occ = std::max(o, 1);
            cfg->occ_smem = smem;
        }
        occ = cfg->occ;
    }
    Rows2DFusedGeom g;
    g.ny = p->ny; g.nx = p->nx;
    g.strips = (p->nx + kFused2DTile - 1) / kFused2DTile;
    g.stages = stages;
    g.nlev = nlev;
    int chunk = p->chunk_z;                          // the streamed axis of a 2D grid is y
    if (chunk <= 0) {
        // A unit reads chunk + 2*nlev*R rows in batches of YB and recomputes the 2*nlev*R extra ones at
        // every level, so chunks should be long; as many (strip, chunk) units as fill the machine's
        // resident warp slots once, never more (10240^2: 248-row chunks 2082 G updates/s, 504-row
        // chunks, half a wave, 1479; 120-row chunks 1843).
        const int H = nlev * p->radius;
        const int slots = occ * sm_count() * cfg->NW;
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

int launch_fused(stencil_plan_s* p, const float* src, float* dst, int nlev, cudaStream_t st) {
    const FusedConfig* cfg = p->fused_cfg;
    const CUtensorMap* map = nullptr;
    int rc = get_tensor_map(p, cfg, cfg->pw, cfg->tye, src, &map);   // a box is at most 256 wide
    if (rc != STENCIL_OK) return rc;
    const int R = p->radius, T = cfg->T;
    FusedGeom g;
    g.nz = p->nz; g.ny = p->ny; g.nx = p->nx;
    g.nlev = nlev;
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
    while (stages > 2 && smem_for(stages) > 227 * 1024) --stages;
    const size_t smem = smem_for(stages);
    if (smem > 227 * 1024) return STENCIL_ERR_UNSUPPORTED;
    g.stages = stages;
    const int tiles = g.tiles_x * g.tiles_y;
    int occ = 1;
    {
        // shared-memory limit and occupancy of the kernel, asked once per device and size
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return STENCIL_ERR_CUDA; }
        std::lock_guard<std::mutex> lock(g_config_mutex);
        if (dev != cfg->cache_device) { cfg->smem_allowed = 0; cfg->occ_smem = 0; cfg->cache_device = dev; }
        if (smem > cfg->smem_allowed) {
            if (cudaFuncSetAttribute(cfg->kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
                    cudaSuccess ||
                cudaFuncSetAttribute(cfg->kernel_spec, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
                    cudaSuccess ||
                cudaFuncSetAttribute(cfg->kernel_wrap, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
                    cudaSuccess) {
                cudaGetLastError();
                return STENCIL_ERR_CUDA;
            }
            cfg->smem_allowed = smem;
        }
        if (cfg->occ_smem != smem) {
            int o = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, cfg->kernel, cfg->threads, smem) != cudaSuccess) {
                cudaGetLastError();
                o = 0;
            }
            cfg->occ = std::max(o, 1);
            cfg->occ_smem = smem;
        }
        occ = cfg->occ;
    }
    int chunk = p->chunk_z;
    if (chunk <= 0) {
        // The kernel is bound by instruction issue, so every SM should get the same number of
        // planes: cut z into the number of chunks whose CTAs fill whole waves of the machine's
        // resident-CTA slots at the least total cost, a chunk costing its planes plus the
        // 2*T*R extra input planes and the start-up of its pipeline.
        const int slots = occ * sm_count();
        const int max_chunks = std::max(1, p->nz / (4 * T * R));
        const double fill = 4.0;
        double best = 1e300;
        int best_n = 1;
        for (int n = 1; n <= max_chunks; ++n) {
            const int c = (p->nz + n - 1) / n;
            const int real_n = (p->nz + c - 1) / c;
            const int64_t ctas = (int64_t)tiles * real_n;
            const double waves = (double)((ctas + slots - 1) / slots);
            const double cost = waves * (c + 2 * T * R + fill);
            if (cost < best * 0.999) { best = cost; best_n = real_n; }
        }
        chunk = (p->nz + best_n - 1) / best_n;
    }
    chunk = std::max(1, std::min(chunk, p->nz));
    g.chunk_z = chunk;
    const int64_t grid64 = (int64_t)tiles * ((p->nz + chunk - 1) / chunk);
    if (grid64 > 0x7fffffffLL) return STENCIL_ERR_UNSUPPORTED;
    // full passes over rows of exactly one region take the instantiation with those facts compiled in
    // ... and the one that also wraps x and z when the pass belongs to a periodic apply (fused_wrap_ok tells
    // the caller beforehand that it will)
    const bool spec = nlev == T && p->nx == cfg->txe;
    auto launch = !spec ? cfg->launch : (p->fused_wrap ? cfg->launch_wrap : cfg->launch_spec);
    if (p->fused_wrap && !spec) return STENCIL_ERR_UNSUPPORTED;
    if (launch(p, *map, dst, g, (int)grid64, smem, st) != cudaSuccess) return STENCIL_ERR_CUDA;
    p->launches++;
    return STENCIL_OK;
}

int launch_sweep(stencil_plan_s* p, const float* src, float* dst, cudaStream_t st) {
    switch (p->variant) {
        case STENCIL_VARIANT_STREAM:
            return p->ndim == 2 ? launch_rows2d(p, src, dst, st) : launch_stream(p, src, dst, st);
        default: return launch_generic(p, src, dst, st);
    }
}

// The sweep launchers read the grid they work on from the plan.  Some applies sweep a plan-owned
// stand-in for the caller's grid (padded rows, a padded periodic copy); this guard swaps the
// stand-in's extents, row length for the tensor maps and boundary into the plan for the
// duration of those launches and puts the plan's own back on every path out.
class ScopedGridView {
public:
    ScopedGridView(stencil_plan_s* p, int nz, int ny, int nx, int tmap_nx, int boundary)
        : p_(p), nz_(p->nz), ny_(p->ny), nx_(p->nx), tmap_nx_(p->tmap_nx), boundary_(p->boundary) {
        p->nz = nz; p->ny = ny; p->nx = nx; p->tmap_nx = tmap_nx; p->boundary = boundary;
    }
    ~ScopedGridView() {
        p_->nz = nz_; p_->ny = ny_; p_->nx = nx_; p_->tmap_nx = tmap_nx_; p_->boundary = boundary_;
        p_->chained = false;
    }
    ScopedGridView(const ScopedGridView&) = delete;
    ScopedGridView& operator=(const ScopedGridView&) = delete;
private:
    stencil_plan_s* p_;
    int nz_, ny_, nx_, tmap_nx_, boundary_;
};

template <typename T>
int repitch_rows(stencil_plan_s* p, const T* src, T* dst, int nx, int src_pitch, int dst_pitch,
                 cudaStream_t st) {
    const int64_t rows = (int64_t)p->nz * p->ny;
    int lanes_log2 = 0;
    while ((1 << lanes_log2) < nx && lanes_log2 < 8) ++lanes_log2;
    const int rows_per_cta = 256 >> lanes_log2;
    const int64_t ctas = (rows + 4 * rows_per_cta - 1) / (4 * rows_per_cta);      // a thread takes 4 rows per round
    const int grid = (int)std::min<int64_t>(ctas, (int64_t)sm_count() * 16);
    stencil_repitch_rows_kernel<T><<<grid, 256, 0, st>>>(src, dst, rows, nx, src_pitch, dst_pitch, lanes_log2);
    if (cudaGetLastError() != cudaSuccess) return STENCIL_ERR_CUDA;
    p->launches++;
    return STENCIL_OK;
}

// Zero-boundary grid whose rows are not a multiple of 4 floats, on the tiled kernels: copy `in`
// into a grid with padded rows, sweep `steps` times between that grid and a second one, copy
// the result into `out`.  While the sweeps run the plan's row length is the padded one (pitch
// of both grids, tile counts, store bounds) and the tensor maps end every row at the true
// length, so the cells the kernels write into the padding never enter a later sweep.
int apply_row_padded(stencil_plan_s* p, const float* in, float* out, int steps, cudaStream_t st) {
    const int nx = p->nx, pitch = (nx + 3) & ~3;
    const int64_t cells = (int64_t)p->nz * p->ny * pitch;
    int rc;
    if ((rc = ensure_grid(&p->pad, cells)) != STENCIL_OK) return rc;
    if ((rc = ensure_grid(&p->pad2, cells)) != STENCIL_OK) return rc;
    if ((rc = repitch_rows(p, in, p->pad, nx, nx, pitch, st)) != STENCIL_OK) return rc;
    float* src = p->pad;
    float* dst = p->pad2;
    {
        ScopedGridView view(p, p->nz, p->ny, pitch, nx, STENCIL_ZERO);
        for (int k = 0; k < steps && rc == STENCIL_OK; ++k) {
            p->chained = p->chain_launches && k > 0;
            rc = launch_sweep(p, src, dst, st);
            std::swap(src, dst);
        }
    }
    if (rc != STENCIL_OK) return rc;
    return repitch_rows(p, src, out, nx, pitch, nx, st);
}


// ---------------------------------------------------------------------------
// FP64 plans: the generic kernel for everything, the row-streaming kernel for
// 2D grids with a zero boundary (the paper's own case)
// ---------------------------------------------------------------------------
inline double dense_w64(const stencil_plan_s* p, int dy, int dx) {
    const int R = p->radius, side = 2 * R + 1;
    return p->w64[(size_t)(dy + R) * side + (dx + R)];
}

template <int R, bool BOX, int YB, int NW>
cudaError_t launch_rows2d64_t(const stencil_plan_s* p, const CUtensorMap& map, double* out, const Rows2DGeom& g,
                              int grid, size_t smem, cudaStream_t st) {
    Weights2D64<R> wt;
    for (int a = -R; a <= R; ++a)
        for (int b = -R; b <= R; ++b) wt.w[a + R][b + R] = dense_w64(p, a, b);
    return launch_kernel(&stencil_rows2d_f64_kernel<R, BOX, YB, NW>, grid, NW * 32, smem, st, p->chained, map, out,
                         g, wt, p->d_status);
}

template <int R, bool BOX, int YB, int NW>
Rows2D64Config make_rows2d64() {
    Rows2D64Config c;
    c.radius = R; c.box = BOX; c.YB = YB; c.NW = NW; c.px = StreamHalo64<R>::PX;
    c.batch_bytes = Rows2D64Shape<YB, StreamHalo64<R>::PX>::BATCH_BYTES;
    c.kernel = reinterpret_cast<const void*>(&stencil_rows2d_f64_kernel<R, BOX, YB, NW>);
    c.smem_allowed = 0; c.cache_device = -1;
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

inline double dense_w64_3d(const stencil_plan_s* p, int dz, int dy, int dx) {
    const int R = p->radius, side = 2 * R + 1;
    return p->w64[((size_t)(dz + R) * side + (dy + R)) * side + (dx + R)];
}

template <int R, bool BOX, int K, int NW, int MINB>
cudaError_t launch_stream64_t(const stencil_plan_s* p, const CUtensorMap& map, double* out, const StreamGeom& g,
                              int grid, size_t smem, cudaStream_t st) {
    StarWeights64<R> sw;
    BoxWeights64<BOX ? R : 0> bw;
    std::memset(&sw, 0, sizeof(sw));
    std::memset(&bw, 0, sizeof(bw));
    if (!BOX) {
        sw.c = dense_w64_3d(p, 0, 0, 0);
        for (int d = -R; d <= R; ++d) {
            if (d == 0) continue;
            sw.x[d + R] = dense_w64_3d(p, 0, 0, d);
            sw.y[d + R] = dense_w64_3d(p, 0, d, 0);
            sw.z[d + R] = dense_w64_3d(p, d, 0, 0);
        }
    } else {
        constexpr int RB = BOX ? R : 0;
        for (int a = -RB; a <= RB; ++a)
            for (int b = -RB; b <= RB; ++b)
                for (int c = -RB; c <= RB; ++c) bw.w[a + RB][b + RB][c + RB] = dense_w64_3d(p, a, b, c);
    }
    return launch_kernel(&stencil_stream_f64_kernel<R, BOX, K, NW, MINB>, grid, Stream64Shape<R, K, NW>::THREADS,
                         smem, st, p->chained, map, out, g, sw, bw, p->d_status);
}

template <int R, bool BOX, int K, int NW, int MINB>
cudaError_t launch_stream64_wrap_t(const stencil_plan_s* p, const CUtensorMap& map, const CUtensorMap& map_xs,
                                   const CUtensorMap& map_ys, const CUtensorMap& map_cs, double* out,
                                   const StreamGeom& g, int grid, size_t smem, cudaStream_t st) {
    StarWeights64<R> sw;
    BoxWeights64<BOX ? R : 0> bw;
    std::memset(&sw, 0, sizeof(sw));
    std::memset(&bw, 0, sizeof(bw));
    if (!BOX) {
        sw.c = dense_w64_3d(p, 0, 0, 0);
        for (int d = -R; d <= R; ++d) {
            if (d == 0) continue;
            sw.x[d + R] = dense_w64_3d(p, 0, 0, d);
            sw.y[d + R] = dense_w64_3d(p, 0, d, 0);
            sw.z[d + R] = dense_w64_3d(p, d, 0, 0);
        }
    } else {
        constexpr int RB = BOX ? R : 0;
        for (int a = -RB; a <= RB; ++a)
            for (int b = -RB; b <= RB; ++b)
                for (int c = -RB; c <= RB; ++c) bw.w[a + RB][b + RB][c + RB] = dense_w64_3d(p, a, b, c);
    }
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
    c.smem_allowed = 0; c.occ_smem = 0; c.occ = 0; c.cache_device = -1;
    c.launch = &launch_stream64_t<R, BOX, K, NW, MINB>;
    c.kernel_wrap = nullptr; c.launch_wrap = nullptr; c.stage_bytes = 0; c.smem_allowed_wrap = 0;
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
    for (int a = -R; a <= R; ++a)
        for (int b = -R; b <= R; ++b) wt.w[a + R][b + R] = dense_w64(p, a, b);
    return launch_kernel(&stencil_rows2d_fused_f64_kernel<R, BOX, T, YB, NW>, grid, NW * 32, smem, st, p->chained,
                         map, out, g, wt, p->d_status);
}

template <int R, bool BOX, int T, int YB, int NW>
Rows2DFused64Config make_rows2d_fused64() {
    Rows2DFused64Config c;
    c.radius = R; c.box = BOX; c.T = T; c.YB = YB; c.NW = NW; c.batch_bytes = Rows2D64Shape<YB>::BATCH_BYTES;
    c.kernel = reinterpret_cast<const void*>(&stencil_rows2d_fused_f64_kernel<R, BOX, T, YB, NW>);
    c.smem_allowed = 0; c.occ_smem = 0; c.occ = 0; c.cache_device = -1;
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
        return STENCIL_OK;
    }
    if (want == STENCIL_VARIANT_STREAM && (c2 || c3)) {
        p->variant = want; p->rows2d64_cfg = c2; p->stream64_cfg = c3;
        p->fused2d64_cfg = c2 ? pick_fused2d64(p) : nullptr;
        return STENCIL_OK;
    }
    return STENCIL_ERR_UNSUPPORTED;
}

int get_tensor_map_f64(stencil_plan_s* p, const void* cfg, int box_x, int box_y, const double* src,
                       const CUtensorMap** out, int tnx = 0, int tny = 0, int tnz = 0) {
    if (tnx == 0) { tnx = p->nx; tny = p->ny; tnz = p->nz; }     // extents of the tensor `src` points at
    const void* key = src;
    for (auto& e : p->maps)
        if (e.ptr == key && e.cfg == cfg) { *out = &e.map; return STENCIL_OK; }
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return STENCIL_ERR_CUDA;
    stencil_plan_s::MapEntry e;
    e.ptr = key; e.cfg = cfg;
    // padded rows: the pitch is p->nx, the cell past the true row length reads as out of grid (zero)
    const cuuint64_t dims[3] = {(cuuint64_t)(p->tmap_nx > 0 ? p->tmap_nx : tnx), (cuuint64_t)tny,
                                (cuuint64_t)tnz};
    const cuuint64_t strides[2] = {(cuuint64_t)tnx * 8, (cuuint64_t)tnx * (cuuint64_t)tny * 8};
    const cuuint32_t box[3] = {(cuuint32_t)box_x, (cuuint32_t)box_y, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(&e.map, CU_TENSOR_MAP_DATA_TYPE_FLOAT64, 3, const_cast<double*>(src), dims, strides, box,
                     estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return STENCIL_ERR_CUDA;
    if (p->maps.size() >= 16) p->maps.erase(p->maps.begin());
    p->maps.push_back(e);
    *out = &p->maps.back().map;
    return STENCIL_OK;
}

// One fused pass of a 2D FP64 grid: nlev time steps (1..T) from src to dst.
int launch_rows2d_fused64(stencil_plan_s* p, const double* src, double* dst, int nlev, cudaStream_t st) {
    const Rows2DFused64Config* cfg = p->fused2d64_cfg;
    const CUtensorMap* map = nullptr;
    int rc = get_tensor_map_f64(p, cfg, kPX64, cfg->YB, src, &map);
    if (rc != STENCIL_OK) return rc;
    int stages = p->stages > 0 ? std::min(p->stages, kMaxStages) : 2;
    auto smem_for = [&](int s_) { return (size_t)cfg->NW * s_ * cfg->batch_bytes + 128 + (size_t)cfg->NW * kMaxStages * 8; };
    while (stages > 2 && smem_for(stages) > 227 * 1024) --stages;      // a ring deeper than shared memory holds is cut back
    const size_t smem = smem_for(stages);
    if (smem > 227 * 1024) return STENCIL_ERR_UNSUPPORTED;
    int dev = -1, occ = 1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return STENCIL_ERR_CUDA; }
    {
        std::lock_guard<std::mutex> lock(g_config_mutex);
        if (dev != cfg->cache_device) { cfg->smem_allowed = 0; cfg->occ_smem = 0; cfg->cache_device = dev; }
        if (smem > cfg->smem_allowed) {
            if (cudaFuncSetAttribute(cfg->kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
                cudaSuccess) {
                cudaGetLastError();
                return STENCIL_ERR_CUDA;
            }
            cfg->smem_allowed = smem;
        }
        if (cfg->occ_smem != smem) {
            int o = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, cfg->kernel, cfg->NW * 32, smem) != cudaSuccess) {
                cudaGetLastError();
                o = 0;
            }
            cfg->occ = std::max(o, 1);
            cfg->occ_smem = smem;
        }
        occ = cfg->occ;
    }
    Rows2DFusedGeom g;
    g.ny = p->ny; g.nx = p->nx;
    g.strips = (p->nx + kFused2D64Tile - 1) / kFused2D64Tile;
    g.stages = stages;
    g.nlev = nlev;
    int chunk = p->chunk_z;
    if (chunk <= 0) {                                 // same sizing rule as the fp32 kernel
        const int H = nlev * p->radius;
        const int slots = occ * sm_count() * cfg->NW;
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
int launch_sweep_f64(stencil_plan_s* p, const double* src, double* dst, cudaStream_t st, int begin = 0, int end = 0) {
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
        while (stages > 2 && smem_for(stages) > 227 * 1024) --stages;      // a ring deeper than shared memory holds is cut back
        const size_t smem = smem_for(stages);
        if (smem > 227 * 1024) return STENCIL_ERR_UNSUPPORTED;
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return STENCIL_ERR_CUDA; }
        {
            std::lock_guard<std::mutex> lock(g_config_mutex);
            if (dev != cfg->cache_device) {
                cfg->smem_allowed = 0; cfg->smem_allowed_wrap = 0; cfg->occ_smem = 0; cfg->cache_device = dev;
            }
            size_t& allowed = wrap ? cfg->smem_allowed_wrap : cfg->smem_allowed;
            if (smem > allowed) {
                if (cudaFuncSetAttribute(wrap ? cfg->kernel_wrap : cfg->kernel,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
                    cudaGetLastError();
                    return STENCIL_ERR_CUDA;
                }
                allowed = smem;
            }
        }
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
        g.wait_polls = p->wait_polls; g.drop_plane = -1;
        // many short CTAs, as for the bandwidth-bound fp32 sweeps; the wide stars re-read 2R halo
        // planes per chunk, so they get longer chunks (measured on 512^3)
        const int want_chunk = p->radius >= 3 ? 64 : 32;
        int chunk = p->chunk_z > 0 ? p->chunk_z : (span >= 2 * want_chunk ? want_chunk : span);
        if (p->chunk_z <= 0 && p->shape == STENCIL_STAR && p->radius == 1 && span >= 16) {
            int occ64 = 0;                            // the 7-point star: very short chunks, as in fp32
            {
                std::lock_guard<std::mutex> lock(g_config_mutex);
                if (cfg->occ_smem != smem) {          // asked once per device and size
                    int o = 0;
                    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, cfg->kernel, cfg->threads, smem) !=
                        cudaSuccess) {
                        cudaGetLastError();
                        o = 0;
                    }
                    cfg->occ = std::max(o, 1);
                    cfg->occ_smem = smem;
                }
                occ64 = cfg->occ;
            }
            chunk = short_chunk_star1(span, (int64_t)g.tiles_x * g.tiles_y, (int64_t)occ64 * sm_count());
        }
        if (p->chunk_z <= 0 && (p->radius >= 4 || (p->shape == STENCIL_BOX && p->radius >= 2))) {
            // The radius-4 star is no longer bound by memory alone (25 DFMA and 15 shared-memory
            // loads per pair of points) and the 125-point box is bound by the FP64 pipe: every SM
            // should get the same number of planes and as
            // few re-read halo planes as possible, so z is cut into the number of chunks whose
            // CTAs fill whole waves of the two-per-SM slots at the least cost (512^3: one chunk,
            // 296 CTAs, 356 against 313 GPoints/s with 64-plane chunks).
            const int64_t tiles = (int64_t)g.tiles_x * g.tiles_y;
            const int64_t slots = 2 * (int64_t)sm_count();
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
        while (stages > 2 && smem_for(stages) > 227 * 1024) --stages;      // a ring deeper than shared memory holds is cut back
        const size_t smem = smem_for(stages);
        if (smem > 227 * 1024) return STENCIL_ERR_UNSUPPORTED;
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return STENCIL_ERR_CUDA; }
        {
            std::lock_guard<std::mutex> lock(g_config_mutex);
            if (dev != cfg->cache_device) { cfg->smem_allowed = 0; cfg->cache_device = dev; }
            if (smem > cfg->smem_allowed) {
                if (cudaFuncSetAttribute(cfg->kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
                    cudaSuccess) {
                    cudaGetLastError();
                    return STENCIL_ERR_CUDA;
                }
                cfg->smem_allowed = smem;
            }
        }
        Rows2DGeom g;
        g.ny = p->ny; g.nx = p->nx;
        g.strips = (p->nx + kStrip64 - 1) / kStrip64;
        g.stages = stages;
        g.in_off_x = periodic ? kPadX : 0;
        g.in_off_y = periodic ? p->radius : 0;
        int chunk = p->chunk_z;
        if (chunk <= 0) {                             // same sizing rule as the fp32 kernel
            const int R = p->radius;
            const int slots = 2 * sm_count() * cfg->NW;
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
        const int64_t units = (int64_t)g.strips * g.nchunks;
        const int64_t grid64 = (units + cfg->NW - 1) / cfg->NW;
        if (grid64 > 0x7fffffffLL) return STENCIL_ERR_UNSUPPORTED;
        if (cfg->launch(p, *map, dst, g, (int)grid64, smem, st) != cudaSuccess) return STENCIL_ERR_CUDA;
        p->launches++;
        return STENCIL_OK;
    }
    Grid g{p->nz, p->ny, p->nx};
    const int grid = generic_grid_size(g, sm_count());
    const int ntaps = (int)p->taps64.size();
    if (p->boundary == STENCIL_PERIODIC)
        stencil_generic_kernel<true, double><<<grid, kGenericThreads, 0, st>>>(src, dst, g, p->d_taps64, ntaps);
    else
        stencil_generic_kernel<false, double><<<grid, kGenericThreads, 0, st>>>(src, dst, g, p->d_taps64, ntaps);
    if (cudaGetLastError() != cudaSuccess) return STENCIL_ERR_CUDA;
    p->launches++;
    return STENCIL_OK;
}

int sweep_any(stencil_plan_s* p, const float* src, float* dst, cudaStream_t st) { return launch_sweep(p, src, dst, st); }
int sweep_any(stencil_plan_s* p, const double* src, double* dst, cudaStream_t st) {
    return launch_sweep_f64(p, src, dst, st);
}

// Iterated periodic apply on the tiled kernels.  `in` is copied once into a padded grid with
// wrapped halos.  Every step but the last sweeps the whole padded grid as if it were a grid
// with a zero boundary (the interior comes out right, the halo cells do not) into a second
// padded grid and then rewrites that grid's halo cells from its interior; the last step reads
// the padded grid with shifted coordinates and writes `out`.  Per step: one sweep over a
// slightly larger grid and a copy of the halo shell, instead of a padded copy of everything.
template <typename T>
int apply_periodic(stencil_plan_s* p, const T* in, T* out, int steps, cudaStream_t st) {
    const int R = p->radius, rz = p->ndim == 3 ? R : 0;
    int pnx, pny, pnz, rc;
    const T* padded = nullptr;
    if ((rc = pad_periodic(p, in, st, &padded, &pnx, &pny, &pnz)) != STENCIL_OK) return rc;
    const int64_t cells = (int64_t)pnx * pny * pnz;
    if ((rc = ensure_grid(&p->pad2, cells * (int64_t)(sizeof(T) / sizeof(float)))) != STENCIL_OK) return rc;
    T* a = reinterpret_cast<T*>(p->pad);
    T* b = reinterpret_cast<T*>(p->pad2);
    const Grid g{p->nz, p->ny, p->nx};
    const int nz = p->nz, ny = p->ny, nx = p->nx;
    const int64_t shell = cells / Vec16<T>::n - (int64_t)nz * ny * (nx / Vec16<T>::n);
    const int shell_grid = (int)std::max<int64_t>(1, std::min<int64_t>((shell + 255) / 256, (int64_t)sm_count() * 16));
    for (int k = 0; k + 1 < steps && rc == STENCIL_OK; ++k) {
        {
            ScopedGridView view(p, pnz, pny, pnx, 0, STENCIL_ZERO);
            rc = sweep_any(p, static_cast<const T*>(a), b, st);
        }
        if (rc != STENCIL_OK) break;
        stencil_refresh_halo_kernel<T><<<shell_grid, 256, 0, st>>>(b, g, R, rz);
        if (cudaGetLastError() != cudaSuccess) rc = STENCIL_ERR_CUDA;
        p->launches++;
        std::swap(a, b);
    }
    if (rc != STENCIL_OK) return rc;
    p->src_padded = true;
    rc = sweep_any(p, static_cast<const T*>(a), out, st);
    p->src_padded = false;
    return rc;
}

inline const Tap* device_taps(const stencil_plan_s* p, const float*) { return p->d_taps; }
inline const TapT<double>* device_taps(const stencil_plan_s* p, const double*) { return p->d_taps64; }
inline int tap_count(const stencil_plan_s* p, const float*) { return (int)p->taps.size(); }
inline int tap_count(const stencil_plan_s* p, const double*) { return (int)p->taps64.size(); }

// The wrap-correction route needs the three parts of the boundary shell to be disjoint.
bool wrap_correction_fits(const stencil_plan_s* p) {
    const int R = p->radius;
    return p->nx >= 2 * R && p->ny >= 2 * R && (p->ndim == 2 || p->nz >= 2 * R);
}

// Which periodic route an apply of `steps` steps takes: true = zero-boundary sweep plus wrap
// correction, false = padded copy.  The correction costs one pass over the taps of every
// shell point, the padded route one copy of the grid per apply (plus a shell copy per step):
// measured on 512^3, the correction wins except for the 125-tap box and, when the copy is
// spread over several steps, for the wide 3D stars.
bool use_wrap_correction(const stencil_plan_s* p, int steps) {
    if (p->radius > 4) return true;                 // the only periodic route of the wide stars (see stream_supported)
    if (p->periodic_route == 1 || !wrap_correction_fits(p)) return false;
    if (p->periodic_route == 2) return true;
    if (p->ndim == 3 && p->shape == STENCIL_BOX && p->radius >= 2) return false;
    if (p->ndim == 3 && p->shape == STENCIL_STAR && p->radius >= 3 && steps > 1) return false;
    return true;
}

// Periodic apply on the tiled kernels without a padded copy: every step is a zero-boundary
// sweep followed by stencil_wrap_correction_kernel, which adds the wrapped taps to the points
// within R of a face.  `other` is the plan's ping-pong grid (used when steps > 1).
template <typename T>
int apply_periodic_corrected(stencil_plan_s* p, const T* in, T* out, T* other, int steps, cudaStream_t st) {
    const int R = p->radius, rz = p->ndim == 3 ? R : 0;
    const Grid g{p->nz, p->ny, p->nx};
    const int64_t shell = (int64_t)2 * rz * g.ny * g.nx + (int64_t)(g.nz - 2 * rz) * 2 * R * g.nx +
                          (int64_t)(g.nz - 2 * rz) * (g.ny - 2 * R) * 2 * R;
    const int shell_grid = (int)std::max<int64_t>(1, std::min<int64_t>((shell + 255) / 256, (int64_t)sm_count() * 16));
    const T* src = in;
    for (int k = 0; k < steps; ++k) {
        T* dst = ((steps - 1 - k) % 2 == 0) ? out : other;
        int rc;
        {
            ScopedGridView view(p, p->nz, p->ny, p->nx, 0, STENCIL_ZERO);
            rc = sweep_any(p, src, dst, st);
        }
        if (rc != STENCIL_OK) return rc;
        if (shell > 0) {
            stencil_wrap_correction_kernel<T><<<shell_grid, 256, 0, st>>>(src, dst, g, R, rz, device_taps(p, src),
                                                                           tap_count(p, src));
            if (cudaGetLastError() != cudaSuccess) return STENCIL_ERR_CUDA;
            p->launches++;
        }
        src = dst;
    }
    return STENCIL_OK;
}

// A periodic 3D star of radius <= 4 or box whose rows are a whole number of tiles is swept by
// the kernel that wraps all three axes itself: no correction pass, no padded copy.
bool stream_wrap_ok(const stencil_plan_s* p) {
    if (p->ndim != 3 || p->variant != STENCIL_VARIANT_STREAM || !wrap_correction_fits(p)) return false;
    if (p->f64) return p->stream64_cfg && p->stream64_cfg->launch_wrap && p->nx % kStream64TX == 0;
    return p->stream_cfg && p->stream_cfg->launch_wrap && p->nx % kStreamTX == 0;
}

int launch_sweep_f64(stencil_plan_s* p, const double* src, double* dst, cudaStream_t st, int begin, int end);
inline int wrapped_sweep(stencil_plan_s* p, const float* src, float* dst, cudaStream_t st) {
    return launch_stream(p, src, dst, st);
}
inline int wrapped_sweep(stencil_plan_s* p, const double* src, double* dst, cudaStream_t st) {
    return launch_sweep_f64(p, src, dst, st, 0, 0);
}

template <typename T>
int apply_periodic_inkernel(stencil_plan_s* p, const T* in, T* out, T* other, int steps, cudaStream_t st) {
    const T* src = in;
    for (int k = 0; k < steps; ++k) {
        T* dst = ((steps - 1 - k) % 2 == 0) ? out : other;
        int rc;
        {
            ScopedGridView view(p, p->nz, p->ny, p->nx, 0, STENCIL_ZERO);
            p->stream_wrap = true;
            p->chained = p->chain_launches && k > 0;
            rc = wrapped_sweep(p, src, dst, st);
            p->stream_wrap = false;
        }
        if (rc != STENCIL_OK) return rc;
        src = dst;
    }
    return STENCIL_OK;
}

// Taps of the operator applied L times in a row (its L-fold self-convolution: the sweep is a
// cross-correlation, and correlating with w twice is correlating with w * w), as doubles on the
// device.  Built from the plan's own weights at first need.
int composite_taps(stencil_plan_s* p, int L, const TapT<double>** taps, int* ntaps) {
    if (L < 1 || L > kMaxFuseLevels) return STENCIL_ERR_UNSUPPORTED;
    if (!p->d_ctaps[L]) {
        const int R = p->radius, side = 2 * R + 1, sz = p->ndim == 3 ? side : 1;
        std::vector<TapT<double>> out;
        try {
            std::vector<double> w((size_t)sz * side * side);
            for (size_t f = 0; f < w.size(); ++f) w[f] = p->f64 ? p->w64[f] : (double)p->w[f];
            std::vector<double> c = w;                                   // composite of l steps, radius l * R
            for (int l = 2; l <= L; ++l) {
                const int cs = 2 * (l - 1) * R + 1, cz = p->ndim == 3 ? cs : 1;
                const int ns = cs + 2 * R, nz = p->ndim == 3 ? ns : 1;
                std::vector<double> n((size_t)nz * ns * ns, 0.0);
                for (int az = 0; az < cz; ++az)
                    for (int ay = 0; ay < cs; ++ay)
                        for (int ax = 0; ax < cs; ++ax) {
                            const double cv = c[((size_t)az * cs + ay) * cs + ax];
                            if (cv == 0.0) continue;
                            for (int bz = 0; bz < sz; ++bz)
                                for (int by = 0; by < side; ++by)
                                    for (int bx = 0; bx < side; ++bx)
                                        n[((size_t)(az + bz) * ns + (ay + by)) * ns + (ax + bx)] +=
                                            cv * w[((size_t)bz * side + by) * side + bx];
                        }
                c.swap(n);
            }
            const int H = L * R, cs = 2 * H + 1, cz = p->ndim == 3 ? cs : 1;
            for (int z = 0; z < cz; ++z)
                for (int y = 0; y < cs; ++y)
                    for (int x = 0; x < cs; ++x) {
                        const double v = c[((size_t)z * cs + y) * cs + x];
                        if (v != 0.0) out.push_back(TapT<double>{p->ndim == 3 ? z - H : 0, y - H, x - H, v});
                    }
        } catch (...) {
            return STENCIL_ERR_ALLOC;
        }
        if (out.empty()) out.push_back(TapT<double>{0, 0, 0, 0.0});      // an all-zero operator
        TapT<double>* d = nullptr;
        const size_t bytes = out.size() * sizeof(TapT<double>);
        if (cudaMalloc(&d, bytes) != cudaSuccess) { cudaGetLastError(); return STENCIL_ERR_ALLOC; }
        if (cudaMemcpy(d, out.data(), bytes, cudaMemcpyHostToDevice) != cudaSuccess) {
            cudaGetLastError();
            cudaFree(d);
            return STENCIL_ERR_CUDA;
        }
        p->ctaps[L].swap(out);
        p->d_ctaps[L] = d;
    }
    *taps = p->d_ctaps[L];
    *ntaps = (int)p->ctaps[L].size();
    return STENCIL_OK;
}

// One periodic step with the kernel that wraps all three axes, where it applies (fp32 3D stars).
bool sweep_wrapped(stencil_plan_s* p, const float* src, float* dst, cudaStream_t st, int* rc) {
    if (!stream_wrap_ok(p)) return false;
    ScopedGridView view(p, p->nz, p->ny, p->nx, 0, STENCIL_ZERO);
    p->stream_wrap = true;
    *rc = launch_stream(p, src, dst, st);
    p->stream_wrap = false;
    return true;
}
bool sweep_wrapped(stencil_plan_s*, const double*, double*, cudaStream_t, int*) { return false; }

int fused_any(stencil_plan_s* p, const float* src, float* dst, int nlev, cudaStream_t st) {
    return p->ndim == 3 ? launch_fused(p, src, dst, nlev, st) : launch_rows2d_fused(p, src, dst, nlev, st);
}
int fused_any(stencil_plan_s* p, const double* src, double* dst, int nlev, cudaStream_t st) {
    return launch_rows2d_fused64(p, src, dst, nlev, st);
}

// A full 3D pass over rows of exactly one region can wrap x and z inside the fused kernel; only the
// rows next to the y faces are then left to put right.
bool fused_wrap_ok(const stencil_plan_s* p, int nlev) {
    return !p->f64 && p->ndim == 3 && p->fused_cfg && nlev == p->fused_cfg->T && p->nx == p->fused_cfg->txe;
}

// Iterated periodic apply under temporal blocking: every pass is a fused zero-boundary pass of
// L <= T steps, right everywhere but within L*R cells of a face, followed by
// stencil_shell_compose_kernel, which rewrites that shell from the pass's input.
template <typename T>
int apply_periodic_fused(stencil_plan_s* p, const T* in, T* out, T* other, int steps, int depth, cudaStream_t st) {
    const int R = p->radius;
    const Grid g{p->nz, p->ny, p->nx};
    const int passes = (steps + depth - 1) / depth;
    const T* src = in;
    int done = 0;
    for (int k = 0; k < passes; ++k) {
        T* dst = ((passes - 1 - k) % 2 == 0) ? out : other;
        const int L = std::min(depth, steps - done);
        const TapT<double>* taps = nullptr;
        int ntaps = 0, rc;
        if ((rc = composite_taps(p, L, &taps, &ntaps)) != STENCIL_OK) return rc;
        if (L == 1 && sweep_wrapped(p, src, dst, st, &rc)) {       // a last single step needs no shell kernel
            if (rc != STENCIL_OK) return rc;
            done += L;
            src = dst;
            continue;
        }
        const bool wrapped = L > 1 && fused_wrap_ok(p, L);
        {
            ScopedGridView view(p, p->nz, p->ny, p->nx, 0, STENCIL_ZERO);
            p->fused_wrap = wrapped;
            // a programmatic dependent launch behind the previous pass's shell kernel: the preamble runs
            // while that kernel drains, and the pass waits for all of it before it touches global memory
            p->chained = p->chain_launches && k > 0;
            rc = L > 1 ? fused_any(p, src, dst, L, st) : sweep_any(p, src, dst, st);
            p->fused_wrap = false;
        }
        if (rc != STENCIL_OK) return rc;
        const int H = L * R;
        if (wrapped) {
            // x and z are right already: the 2H rows next to the y faces of every plane remain (the row
            // kernel with a z shell of depth 0 walks exactly those, wrapping the taps' planes itself)
            const int xchunks = (g.nx + kShellRowChunk - 1) / kShellRowChunk;
            const int64_t nrows = (int64_t)g.nz * 2 * H * xchunks;
            if (ntaps <= kShellTaps && nrows <= 0x7fffffffLL) {
                if (launch_kernel(&stencil_shell_rows_kernel<T>, (int)nrows, 256, 0, st, p->chain_launches, src, dst, g, H,
                                  0, taps, ntaps, xchunks) != cudaSuccess)
                    return STENCIL_ERR_CUDA;
                p->launches++;
                done += L;
                src = dst;
                continue;
            }
            // (an operator with too many composite taps for the row kernel: the whole shell below, which
            // rewrites the x and z faces with the values they already have)
        }
        const int hz = p->ndim == 3 ? H : 0;
        // 3D: whole rows of the shell and the ends of the other rows go to their own kernels (512^3,
        // 7-point star, two steps per pass: 74 us against 124 us for the point-by-point walk).
        // Operators with very many composite taps, shells too deep for the tile, rows too short to
        // occupy a CTA each and 2D grids (whose shell is a few rows and columns: the walk spreads
        // them over more threads, 10240^2 5-point 1924 against 1838 G updates/s) take the walk.
        const int inner_z = g.nz - 2 * hz, inner_y = g.ny - 2 * H;
        const int tz = shell_tz(H, hz);
        const size_t seg_bytes = (size_t)(tz + 2 * hz) * (kShellTY + 2 * H) * 4 * H * sizeof(T);
        const int xchunks = (g.nx + kShellRowChunk - 1) / kShellRowChunk;
        const int64_t nrows = ((int64_t)2 * hz * g.ny + (int64_t)inner_z * 2 * H) * xchunks;     // CTAs of the row kernel
        const int64_t xtiles = (inner_z > 0 && inner_y > 0)
                                   ? (int64_t)((inner_y + kShellTY - 1) / kShellTY) * ((inner_z + tz - 1) / tz) : 0;
        if (p->ndim == 3 && ntaps <= kShellTaps && seg_bytes <= 40 * 1024 && g.nx >= 64 && nrows <= 0x7fffffffLL &&
            xtiles <= 0x7fffffffLL) {
            if (nrows > 0) {
                stencil_shell_rows_kernel<T><<<(int)nrows, 256, 0, st>>>(src, dst, g, H, hz, taps, ntaps, xchunks);
                if (cudaGetLastError() != cudaSuccess) return STENCIL_ERR_CUDA;
                p->launches++;
            }
            if (xtiles > 0) {
                stencil_shell_xfaces_kernel<T><<<(int)xtiles, 256, seg_bytes, st>>>(src, dst, g, H, hz, taps, ntaps);
                if (cudaGetLastError() != cudaSuccess) return STENCIL_ERR_CUDA;
                p->launches++;
            }
        } else {
            const int64_t shell = (int64_t)2 * hz * g.ny * g.nx + (int64_t)inner_z * 2 * H * g.nx +
                                  (int64_t)inner_z * inner_y * 2 * H;
            const int shell_grid = (int)std::max<int64_t>(1, std::min<int64_t>((shell + 255) / 256, (int64_t)sm_count() * 16));
            // 32-bit indices where the grid leaves room for the grid-stride loop's last increment
            if (p->npoints < ((int64_t)1 << 31) - ((int64_t)1 << 24))
                stencil_shell_compose_kernel<T, int><<<shell_grid, 256, 0, st>>>(src, dst, g, H, hz, taps, ntaps);
            else
                stencil_shell_compose_kernel<T, int64_t><<<shell_grid, 256, 0, st>>>(src, dst, g, H, hz, taps, ntaps);
            if (cudaGetLastError() != cudaSuccess) return STENCIL_ERR_CUDA;
            p->launches++;
        }
        done += L;
        src = dst;
    }
    return STENCIL_OK;
}


// FP64 twin of apply_row_padded: rows of an odd number of doubles, pitch rounded up to even.
// The two padded grids live in the same plan slots, sized in doubles.
int apply_row_padded_f64(stencil_plan_s* p, const double* in, double* out, int steps, cudaStream_t st) {
    const int nx = p->nx, pitch = nx + 1;
    const int64_t cells = (int64_t)p->nz * p->ny * pitch;
    int rc;
    if ((rc = ensure_grid(&p->pad, 2 * cells)) != STENCIL_OK) return rc;
    if ((rc = ensure_grid(&p->pad2, 2 * cells)) != STENCIL_OK) return rc;
    double* src = reinterpret_cast<double*>(p->pad);
    double* dst = reinterpret_cast<double*>(p->pad2);
    if ((rc = repitch_rows(p, in, src, nx, nx, pitch, st)) != STENCIL_OK) return rc;
    {
        ScopedGridView view(p, p->nz, p->ny, pitch, nx, STENCIL_ZERO);
        for (int k = 0; k < steps && rc == STENCIL_OK; ++k) {
            p->chained = p->chain_launches && k > 0;
            rc = launch_sweep_f64(p, src, dst, st);
            std::swap(src, dst);
        }
    }
    if (rc != STENCIL_OK) return rc;
    return repitch_rows(p, static_cast<const double*>(src), out, nx, pitch, nx, st);
}

bool valid_plan(const stencil_plan_s* p) { return p && p->magic == kPlanMagic; }

// ---------------------------------------------------------------------------
// plan construction, shared by the fp32 and the FP64 entry point
// ---------------------------------------------------------------------------
template <typename T>
int make_plan(stencil_plan_t* plan_out, int ndim, const int64_t* dims, int radius, int shape,
              const T* weights, int boundary) {
    constexpr bool kF64 = sizeof(T) == 8;
    if (!plan_out) return STENCIL_ERR_INVALID;
    *plan_out = nullptr;
    if ((ndim != 2 && ndim != 3) || !dims || !weights) return STENCIL_ERR_INVALID;
    if (shape != STENCIL_STAR && shape != STENCIL_BOX) return STENCIL_ERR_INVALID;
    if (boundary != STENCIL_ZERO && boundary != STENCIL_PERIODIC) return STENCIL_ERR_INVALID;
    if (radius < 1) return STENCIL_ERR_INVALID;
    if (radius > kMaxRadius) return STENCIL_ERR_UNSUPPORTED;
    int64_t n = 1;
    for (int i = 0; i < ndim; ++i) {
        if (dims[i] < 1) return STENCIL_ERR_INVALID;
        if (dims[i] > 0x7fffffffLL) return STENCIL_ERR_UNSUPPORTED;
        if (n > (int64_t)1 << 40) return STENCIL_ERR_UNSUPPORTED;
        n *= dims[i];
    }

    stencil_plan_s* p = new (std::nothrow) stencil_plan_s();
    if (!p) return STENCIL_ERR_ALLOC;
    p->magic = kPlanMagic;
    p->f64 = kF64;
    p->ndim = ndim;
    p->nz = ndim == 3 ? (int)dims[0] : 1;
    p->ny = ndim == 3 ? (int)dims[1] : (int)dims[0];
    p->nx = ndim == 3 ? (int)dims[2] : (int)dims[1];
    p->npoints = n;
    p->radius = radius; p->shape = shape; p->boundary = boundary;
    p->device = -1;
    p->d_taps = nullptr; p->d_status = nullptr; p->scratch = nullptr; p->pad = nullptr; p->pad2 = nullptr; p->tmap_nx = 0; p->src_padded = false; p->fused_wrap = false; p->stream_wrap = false; p->periodic_route = 0;
    for (int l = 0; l <= kMaxFuseLevels; ++l) p->d_ctaps[l] = nullptr;
    p->d_taps64 = nullptr; p->scratch64 = nullptr; p->rows2d64_cfg = nullptr; p->stream64_cfg = nullptr; p->fused2d64_cfg = nullptr;
    p->host_in = nullptr; p->host_out = nullptr;
    p->copy_in = nullptr; p->copy_out = nullptr;
    p->variant = STENCIL_VARIANT_GENERIC;
    p->tile_y = 0; p->rows_per_thread = 0; p->chunk_z = 0; p->stages = 0; p->fuse_steps = 0; p->streaming_store = 0;
    p->stream_cfg = nullptr; p->fused_cfg = nullptr; p->rows2d_cfg = nullptr; p->fused2d_cfg = nullptr; p->tile_x = 0; p->fused_tile_y = 0;
    p->stream_cfg_fixed = false; p->stream_cfg_tuned = false;
    p->wait_polls = kWaitPolls; p->drop_plane = -1;
    p->chain_launches = true; p->chained = false;
    p->launches = 0; p->last_stream = nullptr; p->used = false;

    const int side = 2 * radius + 1;
    size_t count = 1;
    for (int i = 0; i < ndim; ++i) count *= (size_t)side;
    try {
        if constexpr (kF64) p->w64.assign(weights, weights + count);
        else p->w.assign(weights, weights + count);
        for (size_t f = 0; f < count; ++f) {
            const T wv = weights[f];
            int dx = (int)(f % side) - radius;
            int dy = (int)((f / side) % side) - radius;
            int dz = ndim == 3 ? (int)(f / ((size_t)side * side)) - radius : 0;
            const int nonzero_axes = (dx != 0) + (dy != 0) + (dz != 0);
            if (shape == STENCIL_STAR && nonzero_axes > 1 && wv != T(0)) {
                delete p;
                return STENCIL_ERR_INVALID;       // STAR promises zero off-axis weights
            }
            if (wv != T(0)) {
                if constexpr (kF64) p->taps64.push_back(TapT<double>{dz, dy, dx, wv});
                else p->taps.push_back(Tap{dz, dy, dx, wv});
            }
        }
    } catch (...) {
        delete p;
        return STENCIL_ERR_ALLOC;
    }
    if (kF64) resolve_variant_f64(p, STENCIL_VARIANT_AUTO);
    else resolve_variant(p, STENCIL_VARIANT_AUTO);
    *plan_out = p;
    return STENCIL_OK;
}


// ---------------------------------------------------------------------------
// Fixed scratch for stencil_apply_static: the ping-pong grid and the tap list
// live in one file-scope device array, so that entry point never allocates.
// Every GPU that loads the library holds these bytes until the process exits.
// ---------------------------------------------------------------------------
constexpr int64_t kStaticMaxPoints = STENCIL_STATIC_MAX_POINTS;
constexpr int kStaticMaxTaps = (2 * kMaxRadius + 1) * (2 * kMaxRadius + 1) * (2 * kMaxRadius + 1);
constexpr size_t kStaticGridBytes = (size_t)kStaticMaxPoints * sizeof(float);
constexpr size_t kStaticTapBytes = ((size_t)kStaticMaxTaps * sizeof(Tap) + 255) / 256 * 256;
constexpr int kStaticMaxDevices = 64;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticGridBytes + kStaticTapBytes];

// In host code `g_static_scratch` is only a handle; the device address has to be
// asked for, once per device, while that device is current.
std::mutex g_static_mutex;
unsigned char* g_static_ptr[kStaticMaxDevices] = {nullptr};

int static_scratch_address(unsigned char** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return STENCIL_ERR_CUDA; }
    if (dev < 0 || dev >= kStaticMaxDevices) return STENCIL_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return STENCIL_ERR_CUDA;
        }
        g_static_ptr[dev] = static_cast<unsigned char*>(ptr);
    }
    *out = g_static_ptr[dev];
    return STENCIL_OK;
}

}  // namespace

// ===========================================================================
// C ABI
// ===========================================================================
extern "C" {

int stencil_plan(stencil_plan_t* plan_out, int ndim, const int64_t* dims, int radius, int shape,
                 const float* weights, int boundary) {
    return make_plan<float>(plan_out, ndim, dims, radius, shape, weights, boundary);
}

int stencil_plan_f64(stencil_plan_t* plan_out, int ndim, const int64_t* dims, int radius, int shape,
                     const double* weights, int boundary) {
    return make_plan<double>(plan_out, ndim, dims, radius, shape, weights, boundary);
}

int stencil_apply(stencil_plan_t p, const float* in, float* out, int steps, void* stream) {
    if (!valid_plan(p) || p->f64 || !in || !out || steps < 0) return STENCIL_ERR_INVALID;
    const uintptr_t a = reinterpret_cast<uintptr_t>(in), b = reinterpret_cast<uintptr_t>(out);
    if ((a | b) & 15u) return STENCIL_ERR_INVALID;
    const uintptr_t bytes = (uintptr_t)p->npoints * sizeof(float);
    if (a < b + bytes && b < a + bytes) return STENCIL_ERR_INVALID;      // overlap (covers in == out)
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

    int rc = ensure_device_state(p);
    if (rc != STENCIL_OK) return rc;
    p->last_stream = st;
    p->used = true;

    if (steps == 0) {
        if (cudaMemcpyAsync(out, in, bytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess) {
            cudaGetLastError();
            return STENCIL_ERR_CUDA;
        }
        return STENCIL_OK;
    }
    if (p->variant == STENCIL_VARIANT_STREAM && p->nx % 4 != 0) return apply_row_padded(p, in, out, steps, st);
    if (steps > 1) {
        rc = ensure_grid(&p->scratch, p->npoints);
        if (rc != STENCIL_OK) return rc;
    }
    if (p->variant == STENCIL_VARIANT_STREAM && p->boundary == STENCIL_PERIODIC) {
        const int depth = p->fused_cfg ? p->fused_cfg->T : p->fused2d_cfg ? p->fused2d_cfg->T : 1;
        if (steps > 1 && depth > 1 && p->periodic_route != 1)
            return apply_periodic_fused(p, in, out, p->scratch, steps, depth, st);
        if (p->periodic_route == 0 && stream_wrap_ok(p)) return apply_periodic_inkernel(p, in, out, p->scratch, steps, st);
        if (use_wrap_correction(p, steps)) return apply_periodic_corrected(p, in, out, p->scratch, steps, st);
        if (steps > 1) return apply_periodic(p, in, out, steps, st);
    }
    // A pass advances the field by T time steps (T = 1 without temporal blocking).
    // Ping-pong between `out` and the scratch grid so that the last pass writes
    // `out` and `in` stays intact.
    const bool fuse3d = p->variant == STENCIL_VARIANT_STREAM && p->fused_cfg != nullptr && steps > 1;
    const bool fuse2d = p->variant == STENCIL_VARIANT_STREAM && p->fused2d_cfg != nullptr && steps > 1;
    const bool fuse = fuse3d || fuse2d;
    const int T = fuse3d ? p->fused_cfg->T : fuse2d ? p->fused2d_cfg->T : 1;
    const int passes = (steps + T - 1) / T;
    const float* src = in;
    int done = 0;
    for (int k = 0; k < passes; ++k) {
        const int remaining = passes - 1 - k;
        float* dst = (remaining % 2 == 0) ? out : p->scratch;
        const int nlev = std::min(T, steps - done);
        p->chained = p->chain_launches && k > 0;
        rc = !(fuse && nlev > 1) ? launch_sweep(p, src, dst, st)
             : fuse3d           ? launch_fused(p, src, dst, nlev, st)
                                : launch_rows2d_fused(p, src, dst, nlev, st);
        p->chained = false;
        if (rc != STENCIL_OK) return rc;
        done += nlev;
        src = dst;
    }
    return STENCIL_OK;
}

int stencil_apply_planes(stencil_plan_t p, const float* in, float* out, int64_t z_begin, int64_t z_end,
                         void* stream) {
    if (!valid_plan(p) || p->f64 || !in || !out) return STENCIL_ERR_INVALID;
    const uintptr_t a = reinterpret_cast<uintptr_t>(in), b = reinterpret_cast<uintptr_t>(out);
    if ((a | b) & 15u) return STENCIL_ERR_INVALID;
    const uintptr_t bytes = (uintptr_t)p->npoints * sizeof(float);
    if (a < b + bytes && b < a + bytes) return STENCIL_ERR_INVALID;
    const int slow = p->ndim == 3 ? p->nz : p->ny;
    if (z_begin < 0 || z_end > slow || z_begin >= z_end) return STENCIL_ERR_INVALID;
    if (p->variant != STENCIL_VARIANT_STREAM || p->boundary != STENCIL_ZERO || p->nx % 4 != 0)
        return STENCIL_ERR_UNSUPPORTED;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int rc = ensure_device_state(p);
    if (rc != STENCIL_OK) return rc;
    p->last_stream = st;
    p->used = true;
    return p->ndim == 3 ? launch_stream(p, in, out, st, (int)z_begin, (int)z_end)
                        : launch_rows2d(p, in, out, st, (int)z_begin, (int)z_end);
}

int stencil_apply_planes_f64(stencil_plan_t p, const double* in, double* out, int64_t z_begin, int64_t z_end,
                             void* stream) {
    if (!valid_plan(p) || !p->f64 || !in || !out) return STENCIL_ERR_INVALID;
    const uintptr_t a = reinterpret_cast<uintptr_t>(in), b = reinterpret_cast<uintptr_t>(out);
    if ((a | b) & 15u) return STENCIL_ERR_INVALID;
    const uintptr_t bytes = (uintptr_t)p->npoints * sizeof(double);
    if (a < b + bytes && b < a + bytes) return STENCIL_ERR_INVALID;
    const int slow = p->ndim == 3 ? p->nz : p->ny;
    if (z_begin < 0 || z_end > slow || z_begin >= z_end) return STENCIL_ERR_INVALID;
    if (p->variant != STENCIL_VARIANT_STREAM || p->boundary != STENCIL_ZERO || p->nx % 2 != 0)
        return STENCIL_ERR_UNSUPPORTED;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int rc = ensure_device_state(p);
    if (rc != STENCIL_OK) return rc;
    p->last_stream = st;
    p->used = true;
    return launch_sweep_f64(p, in, out, st, (int)z_begin, (int)z_end);
}

int stencil_apply_f64(stencil_plan_t p, const double* in, double* out, int steps, void* stream) {
    if (!valid_plan(p) || !p->f64 || !in || !out || steps < 0) return STENCIL_ERR_INVALID;
    const uintptr_t a = reinterpret_cast<uintptr_t>(in), b = reinterpret_cast<uintptr_t>(out);
    if ((a | b) & 15u) return STENCIL_ERR_INVALID;
    const uintptr_t bytes = (uintptr_t)p->npoints * sizeof(double);
    if (a < b + bytes && b < a + bytes) return STENCIL_ERR_INVALID;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    int rc = ensure_device_state(p);
    if (rc != STENCIL_OK) return rc;
    p->last_stream = st;
    p->used = true;
    if (steps == 0) {
        if (cudaMemcpyAsync(out, in, bytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess) {
            cudaGetLastError();
            return STENCIL_ERR_CUDA;
        }
        return STENCIL_OK;
    }
    if (p->variant == STENCIL_VARIANT_STREAM && p->nx % 2 != 0) return apply_row_padded_f64(p, in, out, steps, st);
    if (steps > 1 && !p->scratch64) {
        if (cudaMalloc(&p->scratch64, bytes) != cudaSuccess) {
            cudaGetLastError();
            p->scratch64 = nullptr;
            return STENCIL_ERR_ALLOC;
        }
    }
    if (p->variant == STENCIL_VARIANT_STREAM && p->boundary == STENCIL_PERIODIC) {
        const int depth = p->fused2d64_cfg ? p->fused2d64_cfg->T : 1;
        if (steps > 1 && depth > 1 && p->periodic_route != 1)
            return apply_periodic_fused(p, in, out, p->scratch64, steps, depth, st);
        if (p->periodic_route == 0 && stream_wrap_ok(p))
            return apply_periodic_inkernel(p, in, out, p->scratch64, steps, st);
        if (use_wrap_correction(p, steps)) return apply_periodic_corrected(p, in, out, p->scratch64, steps, st);
        if (steps > 1) return apply_periodic(p, in, out, steps, st);
    }
    // A pass advances the field by T time steps (T = 1 without temporal blocking), as in stencil_apply.
    const bool fuse = p->variant == STENCIL_VARIANT_STREAM && p->fused2d64_cfg != nullptr && steps > 1;
    const int T = fuse ? p->fused2d64_cfg->T : 1;
    const int passes = (steps + T - 1) / T;
    const double* src = in;
    int done = 0;
    for (int k = 0; k < passes; ++k) {
        const int remaining = passes - 1 - k;
        double* dst = (remaining % 2 == 0) ? out : p->scratch64;
        const int nlev = std::min(T, steps - done);
        p->chained = p->chain_launches && k > 0;
        rc = (fuse && nlev > 1) ? launch_rows2d_fused64(p, src, dst, nlev, st) : launch_sweep_f64(p, src, dst, st);
        p->chained = false;
        if (rc != STENCIL_OK) return rc;
        done += nlev;
        src = dst;
    }
    return STENCIL_OK;
}

int stencil_apply_host(stencil_plan_t p, const float* in_host, float* out_host, int steps, void* stream) {
    if (!valid_plan(p) || p->f64 || !in_host || !out_host || steps < 0) return STENCIL_ERR_INVALID;
    int rc = ensure_device_state(p);
    if (rc != STENCIL_OK) return rc;
    if ((rc = ensure_grid(&p->host_in, p->npoints)) != STENCIL_OK) return rc;
    if ((rc = ensure_grid(&p->host_out, p->npoints)) != STENCIL_OK) return rc;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const size_t bytes = (size_t)p->npoints * sizeof(float);

    // A single 3D sweep on the tiled kernel is cut into slabs of planes so that the upload
    // of slab s+1, the sweep of slab s and the download of slab s-1 overlap (the copies are
    // what costs time: the sweep itself is ~1 % of a PCIe round trip).
    constexpr int kMaxSlabs = 16;
    const int min_planes = std::max(2 * p->radius, 8);           // per slab
    const int kSlabs = p->nz >= kMaxSlabs * 2 * min_planes ? kMaxSlabs : kMaxSlabs / 2;
    const bool pipelined = steps == 1 && p->variant == STENCIL_VARIANT_STREAM && p->ndim == 3 &&
                           p->boundary == STENCIL_ZERO && p->nx % 4 == 0 &&
                           p->nz >= kSlabs * min_planes;
    if (!pipelined) {
        if (cudaMemcpyAsync(p->host_in, in_host, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) {
            cudaGetLastError();
            return STENCIL_ERR_CUDA;
        }
        rc = stencil_apply(p, p->host_in, p->host_out, steps, stream);
        if (rc != STENCIL_OK) return rc;
        if (cudaMemcpyAsync(out_host, p->host_out, bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess) {
            cudaGetLastError();
            return STENCIL_ERR_CUDA;
        }
        return STENCIL_OK;
    }

    auto fail = [&]() { cudaGetLastError(); return STENCIL_ERR_CUDA; };
    if (!p->copy_in && cudaStreamCreateWithFlags(&p->copy_in, cudaStreamNonBlocking) != cudaSuccess) return fail();
    if (!p->copy_out && cudaStreamCreateWithFlags(&p->copy_out, cudaStreamNonBlocking) != cudaSuccess) return fail();
    while ((int)p->events.size() < 2 * kMaxSlabs + 2) {
        cudaEvent_t e;
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return fail();
        p->events.push_back(e);
    }
    cudaEvent_t* up = p->events.data();              // up[s]: slab s is on the device
    cudaEvent_t* swept = p->events.data() + kMaxSlabs;  // swept[s]: slab s of the result is ready
    cudaEvent_t start = p->events[2 * kMaxSlabs], finished = p->events[2 * kMaxSlabs + 1];
    p->last_stream = st;
    p->used = true;

    const size_t plane = (size_t)p->ny * p->nx;
    auto slab_begin = [&](int s) { return (int)((int64_t)p->nz * s / kSlabs); };
    if (cudaEventRecord(start, st) != cudaSuccess) return fail();
    if (cudaStreamWaitEvent(p->copy_in, start, 0) != cudaSuccess) return fail();
    if (cudaStreamWaitEvent(p->copy_out, start, 0) != cudaSuccess) return fail();
    for (int s = 0; s < kSlabs; ++s) {
        const int z0 = slab_begin(s), z1 = slab_begin(s + 1);
        if (cudaMemcpyAsync(p->host_in + z0 * plane, in_host + z0 * plane, (z1 - z0) * plane * sizeof(float),
                            cudaMemcpyHostToDevice, p->copy_in) != cudaSuccess) return fail();
        if (cudaEventRecord(up[s], p->copy_in) != cudaSuccess) return fail();
    }
    for (int s = 0; s < kSlabs; ++s) {
        const int z0 = slab_begin(s), z1 = slab_begin(s + 1);
        // the sweep of slab s reads R planes of slab s+1 as well
        if (cudaStreamWaitEvent(st, up[std::min(s + 1, kSlabs - 1)], 0) != cudaSuccess) return fail();
        rc = launch_stream(p, p->host_in, p->host_out, st, z0, z1);
        if (rc != STENCIL_OK) return rc;
        if (cudaEventRecord(swept[s], st) != cudaSuccess) return fail();
        if (cudaStreamWaitEvent(p->copy_out, swept[s], 0) != cudaSuccess) return fail();
        if (cudaMemcpyAsync(out_host + z0 * plane, p->host_out + z0 * plane, (z1 - z0) * plane * sizeof(float),
                            cudaMemcpyDeviceToHost, p->copy_out) != cudaSuccess) return fail();
    }
    if (cudaEventRecord(finished, p->copy_out) != cudaSuccess) return fail();
    if (cudaStreamWaitEvent(st, finished, 0) != cudaSuccess) return fail();
    if (cudaStreamSynchronize(st) != cudaSuccess) return fail();
    return STENCIL_OK;
}

int stencil_apply_static(stencil_plan_t p, const float* in, float* out, int steps, void* stream) {
    if (!valid_plan(p) || p->f64 || !in || !out || steps < 0) return STENCIL_ERR_INVALID;
    const uintptr_t a = reinterpret_cast<uintptr_t>(in), b = reinterpret_cast<uintptr_t>(out);
    if ((a | b) & 15u) return STENCIL_ERR_INVALID;
    const uintptr_t bytes = (uintptr_t)p->npoints * sizeof(float);
    if (a < b + bytes && b < a + bytes) return STENCIL_ERR_INVALID;
    if (p->npoints > kStaticMaxPoints || (int64_t)p->taps.size() > kStaticMaxTaps) return STENCIL_ERR_TOO_LARGE;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

    unsigned char* base = nullptr;                 // first call on a device also looks the array up
    int rc = static_scratch_address(&base);
    if (rc != STENCIL_OK) return rc;
    float* grid = reinterpret_cast<float*>(base);
    Tap* taps = reinterpret_cast<Tap*>(base + kStaticGridBytes);

    if (steps == 0) {
        if (cudaMemcpyAsync(out, in, bytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess) {
            cudaGetLastError();
            return STENCIL_ERR_CUDA;
        }
        return STENCIL_OK;
    }
    const int ntaps = (int)p->taps.size();
    if (ntaps > 0 && cudaMemcpyAsync(taps, p->taps.data(), (size_t)ntaps * sizeof(Tap), cudaMemcpyHostToDevice,
                                     st) != cudaSuccess) {
        cudaGetLastError();
        return STENCIL_ERR_CUDA;
    }
    // Same ping-pong as stencil_apply, with the fixed array in place of the plan's
    // scratch grid.  Every cell of it is written before it is read, so nothing of
    // an earlier call's contents has to be cleared.
    Grid g{p->nz, p->ny, p->nx};
    const int nblocks = generic_grid_size(g, sm_count());
    const float* src = in;
    for (int k = 0; k < steps; ++k) {
        const int remaining = steps - 1 - k;
        float* dst = (remaining % 2 == 0) ? out : grid;
        if (p->boundary == STENCIL_PERIODIC)
            stencil_generic_kernel<true><<<nblocks, kGenericThreads, 0, st>>>(src, dst, g, taps, ntaps);
        else
            stencil_generic_kernel<false><<<nblocks, kGenericThreads, 0, st>>>(src, dst, g, taps, ntaps);
        if (cudaGetLastError() != cudaSuccess) return STENCIL_ERR_CUDA;
        p->launches++;
        src = dst;
    }
    return STENCIL_OK;
}

int stencil_destroy(stencil_plan_t p) {
    if (!p) return STENCIL_OK;
    if (!valid_plan(p)) return STENCIL_ERR_INVALID;
    int rc = STENCIL_OK;
    bool composite = false;
    for (int l = 0; l <= kMaxFuseLevels; ++l) composite = composite || p->d_ctaps[l];
    if (p->d_status || p->scratch || p->host_in || p->host_out || p->d_taps || p->d_taps64 || p->scratch64 ||
        p->pad || p->pad2 || composite) {
        int cur = -1;
        cudaGetDevice(&cur);
        if (p->device >= 0 && cur != p->device) cudaSetDevice(p->device);
        if (p->used) cudaStreamSynchronize(p->last_stream);
        void* ptrs[] = {p->d_status, p->scratch, p->host_in, p->host_out, p->d_taps, p->d_taps64, p->scratch64,
                        p->pad, p->pad2};
        for (void* q : ptrs)
            if (q && cudaFree(q) != cudaSuccess) rc = STENCIL_ERR_CUDA;
        for (int l = 0; l <= kMaxFuseLevels; ++l)
            if (p->d_ctaps[l] && cudaFree(p->d_ctaps[l]) != cudaSuccess) rc = STENCIL_ERR_CUDA;
        for (cudaEvent_t e : p->events) cudaEventDestroy(e);
        if (p->copy_in) cudaStreamDestroy(p->copy_in);
        if (p->copy_out) cudaStreamDestroy(p->copy_out);
        if (p->device >= 0 && cur >= 0 && cur != p->device) cudaSetDevice(cur);
        cudaGetLastError();
    }
    p->magic = 0;
    delete p;
    return rc;
}

const char* stencil_status_string(int status) {
    switch (status) {
        case STENCIL_OK: return "ok";
        case STENCIL_ERR_INVALID: return "invalid argument";
        case STENCIL_ERR_UNSUPPORTED: return "unsupported request";
        case STENCIL_ERR_CUDA: return "CUDA call failed or no device";
        case STENCIL_ERR_ALLOC: return "allocation failed";
        case STENCIL_ERR_TIMEOUT: return "bounded device wait expired";
        case STENCIL_ERR_TOO_LARGE: return "grid exceeds the fixed scratch of stencil_apply_static";
        default: return "unknown status";
    }
}

const char* stencil_variant_name(int variant) {
    switch (variant) {
        case STENCIL_VARIANT_AUTO: return "auto";
        case STENCIL_VARIANT_GENERIC: return "generic";
        case STENCIL_VARIANT_STREAM: return "stream";
        case STENCIL_VARIANT_FUSED: return "fused";
        default: return "unknown";
    }
}

int stencil_query_status(stencil_plan_t p) {
    if (!valid_plan(p)) return STENCIL_ERR_INVALID;
    if (!p->d_status) return STENCIL_OK;               // nothing has run yet
    if (cudaStreamSynchronize(p->last_stream) != cudaSuccess) { cudaGetLastError(); return STENCIL_ERR_CUDA; }
    int word = 0;
    if (cudaMemcpy(&word, p->d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemset(p->d_status, 0, sizeof(int)) != cudaSuccess) {
        cudaGetLastError();
        return STENCIL_ERR_CUDA;
    }
    return word == 0 ? STENCIL_OK : STENCIL_ERR_TIMEOUT;
}

int stencil_plan_set(stencil_plan_t p, int key, int64_t value) {
    if (!valid_plan(p)) return STENCIL_ERR_INVALID;
    switch (key) {
        case STENCIL_KEY_VARIANT: {
            if (p->f64) return resolve_variant_f64(p, (int)value);
            const int old_variant = p->variant;
            const StreamConfig* old_cfg = p->stream_cfg;
            const FusedConfig* old_fused = p->fused_cfg;
            int rc = resolve_variant(p, (int)value);
            if (rc != STENCIL_OK) { p->variant = old_variant; p->stream_cfg = old_cfg; p->fused_cfg = old_fused; }
            return rc;
        }
        case STENCIL_KEY_TILE_X:
        case STENCIL_KEY_FUSE_STEPS: {
            if (p->f64) {
                // FP64: only the 2D register cascade exists; 0 = use it, 1 = off, T = its depth
                if (key == STENCIL_KEY_TILE_X) return value == 0 ? STENCIL_OK : STENCIL_ERR_UNSUPPORTED;
                if (value < 0) return STENCIL_ERR_INVALID;
                const int old = p->fuse_steps;
                p->fuse_steps = (int)value;
                const Rows2DFused64Config* f2 =
                    (p->variant == STENCIL_VARIANT_STREAM && p->rows2d64_cfg) ? pick_fused2d64(p) : nullptr;
                if (!f2 && value > 1) { p->fuse_steps = old; return STENCIL_ERR_UNSUPPORTED; }
                p->fused2d64_cfg = f2;
                return STENCIL_OK;
            }
            // region width (128, 256 or 512) and time steps per pass of the fused kernel
            if (value < 0) return STENCIL_ERR_INVALID;
            const int old_fuse = p->fuse_steps, old_tx = p->tile_x;
            if (key == STENCIL_KEY_TILE_X) p->tile_x = (int)value; else p->fuse_steps = (int)value;
            if (p->variant == STENCIL_VARIANT_STREAM && p->ndim == 2) {
                // a 2D operator has one fused depth: 0 = use it, 1 = off, T = that depth
                const Rows2DFusedConfig* f2 = pick_fused2d(p);
                if ((!f2 && p->fuse_steps > 1) || (key == STENCIL_KEY_TILE_X && value != 0)) {
                    p->fuse_steps = old_fuse; p->tile_x = old_tx;
                    return STENCIL_ERR_UNSUPPORTED;
                }
                p->fused2d_cfg = f2;
            } else if (p->variant == STENCIL_VARIANT_STREAM) {
                const FusedConfig* f = pick_fused(p);
                const bool wants_fusion = p->fuse_steps > 1 || (key == STENCIL_KEY_TILE_X && value != 0 && p->fuse_steps != 1);
                if (!f && wants_fusion) { p->fuse_steps = old_fuse; p->tile_x = old_tx; return STENCIL_ERR_UNSUPPORTED; }
                p->fused_cfg = f;
            } else if (p->fuse_steps > 1) {
                p->fuse_steps = old_fuse; p->tile_x = old_tx;
                return STENCIL_ERR_UNSUPPORTED;
            }
            return STENCIL_OK;
        }
        case STENCIL_KEY_TILE_Y:
        case STENCIL_KEY_ROWS_PER_THREAD: {
            if (value < 0) return STENCIL_ERR_INVALID;
            if (p->f64) return value == 0 ? STENCIL_OK : STENCIL_ERR_UNSUPPORTED;
            int ty = key == STENCIL_KEY_TILE_Y ? (int)value : p->tile_y;
            int k = key == STENCIL_KEY_ROWS_PER_THREAD ? (int)value : p->rows_per_thread;
            if (p->variant == STENCIL_VARIANT_STREAM && p->ndim == 2) return value == 0 ? STENCIL_OK : STENCIL_ERR_UNSUPPORTED;
            if (p->variant == STENCIL_VARIANT_STREAM) {
                const StreamConfig* c = find_stream_cfg(p->radius, p->shape == STENCIL_BOX, ty, k);
                if (!c) return STENCIL_ERR_UNSUPPORTED;
                p->stream_cfg = c;
            }
            p->tile_y = ty;
            p->rows_per_thread = k;
            p->stream_cfg_fixed = ty != 0;
            p->stream_cfg_tuned = false;
            return STENCIL_OK;
        }
        case STENCIL_KEY_CHUNK_Z:
            if (value < 0) return STENCIL_ERR_INVALID;
            p->chunk_z = (int)std::min<int64_t>(value, 0x7fffffff);
            return STENCIL_OK;
        case STENCIL_KEY_STAGES:
            if (value < 0 || value > kMaxStages || value == 1) return STENCIL_ERR_INVALID;
            p->stages = (int)value;
            return STENCIL_OK;
        case STENCIL_KEY_STREAMING_STORE:
            p->streaming_store = value ? 1 : 0;
            return STENCIL_OK;
        case STENCIL_KEY_CHAIN_LAUNCHES:
            p->chain_launches = value != 0;
            return STENCIL_OK;
        case STENCIL_KEY_PERIODIC_ROUTE:
            if (value < 0 || value > 2) return STENCIL_ERR_INVALID;
            p->periodic_route = (int)value;
            return STENCIL_OK;
        case STENCIL_KEY_FUSED_TILE_Y: {
            if (value < 0) return STENCIL_ERR_INVALID;
            const int old = p->fused_tile_y;
            p->fused_tile_y = (int)value;
            if (p->variant == STENCIL_VARIANT_STREAM && !p->f64 && p->ndim == 3) {
                const FusedConfig* f = pick_fused(p);
                if (!f && value != 0) { p->fused_tile_y = old; return STENCIL_ERR_UNSUPPORTED; }
                p->fused_cfg = f;
            }
            return STENCIL_OK;
        }
        case STENCIL_KEY_WAIT_POLLS:
            if (value < 1 || value > (int64_t)kWaitPolls) return STENCIL_ERR_INVALID;
            p->wait_polls = (unsigned)value;
            return STENCIL_OK;
        case STENCIL_KEY_TEST_DROP_PLANE:
            if (value < -1 || value > 0x7fffffff) return STENCIL_ERR_INVALID;
            p->drop_plane = (int)value;
            return STENCIL_OK;
        default:
            return STENCIL_ERR_INVALID;
    }
}

int stencil_plan_get(stencil_plan_t p, int key, int64_t* value) {
    if (!valid_plan(p) || !value) return STENCIL_ERR_INVALID;
    switch (key) {
        case STENCIL_KEY_VARIANT: *value = p->variant; return STENCIL_OK;
        case STENCIL_KEY_TILE_X:
            *value = p->variant != STENCIL_VARIANT_STREAM ? 0 : (p->fused_cfg ? p->fused_cfg->txe : kStreamTX);
            if (p->ndim == 2 && p->variant == STENCIL_VARIANT_STREAM) *value = kStreamTX;
            return STENCIL_OK;
        case STENCIL_KEY_TILE_Y:
            *value = (p->variant == STENCIL_VARIANT_STREAM && p->stream_cfg) ? p->stream_cfg->tile_y : 0;
            return STENCIL_OK;
        case STENCIL_KEY_ROWS_PER_THREAD:
            *value = (p->variant == STENCIL_VARIANT_STREAM && p->stream_cfg) ? p->stream_cfg->K : 0;
            return STENCIL_OK;
        case STENCIL_KEY_FUSE_STEPS:
            *value = p->variant != STENCIL_VARIANT_STREAM ? 1
                     : p->fused_cfg                           ? p->fused_cfg->T
                     : p->fused2d_cfg                         ? p->fused2d_cfg->T
                     : p->fused2d64_cfg                       ? p->fused2d64_cfg->T
                                                              : 1;
            return STENCIL_OK;
        case STENCIL_KEY_LAUNCHES: *value = p->launches; return STENCIL_OK;
        case STENCIL_KEY_SCRATCH_BYTES: {
            const int64_t grids = (p->scratch != nullptr) + (p->host_in != nullptr) + (p->host_out != nullptr);
            const int64_t elem = p->f64 ? sizeof(double) : sizeof(float);
            // the padded grids: wrapped halos (periodic) or rows rounded up to 16 bytes (zero boundary)
            const int64_t padded_grid =
                p->boundary == STENCIL_PERIODIC
                    ? (int64_t)(p->nx + 2 * kPadX) * (p->ny + 2 * p->radius) *
                          (p->nz + (p->ndim == 3 ? 2 * p->radius : 0)) * elem
                    : (int64_t)p->nz * p->ny * (p->f64 ? (int64_t)(p->nx + 1) : (int64_t)((p->nx + 3) & ~3)) * elem;
            *value = grids * p->npoints * (int64_t)sizeof(float) +
                     (p->scratch64 ? p->npoints * (int64_t)sizeof(double) : 0) +
                     ((p->pad != nullptr) + (p->pad2 != nullptr)) * padded_grid;
            return STENCIL_OK;
        }
        case STENCIL_KEY_CHUNK_Z: *value = p->chunk_z; return STENCIL_OK;
        case STENCIL_KEY_STAGES: *value = p->stages; return STENCIL_OK;
        case STENCIL_KEY_STREAMING_STORE: *value = p->streaming_store; return STENCIL_OK;
        case STENCIL_KEY_CHAIN_LAUNCHES: *value = p->chain_launches ? 1 : 0; return STENCIL_OK;
        case STENCIL_KEY_PERIODIC_ROUTE: *value = p->periodic_route; return STENCIL_OK;
        case STENCIL_KEY_FUSED_TILE_Y:
            *value = (p->variant == STENCIL_VARIANT_STREAM && p->fused_cfg) ? p->fused_cfg->tye : 0;
            return STENCIL_OK;
        case STENCIL_KEY_WAIT_POLLS: *value = p->wait_polls; return STENCIL_OK;
        case STENCIL_KEY_TEST_DROP_PLANE: *value = p->drop_plane; return STENCIL_OK;
        default: return STENCIL_ERR_INVALID;
    }
}

}  // extern "C"
