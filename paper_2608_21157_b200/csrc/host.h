// Internal header of the host side: the plan object, the configuration tables of the kernel
// families, and the functions the translation units call across each other.
//
//   host_common.cu    device state, tensor maps, the one-thread-per-point kernel
//   host_stream.cu    3D single sweeps (fp32)
//   host_fused.cu     3D temporal blocking (fp32)
//   host_rows2d.cu    2D sweeps and 2D temporal blocking (fp32)
//   host_f64.cu       the FP64 kernels
//   host_periodic.cu  periodic routes, grids with padded rows
//   abi.cu            plan construction and the extern "C" boundary (include/stencil.h)
//
// Each unit includes only the kernel headers it instantiates, so a change to one kernel
// recompiles one unit.  Nothing here is exported: the library is built with hidden visibility
// and only the entry points of include/stencil.h are marked visible.
#pragma once
#include "../../include/stencil.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <functional>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "common.cuh"
#include "geom.cuh"

namespace stencil_host {
using namespace stencil;

constexpr uint32_t kPlanMagic = 0x5354434cu;   // "STCL"
constexpr int kMaxRadius = 8;
constexpr int kMaxFuseLevels = 4;              // deepest temporal blocking of any fused kernel
constexpr size_t kMaxSmemBytes = 227 * 1024;   // dynamic shared memory a CTA can be granted

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
extern std::mutex g_config_mutex;

// Per-device facts of one kernel, cached in its configuration (guarded by g_config_mutex).
struct KernelLimits {
    size_t smem_allowed = 0;     // dynamic shared memory the kernel has been granted (it only ever grows)
    size_t occ_smem = 0;         // the shared-memory size `occ` was measured at
    int occ = 0;                 // resident CTAs per SM at that size
    int device = -1;             // the device these facts belong to
};
// Makes sure `kernel` may use `smem` bytes of dynamic shared memory on device `dev` (the current one) and
// returns its resident CTAs per SM at that size (>= 1; 1 without a query when `want_occ` is false), or -1
// when a CUDA call fails.
int kernel_limits(const void* kernel, int threads, size_t smem, int dev, KernelLimits& lim, bool want_occ);

}  // namespace stencil_host

struct stencil_plan_s;

namespace stencil_host {

// ---------------------------------------------------------------------------
// STREAM kernel configurations (3D single sweep)
// ---------------------------------------------------------------------------
struct StreamConfig {
    int radius;
    bool box;
    int K, NW;            // rows per thread, consumer warps
    int tile_y;           // K * NW
    int plane_bytes, box_rows, threads;
    int px;               // columns of the TMA box: the tile plus its halo on both sides
    mutable KernelLimits lim, lim_wrap;      // of `kernel` and `kernel_wrap`
    const void* kernel;
    cudaError_t (*launch)(const stencil_plan_s*, const StreamConfig&, const CUtensorMap&,
                          float*, const StreamGeom&, int grid, size_t smem, cudaStream_t);
    // the sweep of a periodic grid inside the kernel (stars of radius <= 4 and the boxes; null otherwise)
    const void* kernel_wrap;
    int stage_bytes;                         // per ring slot, beside the plane
    cudaError_t (*launch_wrap)(const stencil_plan_s*, const CUtensorMap&, const CUtensorMap&,
                               const CUtensorMap&, const CUtensorMap&, float*, const StreamGeom&, int grid,
                               size_t smem, cudaStream_t);
};

// ---------------------------------------------------------------------------
// FUSED kernel configurations (temporal blocking, 3D)
// ---------------------------------------------------------------------------
struct FusedConfig {
    int radius, T, K, XW, NWY;
    bool box;
    bool f64;                                // FP64 instantiation (two doubles per lane: 64 columns per warp)
    int txe, tye, threads, slot_bytes;
    int pw;                                  // width of the TMA boxes a plane is loaded as
    const void* kernel;
    const void* kernel_spec;                 // the instantiation for full passes over rows of exactly txe points
    const void* kernel_wrap;                 // ... and the one of those that wraps x and z (passes of a periodic grid)
    mutable KernelLimits lim, lim_spec, lim_wrap;   // of the three kernels
    // `out` is a float* or double* as the configuration's element type says
    cudaError_t (*launch)(const stencil_plan_s*, const CUtensorMap&, void* out, const FusedGeom&,
                          int grid, size_t smem, cudaStream_t);
    cudaError_t (*launch_spec)(const stencil_plan_s*, const CUtensorMap&, void* out, const FusedGeom&,
                               int grid, size_t smem, cudaStream_t);
    cudaError_t (*launch_wrap)(const stencil_plan_s*, const CUtensorMap&, void* out, const FusedGeom&,
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
    mutable KernelLimits lim;
    cudaError_t (*launch)(const stencil_plan_s*, const CUtensorMap&, float*, const Rows2DGeom&,
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
    mutable KernelLimits lim;
    cudaError_t (*launch)(const stencil_plan_s*, const CUtensorMap&, float*, const Rows2DFusedGeom&,
                          int grid, size_t smem, cudaStream_t);
};

// ---------------------------------------------------------------------------
// the FP64 twins
// ---------------------------------------------------------------------------
struct Rows2DFused64Config {
    int radius;
    bool box;
    int T, YB, NW, batch_bytes;
    const void* kernel;
    mutable KernelLimits lim;
    cudaError_t (*launch)(const stencil_plan_s*, const CUtensorMap&, double*, const Rows2DFusedGeom&,
                          int grid, size_t smem, cudaStream_t);
};

struct Rows2D64Config {
    int radius;
    bool box;
    int YB, NW, batch_bytes, px;
    const void* kernel;
    mutable KernelLimits lim;
    cudaError_t (*launch)(const stencil_plan_s*, const CUtensorMap&, double*, const Rows2DGeom&,
                          int grid, size_t smem, cudaStream_t);
};

struct Stream64Config {
    int radius;
    bool box;
    int tile_y, plane_bytes, box_rows, threads, px;
    const void* kernel;
    mutable KernelLimits lim, lim_wrap;      // of `kernel` and `kernel_wrap`
    cudaError_t (*launch)(const stencil_plan_s*, const CUtensorMap&, double*, const StreamGeom&,
                          int grid, size_t smem, cudaStream_t);
    // the sweep of a periodic grid inside the kernel (stars of radius <= 4; null otherwise)
    const void* kernel_wrap;
    int stage_bytes;                         // per ring slot, beside the plane
    cudaError_t (*launch_wrap)(const stencil_plan_s*, const CUtensorMap&, const CUtensorMap&,
                               const CUtensorMap&, const CUtensorMap&, double*, const StreamGeom&, int grid,
                               size_t smem, cudaStream_t);
};

}  // namespace stencil_host

struct stencil_plan_s {
    uint32_t magic;
    uint64_t serial;               // unique per plan of this process, never reused
    int ndim;
    int nz, ny, nx;
    int64_t npoints;
    int radius, shape, boundary;
    bool f64;                      // FP64 plan (stencil_plan_f64): only the *_f64 calls accept it
    std::vector<float> w;          // dense (2R+1)^ndim, as given
    std::vector<stencil::Tap> taps;         // non-zero taps, dense C order
    std::vector<double> w64;       // the same for FP64 plans
    std::vector<stencil::TapT<double>> taps64;
    stencil::TapT<double>* d_taps64;
    // taps of the operator's L-fold self-convolution, L = 1..kMaxFuseLevels (periodic boundary under
    // temporal blocking); built and uploaded at first need
    std::vector<stencil::TapT<double>> ctaps[stencil_host::kMaxFuseLevels + 1];
    stencil::TapT<double>* d_ctaps[stencil_host::kMaxFuseLevels + 1];
    double* scratch64;             // N doubles, iteration ping-pong of FP64 plans
    const stencil_host::Rows2D64Config* rows2d64_cfg;
    const stencil_host::Rows2DFused64Config* fused2d64_cfg;   // non-null: iterated applies of a 2D FP64 grid run fused passes
    const stencil_host::Stream64Config* stream64_cfg;
    const stencil_host::FusedConfig* fused64_cfg;      // non-null: iterated applies of a 3D FP64 grid run fused passes
    // device state (created lazily, on the device current at first apply)
    int device;
    int sms;                       // multiprocessors of that device
    stencil::Tap* d_taps;
    int* d_status;
    float* scratch;                // N floats, iteration ping-pong
    float* pad;                    // padded copy of the input (periodic boundary on the tiled kernels;
                                   // first of the two padded-row grids when nx is not a multiple of 4)
    float* pad2;                   // second padded-row grid
    int tmap_nx;                   // non-zero while a padded-row sweep runs: the true row length
    int periodic_route;            // knob: 0 = by measured cost, 1 = padded copy, 2 = wrap correction where it fits
    // the z cut of the fused passes, found once per configuration and view of the grid
    struct FusedSchedule { const void* cfg = nullptr; int nz = 0, tiles = 0, slots = 0, chunk = 0, rest = 0, rest_chunk = 1; };
    FusedSchedule fused_schedule;
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
    unsigned wait_polls;           // cap of the bounded device waits
    int drop_plane;                // test hook, -1 = off
    int64_t debug_shrink;          // debug builds, test hook: the store checks take the output grid to be this many
                                   // points shorter than it is
    const stencil_host::StreamConfig* stream_cfg;
    bool stream_cfg_fixed;         // the caller chose the tile shape
    bool stream_cfg_tuned;         // the library has chosen it for this grid
    const stencil_host::FusedConfig* fused_cfg;  // non-null: iterated applies run fused passes
    const stencil_host::Rows2DConfig* rows2d_cfg; // non-null: 2D grid on the row-streaming kernel
    const stencil_host::Rows2DFusedConfig* fused2d_cfg;  // non-null: iterated applies of a 2D grid run fused passes
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

namespace stencil_host {

// Debug builds: the extent that a launch's stores are checked against (the grid as the plan sees it now).
#ifdef STENCIL_DEBUG
#define STENCIL_SET_OUT_POINTS(g, p) \
    ((g).out_points = (long long)(p)->nz * (p)->ny * (p)->nx - (long long)(p)->debug_shrink)
#else
#define STENCIL_SET_OUT_POINTS(g, p) ((void)0)
#endif

inline bool valid_plan(const stencil_plan_s* p) { return p && p->magic == kPlanMagic; }

// entry [dz+R][dy+R][dx+R] of the plan's dense weights in the plan's own precision
template <typename E>
inline E dense_tap(const stencil_plan_s* p, int dz, int dy, int dx) {
    const int R = p->radius, side = 2 * R + 1;
    const size_t f = p->ndim == 3 ? ((size_t)(dz + R) * side + (dy + R)) * side + (dx + R)
                                  : (size_t)(dy + R) * side + (dx + R);
    if constexpr (sizeof(E) == 8) return p->w64[f];
    else return p->w[f];
}

// The taps of a 3D star (members c, x[], y[], z[], index d + R) or box (member w[][][]) as the kernels take them.
template <typename E, int R, typename SW>
inline void pack_star3d(const stencil_plan_s* p, SW& sw) {
    std::memset(&sw, 0, sizeof(sw));
    sw.c = dense_tap<E>(p, 0, 0, 0);
    for (int d = -R; d <= R; ++d) {
        if (d == 0) continue;
        sw.x[d + R] = dense_tap<E>(p, 0, 0, d);
        sw.y[d + R] = dense_tap<E>(p, 0, d, 0);
        sw.z[d + R] = dense_tap<E>(p, d, 0, 0);
    }
}
template <typename E, int R, typename BW>
inline void pack_box3d(const stencil_plan_s* p, BW& bw) {
    std::memset(&bw, 0, sizeof(bw));
    for (int a = -R; a <= R; ++a)
        for (int b = -R; b <= R; ++b)
            for (int c = -R; c <= R; ++c) bw.w[a + R][b + R][c + R] = dense_tap<E>(p, a, b, c);
}
// star or box, whichever the kernel instantiation reads (the other stays zero)
template <typename E, int R, bool BOX, typename SW, typename BW>
inline void pack_taps3d(const stencil_plan_s* p, SW& sw, BW& bw) {
    std::memset(&sw, 0, sizeof(sw));
    std::memset(&bw, 0, sizeof(bw));
    if constexpr (BOX) pack_box3d<E, R>(p, bw);
    else pack_star3d<E, R>(p, sw);
}
// the dense (2R+1)^2 weights of a 2D operator (member w[][])
template <typename E, int R, typename W2>
inline void pack_taps2d(const stencil_plan_s* p, W2& wt) {
    for (int a = -R; a <= R; ++a)
        for (int b = -R; b <= R; ++b) wt.w[a + R][b + R] = dense_tap<E>(p, 0, a, b);
}

// A periodic grid takes fused passes of L steps as zero-boundary passes whose shell of depth
// H = L * R is then rewritten (stencil_shell_compose_kernel): every extent must hold both shells.
inline bool shell_fits(const stencil_plan_s* p, int H) {
    return p->nx >= 2 * H && p->ny >= 2 * H && (p->ndim == 2 || p->nz >= 2 * H);
}

// The wrap-correction route needs the three parts of the boundary shell to be disjoint.
inline bool wrap_correction_fits(const stencil_plan_s* p) {
    const int R = p->radius;
    return p->nx >= 2 * R && p->ny >= 2 * R && (p->ndim == 2 || p->nz >= 2 * R);
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

// ---- host_common.cu ---------------------------------------------------------
int sm_count();                    // multiprocessors of the current device
inline int plan_sms(const stencil_plan_s* p) { return p->sms > 0 ? p->sms : sm_count(); }
int ensure_device_state(stencil_plan_s* p);
int check_device(const stencil_plan_s* p);
int ensure_grid(float** slot, int64_t npoints);
int get_tensor_map(stencil_plan_s* p, const void* cfg, int box_x, int box_y, const float* src,
                   const CUtensorMap** out, int tnx = 0, int tny = 0, int tnz = 0);
int get_tensor_map_f64(stencil_plan_s* p, const void* cfg, int box_x, int box_y, const double* src,
                       const CUtensorMap** out, int tnx = 0, int tny = 0, int tnz = 0);
int launch_generic(stencil_plan_s* p, const float* src, float* dst, cudaStream_t st);
int launch_generic_f64(stencil_plan_s* p, const double* src, double* dst, cudaStream_t st);
// the one-thread-per-point kernel on caller-given taps (stencil_apply_static)
int launch_generic_taps(stencil_plan_s* p, const float* src, float* dst, const Tap* d_taps, int ntaps,
                        cudaStream_t st);

// ---- host_stream.cu ---------------------------------------------------------
const StreamConfig* find_stream_cfg(int radius, bool box, int tile_y, int rows_per_thread);
int short_chunk_star1(int nz, int64_t tiles, int64_t slots);
// dst[z_begin, z_end) = one sweep of src; the whole grid when z_end <= z_begin
int launch_stream(stencil_plan_s* p, const float* src, float* dst, cudaStream_t st, int z_begin = 0, int z_end = 0);

// ---- host_fused.cu ----------------------------------------------------------
const FusedConfig* pick_fused(const stencil_plan_s* p);
const FusedConfig* pick_fused64(const stencil_plan_s* p);
// one fused pass: dst = S^nlev(src), nlev <= the configuration's T (grids of the plan's element type)
int launch_fused(stencil_plan_s* p, const void* src, void* dst, int nlev, cudaStream_t st);

// ---- host_rows2d.cu ---------------------------------------------------------
const Rows2DConfig* find_rows2d_cfg(int radius, bool box);
const Rows2DFusedConfig* pick_fused2d(const stencil_plan_s* p);
int short_chunk_2d(const stencil_plan_s* p, int YB);
int launch_rows2d(stencil_plan_s* p, const float* src, float* dst, cudaStream_t st, int y_begin = 0, int y_end = 0);
int launch_rows2d_fused(stencil_plan_s* p, const float* src, float* dst, int nlev, cudaStream_t st);

// ---- host_f64.cu ------------------------------------------------------------
int resolve_variant_f64(stencil_plan_s* p, int want);
const Rows2DFused64Config* pick_fused2d64(const stencil_plan_s* p);
int launch_rows2d_fused64(stencil_plan_s* p, const double* src, double* dst, int nlev, cudaStream_t st);
// dst = one sweep of src; with begin < end only the output planes (3D) or rows (2D) [begin, end)
int launch_sweep_f64(stencil_plan_s* p, const double* src, double* dst, cudaStream_t st, int begin = 0, int end = 0);
int fp64_stream_tile_x();      // tile width of the 3D FP64 kernel

// ---- host_periodic.cu -------------------------------------------------------
// Periodic boundary: copy `src` into the plan's padded grid (wrapped halos) on `st`.
template <typename T>
int pad_periodic(stencil_plan_s* p, const T* src, cudaStream_t st, const T** padded, int* pnx, int* pny, int* pnz);
bool use_wrap_correction(const stencil_plan_s* p, int steps);
bool stream_wrap_ok(const stencil_plan_s* p);
template <typename T> int apply_periodic(stencil_plan_s* p, const T* in, T* out, int steps, cudaStream_t st);
template <typename T>
int apply_periodic_corrected(stencil_plan_s* p, const T* in, T* out, T* other, int steps, cudaStream_t st);
template <typename T>
int apply_periodic_inkernel(stencil_plan_s* p, const T* in, T* out, T* other, int steps, cudaStream_t st);
template <typename T>
int apply_periodic_fused(stencil_plan_s* p, const T* in, T* out, T* other, int steps, int depth, cudaStream_t st);
int apply_row_padded(stencil_plan_s* p, const float* in, float* out, int steps, cudaStream_t st);
int apply_row_padded_f64(stencil_plan_s* p, const double* in, double* out, int steps, cudaStream_t st);

// ---- abi.cu -----------------------------------------------------------------
bool stream_supported(const stencil_plan_s* p);
int launch_sweep(stencil_plan_s* p, const float* src, float* dst, cudaStream_t st);

}  // namespace stencil_host
