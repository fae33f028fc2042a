// Plan construction, kernel selection and the extern "C" boundary declared in include/stencil.h.
// No CPU compute path exists here: every sweep runs in the CUDA kernels.
#include "host.h"
#include "ptx.cuh"

namespace stencil_host {

bool stream_supported(const stencil_plan_s* p) {
    if (p->nx % 4 != 0 && p->boundary != STENCIL_ZERO) return false;
    // radius > 4: the padded periodic copy has only 4 halo columns, so the wrap correction must fit
    if (p->radius > 4 && p->boundary == STENCIL_PERIODIC && !wrap_correction_fits(p)) return false;
    const bool box = p->shape == STENCIL_BOX;
    if (p->ndim == 2) return find_rows2d_cfg(p->radius, box) != nullptr;
    return find_stream_cfg(p->radius, box, 0, 0) != nullptr;
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

int launch_sweep(stencil_plan_s* p, const float* src, float* dst, cudaStream_t st) {
    switch (p->variant) {
        case STENCIL_VARIANT_STREAM:
            return p->ndim == 2 ? launch_rows2d(p, src, dst, st) : launch_stream(p, src, dst, st);
        default: return launch_generic(p, src, dst, st);
    }
}

// ---------------------------------------------------------------------------
// plan construction, shared by the fp32 and the FP64 entry point
// ---------------------------------------------------------------------------
uint64_t next_plan_serial() {
    static std::mutex m;
    static uint64_t n = 0;
    std::lock_guard<std::mutex> lock(m);
    return ++n;
}

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
    p->serial = next_plan_serial();
    p->f64 = kF64;
    p->ndim = ndim;
    p->nz = ndim == 3 ? (int)dims[0] : 1;
    p->ny = ndim == 3 ? (int)dims[1] : (int)dims[0];
    p->nx = ndim == 3 ? (int)dims[2] : (int)dims[1];
    p->npoints = n;
    p->radius = radius; p->shape = shape; p->boundary = boundary;
    p->device = -1; p->sms = 0;
    p->d_taps = nullptr; p->d_status = nullptr; p->scratch = nullptr; p->pad = nullptr; p->pad2 = nullptr; p->tmap_nx = 0; p->src_padded = false; p->fused_wrap = false; p->stream_wrap = false; p->debug_shrink = 0; p->periodic_route = 0;
    for (int l = 0; l <= kMaxFuseLevels; ++l) p->d_ctaps[l] = nullptr;
    p->d_taps64 = nullptr; p->scratch64 = nullptr; p->rows2d64_cfg = nullptr; p->stream64_cfg = nullptr; p->fused2d64_cfg = nullptr; p->fused64_cfg = nullptr;
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

}  // namespace stencil_host

using namespace stencil_host;

namespace {

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
// serial number of the plan whose taps were last uploaded into the array, per device (0: none)
uint64_t g_static_tap_owner[kStaticMaxDevices] = {0};

// `upload` comes back true when the array does not hold the taps of plan `serial` yet; the caller
// then uploads them (the array is marked as that plan's at once: calls do not overlap, by contract).
int static_scratch_address(unsigned char** out, uint64_t serial, bool* upload) {
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
    *upload = g_static_tap_owner[dev] != serial;
    g_static_tap_owner[dev] = serial;
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
    if (rc == STENCIL_OK) rc = check_device(p);
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
    int rc = ensure_device_state(p);
    if (rc == STENCIL_OK) rc = check_device(p);
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
    int rc = ensure_device_state(p);
    if (rc == STENCIL_OK) rc = check_device(p);
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
    if (rc == STENCIL_OK) rc = check_device(p);
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
    const bool fuse3d = p->variant == STENCIL_VARIANT_STREAM && p->fused64_cfg != nullptr && steps > 1;
    const bool fuse = fuse3d || (p->variant == STENCIL_VARIANT_STREAM && p->fused2d64_cfg != nullptr && steps > 1);
    const int T = fuse3d ? p->fused64_cfg->T : fuse ? p->fused2d64_cfg->T : 1;
    const int passes = (steps + T - 1) / T;
    const double* src = in;
    int done = 0;
    for (int k = 0; k < passes; ++k) {
        const int remaining = passes - 1 - k;
        double* dst = (remaining % 2 == 0) ? out : p->scratch64;
        const int nlev = std::min(T, steps - done);
        p->chained = p->chain_launches && k > 0;
        rc = !(fuse && nlev > 1) ? launch_sweep_f64(p, src, dst, st)
             : fuse3d           ? launch_fused(p, src, dst, nlev, st)
                                : launch_rows2d_fused64(p, src, dst, nlev, st);
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
    if (rc == STENCIL_OK) rc = check_device(p);
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

    if (steps == 0) {
        if (cudaMemcpyAsync(out, in, bytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess) {
            cudaGetLastError();
            return STENCIL_ERR_CUDA;
        }
        return STENCIL_OK;
    }
    unsigned char* base = nullptr;                 // first call on a device also looks the array up
    bool upload = true;
    int rc = static_scratch_address(&base, p->serial, &upload);
    if (rc != STENCIL_OK) return rc;
    float* grid = reinterpret_cast<float*>(base);
    Tap* taps = reinterpret_cast<Tap*>(base + kStaticGridBytes);
    const int ntaps = (int)p->taps.size();
    // The taps go up only when the array holds another plan's (or nothing yet): a plan that calls
    // again finds them in place and enqueues nothing but its kernels.
    if (upload && ntaps > 0 &&
        cudaMemcpyAsync(taps, p->taps.data(), (size_t)ntaps * sizeof(Tap), cudaMemcpyHostToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        return STENCIL_ERR_CUDA;
    }
    // Same ping-pong as stencil_apply, with the fixed array in place of the plan's
    // scratch grid.  Every cell of it is written before it is read, so nothing of
    // an earlier call's contents has to be cleared.
    const float* src = in;
    for (int k = 0; k < steps; ++k) {
        const int remaining = steps - 1 - k;
        float* dst = (remaining % 2 == 0) ? out : grid;
        rc = launch_generic_taps(p, src, dst, taps, ntaps, st);
        if (rc != STENCIL_OK) return rc;
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
        case STENCIL_ERR_BOUNDS: return "a store outside the output grid was skipped (debug build)";
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
    return word == 0 ? STENCIL_OK : word == stencil::kStatusBounds ? STENCIL_ERR_BOUNDS : STENCIL_ERR_TIMEOUT;
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
                if (value < 0) return STENCIL_ERR_INVALID;
                if (p->ndim == 3) {
                    // FP64 3D stars of radius 1: region width 128 or 256, two or three steps per pass
                    const int old_fuse = p->fuse_steps, old_tx = p->tile_x;
                    if (key == STENCIL_KEY_TILE_X) p->tile_x = (int)value; else p->fuse_steps = (int)value;
                    const FusedConfig* f3 =
                        (p->variant == STENCIL_VARIANT_STREAM && p->stream64_cfg) ? pick_fused64(p) : nullptr;
                    const bool wants = p->fuse_steps > 1 || (key == STENCIL_KEY_TILE_X && value != 0 && p->fuse_steps != 1);
                    if (!f3 && wants) { p->fuse_steps = old_fuse; p->tile_x = old_tx; return STENCIL_ERR_UNSUPPORTED; }
                    p->fused64_cfg = f3;
                    return STENCIL_OK;
                }
                // FP64 2D: only the register cascade exists; 0 = use it, 1 = off, T = its depth
                if (key == STENCIL_KEY_TILE_X) return value == 0 ? STENCIL_OK : STENCIL_ERR_UNSUPPORTED;
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
            } else if (p->variant == STENCIL_VARIANT_STREAM && p->f64 && p->ndim == 3 && p->stream64_cfg) {
                const FusedConfig* f = pick_fused64(p);
                if (!f && value != 0) { p->fused_tile_y = old; return STENCIL_ERR_UNSUPPORTED; }
                p->fused64_cfg = f;
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
        case STENCIL_KEY_DEBUG_SHRINK:
#ifdef STENCIL_DEBUG
            if (value < 0 || value > p->npoints) return STENCIL_ERR_INVALID;
            p->debug_shrink = value;
            return STENCIL_OK;
#else
            return STENCIL_ERR_UNSUPPORTED;
#endif
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
                     : p->fused64_cfg                         ? p->fused64_cfg->T
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
            *value = p->variant != STENCIL_VARIANT_STREAM ? 0
                     : p->f64 ? (p->fused64_cfg ? p->fused64_cfg->tye : 0) : (p->fused_cfg ? p->fused_cfg->tye : 0);
            return STENCIL_OK;
        case STENCIL_KEY_DEVICE: *value = p->device; return STENCIL_OK;
        case STENCIL_KEY_WAIT_POLLS: *value = p->wait_polls; return STENCIL_OK;
        case STENCIL_KEY_TEST_DROP_PLANE: *value = p->drop_plane; return STENCIL_OK;
        case STENCIL_KEY_DEBUG_SHRINK:
#ifdef STENCIL_DEBUG
            *value = p->debug_shrink;
            return STENCIL_OK;
#else
            return STENCIL_ERR_UNSUPPORTED;
#endif
        default: return STENCIL_ERR_INVALID;
    }
}

}  // extern "C"
