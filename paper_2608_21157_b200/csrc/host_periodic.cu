// Host side of the periodic boundary on the tiled kernels (padded copy, wrap correction, the sweep
// that wraps inside the kernel, fused passes with a rewritten shell) and of grids whose rows are
// not 16-byte multiples.
#include "host.h"
#include "kernel_pad.cuh"

namespace stencil_host {

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
    const int grid = (int)std::min<int64_t>((cells + 255) / 256, (int64_t)plan_sms(p) * 32);
    stencil_pad_periodic_kernel<T><<<grid, 256, 0, st>>>(src, reinterpret_cast<T*>(p->pad), g, R, rz);
    if (cudaGetLastError() != cudaSuccess) return STENCIL_ERR_CUDA;
    p->launches++;
    *padded = reinterpret_cast<const T*>(p->pad);
    return STENCIL_OK;
}

template <typename T>
int repitch_rows(stencil_plan_s* p, const T* src, T* dst, int nx, int src_pitch, int dst_pitch,
                 cudaStream_t st) {
    const int64_t rows = (int64_t)p->nz * p->ny;
    int lanes_log2 = 0;
    while ((1 << lanes_log2) < nx && lanes_log2 < 8) ++lanes_log2;
    const int rows_per_cta = 256 >> lanes_log2;
    const int64_t ctas = (rows + 4 * rows_per_cta - 1) / (4 * rows_per_cta);      // a thread takes 4 rows per round
    const int grid = (int)std::min<int64_t>(ctas, (int64_t)plan_sms(p) * 16);
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
    const int shell_grid = (int)std::max<int64_t>(1, std::min<int64_t>((shell + 255) / 256, (int64_t)plan_sms(p) * 16));
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
    const int shell_grid = (int)std::max<int64_t>(1, std::min<int64_t>((shell + 255) / 256, (int64_t)plan_sms(p) * 16));
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
    if (p->f64) return p->stream64_cfg && p->stream64_cfg->launch_wrap && p->nx % fp64_stream_tile_x() == 0;
    return p->stream_cfg && p->stream_cfg->launch_wrap && p->nx % kStreamTX == 0;
}

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
                const bool small = p->npoints + 2 * (int64_t)p->nx < 0x7fffffffLL;    // room for an index before its wrap
                if ((small ? launch_kernel(&stencil_shell_rows_kernel<T, int>, (int)nrows, 256, 0, st, p->chain_launches,
                                           src, dst, g, H, 0, taps, ntaps, xchunks)
                           : launch_kernel(&stencil_shell_rows_kernel<T, int64_t>, (int)nrows, 256, 0, st,
                                           p->chain_launches, src, dst, g, H, 0, taps, ntaps, xchunks)) != cudaSuccess)
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
                if (p->npoints + 2 * (int64_t)p->nx < 0x7fffffffLL)
                    stencil_shell_rows_kernel<T, int><<<(int)nrows, 256, 0, st>>>(src, dst, g, H, hz, taps, ntaps, xchunks);
                else
                    stencil_shell_rows_kernel<T, int64_t><<<(int)nrows, 256, 0, st>>>(src, dst, g, H, hz, taps, ntaps, xchunks);
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
            const int shell_grid = (int)std::max<int64_t>(1, std::min<int64_t>((shell + 255) / 256, (int64_t)plan_sms(p) * 16));
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

// the instantiations the other units call
template int pad_periodic<float>(stencil_plan_s*, const float*, cudaStream_t, const float**, int*, int*, int*);
template int pad_periodic<double>(stencil_plan_s*, const double*, cudaStream_t, const double**, int*, int*, int*);
template int apply_periodic<float>(stencil_plan_s*, const float*, float*, int, cudaStream_t);
template int apply_periodic<double>(stencil_plan_s*, const double*, double*, int, cudaStream_t);
template int apply_periodic_corrected<float>(stencil_plan_s*, const float*, float*, float*, int, cudaStream_t);
template int apply_periodic_corrected<double>(stencil_plan_s*, const double*, double*, double*, int, cudaStream_t);
template int apply_periodic_inkernel<float>(stencil_plan_s*, const float*, float*, float*, int, cudaStream_t);
template int apply_periodic_inkernel<double>(stencil_plan_s*, const double*, double*, double*, int, cudaStream_t);
template int apply_periodic_fused<float>(stencil_plan_s*, const float*, float*, float*, int, int, cudaStream_t);
template int apply_periodic_fused<double>(stencil_plan_s*, const double*, double*, double*, int, int, cudaStream_t);

}  // namespace stencil_host
