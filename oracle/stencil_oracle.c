/*
 * CPU oracle for the fixed-coefficient stencil sweep.  TEST INFRASTRUCTURE ONLY:
 * it is the slow, plain definition that the CUDA path is checked against and
 * the CPU baseline that the benchmark times.  It shares no code, header, table
 * or helper with the CUDA library, and the library never calls it.
 *
 * What it computes (paper, "Case-study protocol": a box stencil of radius R is
 * the single-channel (2R+1)^d zero-padded cross-correlation with padding R and
 * stride 1, repeated for a number of time steps):
 *
 *     out[p] = sum_o  w[o] * in[p + o]          for every grid point p,
 *
 * o ranging over the dense (2R+1)^d offset cube, no kernel flip, taps that
 * fall outside the grid contributing zero (ZERO boundary) or wrapping around
 * (PERIODIC boundary).  Iteration feeds each result back as the next input;
 * every intermediate field is a float32 array.
 *
 * Precision: the sum is accumulated in double over the float32 weights and
 * float32 inputs, in dense C order of the offsets, and rounded to float32
 * once per point per step.  Weights that are exactly zero are skipped (a star
 * stencil is a dense cube with zeros off the axes).  The paper's own case
 * study runs in FP64; the *_f64 entry points take double weights and fields,
 * accumulate in long double and round to double once per point per step.
 *
 * Every part of this file is pinned by the CPU test-suite against closed
 * forms, invariants, brute force and library routines; nothing here is
 * "parity unpinned".
 *
 * Layout: dims[] slowest axis first, x contiguous; weights[] dense C order in
 * the same axis order, entry [dz+R][dy+R][dx+R].
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_ZERO = 0, ORACLE_PERIODIC = 1 };

typedef struct {
    int dz, dy, dx;
    double w;
} tap_t;

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* non-negative remainder */
static inline int64_t wrap(int64_t q, int64_t n)
{
    q %= n;
    return q < 0 ? q + n : q;
}

/* Collect the non-zero taps in dense C order.  2D grids are treated as 3D
 * with nz = 1 and dz = 0 only. */
static int build_taps(int ndim, int R, const float *weights, tap_t **taps_out)
{
    int side = 2 * R + 1;
    int total = (ndim == 3) ? side * side * side : side * side;
    tap_t *taps = (tap_t *)malloc(sizeof(tap_t) * (size_t)total);
    int n = 0;
    if (!taps) return -1;
    if (ndim == 3) {
        for (int a = 0; a < side; ++a)
            for (int b = 0; b < side; ++b)
                for (int c = 0; c < side; ++c) {
                    float w = weights[((size_t)a * side + b) * side + c];
                    if (w != 0.0f) {
                        taps[n].dz = a - R; taps[n].dy = b - R; taps[n].dx = c - R;
                        taps[n].w = (double)w;
                        ++n;
                    }
                }
    } else {
        for (int b = 0; b < side; ++b)
            for (int c = 0; c < side; ++c) {
                float w = weights[(size_t)b * side + c];
                if (w != 0.0f) {
                    taps[n].dz = 0; taps[n].dy = b - R; taps[n].dx = c - R;
                    taps[n].w = (double)w;
                    ++n;
                }
            }
    }
    *taps_out = taps;
    return n;
}

/* One point of one sweep, straight from the definition. */
static inline float point_value(const float *a, int64_t nz, int64_t ny, int64_t nx,
                                int64_t z, int64_t y, int64_t x,
                                const tap_t *taps, int ntaps, int boundary)
{
    double acc = 0.0;
    for (int t = 0; t < ntaps; ++t) {
        int64_t qz = z + taps[t].dz, qy = y + taps[t].dy, qx = x + taps[t].dx;
        if (boundary == ORACLE_PERIODIC) {
            qz = wrap(qz, nz); qy = wrap(qy, ny); qx = wrap(qx, nx);
        } else if (qz < 0 || qz >= nz || qy < 0 || qy >= ny || qx < 0 || qx >= nx) {
            continue;
        }
        acc += taps[t].w * (double)a[(qz * ny + qy) * nx + qx];
    }
    return (float)acc;
}

/*
 * steps-fold application.  in/out: N floats each, must not overlap.
 * steps == 0 copies.  Returns 0, or -1 on bad arguments / allocation failure.
 */
int oracle_stencil_apply(int ndim, const int64_t *dims, int radius, const float *weights,
                         int boundary, int steps, const float *in, float *out)
{
    if ((ndim != 2 && ndim != 3) || !dims || radius < 1 || !weights || !in || !out || steps < 0)
        return -1;
    if (boundary != ORACLE_ZERO && boundary != ORACLE_PERIODIC) return -1;
    int64_t nz = (ndim == 3) ? dims[0] : 1;
    int64_t ny = (ndim == 3) ? dims[1] : dims[0];
    int64_t nx = (ndim == 3) ? dims[2] : dims[1];
    if (nz < 1 || ny < 1 || nx < 1) return -1;
    size_t N = (size_t)nz * (size_t)ny * (size_t)nx;

    if (steps == 0) {
        memcpy(out, in, N * sizeof(float));
        return 0;
    }

    tap_t *taps = NULL;
    int ntaps = build_taps(ndim, radius, weights, &taps);
    if (ntaps < 0) return -1;

    /* ping-pong: cur holds u^k, nxt receives u^{k+1}; the last step lands in out */
    float *tmp = NULL;
    if (steps > 1) {
        tmp = (float *)malloc(N * sizeof(float));
        if (!tmp) { free(taps); return -1; }
    }
    const float *cur = in;
    for (int k = 0; k < steps; ++k) {
        int remaining = steps - 1 - k;               /* sweeps after this one */
        float *nxt = (remaining % 2 == 0) ? out : tmp;
        /* parallel over the outermost populated axis only; no tiling */
        if (nz > 1) {
#pragma omp parallel for schedule(static)
            for (int64_t z = 0; z < nz; ++z)
                for (int64_t y = 0; y < ny; ++y)
                    for (int64_t x = 0; x < nx; ++x)
                        nxt[(z * ny + y) * nx + x] =
                            point_value(cur, nz, ny, nx, z, y, x, taps, ntaps, boundary);
        } else {
#pragma omp parallel for schedule(static)
            for (int64_t y = 0; y < ny; ++y)
                for (int64_t x = 0; x < nx; ++x)
                    nxt[y * nx + x] = point_value(cur, 1, ny, nx, 0, y, x, taps, ntaps, boundary);
        }
        cur = nxt;
    }
    free(tmp);
    free(taps);
    return 0;
}

/*
 * One sweep evaluated only at the listed points (flat C-order indices); for
 * spot checks on grids where a full sweep is not wanted.
 */
int oracle_stencil_points(int ndim, const int64_t *dims, int radius, const float *weights,
                          int boundary, const float *in, int64_t npts, const int64_t *flat_index,
                          float *out_values)
{
    if ((ndim != 2 && ndim != 3) || !dims || radius < 1 || !weights || !in || npts < 0)
        return -1;
    int64_t nz = (ndim == 3) ? dims[0] : 1;
    int64_t ny = (ndim == 3) ? dims[1] : dims[0];
    int64_t nx = (ndim == 3) ? dims[2] : dims[1];
    tap_t *taps = NULL;
    int ntaps = build_taps(ndim, radius, weights, &taps);
    if (ntaps < 0) return -1;
    for (int64_t i = 0; i < npts; ++i) {
        int64_t f = flat_index[i];
        if (f < 0 || f >= nz * ny * nx) { free(taps); return -1; }
        int64_t x = f % nx, y = (f / nx) % ny, z = f / (nx * ny);
        out_values[i] = point_value(in, nz, ny, nx, z, y, x, taps, ntaps, boundary);
    }
    free(taps);
    return 0;
}

/* ------------------------------------------------------------------------ */
/* FP64 fields (the precision of the paper's case study): same definition,    */
/* long double accumulation, one rounding to double per point per step.       */
/* ------------------------------------------------------------------------ */
typedef struct {
    int dz, dy, dx;
    long double w;
} tapl_t;

static int build_taps_f64(int ndim, int R, const double *weights, tapl_t **taps_out)
{
    int side = 2 * R + 1;
    int total = (ndim == 3) ? side * side * side : side * side;
    tapl_t *taps = (tapl_t *)malloc(sizeof(tapl_t) * (size_t)total);
    int n = 0;
    if (!taps) return -1;
    for (int f = 0; f < total; ++f) {
        double w = weights[f];
        if (w == 0.0) continue;
        int c = f % side, b = (f / side) % side, a = (ndim == 3) ? f / (side * side) : R;
        taps[n].dz = a - R; taps[n].dy = b - R; taps[n].dx = c - R;
        taps[n].w = (long double)w;
        ++n;
    }
    *taps_out = taps;
    return n;
}

static inline double point_value_f64(const double *a, int64_t nz, int64_t ny, int64_t nx,
                                     int64_t z, int64_t y, int64_t x,
                                     const tapl_t *taps, int ntaps, int boundary)
{
    long double acc = 0.0L;
    for (int t = 0; t < ntaps; ++t) {
        int64_t qz = z + taps[t].dz, qy = y + taps[t].dy, qx = x + taps[t].dx;
        if (boundary == ORACLE_PERIODIC) {
            qz = wrap(qz, nz); qy = wrap(qy, ny); qx = wrap(qx, nx);
        } else if (qz < 0 || qz >= nz || qy < 0 || qy >= ny || qx < 0 || qx >= nx) {
            continue;
        }
        acc += taps[t].w * (long double)a[(qz * ny + qy) * nx + qx];
    }
    return (double)acc;
}

int oracle_stencil_apply_f64(int ndim, const int64_t *dims, int radius, const double *weights,
                             int boundary, int steps, const double *in, double *out)
{
    if ((ndim != 2 && ndim != 3) || !dims || radius < 1 || !weights || !in || !out || steps < 0)
        return -1;
    if (boundary != ORACLE_ZERO && boundary != ORACLE_PERIODIC) return -1;
    int64_t nz = (ndim == 3) ? dims[0] : 1;
    int64_t ny = (ndim == 3) ? dims[1] : dims[0];
    int64_t nx = (ndim == 3) ? dims[2] : dims[1];
    if (nz < 1 || ny < 1 || nx < 1) return -1;
    size_t N = (size_t)nz * (size_t)ny * (size_t)nx;
    if (steps == 0) {
        memcpy(out, in, N * sizeof(double));
        return 0;
    }
    tapl_t *taps = NULL;
    int ntaps = build_taps_f64(ndim, radius, weights, &taps);
    if (ntaps < 0) return -1;
    double *tmp = NULL;
    if (steps > 1) {
        tmp = (double *)malloc(N * sizeof(double));
        if (!tmp) { free(taps); return -1; }
    }
    const double *cur = in;
    for (int k = 0; k < steps; ++k) {
        int remaining = steps - 1 - k;
        double *nxt = (remaining % 2 == 0) ? out : tmp;
        if (nz > 1) {
#pragma omp parallel for schedule(static)
            for (int64_t z = 0; z < nz; ++z)
                for (int64_t y = 0; y < ny; ++y)
                    for (int64_t x = 0; x < nx; ++x)
                        nxt[(z * ny + y) * nx + x] =
                            point_value_f64(cur, nz, ny, nx, z, y, x, taps, ntaps, boundary);
        } else {
#pragma omp parallel for schedule(static)
            for (int64_t y = 0; y < ny; ++y)
                for (int64_t x = 0; x < nx; ++x)
                    nxt[y * nx + x] = point_value_f64(cur, 1, ny, nx, 0, y, x, taps, ntaps, boundary);
        }
        cur = nxt;
    }
    free(tmp);
    free(taps);
    return 0;
}
