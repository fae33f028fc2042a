/*
 * stencil.h — C ABI of the sm_100a stencil-sweep library (libstencil_b200.so).
 *
 * The operation is the one the paper's case-study protocol defines: a stencil
 * of radius R is the single-channel (2R+1)^d cross-correlation with zero
 * padding R and stride 1,
 *
 *     out[p] = sum_o  w[o] * in[p + o]        for every grid point p,
 *
 * applied once or iterated over time steps (the protocol repeats the sweep and
 * reports the amortised per-step latency).  This library generalises the
 * paper's 2D box to 2D/3D, star or box neighbourhoods, on fp32 grids
 * (stencil_plan / stencil_apply) and on FP64 grids, the paper's own precision
 * (stencil_plan_f64 / stencil_apply_f64).
 *
 * Conventions for every call
 *   - returns a status (STENCIL_OK or a negative STENCIL_ERR_*); never throws,
 *     aborts or prints; results come back through pointers.
 *   - dims are slowest axis first: (ny, nx) or (nz, ny, nx); x is contiguous,
 *     rows are not padded.
 *   - "HOST" / "DEVICE" beside a pointer says where the memory must live.
 *   - there is no CPU fallback: without a CUDA device every compute call
 *     returns STENCIL_ERR_CUDA.
 */
#ifndef STENCIL_B200_H
#define STENCIL_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define STENCIL_API __attribute__((visibility("default")))
#else
#define STENCIL_API
#endif

typedef struct stencil_plan_s* stencil_plan_t;   /* opaque, owned by the library */

enum { STENCIL_STAR = 0, STENCIL_BOX = 1 };      /* shape    */
enum { STENCIL_ZERO = 0, STENCIL_PERIODIC = 1 }; /* boundary */

enum {
    STENCIL_OK              =  0,
    STENCIL_ERR_INVALID     = -1,  /* bad argument (NULL, size, enum, alignment, aliasing)      */
    STENCIL_ERR_UNSUPPORTED = -2,  /* valid request outside what the kernels cover               */
    STENCIL_ERR_CUDA        = -3,  /* a CUDA runtime/driver call failed (or no device)           */
    STENCIL_ERR_ALLOC       = -4,  /* host or device allocation failed                           */
    STENCIL_ERR_TIMEOUT     = -5,  /* a bounded device-side wait gave up (see query_status)      */
    STENCIL_ERR_TOO_LARGE   = -6,  /* grid larger than stencil_apply_static's fixed scratch      */
    STENCIL_ERR_BOUNDS      = -7   /* debug build only: a kernel's store fell outside the output  */
};

/* Largest grid, in points, that stencil_apply_static accepts (8 MiB of fp32). */
#define STENCIL_STATIC_MAX_POINTS (1 << 21)

/* Kernel families a plan can run.  AUTO lets the plan choose. */
enum {
    STENCIL_VARIANT_AUTO    = 0,
    STENCIL_VARIANT_GENERIC = 1,   /* one thread per point, global-memory gather; any request    */
    STENCIL_VARIANT_STREAM  = 2,   /* TMA-staged x-y tiles streamed along the slowest axis       */
    STENCIL_VARIANT_FUSED   = 3    /* set only: STREAM, and fail unless iterated applies can fuse
                                      several time steps per pass; reads back as STREAM with
                                      STENCIL_KEY_FUSE_STEPS >= 2                                */
};

/* Keys of stencil_plan_set / stencil_plan_get. */
enum {
    STENCIL_KEY_VARIANT      = 0,  /* set/get: STENCIL_VARIANT_*                                 */
    STENCIL_KEY_TILE_X       = 1,  /* set/get: region width of fused 3D passes, 128, 256, 384 or 512
                                      (FP64: 128 or 256; 0 = auto)                               */
    STENCIL_KEY_TILE_Y       = 2,  /* set/get: tile height in rows   (0 = default)               */
    STENCIL_KEY_FUSE_STEPS   = 3,  /* set: time steps fused per pass (0 = auto, 1 = off; 3D fp32
                                      stars: 2-4; 3D FP64 stars of radius 1 with a zero boundary:
                                      2 or 3; 2D grids: the one depth the operator's fused
                                      kernel has: star and box R=1: 4, star R=2: 3, box R=2: 2,
                                      fp32 stars R=3 and 4: 2);
                                      get: the number iterated applies will use (1 = none)       */
    STENCIL_KEY_LAUNCHES     = 4,  /* get: kernels launched by this plan so far                  */
    STENCIL_KEY_SCRATCH_BYTES= 5,  /* get: device bytes the plan currently owns as scratch       */
    STENCIL_KEY_CHUNK_Z      = 6,  /* set/get: planes per CTA along the streamed axis (0 = auto) */
    STENCIL_KEY_STAGES       = 7,  /* set/get: depth of the shared-memory plane ring (0 = auto)  */
    STENCIL_KEY_STREAMING_STORE = 8, /* set/get: 1 = write results with evict-first stores       */
    STENCIL_KEY_ROWS_PER_THREAD = 9, /* set/get: tile rows each thread computes (0 = default)    */
    STENCIL_KEY_WAIT_POLLS   = 10, /* set/get: polls after which a device-side wait of the tiled
                                      kernels gives up (each poll sleeps <= 20 us)               */
    STENCIL_KEY_CHAIN_LAUNCHES = 12, /* set/get: 1 (default) = launches 2..n of an iterated apply are
                                      programmatic dependent launches: each begins its preamble
                                      while its predecessor drains and waits for it before it
                                      touches global memory; 0 = ordinary launches             */
    STENCIL_KEY_FUSED_TILE_Y = 13,   /* set/get: region height of fused 3D passes, 16, 20 or 32 (FP64: 16
                                      or 32); 0 = auto                                           */
    STENCIL_KEY_PERIODIC_ROUTE = 14, /* set/get: how the tiled kernels handle a periodic boundary
                                      where the sweep does not wrap by itself (it does for 3D
                                      stars of radius <= 4 and 3D boxes with nx a multiple of
                                      128, in FP64 of 64, unless this key is 1 or 2).
                                      1 = sweep from a padded copy with wrapped halos; 2 = zero-
                                      boundary sweep plus a correction of the points within R of
                                      a face (needs every extent >= 2R, else as 1); 0 (default)
                                      = whichever of the two is cheaper for the operator.
                                      Iterated applies of an operator with a fused kernel run
                                      fused zero-boundary passes of L steps and rewrite the points
                                      within L*R of a face afterwards (every extent >= 2*L*R),
                                      unless this key is 1 or STENCIL_KEY_FUSE_STEPS is 1         */
    STENCIL_KEY_TEST_DROP_PLANE = 11, /* set/get, test hook: every CTA (2D kernels: every warp) of the
                                      tiled kernels never loads its input plane (2D: batch of
                                      rows) of this index, so the bounded wait for it expires and
                                      stencil_query_status reports STENCIL_ERR_TIMEOUT; nothing
                                      faults (-1 = off, the default)                             */
    STENCIL_KEY_DEVICE       = 15,   /* get: the CUDA device the plan's device state lives on
                                      (the one current at its first apply; -1 before that).
                                      Later applies must run with that device current
                                      (STENCIL_ERR_INVALID otherwise)                            */
    STENCIL_KEY_DEBUG_SHRINK = 16    /* set/get, debug builds of the library only (compiled with
                                      -DSTENCIL_DEBUG; STENCIL_ERR_UNSUPPORTED otherwise, which
                                      is also how a caller tells the two builds apart).  A debug
                                      build checks every global store of the tiled kernels
                                      against the extent of the output grid; a store outside it
                                      is skipped and stencil_query_status reports
                                      STENCIL_ERR_BOUNDS.  This test hook makes the checks take
                                      the grid to be `value` points shorter than it is (0, the
                                      default: its true extent), so that the stores to its last
                                      points trip them; nothing faults                           */
};

/*
 * stencil_plan — validate a stencil and prepare to run it.
 * Paper: "Case-study protocol" (radius R, (2R+1)^d neighbourhood, zero padding
 * R, stride 1, cross-correlation orientation).
 *
 *   plan_out  HOST, receives the handle; set to NULL on any error.
 *   ndim      2 or 3.
 *   dims      HOST, ndim entries, slowest axis first, each >= 1.
 *   radius    R >= 1; R <= 8 (larger: STENCIL_ERR_UNSUPPORTED).  The TMA-staged kernels
 *             cover, in fp32 and FP64, stars up to radius 8, 3D boxes up to radius 2
 *             and 2D boxes up to radius 4; other requests run on the
 *             one-thread-per-point kernel.
 *   shape     STENCIL_STAR or STENCIL_BOX.
 *   weights   HOST, dense (2R+1)^ndim floats in C order, same axis order as
 *             dims: entry [dz+R][dy+R][dx+R] multiplies in[p+(dz,dy,dx)]
 *             (byte-for-byte the weight of a 1-channel conv2d/conv3d).  Copied;
 *             the caller keeps ownership.  STAR is a promise that every
 *             off-axis entry is exactly zero, and is checked
 *             (STENCIL_ERR_INVALID otherwise).  Zero entries cost nothing.
 *   boundary  STENCIL_ZERO (taps outside the grid contribute 0; every grid
 *             point is an output) or STENCIL_PERIODIC (indices wrap).
 *
 * Plan-owned device memory, all allocated at first need by an apply: one
 * scratch grid of N floats for steps > 1; two grids with rows padded to 16
 * bytes when nx is not a multiple of 4 (zero boundary); one or two padded
 * copies of the grid with wrapped halos when a periodic apply takes the
 * padded-copy route (STENCIL_KEY_PERIODIC_ROUTE).  STENCIL_KEY_SCRATCH_BYTES
 * reports the total.
 *
 * Needs no device memory until the first apply.  Errors: INVALID, UNSUPPORTED,
 * ALLOC.
 */
STENCIL_API int stencil_plan(stencil_plan_t* plan_out, int ndim, const int64_t* dims, int radius,
                 int shape, const float* weights, int boundary);

/*
 * stencil_apply — enqueue `steps` sweeps on `stream`:  out = S^steps(in).
 * Paper: "Case-study protocol" (the sweep, and its repetition over time steps
 * with each step consuming the previous result).
 *
 *   in, out   DEVICE, N = prod(dims) floats each, 16-byte aligned, must not
 *             overlap; caller-owned.  `in` is never written.
 *   steps     >= 0.  0 copies in to out.  k > 1 iterates; every intermediate
 *             field is an fp32 grid (ping-pong between `out` and one
 *             plan-owned scratch grid of N floats, allocated on first need).
 *   stream    a cudaStream_t (NULL = the legacy default stream).
 *
 * Enqueue only: returns without waiting for the GPU.  A plan must not be used
 * by two applies that overlap in time (they would share the scratch grid).
 * Errors: INVALID (NULL plan/pointers, misaligned, overlapping, steps < 0),
 * ALLOC (scratch), CUDA (launch or tensor-map encode failed).
 */
STENCIL_API int stencil_apply(stencil_plan_t plan, const float* in, float* out, int steps, void* stream);

/*
 * stencil_plan_f64 / stencil_apply_f64 — the same operation on FP64 grids, the
 * precision of the paper's own case study ("Case-study protocol": FP64).
 * Arguments, layout, ownership and errors are those of stencil_plan and
 * stencil_apply with double in place of float.  A plan made by one of the two
 * plan calls is only accepted by the matching apply call (STENCIL_ERR_INVALID
 * otherwise); stencil_destroy, stencil_query_status and the knobs serve both.
 * TMA-staged kernels cover stars up to radius 8 (2D and 3D), 2D boxes up to
 * radius 4 and 3D boxes up to radius 2, with a zero boundary (rows of an odd
 * number of doubles through grids with padded rows) or a periodic one (even
 * nx); everything else runs on the one-thread-per-point kernel.  Temporal
 * blocking in FP64 exists for 2D grids with radius <= 2 and for 3D stars of
 * radius 1 with a zero boundary (even nx).
 */
STENCIL_API int stencil_plan_f64(stencil_plan_t* plan_out, int ndim, const int64_t* dims, int radius,
                                 int shape, const double* weights, int boundary);
STENCIL_API int stencil_apply_f64(stencil_plan_t plan, const double* in, double* out, int steps,
                                  void* stream);

/*
 * stencil_apply_planes / stencil_apply_planes_f64 — one sweep restricted to the
 * output planes [z_begin, z_end) of a 3D grid (rows [z_begin, z_end) of a 2D
 * grid: the range always runs along the slowest axis):  out[z] = S(in)[z] for
 * those planes, the rest of `out` is left untouched.  All of `in` the planes
 * depend on (R planes on either side, inside the grid) must be valid.  Lets a
 * caller that owns a slab of a larger grid sweep the planes that do not depend
 * on its neighbours' data while that data is still on its way, and the others
 * afterwards.  The paper has no counterpart (it runs on one GPU).
 *
 * Plans on the tiled kernels with a zero boundary and rows that are a multiple
 * of 16 bytes only; STENCIL_ERR_UNSUPPORTED otherwise (periodic, generic
 * variant, other row lengths).  Pointers and errors as for stencil_apply
 * (stencil_apply_f64); INVALID also for z_begin < 0, z_end beyond the slowest
 * extent or z_begin >= z_end.  Enqueue only.
 */
STENCIL_API int stencil_apply_planes(stencil_plan_t plan, const float* in, float* out, int64_t z_begin,
                                     int64_t z_end, void* stream);
STENCIL_API int stencil_apply_planes_f64(stencil_plan_t plan, const double* in, double* out, int64_t z_begin,
                                         int64_t z_end, void* stream);

/*
 * stencil_apply_host — the same operation on HOST buffers (an addition of this
 * library for end-to-end use; the paper's protocol times device-resident
 * grids and has no counterpart): copies `in_host`
 * to a plan-owned device grid, runs stencil_apply, copies the result back to
 * `out_host` and waits for it.  Pinned host memory makes the copies
 * asynchronous up to the final wait; pageable memory works but is slower.
 * `in_host` and `out_host` may be the same buffer.  Allocates two plan-owned
 * device grids of N floats on first use.  A single sweep (steps == 1) of a 3D
 * grid on the tiled kernel is pipelined: the grid is cut into 8 or 16 slabs of planes
 * and the upload of one slab, the sweep of the previous one and the download
 * of the one before overlap on two plan-owned copy streams (ordered after the
 * work already queued on `stream`), which needs pinned host memory to pay off.
 */
STENCIL_API int stencil_apply_host(stencil_plan_t plan, const float* in_host, float* out_host, int steps,
                       void* stream);

/*
 * stencil_apply_static — stencil_apply for callers that must not allocate
 * device memory.  (An addition of this library; the paper has no counterpart.)
 *
 * Some programs cannot call cudaMalloc where they run the sweep: a solver or
 * server that has already handed all device memory to its own pool, or a
 * time-stepping loop that cannot afford the device-wide stall cudaMalloc and
 * cudaFree bring.  stencil_apply allocates on first use (a status word, the tap
 * list, and for steps > 1 a scratch grid).  This entry point allocates nothing,
 * neither through the CUDA runtime nor through any library: its ping-pong grid
 * and tap list sit in one fixed array inside the library, 8 MiB + 77 KiB
 * (8,467,456 bytes) of device memory that every GPU which loads the library
 * holds until the process ends.
 *
 *   in, out, steps, stream   exactly as for stencil_apply; the result is the
 *                            same up to fp32 summation order (it runs the
 *                            one-thread-per-point kernel, whatever the plan's
 *                            variant).
 *   limit                    prod(dims) <= STENCIL_STATIC_MAX_POINTS, else
 *                            STENCIL_ERR_TOO_LARGE and nothing is enqueued.
 *
 * The first call on each device also looks up the array's device address (the
 * name of the array is not an address on the host); make that first call with
 * the device current and before starting any stream capture.  A call whose
 * plan's taps are not in the array (the plan's first call, or after a call of
 * another plan) uploads them with an asynchronous copy from the plan's own,
 * pageable host memory: that copy may make the host wait for earlier work on
 * `stream`, and it does not belong inside a stream capture either; a plan that
 * calls again straight after itself uploads nothing.  All calls, from all plans,
 * share the one array: two calls whose GPU work overlaps (different streams, or
 * different host threads) race on it and on the tap list, so serialise them.
 * Nothing has to be cleared between calls: every scratch cell is written before
 * it is read, and the taps are replaced whenever another plan's are in place.
 */
STENCIL_API int stencil_apply_static(stencil_plan_t plan, const float* in, float* out, int steps,
                                     void* stream);

/*
 * stencil_destroy — free the plan and everything it owns (its device memory on
 * the device it lives on, after waiting for the stream of its last apply).
 * NULL is a no-op.  Housekeeping of this library: no passage of the paper
 * defines it.
 */
STENCIL_API int stencil_destroy(stencil_plan_t plan);

/* Static, NUL-terminated description of a status code. */
STENCIL_API const char* stencil_status_string(int status);

/* Static name of a STENCIL_VARIANT_* value ("generic", "stream", ...). */
STENCIL_API const char* stencil_variant_name(int variant);

/*
 * stencil_query_status — wait for the stream of the plan's last apply and
 * return the device status word: STENCIL_OK, or STENCIL_ERR_TIMEOUT if a
 * bounded wait inside a kernel expired (the kernel then returned early and
 * `out` is not valid), or, from a debug build of the library,
 * STENCIL_ERR_BOUNDS if a kernel skipped a store that fell outside the output
 * grid (see STENCIL_KEY_DEBUG_SHRINK).  The word is cleared by the query.
 */
STENCIL_API int stencil_query_status(stencil_plan_t plan);

/*
 * stencil_plan_set / stencil_plan_get — tuning knobs and counters
 * (STENCIL_KEY_*).  Setting a variant the plan cannot run for its
 * dims/radius/boundary returns STENCIL_ERR_UNSUPPORTED and leaves the plan
 * unchanged.  `value` of get is HOST.
 */
STENCIL_API int stencil_plan_set(stencil_plan_t plan, int key, int64_t value);
STENCIL_API int stencil_plan_get(stencil_plan_t plan, int key, int64_t* value);

#ifdef __cplusplus
}
#endif
#endif /* STENCIL_B200_H */
