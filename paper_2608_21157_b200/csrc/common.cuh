// Shared device-side definitions of the stencil library (CUDA path only).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace stencil {

// One non-zero tap: in[p + (dz,dy,dx)] * w.
template <typename T>
struct TapT {
    int dz, dy, dx;
    T w;
};
using Tap = TapT<float>;

__device__ __forceinline__ float fma_t(float a, float b, float c) { return fmaf(a, b, c); }
__device__ __forceinline__ double fma_t(double a, double b, double c) { return fma(a, b, c); }

// Packed fp32 arithmetic: one instruction does two IEEE operations, each rounded exactly like
// fmaf / * on its own half (round to nearest even, denormals kept), so results are bit-identical to
// the scalar forms.  It halves the issue slots of FMA chains whose operands sit in aligned
// register pairs (the two halves of a float4).  All three operands are register pairs, the
// weight (w, w) included: it pays where a few weights serve many FMAs (the stars), not where every
// FMA has a weight of its own (the boxes).
__device__ __forceinline__ float2 fma2(float w, float2 v, float2 a) { return __ffma2_rn(make_float2(w, w), v, a); }
__device__ __forceinline__ float2 mul2(float w, float2 v) { return __fmul2_rn(make_float2(w, w), v); }
__device__ __forceinline__ float2 lo2(const float4& v) { return make_float2(v.x, v.y); }
__device__ __forceinline__ float2 hi2(const float4& v) { return make_float2(v.z, v.w); }
__device__ __forceinline__ float4 join4(float2 lo, float2 hi) { return make_float4(lo.x, lo.y, hi.x, hi.y); }
// a = w * v + a on all four lanes of a float4
__device__ __forceinline__ void fma4(float4& a, float w, const float4& v) {
    a = join4(fma2(w, lo2(v), lo2(a)), fma2(w, hi2(v), hi2(a)));
}
__device__ __forceinline__ float4 fma4r(float w, const float4& v, const float4& a) {
    return join4(fma2(w, lo2(v), lo2(a)), fma2(w, hi2(v), hi2(a)));
}
__device__ __forceinline__ float4 mul4(float w, const float4& v) { return join4(mul2(w, lo2(v)), mul2(w, hi2(v))); }

// The same operations on a double2 (two plain FP64 FMAs), so that kernels written for either
// 16-byte vector share their arithmetic.
__device__ __forceinline__ void fma4(double2& a, double w, const double2& v) {
    a.x = fma(w, v.x, a.x); a.y = fma(w, v.y, a.y);
}
__device__ __forceinline__ double2 fma4r(double w, const double2& v, const double2& a) {
    return make_double2(fma(w, v.x, a.x), fma(w, v.y, a.y));
}
__device__ __forceinline__ double2 mul4(double w, const double2& v) { return make_double2(w * v.x, w * v.y); }

template <typename V> __device__ __forceinline__ V vzero();
template <> __device__ __forceinline__ float4 vzero<float4>() { return make_float4(0.f, 0.f, 0.f, 0.f); }
template <> __device__ __forceinline__ double2 vzero<double2>() { return make_double2(0.0, 0.0); }
__device__ __forceinline__ void vunpack(const float4& v, float (&a)[4]) { a[0] = v.x; a[1] = v.y; a[2] = v.z; a[3] = v.w; }
__device__ __forceinline__ void vunpack(const double2& v, double (&a)[2]) { a[0] = v.x; a[1] = v.y; }
template <typename V> __device__ __forceinline__ V vpack(const float (&a)[4]) { return make_float4(a[0], a[1], a[2], a[3]); }
template <typename V> __device__ __forceinline__ V vpack(const double (&a)[2]) { return make_double2(a[0], a[1]); }

// Grid extents as the kernels see them; 2D grids have nz == 1.
struct Grid {
    int nz, ny, nx;
};

// Value of the plan's device status word once a bounded wait has given up.
constexpr int kStatusTimeout = -5;
constexpr int kStatusBounds = -7;

// Debug builds (compiled with -DSTENCIL_DEBUG) check every global store of the tiled kernels against the extent
// of the output grid: a store of n elements at p that would not lie inside [out, out + g.out_points) is skipped
// and recorded in the status word (STENCIL_ERR_BOUNDS at the next stencil_query_status).  Release builds compile
// the check away.
template <typename E, typename G>
__device__ __forceinline__ bool store_in_grid(const E* p, int n, const E* out, const G& g, int* status) {
#ifdef STENCIL_DEBUG
    const long long i = p - out;
    if (i < 0 || i + n > g.out_points) {
        atomicExch(status, kStatusBounds);
        return false;
    }
#else
    (void)p; (void)n; (void)out; (void)g; (void)status;
#endif
    return true;
}

}  // namespace stencil
