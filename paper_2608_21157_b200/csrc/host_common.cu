// Host side shared by every kernel family: device state of a plan, tensor maps, and the launches of
// the one-thread-per-point kernel.
#include "host.h"
#include "kernel_generic.cuh"

namespace stencil_host {

// driver entry point for tensor-map encoding, fetched at run time so that the library loads on
// machines without a driver
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

std::mutex g_config_mutex;

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

int kernel_limits(const void* kernel, int threads, size_t smem, int dev, KernelLimits& lim, bool want_occ) {
    std::lock_guard<std::mutex> lock(g_config_mutex);
    if (dev != lim.device) {                       // function attributes are per device
        lim = KernelLimits{};
        lim.device = dev;
    }
    if (smem > lim.smem_allowed) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
            cudaGetLastError();
            return -1;
        }
        lim.smem_allowed = smem;
    }
    if (!want_occ) return 1;
    if (lim.occ_smem != smem || lim.occ <= 0) {
        int o = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o, kernel, threads, smem) != cudaSuccess) {
            cudaGetLastError();
            o = 0;
        }
        lim.occ = std::max(o, 1);
        lim.occ_smem = smem;
    }
    return lim.occ;
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
    p->sms = sm_count();
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

// Multiprocessors of the current device (asked once per device).
int sm_count() {
    constexpr int kMaxDevices = 64;
    static int cache[kMaxDevices] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 148; }
    if (dev >= 0 && dev < kMaxDevices && cache[dev] > 0) return cache[dev];
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) {
        cudaGetLastError();
        return 148;
    }
    if (dev >= 0 && dev < kMaxDevices) cache[dev] = v;      // a benign race: every writer stores the same value
    return v;
}

// A plan's device state (status word, taps, scratch grids, tensor maps) belongs to the device
// that was current at its first apply; later applies must run with the same device current.
int check_device(const stencil_plan_s* p) {
    if (p->device < 0) return STENCIL_OK;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return STENCIL_ERR_CUDA; }
    return dev == p->device ? STENCIL_OK : STENCIL_ERR_INVALID;
}

int get_tensor_map(stencil_plan_s* p, const void* cfg, int box_x, int box_y, const float* src,
                   const CUtensorMap** out, int tnx, int tny, int tnz) {
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

int get_tensor_map_f64(stencil_plan_s* p, const void* cfg, int box_x, int box_y, const double* src,
                       const CUtensorMap** out, int tnx, int tny, int tnz) {
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

int launch_generic(stencil_plan_s* p, const float* src, float* dst, cudaStream_t st) {
    return launch_generic_taps(p, src, dst, p->d_taps, (int)p->taps.size(), st);
}

int launch_generic_f64(stencil_plan_s* p, const double* src, double* dst, cudaStream_t st) {
    Grid g{p->nz, p->ny, p->nx};
    const int grid = generic_grid_size(g, plan_sms(p));
    const int ntaps = (int)p->taps64.size();
    if (p->boundary == STENCIL_PERIODIC)
        stencil_generic_kernel<true, double><<<grid, kGenericThreads, 0, st>>>(src, dst, g, p->d_taps64, ntaps);
    else
        stencil_generic_kernel<false, double><<<grid, kGenericThreads, 0, st>>>(src, dst, g, p->d_taps64, ntaps);
    if (cudaGetLastError() != cudaSuccess) return STENCIL_ERR_CUDA;
    p->launches++;
    return STENCIL_OK;
}

int launch_generic_taps(stencil_plan_s* p, const float* src, float* dst, const Tap* d_taps, int ntaps,
                        cudaStream_t st) {
    Grid g{p->nz, p->ny, p->nx};
    const int grid = generic_grid_size(g, plan_sms(p));
    if (p->boundary == STENCIL_PERIODIC)
        stencil_generic_kernel<true><<<grid, kGenericThreads, 0, st>>>(src, dst, g, d_taps, ntaps);
    else
        stencil_generic_kernel<false><<<grid, kGenericThreads, 0, st>>>(src, dst, g, d_taps, ntaps);
    if (cudaGetLastError() != cudaSuccess) return STENCIL_ERR_CUDA;
    p->launches++;
    return STENCIL_OK;
}

}  // namespace stencil_host
