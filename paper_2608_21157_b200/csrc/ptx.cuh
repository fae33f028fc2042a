// Thin inline-PTX wrappers used by the tiled kernels: shared-memory mbarriers
// and TMA tile loads (cp.async.bulk.tensor, the plain non-multicast form).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace stencil {

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

// Makes freshly initialised barriers visible to the async (TMA) proxy.
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Arrival by the lanes where `take` holds, as a predicated instruction (no branch).
__device__ __forceinline__ void mbar_arrive_if(bool take, uint32_t bar) {
    asm volatile(
        "{\n\t.reg .pred q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "@q mbarrier.arrive.shared::cta.b64 _, [%0];\n\t}"
        ::"r"(bar), "r"((uint32_t)take)
        : "memory");
}

// One poll; the thread may sleep inside it for up to kWaitHintNs nanoseconds
// (a hint to the hardware), which keeps waiting warps out of the issue slots.
constexpr uint32_t kWaitHintNs = 20000;

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(kWaitHintNs)
        : "memory");
    return ok != 0;
}

// Every wait in the library is bounded: after kWaitPolls unsuccessful polls
// (each at most kWaitHintNs long, so some seconds in total at worst) the caller
// records a timeout in the plan's status word and leaves the kernel.
constexpr uint32_t kWaitPolls = 1u << 20;

__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t polls = kWaitPolls) {
    if (mbar_try_wait(bar, parity)) return true;          // the usual case: already complete
    for (uint32_t it = 1; it < polls; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

// 3D tile load global -> shared, completion counted in bytes on `bar`.
// Coordinates are signed; elements outside the tensor arrive as zero.
// x * sizeof(float) must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int x, int y, int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
        : "memory");
}

// Programmatic dependent launch.  A kernel launched with the "programmatic stream
// serialization" attribute may start while the previous kernel of the stream is still
// draining; dependency_wait() then blocks until that kernel has completed and its writes
// are visible.  Everything a kernel reads from or writes to global memory must come after
// it.  allow_dependents() lets the next kernel of the stream begin its own preamble early.
// Both are no-ops in a kernel launched the ordinary way.
__device__ __forceinline__ void dependency_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
__device__ __forceinline__ void allow_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

}  // namespace stencil
