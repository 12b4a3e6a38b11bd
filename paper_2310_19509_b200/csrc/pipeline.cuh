// Device helpers shared by the kernels: packed fp32 pairs, mbarrier waits with an iteration cap,
// bulk asynchronous copies (global -> shared, completion counted on an mbarrier).
#pragma once

#include <stdint.h>

namespace sbnn {

// ---- packed pair of fp32 values in one 64-bit register ------------------------------------------
// fma2 is two independent fp32 FMAs (each rounded to nearest even) issued as one instruction; it
// halves the issue slots the FMAs take, which leaves room for the operand loads.
typedef unsigned long long f32x2;

__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
// (v, v).  (Building the copy on the integer pipe with a byte-permute, or storing weights twice in the
// stream so they load as ready pairs, were both measured slower than the plain register move.)
__device__ __forceinline__ f32x2 dup2(float v) { return pack2(v, v); }
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void fma2(f32x2& d, f32x2 a, f32x2 b) {
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b));
}

// ---- programmatic dependent launch ---------------------------------------------------------------
// grid_dependency_wait: returns once every kernel this one depends on in its stream has completed and its writes are
// visible (immediately if the kernel was launched without programmatic serialization).  Code before it may only
// touch memory no other kernel of the stream writes (weights, its own shared memory).  grid_dependency_release lets
// the next kernel of the stream become resident as SM resources free up; that kernel still waits, in its own
// grid_dependency_wait, for this one to finish.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- mbarrier -------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Largest number of polls before a wait gives up (each poll may itself block for a while inside
// the hardware; in practice this is on the order of a second).
constexpr uint32_t kWaitLimit = 1u << 22;

// Waits for the phase with the given parity.  Returns false, after recording `code` in *status,
// when the cap is reached or another thread of the CTA has already given up (*abort != 0).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort, int* status, int code,
                                          uint32_t limit = kWaitLimit) {
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 64) {
            if (*abort) return false;
            __nanosleep(64);
        }
    }
    *abort = 1;
    atomicCAS(status, 0, code);
    return false;
}

// ---- bulk copy global -> shared (addresses 16-byte aligned, size a multiple of 16 bytes) --------
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst_smem)), "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// ---- tiled copy global -> shared through a 2-D tensor map (opaque 128-byte descriptor made on the host) ----
// Brings the box whose first element is (x, y) -- x along the contiguous dimension -- as [box rows][box width];
// x * element size must be a multiple of 16 bytes, the destination 128-byte aligned.  Elements outside the
// tensor arrive as zeros and count towards the completed bytes.
__device__ __forceinline__ void tensor_g2s_2d(void* dst_smem, const void* tensor_map, int x, int y, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(dst_smem)), "l"(tensor_map), "r"(x), "r"(y), "r"(smem_u32(bar))
                 : "memory");
}

// The same for a 3-D tensor map: box origin (x, y, z), x along the contiguous dimension.
__device__ __forceinline__ void tensor_g2s_3d(void* dst_smem, const void* tensor_map, int x, int y, int z, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(smem_u32(dst_smem)), "l"(tensor_map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
                 : "memory");
}

// ---- tiled copy shared -> global through a 2-D tensor map, tracked by the issuing thread's bulk groups ----
// Stores the [box rows][box width] block at src_smem (laid out as the map's swizzle mode says, 128-byte aligned, 1024
// with the 128-byte swizzle) to the box whose first element is (x, y); the part of the box outside the tensor is not
// written (along x in whole 16-byte pieces).  x * element size must be a multiple of 16 bytes and neither coordinate
// negative.  Shared-memory writes made with ordinary stores must be followed by fence_async_smem() in the writing
// threads, and a barrier, before the copy is issued.
__device__ __forceinline__ void tensor_s2g_2d(const void* tensor_map, int x, int y, const void* src_smem) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(tensor_map), "r"(x), "r"(y), "r"(smem_u32(src_smem))
                 : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Waits until all but the most recent one of the calling thread's bulk groups have finished READING their shared-memory source.
__device__ __forceinline__ void bulk_wait_read_pending1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
// Waits until the calling thread's bulk groups have completed altogether (their global writes are performed).
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

}  // namespace sbnn
