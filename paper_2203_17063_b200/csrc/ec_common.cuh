// Shared device/host helpers of the eventually consistent collectives library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "ec.h"

struct ec_ctx;

namespace ec {

extern thread_local int g_last_cuda_error;

// Internal: whether this context's apply kernels are launched as programmatic dependents of whatever precedes them in
// the stream (the default) - they start while their predecessor's last blocks still run and wait on the device
// (griddepcontrol.wait, their first instruction) until it has completed and its writes are visible.  Results do not
// change; the gaps between the applies of an epoch go (config 2 epoch: 0.191 -> 0.187 ms).
void allreduce_set_dependent_launch(ec_ctx* ctx, bool on);

// Programmatic dependent launch: the device-side wait (returns at once in a kernel launched the ordinary way) ...
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ... and the launch.
template <class... KArgs, class... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(block); cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

inline int cuda_fail(cudaError_t e) {
    g_last_cuda_error = (int)e;
    return EC_ERR_CUDA;
}

#define EC_CUDA(call)                                  \
    do {                                               \
        cudaError_t e__ = (call);                      \
        if (e__ != cudaSuccess) return ec::cuda_fail(e__); \
    } while (0)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline size_t in_bytes(int dtype) { return dtype == EC_F32 ? 4 : dtype == EC_BF16 ? 2 : 8; }
inline size_t out_bytes(int dtype) { return (dtype == EC_F32 || dtype == EC_BF16) ? 4 : 8; }

// Pointer table passed by value in the kernel parameters: stream-ordered, nothing to upload.
template <int CAP>
struct PtrTable {
    const void* p[CAP];
};

// ---- streaming 128-bit accesses -------------------------------------------------------------
// Rank buffers are read exactly once: keep them out of L1 and mark them evict-first in L2 so
// that they do not push out the partial result, which the next round reads again.
__device__ __forceinline__ uint64_t evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint4 ld_stream16(const void* p, uint64_t pol) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p), "l"(pol));
    return v;
}
__device__ __forceinline__ uint2 ld_stream8(const void* p, uint64_t pol) {
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v2.u32 {%0,%1}, [%2], %3;"
                 : "=r"(v.x), "=r"(v.y)
                 : "l"(p), "l"(pol));
    return v;
}
__device__ __forceinline__ uint4 ld_plain16(const void* p) { return *reinterpret_cast<const uint4*>(p); }
__device__ __forceinline__ void st_plain16(void* p, uint4 v) { *reinterpret_cast<uint4*>(p) = v; }

// Result accesses with an explicit L2 policy (0 normal, 1 evict-last = keep for the next round, 2 evict-first).
__device__ __forceinline__ uint64_t result_policy(int hint) {
    uint64_t pol;
    if (hint == 1) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    else if (hint == 2) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    else asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint4 ld_hint16(const void* p, uint64_t pol) {
    uint4 v;
    asm volatile("ld.global.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p), "l"(pol)
                 : "memory");
    return v;
}
__device__ __forceinline__ void st_hint16(void* p, uint4 v, uint64_t pol) {
    asm volatile("st.global.L2::cache_hint.v4.u32 [%0], {%1,%2,%3,%4}, %5;"
                 :
                 : "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "l"(pol)
                 : "memory");
}

}  // namespace ec
