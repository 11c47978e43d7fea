// Shared host/device helpers for the libregione kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "regione.h"

namespace regione {

// Records the first device-side anomaly; later ones do not overwrite it.
__device__ __forceinline__ void record_status(int32_t* dev_status, int code) {
    if (dev_status != nullptr) atomicCAS(dev_status, REGIONE_DEV_OK, code);
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Two fp32 -> packed bf16x2 (round to nearest even); `lo` lands in bits [15:0].
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&p);
}

// 2^x on the special-function unit (flush-to-zero, ~2 ulp); 2^-inf = 0.
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint4 ldg128(const void* p) {
    return __ldg(reinterpret_cast<const uint4*>(p));
}

// Streaming 128-bit load for data that is read exactly once (bypasses L1 allocation).
__device__ __forceinline__ uint4 ld_stream128(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

// Programmatic dependent launch.  Every kernel of the library starts with grid_dependency_wait():
// it returns once the kernel ahead of it in the stream has completed and its writes are visible,
// which is the ordinary stream order, but lets the launch itself (scheduling the grid, making its
// thread blocks resident) overlap the tail of that kernel.  grid_launch_dependents() tells the
// runtime that the kernel behind this one may be made resident.
__device__ __forceinline__ void grid_dependency_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
__device__ __forceinline__ void grid_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Launches `kernel` with programmatic stream serialization (see grid_dependency_wait).
template <typename... Params, typename... Args>
inline cudaError_t launch_overlapped(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem,
                                     cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Per-request scalars (sampler time, step length, decay product) reach a kernel by value, a chunk
// of requests per launch: the host arrays of the C ABI never have to be copied to device memory.
constexpr int kReqChunk = 128;
struct PerRequestF {
    float v[kReqChunk];
};

// The cache refresh a full attention step can carry along (regione_full_attention_store).
struct CacheStore {
    const int32_t* keep_rows;   // dev [B, cap], ascending per request
    const int32_t* n_keep;      // dev [B]
    int cap;
    uint16_t* k_cache;          // dev [B, cap, H, D]
    uint16_t* v_cache;
};

// Host-side argument checks shared by every region-attention entry point (defined in api.cu).
// Returns REGIONE_OK when the call may proceed; *nothing_to_do is set for B == 0 or Nq_cap == 0.
int check_attention_args(const void* q, const void* k_fresh, const void* v_fresh, const void* k_cache,
                         const void* v_cache, const void* n_q, const void* n_fresh, const void* n_cache,
                         int B, int Nq_cap, int Nf_cap, int Nc_cap, int H, int D, const void* out,
                         bool* nothing_to_do);

inline int launch_status(cudaError_t e) { return e == cudaSuccess ? REGIONE_OK : REGIONE_CUDA_ERROR; }

}  // namespace regione
