// Shared host/device helpers of the library (no method arithmetic lives here).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "dash.h"

#define DASH_CUDA_TRY(expr)                          \
    do {                                             \
        cudaError_t e__ = (expr);                    \
        if (e__ != cudaSuccess) return DASH_ERR_CUDA; \
    } while (0)

namespace dash {

// polls before a device-side wait gives up and records DASH_ERR_TIMEOUT
constexpr uint32_t kSpinLimit = 1u << 22;

// Device address of the per-device status word (host side; one word per GPU).
int* status_word_ptr();

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int sm_count() {
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms > 0 ? sms : 148;
}

// cudaFuncAttributeMaxDynamicSharedMemorySize of `kernel`, set once per device: bit `device` of `done` remembers it (the call
// is idempotent, so two threads that race here only repeat it)
template <typename K>
inline bool set_max_smem_once(K kernel, int smem_bytes, std::atomic<uint64_t>& done) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    const uint64_t bit = (dev >= 0 && dev < 64) ? (1ull << dev) : 0ull;
    if (bit && (done.load(std::memory_order_acquire) & bit)) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) != cudaSuccess) return false;
    if (bit) done.fetch_or(bit, std::memory_order_release);
    return true;
}

// Launch of a kernel that calls pdl_wait() before its first global access: it may start while the kernel in front of it in
// the stream drains (programmatic dependent launch); behind anything else it is an ordinary launch.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3((unsigned)block, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

__device__ __forceinline__ uint4 ld_nc_v4(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
// coherent 128-bit load: for data that this very launch may also write (an output that aliases an input)
__device__ __forceinline__ uint4 ld_v4(const void* p) {
    uint4 v;
    asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_v4(void* p, uint4 v) {
    asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Copy one row of `bytes` (multiple of 16, 16-byte aligned ends) with a warp.
__device__ __forceinline__ void warp_copy_row16(const char* __restrict__ src, char* __restrict__ dst, int64_t bytes, int lane) {
    const int nvec = (int)(bytes >> 4);
    constexpr int UN = 8;                       // 8 x 16 B per lane in flight: 4 KB per warp
    for (int base = 0; base < nvec; base += 32 * UN) {
        uint4 r[UN];
#pragma unroll
        for (int k = 0; k < UN; ++k) {
            int v = base + k * 32 + lane;
            if (v < nvec) r[k] = ld_nc_v4(src + ((int64_t)v << 4));
        }
#pragma unroll
        for (int k = 0; k < UN; ++k) {
            int v = base + k * 32 + lane;
            if (v < nvec) st_v4(dst + ((int64_t)v << 4), r[k]);
        }
    }
}
// Same for rows that are only 4-byte granular.
__device__ __forceinline__ void warp_copy_row4(const char* __restrict__ src, char* __restrict__ dst, int64_t bytes, int lane) {
    const int nw = (int)(bytes >> 2);
    for (int v = lane; v < nw; v += 32)
        reinterpret_cast<uint32_t*>(dst)[v] = reinterpret_cast<const uint32_t*>(src)[v];
}

// sequence that holds packed row t: largest s with cu[s] <= t (skips empty sequences)
__device__ __forceinline__ int find_seq(const int32_t* __restrict__ cu, int S, int t) {
    int lo = 0, hi = S;   // invariant: cu[lo] <= t < cu[hi]
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (cu[mid] <= t) lo = mid; else hi = mid;
    }
    return lo;
}

}  // namespace dash
