// Shared host/device helpers of libdeeprebirth (status codes, launch accounting, bf16 packing).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/dr.h"

namespace dr {

extern std::atomic<long long> g_launches;   // kernels launched by this process
inline void count_launch(int n = 1) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// Record left by a kernel whose bounded wait ran out: {code, site, block, tile}.  The words
// live in one file-scope device array; kernels receive its device address as an argument.
// First writer wins (code is claimed with atomicCAS).
int* dev_status_ptr();   // device address of the record on the current device (host call)
int num_sms();

// A "done once" flag kept per device: function attributes (opt-in shared memory sizes) and occupancy figures belong
// to the device that was current when they were set or queried.
struct PerDeviceFlag {
    std::atomic<unsigned long long> bits{0};
    static int dev() { int d = 0; (void)cudaGetDevice(&d); return d & 63; }
    bool get() const { return (bits.load(std::memory_order_acquire) >> dev()) & 1ull; }
    void set() { bits.fetch_or(1ull << dev(), std::memory_order_release); }
};

__device__ __forceinline__ void report_timeout(int* status, int site, int tile) {
    if (atomicCAS(&status[0], 0, DR_ERR_DEVICE_TIMEOUT) == 0) {
        status[1] = site;
        status[2] = (int)blockIdx.x;
        status[3] = tile;
    }
}

inline int cuda_status(cudaError_t e) { return e == cudaSuccess ? DR_OK : DR_ERR_CUDA; }
inline int launch_status() { return cuda_status(cudaGetLastError()); }
// Set by the network executor around its own pooling launches: the kernel is then launched with programmatic stream
// serialization (it may be scheduled while the layer before it drains and waits for that layer before its first load).
extern thread_local bool g_pool_pdl;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);   // .x = lo (low 16 bits), round to nearest even
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_to_float(const __nv_bfloat16 v) { return __bfloat162float(v); }

// scale^(-beta) for LRN; beta = 0.75 (the usual value) avoids the general pow.
__device__ __forceinline__ float lrn_pow(float s, float beta) {
    if (beta == 0.75f) {
        const float r = rsqrtf(s);              // s^(-1/2)
        return r * (r * rsqrtf(r));             // s^(-1/2) * sqrt(s^(-1/2)), sqrt(r) = r * rsqrt(r): no correctly-rounded sqrt sequence
    }
    return exp2f(-beta * log2f(s));
}

}  // namespace dr
