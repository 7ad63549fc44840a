// Device helpers shared by the psmc kernels: counter hash, warp/block collectives, status word.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/psmc.h"

namespace psmc {

constexpr int kWarp = 32;
constexpr unsigned kFull = 0xffffffffu;

// ---- programmatic dependent launch: a kernel launched with launch_chained() may be scheduled while the kernel
// before it on the stream is still running.  chain_begin() lets the next kernel of the stream be scheduled early in
// turn, then waits until the previous kernel has completed and its writes are visible; nothing that reads or
// writes global memory may come before it.  Both are no-ops in a kernel launched the ordinary way. ----
__device__ __forceinline__ void chain_begin() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// ---- sticky device status word: the first error wins ----
__device__ __forceinline__ void raise_status(int32_t* word, int code) {
    if (word) atomicCAS(word, 0, code);
}

// ---- counter hash (splitmix64 finaliser chained over five parts) ----
__host__ __device__ __forceinline__ uint64_t sm64(uint64_t x) {
    uint64_t z = x + 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
__host__ __device__ __forceinline__ uint64_t hash5(uint64_t a, uint64_t b, uint64_t c, uint64_t d, uint64_t e) {
    uint64_t h = sm64(a);
    h = sm64(h ^ b);
    h = sm64(h ^ c);
    h = sm64(h ^ d);
    return sm64(h ^ e);
}
// top 52 bits, centred: exact in double, strictly inside (0,1)
__host__ __device__ __forceinline__ double hash_uniform(uint64_t h) {
    return ((double)(h >> 12) + 0.5) * (1.0 / 4503599627370496.0);
}
enum : uint64_t { kStreamToken = 1, kStreamResample = 2, kStreamSelect = 3 };

// ---- warp collectives; butterfly sums give every lane the same bits ----
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFull, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}
__device__ __forceinline__ double warp_max(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(kFull, v, o));
    return v;
}
__device__ __forceinline__ int warp_max(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(kFull, v, o));
    return v;
}
// inclusive scan across the lanes of a warp
template <typename T>
__device__ __forceinline__ T warp_scan_incl(T v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        T n = __shfl_up_sync(kFull, v, o);
        if (lane >= o) v += n;
    }
    return v;
}

// ---- block collectives for up to 1024 threads (32 warps); `sh` holds 33 items ----
// Every thread of the CTA calls them; only the first `nwarp` warps carry data (the others pass the identity).
// With nwarp == 1 they are plain warp collectives without any CTA barrier, to be called by warp 0 alone.
// Inclusive scan over threadIdx.x order.  Also returns the block total.  The order of additions is
// fixed by the thread index, so results do not depend on scheduling.
template <typename T>
__device__ __forceinline__ T block_scan_incl(T v, T* sh, T* total, int nwarp) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    T incl = warp_scan_incl(v, lane);
    if (nwarp == 1) {
        if (total) *total = __shfl_sync(kFull, incl, 31);
        return incl;
    }
    __syncthreads();  // sh may still be read by a previous call
    if (lane == 31 && warp < nwarp) sh[warp] = incl;
    __syncthreads();
    T before = T(0), all = T(0);
    for (int w = 0; w < nwarp; ++w) {
        T x = sh[w];
        if (w < warp) before += x;
        all += x;
    }
    if (total) *total = all;
    return before + incl;
}
template <typename T>
__device__ __forceinline__ T block_max(T v, T* sh, int nwarp) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = warp_max(v);
    if (nwarp == 1) return v;
    __syncthreads();
    if (lane == 0 && warp < nwarp) sh[warp] = v;
    __syncthreads();
    T m = sh[0];
    for (int w = 1; w < nwarp; ++w) m = m > sh[w] ? m : sh[w];
    return m;
}
__device__ __forceinline__ double block_sum(double v, double* sh, int nwarp) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = warp_sum(v);
    if (nwarp == 1) return v;
    __syncthreads();
    if (lane == 0 && warp < nwarp) sh[warp] = v;
    __syncthreads();
    double s = 0.0;
    for (int w = 0; w < nwarp; ++w) s += sh[w];
    return s;
}

// CTA barrier, or a warp barrier when a single warp is at work
__device__ __forceinline__ void group_sync(int nwarp) {
    if (nwarp == 1) __syncwarp();
    else __syncthreads();
}

}  // namespace psmc
