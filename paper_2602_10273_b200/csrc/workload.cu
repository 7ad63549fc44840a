// CUDA twin of the numpy input generators (synthetic first-order LM logits, hashed KV fill).
// Workload code, not part of the sampler: built into libpsmc_workload.so, used by tests and bench.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

__device__ __forceinline__ uint64_t sm64(uint64_t x) {
    uint64_t z = x + 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
__device__ __forceinline__ double box_muller(uint64_t h) {
    const double u1 = ((double)(uint32_t)(h >> 32) + 0.5) * (1.0 / 4294967296.0);
    const double u2 = ((double)(uint32_t)(h & 0xFFFFFFFFull) + 0.5) * (1.0 / 4294967296.0);
    return sqrt(-2.0 * log(u1)) * cos(2.0 * 3.141592653589793 * u2);
}
__device__ __forceinline__ uint16_t f32_to_bf16_rne(float f) {
    uint32_t b = __float_as_uint(f);
    b += 0x7FFFu + ((b >> 16) & 1u);
    return (uint16_t)(b >> 16);
}
__device__ __forceinline__ void store(void* dst, int dt, int64_t i, double x) {
    const float f = (float)x;
    if (dt == 0) reinterpret_cast<float*>(dst)[i] = f;
    else reinterpret_cast<uint16_t*>(dst)[i] = f32_to_bf16_rne(f);
}

enum : uint64_t { kLogit = 4, kKv = 6 };

__global__ void logits_kernel(void* dst, int dt, int R, int V, int64_t ld, uint64_t seed, int t, int g0, int N,
                              const int32_t* prev, double scale, const double* bias) {
    const int r = blockIdx.y;
    const uint64_t g = (uint64_t)(g0 + r / N);
    uint64_t h = sm64(seed);
    h = sm64(h ^ (kLogit ^ (g << 8)));
    h = sm64(h ^ (uint64_t)t);
    h = sm64(h ^ (uint64_t)(int64_t)prev[r]);
    for (int v = blockIdx.x * blockDim.x + threadIdx.x; v < V; v += gridDim.x * blockDim.x)
        store(dst, dt, (int64_t)r * ld + v, scale * box_muller(sm64(h ^ (uint64_t)v)) + bias[v]);
}

__global__ void kv_kernel(void* dst, int dt, uint64_t seed, int layer, int which, int row0, int R, int H, int max_len,
                          int D) {
    const int64_t per_row = (int64_t)H * max_len * D, total = (int64_t)R * per_row;
    const uint64_t tag = kKv ^ ((uint64_t)layer << 8) ^ ((uint64_t)which << 40);
    const uint64_t h1 = sm64(sm64(seed) ^ tag);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / per_row, rem = i - r * per_row;
        const int64_t hp = rem / D, d = rem - hp * D;  // hp = head * max_len + pos
        uint64_t h = sm64(h1 ^ (uint64_t)(row0 + r));
        h = sm64(h ^ (uint64_t)hp);
        store(dst, dt, i, box_muller(sm64(h ^ (uint64_t)d)));
    }
}

}  // namespace

// dst: DEVICE [R, ld]; prev: DEVICE [R] previous tokens; bias: DEVICE [V] doubles.  dt 0 = fp32, 1 = bf16.
extern "C" int psmc_wl_logits(void* dst, int dt, int R, int V, int64_t ld, uint64_t seed, int t, int g0, int N,
                              const int32_t* prev, double scale, const double* bias, void* stream) {
    dim3 grid((unsigned)((V + 1023) / 1024), (unsigned)R);
    logits_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(dst, dt, R, V, ld, seed, t, g0, N, prev, scale,
                                                                         bias);
    return (int)cudaGetLastError();
}

// dst: DEVICE contiguous [R, H, max_len, D] for rows row0 .. row0+R-1 of (layer, which = 0 K / 1 V).
extern "C" int psmc_wl_kv(void* dst, int dt, uint64_t seed, int layer, int which, int row0, int R, int H, int max_len,
                          int D, void* stream) {
    kv_kernel<<<148 * 16, 256, 0, static_cast<cudaStream_t>(stream)>>>(dst, dt, seed, layer, which, row0, R, H,
                                                                       max_len, D);
    return (int)cudaGetLastError();
}
