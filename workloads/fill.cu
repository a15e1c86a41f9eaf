// Device twin of workloads/rng.py: fills a tensor with normal(seed, tensor id, flat index) using the same
// 64-bit integer hash, so host slices and device tensors are bit-identical.  Input generation only.
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

__device__ __forceinline__ uint64_t wl_fin(uint64_t x) {
    x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27; x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return x;
}
__device__ __forceinline__ float wl_normal(uint64_t key, uint64_t idx, float scale) {
    const uint64_t h1 = wl_fin((2 * idx) * 0x9E3779B97F4A7C15ull + key);
    const uint64_t h2 = wl_fin((2 * idx + 1) * 0x9E3779B97F4A7C15ull + key);
    int s = 0;
#pragma unroll
    for (int sh = 0; sh < 64; sh += 16) s += (int)((h1 >> sh) & 0xFFFF) + (int)((h2 >> sh) & 0xFFFF);
    return __fmul_rn((float)(2 * s - 8 * 65535), scale);
}
__global__ void wl_fill_bf16_kernel(__nv_bfloat16* out, uint64_t n, uint64_t key, float scale) {
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x)
        out[i] = __float2bfloat16_rn(wl_normal(key, i, scale));
}
__global__ void wl_fill_f32_kernel(float* out, uint64_t n, uint64_t key, float scale) {
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x)
        out[i] = wl_normal(key, i, scale);
}
extern "C" int wl_fill_normal(void* out, uint64_t n, uint64_t key, float scale, int bf16, void* stream) {
    if (n == 0) return 0;
    const unsigned grid = (unsigned)((n + 255) / 256 < 148u * 32u ? (n + 255) / 256 : 148u * 32u);
    if (bf16) wl_fill_bf16_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>((__nv_bfloat16*)out, n, key, scale);
    else wl_fill_f32_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>((float*)out, n, key, scale);
    return (int)cudaGetLastError();
}
