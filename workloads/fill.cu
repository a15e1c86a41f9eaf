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

// Closed-loop stand-in for the target model: the token stream itself.  target[b, i] = the stream token that follows node i's
// path if the tokens on the path from the root to node i equal the stream's continuation (the root is the sequence's last
// token), else a token outside the vocabulary range of the stream (so it never matches).  Input generation only: this is
// what an LM head plus arg-max would hand to acceptance.
__global__ void wl_stream_targets_kernel(const int32_t* tokens, long long row_stride, const int32_t* seq_len, const int32_t* tree_tok,
                                         const int32_t* tree_par, const int32_t* tree_dep, const int32_t* n_nodes, int B, int T, int32_t junk_base,
                                         int32_t* target) {
    const int b = blockIdx.x, i = threadIdx.x;
    if (b >= B || i >= T) return;
    const int n = n_nodes[b], pos = seq_len[b];
    int32_t out = -1;
    if (i < n) {
        const int32_t* s = tokens + (long long)b * row_stride;
        bool on = true;
        int c = i;
        for (int guard = 0; guard < T && c > 0; ++guard) {
            on = on && tree_tok[(long long)b * T + c] == s[pos - 1 + tree_dep[(long long)b * T + c]];
            c = tree_par[(long long)b * T + c];
        }
        out = on ? s[pos + tree_dep[(long long)b * T + i]] : junk_base + i;
    }
    target[(long long)b * T + i] = out;
}
extern "C" int wl_stream_targets(const int32_t* tokens, long long row_stride, const int32_t* seq_len, const int32_t* tree_tok, const int32_t* tree_par,
                                 const int32_t* tree_dep, const int32_t* n_nodes, int B, int T, int32_t junk_base, int32_t* target, void* stream) {
    if (B <= 0 || T <= 0 || T > 1024) return 1;
    wl_stream_targets_kernel<<<B, T, 0, (cudaStream_t)stream>>>(tokens, row_stride, seq_len, tree_tok, tree_par, tree_dep, n_nodes, B, T, junk_base, target);
    return (int)cudaGetLastError();
}

// Turns target ids into logits (and back): row (b, i) of the fp32 logits gets `value` at column target[b, i] where that is a
// vocabulary id, the old entry goes to saved[b, i]; restore != 0 writes the saved entries back.  Input generation only: the
// closed loop's stand-in for an LM head whose arg-max is the given target.
__global__ void wl_plant_logits_kernel(float* logits, long long row_stride, const int32_t* target, const int32_t* n_nodes, int B, int T, int V,
                                       float value, float* saved, int restore) {
    const int b = blockIdx.x, i = threadIdx.x;
    if (b >= B || i >= T || i >= n_nodes[b]) return;
    const int32_t t = target[(long long)b * T + i];
    if (t < 0 || t >= V) return;
    float* p = logits + ((long long)b * T + i) * row_stride + t;
    if (restore) { *p = saved[(long long)b * T + i]; }
    else { saved[(long long)b * T + i] = *p; *p = value; }
}
extern "C" int wl_plant_logits(float* logits, long long row_stride, const int32_t* target, const int32_t* n_nodes, int B, int T, int V, float value,
                               float* saved, int restore, void* stream) {
    if (B <= 0 || T <= 0 || T > 1024) return 1;
    wl_plant_logits_kernel<<<B, T, 0, (cudaStream_t)stream>>>(logits, row_stride, target, n_nodes, B, T, V, value, saved, restore);
    return (int)cudaGetLastError();
}
