// Pipe-rate microbenchmark behind the figures the design doc quotes for the softmax loop of tree attention (one block on one SM):
// cycles per warp instruction for the instructions that loop is made of (ex2, packed fp32 FMA and ADD, bf16x2 conversion,
// three-input max), alone and mixed, with one warp (32 threads), one warp per SM sub-partition (128) and two (256); and the
// wake-up latency of an mbarrier wait, suspended (try_wait) or spinning (test_wait).
//
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -o pipe_rates pipe_rates.cu && ./pipe_rates
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#define CHK(x) do { cudaError_t e = (x); if (e != cudaSuccess) { printf("CUDA %s at %d\n", cudaGetErrorString(e), __LINE__); return 1; } } while (0)

__device__ __forceinline__ float ex2(float x) { float y; asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ uint32_t cvt2(float lo, float hi) { uint32_t r; asm volatile("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo)); return r; }
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b) { uint32_t r; asm volatile("prmt.b32 %0, %1, %2, 0x7632;" : "=r"(r) : "r"(a), "r"(b)); return r; }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) { uint64_t d; asm volatile("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c)); return d; }
__device__ __forceinline__ float fmax3(float a, float b, float c) { float d; asm volatile("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c)); return d; }

constexpr int N = 512;   // iterations, 8 independent chains each

template <int MODE>
__global__ void k(float* out, long long* cyc, float seed) {
    float a[8];
    uint32_t u[8];
    uint64_t w[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) { a[j] = seed * (j + 1 + threadIdx.x); u[j] = __float_as_uint(a[j]); w[j] = ((uint64_t)u[j] << 32) | u[j]; }
    __syncthreads();
    const long long t0 = clock64();
    for (int it = 0; it < N; ++it) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (MODE == 0) a[j] = ex2(a[j]);
            if (MODE == 1) u[j] = cvt2(__uint_as_float(u[j]), __uint_as_float(u[(j + 1) & 7]));
            if (MODE == 2) u[j] = prmt(u[j], u[(j + 1) & 7]);
            if (MODE == 3) w[j] = fma2(w[j], w[j], w[(j + 1) & 7]);
            if (MODE == 4) a[j] = fmax3(a[j], a[(j + 1) & 7], a[(j + 2) & 7]);
            if (MODE == 5) { a[j] = ex2(a[j]); u[j] = cvt2(__uint_as_float(u[j]), a[j]); }                     // 1 ex2 + 1 cvt
            if (MODE == 6) { a[j] = ex2(a[j]); u[j] = prmt(u[j], __float_as_uint(a[j])); }                     // 1 ex2 + 1 prmt
            if (MODE == 7) { a[j] = ex2(a[j]); w[j] = fma2(w[j], w[j], w[(j + 1) & 7]); }                      // 1 ex2 + 1 fma2
            if (MODE == 8) { asm volatile("add.rn.f32x2 %0, %0, %1;" : "+l"(w[j]) : "l"(w[(j + 1) & 7])); }
            if (MODE == 9) { a[j] = a[j] * a[(j + 1) & 7] + 1.0f; }
        }
    }
    const long long t1 = clock64();
    float s = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) s += a[j] + __uint_as_float(u[j]) + __uint_as_float((uint32_t)w[j]);
    out[blockIdx.x * blockDim.x + threadIdx.x] = s;
    if ((threadIdx.x & 31) == 0) cyc[threadIdx.x >> 5] = t1 - t0;
}

// wake-up latency: warp 1 waits on an mbarrier, warp 0 arrives after a delay; reports (waiter's clock after the wait) - (arriver's clock at the arrive)
template <int SPIN>
__global__ void wake(long long* res) {
    __shared__ __align__(8) unsigned long long bar[8];
    __shared__ long long t_arr[8];
    const uint32_t b0 = (uint32_t)__cvta_generic_to_shared(bar);
    if (threadIdx.x == 0) {
        for (int i = 0; i < 8; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(b0 + 8 * i));
    }
    __syncthreads();
    for (int r = 0; r < 8; ++r) {
        const uint32_t b = b0 + 8 * r;
        if (threadIdx.x == 0) {
            const long long t = clock64();
            while (clock64() - t < 3000 + 500 * r) {}
            t_arr[r] = clock64();
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(b) : "memory");
        } else if (threadIdx.x == 32) {
            uint32_t ok = 0;
            long long guard = clock64();
            while (!ok && clock64() - guard < 4000000) {
                if (SPIN)
                    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], 0;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(b) : "memory");
                else
                    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0, 20000;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(b) : "memory");
            }
            const long long t = clock64();
            res[r] = t - *(volatile long long*)&t_arr[r];
        }
        __syncthreads();
    }
}

int main() {
    float* out; long long* cyc;
    CHK(cudaMalloc(&out, 1024 * 4)); CHK(cudaMalloc(&cyc, 64 * 8));
    const char* names[] = {"ex2", "cvt.bf16x2", "prmt", "fma.f32x2", "max3", "ex2+cvt", "ex2+prmt", "ex2+fma2", "add.f32x2", "fma.f32"};
    for (int threads : {32, 128, 256}) {
        for (int m = 0; m < 10; ++m) {
            for (int rep = 0; rep < 2; ++rep) {
                switch (m) {
                    case 0: k<0><<<1, threads>>>(out, cyc, 1e-3f); break; case 1: k<1><<<1, threads>>>(out, cyc, 1e-3f); break;
                    case 2: k<2><<<1, threads>>>(out, cyc, 1e-3f); break; case 3: k<3><<<1, threads>>>(out, cyc, 1e-3f); break;
                    case 4: k<4><<<1, threads>>>(out, cyc, 1e-3f); break; case 5: k<5><<<1, threads>>>(out, cyc, 1e-3f); break;
                    case 6: k<6><<<1, threads>>>(out, cyc, 1e-3f); break; case 7: k<7><<<1, threads>>>(out, cyc, 1e-3f); break;
                    case 8: k<8><<<1, threads>>>(out, cyc, 1e-3f); break; case 9: k<9><<<1, threads>>>(out, cyc, 1e-3f); break;
                }
                CHK(cudaDeviceSynchronize());
            }
            long long h[8]; CHK(cudaMemcpy(h, cyc, sizeof(h), cudaMemcpyDeviceToHost));
            const int per = (m >= 5 && m <= 7) ? 2 : 1;
            printf("threads=%3d %-10s cycles per warp-instruction (warp 0): %.2f  (%d instr per element)\n", threads, names[m], (double)h[0] / (N * 8 * per), per);
        }
    }
    long long* res; CHK(cudaMalloc(&res, 8 * 8));
    for (int spin = 0; spin < 2; ++spin) {
        for (int rep = 0; rep < 2; ++rep) { if (spin) wake<1><<<1, 64>>>(res); else wake<0><<<1, 64>>>(res); CHK(cudaDeviceSynchronize()); }
        long long h[8]; CHK(cudaMemcpy(h, res, sizeof(h), cudaMemcpyDeviceToHost));
        printf("%s wake-up latency (cycles):", spin ? "test_wait spin" : "try_wait suspend");
        for (int i = 0; i < 8; ++i) printf(" %lld", h[i]);
        printf("\n");
    }
    return 0;
}
