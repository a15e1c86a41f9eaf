// Microbenchmark behind the figures the design doc quotes for the tensor-core side of tree attention.
//
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -o mma_issue mma_issue.cu && ./mma_issue
//
// Throughput of tcgen05.mma blocks as the attention kernels issue them: time to issue n MMAs (128x128x16 per SM, bf16) and
// time until their commit completes, for cta_group::1 and for a pair of CTAs with cta_group::2; also 128xNx16 with N = 64
// and N = 256 (cta_group::1, both operands from shared memory).  Operands are whatever
// shared memory holds (zeroed); only timing matters.
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#define CHK(x) do { cudaError_t e = (x); if (e != cudaSuccess) { printf("CUDA %s at %d\n", cudaGetErrorString(e), __LINE__); return 1; } } while (0)
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t clk() { uint32_t c; asm volatile("mov.u32 %0, %%clock;" : "=r"(c)); return c; }
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t desc_lo(uint32_t saddr, uint32_t lbo) { return ((saddr & 0x3FFFFu) >> 4) | ((lbo >> 4) << 16); }
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, bool b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
template <int CG>
__device__ __forceinline__ void mma_ss(uint32_t d, uint32_t alo, uint32_t blo, uint32_t idesc, uint32_t acc) {
    if (CG == 1)
        asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.u32 p, %5, 0;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                     "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}" ::"r"(d), "r"(alo), "r"(blo), "r"(kDescHi), "r"(idesc), "r"(acc) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.u32 p, %5, 0;\n\tmov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                     "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, p;\n\t}" ::"r"(d), "r"(alo), "r"(blo), "r"(kDescHi), "r"(idesc), "r"(acc) : "memory");
}
template <int CG>
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a_tmem, uint32_t blo, uint32_t idesc, uint32_t acc) {
    if (CG == 1)
        asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 db;\n\tsetp.ne.u32 p, %5, 0;\n\tmov.b64 db, {%2, %3};\n\t"
                     "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}" ::"r"(d), "r"(a_tmem), "r"(blo), "r"(kDescHi), "r"(idesc), "r"(acc) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 db;\n\tsetp.ne.u32 p, %5, 0;\n\tmov.b64 db, {%2, %3};\n\t"
                     "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], db, %4, p;\n\t}" ::"r"(d), "r"(a_tmem), "r"(blo), "r"(kDescHi), "r"(idesc), "r"(acc) : "memory");
}

// res[0..]: per repetition (issue cycles, cycles until the commit's barrier completed)
template <int CG, int TS, int NN = 128>
__global__ void __launch_bounds__(128, 1) k(long long* res, int n_mma, int reps) {
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ __align__(8) unsigned long long bar;
    __shared__ uint32_t s_tmem;
    const uint32_t sbase = (smem_u32(smem) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint32_t rank = 0;
    if (CG == 2) asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    for (int i = threadIdx.x; i < (NN > 128 ? 112 : 64) * 1024 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem + (sbase - smem_u32(smem)))[i] = 0u;
    if (warp == 0) {
        if (CG == 1) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&s_tmem)) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&s_tmem)) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        }
    }
    if (threadIdx.x == 32) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (CG == 2) { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s_tmem;
    if (warp == 1 && lane == 0 && rank == 0) {
        const uint32_t idesc = TS ? make_idesc(128 * CG, NN, true) : make_idesc(128 * CG, NN, false);
        const uint32_t alo = desc_lo(sbase, 16), blo = desc_lo(sbase + 32768, TS ? 16384 : 16);
        const uint32_t b = smem_u32(&bar);
        for (int r = 0; r < reps; ++r) {
            const uint32_t t0 = clk();
            for (int m = 0; m < n_mma; ++m) {
                const int ks = m & 7;
                if (TS) mma_ts<CG>(tmem + 256, tmem + (m & 8 ? 128 : 0) + 8 * ks, blo + 128 * ks, idesc, 1u);
                else mma_ss<CG>(tmem + ((m >> 3) & 1) * 128, alo + (ks < 4 ? 2 * ks : 1024 + 2 * (ks - 4)), blo + (ks < 4 ? 2 * ks : (CG == 2 ? 512 : 1024) + 2 * (ks - 4)), idesc, ks ? 1u : 0u);
            }
            const uint32_t t1 = clk();
            if (CG == 1) asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(b) : "memory");
            else asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(b) : "memory");
            const uint32_t t2 = clk();
            uint32_t ok = 0;
            const uint32_t guard = clk();
            while (!ok && clk() - guard < 4000000u)
                asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(b), "r"((uint32_t)(r & 1)) : "memory");
            const uint32_t t3 = clk();
            res[r * 3 + 0] = t1 - t0; res[r * 3 + 1] = t2 - t1; res[r * 3 + 2] = t3 - t0;
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (CG == 2) { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
    if (warp == 0) {
        if (CG == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    }
}

template <int CG, int TS, int NN = 128>
int run(long long* res, const char* name) {
    const int smem = (NN > 128 ? 112 : 64) * 1024 + 1024 + 1024;   // B of N = 256: two 32 KB blocks from offset 32 KB and 48 KB
    CHK(cudaFuncSetAttribute(k<CG, TS, NN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    for (int n : {1, 8, 16, 64}) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(CG); cfg.blockDim = dim3(128); cfg.dynamicSmemBytes = smem;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension; at[0].val.clusterDim.x = CG; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        CHK(cudaLaunchKernelEx(&cfg, k<CG, TS, NN>, res, n, 4));
        CHK(cudaDeviceSynchronize());
        long long h[12]; CHK(cudaMemcpy(h, res, sizeof(h), cudaMemcpyDeviceToHost));
        printf("%-28s n=%2d  issue %lld  commit %lld  until complete %lld cycles  (last of 4 repetitions; %.1f cycles per MMA)\n", name, n, h[9], h[10], h[11],
               (double)h[11] / n);
    }
    return 0;
}

int main() {
    long long* res; CHK(cudaMalloc(&res, 64 * 8));
    if (run<1, 0>(res, "cta_group::1 SS (Q K^T)")) return 1;
    if (run<1, 1>(res, "cta_group::1 TS (P V)")) return 1;
    if (run<1, 0, 64>(res, "cta_group::1 SS, N = 64")) return 1;
    if (run<1, 0, 256>(res, "cta_group::1 SS, N = 256")) return 1;
    if (run<2, 0>(res, "cta_group::2 SS (Q K^T)")) return 1;
    if (run<2, 1>(res, "cta_group::2 TS (P V)")) return 1;
    return 0;
}
