// Device-side building blocks of the tensor-core attention kernels: bounded mbarrier waits, TMA loads, tcgen05 fences,
// TMEM loads and stores, packed fp32 arithmetic, and the shared-memory / instruction descriptors of tcgen05.mma.
// Included by cb_attn_tc.cu only (one translation unit holds both attention kernels and their launcher).
#pragma once
#include <cuda.h>

#include "cb_attn.cuh"

namespace {

constexpr long long kWaitCycles = 1ll << 32;     // bound of every wait, in SM clock cycles (about two seconds)
constexpr uint32_t kSuspendNs = 20000;
constexpr float kRowSumLimit = 1048576.f;        // a tile's row sum of P above which the row takes a new reference maximum
constexpr int kThreads = 384;
constexpr uint32_t kTmemCols = 512;

struct TcMaps { CUtensorMap k_pool, v_pool, k_tree, v_tree, q; };

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_n(uint32_t bar, uint32_t n) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(n) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Potentially blocking test of a barrier phase: the hardware suspends the thread until the phase completes
// or a time limit of about kSuspendNs passes, so waiting warps do not take issue slots from working ones.
__device__ __forceinline__ uint32_t mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(kSuspendNs) : "memory");
    return ok;
}
// Bounded wait. Returns false when the wait ran out or another role already gave up; the first to run out
// records CB_ERR_TIMEOUT and raises the CTA's abort flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t* status) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitCycles) break;
    }
    *abort_flag = 1;
    atomicCAS(status, 0u, (uint32_t)CB_ERR_TIMEOUT);
    return false;
}

// Cluster-scope helpers: address of a shared-memory location in another CTA of the cluster, arrival on a barrier there
// (releasing this thread's earlier writes to the cluster), a 16-byte store there, and a bounded wait that acquires them.
__device__ __forceinline__ uint32_t cluster_addr(uint32_t local, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t remote_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
}
__device__ __forceinline__ void st_cluster_v4(uint32_t raddr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(raddr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(kSuspendNs) : "memory");
    return ok;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t* status) {
    if (mbar_try_cluster(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try_cluster(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitCycles) break;
    }
    *abort_flag = 1;
    atomicCAS(status, 0u, (uint32_t)CB_ERR_TIMEOUT);
    return false;
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

// The cached context is read once per call: its copies are marked as the first to leave L2, so that what the other kernels
// of a step keep coming back to (the n-gram tables) is still there after 100 MB of keys and values have passed through.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void tma_load_4d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3, uint64_t pol) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cta.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(pol) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
#define CB_R32(a, o) "=r"(a[o + 0]), "=r"(a[o + 1]), "=r"(a[o + 2]), "=r"(a[o + 3]), "=r"(a[o + 4]), "=r"(a[o + 5]), \
    "=r"(a[o + 6]), "=r"(a[o + 7]), "=r"(a[o + 8]), "=r"(a[o + 9]), "=r"(a[o + 10]), "=r"(a[o + 11]), "=r"(a[o + 12]), \
    "=r"(a[o + 13]), "=r"(a[o + 14]), "=r"(a[o + 15]), "=r"(a[o + 16]), "=r"(a[o + 17]), "=r"(a[o + 18]), "=r"(a[o + 19]), \
    "=r"(a[o + 20]), "=r"(a[o + 21]), "=r"(a[o + 22]), "=r"(a[o + 23]), "=r"(a[o + 24]), "=r"(a[o + 25]), "=r"(a[o + 26]), \
    "=r"(a[o + 27]), "=r"(a[o + 28]), "=r"(a[o + 29]), "=r"(a[o + 30]), "=r"(a[o + 31])
#define CB_W32(a, o) "r"(a[o + 0]), "r"(a[o + 1]), "r"(a[o + 2]), "r"(a[o + 3]), "r"(a[o + 4]), "r"(a[o + 5]), \
    "r"(a[o + 6]), "r"(a[o + 7]), "r"(a[o + 8]), "r"(a[o + 9]), "r"(a[o + 10]), "r"(a[o + 11]), "r"(a[o + 12]), \
    "r"(a[o + 13]), "r"(a[o + 14]), "r"(a[o + 15]), "r"(a[o + 16]), "r"(a[o + 17]), "r"(a[o + 18]), "r"(a[o + 19]), \
    "r"(a[o + 20]), "r"(a[o + 21]), "r"(a[o + 22]), "r"(a[o + 23]), "r"(a[o + 24]), "r"(a[o + 25]), "r"(a[o + 26]), \
    "r"(a[o + 27]), "r"(a[o + 28]), "r"(a[o + 29]), "r"(a[o + 30]), "r"(a[o + 31])

// 32 consecutive 32-bit columns of this thread's TMEM lane -> registers a[o .. o+32)
#define CB_TMEM_LD32(a, o, taddr)                                                                                    \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, "   \
                 "%13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, "  \
                 "[%32];" : CB_R32(a, o) : "r"(taddr) : "memory")
#define CB_TMEM_ST32(a, o, taddr)                                                                                    \
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, " \
                 "%12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, "   \
                 "%31};" ::CB_W32(a, o), "r"(taddr) : "memory")
#define CB_RW32(a) "+r"(a[0]), "+r"(a[1]), "+r"(a[2]), "+r"(a[3]), "+r"(a[4]), "+r"(a[5]), "+r"(a[6]), "+r"(a[7]), "+r"(a[8]), \
    "+r"(a[9]), "+r"(a[10]), "+r"(a[11]), "+r"(a[12]), "+r"(a[13]), "+r"(a[14]), "+r"(a[15]), "+r"(a[16]), "+r"(a[17]), "+r"(a[18]), \
    "+r"(a[19]), "+r"(a[20]), "+r"(a[21]), "+r"(a[22]), "+r"(a[23]), "+r"(a[24]), "+r"(a[25]), "+r"(a[26]), "+r"(a[27]), "+r"(a[28]), \
    "+r"(a[29]), "+r"(a[30]), "+r"(a[31])
// Waits for this thread's outstanding TMEM loads; naming the destination registers keeps their uses below the wait.
#define CB_TMEM_WAIT_LD32(a) asm volatile("tcgen05.wait::ld.sync.aligned;" : CB_RW32(a) :: "memory")
#define CB_TMEM_LD16(a, taddr)                                                                                       \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, "   \
                 "%13, %14, %15}, [%16];" : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3]), "=r"(a[4]), "=r"(a[5]),  \
                 "=r"(a[6]), "=r"(a[7]), "=r"(a[8]), "=r"(a[9]), "=r"(a[10]), "=r"(a[11]), "=r"(a[12]), "=r"(a[13]), \
                 "=r"(a[14]), "=r"(a[15]) : "r"(taddr) : "memory")
#define CB_TMEM_ST16(a, o, taddr)                                                                                    \
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, " \
                 "%12, %13, %14, %15};" ::"r"(a[o + 0]), "r"(a[o + 1]), "r"(a[o + 2]), "r"(a[o + 3]), "r"(a[o + 4]),  \
                 "r"(a[o + 5]), "r"(a[o + 6]), "r"(a[o + 7]), "r"(a[o + 8]), "r"(a[o + 9]), "r"(a[o + 10]),           \
                 "r"(a[o + 11]), "r"(a[o + 12]), "r"(a[o + 13]), "r"(a[o + 14]), "r"(a[o + 15]), "r"(taddr) : "memory")
// 32-byte store: one instruction fills a whole DRAM sector of this thread's output row
__device__ __forceinline__ void st_global_v8(void* ptr, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t a4, uint32_t a5, uint32_t a6,
                                             uint32_t a7) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(ptr), "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(a4), "r"(a5), "r"(a6),
                 "r"(a7) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Two fp32 values in one 64-bit register pair, for the packed fp32x2 arithmetic of sm_100.
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f2_unpack(uint64_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Instruction descriptor: bf16 x bf16 -> fp32, A K-major, B K-major or MN-major.
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}

// Low and high 32-bit words of a shared-memory matrix descriptor (128-byte swizzle, 1024-byte stride between
// 8-row groups).  All operands live below 256 KB, so stepping the low word by (bytes >> 4) moves the start address.
__device__ __forceinline__ uint32_t desc_lo(uint32_t saddr, uint32_t lbo_bytes) { return ((saddr & 0x3FFFFu) >> 4) | ((lbo_bytes >> 4) << 16); }
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);

// One MMA issuer thread feeds the tensor pipe, so the instructions between two MMAs are kept to a minimum: each
// of the blocks below issues all MMAs of one 128 x 128 x D (or 128 x D x 128) product from a single asm statement.
#define CB_MMA_SS_STEP(OFF)                                                                                          \
    "add.u32 ra, %1, " #OFF ";\n\tadd.u32 rb, %2, " #OFF ";\n\tmov.b64 da, {ra, %3};\n\tmov.b64 db, {rb, %3};\n\t"  \
    "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pt;\n\t"
// S[tmem] = Q[smem, K-major] * K[smem, K-major]^T over D.  qlo / klo: low descriptor words of the first 16-wide slice.
template <int D>
__device__ __forceinline__ void mma_s_block(uint32_t d_tmem, uint32_t qlo, uint32_t klo, uint32_t idesc) {
    if (D == 128) {
        asm volatile(
            "{\n\t.reg .pred pt, pf;\n\t.reg .b64 da, db;\n\t.reg .b32 ra, rb;\n\t"
            "setp.eq.u32 pt, %4, %4;\n\tsetp.ne.u32 pf, %4, %4;\n\t"
            "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pf;\n\t"
            CB_MMA_SS_STEP(2) CB_MMA_SS_STEP(4) CB_MMA_SS_STEP(6) CB_MMA_SS_STEP(1024) CB_MMA_SS_STEP(1026) CB_MMA_SS_STEP(1028)
            CB_MMA_SS_STEP(1030) "}"
            ::"r"(d_tmem), "r"(qlo), "r"(klo), "r"(kDescHi), "r"(idesc) : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred pt, pf;\n\t.reg .b64 da, db;\n\t.reg .b32 ra, rb;\n\t"
            "setp.eq.u32 pt, %4, %4;\n\tsetp.ne.u32 pf, %4, %4;\n\t"
            "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, pf;\n\t"
            CB_MMA_SS_STEP(2) CB_MMA_SS_STEP(4) CB_MMA_SS_STEP(6) "}"
            ::"r"(d_tmem), "r"(qlo), "r"(klo), "r"(kDescHi), "r"(idesc) : "memory");
    }
}
#define CB_MMA_TS_STEP(K)                                                                                            \
    "add.u32 ra, %1, 8 * " #K ";\n\tadd.u32 rb, %2, 128 * " #K ";\n\tmov.b64 db, {rb, %3};\n\t"                     \
    "tcgen05.mma.cta_group::1.kind::f16 [%0], [ra], db, %4, pt;\n\t"
// O[tmem] (+)= P[tmem, packed bf16] * V[smem, MN-major] over the tile's 128 keys.  vlo: low descriptor word of the V tile.
__device__ __forceinline__ void mma_pv_block(uint32_t d_tmem, uint32_t p_tmem, uint32_t vlo, uint32_t idesc, uint32_t accum) {
    asm volatile(
        "{\n\t.reg .pred pt, pa;\n\t.reg .b64 db;\n\t.reg .b32 ra, rb;\n\t"
        "setp.eq.u32 pt, %4, %4;\n\tsetp.ne.u32 pa, %5, 0;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, pa;\n\t"
        CB_MMA_TS_STEP(1) CB_MMA_TS_STEP(2) CB_MMA_TS_STEP(3) CB_MMA_TS_STEP(4) CB_MMA_TS_STEP(5) CB_MMA_TS_STEP(6) CB_MMA_TS_STEP(7) "}"
        ::"r"(d_tmem), "r"(p_tmem), "r"(vlo), "r"(kDescHi), "r"(idesc), "r"(accum) : "memory");
}

template <int REGS> __device__ __forceinline__ void reg_dealloc() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS)); }
template <int REGS> __device__ __forceinline__ void reg_alloc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS)); }
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

}  // namespace
