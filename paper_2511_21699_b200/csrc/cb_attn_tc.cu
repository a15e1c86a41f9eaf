// Tree-masked attention on the 5th-generation tensor cores (tcgen05) with TMA-staged paged K/V.
//
// One CTA handles one (key split, row tile, sequence, kv head).  A row tile packs the GQA group times a
// range of tree nodes into the 128 rows of one MMA tile: row r = node_local * G + g.  Key tiles hold 128
// keys: ceil(ctx/128) tiles of cached keys (eight 16-token pages each, fetched page by page with TMA
// through the block table) followed by one tile with the tree's own keys, masked by the ancestor bits.
//
// Warp roles (192 threads):
//   warp 0      TMA producer: K and V tiles into a ring of 128B-swizzled shared-memory stages
//   warp 1      MMA issuer (one lane): S = Q K^T into a double-buffered TMEM tile, then O += P V with
//               P read from TMEM; owns the TMEM allocation
//   warps 2..5  softmax: one thread per row; S from TMEM to registers, fp32 online softmax in the
//               log2 domain with lazy rescaling of O, P written back to TMEM as packed bf16 over S
// All waits are bounded; a wait that runs out records CB_ERR_TIMEOUT and the CTA drains and exits.
#include <cuda.h>

#include "cb_attn.cuh"

namespace {

constexpr uint32_t kWaitLimit = 1u << 24;
constexpr int kThreads = 192;
constexpr uint32_t kTmemCols = 512;

struct TcMaps { CUtensorMap k_pool, v_pool, k_tree, v_tree; };

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
// Bounded wait. Returns false when the wait ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t* status) {
    for (uint32_t it = 0; it < kWaitLimit; ++it) {
        if (mbar_test(bar, parity)) return true;
        if (it > 64) {
            __nanosleep(40);
            if ((it & 255u) == 0u && *abort_flag) return false;
        }
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

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accum) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accum) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accum) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accum) : "memory");
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
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Shared-memory matrix descriptor, 128-byte swizzle, for tiles whose rows are 128 bytes (64 bf16).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(lbo_bytes >> 4) << 16;
    d |= (uint64_t)(sbo_bytes >> 4) << 32;
    d |= 1ull << 46;
    d |= 2ull << 61;
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, A K-major, B K-major or MN-major.
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}

template <int D>
struct Cfg {
    static constexpr int DB = D / 64;                        // 64-element (128-byte) column blocks per row
    static constexpr int NST = (D == 128) ? 3 : 4;           // K/V stages
    static constexpr uint32_t TILE_BYTES = CB_KT * D * 2;    // one K or V tile
    static constexpr uint32_t Q_BYTES = CB_MT * D * 2;
    static constexpr uint32_t OFF_Q = 0;
    static constexpr uint32_t OFF_K = Q_BYTES;
    static constexpr uint32_t OFF_V = OFF_K + NST * TILE_BYTES;
    static constexpr uint32_t OFF_BAR = OFF_V + NST * TILE_BYTES;
    static constexpr int NBAR = 1 + 3 * NST + 2 + 2 + 1;     // q, k_full, v_full, kv_free, s_full[2], p_ready[2], o_done
    static constexpr uint32_t SMEM = OFF_BAR + NBAR * 8 + 16;
    static constexpr uint32_t SMEM_ALLOC = SMEM + 1024;      // slack to align the base to 1024 bytes
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
cb_attn_tc_kernel(const CbAttnParams p, const __grid_constant__ TcMaps maps) {
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sgen = smem_raw + (sbase - smem_u32(smem_raw));
    const uint32_t bar0 = sbase + C::OFF_BAR;
    const uint32_t bar_q = bar0;
    auto bar_kfull = [&](int s) { return bar0 + 8u * (1 + s); };
    auto bar_vfull = [&](int s) { return bar0 + 8u * (1 + C::NST + s); };
    auto bar_free = [&](int s) { return bar0 + 8u * (1 + 2 * C::NST + s); };
    auto bar_sfull = [&](int s) { return bar0 + 8u * (1 + 3 * C::NST + s); };
    auto bar_pready = [&](int s) { return bar0 + 8u * (3 + 3 * C::NST + s); };
    const uint32_t bar_odone = bar0 + 8u * (5 + 3 * C::NST);
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(sgen + C::OFF_BAR + C::NBAR * 8);
    volatile int* s_abort = reinterpret_cast<volatile int*>(sgen + C::OFF_BAR + C::NBAR * 8 + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int split = blockIdx.x, mt = blockIdx.y, bk = blockIdx.z;
    const int b = bk / p.Hkv, kh = bk % p.Hkv;
    const int n = p.n_nodes[b], ctx = p.ctx_len[b];
    const int nct = (ctx + CB_KT - 1) / CB_KT;               // context tiles; tile nct is the tree tile
    int t_lo, t_hi;
    cb_split_range(ctx, p.nsplit, split, &t_lo, &t_hi);
    const int ntiles = t_hi - t_lo;
    const int RT = p.NPT * p.G;                               // rows of this tile that exist

    // Softmax-thread row bookkeeping (also used by the trivial path)
    const int wq = warp & 3;
    const int row = wq * 32 + lane;
    const int node = mt * p.NPT + row / p.G, g = row % p.G, h = kh * p.G + g;
    const bool row_exists = warp >= 2 && row < RT && node < p.T;
    const bool row_valid = row_exists && node < n;
    const size_t slot = ((size_t)bk * p.MT + mt) * p.nsplit + split;

    if (n <= 0 || ntiles <= 0 || mt * p.NPT >= n) {
        // Nothing to attend from this CTA: zero rows / an empty partial.
        if (warp >= 2) {
            if (p.nsplit == 1) {
                if (row_exists) {
                    uint4* op = reinterpret_cast<uint4*>(p.out + (((size_t)b * p.T + node) * p.Hq + h) * D);
                    for (int c = 0; c < D / 8; ++c) op[c] = make_uint4(0, 0, 0, 0);
                    if (p.lse) p.lse[((size_t)b * p.Hq + h) * p.T + node] = 0.f;
                }
            } else {
                float* pp = p.part + (slot * CB_MT + row) * (D + 4);
                pp[D] = -INFINITY; pp[D + 1] = 0.f;
            }
        }
        return;
    }

    if (tid == 0) {
        mbar_init(bar_q, 128);
        for (int s = 0; s < C::NST; ++s) { mbar_init(bar_kfull(s), 1); mbar_init(bar_vfull(s), 1); mbar_init(bar_free(s), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(bar_sfull(s), 1); mbar_init(bar_pready(s), 128); }
        mbar_init(bar_odone, 1);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *s_tmem;
    const uint32_t tm_S0 = tmem, tm_O = tmem + 256;           // S buffers at columns 0 and 128, O at 256

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        constexpr int NB = 8 * C::DB;                        // boxes (16 keys x 64 dims) per K tile
        const bool active = lane < 2 * NB;
        const bool isV = lane >= NB;
        const int within = lane % NB, j = within % 8, dblk = within / 8;
        const int npages = (ctx + p.P - 1) / p.P;
        for (int it = 0; it < ntiles; ++it) {
            const int tile = t_lo + it, st = it % C::NST;
            if (it >= C::NST) {
                if (!mbar_wait(bar_free(st), ((it / C::NST) - 1) & 1, s_abort, p.status)) break;
            }
            if (lane == 0) { mbar_expect_tx(bar_kfull(st), C::TILE_BYTES); mbar_expect_tx(bar_vfull(st), C::TILE_BYTES); }
            __syncwarp();
            if (active) {
                const uint32_t dst = sbase + (isV ? C::OFF_V : C::OFF_K) + st * C::TILE_BYTES + dblk * (CB_KT * 128) + j * 2048;
                const uint32_t bar = isV ? bar_vfull(st) : bar_kfull(st);
                if (tile < nct) {
                    const int pidx = tile * (CB_KT / 16) + j;
                    // pages past the sequence's end are fetched out of range: the copy fills zeros
                    const int page = pidx < npages ? p.block_table[(size_t)b * p.max_pages + pidx] : p.num_pages;
                    tma_load_4d(dst, isV ? &maps.v_pool : &maps.k_pool, bar, dblk * 64, kh, 0, page);
                } else {
                    tma_load_4d(dst, isV ? &maps.v_tree : &maps.k_tree, bar, dblk * 64, kh, 16 * j, b);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_s = make_idesc(128, CB_KT, false);
            constexpr uint32_t idesc_o = make_idesc(128, D, true);
            bool ok = mbar_wait(bar_q, 0, s_abort, p.status);
            tc_fence_after();
            for (int it = 0; ok && it <= ntiles; ++it) {
                if (it < ntiles) {
                    const int st = it % C::NST, sb = it & 1;
                    if (!(ok = mbar_wait(bar_kfull(st), (it / C::NST) & 1, s_abort, p.status))) break;
                    tc_fence_after();
                    const uint32_t qa = sbase + C::OFF_Q, ka = sbase + C::OFF_K + st * C::TILE_BYTES;
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t off = (kk / 4) * (CB_KT * 128) + (kk % 4) * 32;
                        mma_ss(tm_S0 + sb * 128, make_desc(qa + off, 16, 1024), make_desc(ka + off, 16, 1024), idesc_s, kk > 0);
                    }
                    tc_commit(bar_sfull(sb));
                }
                if (it >= 1) {
                    const int pt = it - 1, st = pt % C::NST, sb = pt & 1;
                    if (!(ok = mbar_wait(bar_vfull(st), (pt / C::NST) & 1, s_abort, p.status))) break;
                    if (!(ok = mbar_wait(bar_pready(sb), (pt >> 1) & 1, s_abort, p.status))) break;
                    tc_fence_after();
                    const uint32_t va = sbase + C::OFF_V + st * C::TILE_BYTES;
#pragma unroll
                    for (int kk = 0; kk < CB_KT / 16; ++kk)
                        mma_ts(tm_O, tm_S0 + sb * 128 + kk * 8, make_desc(va + kk * 2048, CB_KT * 128, 1024), idesc_o,
                               (pt > 0 || kk > 0) ? 1u : 0u);
                    tc_commit(bar_free(st));
                    tc_commit(bar_odone);
                }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ softmax / correction / epilogue
        // Q tile -> shared memory in the 128B-swizzled K-major layout: row r, 16-byte chunk c of column
        // block db lands at db * 16 KB + r * 128 + ((c ^ (r & 7)) * 16).
        {
            constexpr int CPR = C::DB * 8, RPI = 32 / CPR;          // 16-byte chunks per row, rows per iteration
            const int sub = lane / CPR, cc = lane % CPR, db = cc / 8, ch = cc % 8;
            for (int k = 0; k < 32 / RPI; ++k) {
                const int r = wq * 32 + k * RPI + sub;
                const int nd = mt * p.NPT + r / p.G, hh = kh * p.G + r % p.G;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (r < RT && nd < n)
                    v = *reinterpret_cast<const uint4*>(p.q + (((size_t)b * p.T + nd) * p.Hq + hh) * D + db * 64 + ch * 8);
                *reinterpret_cast<uint4*>(sgen + C::OFF_Q + db * (CB_MT * 128) + r * 128 + ((ch ^ (r & 7)) << 4)) = v;
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive(bar_q);

        uint32_t mrow[4] = {0u, 0u, 0u, 0u};
        if (row_valid) for (int k = 0; k < p.W; ++k) mrow[k] = p.tree_mask[((size_t)b * p.T + node) * p.W + k];
        float m_used = -INFINITY, l = 0.f;
        const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
        bool ok = true;
        for (int it = 0; it < ntiles; ++it) {
            const int tile = t_lo + it, sb = it & 1;
            if (!(ok = mbar_wait(bar_sfull(sb), (it >> 1) & 1, s_abort, p.status))) break;
            tc_fence_after();
            uint32_t sr[128];
            const uint32_t ts = tm_S0 + sb * 128 + lane_addr;
            CB_TMEM_LD32(sr, 0, ts);
            CB_TMEM_LD32(sr, 32, ts + 32);
            CB_TMEM_LD32(sr, 64, ts + 64);
            CB_TMEM_LD32(sr, 96, ts + 96);
            tmem_wait_ld();
            const bool is_tree = tile == nct;
            const int kv = is_tree ? n : min(CB_KT, ctx - tile * CB_KT);
            float mloc = -INFINITY;
            if (!row_valid) {
#pragma unroll
                for (int jx = 0; jx < 128; ++jx) sr[jx] = 0xFF800000u;
            } else if (is_tree) {
#pragma unroll
                for (int jx = 0; jx < 128; ++jx) {
                    const bool vis = (mrow[jx >> 5] >> (jx & 31)) & 1u;
                    if (!vis || jx >= kv) sr[jx] = 0xFF800000u;
                    mloc = fmaxf(mloc, __uint_as_float(sr[jx]));
                }
            } else if (kv < CB_KT) {
#pragma unroll
                for (int jx = 0; jx < 128; ++jx) {
                    if (jx >= kv) sr[jx] = 0xFF800000u;
                    mloc = fmaxf(mloc, __uint_as_float(sr[jx]));
                }
            } else {
#pragma unroll
                for (int jx = 0; jx < 128; ++jx) mloc = fmaxf(mloc, __uint_as_float(sr[jx]));
            }
            mloc *= p.scale_log2;
            // lazy rescaling: keep the reference maximum until the running maximum exceeds it by 2^8
            const bool need = mloc > m_used + 8.0f;
            const float alpha = need ? ex2(m_used - mloc) : 1.0f;
            if (need) m_used = mloc;
            if (it > 0) {
                if (!(ok = mbar_wait(bar_odone, (it - 1) & 1, s_abort, p.status))) break;
                tc_fence_after();
                if (__any_sync(CB_FULL, need)) {
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t o[32];
                        CB_TMEM_LD32(o, 0, tm_O + lane_addr + c * 32);
                        tmem_wait_ld();
#pragma unroll
                        for (int jx = 0; jx < 32; ++jx) o[jx] = __float_as_uint(__uint_as_float(o[jx]) * alpha);
                        CB_TMEM_ST32(o, 0, tm_O + lane_addr + c * 32);
                    }
                }
            }
            l *= alpha;
            const float mu = (m_used == -INFINITY) ? 0.f : m_used;
            float l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
            uint32_t pk[64];
#pragma unroll
            for (int jx = 0; jx < 128; jx += 4) {
                const float p0 = ex2(fmaf(__uint_as_float(sr[jx]), p.scale_log2, -mu));
                const float p1 = ex2(fmaf(__uint_as_float(sr[jx + 1]), p.scale_log2, -mu));
                const float p2 = ex2(fmaf(__uint_as_float(sr[jx + 2]), p.scale_log2, -mu));
                const float p3 = ex2(fmaf(__uint_as_float(sr[jx + 3]), p.scale_log2, -mu));
                l0 += p0; l1 += p1; l2 += p2; l3 += p3;
                pk[jx >> 1] = pack_bf16(p0, p1);
                pk[(jx >> 1) + 1] = pack_bf16(p2, p3);
            }
            l += (l0 + l1) + (l2 + l3);
            CB_TMEM_ST32(pk, 0, ts);
            CB_TMEM_ST32(pk, 32, ts + 32);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar_pready(sb));
        }
        if (ok) ok = mbar_wait(bar_odone, (ntiles - 1) & 1, s_abort, p.status);
        tc_fence_after();
        if (ok) {
            if (p.nsplit == 1) {
                const float inv = (row_valid && l > 0.f) ? 1.0f / l : 0.f;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t o[32];
                    CB_TMEM_LD32(o, 0, tm_O + lane_addr + c * 32);
                    tmem_wait_ld();
                    if (row_exists) {
                        uint4* op = reinterpret_cast<uint4*>(p.out + (((size_t)b * p.T + node) * p.Hq + h) * D + c * 32);
#pragma unroll
                        for (int v4 = 0; v4 < 4; ++v4) {
                            uint4 w;
                            w.x = pack_bf16(__uint_as_float(o[v4 * 8 + 0]) * inv, __uint_as_float(o[v4 * 8 + 1]) * inv);
                            w.y = pack_bf16(__uint_as_float(o[v4 * 8 + 2]) * inv, __uint_as_float(o[v4 * 8 + 3]) * inv);
                            w.z = pack_bf16(__uint_as_float(o[v4 * 8 + 4]) * inv, __uint_as_float(o[v4 * 8 + 5]) * inv);
                            w.w = pack_bf16(__uint_as_float(o[v4 * 8 + 6]) * inv, __uint_as_float(o[v4 * 8 + 7]) * inv);
                            op[v4] = w;
                        }
                    }
                }
                if (row_exists && p.lse)
                    p.lse[((size_t)b * p.Hq + h) * p.T + node] = (row_valid && l > 0.f) ? (m_used + log2f(l)) * 0.6931471805599453f : 0.f;
            } else {
                float* pp = p.part + (slot * CB_MT + row) * (D + 4);
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t o[32];
                    CB_TMEM_LD32(o, 0, tm_O + lane_addr + c * 32);
                    tmem_wait_ld();
                    if (row_valid) {
#pragma unroll
                        for (int v4 = 0; v4 < 8; ++v4)
                            *reinterpret_cast<uint4*>(pp + c * 32 + v4 * 4) = make_uint4(o[v4 * 4], o[v4 * 4 + 1], o[v4 * 4 + 2], o[v4 * 4 + 3]);
                    }
                }
                pp[D] = row_valid ? m_used : -INFINITY;
                pp[D + 1] = row_valid ? l : 0.f;
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    if (*s_abort) {
        // give copies that are still in flight time to land before the shared memory is released
        for (int k = 0; k < 64; ++k) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)ptr;
    }
    return fn;
}

// 4-D view (d, kv head, row, block) of a [blocks, rows, Hkv, D] bf16 tensor; box = 64 dims x 1 head x 16 rows.
bool encode_kv_map(CUtensorMap* m, const void* base, int D, int Hkv, int rows, long blocks) {
    EncodeTiledFn enc = get_encode();
    if (!enc) { fprintf(stderr, "cacheback: cuTensorMapEncodeTiled entry point not found\n"); return false; }
    cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)Hkv, (cuuint64_t)rows, (cuuint64_t)blocks};
    cuuint64_t strides[3] = {(cuuint64_t)D * 2, (cuuint64_t)Hkv * D * 2, (cuuint64_t)rows * Hkv * D * 2};
    cuuint32_t box[4] = {64, 1, 16, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        fprintf(stderr, "cacheback: tensor map encode failed (%d): D=%d Hkv=%d rows=%d blocks=%ld base=%p\n", (int)r, D, Hkv, rows,
                blocks, base);
    return r == CUDA_SUCCESS;
}

template <int D>
cb_status launch(const CbAttnParams& p, const TcMaps& maps, cudaStream_t st) {
    static bool attr_set = false;
    if (!attr_set) {
        CB_CUDA(cudaFuncSetAttribute(cb_attn_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<D>::SMEM_ALLOC));
        attr_set = true;
    }
    dim3 grid(p.nsplit, p.MT, p.B * p.Hkv);
    cb_attn_tc_kernel<D><<<grid, kThreads, Cfg<D>::SMEM_ALLOC, st>>>(p, maps);
    cb_count_launch(1);
    CB_CUDA(cudaGetLastError());
    return CB_OK;
}

}  // namespace

cb_status cb_attn_launch_tensor(cb_ctx* ctx, const CbAttnParams& p, cudaStream_t st) {
    (void)ctx;
    if (p.P != 16) return CB_ERR_UNSUPPORTED;
    TcMaps maps;
    if (!encode_kv_map(&maps.k_pool, p.k_pool, p.D, p.Hkv, p.P, p.num_pages)) return CB_ERR_CUDA;
    if (!encode_kv_map(&maps.v_pool, p.v_pool, p.D, p.Hkv, p.P, p.num_pages)) return CB_ERR_CUDA;
    if (!encode_kv_map(&maps.k_tree, p.k_tree, p.D, p.Hkv, p.T, p.B)) return CB_ERR_CUDA;
    if (!encode_kv_map(&maps.v_tree, p.v_tree, p.D, p.Hkv, p.T, p.B)) return CB_ERR_CUDA;
    return p.D == 128 ? launch<128>(p, maps, st) : launch<64>(p, maps, st);
}
