// Tree-masked attention for launches whose trees need two or more 128-row query tiles (GQA groups, large trees): the
// tensor-bound shapes.  Two CTAs on two SMs form a pair (a thread-block cluster of 2) and issue their products as one
// tcgen05.mma.cta_group::2: the pair works on one unit (sequence, kv head, row group), CTA r holds row tile r of the
// group, and every K or V tile is split between the two: each CTA fetches only its half with its own TMA copies (keys
// [64 r, 64 r + 64) of a K tile, head dimensions [64 r, 64 r + 64) of a V tile) and the tensor cores of both read both
// halves.  No copy is multicast.  Per CTA that halves the shared-memory traffic of the score product, which otherwise is
// what bounds it, and with one row tile per CTA TMEM has room to double-buffer S (S0, S1, O: 384 columns): the scores of
// key tile i + 1 are produced while tile i is in softmax, so the softmax never waits for the tensor pipe and the tensor
// pipe only for the P it needs next.  Softmax is the longer of the two, and a single warp per SM sub-partition leaves
// most of its issue slots empty (dependent instructions, the exponential unit's occupancy), so two warpgroups work on
// every score tile together: thread (warpgroup w, row r) takes row r and key columns [64 w, 64 w + 64), and the row's two
// threads share one reference maximum.
//
// Warp roles (384 threads per CTA):
//   warp 0        TMA producer of this CTA's halves of the K/V tiles (ring of key-tile slots, K half + V half each)
//   warp 1        owns the pair's TMEM allocation; in the leader CTA (rank 0) one lane issues all products of the pair:
//                 S(i) = Q K(i)^T into S[i & 1], then O += P(i - 1) V(i - 1) with P read from TMEM
//   warp 2        TMA loads of this CTA's query tile; zero rows of padding nodes
//   warps 4..11   softmax: two warpgroups, thread (w, r) = row r, key columns [64 w, 64 w + 64) of every tile; S from TMEM,
//                 fp32 online softmax in the log2 domain, P written back over the scores it read as packed bf16;
//                 epilogue of the unit (each warpgroup writes half of the output columns)
// Barriers the issuer waits on live in the leader CTA (TMA completions of both CTAs, "P ready" and "O read" arrivals of
// both CTAs' softmax warps); completions of the tensor core's work are committed to both CTAs' copies of a barrier at
// once.  All waits are bounded; the pair leaves together through the hardware cluster barrier.
//
// Included by cb_attn_tc.cu.
#pragma once
#include "cb_tc_dev.cuh"

namespace {

constexpr int kPairThreads = 384;

struct PairCfg {
    static constexpr int D = 128;
    static constexpr int DB = 2;                                 // 64-element (128-byte) column blocks per row
    static constexpr uint32_t HALF_BYTES = 64 * D * 2;           // half a K tile (64 keys x D) = half a V tile (128 keys x D / 2)
    static constexpr uint32_t SLOT_BYTES = 2 * HALF_BYTES;       // one ring slot: this CTA's halves of the K and V tile of one key tile
    static constexpr uint32_t Q_BYTES = CB_MT * D * 2;
    static constexpr int NSLOT = 5;
    static constexpr uint32_t OFF_Q = 0;
    static constexpr uint32_t OFF_RING = Q_BYTES;
    static constexpr uint32_t OFF_BAR = OFF_RING + NSLOT * SLOT_BYTES;
    // slot_full[NSLOT], slot_free[NSLOT], q_full, q_free, s_full[2], p_ready[2], o_full, o_free, pair[4]
    static constexpr int NBAR = 2 * NSLOT + 12;
    static constexpr uint32_t OFF_MISC = OFF_BAR + NBAR * 8;     // schedule, tmem base, abort flag, pair flags
    static constexpr uint32_t OFF_XCHG = OFF_MISC + 112;         // [2 warpgroups][128 rows] floats passed between a row's two threads
    static constexpr uint32_t SMEM = OFF_XCHG + 2 * CB_MT * 4;
    static constexpr uint32_t SMEM_ALLOC = SMEM + 1024;          // slack to align the base to 1024 bytes
    static constexpr uint32_t O_COL = 256;                       // TMEM columns: S0 at 0, S1 at 128, O at 256
};
static_assert(PairCfg::SMEM_ALLOC <= 227 * 1024, "shared memory of a pair CTA");

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void mbar_expect_tx_only(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// TMA copies of a CTA pair: the destination is this CTA's shared memory, the completion is counted on a barrier that may
// live in the other CTA of the pair (the leader's).
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int c0, int c1, int c2, int c3,
                                                      uint64_t pol) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
        ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(pol) : "memory");
}
// Arrival on a barrier of the pair's other CTA that carries no data in shared or global memory with it (what it signals was
// written to TMEM and ordered by the tcgen05 fences around it), hence with the default CTA-scope semantics: a release at
// cluster scope would make every arrival wait for the thread's earlier memory traffic to become visible to the whole pair.
__device__ __forceinline__ void mbar_arrive_peer(uint32_t remote_bar) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
}
// Completion of all products issued so far, signalled on the same barrier in both CTAs of the pair.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar), "h"((uint16_t)3)
                 : "memory");
}

#define CB_MMA2_SS_STEP(AOFF, BOFF)                                                                                  \
    "add.u32 ra, %1, " #AOFF ";\n\tadd.u32 rb, %2, " #BOFF ";\n\tmov.b64 da, {ra, %3};\n\tmov.b64 db, {rb, %3};\n\t" \
    "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, pt;\n\t"
// S[tmem of both CTAs] = Q[each CTA's 128 rows, K-major] * K[64 keys in each CTA, K-major]^T over D = 128.
// qlo / klo: low descriptor words of the first 16-wide slice; the second 64-element block of Q lies 16 KB further, that
// of the K half 8 KB further.
__device__ __forceinline__ void mma2_s_block(uint32_t d_tmem, uint32_t qlo, uint32_t klo, uint32_t idesc) {
    asm volatile(
        "{\n\t.reg .pred pt, pf;\n\t.reg .b64 da, db;\n\t.reg .b32 ra, rb;\n\t"
        "setp.eq.u32 pt, %4, %4;\n\tsetp.ne.u32 pf, %4, %4;\n\t"
        "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, pf;\n\t"
        CB_MMA2_SS_STEP(2, 2) CB_MMA2_SS_STEP(4, 4) CB_MMA2_SS_STEP(6, 6) CB_MMA2_SS_STEP(1024, 512) CB_MMA2_SS_STEP(1026, 514)
        CB_MMA2_SS_STEP(1028, 516) CB_MMA2_SS_STEP(1030, 518) "}"
        ::"r"(d_tmem), "r"(qlo), "r"(klo), "r"(kDescHi), "r"(idesc) : "memory");
}
#define CB_MMA2_TS_STEP(K, PCOL)                                                                                     \
    "add.u32 ra, %1, " #PCOL ";\n\tadd.u32 rb, %2, 128 * " #K ";\n\tmov.b64 db, {rb, %3};\n\t"                      \
    "tcgen05.mma.cta_group::2.kind::f16 [%0], [ra], db, %4, pt;\n\t"
// O[tmem of both CTAs] (+)= P[each CTA's TMEM, packed bf16] * V[64 head dimensions in each CTA, MN-major] over the tile's 128 keys.
// P of keys 0..63 is packed into columns 0..31 of the S buffer and P of keys 64..127 into columns 64..95: each half is
// written by the softmax warpgroup that read the scores it replaces.
__device__ __forceinline__ void mma2_pv_block(uint32_t d_tmem, uint32_t p_tmem, uint32_t vlo, uint32_t idesc, uint32_t accum) {
    asm volatile(
        "{\n\t.reg .pred pt, pa;\n\t.reg .b64 db;\n\t.reg .b32 ra, rb;\n\t"
        "setp.eq.u32 pt, %4, %4;\n\tsetp.ne.u32 pa, %5, 0;\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], db, %4, pa;\n\t"
        CB_MMA2_TS_STEP(1, 8) CB_MMA2_TS_STEP(2, 16) CB_MMA2_TS_STEP(3, 24) CB_MMA2_TS_STEP(4, 64) CB_MMA2_TS_STEP(5, 72) CB_MMA2_TS_STEP(6, 80)
        CB_MMA2_TS_STEP(7, 88) "}"
        ::"r"(d_tmem), "r"(p_tmem), "r"(vlo), "r"(kDescHi), "r"(idesc), "r"(accum) : "memory");
}

// The rare step of the online softmax: a row moves to a new reference, so what was accumulated against the old one is
// multiplied by alpha = 2^(old - new): here n_chunks 16-column chunks of the row's accumulator, starting at tm_O.  Kept out
// of line: it runs for a few tiles per unit at most.
__device__ __noinline__ void rescale_row(uint32_t tm_O, int n_chunks, float alpha) {
    for (int ox = 0; ox < n_chunks; ++ox) {
        uint32_t o[16];
        CB_TMEM_LD16(o, tm_O + ox * 16);
        tmem_wait_ld();
#pragma unroll
        for (int jx = 0; jx < 16; ++jx) o[jx] = __float_as_uint(__uint_as_float(o[jx]) * alpha);
        CB_TMEM_ST16(o, 0, tm_O + ox * 16);
    }
    tmem_wait_st();
}

__global__ void __launch_bounds__(kPairThreads, 1)
cb_attn_pair_kernel(const CbAttnParams p, const __grid_constant__ TcMaps maps) {
    using C = PairCfg;
    constexpr int D = C::D;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sgen = smem_raw + (sbase - smem_u32(smem_raw));
    const uint32_t bar0 = sbase + C::OFF_BAR;
    auto bar_full = [&](int s) { return bar0 + 8u * s; };
    auto bar_free = [&](int s) { return bar0 + 8u * (C::NSLOT + s); };
    const uint32_t bar_qfull = bar0 + 8u * (2 * C::NSLOT), bar_qfree = bar_qfull + 8u;
    auto bar_sfull = [&](int s) { return bar0 + 8u * (2 * C::NSLOT + 2 + s); };
    auto bar_pready = [&](int s) { return bar0 + 8u * (2 * C::NSLOT + 4 + s); };
    const uint32_t bar_ofull = bar0 + 8u * (2 * C::NSLOT + 6), bar_ofree = bar_ofull + 8u;
    const uint32_t bar_pair0 = bar_ofree + 8u;                  // one per TMEM lane quarter: the two softmax warps that share 32 rows
    SchedSmem* s_sched = reinterpret_cast<SchedSmem*>(sgen + C::OFF_MISC);
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(sgen + C::OFF_MISC + 64);
    volatile int* s_abort = reinterpret_cast<volatile int*>(sgen + C::OFF_MISC + 68);
    volatile uint32_t* s_over = reinterpret_cast<volatile uint32_t*>(sgen + C::OFF_MISC + 72);   // [4 quarters][2]
    volatile float* s_xchg = reinterpret_cast<volatile float*>(sgen + C::OFF_XCHG);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();                    // 0: the leader, whose barriers the issuer waits on
    const int pair = blockIdx.x >> 1;
    const int RT = p.NPT * p.G;                                 // rows of a row tile that exist
    // Set-up that reads no input runs before the wait for the kernels earlier in the stream.
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else if (warp == 2 && lane == 0) {
        for (int s = 0; s < C::NSLOT; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_free(s), 1); }
        mbar_init(bar_qfull, 1); mbar_init(bar_qfree, 1);
        for (int s = 0; s < 2; ++s) { mbar_init(bar_sfull(s), 1); mbar_init(bar_pready(s), 16); }   // one arrival per softmax warp of both CTAs
        mbar_init(bar_ofull, 1); mbar_init(bar_ofree, 16);
        for (int s = 0; s < 4; ++s) { mbar_init(bar_pair0 + 8u * s, 64); s_over[2 * s] = 0u; s_over[2 * s + 1] = 0u; }
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tma_prefetch_desc(&maps.k_pool); tma_prefetch_desc(&maps.v_pool); tma_prefetch_desc(&maps.q);
        tma_prefetch_desc(&maps.k_tree); tma_prefetch_desc(&maps.v_tree);
    }
    CB_PDL_ENTRY();
    if (warp == 0) {
        // this pair's range of the global tile sequence
        const long long tot = cb_sched_total(p, lane);
        const long long g0 = cb_range_start(tot, p.nc, pair), g1 = cb_range_start(tot, p.nc, pair + 1);
        int b0 = 0, rg0 = 0;
        long long pre0 = 0;
        if (g0 < g1) cb_sched_locate(p, g0, lane, &rg0, &b0, &pre0);
        if (lane == 0) { s_sched->g0 = g0; s_sched->g1 = g1; s_sched->b0 = b0; s_sched->rg0 = rg0; s_sched->pre0 = pre0; }
    }
    tc_fence_before();
    __syncthreads();
    // the peer's barriers must exist before anything arrives on them
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    tc_fence_after();
    const uint32_t tmem = *s_tmem;
    CbWalker wk;
    wk.init(p, s_sched->g0, s_sched->g1, s_sched->rg0, s_sched->b0, s_sched->pre0);
    CbUnit u;

    if (warp == 0) {
        // ---------------------------------------------------------------------- K/V producer: this CTA's halves
        // lanes 0..7: the K half (keys 64 rank .. 64 rank + 63: four pages, two 64-dim blocks); lanes 8..15: the V half (all
        // eight pages of the tile, 64-dim block `rank`)
        const bool active = lane < 16, isV = lane >= 8;
        const int j = isV ? lane - 8 : (lane & 3);              // page of the tile (V) or of this CTA's half (K)
        const int dblk = isV ? (int)rank : (lane >> 2);
        const int pg_in_tile = isV ? j : (int)rank * 4 + j;
        const uint32_t dst_off = isV ? C::HALF_BYTES + (uint32_t)j * 2048u : (uint32_t)dblk * 8192u + (uint32_t)j * 2048u;
        uint32_t c = 0;
        bool ok = true;
        const uint64_t pol = l2_evict_first_policy();
        while (ok && wk.next(p, &u)) {
            const int npages = (u.ctx + p.P - 1) / p.P, nct = u.tiles - 1;
            const int32_t* bt = p.block_table + (size_t)u.b * p.max_pages;
            for (int i = u.t0; i < u.t1; ++i, ++c) {
                int page = p.num_pages;                          // out of range: the copy fills zeros
                if (active && i < nct) {
                    const int pidx = i * (CB_KT / 16) + pg_in_tile;
                    if (pidx < npages) {
                        page = bt[pidx];
                        if (!cb_dbg_in(page, p.num_pages, p.status)) page = p.num_pages;   // the copy then fills zeros
                    }
                }
                const uint32_t slot = c % C::NSLOT;
                if (c >= (uint32_t)C::NSLOT && !(ok = mbar_wait(bar_free(slot), (c / C::NSLOT - 1) & 1, s_abort, p.status))) break;
                if (rank == 0 && lane == 0) mbar_expect_tx_only(bar_full(slot), 2 * C::SLOT_BYTES);   // both CTAs' halves
                __syncwarp();
                if (active) {
                    const uint32_t dst = sbase + C::OFF_RING + slot * C::SLOT_BYTES + dst_off;
                    const uint32_t lbar = cluster_addr(bar_full(slot), 0);
                    if (i < nct) tma_load_4d_pair_hint(dst, isV ? &maps.v_pool : &maps.k_pool, lbar, dblk * 64, u.kh, 0, page, pol);
                    else tma_load_4d_pair(dst, isV ? &maps.v_tree : &maps.k_tree, lbar, dblk * 64, u.kh, 16 * pg_in_tile, u.b);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------------- MMA issuer (leader CTA only)
        if (rank == 0 && lane == 0) {
            constexpr uint32_t idesc_s = make_idesc(256, CB_KT, false);
            constexpr uint32_t idesc_o = make_idesc(256, D, true);
            uint32_t c = 0, uq = 0;
            bool ok = true;
            const uint32_t q_lo = desc_lo(sbase + C::OFF_Q, 16), k_lo0 = desc_lo(sbase + C::OFF_RING, 16);
            const uint32_t v_lo0 = desc_lo(sbase + C::OFF_RING + C::HALF_BYTES, 16);
            while (ok && wk.next(p, &u)) {
                if (!(ok = mbar_wait(bar_qfull, uq & 1, s_abort, p.status))) break;
                tc_fence_after();
                for (int i = u.t0; ok && i <= u.t1; ++i) {
                    if (i < u.t1) {
                        const uint32_t cc = c + (uint32_t)(i - u.t0), slot = cc % C::NSLOT, buf = cc & 1u;
                        if (!(ok = mbar_wait(bar_full(slot), (cc / C::NSLOT) & 1, s_abort, p.status))) break;
                        tc_fence_after();
                        mma2_s_block(tmem + buf * 128, q_lo, k_lo0 + slot * (C::SLOT_BYTES >> 4), idesc_s);
                        tc_commit_pair(bar_sfull(buf));
                        if (i == u.t1 - 1) tc_commit_pair(bar_qfree);
                    }
                    if (i > u.t0) {
                        const uint32_t cp = c + (uint32_t)(i - 1 - u.t0), slot = cp % C::NSLOT, buf = cp & 1u;
                        if (!(ok = mbar_wait(bar_pready(buf), (cp >> 1) & 1, s_abort, p.status))) break;
                        if (i == u.t0 + 1 && uq > 0 && !(ok = mbar_wait(bar_ofree, (uq - 1) & 1, s_abort, p.status))) break;
                        tc_fence_after();
                        mma2_pv_block(tmem + C::O_COL, tmem + buf * 128, v_lo0 + slot * (C::SLOT_BYTES >> 4), idesc_o, i > u.t0 + 1 ? 1u : 0u);
                        tc_commit_pair(bar_free(slot));
                        if (i == u.t1) tc_commit_pair(bar_ofull);
                    }
                }
                c += (uint32_t)(u.t1 - u.t0);
                ++uq;
            }
        }
        __syncwarp();
    } else if (warp == 2) {
        // ---------------------------------------------------------------------- query loader, then zero rows of padding nodes
        uint32_t uq = 0;
        bool have = wk.next(p, &u);
        auto load_q = [&]() {
            if (rank == 0) mbar_expect_tx_only(bar_qfull, (uint32_t)(u.nrt * C::DB * RT * 128));
            if ((int)rank < u.nrt) {
                const uint32_t lbar = cluster_addr(bar_qfull, 0);
                for (int db = 0; db < C::DB; ++db)
                    tma_load_4d_pair(sbase + C::OFF_Q + db * (CB_MT * 128), &maps.q, lbar, db * 64, u.kh * p.G, (u.rg * 2 + (int)rank) * p.NPT, u.b);
            }
        };
        if (have && lane == 0) load_q();
        __syncwarp();
        {
            const int per_row = p.Hq * D / 8;                    // 16-byte chunks per node row
            for (int idx = blockIdx.x; idx < p.B * p.T; idx += gridDim.x) {
                const int b = idx / p.T, node = idx % p.T;
                const int n = min(max(p.n_nodes[b], 0), p.T);
                if (node < n) continue;
                uint4* op = reinterpret_cast<uint4*>(p.out + (size_t)idx * p.Hq * D);
                for (int k = lane; k < per_row; k += 32) op[k] = make_uint4(0, 0, 0, 0);
                if (p.lse) for (int h = lane; h < p.Hq; h += 32) p.lse[((size_t)b * p.Hq + h) * p.T + node] = 0.f;
            }
        }
        if (lane == 0 && have) {
            uq = 1;
            while (wk.next(p, &u)) {
                if (!mbar_wait(bar_qfree, (uq - 1) & 1, s_abort, p.status)) break;
                load_q();
                ++uq;
            }
        }
        __syncwarp();
    } else if (warp >= 4) {
        // ---------------------------------------------------------------------- softmax / correction / epilogue
        const int wg = (warp - 4) >> 2;                         // which half of every tile's key columns this thread takes
        const int wq = warp & 3;                                // TMEM lane quarter this warp may access
        const int row = wq * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
        // The two threads of a row (same lane quarter, one per warpgroup) meet on an mbarrier of their own: every wait in
        // this kernel is bounded, which a named barrier is not.  pp counts the phases used.
        const uint32_t bar_pair = bar_pair0 + 8u * (uint32_t)wq;
        volatile uint32_t* over_flag = s_over + 2 * wq;
        volatile float* x_mine = s_xchg + wg * CB_MT + row;
        volatile float* x_peer = s_xchg + (wg ^ 1) * CB_MT + row;
        uint32_t pp = 0, c = 0, uq = 0;
        bool ok = true;
        auto pair_sync = [&]() {
            mbar_arrive(bar_pair);
            const bool r = mbar_wait(bar_pair, pp & 1, s_abort, p.status);
            ++pp;
            return r;
        };
        // The next unit's shape and this row's ancestor bits (the two words of this thread's columns) are fetched while the
        // current unit is being finished.
        CbUnit un;
        uint32_t mrow_n[2] = {0u, 0u};
        auto fetch_next = [&]() {
            const bool have = wk.next(p, &un);
            mrow_n[0] = mrow_n[1] = 0u;
            if (have && (int)rank < un.nrt) {
                const int nnode = (un.rg * 2 + (int)rank) * p.NPT + row / p.G;
                if (row < RT && nnode < un.n) {
                    const uint32_t* mp = p.tree_mask + ((size_t)un.b * p.T + nnode) * p.W;
                    if (p.W > 2 * wg) mrow_n[0] = mp[2 * wg];
                    if (p.W > 2 * wg + 1) mrow_n[1] = mp[2 * wg + 1];
                }
            }
            return have;
        };
        bool have = fetch_next();
        while (ok && have) {
            u = un;
            const uint32_t mk0 = mrow_n[0], mk1 = mrow_n[1];
            const bool mine = (int)rank < u.nrt;                 // this CTA's row tile exists in the unit
            const int rt = u.rg * 2 + (int)rank;
            const int node = rt * p.NPT + row / p.G, g = row % p.G, h = u.kh * p.G + g;
            const bool row_valid = mine && row < RT && node < u.n;
            // row 0 of the warp is valid: a warp without valid rows skips the arithmetic (both warps of a pair alike)
            const bool warp_active = mine && (wq * 32) < RT && (rt * p.NPT + (wq * 32) / p.G) < u.n;
            const int nct = u.tiles - 1;
            float m_used = -INFINITY, l = 0.f;                   // the row's reference (same in both threads), this thread's part of the row sum
            for (int i = u.t0; i < u.t1; ++i) {
                const uint32_t cc = c + (uint32_t)(i - u.t0), buf = cc & 1u;
                if (!(ok = mbar_wait(bar_sfull(buf), (cc >> 1) & 1, s_abort, p.status))) break;
                if (warp_active) {
                    tc_fence_after();
                    const uint32_t ts = tmem + buf * 128 + lane_addr + 64u * (uint32_t)wg;   // this thread's 64 columns; its P goes over the first 32
                    uint32_t A0[32], A1[32];
                    CB_TMEM_LD32(A0, 0, ts);
                    CB_TMEM_LD32(A1, 0, ts + 32);
                    // visibility of this thread's 64 keys for its row: context keys below ctx, tree keys by the ancestor bits.  A
                    // context tile that lies wholly inside the context needs no masks; rows that do not exist take that path
                    // too: whatever they compute stays in their own row.
                    const bool is_tree = i == nct;
                    const int kv = is_tree ? u.n : min(CB_KT, u.ctx - i * CB_KT);
                    auto below_bits = [](int lo) { return lo >= 32 ? 0xFFFFFFFFu : (lo <= 0 ? 0u : ((1u << lo) - 1u)); };
                    uint32_t vm0 = 0xFFFFFFFFu, vm1 = 0xFFFFFFFFu;
                    bool all_vis = !is_tree && kv == CB_KT;
                    if (!all_vis) {
                        vm0 = row_valid ? ((is_tree ? mk0 : 0xFFFFFFFFu) & below_bits(kv - 64 * wg)) : 0u;
                        vm1 = row_valid ? ((is_tree ? mk1 : 0xFFFFFFFFu) & below_bits(kv - 64 * wg - 32)) : 0u;
                        all_vis = __all_sync(CB_FULL, !row_valid || (vm0 & vm1) == 0xFFFFFFFFu);
                    }
                    CB_TMEM_WAIT_LD32(A0);
                    CB_TMEM_WAIT_LD32(A1);
                    if (!all_vis) {
#pragma unroll
                        for (int jx = 0; jx < 32; ++jx) {
                            if (!((vm0 >> jx) & 1u)) A0[jx] = 0xFF800000u;
                            if (!((vm1 >> jx) & 1u)) A1[jx] = 0xFF800000u;
                        }
                    }
                    // largest visible score of this thread's columns (first tile of a share, and the rare path below)
                    auto half_max = [&]() {
                        float c0 = -INFINITY, c1 = -INFINITY, c2 = -INFINITY, c3 = -INFINITY;
#pragma unroll
                        for (int jx = 0; jx < 32; jx += 8) {
                            c0 = fmax3(c0, __uint_as_float(A0[jx]), __uint_as_float(A0[jx + 1]));
                            c1 = fmax3(c1, __uint_as_float(A0[jx + 2]), __uint_as_float(A0[jx + 3]));
                            c2 = fmax3(c2, __uint_as_float(A0[jx + 4]), __uint_as_float(A0[jx + 5]));
                            c3 = fmax3(c3, __uint_as_float(A0[jx + 6]), __uint_as_float(A0[jx + 7]));
                            c0 = fmax3(c0, __uint_as_float(A1[jx]), __uint_as_float(A1[jx + 1]));
                            c1 = fmax3(c1, __uint_as_float(A1[jx + 2]), __uint_as_float(A1[jx + 3]));
                            c2 = fmax3(c2, __uint_as_float(A1[jx + 4]), __uint_as_float(A1[jx + 5]));
                            c3 = fmax3(c3, __uint_as_float(A1[jx + 6]), __uint_as_float(A1[jx + 7]));
                        }
                        return fmaxf(fmaxf(c0, c1), fmaxf(c2, c3)) * p.scale_log2;
                    };
                    // The reference maximum of a row is shared by its two threads.  A share's first tile sets it to the row's
                    // true maximum (exchanged through shared memory).  Later tiles keep it as long as it serves: the reference
                    // only has to keep 2^(s - reference) and its sums inside fp32 (P is bf16, same exponent range), not to be
                    // the maximum, and no maximum is taken: this thread's row sum of the tile, which is needed anyway, tells
                    // (at most 2^22: no P is above that, and one above 2^16 times 64 would show).  P is stored at once; a
                    // warp that holds a sum out of range (or not finite) leaves this phase's tag in the pair's flag, the two
                    // warps of the rows meet, and only then is P announced, or done again (the scores are still in registers).
                    const bool first = i == u.t0;
                    if (first) {
                        const float hm = half_max();
                        *x_mine = hm;
                        if (!(ok = pair_sync())) break;
                        m_used = fmaxf(hm, *x_peer);
                        if (!(ok = pair_sync())) break;
                    }
                    uint32_t pk[32];
                    const uint64_t scale2 = f2_pack(p.scale_log2, p.scale_log2), zero2 = f2_pack(0.f, 0.f);
                    uint64_t a0, a1, a2, a3;
                    // P = 2^(s * scale - reference) of this thread's 64 scores, packed to bf16 pairs; eight independent partial sums
                    auto exps = [&]() {
                        const float mu = (m_used == -INFINITY) ? 0.f : m_used;
                        const uint64_t negmu2 = f2_pack(-mu, -mu);
                        a0 = a1 = a2 = a3 = zero2;
#pragma unroll
                        for (int hx = 0; hx < 2; ++hx) {
                            const uint32_t* cur = hx ? A1 : A0;
#pragma unroll
                            for (int jx = 0; jx < 32; jx += 8) {
                                float p0, p1, p2, p3, p4, p5, p6, p7;
                                f2_unpack(f2_fma(f2_pack(__uint_as_float(cur[jx]), __uint_as_float(cur[jx + 1])), scale2, negmu2), p0, p1);
                                f2_unpack(f2_fma(f2_pack(__uint_as_float(cur[jx + 2]), __uint_as_float(cur[jx + 3])), scale2, negmu2), p2, p3);
                                f2_unpack(f2_fma(f2_pack(__uint_as_float(cur[jx + 4]), __uint_as_float(cur[jx + 5])), scale2, negmu2), p4, p5);
                                f2_unpack(f2_fma(f2_pack(__uint_as_float(cur[jx + 6]), __uint_as_float(cur[jx + 7])), scale2, negmu2), p6, p7);
                                p0 = ex2(p0); p1 = ex2(p1); p2 = ex2(p2); p3 = ex2(p3); p4 = ex2(p4); p5 = ex2(p5); p6 = ex2(p6); p7 = ex2(p7);
                                a0 = f2_add(a0, f2_pack(p0, p1));
                                a1 = f2_add(a1, f2_pack(p2, p3));
                                a2 = f2_add(a2, f2_pack(p4, p5));
                                a3 = f2_add(a3, f2_pack(p6, p7));
                                pk[hx * 16 + (jx >> 1)] = pack_bf16(p0, p1);
                                pk[hx * 16 + (jx >> 1) + 1] = pack_bf16(p2, p3);
                                pk[hx * 16 + (jx >> 1) + 2] = pack_bf16(p4, p5);
                                pk[hx * 16 + (jx >> 1) + 3] = pack_bf16(p6, p7);
                            }
                        }
                        float s_lo, s_hi;
                        f2_unpack(f2_add(f2_add(a0, a1), f2_add(a2, a3)), s_lo, s_hi);
                        return s_lo + s_hi;
                    };
                    float lt = exps();
                    CB_TMEM_ST16(pk, 0, ts);
                    CB_TMEM_ST16(pk, 16, ts + 16);
                    if (!first) {
                        // rows that do not exist hold anything: they never ask
                        if (__any_sync(CB_FULL, row_valid && !(lt <= 4194304.f)) && lane == 0) over_flag[pp & 1] = pp + 1u;
                        if (!(ok = pair_sync())) break;
                        if (over_flag[(pp - 1u) & 1] == pp) {
                            // Some row of this pair of warps holds a score far above its reference: the pair's threads exchange
                            // their maxima, rows that need it move their reference there and rescale O (each thread its half of
                            // the columns) and their row sums, and P is computed again.
                            const float hm = half_max();
                            *x_mine = hm;
                            if (!(ok = pair_sync())) break;
                            const float row_max = fmaxf(hm, *x_peer);
                            if (!(ok = pair_sync())) break;
                            const bool need = row_max > m_used + 8.0f;
                            const float alpha = need ? ex2(m_used - row_max) : 1.0f;
                            if (need) m_used = row_max;
                            // O must be complete up to the previous tile before it is rescaled: that tile's slot has been released
                            const uint32_t cp = cc - 1u;
                            if (!(ok = mbar_wait(bar_free(cp % C::NSLOT), (cp / C::NSLOT) & 1, s_abort, p.status))) break;
                            tc_fence_after();
                            tmem_wait_st();
                            rescale_row(tmem + C::O_COL + lane_addr + 64u * (uint32_t)wg, 4, alpha);
                            l *= alpha;
                            lt = exps();
                            CB_TMEM_ST16(pk, 0, ts);
                            CB_TMEM_ST16(pk, 16, ts + 16);
                        }
                    }
                    l += lt;
                    tmem_wait_st();
                }
                // P of this warp's rows and columns is in place: one arrival per warp on the leader's barrier
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_peer(cluster_addr(bar_pready(buf), 0));
            }
            if (!ok) break;
            c += (uint32_t)(u.t1 - u.t0);
            have = fetch_next();
            // ---- epilogue of this unit's share.  The row sums of the two column halves are added up through shared memory;
            // the exchange ends with the pair meeting once more, so that the words are free for their next use.
            *x_mine = l;
            if (!(ok = pair_sync())) break;
            l += *x_peer;
            if (!(ok = pair_sync())) break;
            // O is complete once the unit's last PV has finished; each warpgroup writes half of the output columns
            if (!(ok = mbar_wait(bar_ofull, uq & 1, s_abort, p.status))) break;
            tc_fence_after();
            if (warp_active) {
                const bool whole = u.t0 == 0 && u.t1 == u.tiles;
                const float inv = whole ? (l > 0.f ? 1.0f / l : 0.f) : 1.0f;
                const uint32_t t_me = tmem + C::O_COL + lane_addr + 64u * (uint32_t)wg;
                __nv_bfloat16* op = p.out + (((size_t)u.b * p.T + node) * p.Hq + h) * D + 64 * wg;
                const size_t pslot = 2 * (size_t)pair + (u.t0 == 0 ? 1 : 0);
                float* pp_ = p.part + ((pslot * 2 + rank) * CB_MT + row) * (D + 4);
#pragma unroll
                for (int cx = 0; cx < 2; ++cx) {
                    uint32_t o[32];
                    CB_TMEM_LD32(o, 0, t_me + cx * 32);
                    tmem_wait_ld();
                    if (row_valid) {
                        if (whole) {
                            uint32_t w[16];
#pragma unroll
                            for (int k2 = 0; k2 < 16; ++k2) w[k2] = pack_bf16(__uint_as_float(o[2 * k2]) * inv, __uint_as_float(o[2 * k2 + 1]) * inv);
                            st_global_v8(op + cx * 32, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
                            st_global_v8(op + cx * 32 + 16, w[8], w[9], w[10], w[11], w[12], w[13], w[14], w[15]);
                        } else {
                            // partial rows are D + 4 floats long: 16-byte aligned only
#pragma unroll
                            for (int v4 = 0; v4 < 8; ++v4)
                                *reinterpret_cast<uint4*>(pp_ + 64 * wg + cx * 32 + v4 * 4) = make_uint4(o[v4 * 4], o[v4 * 4 + 1], o[v4 * 4 + 2], o[v4 * 4 + 3]);
                        }
                    }
                }
                if (row_valid && wg == 0) {
                    if (whole) {
                        if (p.lse) p.lse[((size_t)u.b * p.Hq + h) * p.T + node] = l > 0.f ? (m_used + log2f(l)) * 0.6931471805599453f : 0.f;
                    } else {
                        pp_[D] = m_used; pp_[D + 1] = l;
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_peer(cluster_addr(bar_ofree, 0));
            ++uq;
        }
    }

    // ---------------------------------------------------------------------- teardown
    if (*s_abort) {
        // give copies that are still in flight time to land before the shared memory is released
        for (int k = 0; k < 64; ++k) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    // neither CTA leaves while the other may still signal its barriers or read its shared memory
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

}  // namespace
