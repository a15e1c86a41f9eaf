// Tree-masked attention on the 5th-generation tensor cores (tcgen05) with TMA-staged paged K/V.
//
// Persistent kernel: one CTA per SM, each working through an equal share of the global sequence of key
// tiles (see cb_attn.cuh).  A CTA holds up to two 128-row query tiles of a unit and streams that unit's
// 128-key tiles through a ring of 128B-swizzled shared-memory slots (K and V tiles alternate in the
// ring; eight 16-token pages per tile, fetched page by page with TMA through the block table).
//
// Warp roles (384 threads, three warpgroups):
//   warp 0        TMA producer for the K tiles (warp 3 for the V tiles): runs ahead across unit boundaries, limited only
//                 by the ring
//   warp 1        MMA issuer (one lane): S = Q K^T into TMEM, then O += P V with P read from TMEM;
//                 owns the TMEM allocation (S0, S1, O0, O1: 4 x 128 columns)
//   warp 2        TMA loader for the query tiles of each unit; in launches where every unit has one row tile it also issues
//                 S = Q K^T, and warp 1 only O += P V (two issuing threads, see two_issuers below)
//   warp 3        writes the zero rows of padding nodes (node >= n_nodes), then TMA producer for the V tiles
//   warps 4..7    softmax warpgroup 0, warps 8..11 softmax warpgroup 1: one thread per query row; S from
//                 TMEM to registers, fp32 online softmax in the log2 domain with lazy rescaling of O,
//                 P written back to TMEM as packed bf16 over S; epilogue of the unit
// A unit with two valid row tiles gives one to each softmax warpgroup (both consume every key tile, so
// the tensor pipe works on one tile's MMAs while the other tile is in softmax).  A unit with one valid
// row tile is handled by warpgroup 0 alone with S double-buffered over S0/S1.
// All waits are bounded; a wait that runs out records CB_ERR_TIMEOUT and the CTA drains and exits.
//
// Cluster mode.  When a launch has so few units that the split above would make every unit a shared one (batch 1), the
// kernel is launched as thread-block clusters instead: cluster k works on unit k, its CTAs take equal parts of the unit's
// key tiles, and at the end they combine their shares through distributed shared memory: row block r of the 128 rows is
// gathered in CTA r, which merges the contributions and writes the output.  No partials go to HBM and no merge pass runs.
#include <cuda.h>

#include <mutex>

#include "cb_tc_dev.cuh"

namespace {

template <int D>
struct Cfg {
    static constexpr int DB = D / 64;                        // 64-element (128-byte) column blocks per row
    static constexpr int NSLOT = (D == 128) ? 5 : 8;         // ring slots, each one K or one V tile
    static constexpr uint32_t TILE_BYTES = CB_KT * D * 2;    // one K or V tile
    static constexpr uint32_t Q_BYTES = CB_MT * D * 2;       // one query row tile
    static constexpr uint32_t OFF_Q = 0;                     // two row tiles
    static constexpr uint32_t OFF_RING = 2 * Q_BYTES;
    static constexpr uint32_t OFF_BAR = OFF_RING + NSLOT * TILE_BYTES;
    // slot_full[NSLOT], slot_free[NSLOT], q_full, q_free, s_full0, p_ready[2], o_free[2], cluster_ready, cluster_data
    static constexpr int NBAR = 2 * NSLOT + 2 + 7 + 2;       // ... and pv_done[2]
    static constexpr uint32_t OFF_MISC = OFF_BAR + NBAR * 8;  // schedule, tmem base, abort flag
    static constexpr uint32_t SMEM = OFF_MISC + 96;
    static constexpr uint32_t SMEM_ALLOC = SMEM + 1024;      // slack to align the base to 1024 bytes
    static constexpr uint32_t O_COL = 256;                   // TMEM columns: S0 at 0, S1 at 128, O0 at 256, O1 at 256 + D
};

struct SchedSmem { long long g0, g1, pre0; int b0, rg0; int c_b, c_kh, c_t0, c_t1, c_tiles, c_n, c_ctx, c_has; };
static_assert(sizeof(SchedSmem) <= 64, "the schedule block is followed by the tmem base and the abort flag");

}  // namespace

#include "cb_attn_pair.cuh"

namespace {

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
cb_attn_tc_kernel(const CbAttnParams p, const __grid_constant__ TcMaps maps) {
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sgen = smem_raw + (sbase - smem_u32(smem_raw));
    const uint32_t bar0 = sbase + C::OFF_BAR;
    auto bar_full = [&](int s) { return bar0 + 8u * s; };
    auto bar_free = [&](int s) { return bar0 + 8u * (C::NSLOT + s); };
    auto slot_base = [&](uint32_t s) { return sbase + C::OFF_RING + s * C::TILE_BYTES; };
    const uint32_t bar_qfull = bar0 + 8u * (2 * C::NSLOT), bar_qfree = bar_qfull + 8u;
    // Completion of the tensor core's work is signalled with as few commits as possible (a second commit behind the
    // same MMA block stalls the issuer): a ring slot's "free" barrier doubles as "the S product that read this K tile is
    // done" and "the PV product that read this V tile is done".  Its phases are a ring revolution apart, so a softmax
    // thread can wait on it by the slot's sequence number alone.  Only row tile 0 of a two-row-tile unit needs a
    // barrier of its own for S, because its S is finished before the K tile is released.
    const uint32_t bar_sfull0 = bar0 + 8u * (2 * C::NSLOT + 2);
    auto bar_pready = [&](int s) { return bar0 + 8u * (2 * C::NSLOT + 3 + s); };
    auto bar_ofree = [&](int s) { return bar0 + 8u * (2 * C::NSLOT + 5 + s); };
    const uint32_t bar_cready = bar0 + 8u * (2 * C::NSLOT + 7), bar_cdata = bar_cready + 8u;   // cluster mode only
    auto bar_pvdone = [&](int s) { return bar0 + 8u * (2 * C::NSLOT + 9 + s); };               // two issuing threads only (see below)
    SchedSmem* s_sched = reinterpret_cast<SchedSmem*>(sgen + C::OFF_MISC);
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(sgen + C::OFF_MISC + 64);
    volatile int* s_abort = reinterpret_cast<volatile int*>(sgen + C::OFF_MISC + 68);
    volatile int* s_one_row = reinterpret_cast<volatile int*>(sgen + C::OFF_MISC + 72);   // every unit of the launch has one row tile

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x;
    const int RT = p.NPT * p.G;                               // rows of a row tile that exist
    // Set-up that reads no input (TMEM allocation, barrier initialisation, descriptor prefetch) runs before the wait for the
    // kernels earlier in the stream, so it overlaps their tail.  The merge pass (like the next kernel of a step) is launched as
    // a programmatic dependent in turn: its blocks may take the SMs that this grid's CTAs leave and do their set-up there;
    // they wait for this whole grid before they read any partial.
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    } else if (warp == 2) {
        if (lane == 0) {
            for (int s = 0; s < C::NSLOT; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_free(s), 1); }
            mbar_init(bar_qfull, 1); mbar_init(bar_qfree, 1); mbar_init(bar_sfull0, 1);
            for (int s = 0; s < 2; ++s) {
                mbar_init(bar_pready(s), 256); mbar_init(bar_ofree(s), 128);
            }
            mbar_init(bar_cready, p.cs > 0 ? (uint32_t)p.cs : 1u); mbar_init(bar_cdata, 128);
            mbar_init(bar_pvdone(0), 1); mbar_init(bar_pvdone(1), 1);
            *s_abort = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            tma_prefetch_desc(&maps.k_pool); tma_prefetch_desc(&maps.v_pool); tma_prefetch_desc(&maps.q);
            tma_prefetch_desc(&maps.k_tree); tma_prefetch_desc(&maps.v_tree);
        }
    }
    CB_PDL_ENTRY();

    if (warp == 0 && p.cs > 0) {
        // Cluster mode: cluster k works on unit k = (sequence, kv head) and its CTAs take equal parts of the unit's key tiles.
        if (lane == 0) {
            const int uid = cta / p.cs, rank = cta % p.cs;
            const int b = uid / p.Hkv;
            const CbSeqShape sh = cb_seq_shape(p, b);
            s_sched->c_b = b; s_sched->c_kh = uid % p.Hkv; s_sched->c_tiles = sh.tiles; s_sched->c_n = sh.n; s_sched->c_ctx = sh.ctx;
            s_sched->c_has = sh.RG > 0 ? 1 : 0;
            s_sched->c_t0 = sh.RG > 0 ? (int)((long long)sh.tiles * rank / p.cs) : 0;
            s_sched->c_t1 = sh.RG > 0 ? (int)((long long)sh.tiles * (rank + 1) / p.cs) : 0;
            s_sched->g0 = 0; s_sched->g1 = 0; s_sched->pre0 = 0; s_sched->b0 = 0; s_sched->rg0 = 0;
            *s_one_row = 1;
        }
    } else if (warp == 0) {
        // this CTA's range of the global tile sequence
        int max_rt = 0;
        const long long tot = cb_sched_total(p, lane, &max_rt);
        const long long g0 = cb_range_start(tot, p.nc, cta), g1 = cb_range_start(tot, p.nc, cta + 1);
        int b0 = 0, rg0 = 0;
        long long pre0 = 0;
        if (g0 < g1) cb_sched_locate(p, g0, lane, &rg0, &b0, &pre0);
        if (lane == 0) {
            s_sched->g0 = g0; s_sched->g1 = g1; s_sched->b0 = b0; s_sched->rg0 = rg0; s_sched->pre0 = pre0;
            *s_one_row = (p.MT == 1 || max_rt <= 1) ? 1 : 0;
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *s_tmem;
    const long long g0 = s_sched->g0, g1 = s_sched->g1, pre0 = s_sched->pre0;
    const int b0 = s_sched->b0, rg0 = s_sched->rg0;
    // When no unit of the launch has two row tiles (the same for every CTA: it follows from n_nodes alone), the products of a
    // key tile get an issuing thread each: warp 2's thread, which loads the query tile, issues S = Q K^T, warp 1's thread
    // issues O += P V.  One thread issuing both spends about 2.0 k cycles per key tile in the two blocks and its loop, and the
    // next S follows the P.V it has to wait for; with two threads the next S only waits for the completion of the P.V that
    // read its buffer two tiles before, and the softmax warpgroup (1.9 k cycles per tile) is what a tile costs.
    const bool two_issuers = *s_one_row != 0;
    constexpr uint32_t ns = (uint32_t)C::NSLOT;
    CbWalker wk;
    if (p.cs > 0) {
        // the peers' barriers must exist before anything arrives on them
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        CbUnit u0;
        u0.b = s_sched->c_b; u0.kh = s_sched->c_kh; u0.rg = 0; u0.t0 = s_sched->c_t0; u0.t1 = s_sched->c_t1;
        u0.tiles = s_sched->c_tiles; u0.n = s_sched->c_n; u0.ctx = s_sched->c_ctx; u0.nrt = 1;
        wk.init_fixed(u0);
    } else {
        wk.init(p, g0, g1, rg0, b0, pre0);
    }
    CbUnit u;

    if (warp < 4) {
        reg_dealloc<120>();
        if (warp == 0 || warp == 3) {
            // ------------------------------------------------------------------ K/V producers: warp 0 the K tiles, warp 3 the V tiles
            // A tile is 8 * DB boxes of 16 keys x 64 dims, one copy instruction each, and the copies of one warp instruction
            // are issued one after the other: two warps issue the two tiles of a key tile side by side.
            const bool isV = warp == 3;
            if (isV) {
                // rows of padding nodes (node >= n_nodes) are written as zeros: once, before the first V tile is wanted
                const int per_row = p.Hq * D / 8;            // 16-byte chunks per node row
                for (int idx = cta; idx < p.B * p.T; idx += gridDim.x) {
                    const int b = idx / p.T, node = idx % p.T;
                    const int n = min(max(p.n_nodes[b], 0), p.T);
                    if (node < n) continue;
                    uint4* op = reinterpret_cast<uint4*>(p.out + (size_t)idx * p.Hq * D);
                    for (int k = lane; k < per_row; k += 32) op[k] = make_uint4(0, 0, 0, 0);
                    if (p.lse) for (int h = lane; h < p.Hq; h += 32) p.lse[((size_t)b * p.Hq + h) * p.T + node] = 0.f;
                }
            }
            constexpr int NB = 8 * C::DB;                    // boxes per tile
            const bool active = lane < NB;
            const int j = lane % 8, dblk = (lane % NB) / 8;
            uint32_t seq = isV ? 1u : 0u;                    // K and V tiles alternate in the ring
            bool ok = true;
            const uint64_t pol = l2_evict_first_policy();
            while (ok && wk.next(p, &u)) {
                const int npages = (u.ctx + p.P - 1) / p.P, nct = u.tiles - 1;
                const int32_t* bt = p.block_table + (size_t)u.b * p.max_pages;
                // The page number of a lane's box comes from the block table: a memory round trip that the copy depends on.
                // It is fetched one tile ahead, so that it is under way while this tile's copies are issued and waited for.
                auto page_of = [&](int i) {
                    int page = p.num_pages;                  // out of range: the copy fills zeros
                    if (active && i < nct) {
                        const int pidx = i * (CB_KT / 16) + j;
                        if (pidx < npages) page = bt[pidx];
                    }
                    return page;
                };
                int page_next = page_of(u.t0);
                for (int i = u.t0; i < u.t1; ++i) {
                    int page = page_next;
                    if (i + 1 < u.t1) page_next = page_of(i + 1);
                    if (!cb_dbg_in(page, p.num_pages + 1, p.status)) page = p.num_pages;   // the copy then fills zeros
                    const uint32_t sl = seq % ns;
                    if (seq >= ns && !(ok = mbar_wait(bar_free(sl), (seq / ns - 1) & 1, s_abort, p.status))) break;
                    if (lane == 0) mbar_expect_tx(bar_full(sl), C::TILE_BYTES);
                    __syncwarp();
                    if (active) {
                        const uint32_t dst = slot_base(sl) + dblk * (CB_KT * 128) + j * 2048;
                        if (i < nct) tma_load_4d_hint(dst, isV ? &maps.v_pool : &maps.k_pool, bar_full(sl), dblk * 64, u.kh, 0, page, pol);
                        else tma_load_4d(dst, isV ? &maps.v_tree : &maps.k_tree, bar_full(sl), dblk * 64, u.kh, 16 * j, u.b);
                    }
                    seq += 2;
                }
            }
        } else if (warp == 1) {
            // ------------------------------------------------------------------ MMA issuer
            if (lane == 0) {
                constexpr uint32_t idesc_s = make_idesc(128, CB_KT, false);
                constexpr uint32_t idesc_o = make_idesc(128, D, true);
                uint32_t seq = 0, uq = 0, c_p[2] = {0u, 0u}, c_of[2] = {0u, 0u};
                bool ok = true;
                const uint32_t q_lo0 = desc_lo(sbase + C::OFF_Q, 16), k_lo0 = desc_lo(sbase + C::OFF_RING, 16);
                const uint32_t v_lo0 = desc_lo(sbase + C::OFF_RING, CB_KT * 128);
                auto issue_s = [&](int rt, int buf, uint32_t kslot) {
                    mma_s_block<D>(tmem + buf * 128, q_lo0 + rt * (C::Q_BYTES >> 4), k_lo0 + kslot * (C::TILE_BYTES >> 4), idesc_s);
                };
                auto issue_pv = [&](int ol, int buf, uint32_t vslot, bool accum) {
                    mma_pv_block(tmem + C::O_COL + ol * D, tmem + buf * 128, v_lo0 + vslot * (C::TILE_BYTES >> 4), idesc_o, accum ? 1u : 0u);
                };
                if (two_issuers) {
                    // O += P V only (S is issued by warp 2's thread).  After every product one more commit reports it on the
                    // barrier of the S buffer whose P it read: the next S into that buffer waits for it.
                    uint32_t c_of0 = 0;
                    while (ok && wk.next(p, &u)) {
                        const uint32_t seq0 = seq;
                        for (int i = u.t0; ok && i < u.t1; ++i) {
                            const int buf = (i - u.t0) & 1;
                            const uint32_t vseq = seq0 + 2u * (uint32_t)(i - u.t0) + 1u, vs = vseq % ns;
                            if (!(ok = mbar_wait(bar_full(vs), (vseq / ns) & 1, s_abort, p.status))) break;
                            if (!(ok = mbar_wait(bar_pready(buf), c_p[buf] & 1, s_abort, p.status))) break;
                            ++c_p[buf];
                            if (i == u.t0) {
                                if (c_of0 > 0 && !(ok = mbar_wait(bar_ofree(0), (c_of0 - 1) & 1, s_abort, p.status))) break;
                                ++c_of0;
                            }
                            tc_fence_after();
                            mma_pv_block(tmem + C::O_COL, tmem + buf * 128, desc_lo(slot_base(vs), CB_KT * 128), idesc_o, i > u.t0 ? 1u : 0u);
                            tc_commit(bar_free(vs));
                            tc_commit(bar_pvdone(buf));
                        }
                        seq = seq0 + 2u * (uint32_t)(u.t1 - u.t0);
                    }
                }
                CbUnit un;
                    bool have = !two_issuers && wk.next(p, &un);
                while (ok && have) {
                    u = un;
                    const bool two = u.nrt == 2;
                    if (!(ok = mbar_wait(bar_qfull, uq & 1, s_abort, p.status))) break;
                    tc_fence_after();
                    const uint32_t seq0 = seq;
                    for (int i = u.t0; ok && i <= u.t1; ++i) {
                        if (i == u.t1) have = wk.next(p, &un);   // its loads overlap the wait for the last P
                        const uint32_t kseq = seq0 + 2 * (i - u.t0), vseq_prev = kseq - 1;
                        const uint32_t ks = kseq % C::NSLOT, vs = vseq_prev % C::NSLOT;
                        if (two) {
                            // per row tile l: PV of the previous key tile, then S of this one, so that the other
                            // tile's softmax always has MMAs to overlap with
                            for (int l = 0; l < 2; ++l) {
                                if (i > u.t0) {
                                    if (l == 0 && !(ok = mbar_wait(bar_full(vs), (vseq_prev / C::NSLOT) & 1, s_abort, p.status))) break;
                                    if (!(ok = mbar_wait(bar_pready(l), c_p[l] & 1, s_abort, p.status))) break;
                                    ++c_p[l];
                                    if (i == u.t0 + 1) {
                                        if (c_of[l] > 0 && !(ok = mbar_wait(bar_ofree(l), (c_of[l] - 1) & 1, s_abort, p.status))) break;
                                        ++c_of[l];
                                    }
                                    tc_fence_after();
                                    issue_pv(l, l, vs, i > u.t0 + 1);
                                    if (l == 1) tc_commit(bar_free(vs));
                                }
                                if (i < u.t1) {
                                    if (l == 0) {
                                        if (!(ok = mbar_wait(bar_full(ks), (kseq / C::NSLOT) & 1, s_abort, p.status))) break;
                                        tc_fence_after();
                                    }
                                    issue_s(l, l, ks);
                                    if (l == 0) {
                                        tc_commit(bar_sfull0);
                                    } else {
                                        tc_commit(bar_free(ks));
                                        if (i == u.t1 - 1) tc_commit(bar_qfree);
                                    }
                                }
                            }
                        } else {
                            if (i < u.t1) {
                                const int buf = (i - u.t0) & 1;
                                if (!(ok = mbar_wait(bar_full(ks), (kseq / C::NSLOT) & 1, s_abort, p.status))) break;
                                tc_fence_after();
                                issue_s(0, buf, ks);
                                tc_commit(bar_free(ks));
                                if (i == u.t1 - 1) tc_commit(bar_qfree);
                            }
                            if (i > u.t0) {
                                const int buf = (i - 1 - u.t0) & 1;
                                if (!(ok = mbar_wait(bar_full(vs), (vseq_prev / C::NSLOT) & 1, s_abort, p.status))) break;
                                if (!(ok = mbar_wait(bar_pready(buf), c_p[buf] & 1, s_abort, p.status))) break;
                                ++c_p[buf];
                                if (i == u.t0 + 1) {
                                    if (c_of[0] > 0 && !(ok = mbar_wait(bar_ofree(0), (c_of[0] - 1) & 1, s_abort, p.status))) break;
                                    ++c_of[0];
                                }
                                tc_fence_after();
                                issue_pv(0, buf, vs, i > u.t0 + 1);
                                tc_commit(bar_free(vs));
                            }
                        }
                    }
                    seq = seq0 + 2 * (u.t1 - u.t0);
                    ++uq;
                }
            }
            __syncwarp();
        } else if (warp == 2) {
            // ------------------------------------------------------------------ query loader
            if (lane == 0) {
                uint32_t uq = 0;
                if (two_issuers) {
                    // query tile, then S = Q K^T of every key tile of the unit.  The k-th S into a buffer waits for the
                    // completion of the P.V that read the (k-1)-th P from it.
                    constexpr uint32_t idesc_s = make_idesc(128, CB_KT, false);
                    const uint32_t q_lo0 = desc_lo(sbase + C::OFF_Q, 16);
                    uint32_t seq = 0, c_s[2] = {0u, 0u};
                    bool ok = true;
                    while (ok && wk.next(p, &u)) {
                        if (uq > 0 && !(ok = mbar_wait(bar_qfree, (uq - 1) & 1, s_abort, p.status))) break;
                        mbar_expect_tx(bar_qfull, (uint32_t)(C::DB * RT * 128));
                        for (int db = 0; db < C::DB; ++db)
                            tma_load_4d(sbase + C::OFF_Q + db * (CB_MT * 128), &maps.q, bar_qfull, db * 64, u.kh * p.G, u.rg * 2 * p.NPT, u.b);
                        if (!(ok = mbar_wait(bar_qfull, uq & 1, s_abort, p.status))) break;
                        ++uq;
                        const uint32_t seq0 = seq;
                        for (int i = u.t0; ok && i < u.t1; ++i) {
                            const int buf = (i - u.t0) & 1;
                            const uint32_t kseq = seq0 + 2u * (uint32_t)(i - u.t0), ks = kseq % ns;
                            if (!(ok = mbar_wait(bar_full(ks), (kseq / ns) & 1, s_abort, p.status))) break;
                            if (c_s[buf] > 0 && !(ok = mbar_wait(bar_pvdone(buf), (c_s[buf] - 1) & 1, s_abort, p.status))) break;
                            ++c_s[buf];
                            tc_fence_after();
                            mma_s_block<D>(tmem + buf * 128, q_lo0, desc_lo(slot_base(ks), 16), idesc_s);
                            tc_commit(bar_free(ks));
                            if (i == u.t1 - 1) tc_commit(bar_qfree);
                        }
                        seq = seq0 + 2u * (uint32_t)(u.t1 - u.t0);
                    }
                }
                while (!two_issuers && wk.next(p, &u)) {
                    if (uq > 0 && !mbar_wait(bar_qfree, (uq - 1) & 1, s_abort, p.status)) break;
                    mbar_expect_tx(bar_qfull, (uint32_t)(u.nrt * C::DB * RT * 128));
                    for (int rt = 0; rt < u.nrt; ++rt)
                        for (int db = 0; db < C::DB; ++db)
                            tma_load_4d(sbase + C::OFF_Q + rt * C::Q_BYTES + db * (CB_MT * 128), &maps.q, bar_qfull, db * 64, u.kh * p.G,
                                        (u.rg * 2 + rt) * p.NPT, u.b);
                    ++uq;
                }
                if (p.cs > 0 && s_sched->c_has) {
                    // Cluster mode: the peers write their rows into this CTA's query tiles, so it reports itself ready to
                    // receive as soon as its last S product has released them (long before its last P.V is done).
                    const int Rv = (min(RT, p.T * p.G) + p.cs - 1) / p.cs;
                    if ((uint32_t)(p.cs * Rv) * (uint32_t)((D + 4) * 4) <= 2u * C::Q_BYTES) {
                        if (uq == 0 || mbar_wait(bar_qfree, 0, s_abort, p.status))
                            for (int r = 0; r < p.cs; ++r) mbar_arrive_remote(cluster_addr(bar_cready, (uint32_t)r));
                    }
                }
            }
            __syncwarp();
        }
    } else {
        // ---------------------------------------------------------------------- softmax / correction / epilogue
        reg_alloc<192>();
        const int wg = (warp - 4) >> 2;                       // softmax warpgroup = row tile of a two-tile unit
        const int wq = warp & 3;                              // TMEM lane quarter this warp may access
        const int row = wq * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
        const uint32_t tm_O = tmem + C::O_COL + wg * D + lane_addr;
        uint32_t c_s0 = 0;                                    // completions of s_full0 consumed so far (warpgroup 0 only)
        uint32_t seq = 0;                                     // ring sequence number of the next unit's first K tile
        bool ok = true;
        // The next unit's shape and this row's ancestor bits are fetched while the current unit is still being finished,
        // so that their memory round trips do not sit between two units.
        CbUnit un;
        uint32_t mrow_n[4] = {0u, 0u, 0u, 0u};
        auto fetch_next = [&]() {
            const bool have = wk.next(p, &un);
            mrow_n[0] = mrow_n[1] = mrow_n[2] = mrow_n[3] = 0u;
            if (have && (wg == 0 || un.nrt == 2)) {
                const int nnode = (un.rg * 2 + wg) * p.NPT + row / p.G;
                if (row < RT && nnode < un.n) {
                    const uint32_t* mp = p.tree_mask + ((size_t)un.b * p.T + nnode) * p.W;
                    mrow_n[0] = mp[0];
                    if (p.W > 1) mrow_n[1] = mp[1];
                    if (p.W > 2) mrow_n[2] = mp[2];
                    if (p.W > 3) mrow_n[3] = mp[3];
                }
            }
            return have;
        };
        float c_m = -INFINITY, c_l = 0.f;                     // cluster mode: this CTA's share of the unit, kept for the exchange
        bool c_share = false;
        bool have = fetch_next();
        while (ok && have) {
            u = un;
            const uint32_t mrow[4] = {mrow_n[0], mrow_n[1], mrow_n[2], mrow_n[3]};
            const bool two = u.nrt == 2;
            const int nt = u.t1 - u.t0;
            const uint32_t seq0 = seq;
            seq += 2u * (uint32_t)nt;
            if (wg == 1 && !two) {
                // Handled by warpgroup 0 alone.  This warpgroup still watches every S completion, in order: waiting on a
                // barrier by parity is only sound for a thread that is at most one phase away from it, and a thread that
                // ran ahead over this unit would later meet ring barriers that are whole revolutions behind it.  It must
                // not fall behind either (it may start late, after a long epilogue): half of every "P ready" arrival is
                // its own, given when it has seen the tile's S, so the products cannot run more than a tile ahead of it.
                for (int i = u.t0; ok && i < u.t1; ++i) {
                    const uint32_t kseq = seq0 + 2u * (uint32_t)(i - u.t0);
                    ok = mbar_wait(bar_free(kseq % ns), (kseq / ns) & 1, s_abort, p.status);
                    mbar_arrive(bar_pready((i - u.t0) & 1));
                }
                have = fetch_next();
                continue;
            }
            // S(i) is done when tile i's K slot is released (or, for row tile 0 of two, when s_full0 completes);
            // every PV up to tile i is done when tile i's V slot is released.
            auto wait_pv = [&](int i) {
                const uint32_t vseq = seq0 + 2u * (uint32_t)(i - u.t0) + 1u;
                return mbar_wait(bar_free(vseq % ns), (vseq / ns) & 1, s_abort, p.status);
            };
            const int rt = u.rg * 2 + wg;
            const int node = rt * p.NPT + row / p.G, g = row % p.G, h = u.kh * p.G + g;
            const bool row_valid = row < RT && node < u.n;
            const bool warp_active = (wq * 32) < RT && (rt * p.NPT + (wq * 32) / p.G) < u.n;   // row 0 of the warp is valid
            const int nct = u.tiles - 1;
            float m_used = -INFINITY, l = 0.f;
            for (int i = u.t0; i < u.t1; ++i) {
                const int buf = two ? wg : ((i - u.t0) & 1);
                if (two && wg == 0) {
                    if (!(ok = mbar_wait(bar_sfull0, c_s0 & 1, s_abort, p.status))) break;
                    ++c_s0;
                } else {
                    const uint32_t kseq = seq0 + 2u * (uint32_t)(i - u.t0);
                    if (!(ok = mbar_wait(bar_free(kseq % ns), (kseq / ns) & 1, s_abort, p.status))) break;
                }
                if (warp_active) {
                    tc_fence_after();
                    const uint32_t ts = tmem + buf * 128 + lane_addr;
                    // visibility of the tile's 128 keys for this row: context keys below ctx, tree keys by the ancestor bits
                    const bool is_tree = i == nct;
                    const int kv = is_tree ? u.n : min(CB_KT, u.ctx - i * CB_KT);
                    uint32_t vm[4] = {0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu};
                    // A context tile that lies wholly inside the context needs no masks.  Rows that do not exist take the fast
                    // path too: whatever they compute stays in their own row.
                    bool all_vis = !is_tree && kv == CB_KT;
                    if (!all_vis) {
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const int lo = kv - 32 * k;
                            const uint32_t below = lo >= 32 ? 0xFFFFFFFFu : (lo <= 0 ? 0u : ((1u << lo) - 1u));
                            vm[k] = row_valid ? (is_tree ? (mrow[k] & below) : below) : 0u;
                        }
                        all_vis = __all_sync(CB_FULL, !row_valid || (vm[0] & vm[1] & vm[2] & vm[3]) == 0xFFFFFFFFu);
                    }
                    uint32_t sa[32], sb[32];
                    // Single pass, tried first on every tile: P against the reference maximum in use, held back in registers so
                    // that S is still whole if the tile has to be done again.  No row maximum is taken.  The reference exists
                    // to keep 2^(s - reference) and its sums inside fp32 (P is bf16, same exponent range), not for precision,
                    // so the tile's row sum tells all that matters: while it stays below 2^20 no score is more than 20
                    // above the reference and the tile stands; above that (or not finite) the two passes below run instead
                    // and move the reference to the new maximum.  A share's first tile has no reference yet and takes the
                    // largest of its first 32 scores.
                    bool single = false;
                    {
                        uint32_t pk[64];
                        CB_TMEM_LD32(sa, 0, ts);
                        CB_TMEM_WAIT_LD32(sa);
                        CB_TMEM_LD32(sb, 0, ts + 32);
                        if (!all_vis) {
#pragma unroll
                            for (int jx = 0; jx < 32; ++jx)
                                if (!((vm[0] >> jx) & 1u)) sa[jx] = 0xFF800000u;
                        }
                        if (i == u.t0) {
                            float c0 = -INFINITY, c1 = -INFINITY, c2 = -INFINITY, c3 = -INFINITY;
#pragma unroll
                            for (int jx = 0; jx < 32; jx += 4) {
                                c0 = fmaxf(c0, __uint_as_float(sa[jx])); c1 = fmaxf(c1, __uint_as_float(sa[jx + 1]));
                                c2 = fmaxf(c2, __uint_as_float(sa[jx + 2])); c3 = fmaxf(c3, __uint_as_float(sa[jx + 3]));
                            }
                            m_used = fmaxf(fmaxf(c0, c1), fmaxf(c2, c3)) * p.scale_log2;   // -inf if the row sees none of them
                        }
                        const float mu = (m_used == -INFINITY) ? 0.f : m_used;
                        const uint64_t scale2 = f2_pack(p.scale_log2, p.scale_log2), negmu2 = f2_pack(-mu, -mu);
                        uint64_t lsa = f2_pack(0.f, 0.f), lsb = f2_pack(0.f, 0.f);
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint32_t* cur = (c & 1) ? sb : sa;
                            uint32_t* nxt = (c & 1) ? sa : sb;
                            if (c > 0) {
                                CB_TMEM_WAIT_LD32(cur);
                                if (c < 3) CB_TMEM_LD32(nxt, 0, ts + 32 * (c + 1));
                                if (!all_vis) {
#pragma unroll
                                    for (int jx = 0; jx < 32; ++jx)
                                        if (!((vm[c] >> jx) & 1u)) cur[jx] = 0xFF800000u;
                                }
                            }
#pragma unroll
                            for (int jx = 0; jx < 32; jx += 4) {
                                float p0, p1, p2, p3;
                                f2_unpack(f2_fma(f2_pack(__uint_as_float(cur[jx]), __uint_as_float(cur[jx + 1])), scale2, negmu2), p0, p1);
                                f2_unpack(f2_fma(f2_pack(__uint_as_float(cur[jx + 2]), __uint_as_float(cur[jx + 3])), scale2, negmu2), p2, p3);
                                p0 = ex2(p0); p1 = ex2(p1); p2 = ex2(p2); p3 = ex2(p3);
                                lsa = f2_add(lsa, f2_pack(p0, p1));
                                lsb = f2_add(lsb, f2_pack(p2, p3));
                                pk[c * 16 + (jx >> 1)] = pack_bf16(p0, p1);
                                pk[c * 16 + (jx >> 1) + 1] = pack_bf16(p2, p3);
                            }
                        }
                        float l0, l1, l2, l3;
                        f2_unpack(lsa, l0, l1);
                        f2_unpack(lsb, l2, l3);
                        const float lt = (l0 + l1) + (l2 + l3);
                        if (!__any_sync(CB_FULL, row_valid && !(lt <= kRowSumLimit))) {   // rows that do not exist hold anything: they never ask
                            CB_TMEM_ST16(pk, 0, ts);
                            CB_TMEM_ST16(pk, 16, ts + 16);
                            CB_TMEM_ST16(pk, 32, ts + 32);
                            CB_TMEM_ST16(pk, 48, ts + 48);
                            l += lt;
                            tmem_wait_st();
                            single = true;
                        }
                    }
                    if (!single) {
                    // pass 1: row maximum of the visible scores, 32 columns at a time with the next 32 in flight
                    CB_TMEM_LD32(sa, 0, ts);
                    float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t* cur = (c & 1) ? sb : sa;
                        uint32_t* nxt = (c & 1) ? sa : sb;
                        CB_TMEM_WAIT_LD32(cur);
                        if (c < 3) CB_TMEM_LD32(nxt, 0, ts + 32 * (c + 1));
                        if (all_vis) {
#pragma unroll
                            for (int jx = 0; jx < 32; jx += 4) {
                                m0 = fmaxf(m0, __uint_as_float(cur[jx])); m1 = fmaxf(m1, __uint_as_float(cur[jx + 1]));
                                m2 = fmaxf(m2, __uint_as_float(cur[jx + 2])); m3 = fmaxf(m3, __uint_as_float(cur[jx + 3]));
                            }
                        } else {
#pragma unroll
                            for (int jx = 0; jx < 32; ++jx) m0 = fmaxf(m0, ((vm[c] >> jx) & 1u) ? __uint_as_float(cur[jx]) : -INFINITY);
                        }
                    }
                    float mloc = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
                    CB_TMEM_LD32(sa, 0, ts);                     // first columns of pass 2, in flight during the bookkeeping below
                    mloc *= p.scale_log2;
                    // lazy rescaling: keep the reference maximum until the running maximum exceeds it by 2^8 (a tile that
                    // comes here from the single pass holds a score at least 2^13 above it)
                    const bool need = mloc > m_used + 8.0f;
                    const float alpha = need ? ex2(m_used - mloc) : 1.0f;
                    if (need) m_used = mloc;
                    if (i > u.t0 && __any_sync(CB_FULL, need)) {
                        // O must be complete up to the previous tile before it is rescaled
                        if (!(ok = wait_pv(i - 1))) break;
                        tc_fence_after();
#pragma unroll
                        for (int c = 0; c < D / 32; ++c) {
                            uint32_t o[32];
                            CB_TMEM_LD32(o, 0, tm_O + c * 32);
                            tmem_wait_ld();
#pragma unroll
                            for (int jx = 0; jx < 32; ++jx) o[jx] = __float_as_uint(__uint_as_float(o[jx]) * alpha);
                            CB_TMEM_ST32(o, 0, tm_O + c * 32);
                        }
                    }
                    l *= alpha;
                    const float mu = (m_used == -INFINITY) ? 0.f : m_used;
                    // pass 2: P = 2^(s * scale - m), written back over S as packed bf16 (64 scores -> 32 columns)
                    const uint64_t scale2 = f2_pack(p.scale_log2, p.scale_log2), negmu2 = f2_pack(-mu, -mu);
                    uint64_t lsa = f2_pack(0.f, 0.f), lsb = f2_pack(0.f, 0.f);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t pk[16];
                        uint32_t* cur = (c & 1) ? sb : sa;
                        uint32_t* nxt = (c & 1) ? sa : sb;
                        CB_TMEM_WAIT_LD32(cur);
                        if (c < 3) CB_TMEM_LD32(nxt, 0, ts + 32 * (c + 1));
                        if (!all_vis) {
#pragma unroll
                            for (int jx = 0; jx < 32; ++jx)
                                if (!((vm[c] >> jx) & 1u)) cur[jx] = 0xFF800000u;
                        }
#pragma unroll
                        for (int jx = 0; jx < 32; jx += 4) {
                            float p0, p1, p2, p3;
                            f2_unpack(f2_fma(f2_pack(__uint_as_float(cur[jx]), __uint_as_float(cur[jx + 1])), scale2, negmu2), p0, p1);
                            f2_unpack(f2_fma(f2_pack(__uint_as_float(cur[jx + 2]), __uint_as_float(cur[jx + 3])), scale2, negmu2), p2, p3);
                            p0 = ex2(p0); p1 = ex2(p1); p2 = ex2(p2); p3 = ex2(p3);
                            lsa = f2_add(lsa, f2_pack(p0, p1));
                            lsb = f2_add(lsb, f2_pack(p2, p3));
                            pk[jx >> 1] = pack_bf16(p0, p1);
                            pk[(jx >> 1) + 1] = pack_bf16(p2, p3);
                        }
                        CB_TMEM_ST16(pk, 0, ts + c * 16);             // the 32 scores just read become 16 columns of packed P
                    }
                    float l0, l1, l2, l3;
                    f2_unpack(lsa, l0, l1);
                    f2_unpack(lsb, l2, l3);
                    l += (l0 + l1) + (l2 + l3);
                    tmem_wait_st();
                    }
                }
                tc_fence_before();
                mbar_arrive_n(bar_pready(buf), two ? 2u : 1u);   // 256 arrivals per phase: the other half is the watching warpgroup's
            }
            if (!ok) break;
            have = fetch_next();
            // ---- epilogue of this unit's share: O is complete once its last PV has finished
            if (!(ok = wait_pv(u.t1 - 1))) break;
            tc_fence_after();
            if (p.cs > 0) {
                c_m = m_used; c_l = l; c_share = true;         // O stays in TMEM until the exchange below
            } else if (warp_active) {
                const bool whole = u.t0 == 0 && u.t1 == u.tiles;
                if (whole) {
                    const float inv = l > 0.f ? 1.0f / l : 0.f;
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t o[32];
                        CB_TMEM_LD32(o, 0, tm_O + c * 32);
                        tmem_wait_ld();
                        if (row_valid) {
                            __nv_bfloat16* op = p.out + (((size_t)u.b * p.T + node) * p.Hq + h) * D + c * 32;
                            uint32_t w[16];
#pragma unroll
                            for (int k2 = 0; k2 < 16; ++k2) w[k2] = pack_bf16(__uint_as_float(o[2 * k2]) * inv, __uint_as_float(o[2 * k2 + 1]) * inv);
                            st_global_v8(op, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
                            st_global_v8(op + 16, w[8], w[9], w[10], w[11], w[12], w[13], w[14], w[15]);
                        }
                    }
                    if (row_valid && p.lse)
                        p.lse[((size_t)u.b * p.Hq + h) * p.T + node] = l > 0.f ? (m_used + log2f(l)) * 0.6931471805599453f : 0.f;
                } else {
                    const size_t slot = 2 * (size_t)cta + (u.t0 == 0 ? 1 : 0);
                    float* pp = p.part + ((slot * 2 + wg) * CB_MT + row) * (D + 4);
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t o[32];
                        CB_TMEM_LD32(o, 0, tm_O + c * 32);
                        tmem_wait_ld();
                        if (row_valid) {
                            // partial rows are D + 4 floats long: 16-byte aligned only
#pragma unroll
                            for (int v4 = 0; v4 < 8; ++v4)
                                *reinterpret_cast<uint4*>(pp + c * 32 + v4 * 4) = make_uint4(o[v4 * 4], o[v4 * 4 + 1], o[v4 * 4 + 2], o[v4 * 4 + 3]);
                        }
                    }
                    if (row_valid) { pp[D] = m_used; pp[D + 1] = l; }
                }
            }
            tc_fence_before();
            mbar_arrive(bar_ofree(wg));
        }
        if (p.cs > 0 && s_sched->c_has) {
            // ------------------------------------------------------------------ cluster mode: combine the unit's shares
            // Every CTA of the cluster holds the unnormalised rows of its share (O in TMEM, running maximum and sum in
            // registers).  Row i is combined by CTA i % cs: each CTA writes its copy of the row into that CTA's shared memory,
            // arrives on its data barrier, and the owner merges the cs contributions and writes the output row.  The rows are
            // received in the two query tiles when they fit (they are idle from a CTA's last S product on, which the query
            // loader reports), otherwise in the K/V ring (idle from the last P.V on, reported here).
            const int cs = p.cs, rank = cta % cs;
            const int Rv = (min(RT, p.T * p.G) + cs - 1) / cs;   // rows that one CTA may own (rows beyond T nodes never exist)
            const int cb_ = s_sched->c_b, ckh = s_sched->c_kh, cn = s_sched->c_n;
            constexpr uint32_t ROWB = (D + 4) * 4;
            const bool in_q = (uint32_t)(cs * Rv) * ROWB <= 2u * C::Q_BYTES;
            const uint32_t recv = sbase + (in_q ? C::OFF_Q : C::OFF_RING);     // [cs sources][Rv rows][D + 4] floats
            if (ok && !in_q && wg == 0 && row == 0)
                for (int r = 0; r < cs; ++r) mbar_arrive_remote(cluster_addr(bar_cready, (uint32_t)r));
            if (ok) ok = mbar_wait_cluster(bar_cready, 0, s_abort, p.status);
            if (ok && wg == 0) {
                const int dest = row % cs, rl = row / cs;
                const bool valid = row < RT && (row / p.G) < cn;
                const uint32_t ra = cluster_addr(recv + (uint32_t)(rank * Rv + rl) * ROWB, (uint32_t)dest);
                const bool act = (wq * 32) < RT && ((wq * 32) / p.G) < cn;     // row 0 of the warp is valid
                if (act && c_share) {
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t o[32];
                        CB_TMEM_LD32(o, 0, tm_O + c * 32);
                        tmem_wait_ld();
                        if (valid) {
#pragma unroll
                            for (int v4 = 0; v4 < 8; ++v4)
                                st_cluster_v4(ra + (uint32_t)(c * 32 + v4 * 4) * 4u, o[v4 * 4], o[v4 * 4 + 1], o[v4 * 4 + 2], o[v4 * 4 + 3]);
                        }
                    }
                }
                if (valid) st_cluster_v4(ra + D * 4u, __float_as_uint(c_share ? c_m : -INFINITY), __float_as_uint(c_share ? c_l : 0.f), 0u, 0u);
                mbar_arrive_remote(cluster_addr(bar_cdata, (uint32_t)dest));
            }
            if (ok) ok = mbar_wait_cluster(bar_cdata, 0, s_abort, p.status);
            if (ok) {
                // up to 256 threads: tpr threads per row, each a run of D / tpr >= 8 columns in groups of 8
                int tpr = D / 8;                                 // a power of two
                while (tpr * Rv > 256) tpr >>= 1;
                const int t = wg * 128 + row, rl = t / tpr, sub = t % tpr;
                const int gr = rl * cs + rank, node = gr / p.G, h = ckh * p.G + gr % p.G;
                if (rl < Rv && gr < RT && node < cn) {
                    float mx = -INFINITY;
                    for (int sidx = 0; sidx < cs; ++sidx) {
                        float ms;
                        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(ms) : "r"(recv + (uint32_t)(sidx * Rv + rl) * ROWB + D * 4u));
                        mx = fmaxf(mx, ms);
                    }
                    float wsum = 0.f;
                    for (int sidx = 0; sidx < cs; ++sidx) {
                        float ms, ls;
                        asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(ms), "=f"(ls) : "r"(recv + (uint32_t)(sidx * Rv + rl) * ROWB + D * 4u));
                        wsum += (ms == -INFINITY) ? 0.f : ex2(ms - mx) * ls;
                    }
                    const float inv = wsum > 0.f ? 1.0f / wsum : 0.f;
                    const int cols = D / tpr;
                    for (int g8 = 0; g8 < cols; g8 += 8) {
                        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                        for (int sidx = 0; sidx < cs; ++sidx) {
                            const uint32_t base = recv + (uint32_t)(sidx * Rv + rl) * ROWB;
                            float ms;
                            asm volatile("ld.shared.f32 %0, [%1];" : "=f"(ms) : "r"(base + D * 4u));
                            if (ms == -INFINITY) continue;      // that CTA had no tiles: its row was not written
                            const float w = ex2(ms - mx);
                            float v[8];
                            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3])
                                         : "r"(base + (uint32_t)(sub * cols + g8) * 4u));
                            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
                                         : "r"(base + (uint32_t)(sub * cols + g8 + 4) * 4u));
#pragma unroll
                            for (int k = 0; k < 8; ++k) acc[k] += w * v[k];
                        }
                        __nv_bfloat16* op = p.out + (((size_t)cb_ * p.T + node) * p.Hq + h) * D + sub * cols + g8;
                        *reinterpret_cast<uint4*>(op) = make_uint4(pack_bf16(acc[0] * inv, acc[1] * inv), pack_bf16(acc[2] * inv, acc[3] * inv),
                                                                   pack_bf16(acc[4] * inv, acc[5] * inv), pack_bf16(acc[6] * inv, acc[7] * inv));
                    }
                    if (sub == 0 && p.lse)
                        p.lse[((size_t)cb_ * p.Hq + h) * p.T + node] = wsum > 0.f ? (mx + log2f(wsum)) * 0.6931471805599453f : 0.f;
                }
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

// Merge pass: block (c, *) looks at the unit that CTA c of the attention kernel started but did not finish,
// and combines the partials that CTA c and the following CTAs left for it.  One warp per output row.
// Every block waits for the attention grid before it leaves, also the ones that find nothing to merge: the next kernel
// in the stream is ordered behind this grid only, so this grid must not end while the attention kernel still runs.
template <int D>
__global__ void __launch_bounds__(256) cb_attn_merge_kernel(const CbAttnParams p) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the wait comes below, after the set-up that reads inputs only
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int c = blockIdx.x;
    const long long tot = cb_sched_total(p, lane);
    bool nothing = tot <= 0;
    long long g0 = 0, g1 = 0, pre = 0, ustart = 0;
    int b = 0, rg = 0, j = 0, vt = 1;
    CbSeqShape s = {};
    if (!nothing) {
        g0 = cb_range_start(tot, p.nc, c); g1 = cb_range_start(tot, p.nc, c + 1);
        nothing = g1 <= g0 || g1 >= tot;                      // empty range, or the last range
    }
    if (!nothing) {
        cb_sched_locate(p, g1 - 1, lane, &rg, &b, &pre);
        s = cb_seq_shape(p, b);
        const long long off = g1 - 1 - pre;
        vt = s.tiles + s.ov;                                  // positions of one unit: padding, then its key tiles
        j = (int)(off / vt);
        ustart = pre + (long long)j * vt;
        const long long first_tile = ustart + s.ov;
        nothing = (int)(off - (long long)j * vt) == vt - 1    // the unit ends with this range
                  || first_tile < g0                          // started by an earlier CTA: that CTA's block merges it
                  || first_tile >= g1;                        // only padding so far: the next CTA starts the unit
    }
    if (nothing) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        return;
    }
    const int c_last = cb_cta_of(tot, p.nc, ustart + vt - 1);
    const int kh = j;                                         // units of (row group, sequence) are its kv heads
    const int nrt = p.MT == 1 ? 1 : min(2, s.mtn - 2 * rg);
    const int RT = p.NPT * p.G;
    constexpr int PER = D / 32;
    // partial slots of this unit, listed once per block: CTA c's "started here" slot, then the "continued" slots of
    // the following CTAs that have a non-empty range
    __shared__ int s_slot[CB_ATTN_MAX_CTAS];
    __shared__ int s_nparts;
    if (warp == 0) {
        int np = 0;
        for (int base = c; base <= c_last; base += 32) {
            const int cc = base + lane;
            const bool valid = cc <= c_last && cb_range_start(tot, p.nc, cc) < cb_range_start(tot, p.nc, cc + 1);
            const uint32_t m = __ballot_sync(CB_FULL, valid);
            if (valid) s_slot[np + __popc(m & ((1u << lane) - 1u))] = 2 * cc + (cc == c ? 1 : 0);
            np += __popc(m);
        }
        if (lane == 0) s_nparts = np;
    }
    __syncthreads();
    const int nparts = s_nparts;
    asm volatile("griddepcontrol.wait;" ::: "memory");       // the attention grid has finished and its writes are visible
    const size_t rstride = (size_t)(D + 4), sstride = (size_t)2 * CB_MT * rstride;
    for (int r2 = blockIdx.y * 8 + warp; r2 < nrt * CB_MT; r2 += gridDim.y * 8) {
        const int wg = r2 / CB_MT, row = r2 % CB_MT;
        const int node = (rg * 2 + wg) * p.NPT + row / p.G, h = kh * p.G + row % p.G;
        if (row >= RT || node >= s.n) continue;
        const float* base = p.part + ((size_t)wg * CB_MT + row) * rstride;
        // lanes fetch the running maxima of up to 32 parts at a time
        float M = -INFINITY;
        for (int k0 = 0; k0 < nparts; k0 += 32) {
            const int k = k0 + lane;
            const float ms = k < nparts ? base[(size_t)s_slot[k] * sstride + D] : -INFINITY;
            M = fmaxf(M, ms);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(CB_FULL, M, o));
        float o[PER], Lsum = 0.f;
#pragma unroll
        for (int d = 0; d < PER; ++d) o[d] = 0.f;
        for (int k = 0; k < nparts; ++k) {
            const float* pp = base + (size_t)s_slot[k] * sstride;
            const float ms = pp[D];
            const float w = ms == -INFINITY ? 0.f : exp2f(ms - M);
            Lsum = fmaf(w, pp[D + 1], Lsum);
            if constexpr (PER == 4) {
                const float4 v = *reinterpret_cast<const float4*>(pp + lane * 4);
                o[0] = fmaf(w, v.x, o[0]); o[1] = fmaf(w, v.y, o[1]); o[2] = fmaf(w, v.z, o[2]); o[3] = fmaf(w, v.w, o[3]);
            } else {
                const float2 v = *reinterpret_cast<const float2*>(pp + lane * 2);
                o[0] = fmaf(w, v.x, o[0]); o[1] = fmaf(w, v.y, o[1]);
            }
        }
        const float inv = Lsum > 0.f ? 1.f / Lsum : 0.f;
        __nv_bfloat16* op = p.out + (((size_t)b * p.T + node) * p.Hq + h) * D + lane * PER;
#pragma unroll
        for (int d = 0; d < PER; ++d) op[d] = __float2bfloat16_rn(o[d] * inv);
        if (p.lse && lane == 0) p.lse[((size_t)b * p.Hq + h) * p.T + node] = Lsum > 0.f ? (M + log2f(Lsum)) * 0.6931471805599453f : 0.f;
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

// 4-D view (d, head, row, block) of a [blocks, rows, heads, D] bf16 tensor; box = 64 dims x box_heads x box_rows.
bool encode_map(CUtensorMap* m, const void* base, int D, int heads, int rows, long blocks, int box_heads, int box_rows) {
    EncodeTiledFn enc = get_encode();
    if (!enc) { fprintf(stderr, "cacheback: cuTensorMapEncodeTiled entry point not found\n"); return false; }
    cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)heads, (cuuint64_t)rows, (cuuint64_t)blocks};
    cuuint64_t strides[3] = {(cuuint64_t)D * 2, (cuuint64_t)heads * D * 2, (cuuint64_t)rows * heads * D * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)box_heads, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           // a head's row is D * 2 bytes contiguous and is fetched as 128-byte halves by two boxes: with D = 128 let the
                           // first one bring the whole row into L2
                           D >= 128 ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
        fprintf(stderr, "cacheback: tensor map encode failed (%d): D=%d heads=%d rows=%d blocks=%ld base=%p\n", (int)r, D, heads, rows,
                blocks, base);
    return r == CUDA_SUCCESS;
}

// Cluster mode is for launches with few units, where the stream-K split would make every unit a shared one: all trees fit
// one row tile (so a unit is one (sequence, kv head)), units times a cluster size of 8, 4 or 2 does not exceed the SMs, that
// many clusters can be resident at once, and a CTA's part of a unit (tiles / cs) is shorter than a CTA's range under the
// stream-K split plus what its partials and merge pass cost (about three tiles).  Returns the cluster size or 0.
template <int D>
int pick_cluster_size(const CbAttnParams& p, int num_sms) {
    if (p.MT != 1) return 0;
    const long long units = (long long)p.B * p.Hkv;
    for (int cs = 8; cs >= 2; cs >>= 1) {
        if (units * cs > num_sms) continue;
        const long long in_cluster = (p.max_tiles + cs - 1) / cs, stream_k = units * (p.max_tiles + 2) / num_sms + 3;
        if (in_cluster >= stream_k) continue;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(units * cs)); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = Cfg<D>::SMEM_ALLOC;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = (unsigned)cs; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        int nclusters = 0;
        if (cudaOccupancyMaxActiveClusters(&nclusters, cb_attn_tc_kernel<D>, &cfg) != cudaSuccess) { (void)cudaGetLastError(); continue; }
        if (nclusters >= units) return cs;
    }
    return 0;
}

// Host state of the launcher, per device and guarded: the opt-in to large dynamic shared memory is a per-device function
// attribute, and the cluster size chosen for a shape is remembered for the shapes seen last.
constexpr int kMaxDevices = 64;
constexpr int kShapeMemo = 8;
struct ShapeMemo { int key[6]; int cs; };
std::mutex g_launch_mutex;
bool g_attr_set[2][kMaxDevices];
ShapeMemo g_shape_memo[kShapeMemo];
int g_shape_used = 0, g_shape_next = 0;

int g_pairs[kMaxDevices];              // CTA pairs that can be resident at once (0 = not asked yet, -1 = none)

// On request (CB_FLAG_ATTN_CTA_PAIRS), launches with two or more row tiles per unit and head_dim 128 run as pairs of CTAs
// (cb_attn_pair.cuh): as many pairs as can be resident together, each taking an equal range of the global tile sequence.
cb_status launch_pairs(CbAttnParams p, const TcMaps& maps, cudaStream_t st, int num_sms, int device, bool* done) {
    *done = false;
    const int di = device >= 0 && device < kMaxDevices ? device : -1;
    if (di < 0) return CB_OK;
    int npairs;
    {
        std::lock_guard<std::mutex> lock(g_launch_mutex);
        if (g_pairs[di] == 0) {
            g_pairs[di] = -1;
            if (cudaFuncSetAttribute(cb_attn_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PairCfg::SMEM_ALLOC) == cudaSuccess) {
                cudaLaunchConfig_t cfg = {};
                cfg.gridDim = dim3((unsigned)(num_sms / 2 * 2)); cfg.blockDim = dim3(kPairThreads); cfg.dynamicSmemBytes = PairCfg::SMEM_ALLOC;
                cudaLaunchAttribute at[1];
                at[0].id = cudaLaunchAttributeClusterDimension;
                at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
                cfg.attrs = at; cfg.numAttrs = 1;
                int n = 0;
                if (cudaOccupancyMaxActiveClusters(&n, cb_attn_pair_kernel, &cfg) == cudaSuccess && n > 0) g_pairs[di] = n < num_sms / 2 ? n : num_sms / 2;
            }
            (void)cudaGetLastError();
        }
        npairs = g_pairs[di];
    }
    if (npairs <= 0) return CB_OK;
    // The units that stream the same keys (the row groups of one (sequence, kv head)) lie 1 / row-groups of the tile sequence
    // apart: with a number of ranges that is a multiple of the row groups they are at the same point of their ranges at the
    // same time, so that one fetch from HBM serves all of them.
    const int row_groups = (p.MT + 1) / 2;
    if (npairs > row_groups) npairs -= npairs % row_groups;
    p.nc = npairs; p.cs = 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * npairs)); cfg.blockDim = dim3(kPairThreads); cfg.dynamicSmemBytes = PairCfg::SMEM_ALLOC; cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 2;
    CB_CUDA(cudaLaunchKernelEx(&cfg, cb_attn_pair_kernel, p, maps));
    CB_CUDA(cb_launch_pdl(cb_attn_merge_kernel<128>, dim3(p.nc, 4), dim3(256), 0, st, p));
    cb_count_launch(2);
    CB_CUDA(cudaGetLastError());
    *done = true;
    return CB_OK;
}

template <int D>
cb_status launch(CbAttnParams p, const TcMaps& maps, cudaStream_t st, int num_sms, int device) {
    {
        std::lock_guard<std::mutex> lock(g_launch_mutex);
        const int di = device >= 0 && device < kMaxDevices ? device : -1;
        if (di < 0 || !g_attr_set[D == 128][di]) {
            CB_CUDA(cudaFuncSetAttribute(cb_attn_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<D>::SMEM_ALLOC));
            if (di >= 0) g_attr_set[D == 128][di] = true;
        }
        // the choice depends on the shape only
        const int key[6] = {p.B, p.Hkv, p.MT, num_sms, p.max_tiles, D * kMaxDevices + (di < 0 ? 0 : di)};
        int found = -1;
        for (int i = 0; i < g_shape_used && found < 0; ++i) {
            bool same = true;
            for (int k = 0; k < 6; ++k) same = same && g_shape_memo[i].key[k] == key[k];
            if (same) found = i;
        }
        if (found < 0) {
            found = g_shape_used < kShapeMemo ? g_shape_used++ : (g_shape_next++ % kShapeMemo);
            for (int k = 0; k < 6; ++k) g_shape_memo[found].key[k] = key[k];
            g_shape_memo[found].cs = pick_cluster_size<D>(p, num_sms);
        }
        p.cs = g_shape_memo[found].cs;
    }
    if (p.cs > 0) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(p.B * p.Hkv * p.cs)); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = Cfg<D>::SMEM_ALLOC; cfg.stream = st;
        cudaLaunchAttribute at[2];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = (unsigned)p.cs; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at; cfg.numAttrs = 2;
        CB_CUDA(cudaLaunchKernelEx(&cfg, cb_attn_tc_kernel<D>, p, maps));
        cb_count_launch(1);
        return CB_OK;
    }
    CB_CUDA(cb_launch_pdl(cb_attn_tc_kernel<D>, dim3(p.nc), dim3(kThreads), Cfg<D>::SMEM_ALLOC, st, p, maps));
    CB_CUDA(cb_launch_pdl(cb_attn_merge_kernel<D>, dim3(p.nc, 4), dim3(256), 0, st, p));
    cb_count_launch(2);
    CB_CUDA(cudaGetLastError());
    return CB_OK;
}

}  // namespace

// Encoding five tensor maps costs several microseconds of host time, which matters at batch 1: the maps of the most
// recent argument sets are kept (they depend only on the base pointers and the shape).
namespace {
struct MapKey {
    const void *q, *k_pool, *v_pool, *k_tree, *v_tree;
    int D, Hq, Hkv, P, T, B, G, NPT, num_pages;
    bool operator==(const MapKey& o) const {
        return q == o.q && k_pool == o.k_pool && v_pool == o.v_pool && k_tree == o.k_tree && v_tree == o.v_tree && D == o.D && Hq == o.Hq &&
               Hkv == o.Hkv && P == o.P && T == o.T && B == o.B && G == o.G && NPT == o.NPT && num_pages == o.num_pages;
    }
};
constexpr int kMapCache = 16;
MapKey g_map_keys[kMapCache];
TcMaps g_map_vals[kMapCache];
int g_map_used = 0, g_map_next = 0;
std::mutex g_map_mutex;
}  // namespace

cb_status cb_attn_launch_tensor(cb_ctx* ctx, const CbAttnParams& p, cudaStream_t st) {
    if (p.P != 16) return CB_ERR_UNSUPPORTED;
    const bool pairs = p.D == 128 && p.MT > 1 && (ctx->cfg.flags & CB_FLAG_ATTN_CTA_PAIRS);
    const MapKey key = {p.q, p.k_pool, p.v_pool, p.k_tree, p.v_tree, p.D, p.Hq, p.Hkv, p.P, p.T, p.B, p.G, p.NPT, p.num_pages};
    TcMaps maps;
    bool hit = false;
    {
        std::lock_guard<std::mutex> lock(g_map_mutex);
        for (int i = 0; i < g_map_used && !hit; ++i)
            if (g_map_keys[i] == key) { maps = g_map_vals[i]; hit = true; }
    }
    if (!hit) {
        if (!encode_map(&maps.k_pool, p.k_pool, p.D, p.Hkv, p.P, p.num_pages, 1, 16)) return CB_ERR_CUDA;
        if (!encode_map(&maps.v_pool, p.v_pool, p.D, p.Hkv, p.P, p.num_pages, 1, 16)) return CB_ERR_CUDA;
        if (!encode_map(&maps.k_tree, p.k_tree, p.D, p.Hkv, p.T, p.B, 1, 16)) return CB_ERR_CUDA;
        if (!encode_map(&maps.v_tree, p.v_tree, p.D, p.Hkv, p.T, p.B, 1, 16)) return CB_ERR_CUDA;
        if (!encode_map(&maps.q, p.q, p.D, p.Hq, p.T, p.B, p.G, p.NPT)) return CB_ERR_CUDA;
        std::lock_guard<std::mutex> lock(g_map_mutex);
        const int slot = g_map_used < kMapCache ? g_map_used++ : (g_map_next++ % kMapCache);
        g_map_keys[slot] = key;
        g_map_vals[slot] = maps;
    }
    if (pairs) {
        bool done = false;
        const cb_status r = launch_pairs(p, maps, st, ctx->num_sms, ctx->device, &done);
        if (r != CB_OK || done) return r;
    }
    return p.D == 128 ? launch<128>(p, maps, st, ctx->num_sms, ctx->device) : launch<64>(p, maps, st, ctx->num_sms, ctx->device);
}
