// Order-free form of the bulk update (prompt initialisation, Section 3.3), used by cb_update_bulk when the caller has
// attached scratch memory (cb_bulk_scratch_attach).  Included by cb_table.cu after the table helpers.
//
// When no leader can be evicted during a run of insertions and a stored follower is refreshed by re-insertion, the state
// after the run does not depend on the order of the windows (Section 3.1: both lists are least-recently-used lists, and the
// content of such a list after a run is the most recently touched distinct items):
//   * a leader's stamp is that of its last window in the run;
//   * its followers are the FC distinct followers with the latest last occurrence, taken over what the entry held before
//     (all older than the run) and the run's windows; a follower's stamp is that of its last occurrence.
// So the run is reduced first, with one thread per window and no warp owning a leader's history:
//   1. every window finds or claims the slot of its (leader, follower) pair in a scratch hash table and of its leader in a
//      second one, and raises their "last index" with atomicMax; the thread that creates a pair counts it for its leader;
//   2. every leader takes a range of the group array (a block scan over 256 slots, then one atomicAdd on a cursor),
//   3. every pair writes itself into its leader's range;
//   4. the leaders are applied to the table, 32 slots per warp: a leader that is not in the table yet and has few followers
//      is written by one lane alone (entry id from the leader count, key, followers, stamps), every other one by the whole
//      warp, which finds or creates the entry, sets the leader's stamp, and inserts the leader's pairs with the usual
//      follower-list code, or only the FC latest of them when there are more (threshold by bisection on the last index).
//      Those FC are newer than anything stored, so inserting them in any order evicts stored followers oldest first and
//      never one of them: the result is the sequential one.  Which place a follower takes in the entry, and which entry id
//      a leader gets, may differ from the sequential run; nothing reads either.
// Keys are compared by reading the tokens at the position a slot's first claimant recorded.  All loops are bounded.
#pragma once

namespace {

struct BulkFreeHdr {          // head of the scratch buffer (device)
    uint32_t m_total;         // windows of all order-free sequences of this call
    uint32_t s_eff;           // slots in use of either hash table: a power of two >= 2 * m_total
    uint32_t cursor;          // next free place of the group array
    uint32_t pad[13];
};

struct BulkFreeView {
    BulkFreeHdr* hdr;
    uint32_t* off;            // [B + 1] first window of every sequence among the order-free ones
    unsigned long long* prep; // [S] pair slots: (sequence << 32) | (window position + 1) of the first claimant, 0 = empty
    uint32_t* plast;          // [S] last index + 1 of the pair within its sequence's run
    uint32_t* pl;             // [S] the pair's leader slot
    unsigned long long* lrep; // [S] leader slots, as prep
    uint32_t* llast;          // [S]
    uint32_t* lcount;         // [S] distinct pairs of the leader
    uint32_t* lbase;          // [S] start of the leader's range in group
    uint32_t* lfill;          // [S]
    uint32_t* group;          // [W] pair slots grouped by leader
    uint32_t S, W;            // capacity: slots (power of two), windows (S / 2)
};

struct BulkFreeLayout { size_t off_off, off_prep, off_plast, off_pl, off_lrep, off_llast, off_lcount, off_lbase, off_lfill, off_group, total; };

inline BulkFreeLayout bulk_free_layout(uint32_t S, int B) {
    BulkFreeLayout L;
    size_t o = sizeof(BulkFreeHdr);
    auto take = [&](size_t bytes) { const size_t at = o; o += (bytes + 255) / 256 * 256; return at; };
    L.off_off = take((size_t)(B + 1) * 4);
    L.off_prep = take((size_t)S * 8); L.off_plast = take((size_t)S * 4); L.off_pl = take((size_t)S * 4);
    L.off_lrep = take((size_t)S * 8); L.off_llast = take((size_t)S * 4); L.off_lcount = take((size_t)S * 4);
    L.off_lbase = take((size_t)S * 4); L.off_lfill = take((size_t)S * 4);
    L.off_group = take((size_t)(S / 2) * 4);
    L.total = o;
    return L;
}

inline BulkFreeView bulk_free_view(void* scratch, uint32_t S, int B) {
    const BulkFreeLayout L = bulk_free_layout(S, B);
    char* p = static_cast<char*>(scratch);
    BulkFreeView v;
    v.hdr = reinterpret_cast<BulkFreeHdr*>(p);
    v.off = reinterpret_cast<uint32_t*>(p + L.off_off);
    v.prep = reinterpret_cast<unsigned long long*>(p + L.off_prep);
    v.plast = reinterpret_cast<uint32_t*>(p + L.off_plast);
    v.pl = reinterpret_cast<uint32_t*>(p + L.off_pl);
    v.lrep = reinterpret_cast<unsigned long long*>(p + L.off_lrep);
    v.llast = reinterpret_cast<uint32_t*>(p + L.off_llast);
    v.lcount = reinterpret_cast<uint32_t*>(p + L.off_lcount);
    v.lbase = reinterpret_cast<uint32_t*>(p + L.off_lbase);
    v.lfill = reinterpret_cast<uint32_t*>(p + L.off_lfill);
    v.group = reinterpret_cast<uint32_t*>(p + L.off_group);
    v.S = S; v.W = S / 2;
    return v;
}

constexpr int kBulkFreeMaxBatch = 4096;      // the plan kernel keeps one word per sequence in shared memory

// Plan: what cb_bulk_plan_kernel decides, plus which of the qualifying sequences fit the scratch (taken in order) and
// where their windows start in the global numbering.  One block.
__global__ void __launch_bounds__(1024) cb_bulk_free_plan_kernel(CbTables t, int B, const int32_t* __restrict__ n_old,
                                                                const int32_t* __restrict__ n_new, BulkPlan* plan, BulkFreeView v,
                                                                unsigned long long* counters) {
    CB_PDL_ENTRY();
    __shared__ uint32_t s_nwin[kBulkFreeMaxBatch];
    const int w = t.LL + t.FL;
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
        const CbSeq s = cb_seq(t, b);
        const int first = max(0, n_old[b] - w + 1);
        const int nwin = max(0, n_new[b] - w + 1 - first);
        BulkPlan p;
        p.clock0 = s.hdr[0];
        p.first = (uint32_t)first;
        p.nwin = (uint32_t)nwin;
        p.parallel = (nwin >= 64 && (unsigned long long)s.hdr[1] + (unsigned long long)nwin <= (unsigned long long)t.LC) ? 1u : 0u;
        if (p.parallel) s.hdr[0] = p.clock0 + (uint32_t)nwin;
        plan[b] = p;
        s_nwin[b] = (p.parallel && t.refresh) ? (uint32_t)nwin : 0u;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t at = 0;
        unsigned long long ins = 0;
        for (int b = 0; b < B; ++b) {
            v.off[b] = at;
            const uint32_t n = s_nwin[b];
            if (n > 0 && at + n <= v.W) {
                at += n;
                ins += n;
                plan[b].parallel = 2u;
            }
        }
        v.off[B] = at;
        uint32_t s_eff = 1024;
        while (s_eff < 2u * at) s_eff <<= 1;
        v.hdr->m_total = at;
        v.hdr->s_eff = min(s_eff, v.S);
        v.hdr->cursor = 0;
        if (ins) atomicAdd(&counters[CB_CNT_INSERTS], ins);
    }
}

__global__ void cb_bulk_free_clear_kernel(BulkFreeView v) {
    CB_PDL_ENTRY();
    if (v.hdr->m_total == 0) return;
    const uint32_t S = v.hdr->s_eff;
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < S; i += gridDim.x * blockDim.x) {
        v.prep[i] = 0ull; v.plast[i] = 0u; v.lrep[i] = 0ull; v.llast[i] = 0u; v.lcount[i] = 0u;
    }
}

__device__ __forceinline__ uint64_t bulk_free_hash(int b, const int32_t* p, int n) {
    uint64_t h = 0x9E3779B97F4A7C15ull ^ ((uint64_t)(uint32_t)b * 0xD6E8FEB86659FD93ull);
    for (int j = 0; j < n; ++j) { h = (h ^ (uint32_t)p[j]) * 0xFF51AFD7ED558CCDull; h ^= h >> 32; }
    h ^= h >> 33; h *= 0xC4CEB9FE1A85EC53ull; h ^= h >> 33;
    return h;
}

// Finds or claims the slot of the n-token key at position i of sequence b (row = that sequence's tokens).  Returns the
// slot, or 0xFFFFFFFF when every slot was visited (excluded by the sizing: at most half of the slots are ever taken).
__device__ __forceinline__ uint32_t bulk_free_slot(unsigned long long* rep, uint32_t S, const int32_t* row, int b, uint32_t i, int n, bool* created) {
    const unsigned long long me = ((unsigned long long)(uint32_t)b << 32) | (unsigned long long)(i + 1u);
    uint32_t slot = (uint32_t)bulk_free_hash(b, row + i, n) & (S - 1u);
    *created = false;
    for (uint32_t probes = 0; probes < S; ++probes) {
        unsigned long long cur = __ldcg(&rep[slot]);
        if (cur == 0ull) {
            cur = atomicCAS(&rep[slot], 0ull, me);
            if (cur == 0ull) { *created = true; return slot; }
        }
        if ((uint32_t)(cur >> 32) == (uint32_t)b) {
            const int32_t* q = row + ((uint32_t)cur - 1u);
            bool same = true;
            for (int j = 0; j < n; ++j) same = same && (q[j] == row[i + j]);
            if (same) return slot;
        }
        slot = (slot + 1u) & (S - 1u);
    }
    return 0xFFFFFFFFu;
}

// global window number -> sequence (off is non-decreasing; sequences outside the order-free path have empty ranges)
__device__ __forceinline__ int bulk_free_seq_of(const uint32_t* off, int B, uint32_t g) {
    int lo = 0, hi = B - 1;                                    // the last b with off[b] <= g
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (off[mid] <= g) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// 1. one thread per window
__global__ void __launch_bounds__(256) cb_bulk_free_reduce_kernel(CbTables t, int B, const int32_t* __restrict__ tokens, int64_t row_stride,
                                                                  const BulkPlan* __restrict__ plan, BulkFreeView v, uint32_t* status) {
    CB_PDL_ENTRY();
    const uint32_t M = v.hdr->m_total, S = v.hdr->s_eff;
    const int w = t.LL + t.FL;
    for (uint32_t g = blockIdx.x * blockDim.x + threadIdx.x; g < M; g += gridDim.x * blockDim.x) {
        const int b = bulk_free_seq_of(v.off, B, g);
        const uint32_t k = g - v.off[b];
        const uint32_t i = plan[b].first + k;
        const int32_t* row = tokens + (size_t)b * row_stride;
        bool made_l, made_p;
        const uint32_t ls = bulk_free_slot(v.lrep, S, row, b, i, t.LL, &made_l);
        const uint32_t ps = ls == 0xFFFFFFFFu ? ls : bulk_free_slot(v.prep, S, row, b, i, w, &made_p);
        if (ps == 0xFFFFFFFFu) { atomicCAS(status, 0u, (uint32_t)CB_ERR_PROBE_LIMIT); continue; }
        atomicMax(&v.llast[ls], k + 1u);
        if (made_p) { v.pl[ps] = ls; atomicAdd(&v.lcount[ls], 1u); }
        atomicMax(&v.plast[ps], k + 1u);
    }
}

// 2. every leader takes its range of the group array (one atomicAdd per block and 256 slots: their ranges lie side by side)
__global__ void __launch_bounds__(256) cb_bulk_free_ranges_kernel(BulkFreeView v) {
    CB_PDL_ENTRY();
    if (v.hdr->m_total == 0) return;
    const uint32_t S = v.hdr->s_eff;                             // a multiple of 256
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __shared__ uint32_t s_tot[8], s_start;
    for (uint32_t i0 = blockIdx.x * 256u; i0 < S; i0 += gridDim.x * 256u) {
        const uint32_t i = i0 + threadIdx.x;
        const uint32_t n = v.lrep[i] != 0ull ? v.lcount[i] : 0u;
        uint32_t incl = n;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t up = __shfl_up_sync(CB_FULL, incl, o);
            if (lane >= o) incl += up;
        }
        if (lane == 31) s_tot[warp] = incl;
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t total = 0;
            for (int k = 0; k < 8; ++k) { const uint32_t c = s_tot[k]; s_tot[k] = total; total += c; }
            s_start = total ? atomicAdd(&v.hdr->cursor, total) : 0u;
        }
        __syncthreads();
        if (n) { v.lbase[i] = s_start + s_tot[warp] + incl - n; v.lfill[i] = 0u; }
        __syncthreads();                                         // the shared words are rewritten by the next round
    }
}

// 3. every pair goes into its leader's range
__global__ void __launch_bounds__(256) cb_bulk_free_scatter_kernel(BulkFreeView v) {
    CB_PDL_ENTRY();
    if (v.hdr->m_total == 0) return;
    const uint32_t S = v.hdr->s_eff;
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < S; i += gridDim.x * blockDim.x) {
        if (v.prep[i] == 0ull) continue;
        const uint32_t ls = v.pl[i];
        const uint32_t at = v.lbase[ls] + atomicAdd(&v.lfill[ls], 1u);
        if (at < v.W) v.group[at] = i;
    }
}

// 4. one warp per leader: entry, leader stamp, followers.  A warp takes 32 leader slots at a time.  What does not need the
// whole warp is done by the lanes side by side, each for its own slot: the slot's figures, the leader's tokens and hash, a
// prefetch of its index bucket and of its part of the group array, and at the end the publication of the new entries in
// the index (one fence for all of them instead of one each).
__global__ void __launch_bounds__(256) cb_bulk_free_apply_kernel(CbTables t, int B, const int32_t* __restrict__ tokens, int64_t row_stride,
                                                                 const BulkPlan* __restrict__ plan, BulkFreeView v, uint32_t* status,
                                                                 unsigned long long* counters) {
    CB_PDL_ENTRY();
    if (v.hdr->m_total == 0) return;
    const uint32_t S = v.hdr->s_eff;
    const int lane = threadIdx.x & 31;
    const uint32_t gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nw = (gridDim.x * blockDim.x) >> 5;
    TblCounters cnt = {0, 0, 0, 0};
    for (uint32_t base = gw * 32u; base < S; base += nw * 32u) {
        // ---- per lane: this lane's slot
        const unsigned long long my_rep = v.lrep[base + lane];
        const bool occ = my_rep != 0ull && (int)(my_rep >> 32) < B;
        uint32_t my_n = 0, my_gbase = 0, my_last = 0;
        int32_t my_k[CB_MAX_LL] = {0, 0, 0, 0};
        uint64_t my_h = 0;
        if (occ) {
            const int b = (int)(my_rep >> 32);
            const int32_t* row = tokens + (size_t)b * row_stride + ((uint32_t)my_rep - 1u);
            my_n = v.lcount[base + lane]; my_gbase = v.lbase[base + lane]; my_last = v.llast[base + lane];
            for (int j = 0; j < t.LL; ++j) my_k[j] = row[j];
            my_h = cb_hash4(my_k[0], my_k[1], my_k[2], my_k[3], t.LL);
            const uint32_t* bucket = cb_seq(t, b).index + (size_t)cb_hash_bucket(my_h, t.nslots) * 32;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(bucket));
            if (my_gbase < v.W) asm volatile("prefetch.global.L2 [%0];" ::"l"(v.group + my_gbase));
        }
        // what this lane's leader still needs at the end: its new entry's index word and the slot found free for it
        uint32_t my_word = 0, my_free = 0xFFFFFFFFu;
        // ---- per lane: the common case of a prompt, a leader that is not in the table yet and has a few followers, is done
        // by its lane alone (32 leaders side by side instead of one after the other): the home bucket shows no index word
        // with the leader's tag and has room, so the leader is absent and its word goes there; the lane takes an entry and
        // writes it.  Every other case (a word with the tag, a full bucket, many followers) is left to the whole warp below.
        bool handled = false;
        if (occ && my_n <= (uint32_t)min(t.FC, 8)) {
            const int b = (int)(my_rep >> 32);
            const CbSeq s = cb_seq(t, b);
            const uint32_t bucket = cb_hash_bucket(my_h, t.nslots), tag = cb_hash_tag(my_h);
            const uint4* bp = reinterpret_cast<const uint4*>(s.index + (size_t)bucket * 32);
            uint32_t w[32];
#pragma unroll
            for (int q = 0; q < 8; ++q) { const uint4 x = __ldcg(bp + q); w[4 * q] = x.x; w[4 * q + 1] = x.y; w[4 * q + 2] = x.z; w[4 * q + 3] = x.w; }
            bool tagged = false, has_empty = false;
            int first_free = -1;
#pragma unroll
            for (int q = 0; q < 32; ++q) {
                const bool emp = w[q] == CB_IDX_EMPTY, tomb = w[q] == CB_IDX_TOMB;
                has_empty = has_empty || emp;
                if ((emp || tomb) && first_free < 0) first_free = q;
                tagged = tagged || (!emp && !tomb && (w[q] >> CB_EID_BITS) == tag);
            }
            if (!tagged && has_empty && my_gbase + my_n <= v.W) {
                const uint32_t got = atomicAdd(&s.hdr[1], 1u);
                if (got < (uint32_t)t.LC) {                     // anything else is excluded by the plan
                    const uint32_t clock0 = plan[b].clock0;
                    const int32_t* row = tokens + (size_t)b * row_stride;
                    uint32_t* e = s.entries + (size_t)got * t.E;
                    for (int j = 0; j < t.LL; ++j) e[j] = (uint32_t)my_k[j];
                    // loads first, level by level, so that the followers' round trips overlap
                    uint32_t ps[8], fl[8], fp[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) ps[j] = (uint32_t)j < my_n ? v.group[my_gbase + j] : 0u;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        fl[j] = (uint32_t)j < my_n ? v.plast[ps[j]] : 0u;
                        fp[j] = (uint32_t)j < my_n ? (uint32_t)v.prep[ps[j]] - 1u : 0u;
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if ((uint32_t)j >= my_n) break;
                        int32_t ft[CB_MAX_FL];
#pragma unroll
                        for (int f = 0; f < CB_MAX_FL; ++f) ft[f] = f < t.FL ? row[fp[j] + t.LL + f] : 0;
                        e[t.LL + j] = clock0 + fl[j];
#pragma unroll
                        for (int f = 0; f < CB_MAX_FL; ++f) if (f < t.FL) e[t.LL + t.FC + j * t.FL + f] = (uint32_t)ft[f];
                    }
                    for (int f = (int)my_n; f < t.FC; ++f) e[t.LL + f] = 0u;
                    s.lstamp[got] = clock0 + my_last;
                    my_word = (tag << CB_EID_BITS) | got;
                    my_free = bucket * 32u + (uint32_t)first_free;
                    handled = true;
                }
            }
        }
        uint32_t todo = __ballot_sync(CB_FULL, occ && !handled);
        while (todo) {
            const int src = __ffs(todo) - 1;
            todo &= todo - 1;
            const unsigned long long rep = __shfl_sync(CB_FULL, my_rep, src);
            const int b = (int)(rep >> 32);
            const CbSeq s = cb_seq(t, b);
            const BulkPlan pl = plan[b];
            const int32_t* row = tokens + (size_t)b * row_stride;
            const int32_t k0 = __shfl_sync(CB_FULL, my_k[0], src), k1 = __shfl_sync(CB_FULL, my_k[1], src),
                          k2 = __shfl_sync(CB_FULL, my_k[2], src), k3 = __shfl_sync(CB_FULL, my_k[3], src);
            const int32_t mykey = lane == 0 ? k0 : (lane == 1 ? k1 : (lane == 2 ? k2 : (lane == 3 ? k3 : 0)));
            const uint32_t n = __shfl_sync(CB_FULL, my_n, src), gbase = __shfl_sync(CB_FULL, my_gbase, src);
            const uint32_t cL = pl.clock0 + __shfl_sync(CB_FULL, my_last, src);
            const uint64_t h = __shfl_sync(CB_FULL, my_h, src);
            if (gbase + n > v.W) continue;                       // cannot happen: the ranges partition at most W pairs
            // ---- the leader's entry: found, or taken from the unused ones and filled here (published below)
            const Probe pr = tbl_find<true>(t, s, mykey, h, lane);
            cnt.maxprobe = max(cnt.maxprobe, pr.probes);
            int eid = pr.eid;
            bool fresh = false;
            if (eid == -1 && pr.free_slot != 0xFFFFFFFFu) {
                uint32_t got = 0;
                if (lane == 0) got = atomicAdd(&s.hdr[1], 1u);
                got = __shfl_sync(CB_FULL, got, 0);
                if (got < (uint32_t)t.LC) {                     // anything else is excluded by the plan
                    eid = (int)got;
                    fresh = true;
                    uint32_t* e = s.entries + (size_t)eid * t.E;
                    if (lane < t.LL) e[lane] = (uint32_t)mykey;
                    for (int f = lane + (int)min(n, (uint32_t)t.FC); f < t.FC; f += 32) e[t.LL + f] = 0u;   // the places the followers below leave free
                    if (lane == src) { my_word = (cb_hash_tag(h) << CB_EID_BITS) | (uint32_t)eid; my_free = pr.free_slot; }
                }
            }
            if (eid < 0) {
                if (lane == 0) atomicCAS(status, 0u, (uint32_t)CB_ERR_PROBE_LIMIT);
                continue;
            }
            uint32_t* e = s.entries + (size_t)eid * t.E;
            if (lane == 0) s.lstamp[eid] = cL;
            // ---- with more than FC distinct followers only the FC latest count: the largest thr with FC pairs at or above it
            uint32_t thr = 0;
            if (n > (uint32_t)t.FC) {
                uint32_t lo = 1, hi = pl.nwin;                   // count(last >= lo) >= FC holds for lo = 1
                while (lo < hi) {
                    const uint32_t mid = lo + (hi - lo + 1u) / 2u;
                    uint32_t c = 0;
                    for (uint32_t j = lane; j < n; j += 32) c += v.plast[v.group[gbase + j]] >= mid ? 1u : 0u;
                    c = __reduce_add_sync(CB_FULL, c);
                    if (c >= (uint32_t)t.FC) lo = mid; else hi = mid - 1u;
                }
                thr = lo;
            }
            // ---- the followers: a new entry's places are taken in turn, an old one goes through the follower-list code
            uint32_t placed = 0;
            for (uint32_t j0 = 0; j0 < n; j0 += 32) {
                const uint32_t j = j0 + lane;
                uint32_t last = 0, fpos = 0;
                if (j < n) {
                    const uint32_t ps = v.group[gbase + j];
                    last = v.plast[ps];
                    fpos = (uint32_t)v.prep[ps] - 1u;
                }
                const uint32_t keep = __ballot_sync(CB_FULL, j < n && last >= thr && last > 0u);
                if (fresh) {
                    // lane q writes its own follower's tokens and stamp
                    const uint32_t place = placed + __popc(keep & ((1u << lane) - 1u));
                    if (((keep >> lane) & 1u) && place < (uint32_t)t.FC) {
                        for (int f = 0; f < t.FL; ++f) e[t.LL + t.FC + place * t.FL + f] = (uint32_t)row[fpos + t.LL + f];
                        e[t.LL + place] = pl.clock0 + last;
                    }
                    placed += __popc(keep);
                } else {
                    uint32_t k = keep;
                    while (k) {
                        const int q = __ffs(k) - 1;
                        k &= k - 1;
                        const uint32_t fi = __shfl_sync(CB_FULL, fpos, q);
                        const uint32_t c = pl.clock0 + __shfl_sync(CB_FULL, last, q);
                        const int32_t myfol = lane < t.FL ? row[fi + t.LL + lane] : 0;
                        tbl_put_follower(t, e, myfol, c, lane, cnt);
                        __syncwarp();
                    }
                }
            }
        }
        // ---- publication of the new entries: they are complete (fence), each lane claims the slot found for its leader
        __threadfence();
        __syncwarp();
        bool retry = false;
        if (my_free != 0xFFFFFFFFu) {
            const CbSeq s = cb_seq(t, (int)(my_rep >> 32));
            uint32_t old = atomicCAS(&s.index[my_free], CB_IDX_EMPTY, my_word);
            if (old == CB_IDX_TOMB) old = atomicCAS(&s.index[my_free], CB_IDX_TOMB, my_word) == CB_IDX_TOMB ? CB_IDX_EMPTY : 1u;
            retry = old != CB_IDX_EMPTY;                        // another leader took the slot meanwhile
        }
        uint32_t again = __ballot_sync(CB_FULL, retry);
        while (again) {
            const int src = __ffs(again) - 1;
            again &= again - 1;
            const int b = (int)(__shfl_sync(CB_FULL, my_rep, src) >> 32);
            const CbSeq s = cb_seq(t, b);
            const int32_t k0 = __shfl_sync(CB_FULL, my_k[0], src), k1 = __shfl_sync(CB_FULL, my_k[1], src),
                          k2 = __shfl_sync(CB_FULL, my_k[2], src), k3 = __shfl_sync(CB_FULL, my_k[3], src);
            const int32_t mykey = lane == 0 ? k0 : (lane == 1 ? k1 : (lane == 2 ? k2 : (lane == 3 ? k3 : 0)));
            const uint64_t h = __shfl_sync(CB_FULL, my_h, src);
            const uint32_t word = __shfl_sync(CB_FULL, my_word, src);
            bool done = false;
            for (int attempt = 0; attempt < 64 && !done; ++attempt) {
                const Probe pr = tbl_find<true>(t, s, mykey, h, lane);
                cnt.maxprobe = max(cnt.maxprobe, pr.probes);
                if (pr.eid != -1 || pr.free_slot == 0xFFFFFFFFu) break;
                uint32_t old = 0;
                if (lane == 0) {
                    old = atomicCAS(&s.index[pr.free_slot], CB_IDX_EMPTY, word);
                    if (old == CB_IDX_TOMB) old = atomicCAS(&s.index[pr.free_slot], CB_IDX_TOMB, word) == CB_IDX_TOMB ? CB_IDX_EMPTY : 1u;
                }
                done = __shfl_sync(CB_FULL, old, 0) == CB_IDX_EMPTY;
            }
            if (!done && lane == 0) atomicCAS(status, 0u, (uint32_t)CB_ERR_PROBE_LIMIT);
        }
    }
    if (lane == 0) {
        if (cnt.fevict) atomicAdd(&counters[CB_CNT_FOLLOWER_EVICTIONS], (unsigned long long)cnt.fevict);
        if (cnt.maxprobe) atomicMax(&counters[CB_CNT_MAX_PROBE], (unsigned long long)cnt.maxprobe);
    }
}

}  // namespace
