// Per-sequence LRU cache table kernels: sliding-window update and batched draft-tree expansion.
//
// Every table operation is executed by one warp acting as a unit: the 32 lanes probe the 32 slots of an
// index bucket with one coalesced load, compare the FC followers of an entry in parallel, and scan the
// dense stamp array for the least recently used leader.  Recency is a per-sequence operation counter
// ("clock"); a leader or follower stamp is the clock value of the operation that last touched it.
#include <algorithm>
#include <mutex>

#include "cb_accept_dev.cuh"

namespace {

struct Probe {
    int eid;             // entry id, -1 absent, -2 probe limit
    uint32_t slot;       // index slot holding the entry (when found)
    uint32_t free_slot;  // first reusable slot on the probe path (when absent), 0xFFFFFFFF if none seen
    uint32_t probes;     // buckets visited
};

// Warp-wide lookup of a leader. mykey = key[lane] for lane < LL (0 otherwise), identical call in all lanes.
// SHARED: other SMs publish index words and entries while this warp probes (bulk update), so index and key are read
// through to L2 instead of from an L1 line that may be stale.
// FETCH (tables with FC <= 32, so that lane l owns follower l alone): the follower's stamp and tokens are loaded together
// with the key when an index word's tag matches, which saves the callers two dependent memory round trips.
// FETCH == 2 (larger FC): the stamps of all the lane's followers come with the key (one round trip saved); the tokens are
// loaded when they are known to be needed.
struct EntryRegs {
    uint32_t fs;
    int32_t tok[CB_MAX_FL];
    uint32_t fs4[CB_MAX_FC / 32];
};
template <bool SHARED = false, int FETCH = 0>
__device__ __forceinline__ Probe tbl_find(const CbTables& t, const CbSeq& s, int32_t mykey, uint64_t h, int lane, EntryRegs* er = nullptr) {
    Probe r;
    r.eid = -2; r.slot = 0; r.free_slot = 0xFFFFFFFFu; r.probes = 0;
    const uint32_t nb = t.nslots >> 5, tag = cb_hash_tag(h);
    uint32_t bucket = cb_hash_bucket(h, t.nslots);
    for (uint32_t p = 0; p < nb; ++p) {
        r.probes = p + 1;
        const uint32_t w = SHARED ? __ldcg(&s.index[bucket * 32 + lane]) : s.index[bucket * 32 + lane];
        uint32_t cand = __ballot_sync(CB_FULL, w != CB_IDX_EMPTY && w != CB_IDX_TOMB && (w >> CB_EID_BITS) == tag);
        while (cand) {
            const int l = __ffs(cand) - 1;
            cand &= cand - 1;
            const uint32_t eid = __shfl_sync(CB_FULL, w, l) & CB_EID_MASK;
            if (!cb_dbg_in(eid, t.LC, t.dbg_status)) continue;                // an index word naming an entry that cannot exist
            bool eq = true;
            if (FETCH == 2) {
                const uint32_t* e = s.entries + (size_t)eid * t.E;
                const uint32_t kv = lane < t.LL ? e[lane] : 0u;
#pragma unroll
                for (int c = 0; c < CB_MAX_FC / 32; ++c) er->fs4[c] = (c * 32 + lane) < t.FC ? e[t.LL + c * 32 + lane] : 0u;
                if (lane < t.LL) eq = (int32_t)kv == mykey;
            } else if (FETCH == 1) {
                const uint32_t* e = s.entries + (size_t)eid * t.E;
                const bool mine = lane < t.FC;
                const uint32_t kv = lane < t.LL ? e[lane] : 0u;
                er->fs = mine ? e[t.LL + lane] : 0u;
#pragma unroll
                for (int j = 0; j < CB_MAX_FL; ++j) er->tok[j] = (mine && j < t.FL) ? (int32_t)e[t.LL + t.FC + lane * t.FL + j] : -1;
                if (lane < t.LL) eq = (int32_t)kv == mykey;
            } else if (lane < t.LL) {
                const uint32_t* kp = &s.entries[(size_t)eid * t.E + lane];
                eq = ((int32_t)(SHARED ? __ldcg(kp) : *kp) == mykey);
            }
            if (__all_sync(CB_FULL, eq)) { r.eid = (int)eid; r.slot = bucket * 32 + l; return r; }
        }
        const uint32_t fr = __ballot_sync(CB_FULL, w == CB_IDX_EMPTY || w == CB_IDX_TOMB);
        if (r.free_slot == 0xFFFFFFFFu && fr) r.free_slot = bucket * 32 + (__ffs(fr) - 1);
        if (__ballot_sync(CB_FULL, w == CB_IDX_EMPTY)) { r.eid = -1; return r; }
        bucket = (bucket + 1) & (nb - 1);
    }
    return r;
}

__device__ __forceinline__ uint64_t warp_hash(const CbTables& t, int32_t mykey) {
    const int32_t k0 = __shfl_sync(CB_FULL, mykey, 0), k1 = __shfl_sync(CB_FULL, mykey, 1),
                  k2 = __shfl_sync(CB_FULL, mykey, 2), k3 = __shfl_sync(CB_FULL, mykey, 3);
    return cb_hash4(k0, k1, k2, k3, t.LL);
}

// Removes the least recently used leader from the index and returns its entry id for reuse.
__device__ int tbl_evict_lru(const CbTables& t, const CbSeq& s, int lane, uint32_t* status) {
    uint32_t minv = 0xFFFFFFFFu;
    int mine = 0;
#pragma unroll 4
    for (int i = lane; i < t.LC; i += 32) {
        const uint32_t v = s.lstamp[i];
        if (v < minv) { minv = v; mine = i; }
    }
    const uint32_t g = __reduce_min_sync(CB_FULL, minv);
    const int wl = __ffs(__ballot_sync(CB_FULL, minv == g)) - 1;   // stamps are unique
    const int eid = __shfl_sync(CB_FULL, mine, wl);
    const int32_t vkey = lane < t.LL ? (int32_t)s.entries[(size_t)eid * t.E + lane] : 0;
    const uint64_t h = warp_hash(t, vkey);
    const uint32_t nb = t.nslots >> 5, word = (cb_hash_tag(h) << CB_EID_BITS) | (uint32_t)eid;
    uint32_t bucket = cb_hash_bucket(h, t.nslots);
    for (uint32_t p = 0; p < nb; ++p) {
        const uint32_t w = s.index[bucket * 32 + lane];
        const uint32_t hit = __ballot_sync(CB_FULL, w == word);
        const uint32_t empties = __ballot_sync(CB_FULL, w == CB_IDX_EMPTY);
        if (hit) {
            // A bucket that still has an empty slot is the end of every probe path through it, so the
            // slot can simply become empty again; otherwise later buckets may hold keys that probed
            // past this one and the slot must stay marked as deleted.
            if (lane == __ffs(hit) - 1) s.index[bucket * 32 + lane] = empties ? CB_IDX_EMPTY : CB_IDX_TOMB;
            __syncwarp();
            return eid;
        }
        if (empties) break;
        bucket = (bucket + 1) & (nb - 1);
    }
    if (lane == 0) atomicCAS(status, 0u, (uint32_t)CB_ERR_PROBE_LIMIT);   // index and entries disagree
    return eid;
}

struct TblCounters { uint32_t inserts, levict, fevict, maxprobe; };

// Follower list of an existing leader (Section 3.1): a stored copy of the follower is refreshed, otherwise the follower takes
// the lowest free place or replaces the least recently inserted one.  e = the leader's entry, c = this operation's stamp.
// The same with the follower's stamp and tokens already in registers (FC <= 32).
__device__ __forceinline__ void tbl_put_follower_regs(const CbTables& t, uint32_t* e, const EntryRegs& er, int32_t myfol, uint32_t c, int lane,
                                                      TblCounters& cnt) {
    const bool mine = lane < t.FC;
    bool match = mine && er.fs != 0u;
#pragma unroll
    for (int j = 0; j < CB_MAX_FL; ++j) {
        const int32_t fj = __shfl_sync(CB_FULL, myfol, j);
        if (j < t.FL) match = match && (er.tok[j] == fj);
    }
    const uint32_t mm = __ballot_sync(CB_FULL, match);
    if (mm) {
        if (t.refresh && lane == 0) e[t.LL + (__ffs(mm) - 1)] = c;
        return;
    }
    const uint32_t freem = __ballot_sync(CB_FULL, mine && er.fs == 0u);
    int tgt;
    if (freem) {
        tgt = __ffs(freem) - 1;
    } else {
        const uint32_t g = __reduce_min_sync(CB_FULL, mine ? er.fs : 0xFFFFFFFFu);
        tgt = __ffs(__ballot_sync(CB_FULL, mine && er.fs == g)) - 1;
        cnt.fevict++;
    }
    if (lane < t.FL) e[t.LL + t.FC + tgt * t.FL + lane] = (uint32_t)myfol;
    if (lane == 0) e[t.LL + tgt] = c;
}

template <bool PRE = false>
__device__ __forceinline__ void tbl_put_follower(const CbTables& t, uint32_t* e, int32_t myfol, uint32_t c, int lane, TblCounters& cnt,
                                                 const EntryRegs* er = nullptr) {
    // Lane l looks after followers l, l + 32, ...: one pass finds a stored copy of the follower, the lowest free place
    // and the least recently inserted follower.  PRE: the stamps came with the lookup.
    int match_f = -1, free_f = -1, lru_f = -1;
    uint32_t lru_stamp = 0xFFFFFFFFu;
#pragma unroll
    for (int ch = 0; ch < CB_MAX_FC / 32; ++ch) {
        const int base = ch * 32;
        if (base >= t.FC || match_f >= 0) break;
        const int f = base + lane;
        const bool mine = f < t.FC;
        const uint32_t fs = PRE ? er->fs4[ch] : (mine ? e[t.LL + f] : 0u);
        bool match = mine && fs != 0u;
        for (int j = 0; j < t.FL; ++j) {
            const int32_t fj = __shfl_sync(CB_FULL, myfol, j);
            if (match) match = ((int32_t)e[t.LL + t.FC + f * t.FL + j] == fj);
        }
        const uint32_t mm = __ballot_sync(CB_FULL, match);
        if (mm) { match_f = base + __ffs(mm) - 1; break; }
        const uint32_t freem = __ballot_sync(CB_FULL, mine && fs == 0u);
        if (free_f < 0 && freem) free_f = base + __ffs(freem) - 1;
        const uint32_t g = __reduce_min_sync(CB_FULL, (mine && fs != 0u) ? fs : 0xFFFFFFFFu);
        if (g < lru_stamp) { lru_stamp = g; lru_f = base + __ffs(__ballot_sync(CB_FULL, mine && fs == g)) - 1; }
    }
    if (match_f >= 0) {
        if (t.refresh && lane == 0) e[t.LL + match_f] = c;
    } else {
        int tgt = free_f;
        if (tgt < 0) { tgt = lru_f; cnt.fevict++; }
        if (lane < t.FL) e[t.LL + t.FC + tgt * t.FL + lane] = (uint32_t)myfol;
        if (lane == 0) e[t.LL + tgt] = c;
    }
}

// One insertion (Section 3.1). mykey = leader[lane] (lane < LL), myfol = follower[lane] (lane < FL).
template <int FETCH = 0>
__device__ void tbl_insert(const CbTables& t, const CbSeq& s, int32_t mykey, int32_t myfol, uint32_t& clock,
                           uint32_t& count, int lane, uint32_t* status, TblCounters& cnt) {
    const uint32_t c = ++clock;
    cnt.inserts++;
    const uint64_t h = warp_hash(t, mykey);
    EntryRegs er;
    Probe pr = tbl_find<false, FETCH>(t, s, mykey, h, lane, &er);
    cnt.maxprobe = max(cnt.maxprobe, pr.probes);
    if (pr.eid >= 0) {
        uint32_t* e = s.entries + (size_t)pr.eid * t.E;
        if (lane == 0) s.lstamp[pr.eid] = c;
        if (FETCH == 1) tbl_put_follower_regs(t, e, er, myfol, c, lane, cnt);
        else if (FETCH == 2) tbl_put_follower<true>(t, e, myfol, c, lane, cnt, &er);
        else tbl_put_follower(t, e, myfol, c, lane, cnt);
    } else if (pr.eid == -1) {
        int eid;
        if (count < (uint32_t)t.LC) {
            eid = (int)count++;
        } else {
            eid = tbl_evict_lru(t, s, lane, status);
            cnt.levict++;
            pr = tbl_find(t, s, mykey, h, lane);           // the eviction may have opened a nearer slot
        }
        if (pr.free_slot == 0xFFFFFFFFu) {
            if (lane == 0) atomicCAS(status, 0u, (uint32_t)CB_ERR_PROBE_LIMIT);
        } else {
            uint32_t* e = s.entries + (size_t)eid * t.E;
            if (lane < t.LL) e[lane] = (uint32_t)mykey;
            for (int f = lane; f < t.FC; f += 32) e[t.LL + f] = f == 0 ? c : 0u;
            if (lane < t.FL) e[t.LL + t.FC + lane] = (uint32_t)myfol;
            if (lane == 0) {
                s.lstamp[eid] = c;
                s.index[pr.free_slot] = (cb_hash_tag(h) << CB_EID_BITS) | (uint32_t)eid;
            }
        }
    } else {
        if (lane == 0) atomicCAS(status, 0u, (uint32_t)CB_ERR_PROBE_LIMIT);
    }
    __syncwarp();
}

// One warp per sequence; windows are applied in increasing position.
template <int FETCH>
__device__ __forceinline__ void update_seq(const CbTables& t, int b, const int32_t* tokens, int64_t row_stride, int n0, int n1,
                                           int lane, uint32_t* status, unsigned long long* counters) {
    const CbSeq s = cb_seq(t, b);
    const int w = t.LL + t.FL;
    uint32_t clock = s.hdr[0], count = s.hdr[1];
    TblCounters cnt = {0, 0, 0, 0};
    const int32_t* row = tokens + (size_t)b * row_stride;
    for (int i = max(0, n0 - w + 1); i + w <= n1; ++i) {
        const int32_t mykey = lane < t.LL ? row[i + lane] : 0;
        const int32_t myfol = lane < t.FL ? row[i + t.LL + lane] : 0;
        tbl_insert<FETCH>(t, s, mykey, myfol, clock, count, lane, status, cnt);
    }
    if (lane == 0) {
        s.hdr[0] = clock; s.hdr[1] = count;
        if (cnt.inserts) atomicAdd(&counters[CB_CNT_INSERTS], (unsigned long long)cnt.inserts);
        if (cnt.levict) atomicAdd(&counters[CB_CNT_LEADER_EVICTIONS], (unsigned long long)cnt.levict);
        if (cnt.fevict) atomicAdd(&counters[CB_CNT_FOLLOWER_EVICTIONS], (unsigned long long)cnt.fevict);
        if (cnt.maxprobe) atomicMax(&counters[CB_CNT_MAX_PROBE], (unsigned long long)cnt.maxprobe);
    }
}

template <int FETCH>
__global__ void __launch_bounds__(128) cb_update_kernel(CbTables t, int B, const int32_t* __restrict__ tokens,
                                                        int64_t row_stride, const int32_t* __restrict__ n_old,
                                                        const int32_t* __restrict__ n_new, uint32_t* status,
                                                        unsigned long long* counters) {
    CB_PDL_ENTRY();
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (b >= B) return;
    update_seq<FETCH>(t, b, tokens, row_stride, n_old[b], n_new[b], lane, status, counters);
}

// ---------------------------------------------------------------------------------------------------
// Bulk update (prompt initialisation and other long runs of new tokens): many warps per sequence.
//
// The result of a run of insertions depends on their order only within one leader (its recency and its follower list)
// and, across leaders, through leader eviction.  Stamps are a function of the window's position (the clock ticks once per
// window), so when no leader can be evicted during the run (leaders stored + windows <= LC) the windows may be dealt out
// to warps by a hash of their leader: every leader is handled by one warp, in increasing position, exactly as the
// sequential kernel would, and different leaders touch disjoint entries.  What the warps share is the leader counter
// (atomicAdd hands out entry ids) and the index, whose slots are claimed with atomicCAS; an entry is complete before its
// index word is published.  A plan kernel takes that decision once per sequence, before any warp changes the table;
// sequences that do not qualify (short runs, possible eviction) are done by their first warp alone, in order.
struct BulkPlan { uint32_t parallel, clock0, first, nwin; };   // parallel: 0 one warp in order, 1 warps by leader, 2 order-free path (cb_bulk_free.cuh)

__global__ void cb_bulk_plan_kernel(CbTables t, int B, const int32_t* __restrict__ n_old, const int32_t* __restrict__ n_new,
                                    BulkPlan* plan) {
    CB_PDL_ENTRY();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const CbSeq s = cb_seq(t, b);
    const int w = t.LL + t.FL;
    const int first = max(0, n_old[b] - w + 1);
    const int nwin = max(0, n_new[b] - w + 1 - first);
    BulkPlan p;
    p.clock0 = s.hdr[0];
    p.first = (uint32_t)first;
    p.nwin = (uint32_t)nwin;
    p.parallel = (nwin >= 64 && (unsigned long long)s.hdr[1] + (unsigned long long)nwin <= (unsigned long long)t.LC) ? 1u : 0u;
    if (p.parallel) s.hdr[0] = p.clock0 + (uint32_t)nwin;      // the clock after the run; the warps take stamps from positions
    plan[b] = p;
}

// One insertion of the parallel path: c is the operation's stamp; no leader is ever evicted here.  Returns the leader's
// entry id (-1 if the insertion failed).
__device__ int tbl_insert_shared(const CbTables& t, const CbSeq& s, int32_t mykey, int32_t myfol, uint32_t c, int lane,
                                 uint32_t* status, TblCounters& cnt) {
    cnt.inserts++;
    const uint64_t h = warp_hash(t, mykey);
    const uint32_t tagword = cb_hash_tag(h) << CB_EID_BITS;
    int eid = -1;
    for (int attempt = 0; attempt < 64; ++attempt) {            // a claim can lose its slot to another warp's leader: look again
        const Probe pr = tbl_find<true>(t, s, mykey, h, lane);
        cnt.maxprobe = max(cnt.maxprobe, pr.probes);
        if (pr.eid >= 0) {
            uint32_t* e = s.entries + (size_t)pr.eid * t.E;
            if (lane == 0) s.lstamp[pr.eid] = c;
            tbl_put_follower(t, e, myfol, c, lane, cnt);
            __syncwarp();
            return pr.eid;
        }
        if (pr.eid != -1 || pr.free_slot == 0xFFFFFFFFu) break;
        if (eid < 0) {
            // new leader: take an entry, fill it, then publish it
            uint32_t got = 0;
            if (lane == 0) got = atomicAdd(&s.hdr[1], 1u);
            got = __shfl_sync(CB_FULL, got, 0);
            if (got >= (uint32_t)t.LC) break;                  // excluded by the plan
            eid = (int)got;
            uint32_t* e = s.entries + (size_t)eid * t.E;
            if (lane < t.LL) e[lane] = (uint32_t)mykey;
            for (int f = lane; f < t.FC; f += 32) e[t.LL + f] = f == 0 ? c : 0u;
            if (lane < t.FL) e[t.LL + t.FC + lane] = (uint32_t)myfol;
            if (lane == 0) s.lstamp[eid] = c;
            __threadfence();
            __syncwarp();
        }
        uint32_t old = 0;
        if (lane == 0) old = atomicCAS(&s.index[pr.free_slot], CB_IDX_EMPTY, tagword | (uint32_t)eid);
        old = __shfl_sync(CB_FULL, old, 0);
        if (old == CB_IDX_EMPTY) return eid;
        if (old == CB_IDX_TOMB) {                              // a deleted slot is as good as an empty one
            if (lane == 0) old = atomicCAS(&s.index[pr.free_slot], CB_IDX_TOMB, tagword | (uint32_t)eid);
            old = __shfl_sync(CB_FULL, old, 0);
            if (old == CB_IDX_TOMB) return eid;
        }
    }
    if (lane == 0) atomicCAS(status, 0u, (uint32_t)CB_ERR_PROBE_LIMIT);
    return -1;
}

// The warp that owns a frequent leader meets it again and again (with unigram leaders a handful of tokens own a third of
// the windows), and every insertion into a leader that is in the table is a chain of four dependent memory round trips.  So
// every warp keeps the entries it touched last in shared memory (WAYS of them: key, follower stamps and tokens, leader
// stamp): an insertion into a kept entry is the same follower-list code running on the shared-memory copy, and the copy goes
// back to the table when its place is needed or the run ends.  No other warp touches these leaders during the run.
__global__ void __launch_bounds__(256) cb_update_bulk_kernel(CbTables t, int B, int WPS, int WAYS, const int32_t* __restrict__ tokens, int64_t row_stride,
                                                             const int32_t* __restrict__ n_old, const int32_t* __restrict__ n_new,
                                                             const BulkPlan* __restrict__ plan, uint32_t* status, unsigned long long* counters) {
    CB_PDL_ENTRY();
    extern __shared__ uint32_t bulk_smem[];
    const int lane = threadIdx.x & 31;
    // this warp's kept entries: WAYS x (E words of the entry, then entry id + 1 (0 = free), leader stamp, last use, unused)
    const uint32_t way_words = t.E + 4;
    uint32_t* ways = bulk_smem + (size_t)(threadIdx.x >> 5) * WAYS * way_words;
    for (int w = lane; w < WAYS; w += 32) ways[(size_t)w * way_words + t.E] = 0u;
    __syncwarp();
    uint32_t use_clock = 0;
    const int gw = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int b = gw / WPS, wi = gw % WPS;
    if (b >= B) return;
    const CbSeq s = cb_seq(t, b);
    const BulkPlan pl = plan[b];
    if (pl.parallel == 2u) return;                              // done by the order-free kernels
    const int32_t* row = tokens + (size_t)b * row_stride;
    TblCounters cnt = {0, 0, 0, 0};
    if (!pl.parallel) {
        if (wi != 0) return;
        uint32_t clock = s.hdr[0], count = s.hdr[1];
        for (uint32_t k = 0; k < pl.nwin; ++k) {
            const int i = (int)(pl.first + k);
            const int32_t mykey = lane < t.LL ? row[i + lane] : 0;
            const int32_t myfol = lane < t.FL ? row[i + t.LL + lane] : 0;
            tbl_insert(t, s, mykey, myfol, clock, count, lane, status, cnt);
        }
        if (lane == 0) { s.hdr[0] = clock; s.hdr[1] = count; }
    } else {
        // 32 windows at a time: every lane hashes one leader, the warp keeps those that are its own and inserts them in order
        for (uint32_t k0 = 0; k0 < pl.nwin; k0 += 32) {
            const uint32_t k = k0 + lane;
            bool mine = false;
            if (k < pl.nwin) {
                const int i = (int)(pl.first + k);
                int32_t k4[4] = {0, 0, 0, 0};
                for (int j = 0; j < t.LL; ++j) k4[j] = row[i + j];
                const uint64_t h = cb_hash4(k4[0], k4[1], k4[2], k4[3], t.LL);
                mine = (uint32_t)((h >> 17) % (uint64_t)WPS) == (uint32_t)wi;
            }
            uint32_t todo = __ballot_sync(CB_FULL, mine);
            while (todo) {
                const int l = __ffs(todo) - 1;
                todo &= todo - 1;
                const int i = (int)(pl.first + k0 + l);
                const int32_t mykey = lane < t.LL ? row[i + lane] : 0;
                const int32_t myfol = lane < t.FL ? row[i + t.LL + lane] : 0;
                const uint32_t c = pl.clock0 + k0 + (uint32_t)l + 1u;
                // is the leader among the kept entries?  lane w compares way w's key
                bool match = lane < WAYS && ways[(size_t)lane * way_words + t.E] != 0u;
                for (int j = 0; j < t.LL; ++j) {
                    const int32_t kj = __shfl_sync(CB_FULL, mykey, j);
                    if (match) match = (int32_t)ways[(size_t)lane * way_words + j] == kj;
                }
                const uint32_t hit = __ballot_sync(CB_FULL, match);
                ++use_clock;
                if (hit) {
                    uint32_t* e = ways + (size_t)(__ffs(hit) - 1) * way_words;
                    cnt.inserts++;
                    if (lane == 0) { e[t.E + 1] = c; e[t.E + 2] = use_clock; }
                    tbl_put_follower(t, e, myfol, c, lane, cnt);
                    __syncwarp();
                    continue;
                }
                const int eid = tbl_insert_shared(t, s, mykey, myfol, c, lane, status, cnt);
                if (eid < 0) continue;
                // keep it: in a free way, else in place of the way used longest ago (whose copy goes back to the table first)
                uint32_t u = lane < WAYS ? (ways[(size_t)lane * way_words + t.E] == 0u ? 0u : ways[(size_t)lane * way_words + t.E + 2]) : 0xFFFFFFFFu;
                const uint32_t umin = __reduce_min_sync(CB_FULL, u);
                uint32_t* e = ways + (size_t)(__ffs(__ballot_sync(CB_FULL, u == umin)) - 1) * way_words;
                const uint32_t old = e[t.E];
                if (old != 0u) {
                    uint32_t* g = s.entries + (size_t)(old - 1u) * t.E;
                    for (uint32_t k = lane; k < t.E; k += 32) g[k] = e[k];
                    if (lane == 0) s.lstamp[old - 1u] = e[t.E + 1];
                }
                __syncwarp();
                const uint32_t* g = s.entries + (size_t)eid * t.E;
                for (uint32_t k = lane; k < t.E; k += 32) e[k] = __ldcg(g + k);
                if (lane == 0) { e[t.E] = (uint32_t)eid + 1u; e[t.E + 1] = c; e[t.E + 2] = use_clock; }
                __syncwarp();
            }
        }
        // the kept entries go back to the table
        for (int w = 0; w < WAYS; ++w) {
            const uint32_t* e = ways + (size_t)w * way_words;
            const uint32_t id = e[t.E];
            if (id == 0u) continue;
            uint32_t* g = s.entries + (size_t)(id - 1u) * t.E;
            for (uint32_t k = lane; k < t.E; k += 32) g[k] = e[k];
            if (lane == 0) s.lstamp[id - 1u] = e[t.E + 1];
        }
    }
    if (lane == 0) {
        if (cnt.inserts) atomicAdd(&counters[CB_CNT_INSERTS], (unsigned long long)cnt.inserts);
        if (cnt.levict) atomicAdd(&counters[CB_CNT_LEADER_EVICTIONS], (unsigned long long)cnt.levict);
        if (cnt.fevict) atomicAdd(&counters[CB_CNT_FOLLOWER_EVICTIONS], (unsigned long long)cnt.fevict);
        if (cnt.maxprobe) atomicMax(&counters[CB_CNT_MAX_PROBE], (unsigned long long)cnt.maxprobe);
    }
}

}  // namespace

#include "cb_bulk_free.cuh"

namespace {

// ---------------------------------------------------------------------------------------------------
// Draft-tree expansion: one CTA per sequence, one warp per frontier leaf ("branch") for the lookups.
// Each level: (1) warps look up the keys of all frontier leaves in parallel and stage the followers,
// most recent first, in shared memory; (2) one thread replays the sequential breadth-first order over
// the staged results, which fixes node indices, the point where the size cap ends the level and the
// ordinal of every query that the sequential order would have issued; (3) the leaders of those queries
// get their new recency stamp with an atomic max (two leaves of one level may share a leader).
// With a frozen table attached (Section 3.3) a second pass follows while the tree is below the size cap: its first
// frontier is every node that was a frontier leaf of the first pass, in creation order, and its lookups go to the
// frozen table, which is shared by all sequences and only read (no clock tick, no stamp).
struct DraftSmem {
    int32_t* tok; int32_t* par; int32_t* dep;
    int32_t* front; int32_t* next; int32_t* pts;
    int32_t* r_eid; int32_t* r_nf; int32_t* r_ok; uint32_t* r_stamp;
    int32_t* r_n0; int32_t* r_cl; int32_t* r_tot; int32_t* r_nn0;     // plan of a leaf's attachment: first node, chain length, nodes, first frontier place
    int32_t* fol;
};

// The work of the CTA that drafts sequence b, whose history holds L tokens.  upd_n_old >= 0: the windows that the tokens
// from upd_n_old on complete are inserted first (cb_update_draft_tree and the call that follows an acceptance).  The
// history may have been extended by this CTA just before (no read-only path to it).
template <int FETCH>
__device__ __forceinline__ void draft_body(const CbTables& t, const CbTables& tf, int T, int crt, int max_depth, int NL, int KF,
                                           const int32_t* tokens, int64_t row_stride, int b, int L, int upd_n_old,
                                           int32_t* __restrict__ o_tok, int32_t* __restrict__ o_par,
                                           int32_t* __restrict__ o_dep, uint32_t* __restrict__ o_mask,
                                           int32_t* __restrict__ o_n, uint32_t* status,
                                           unsigned long long* counters, int32_t* smem) {
    DraftSmem S;
    S.tok = smem; S.par = S.tok + T; S.dep = S.par + T;
    S.front = S.dep + T; S.next = S.front + NL; S.pts = S.next + NL;
    S.r_eid = S.pts + NL; S.r_nf = S.r_eid + NL; S.r_ok = S.r_nf + NL; S.r_stamp = (uint32_t*)(S.r_ok + NL);
    S.r_n0 = (int32_t*)(S.r_stamp + NL); S.r_cl = S.r_n0 + NL; S.r_tot = S.r_cl + NL; S.r_nn0 = S.r_tot + NL;
    S.fol = S.r_nn0 + NL;
    __shared__ int sh_n, sh_nfront, sh_nnext, sh_npts, sh_q, sh_hits, sh_fq, sh_fhits;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    const CbSeq s = cb_seq(t, b);
    const int32_t* row = tokens + (size_t)b * row_stride;
    if (upd_n_old >= 0) {
        // cb_update_draft_tree: the sequence's new windows go into the table first (one warp, in order, exactly as
        // cb_update does), then the whole CTA drafts from the updated table.
        if (warp == 0) update_seq<FETCH>(t, b, tokens, row_stride, upd_n_old, L, lane, status, counters);
        __threadfence_block();
        __syncthreads();
    }
    const int W = (T + 31) >> 5;
    const int FLFC = t.FL * KF;                               // staged followers per leaf: the KF best
    const uint32_t clock0 = s.hdr[0];
    const bool has_frozen = tf.index != nullptr;

    for (int i = tid; i < T; i += blockDim.x) { S.tok[i] = -1; S.par[i] = -1; S.dep[i] = -1; }
    if (tid == 0) {
        sh_n = 0; sh_nfront = 0; sh_npts = 0; sh_q = 0; sh_hits = 0; sh_fq = 0; sh_fhits = 0;
    }
    __syncthreads();
    if (tid == 0 && L >= 1) {
        S.tok[0] = row[L - 1]; S.dep[0] = 0; sh_n = 1; S.front[0] = 0; sh_nfront = 1; S.pts[0] = 0; sh_npts = 1;
    }
    __syncthreads();

    for (int pass = 0; pass < (has_frozen ? 2 : 1); ++pass) {
        const CbTables& tt = pass ? tf : t;
        const CbSeq ss = pass ? cb_seq(tf, 0) : s;
        if (pass == 1) {
            // the frozen pass starts from every frontier leaf the dynamic pass had
            const int np = sh_npts;
            __syncthreads();
            for (int i = tid; i < np; i += blockDim.x) S.front[i] = S.pts[i];
            if (tid == 0) sh_nfront = np;
            __syncthreads();
        }
        while (true) {
            const int nfront = sh_nfront;
            if (nfront == 0 || sh_n >= T) break;
            for (int li = tid; li < nfront; li += blockDim.x) S.r_stamp[li] = 0u;
            if (tid == 0) sh_nnext = 0;
            __syncthreads();
            // With long follower lists the frontier is worked off in batches of one leaf per warp, lookups then replay, so that a
            // level ends as soon as the tree is full (the first leaves of a level then usually take all the room).
            const int BS = tt.FC > 32 ? nwarps : nfront;          // short follower lists: the whole frontier at once
            for (int base = 0; base < nfront; base += BS) {
                const int n_now = sh_n;
                if (n_now >= T) break;
                // (1) parallel lookups, one warp per leaf
                for (int li = base + warp; li < min(nfront, base + BS); li += nwarps) {
                    const int leaf = S.front[li];
                    const int d = S.dep[leaf];
                    // key = last LL tokens of (row[0 .. L-1) ++ root->leaf path); lane j < LL holds key[j]
                    int32_t mykey = 0;
                    bool ok = d < max_depth;
                    if (lane < t.LL) {
                        const int back = t.LL - 1 - lane;     // distance from the leaf along the sequence
                        if (back <= d) {
                            int c = leaf;
                            for (int k = 0; k < back; ++k) c = S.par[c];
                            mykey = S.tok[c];
                        } else {
                            const int pos = L - 1 - (back - d);
                            mykey = pos >= 0 ? row[pos] : -1;
                        }
                    }
                    ok = ok && __all_sync(CB_FULL, mykey >= 0);
                    int eid = -1, nf = 0;
                    if (ok) {
                        const uint64_t h = warp_hash(tt, mykey);
                        EntryRegs er;
                        const Probe pr = tbl_find<false, FETCH>(tt, ss, mykey, h, lane, &er);
                        if (pr.eid == -2 && lane == 0) atomicCAS(status, 0u, (uint32_t)CB_ERR_PROBE_LIMIT);
                        if (pr.eid >= 0) {
                            eid = pr.eid;
                            const uint32_t* e = ss.entries + (size_t)eid * tt.E;
                            // Lane l holds the stamps of followers l, l + 32, ...  The followers are wanted by falling stamp
                            // (most recently inserted first in the dynamic table, most frequent first in the frozen one),
                            // and only as many as the tree still has room for: they are picked one by one with a warp-wide
                            // maximum (stamps are unique) and staged in that order.
                            uint32_t fs[CB_MAX_FC / 32];
#pragma unroll
                            for (int c = 0; c < CB_MAX_FC / 32; ++c) {
                                if (FETCH == 1) fs[c] = c == 0 ? er.fs : 0u;       // FC <= 32: stamp and tokens came with the lookup
                                else if (FETCH == 2) fs[c] = er.fs4[c];            // the stamps came with the lookup
                                else fs[c] = (c * 32 + lane) < tt.FC ? e[tt.LL + c * 32 + lane] : 0u;
                                nf += __popc(__ballot_sync(CB_FULL, fs[c] != 0u));
                            }
                            nf = min(nf, min(KF, (leaf == 0 ? max(1, T - crt) : T) - n_now));
                            int rank[CB_MAX_FC / 32];
#pragma unroll
                            for (int c = 0; c < CB_MAX_FC / 32; ++c) rank[c] = -1;
                            if (nf <= 16) {
                                for (int r = 0; r < nf; ++r) {
                                    uint32_t m = fs[0];
#pragma unroll
                                    for (int c = 1; c < CB_MAX_FC / 32; ++c) m = max(m, fs[c]);
                                    const uint32_t g = __reduce_max_sync(CB_FULL, m);
#pragma unroll
                                    for (int c = 0; c < CB_MAX_FC / 32; ++c)
                                        if (fs[c] == g) { rank[c] = r; fs[c] = 0u; }
                                }
                            } else {
                                // many are wanted: rank every follower by counting the larger stamps (independent shuffles,
                                // where the repeated maximum is a chain of reductions)
                                int cntr[CB_MAX_FC / 32];
#pragma unroll
                                for (int c = 0; c < CB_MAX_FC / 32; ++c) cntr[c] = 0;
#pragma unroll
                                for (int c2 = 0; c2 < CB_MAX_FC / 32; ++c2) {
                                    if (c2 * 32 >= tt.FC) break;
                                    for (int l = 0; l < 32; ++l) {
                                        const uint32_t o = __shfl_sync(CB_FULL, fs[c2], l);
#pragma unroll
                                        for (int c = 0; c < CB_MAX_FC / 32; ++c) cntr[c] += (o > fs[c]) ? 1 : 0;
                                    }
                                }
#pragma unroll
                                for (int c = 0; c < CB_MAX_FC / 32; ++c)
                                    if (fs[c] != 0u && cntr[c] < nf) rank[c] = cntr[c];
                            }
                            // every lane copies the tokens of its picked followers
#pragma unroll
                            for (int c = 0; c < CB_MAX_FC / 32; ++c) {
                                if (rank[c] >= 0) {
                                    const int f = c * 32 + lane;
                                    if (FETCH == 1) {
#pragma unroll
                                        for (int j = 0; j < CB_MAX_FL; ++j)
                                            if (j < tt.FL) S.fol[li * FLFC + rank[c] * tt.FL + j] = er.tok[j];
                                    } else {
                                        for (int j = 0; j < tt.FL; ++j)
                                            S.fol[li * FLFC + rank[c] * tt.FL + j] = (int32_t)e[tt.LL + tt.FC + f * tt.FL + j];
                                    }
                                }
                            }
                        }
                    }
                    if (lane == 0) { S.r_eid[li] = eid; S.r_nf[li] = nf; S.r_ok[li] = ok ? 1 : 0; }
                }
                __syncthreads();
                // (2) the sequential breadth-first order, planned by one thread and filled in by all.  A query at the root (the only
                // leaf of level 1) is issued, and its followers attached, while the tree has fewer than max(1, T - crt) nodes; any
                // other while fewer than T.  Below a leaf of depth d every follower is a chain of min(FL, max_depth - d) nodes, the
                // chains follow one another until the cap cuts the last one short, and a chain of FL nodes ends in a leaf of the
                // next level: so a leaf's nodes and frontier places follow from where it starts, and only that is sequential.
                const int lend = min(nfront, base + BS);
                if (tid == 0) {
                    int n = n_now, q = 0, hits = 0, nn = sh_nnext;
                    for (int l2 = base; l2 < lend; ++l2) {
                        S.r_tot[l2] = 0;
                        if (n >= T) continue;
                        const int leaf = S.front[l2];
                        const int cap = leaf == 0 ? max(1, T - crt) : T;
                        if (n >= cap) continue;
                        if (!S.r_ok[l2]) continue;
                        ++q;                                    // this query is issued: the dynamic table's clock ticks
                        if (S.r_eid[l2] < 0) continue;
                        ++hits;
                        if (pass == 0) S.r_stamp[l2] = clock0 + (uint32_t)(sh_q + q);
                        const int cl = min(t.FL, max_depth - S.dep[leaf]);
                        const int tot = min(max(S.r_nf[l2], 0) * cl, cap - n);
                        S.r_n0[l2] = n; S.r_cl[l2] = cl; S.r_tot[l2] = tot; S.r_nn0[l2] = nn;
                        n += tot;
                        if (cl == t.FL) nn += tot / t.FL;
                    }
                    sh_n = n; sh_nnext = nn;
                    if (pass == 0) { sh_q += q; sh_hits += hits; } else { sh_fq += q; sh_fhits += hits; }
                }
                __syncthreads();
                for (int l2 = base; l2 < lend; ++l2) {
                    const int tot = S.r_tot[l2];
                    if (tot == 0) continue;
                    const int leaf = S.front[l2], n0 = S.r_n0[l2], cl = S.r_cl[l2], d = S.dep[leaf];
                    for (int x = tid; x < tot; x += blockDim.x) {
                        const int f = x / cl, j = x - f * cl;
                        S.tok[n0 + x] = S.fol[l2 * FLFC + f * t.FL + j];
                        S.par[n0 + x] = j == 0 ? leaf : n0 + x - 1;
                        S.dep[n0 + x] = d + j + 1;
                    }
                    if (cl == t.FL)
                        for (int c = tid; c < tot / t.FL; c += blockDim.x) S.next[S.r_nn0[l2] + c] = n0 + c * t.FL + t.FL - 1;
                }
            }
            // (3) stamp the leaders the sequential order reached; publish the next frontier
            if (pass == 0)
                for (int li = tid; li < nfront; li += blockDim.x)
                    if (S.r_stamp[li] != 0u) atomicMax(&s.lstamp[S.r_eid[li]], S.r_stamp[li]);
            const int nn = sh_nnext, np = sh_npts;
            __syncthreads();
            for (int i = tid; i < nn; i += blockDim.x) {
                S.front[i] = S.next[i];
                if (pass == 0 && has_frozen) S.pts[np + i] = S.next[i];
            }
            if (tid == 0) { sh_nfront = nn; if (pass == 0 && has_frozen) sh_npts = np + nn; }
            __syncthreads();
        }
    }

    const int n = sh_n;
    if (tid == 0) {
        s.hdr[0] = clock0 + (uint32_t)sh_q;
        o_n[b] = n;
        if (sh_q) atomicAdd(&counters[CB_CNT_QUERIES], (unsigned long long)sh_q);
        if (sh_hits) atomicAdd(&counters[CB_CNT_QUERY_HITS], (unsigned long long)sh_hits);
        if (sh_fq) atomicAdd(&counters[CB_CNT_FROZEN_QUERIES], (unsigned long long)sh_fq);
        if (sh_fhits) atomicAdd(&counters[CB_CNT_FROZEN_HITS], (unsigned long long)sh_fhits);
    }
    for (int i = tid; i < T; i += blockDim.x) {
        o_tok[(size_t)b * T + i] = S.tok[i];
        o_par[(size_t)b * T + i] = S.par[i];
        o_dep[(size_t)b * T + i] = S.dep[i];
        uint32_t m[4] = {0u, 0u, 0u, 0u};
        if (i < n) for (int c = i; c >= 0; c = S.par[c]) m[c >> 5] |= 1u << (c & 31);
        for (int k = 0; k < W; ++k) o_mask[((size_t)b * T + i) * W + k] = m[k];
    }
}

template <int FETCH>
__global__ void __launch_bounds__(256) cb_draft_kernel(CbTables t, CbTables tf, int T, int crt, int max_depth, int NL, int KF,
                                                       const int32_t* __restrict__ tokens, int64_t row_stride,
                                                       const int32_t* __restrict__ seq_len, const int32_t* __restrict__ upd_n_old,
                                                       int32_t* __restrict__ o_tok, int32_t* __restrict__ o_par,
                                                       int32_t* __restrict__ o_dep, uint32_t* __restrict__ o_mask,
                                                       int32_t* __restrict__ o_n, uint32_t* status,
                                                       unsigned long long* counters) {
    CB_PDL_ENTRY();
    extern __shared__ int32_t smem[];
    const int b = blockIdx.x;
    draft_body<FETCH>(t, tf, T, crt, max_depth, NL, KF, tokens, row_stride, b, seq_len[b], upd_n_old ? upd_n_old[b] : -1, o_tok, o_par, o_dep,
                      o_mask, o_n, status, counters, smem);
}

// Acceptance of one step and update + draft of the next in one launch (the three are a chain per sequence: Fig. 2).  The
// grid is the acceptance kernel's; the CTA that ends a sequence's acceptance appends the emitted tokens (accepted ones and
// the bonus token) to the sequence's history, advances its length, and goes on as that sequence's update-and-draft CTA.
struct AcceptArgs {
    int V, Dmax, chunk, chunks_per_row;
    const void* logits; int64_t logits_row_stride;
    const int32_t* tok; const int32_t* par; const int32_t* dep; const int32_t* n_nodes;
    unsigned long long* rowmax; uint32_t* ticket;
    int32_t* n_accept; int32_t* accept_nodes; int32_t* out_tokens; int32_t* target_out;
};

template <int FETCH, bool BF16>
__global__ void __launch_bounds__(256) cb_accept_draft_kernel(AcceptArgs a, CbTables t, CbTables tf, int T, int crt, int max_depth, int NL, int KF,
                                                              int32_t* tokens, int64_t row_stride, int32_t* seq_len,
                                                              int32_t* o_tok, int32_t* o_par, int32_t* o_dep, uint32_t* o_mask, int32_t* o_n,
                                                              uint32_t* status, unsigned long long* counters) {
    CB_PDL_ENTRY();
    extern __shared__ int32_t smem[];
    if (!accept_rows<BF16>(T, a.V, a.Dmax, a.chunk, a.chunks_per_row, a.logits, a.logits_row_stride, a.tok, a.par, a.dep, a.n_nodes, a.rowmax,
                           a.ticket, a.n_accept, a.accept_nodes, a.out_tokens, a.target_out))
        return;
    __threadfence_block();
    __syncthreads();                                            // the walk (first warp) has written the sequence's result
    const int b = blockIdx.z, tid = threadIdx.x;
    const int m = __ldcg(&a.n_accept[b]);
    const int have = min(max(__ldcg(&a.n_nodes[b]), 0), T) > 0 ? m + 1 : 0;   // tokens emitted (an empty tree emits none)
    const int L = seq_len[b];
    int L1 = L + have;
    if (L1 > row_stride) {
        // no room in the history: nothing is appended and the step is reported; the draft below continues from what is there
        if (tid == 0) atomicCAS(status, 0u, (uint32_t)CB_ERR_INVALID_ARG);
        L1 = L;
    } else if (tid < have) {
        tokens[(size_t)b * row_stride + L + tid] = __ldcg(&a.out_tokens[(size_t)b * (a.Dmax + 1) + tid]);
    }
    __threadfence_block();
    __syncthreads();
    if (tid == 0) seq_len[b] = L1;
    draft_body<FETCH>(t, tf, T, crt, max_depth, NL, KF, tokens, row_stride, b, L1, L, o_tok, o_par, o_dep, o_mask, o_n, status, counters, smem);
}

}  // namespace

extern "C" cb_status cb_update(cb_ctx* ctx, const int32_t* tokens, int64_t row_stride, const int32_t* n_old,
                               const int32_t* n_new, void* stream) {
    CB_CHECK_ARG(ctx && tokens && n_old && n_new && row_stride >= 1);
    const int B = ctx->cfg.batch, wpb = 4;
    CB_CUDA(cb_launch_pdl(ctx->cfg.FC <= 32 ? cb_update_kernel<1> : cb_update_kernel<2>, dim3((B + wpb - 1) / wpb), dim3(wpb * 32), 0, (cudaStream_t)stream, ctx->tables, B, tokens, row_stride,
                          n_old, n_new, ctx->d_status, ctx->d_counters));
    cb_count_launch(1);
    return CB_OK;
}

extern "C" cb_status cb_update_bulk(cb_ctx* ctx, const int32_t* tokens, int64_t row_stride, const int32_t* n_old,
                                    const int32_t* n_new, void* stream) {
    CB_CHECK_ARG(ctx && tokens && n_old && n_new && row_stride >= 1);
    const int B = ctx->cfg.batch;
    // enough warps per sequence to fill the GPU at small batch, fewer at large batch
    int wps = 1;
    while (wps < 256 && (long long)B * wps * 2 <= (long long)ctx->num_sms * 64) wps *= 2;
    BulkPlan* plan = reinterpret_cast<BulkPlan*>(ctx->d_bulk_plan);
    const bool free_path = ctx->bulk_scratch && B <= kBulkFreeMaxBatch && ctx->tables.refresh;
    if (free_path) {
        // order-free path for the sequences that qualify and fit the attached scratch; the kernel below does the others
        const BulkFreeView v = bulk_free_view(ctx->bulk_scratch, ctx->bulk_slots, B);
        const cudaStream_t st = (cudaStream_t)stream;
        const unsigned blocks = (unsigned)std::min<long long>((long long)v.S / 256, (long long)ctx->num_sms * 8);
        const unsigned wide = (unsigned)std::min<long long>((long long)v.S / 256, (long long)ctx->num_sms * 32);   // one item per thread, or a few
        CB_CUDA(cb_launch_pdl(cb_bulk_free_plan_kernel, dim3(1), dim3(1024), 0, st, ctx->tables, B, n_old, n_new, plan, v, ctx->d_counters));
        CB_CUDA(cb_launch_pdl(cb_bulk_free_clear_kernel, dim3(wide), dim3(256), 0, st, v));
        CB_CUDA(cb_launch_pdl(cb_bulk_free_reduce_kernel, dim3(wide), dim3(256), 0, st, ctx->tables, B, tokens, row_stride, (const BulkPlan*)plan, v,
                              ctx->d_status));
        CB_CUDA(cb_launch_pdl(cb_bulk_free_ranges_kernel, dim3(wide), dim3(256), 0, st, v));
        CB_CUDA(cb_launch_pdl(cb_bulk_free_scatter_kernel, dim3(wide), dim3(256), 0, st, v));
        CB_CUDA(cb_launch_pdl(cb_bulk_free_apply_kernel, dim3(blocks), dim3(256), 0, st, ctx->tables, B, tokens, row_stride, (const BulkPlan*)plan, v,
                              ctx->d_status, ctx->d_counters));
        cb_count_launch(6);
    } else {
        CB_CUDA(cb_launch_pdl(cb_bulk_plan_kernel, dim3((B + 127) / 128), dim3(128), 0, (cudaStream_t)stream, ctx->tables, B, n_old, n_new, plan));
        cb_count_launch(1);
    }
    const long long warps = (long long)B * wps;
    // kept entries per warp: four, fewer where 96 KB of shared memory per CTA (8 warps) do not hold that many
    const size_t way_bytes = ((size_t)ctx->tables.E + 4) * 4;
    const int n_ways = (int)std::max<size_t>(1, std::min<size_t>(4, (96 * 1024) / (8 * way_bytes)));
    const size_t smem = 8 * (size_t)n_ways * way_bytes;
    if (smem > 200 * 1024) return CB_ERR_UNSUPPORTED;
    if (smem > 48 * 1024) {
        static size_t opted[64] = {0};                         // largest size opted into so far, per device
        const int d = ctx->device & 63;
        if (opted[d] < smem) {
            CB_CUDA(cudaFuncSetAttribute(cb_update_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            opted[d] = smem;
        }
    }
    CB_CUDA(cb_launch_pdl(cb_update_bulk_kernel, dim3((unsigned)((warps + 7) / 8)), dim3(256), smem, (cudaStream_t)stream, ctx->tables, B, wps, n_ways,
                          tokens, row_stride, n_old, n_new, (const BulkPlan*)plan, ctx->d_status, ctx->d_counters));
    cb_count_launch(1);
    return CB_OK;
}

extern "C" cb_status cb_bulk_scratch_bytes(const cb_config* cfg, int64_t max_windows, size_t* bytes) {
    CB_CHECK_ARG(cfg && bytes && cfg->batch >= 1 && max_windows >= 1 && max_windows <= (int64_t)1 << 29);
    uint32_t S = 2048;
    while ((int64_t)S < 2 * max_windows) S <<= 1;
    *bytes = bulk_free_layout(S, cfg->batch).total;
    return CB_OK;
}

extern "C" cb_status cb_bulk_scratch_attach(cb_ctx* ctx, void* dev_scratch, size_t bytes) {
    CB_CHECK_ARG(ctx);
    ctx->bulk_scratch = nullptr;
    ctx->bulk_slots = 0;
    if (!dev_scratch) return CB_OK;
    CB_CHECK_ARG((reinterpret_cast<uintptr_t>(dev_scratch) & 255u) == 0);
    // the largest power-of-two slot count whose layout fits
    uint32_t S = 0;
    for (uint32_t c = 2048; c != 0 && c <= (1u << 30) && bulk_free_layout(c, ctx->cfg.batch).total <= bytes; c <<= 1) S = c;
    CB_CHECK_ARG(S != 0);
    ctx->bulk_scratch = dev_scratch;
    ctx->bulk_slots = S;
    return CB_OK;
}

static cb_status draft_launch(cb_ctx* ctx, const int32_t* tokens, int64_t row_stride, const int32_t* seq_len, const int32_t* upd_n_old,
                              int32_t* tree_tokens, int32_t* tree_parent, int32_t* tree_depth,
                              uint32_t* tree_mask, int32_t* n_nodes, void* stream) {
    CB_CHECK_ARG(ctx && tokens && seq_len && tree_tokens && tree_parent && tree_depth && tree_mask && n_nodes);
    CB_CHECK_ARG(row_stride >= 1);
    const cb_config& c = ctx->cfg;
    const int T = c.max_nodes;
    const int NL = min(T, (T - 1) / c.FL + 1);
    // A leaf can receive at most T - 1 followers (each adds a node), so no more than that many are staged per lookup.
    const int FCmax = ctx->has_frozen ? max(c.FC, ctx->frozen.FC) : c.FC;
    const int KF = max(1, min(FCmax, T - 1));
    const size_t smem = sizeof(int32_t) * ((size_t)3 * T + (size_t)11 * NL + (size_t)NL * c.FL * KF);
    if (smem > 200 * 1024) return CB_ERR_UNSUPPORTED;
    if (smem > 48 * 1024) {
        static size_t opted[64] = {0};                         // largest size opted into so far, per device
        const int d = ctx->device & 63;
        if (opted[d] < smem) {
            CB_CUDA(cudaFuncSetAttribute(cb_draft_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            CB_CUDA(cudaFuncSetAttribute(cb_draft_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            opted[d] = smem;
        }
    }
    const int threads = 32 * max(1, min(8, NL));
    CbTables tf = {};
    if (ctx->has_frozen) tf = ctx->frozen;
    CB_CUDA(cb_launch_pdl(FCmax <= 32 ? cb_draft_kernel<1> : cb_draft_kernel<2>, dim3(c.batch), dim3(threads), smem, (cudaStream_t)stream, ctx->tables, tf, T, c.crt, c.max_depth, NL, KF,
                          tokens, row_stride, seq_len, upd_n_old, tree_tokens, tree_parent, tree_depth, tree_mask, n_nodes, ctx->d_status, ctx->d_counters));
    cb_count_launch(1);
    return CB_OK;
}

extern "C" cb_status cb_draft_tree(cb_ctx* ctx, const int32_t* tokens, int64_t row_stride, const int32_t* seq_len,
                                   int32_t* tree_tokens, int32_t* tree_parent, int32_t* tree_depth,
                                   uint32_t* tree_mask, int32_t* n_nodes, void* stream) {
    return draft_launch(ctx, tokens, row_stride, seq_len, nullptr, tree_tokens, tree_parent, tree_depth, tree_mask, n_nodes, stream);
}

extern "C" cb_status cb_update_draft_tree(cb_ctx* ctx, const int32_t* tokens, int64_t row_stride, const int32_t* n_old,
                                          const int32_t* n_new, int32_t* tree_tokens, int32_t* tree_parent,
                                          int32_t* tree_depth, uint32_t* tree_mask, int32_t* n_nodes, void* stream) {
    CB_CHECK_ARG(n_old != nullptr);
    return draft_launch(ctx, tokens, row_stride, n_new, n_old, tree_tokens, tree_parent, tree_depth, tree_mask, n_nodes, stream);
}

extern "C" cb_status cb_accept_update_draft_tree(cb_ctx* ctx, const cb_accept_draft_args* a, void* stream) {
    CB_CHECK_ARG(ctx && a);
    CB_CHECK_ARG(a->logits && a->tree_tokens && a->tree_parent && a->tree_depth && a->n_nodes && a->n_accept && a->accept_nodes && a->out_tokens);
    CB_CHECK_ARG(a->tokens && a->seq_len && a->row_stride >= 1);
    CB_CHECK_ARG(a->next_tokens && a->next_parent && a->next_depth && a->next_mask && a->next_n_nodes);
    const cb_config& c = ctx->cfg;
    CB_CHECK_ARG(a->logits_dtype == CB_DTYPE_F32 || a->logits_dtype == CB_DTYPE_BF16);
    CB_CHECK_ARG(a->logits_row_stride >= c.vocab);
    const int esz = a->logits_dtype == CB_DTYPE_F32 ? 4 : 2;
    CB_CHECK_ARG(((uintptr_t)a->logits & (esz - 1)) == 0);
    if (c.batch > 65535) return CB_ERR_UNSUPPORTED;
    const int T = c.max_nodes;
    // the acceptance grid: about 32 KB of a logits row per CTA, fewer chunks when the batch alone fills the machine
    int chunk = 32768 / esz;
    if ((long)c.batch * T >= 8L * ctx->num_sms) chunk *= 4;
    int cpr = (c.vocab + chunk - 1) / chunk;
    chunk = ((c.vocab + cpr - 1) / cpr + 7) & ~7;
    cpr = (c.vocab + chunk - 1) / chunk;
    AcceptArgs aa;
    aa.V = c.vocab; aa.Dmax = c.max_depth; aa.chunk = chunk; aa.chunks_per_row = cpr;
    aa.logits = a->logits; aa.logits_row_stride = a->logits_row_stride;
    aa.tok = a->tree_tokens; aa.par = a->tree_parent; aa.dep = a->tree_depth; aa.n_nodes = a->n_nodes;
    aa.rowmax = ctx->d_rowmax; aa.ticket = ctx->d_ticket;
    aa.n_accept = a->n_accept; aa.accept_nodes = a->accept_nodes; aa.out_tokens = a->out_tokens; aa.target_out = a->target_ids_out;
    // the drafting CTA's shared memory, as in cb_draft_tree
    const int NL = min(T, (T - 1) / c.FL + 1);
    const int FCmax = ctx->has_frozen ? max(c.FC, ctx->frozen.FC) : c.FC;
    const int KF = max(1, min(FCmax, T - 1));
    const size_t smem = sizeof(int32_t) * ((size_t)3 * T + (size_t)11 * NL + (size_t)NL * c.FL * KF);
    if (smem > 200 * 1024) return CB_ERR_UNSUPPORTED;
    const bool bf = a->logits_dtype == CB_DTYPE_BF16;
    auto kernel = FCmax <= 32 ? (bf ? cb_accept_draft_kernel<1, true> : cb_accept_draft_kernel<1, false>)
                              : (bf ? cb_accept_draft_kernel<2, true> : cb_accept_draft_kernel<2, false>);
    if (smem > 48 * 1024) {
        static std::mutex mu;
        static size_t opted[64][4] = {};                       // largest size opted into so far, per device and kernel
        std::lock_guard<std::mutex> lock(mu);
        const int d = ctx->device & 63, k = (FCmax <= 32 ? 0 : 2) + (bf ? 1 : 0);
        if (opted[d][k] < smem) {
            CB_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            opted[d][k] = smem;
        }
    }
    CbTables tf = {};
    if (ctx->has_frozen) tf = ctx->frozen;
    CB_CUDA(cb_launch_pdl(kernel, dim3(cpr, T, c.batch), dim3(256), smem, (cudaStream_t)stream, aa, ctx->tables, tf, T, c.crt, c.max_depth, NL, KF,
                          a->tokens, a->row_stride, a->seq_len, a->next_tokens, a->next_parent, a->next_depth, a->next_mask, a->next_n_nodes,
                          ctx->d_status, ctx->d_counters));
    cb_count_launch(1);
    return CB_OK;
}
