// Offline construction of a frozen table from a token corpus on the GPU (Section 4: the most frequent LC n-grams of
// length LL become the leaders; each keeps the FC most frequent n-grams of length FL that follow it).
//
// A window is LL + FL consecutive tokens; the corpus of N tokens has M = N - LL - FL + 1 of them.  Everything is counting
// and selection on integers, done without sorting:
//   1. leader counts: every window inserts-or-increments its leader in an open-addressing table whose slots hold the
//      position of one occurrence (keys are compared by reading the corpus there) and a counter;
//   2. the LC best leaders under the order (count falling, tokens rising) are found by a most-significant-digit-first
//      radix select over the distinct leaders (one histogram pass per byte of the composite key), then written into the
//      frozen table's entries and hashed into its index;
//   3. follower counts: windows whose leader was selected insert-or-increment the whole window in a second table; the
//      distinct windows are then grouped by leader into one array (count per leader, exclusive scan, scatter);
//   4. every distinct window scans its leader's group and counts the windows that beat it under (count falling, follower
//      tokens rising), giving up at FC; a rank below FC is that follower's place in the entry.  A histogram of the counts'
//      binary orders of magnitude per leader gives the order below which no window can be among the FC best, so that the
//      many rare windows of a frequent leader leave at once.
// Which occurrence represents a key, and which entry id a leader gets, depends on timing; the table's content (and
// cb_frozen_dump's output) does not.
#include "cb_common.cuh"

namespace {

constexpr uint32_t kEmpty = 0xFFFFFFFFu;
constexpr uint32_t kBigGroup = 2048;          // distinct windows of one leader above which a window is ranked by a warp
constexpr int kMaxWords = 1 + CB_MAX_LL;      // composite selection key: ~count, then the leader's tokens

struct BuildState {                           // head of the scratch buffer
    uint32_t status;
    uint32_t n_uniq;                          // distinct leaders
    uint32_t n_sel;                           // entry ids handed out
    uint32_t n_big;                           // windows of large groups that are ranked by a whole warp each
    uint32_t k_rem;                           // radix select: rank still to be resolved inside the current prefix
    uint32_t prefix[kMaxWords];               // composite key of the LC-th best leader, resolved digit by digit
    uint32_t select_all;                      // no more than LC distinct leaders: all of them are taken
    uint32_t hist[256];
};

struct BuildView {
    BuildState* st;
    uint32_t* h1_pos; uint32_t* h1_cnt; int32_t* h1_eid;          // [S] leaders
    uint32_t* uniq;                                               // [M] slots of the distinct leaders
    uint32_t* h2_pos; uint32_t* h2_cnt; int32_t* h2_eid;          // [S] windows of selected leaders
    uint32_t* seg; uint32_t* seg_cnt;                             // [S] distinct windows grouped by leader: slot, count
    uint32_t* grp_n; uint32_t* grp_off; uint32_t* grp_fill;       // [LC] group size, start, scatter cursor per entry
    uint32_t* grp_hist;                                           // [LC][32] windows per floor(log2(count)); [0] becomes the cut-off order
    uint32_t S;                                                   // slots of each hash table (a power of two)
    const int32_t* corpus;
    uint32_t M;
    int LL, FL, LC, FC;
};

__device__ __forceinline__ uint64_t hash_tokens(const int32_t* p, int n) {
    uint64_t h = 0x9E3779B97F4A7C15ull ^ (uint64_t)n;
    for (int j = 0; j < n; ++j) { h = (h ^ (uint32_t)p[j]) * 0xFF51AFD7ED558CCDull; h ^= h >> 32; }
    h ^= h >> 33; h *= 0xC4CEB9FE1A85EC53ull; h ^= h >> 33;
    return h;
}
__device__ __forceinline__ bool same_tokens(const int32_t* a, const int32_t* b, int n) {
    for (int j = 0; j < n; ++j) if (a[j] != b[j]) return false;
    return true;
}
// Finds or creates the slot of the n-token key at corpus position i.  Returns the slot, or kEmpty when every slot was
// visited (cannot happen at the load factor the tables are sized for; reported as CB_ERR_PROBE_LIMIT).
__device__ __forceinline__ uint32_t find_or_claim(uint32_t* pos, uint32_t S, const int32_t* corpus, uint32_t i, int n, bool* created) {
    uint32_t s = (uint32_t)(hash_tokens(corpus + i, n) >> 20) & (S - 1);
    *created = false;
    for (uint32_t p = 0; p < S; ++p) {
        uint32_t cur = pos[s];
        if (cur == kEmpty) {
            cur = atomicCAS(&pos[s], kEmpty, i);
            if (cur == kEmpty) { *created = true; return s; }
        }
        if (same_tokens(corpus + cur, corpus + i, n)) return s;
        s = (s + 1) & (S - 1);
    }
    return kEmpty;
}
__device__ __forceinline__ uint32_t find_only(const uint32_t* pos, uint32_t S, const int32_t* corpus, uint32_t i, int n) {
    uint32_t s = (uint32_t)(hash_tokens(corpus + i, n) >> 20) & (S - 1);
    for (uint32_t p = 0; p < S; ++p) {
        const uint32_t cur = pos[s];
        if (cur == kEmpty) return kEmpty;
        if (same_tokens(corpus + cur, corpus + i, n)) return s;
        s = (s + 1) & (S - 1);
    }
    return kEmpty;
}

__global__ void fb_init_kernel(BuildView v, CbTables t) {
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = g; i < v.S; i += stride) {
        v.h1_pos[i] = kEmpty; v.h1_cnt[i] = 0u; v.h1_eid[i] = -1;
        v.h2_pos[i] = kEmpty; v.h2_cnt[i] = 0u; v.h2_eid[i] = -1;
    }
    for (size_t i = g; i < (size_t)v.LC; i += stride) { v.grp_n[i] = 0u; v.grp_off[i] = 0u; v.grp_fill[i] = 0u; t.lstamp[i] = 0u; }
    for (size_t i = g; i < (size_t)v.LC * 32; i += stride) v.grp_hist[i] = 0u;
    for (size_t i = g; i < t.nslots; i += stride) t.index[i] = CB_IDX_EMPTY;
    for (size_t i = g; i < (size_t)v.LC * t.E; i += stride) t.entries[i] = 0u;
    if (g < sizeof(BuildState) / 4) reinterpret_cast<uint32_t*>(v.st)[g] = 0u;
    if (g < 4) t.hdr[g] = 0u;
}

// 1. leader counts
__global__ void fb_count_leaders_kernel(BuildView v) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < v.M; i += stride) {
        bool neg = false;
        for (int j = 0; j < v.LL + v.FL; ++j) neg |= v.corpus[i + j] < 0;
        if (neg) { atomicCAS(&v.st->status, 0u, (uint32_t)CB_ERR_INVALID_ARG); continue; }
        bool created;
        const uint32_t s = find_or_claim(v.h1_pos, v.S, v.corpus, (uint32_t)i, v.LL, &created);
        if (s == kEmpty) { atomicCAS(&v.st->status, 0u, (uint32_t)CB_ERR_PROBE_LIMIT); continue; }
        atomicAdd(&v.h1_cnt[s], 1u);
        if (created) v.uniq[atomicAdd(&v.st->n_uniq, 1u)] = s;
    }
}

__device__ __forceinline__ uint32_t sel_word(const BuildView& v, uint32_t slot, int w) {
    return w == 0 ? ~v.h1_cnt[slot] : (uint32_t)v.corpus[v.h1_pos[slot] + (w - 1)];
}

__global__ void fb_select_begin_kernel(BuildView v) {
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        v.st->select_all = v.st->n_uniq <= (uint32_t)v.LC ? 1u : 0u;
        v.st->k_rem = (uint32_t)v.LC;
    }
}
// 2a. histogram of byte `shift` of word `w` over the distinct leaders that match the prefix resolved so far
__global__ void fb_select_hist_kernel(BuildView v, int w, int shift) {
    __shared__ uint32_t sh[256];
    if (v.st->select_all) return;
    sh[threadIdx.x] = 0u;                     // blockDim.x == 256
    __syncthreads();
    const uint32_t n = v.st->n_uniq;
    const uint32_t hi_mask = shift == 24 ? 0u : (0xFFFFFFFFu << (shift + 8));
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const uint32_t slot = v.uniq[i];
        bool ok = true;
        for (int k = 0; k < w && ok; ++k) ok = sel_word(v, slot, k) == v.st->prefix[k];
        if (!ok) continue;
        const uint32_t x = sel_word(v, slot, w);
        if ((x & hi_mask) != (v.st->prefix[w] & hi_mask)) continue;
        atomicAdd(&sh[(x >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (sh[threadIdx.x]) atomicAdd(&v.st->hist[threadIdx.x], sh[threadIdx.x]);
}
// 2b. picks the digit in which the k-th smallest composite key lies
__global__ void fb_select_step_kernel(BuildView v, int w, int shift) {
    if (threadIdx.x != 0 || v.st->select_all) return;
    uint32_t k = v.st->k_rem, cum = 0, d = 255;
    for (uint32_t b = 0; b < 256; ++b) {
        const uint32_t c = v.st->hist[b];
        if (cum + c >= k) { d = b; break; }
        cum += c;
    }
    v.st->k_rem = k - cum;
    v.st->prefix[w] |= d << shift;
    for (int b = 0; b < 256; ++b) v.st->hist[b] = 0u;
}
// 2c. the selected leaders get their entries; their keys go into the frozen table's index
__global__ void fb_place_leaders_kernel(BuildView v, CbTables t) {
    const uint32_t n = v.st->n_uniq;
    const int W = 1 + v.LL;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const uint32_t slot = v.uniq[i];
        bool take = v.st->select_all != 0u;
        if (!take) {
            take = true;                      // composite key <= the threshold, compared word by word
            for (int k = 0; k < W; ++k) {
                const uint32_t x = sel_word(v, slot, k), y = v.st->prefix[k];
                if (x != y) { take = x < y; break; }
            }
        }
        if (!take) continue;
        const uint32_t eid = atomicAdd(&v.st->n_sel, 1u);
        if (eid >= (uint32_t)v.LC) { atomicCAS(&v.st->status, 0u, (uint32_t)CB_ERR_PROBE_LIMIT); continue; }
        v.h1_eid[slot] = (int32_t)eid;
        const int32_t* key = v.corpus + v.h1_pos[slot];
        uint32_t* e = t.entries + (size_t)eid * t.E;
        int32_t k4[4] = {0, 0, 0, 0};
        for (int j = 0; j < v.LL; ++j) { k4[j] = key[j]; e[j] = (uint32_t)key[j]; }
        t.lstamp[eid] = v.h1_cnt[slot];
        const uint64_t h = cb_hash4(k4[0], k4[1], k4[2], k4[3], v.LL);
        const uint32_t nb = t.nslots >> 5, word = (cb_hash_tag(h) << CB_EID_BITS) | eid;
        uint32_t bucket = cb_hash_bucket(h, t.nslots);
        bool placed = false;
        for (uint32_t p = 0; p < nb && !placed; ++p) {
            for (uint32_t l = 0; l < 32 && !placed; ++l) {
                uint32_t* w = &t.index[bucket * 32 + l];
                if (*w == CB_IDX_EMPTY && atomicCAS(w, CB_IDX_EMPTY, word) == CB_IDX_EMPTY) placed = true;
            }
            bucket = (bucket + 1) & (nb - 1);
        }
        if (!placed) atomicCAS(&v.st->status, 0u, (uint32_t)CB_ERR_PROBE_LIMIT);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) t.hdr[1] = min(n, (uint32_t)v.LC);
}

// 3a. follower counts of the selected leaders; every leader learns how many distinct windows it has
__global__ void fb_count_followers_kernel(BuildView v) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < v.M; i += stride) {
        bool neg = false;
        for (int j = 0; j < v.LL + v.FL; ++j) neg |= v.corpus[i + j] < 0;
        if (neg) continue;
        const uint32_t ls = find_only(v.h1_pos, v.S, v.corpus, (uint32_t)i, v.LL);
        if (ls == kEmpty) continue;
        const int32_t eid = v.h1_eid[ls];
        if (eid < 0) continue;
        bool created;
        const uint32_t s = find_or_claim(v.h2_pos, v.S, v.corpus, (uint32_t)i, v.LL + v.FL, &created);
        if (s == kEmpty) { atomicCAS(&v.st->status, 0u, (uint32_t)CB_ERR_PROBE_LIMIT); continue; }
        atomicAdd(&v.h2_cnt[s], 1u);
        if (created) {
            v.h2_eid[s] = eid;
            atomicAdd(&v.grp_n[eid], 1u);
        }
    }
}
// 3b. exclusive scan of the group sizes (one block; each thread owns a contiguous run of entries)
__global__ void __launch_bounds__(1024) fb_group_scan_kernel(BuildView v) {
    __shared__ uint32_t part[1024];
    const uint32_t n = v.st->n_sel < (uint32_t)v.LC ? v.st->n_sel : (uint32_t)v.LC;
    const uint32_t per = (n + 1023u) / 1024u, lo = threadIdx.x * per, hi = min(n, lo + per);
    uint32_t sum = 0;
    for (uint32_t i = lo; i < hi; ++i) sum += v.grp_n[i];
    part[threadIdx.x] = sum;
    __syncthreads();
    for (int o = 1; o < 1024; o <<= 1) {
        const uint32_t add = threadIdx.x >= o ? part[threadIdx.x - o] : 0u;
        __syncthreads();
        part[threadIdx.x] += add;
        __syncthreads();
    }
    uint32_t run = part[threadIdx.x] - sum;
    for (uint32_t i = lo; i < hi; ++i) { v.grp_off[i] = run; run += v.grp_n[i]; }
}
// 3c. the distinct windows, grouped by leader, with their counts beside them
__global__ void fb_group_scatter_kernel(BuildView v) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t s = (size_t)blockIdx.x * blockDim.x + threadIdx.x; s < v.S; s += stride) {
        if (v.h2_pos[s] == kEmpty) continue;
        const int32_t eid = v.h2_eid[s];
        const uint32_t at = v.grp_off[eid] + atomicAdd(&v.grp_fill[eid], 1u);
        v.seg[at] = (uint32_t)s;
        const uint32_t c = v.h2_cnt[s];
        v.seg_cnt[at] = c;
        atomicAdd(&v.grp_hist[(size_t)eid * 32 + (31 - __clz(c))], 1u);
    }
}
// 3d. per leader, the smallest order of magnitude that can still hold one of the FC most frequent windows
__global__ void fb_group_cutoff_kernel(BuildView v) {
    const uint32_t n = v.st->n_sel < (uint32_t)v.LC ? v.st->n_sel : (uint32_t)v.LC;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        uint32_t* h = v.grp_hist + e * 32;
        uint32_t acc = 0;
        int b = 31;
        for (; b > 0; --b) {
            acc += h[b];
            if (acc >= (uint32_t)v.FC) break;
        }
        h[0] = (uint32_t)b;                                  // orders below b hold none of the FC best
    }
}

// 4. rank of every distinct window among its leader's windows; the FC best become the entry's followers
__global__ void fb_rank_followers_kernel(BuildView v, CbTables t) {
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t s = (size_t)blockIdx.x * blockDim.x + threadIdx.x; s < v.S; s += stride) {
        if (v.h2_pos[s] == kEmpty) continue;
        const int32_t eid = v.h2_eid[s];
        const uint32_t mycnt = v.h2_cnt[s];
        if ((uint32_t)(31 - __clz(mycnt)) < v.grp_hist[(size_t)eid * 32]) continue;   // FC windows of higher order exist
        const int32_t* mine = v.corpus + v.h2_pos[s] + v.LL;
        const uint32_t lo = v.grp_off[eid], hi = lo + v.grp_n[eid];
        if (hi - lo > kBigGroup) {                           // a long scan: left to a warp (the list reuses the leaders' array)
            v.uniq[atomicAdd(&v.st->n_big, 1u)] = (uint32_t)s;
            continue;
        }
        int rank = 0;
        for (uint32_t k = lo; k < hi && rank < v.FC; ++k) {
            const uint32_t c = v.seg_cnt[k];
            if (c < mycnt) continue;
            bool beats = c > mycnt;
            if (!beats) {
                const uint32_t o = v.seg[k];
                if (o == (uint32_t)s) continue;
                const int32_t* other = v.corpus + v.h2_pos[o] + v.LL;
                for (int j = 0; j < v.FL; ++j)
                    if (other[j] != mine[j]) { beats = other[j] < mine[j]; break; }
            }
            rank += beats ? 1 : 0;
        }
        if (rank >= v.FC) continue;
        uint32_t* e = t.entries + (size_t)eid * t.E;
        for (int j = 0; j < v.FL; ++j) e[v.LL + v.FC + rank * v.FL + j] = (uint32_t)mine[j];
        e[v.LL + rank] = (uint32_t)(v.FC - rank);
    }
}

// 4b. the same for the windows of large groups, one warp per window: the lanes stride over the group
__global__ void fb_rank_big_kernel(BuildView v, CbTables t) {
    const int lane = threadIdx.x & 31;
    const size_t nwarps = (size_t)gridDim.x * (blockDim.x >> 5);
    const uint32_t n = v.st->n_big;
    for (size_t w = (size_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); w < n; w += nwarps) {
        const uint32_t s = v.uniq[w];
        const int32_t eid = v.h2_eid[s];
        const uint32_t mycnt = v.h2_cnt[s];
        const int32_t* mine = v.corpus + v.h2_pos[s] + v.LL;
        const uint32_t lo = v.grp_off[eid], hi = lo + v.grp_n[eid];
        int rank = 0;
        for (uint32_t k0 = lo; k0 < hi && rank < v.FC; k0 += 32) {
            const uint32_t k = k0 + lane;
            bool beats = false;
            if (k < hi) {
                const uint32_t c = v.seg_cnt[k];
                beats = c > mycnt;
                if (c == mycnt) {
                    const uint32_t o = v.seg[k];
                    if (o != s) {
                        const int32_t* other = v.corpus + v.h2_pos[o] + v.LL;
                        for (int j = 0; j < v.FL; ++j)
                            if (other[j] != mine[j]) { beats = other[j] < mine[j]; break; }
                    }
                }
            }
            rank += __popc(__ballot_sync(0xFFFFFFFFu, beats));
        }
        if (rank >= v.FC) continue;
        uint32_t* e = t.entries + (size_t)eid * t.E;
        if (lane < v.FL) e[v.LL + v.FC + rank * v.FL + lane] = (uint32_t)mine[lane];
        if (lane == 0) e[v.LL + rank] = (uint32_t)(v.FC - rank);
    }
}

size_t fb_align(size_t x) { return (x + 255) / 256 * 256; }

struct BuildLayout {
    uint32_t S;
    size_t off_h1_pos, off_h1_cnt, off_h1_eid, off_uniq, off_h2_pos, off_h2_cnt, off_h2_eid, off_seg, off_seg_cnt, off_grp, off_hist, total;
};

cb_status fb_layout(const cb_frozen_config* c, int64_t n_tokens, BuildLayout* B) {
    if (n_tokens < 0 || n_tokens > (int64_t)1 << 30) return CB_ERR_INVALID_ARG;
    const int64_t M = n_tokens - c->LL - c->FL + 1 > 0 ? n_tokens - c->LL - c->FL + 1 : 0;
    uint64_t S = 1024;
    while (S < 2ull * (uint64_t)M) S <<= 1;
    B->S = (uint32_t)S;
    size_t o = fb_align(sizeof(BuildState));
    B->off_h1_pos = o;  o = fb_align(o + S * 4);
    B->off_h1_cnt = o;  o = fb_align(o + S * 4);
    B->off_h1_eid = o;  o = fb_align(o + S * 4);
    B->off_uniq = o;    o = fb_align(o + (size_t)(M > 0 ? M : 1) * 4);
    B->off_h2_pos = o;  o = fb_align(o + S * 4);
    B->off_h2_cnt = o;  o = fb_align(o + S * 4);
    B->off_h2_eid = o;  o = fb_align(o + S * 4);
    B->off_seg = o;     o = fb_align(o + S * 4);
    B->off_seg_cnt = o; o = fb_align(o + S * 4);
    B->off_grp = o;     o = fb_align(o + (size_t)c->LC * 4 * 3);
    B->off_hist = o;    o = fb_align(o + (size_t)c->LC * 4 * 32);
    B->total = o;
    return CB_OK;
}

}  // namespace

extern "C" cb_status cb_frozen_build_bytes(const cb_frozen_config* cfg, int64_t n_tokens, size_t* scratch_bytes) {
    CbFrozenLayout L;
    BuildLayout B;
    if (!scratch_bytes) return CB_ERR_INVALID_ARG;
    cb_status s = cb_frozen_layout(cfg, &L);
    if (s != CB_OK) return s;
    s = fb_layout(cfg, n_tokens, &B);
    if (s != CB_OK) return s;
    *scratch_bytes = B.total;
    return CB_OK;
}

extern "C" cb_status cb_frozen_build(const cb_frozen_config* cfg, const int32_t* dev_corpus, int64_t n_tokens, void* dev_table,
                                     size_t table_bytes, void* dev_scratch, size_t scratch_bytes, void* stream) {
    CbFrozenLayout L;
    BuildLayout B;
    cb_status s = cb_frozen_layout(cfg, &L);
    if (s != CB_OK) return s;
    s = fb_layout(cfg, n_tokens, &B);
    if (s != CB_OK) return s;
    CB_CHECK_ARG(dev_table && ((uintptr_t)dev_table & 255) == 0 && dev_scratch && ((uintptr_t)dev_scratch & 255) == 0);
    CB_CHECK_ARG(dev_corpus || n_tokens == 0);
    if (table_bytes < L.total || scratch_bytes < B.total) return CB_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = (cudaStream_t)stream;
    CbTables t = cb_frozen_view(cfg, L, dev_table);
    char* base = (char*)dev_scratch;
    BuildView v;
    v.st = (BuildState*)base;
    v.h1_pos = (uint32_t*)(base + B.off_h1_pos); v.h1_cnt = (uint32_t*)(base + B.off_h1_cnt); v.h1_eid = (int32_t*)(base + B.off_h1_eid);
    v.uniq = (uint32_t*)(base + B.off_uniq);
    v.h2_pos = (uint32_t*)(base + B.off_h2_pos); v.h2_cnt = (uint32_t*)(base + B.off_h2_cnt); v.h2_eid = (int32_t*)(base + B.off_h2_eid);
    v.seg = (uint32_t*)(base + B.off_seg); v.seg_cnt = (uint32_t*)(base + B.off_seg_cnt);
    v.grp_n = (uint32_t*)(base + B.off_grp); v.grp_off = v.grp_n + cfg->LC; v.grp_fill = v.grp_off + cfg->LC;
    v.grp_hist = (uint32_t*)(base + B.off_hist);
    v.S = B.S;
    v.corpus = dev_corpus;
    const int64_t M = n_tokens - cfg->LL - cfg->FL + 1;
    v.M = (uint32_t)(M > 0 ? M : 0);
    v.LL = cfg->LL; v.FL = cfg->FL; v.LC = cfg->LC; v.FC = cfg->FC;
    int dev = 0, sms = 0;
    CB_CUDA(cudaGetDevice(&dev));
    CB_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const dim3 grid((unsigned)(sms * 8)), block(256);
    fb_init_kernel<<<grid, block, 0, st>>>(v, t);
    if (v.M > 0) {
        fb_count_leaders_kernel<<<grid, block, 0, st>>>(v);
        fb_select_begin_kernel<<<1, 32, 0, st>>>(v);
        for (int w = 0; w < 1 + cfg->LL; ++w)
            for (int shift = 24; shift >= 0; shift -= 8) {
                fb_select_hist_kernel<<<grid, block, 0, st>>>(v, w, shift);
                fb_select_step_kernel<<<1, 32, 0, st>>>(v, w, shift);
            }
        fb_place_leaders_kernel<<<grid, block, 0, st>>>(v, t);
        fb_count_followers_kernel<<<grid, block, 0, st>>>(v);
        fb_group_scan_kernel<<<1, 1024, 0, st>>>(v);
        fb_group_scatter_kernel<<<grid, block, 0, st>>>(v);
        fb_group_cutoff_kernel<<<grid, block, 0, st>>>(v);
        fb_rank_followers_kernel<<<grid, block, 0, st>>>(v, t);
        fb_rank_big_kernel<<<grid, block, 0, st>>>(v, t);
        cb_count_launch(9 + 8 * (1 + cfg->LL));
    }
    cb_count_launch(1);
    CB_CUDA(cudaGetLastError());
    uint32_t status = 0;
    CB_CUDA(cudaMemcpyAsync(&status, &v.st->status, 4, cudaMemcpyDeviceToHost, st));
    CB_CUDA(cudaStreamSynchronize(st));
    return (cb_status)status;
}
