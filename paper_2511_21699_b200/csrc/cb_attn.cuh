// Tree attention: work decomposition shared by the tensor-core kernels and the merge pass.
//
// Work is measured in key tiles of 128 keys.  Sequence b has tiles_b = ceil(ctx_b / 128) + 1 of them (the
// last one holds the tree's own keys).  A unit is one (sequence, kv head, row group): a row group is a
// pair of 128-row tiles (row = node_local * G + g, NPT = 128 / G nodes per tile), or a single tile when
// the whole tree fits one tile; only row tiles that hold valid nodes form units.  All units laid end to end give one
// global sequence of key tiles; it is cut into `nc` equal ranges, one per persistent CTA (or CTA pair): a stream-K split.
// The order of the units is (row group, sequence, kv head), row group outermost: the units that stream the same keys and
// values (one (sequence, kv head), all its row groups) then lie a fixed fraction of the whole sequence apart, so that they
// are worked on at the same time by different CTAs and the keys and values are fetched from HBM once and found in L2 by
// the others; with the row group innermost one CTA would stream them again and again, each time after everything else
// it holds has passed through L2.  Starting a unit costs about as much as two or
// three tiles (query load, pipeline refill, epilogue), so every unit is preceded by that many padding positions in the
// sequence: they carry no work, they only make a CTA that handles many short units receive fewer tiles.  A CTA therefore finishes whole
// units, plus at most one unit it shares with earlier CTAs and one it shares with later CTAs; shared
// units leave unnormalised partials that the merge pass combines.
#pragma once
#include "cb_common.cuh"

#define CB_KT 128        // keys per tile
#define CB_MT 128        // query rows per tile

struct CbAttnParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k_pool;
    const __nv_bfloat16* v_pool;
    const int32_t* block_table;
    const int32_t* ctx_len;
    const __nv_bfloat16* k_tree;
    const __nv_bfloat16* v_tree;
    const uint32_t* tree_mask;
    const int32_t* n_nodes;
    __nv_bfloat16* out;
    float* lse;
    float* part;          // [2 * nc slots][2 row tiles][128 rows][D + 4]: unnormalised O row, running max (log2 domain), sum
    int B, T, W, Hq, Hkv, G, D, P, max_pages, num_pages;
    int NPT;              // tree nodes per row tile = 128 / G
    int MT;               // row tiles that T nodes need = ceil(T / NPT)
    int nc;               // persistent CTAs (= ranges of the global tile sequence)
    int max_tiles;        // host's upper bound on the key tiles of a unit (from max_ctx, else from the block table's width)
    int cs;               // > 0: cluster mode, one unit per cluster of cs CTAs (see cb_attn_tc.cu); 0: the stream-K split
    float scale_log2;     // softmax scale * log2(e)
    uint32_t* status;
};

// Per-sequence shape of the decomposition.
struct CbSeqShape {
    int n, ctx, tiles, mtn, RG;
    int ov;               // padding positions in front of each unit of this sequence
    long long W;          // positions (padding + key tiles) of all units of this sequence
    // positions of this sequence's units of row group rg (all kv heads); 0 if the tree has no such row group
    __device__ __forceinline__ long long w_of(int Hkv, int rg) const { return rg < RG ? (long long)Hkv * (tiles + ov) : 0ll; }
};

__device__ __forceinline__ CbSeqShape cb_seq_shape(const CbAttnParams& p, int b) {
    CbSeqShape s;
    s.n = min(max(p.n_nodes[b], 0), p.T);
    s.ctx = min(max(p.ctx_len[b], 0), p.max_pages * p.P);
    s.tiles = (s.ctx + CB_KT - 1) / CB_KT + 1;
    s.mtn = (s.n + p.NPT - 1) / p.NPT;
    s.RG = p.MT == 1 ? (s.mtn > 0 ? 1 : 0) : (s.mtn + 1) / 2;
    s.ov = s.mtn >= 2 ? 3 : 2;
    s.W = (long long)p.Hkv * s.RG * (s.tiles + s.ov);
    return s;
}

__device__ __forceinline__ long long cb_range_start(long long total, int nc, int c) { return total * c / nc; }
// CTA whose range holds global tile x.
__device__ __forceinline__ int cb_cta_of(long long total, int nc, long long x) { return (int)(((x + 1) * nc - 1) / total); }

// Row groups a launch can have per sequence (trees of max_nodes nodes).
__device__ __forceinline__ int cb_max_row_groups(const CbAttnParams& p) { return p.MT == 1 ? 1 : (p.MT + 1) / 2; }

// Warp-collective: total weight of all sequences, and the (row group, sequence) holding global position g (with the
// global index at which that sequence's units of that row group start).  Every lane gets the results.
// max_row_tiles (optional): the largest number of row tiles that any sequence's tree has.
__device__ __forceinline__ long long cb_sched_total(const CbAttnParams& p, int lane, int* max_row_tiles = nullptr) {
    long long tot = 0;
    int mt = 0;
    for (int base = 0; base < p.B; base += 32) {
        const int b = base + lane;
        CbSeqShape s = {};
        if (b < p.B) s = cb_seq_shape(p, b);
        long long w = b < p.B ? s.W : 0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) w += __shfl_xor_sync(CB_FULL, w, o);
        tot += w;
        mt = max(mt, b < p.B ? s.mtn : 0);
    }
    if (max_row_tiles) *max_row_tiles = __reduce_max_sync(CB_FULL, mt);
    return tot;
}
__device__ __forceinline__ void cb_sched_locate(const CbAttnParams& p, long long g, int lane, int* rg_out, int* b_out, long long* pre_out) {
    long long run = 0;
    int frg = cb_max_row_groups(p), fb = p.B;
    long long fpre = 0;
    for (int rg = 0; rg < cb_max_row_groups(p) && fb == p.B; ++rg) {
        for (int base = 0; base < p.B; base += 32) {
            const int b = base + lane;
            const long long w = b < p.B ? cb_seq_shape(p, b).w_of(p.Hkv, rg) : 0;
            long long inc = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const long long t = __shfl_up_sync(CB_FULL, inc, o);
                if (lane >= o) inc += t;
            }
            const long long pre = run + inc - w;
            const uint32_t hit = __ballot_sync(CB_FULL, w > 0 && g >= pre && g < pre + w);
            if (hit) {
                const int l = __ffs(hit) - 1;
                frg = rg;
                fb = base + l;
                fpre = __shfl_sync(CB_FULL, pre, l);
                break;
            }
            run += __shfl_sync(CB_FULL, inc, 31);
        }
    }
    *rg_out = frg;
    *b_out = fb;
    *pre_out = fpre;
}

// One unit's share of a CTA's range: key tiles [t0, t1) of the unit's `tiles`.
struct CbUnit {
    int b, kh, rg, t0, t1, tiles, n, ctx, nrt;   // nrt = valid row tiles in the group (1 or 2)
};

// Walks the units of the range [g, g1).  Every role of a CTA runs its own copy and sees the same units.
struct CbWalker {
    long long g, g1, pre;     // pre: global position at which the units of (rg, b) start
    int rg, b;
    long long w;              // positions of the units of (rg, b)
    CbSeqShape s;
    bool fixed, fixed_left;   // cluster mode: the CTA has exactly one share of one unit (or none)
    CbUnit fu;
    __device__ __forceinline__ void init(const CbAttnParams& p, long long g0, long long g1_, int rg0, int b0, long long pre0) {
        g = g0; g1 = g1_; rg = rg0; b = b0; pre = pre0; fixed = false; fixed_left = false; w = 0;
        if (g < g1) { s = cb_seq_shape(p, b); w = s.w_of(p.Hkv, rg); }
    }
    __device__ __forceinline__ void init_fixed(const CbUnit& u0) {
        g = 0; g1 = 0; rg = 0; b = 0; pre = 0; w = 0; fixed = true; fixed_left = u0.t1 > u0.t0; fu = u0;
    }
    __device__ __forceinline__ bool next(const CbAttnParams& p, CbUnit* u) {
        if (fixed) {
            if (!fixed_left) return false;
            fixed_left = false;
            *u = fu;
            return true;
        }
        while (true) {
            if (g >= g1) return false;
            while (g >= pre + w) {                            // on to the next sequence that has this row group, then to the next row group
                pre += w;
                if (++b == p.B) { b = 0; ++rg; }
                s = cb_seq_shape(p, b);
                w = s.w_of(p.Hkv, rg);
            }
            const long long off = g - pre;
            const int vt = s.tiles + s.ov;                    // positions of one unit
            const int kh = (int)(off / vt);
            const int v0 = (int)(off - (long long)kh * vt);
            const int v1 = (int)min((long long)vt, (long long)v0 + (g1 - g));
            g += v1 - v0;
            u->t0 = max(v0 - s.ov, 0);
            u->t1 = max(v1 - s.ov, 0);
            if (u->t1 <= u->t0) continue;                     // only padding of this unit falls into the range
            u->b = b; u->kh = kh; u->rg = rg; u->tiles = s.tiles; u->n = s.n; u->ctx = s.ctx;
            u->nrt = p.MT == 1 ? 1 : min(2, s.mtn - 2 * rg);
            return true;
        }
    }
};

#define CB_ATTN_MAX_CTAS 160   // upper bound on persistent CTAs (>= SM count); sizes the partial buffer
static_assert(CB_ATTN_MAX_UNITS == 4 * CB_ATTN_MAX_CTAS, "partial buffer: two shared units of two row tiles per CTA");

cb_status cb_attn_launch_cuda_cores(cb_ctx* ctx, const CbAttnParams& p, cudaStream_t st);
cb_status cb_attn_launch_tensor(cb_ctx* ctx, const CbAttnParams& p, cudaStream_t st);
