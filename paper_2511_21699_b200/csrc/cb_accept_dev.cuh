// Device code of the greedy acceptance (Section 3.2), shared by the acceptance kernel and by the kernel that goes on to the
// next step's update and draft in the same launch: packed (value, index) maxima, streaming loads, the walk of a tree.
#pragma once
#include "cb_common.cuh"

namespace {

// Order-preserving map of a finite float to uint32 (larger float -> larger integer). -0 is folded into +0
// first so that equal values compare equal.
__device__ __forceinline__ uint32_t f2ord(float x) {
    x += 0.0f;
    const uint32_t u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
// Packed key: larger value wins, then the smaller index.
__device__ __forceinline__ unsigned long long pack(float x, uint32_t idx) {
    return ((unsigned long long)f2ord(x) << 32) | (unsigned long long)(0xFFFFFFFFu - idx);
}
__device__ __forceinline__ unsigned long long umax64(unsigned long long a, unsigned long long b) { return a > b ? a : b; }

// The logits are read once: no L1 allocation, and first to leave L2 (the tables of the step's other kernels stay).
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ float4 ldg_stream4(const float* p, uint64_t pol) {
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.f32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p), "l"(pol));
    return v;
}
__device__ __forceinline__ uint4 ldg_stream4u(const void* p, uint64_t pol) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(pol));
    return v;
}

// Walk of one sequence by one warp (n <= 128 nodes, parents precede children).
// tk, pa, de: the sequence's own tree rows (shared or global memory).
__device__ void accept_walk(int b, int Dmax, const int32_t* tk, const int32_t* pa, const int32_t* de, int n,
                            const int32_t* target_s /*shared, [T]*/,
                            int32_t* __restrict__ n_accept, int32_t* __restrict__ accept_nodes,
                            int32_t* __restrict__ out_tokens, int lane) {
    // key = (depth << 8) | (255 - index) for verified nodes: max = deepest, lowest index among ties
    uint32_t best = 0;
    for (int i = lane; i < n; i += 32) {
        bool good = true;
        int c = i;
        for (int guard = 0; guard < CB_MAX_T && c > 0; ++guard) {
            const int p = pa[c];
            if (p < 0 || p >= c) { good = false; break; }      // malformed tree: treat as unverified
            good = good && (tk[c] == target_s[p]);
            c = p;
        }
        // a depth outside [0, Dmax] cannot come from the drafter (malformed input): such a node counts as unverified, so the
        // winner's depth always fits the output rows
        const int d = de[i];
        if (good && d >= 0 && d <= Dmax) best = max(best, ((uint32_t)d << 8) | (uint32_t)(255 - i));
    }
    best = __reduce_max_sync(CB_FULL, best);
    int node = n > 0 ? 255 - (int)(best & 255u) : 0;
    int m = n > 0 ? (int)(best >> 8) : 0;
    if (node >= n) { node = 0; m = 0; }                        // nothing verified, not even the root (malformed input)
    for (int k = lane; k < Dmax; k += 32) accept_nodes[(size_t)b * Dmax + k] = -1;
    for (int k = lane; k <= Dmax; k += 32) out_tokens[(size_t)b * (Dmax + 1) + k] = -1;
    __syncwarp();
    if (lane == 0) {
        n_accept[b] = m;
        if (n > 0) {
            out_tokens[(size_t)b * (Dmax + 1) + m] = target_s[node];
            int c = node;
            for (int k = m - 1; k >= 0 && c > 0; --k) {
                accept_nodes[(size_t)b * Dmax + k] = c;
                out_tokens[(size_t)b * (Dmax + 1) + k] = tk[c];
                c = pa[c];
            }
        }
    }
}

// The work of one CTA of the acceptance grid (row chunk ck = blockIdx.x, node i = blockIdx.y, sequence b = blockIdx.z): its
// chunk of the node's logits row is reduced into the row's packed maximum; the last CTA of the sequence to arrive turns the
// maxima into the target's tokens, walks the tree and writes the result.  Returns true in that CTA (all its threads), after
// the result has been written; false in all others.
template <bool BF16>
__device__ __forceinline__ bool accept_rows(
    int T, int V, int Dmax, int chunk, int chunks_per_row, const void* __restrict__ logits, int64_t row_stride,
    const int32_t* __restrict__ tok, const int32_t* __restrict__ par, const int32_t* __restrict__ dep,
    const int32_t* __restrict__ n_nodes, unsigned long long* rowmax, uint32_t* ticket,
    int32_t* __restrict__ n_accept, int32_t* __restrict__ accept_nodes, int32_t* __restrict__ out_tokens,
    int32_t* __restrict__ target_out) {
    const int b = blockIdx.z, i = blockIdx.y, ck = blockIdx.x, tid = threadIdx.x;
    const int n = min(max(n_nodes[b], 0), T);
    // Rows past the tree have nothing to add and do not queue for the ticket either (hundreds of atomics on one word at
    // batch 1); an empty tree keeps row 0's CTAs, one of which writes the empty result.
    if (i >= max(n, 1)) return false;
    __shared__ unsigned long long s_red[8];
    __shared__ int32_t s_target[CB_MAX_T], s_tok[CB_MAX_T], s_par[CB_MAX_T], s_dep[CB_MAX_T];
    __shared__ int s_last;
    if (i < n) {
        const int v0 = ck * chunk, v1 = min(V, v0 + chunk);
        unsigned long long best = 0ull;
        const uint64_t pol = l2_evict_first_policy();
        if (!BF16) {
            const float* rowp = (const float*)logits + ((size_t)b * T + i) * row_stride;
            // head up to a 16-byte boundary, vector body, scalar tail
            int v = v0;
            const uintptr_t a = (uintptr_t)(rowp + v);
            int head = (int)(((16 - (a & 15)) & 15) >> 2);
            head = min(head, v1 - v);
            if (tid < head) best = pack(rowp[v + tid], (uint32_t)(v + tid));
            v += head;
            const int nvec = (v1 - v) >> 2;
            const float* base = rowp + v;
            for (int k = tid; k < nvec; k += blockDim.x * 4) {
                float4 x[4];
                int kk[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) { kk[u] = k + u * blockDim.x; if (kk[u] < nvec) x[u] = ldg_stream4(base + 4 * (size_t)kk[u], pol); }
#pragma unroll
                for (int u = 0; u < 4; ++u) if (kk[u] < nvec) {
                    const uint32_t id = (uint32_t)(v + 4 * kk[u]);
                    best = umax64(best, pack(x[u].x, id));
                    best = umax64(best, pack(x[u].y, id + 1));
                    best = umax64(best, pack(x[u].z, id + 2));
                    best = umax64(best, pack(x[u].w, id + 3));
                }
            }
            const int tail0 = v + 4 * nvec;
            if (tail0 + tid < v1) best = umax64(best, pack(rowp[tail0 + tid], (uint32_t)(tail0 + tid)));
        } else {
            const __nv_bfloat16* rowp = (const __nv_bfloat16*)logits + ((size_t)b * T + i) * row_stride;
            int v = v0;
            const uintptr_t a = (uintptr_t)(rowp + v);
            int head = (int)(((16 - (a & 15)) & 15) >> 1);
            head = min(head, v1 - v);
            if (tid < head) best = pack(__bfloat162float(rowp[v + tid]), (uint32_t)(v + tid));
            v += head;
            const int nvec = (v1 - v) >> 3;
            const __nv_bfloat16* base = rowp + v;
            for (int k = tid; k < nvec; k += blockDim.x * 4) {
                uint4 x[4];
                int kk[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) { kk[u] = k + u * blockDim.x; if (kk[u] < nvec) x[u] = ldg_stream4u(base + 8 * (size_t)kk[u], pol); }
#pragma unroll
                for (int u = 0; u < 4; ++u) if (kk[u] < nvec) {
                    const uint32_t id = (uint32_t)(v + 8 * kk[u]);
                    const uint32_t wds[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        best = umax64(best, pack(__uint_as_float(wds[q] << 16), id + 2 * q));
                        best = umax64(best, pack(__uint_as_float(wds[q] & 0xFFFF0000u), id + 2 * q + 1));
                    }
                }
            }
            const int tail0 = v + 8 * nvec;
            if (tail0 + tid < v1) best = umax64(best, pack(__bfloat162float(rowp[tail0 + tid]), (uint32_t)(tail0 + tid)));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) best = umax64(best, __shfl_xor_sync(CB_FULL, best, o));
        if ((tid & 31) == 0) s_red[tid >> 5] = best;
        __syncthreads();
        if (tid == 0) {
            for (int w = 1; w < (int)(blockDim.x >> 5); ++w) best = umax64(best, s_red[w]);
            atomicMax(&rowmax[(size_t)b * T + i], best);
        }
    }
    // The last CTA of this sequence to arrive owns the walk (and re-zeroes the scratch for the next call).
    if (tid == 0) {
        __threadfence();
        const uint32_t total = gridDim.x * (uint32_t)max(n, 1);
        s_last = (atomicAdd(&ticket[b], 1u) == total - 1u) ? 1 : 0;
    }
    __syncthreads();
    if (!s_last) return false;
    __threadfence();
    for (int k = tid; k < T; k += blockDim.x) {
        int32_t tg = -1;
        if (k < n) {
            const unsigned long long r = atomicExch(&rowmax[(size_t)b * T + k], 0ull);
            tg = (int32_t)(0xFFFFFFFFu - (uint32_t)(r & 0xFFFFFFFFull));
        }
        s_target[k] = tg;
        if (target_out) target_out[(size_t)b * T + k] = tg;
        // the tree's rows come along, so that the climb from each node to the root below reads shared memory
        s_tok[k] = k < n ? tok[(size_t)b * T + k] : -1;
        s_par[k] = k < n ? par[(size_t)b * T + k] : -1;
        s_dep[k] = k < n ? dep[(size_t)b * T + k] : -1;
    }
    if (tid == 0) ticket[b] = 0u;
    __syncthreads();
    if (tid < 32) accept_walk(b, Dmax, s_tok, s_par, s_dep, n, s_target, n_accept, accept_nodes, out_tokens, tid);
    return true;
}

}  // namespace
