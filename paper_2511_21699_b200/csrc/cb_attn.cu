// cb_tree_attn entry point, the split-KV combine pass and the plain CUDA-core attention kernel.
//
// The CUDA-core kernel is a debugging aid (CB_FLAG_ATTN_CUDA_CORES): four threads per query row, fp32
// dot products from bf16 tiles staged in shared memory, one online-softmax update per key.  The
// production path is the tensor-core kernel in cb_attn_tc.cu; both write the same partial format.
#include <math.h>

#include "cb_attn.cuh"

namespace {

// ---------------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(512) cb_attn_cc_kernel(CbAttnParams p) {
    constexpr int DQ = D / 4;
    __shared__ __align__(16) __nv_bfloat16 Ks[32][D];
    __shared__ __align__(16) __nv_bfloat16 Vs[32][D];
    const int split = blockIdx.x, mt = blockIdx.y, bk = blockIdx.z;
    const int b = bk / p.Hkv, kh = bk % p.Hkv;
    const int tid = threadIdx.x, rl = tid >> 2, qd = tid & 3;
    const int n = p.n_nodes[b], ctx = p.ctx_len[b];
    const int node = mt * p.NPT + rl / p.G;
    const bool exists = rl < p.NPT * p.G && node < p.T;
    const bool valid = exists && node < n;
    const int i = valid ? node : 0, h = kh * p.G + (valid ? rl % p.G : 0);

    float q[DQ], acc[DQ];
    {
        const __nv_bfloat16* qp = p.q + (((size_t)b * p.T + i) * p.Hq + h) * D + qd * DQ;
#pragma unroll
        for (int d = 0; d < DQ; ++d) { q[d] = valid ? __bfloat162float(qp[d]) * p.scale_log2 : 0.f; acc[d] = 0.f; }
    }
    float m = -INFINITY, l = 0.f;
    uint32_t mrow[4] = {0u, 0u, 0u, 0u};
    if (valid) for (int k = 0; k < p.W; ++k) mrow[k] = p.tree_mask[((size_t)b * p.T + i) * p.W + k];

    int t_lo, t_hi;
    cb_split_range(ctx, p.nsplit, split, &t_lo, &t_hi);
    const int nct = (ctx + CB_KT - 1) / CB_KT;
    for (int tile = t_lo; tile < t_hi; ++tile) {
        const bool is_tree = tile == nct;
        const int kbase = is_tree ? 0 : tile * CB_KT;
        const int klim = is_tree ? n : ctx;
        for (int sub = 0; sub < CB_KT / 32; ++sub) {
            const int k0 = kbase + sub * 32;
            if (k0 >= klim) break;
            __syncthreads();
            // stage 32 keys: thread -> (key, 16-byte chunk)
            constexpr int CH = D / 8;                      // uint4 chunks per row
            if (tid < 32 * CH) {
                const int kk = tid / CH, ch = tid % CH, key = k0 + kk;
                uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
                if (key < klim) {
                    size_t off;
                    if (is_tree) off = (((size_t)b * p.T + key) * p.Hkv + kh) * D;
                    else {
                        const int page = p.block_table[(size_t)b * p.max_pages + key / p.P];
                        off = (((size_t)page * p.P + key % p.P) * p.Hkv + kh) * D;
                    }
                    const __nv_bfloat16* kp = (is_tree ? p.k_tree : p.k_pool) + off;
                    const __nv_bfloat16* vp = (is_tree ? p.v_tree : p.v_pool) + off;
                    kv = *reinterpret_cast<const uint4*>(kp + ch * 8);
                    vv = *reinterpret_cast<const uint4*>(vp + ch * 8);
                }
                *reinterpret_cast<uint4*>(&Ks[kk][ch * 8]) = kv;
                *reinterpret_cast<uint4*>(&Vs[kk][ch * 8]) = vv;
            }
            __syncthreads();
            const int kn = min(32, klim - k0);
            for (int kk = 0; kk < kn; ++kk) {
                float s = 0.f;
#pragma unroll
                for (int d = 0; d < DQ; d += 2) {
                    const float2 kf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&Ks[kk][qd * DQ + d]));
                    s = fmaf(q[d], kf.x, s);
                    s = fmaf(q[d + 1], kf.y, s);
                }
                s += __shfl_xor_sync(CB_FULL, s, 1);
                s += __shfl_xor_sync(CB_FULL, s, 2);
                const int key = k0 + kk;
                const bool vis = valid && (!is_tree || ((mrow[key >> 5] >> (key & 31)) & 1u));
                if (vis) {
                    if (s > m) {
                        const float a = exp2f(m - s);
                        l *= a;
#pragma unroll
                        for (int d = 0; d < DQ; ++d) acc[d] *= a;
                        m = s;
                    }
                    const float pw = exp2f(s - m);
                    l += pw;
#pragma unroll
                    for (int d = 0; d < DQ; d += 2) {
                        const float2 vf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&Vs[kk][qd * DQ + d]));
                        acc[d] = fmaf(pw, vf.x, acc[d]);
                        acc[d + 1] = fmaf(pw, vf.y, acc[d + 1]);
                    }
                }
            }
        }
    }

    if (p.nsplit == 1) {
        if (exists) {
            const int io = node, ho = kh * p.G + rl % p.G;
            __nv_bfloat16* op = p.out + (((size_t)b * p.T + io) * p.Hq + ho) * D + qd * DQ;
            const float inv = (valid && l > 0.f) ? 1.f / l : 0.f;
#pragma unroll
            for (int d = 0; d < DQ; ++d) op[d] = __float2bfloat16_rn(acc[d] * inv);
            if (p.lse && qd == 0) p.lse[((size_t)b * p.Hq + ho) * p.T + io] = (valid && l > 0.f) ? (m + log2f(l)) * 0.6931471805599453f : 0.f;
        }
    } else {
        const size_t slot = ((size_t)bk * p.MT + mt) * p.nsplit + split;
        float* pp = p.part + (slot * CB_MT + rl) * (D + 4);
#pragma unroll
        for (int d = 0; d < DQ; ++d) pp[qd * DQ + d] = acc[d];
        if (qd == 0) { pp[D] = m; pp[D + 1] = l; }
    }
}

// ---------------------------------------------------------------------------------------------------
// Combine: one warp per output row; merges the nsplit partials of its unit.
template <int D>
__global__ void __launch_bounds__(256) cb_attn_combine_kernel(CbAttnParams p) {
    const int lane = threadIdx.x & 31;
    const long row = (long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);   // over B * Hkv * G * T
    const long rows_per_unit = (long)p.G * p.T;
    if (row >= (long)p.B * p.Hkv * rows_per_unit) return;
    const int bk = (int)(row / rows_per_unit), r = (int)(row % rows_per_unit);
    const int b = bk / p.Hkv, kh = bk % p.Hkv;
    const int i = r / p.G, h = kh * p.G + r % p.G;
    const int mt = i / p.NPT, rl = (i % p.NPT) * p.G + r % p.G;
    const int n = p.n_nodes[b];
    constexpr int PER = D / 32;
    float o[PER];
#pragma unroll
    for (int d = 0; d < PER; ++d) o[d] = 0.f;
    float M = -INFINITY, Lsum = 0.f;
    if (i < n) {
        const float* base = p.part + (((size_t)bk * p.MT + mt) * p.nsplit * CB_MT + rl) * (D + 4);
        const size_t sstride = (size_t)CB_MT * (D + 4);
        for (int s = 0; s < p.nsplit; ++s) M = fmaxf(M, base[s * sstride + D]);
        for (int s = 0; s < p.nsplit; ++s) {
            const float* pp = base + s * sstride;
            const float ms = pp[D];
            if (ms == -INFINITY) continue;
            const float w = exp2f(ms - M);
            Lsum += w * pp[D + 1];
#pragma unroll
            for (int d = 0; d < PER; ++d) o[d] = fmaf(w, pp[lane * PER + d], o[d]);
        }
    }
    const float inv = Lsum > 0.f ? 1.f / Lsum : 0.f;
    __nv_bfloat16* op = p.out + (((size_t)b * p.T + i) * p.Hq + h) * D + lane * PER;
#pragma unroll
    for (int d = 0; d < PER; ++d) op[d] = __float2bfloat16_rn(o[d] * inv);
    if (p.lse && lane == 0) p.lse[((size_t)b * p.Hq + h) * p.T + i] = Lsum > 0.f ? (M + log2f(Lsum)) * 0.6931471805599453f : 0.f;
}

}  // namespace

cb_status cb_attn_launch_cuda_cores(cb_ctx* ctx, const CbAttnParams& p, cudaStream_t st) {
    dim3 grid(p.nsplit, p.MT, p.B * p.Hkv);
    if (p.D == 128) cb_attn_cc_kernel<128><<<grid, 512, 0, st>>>(p);
    else cb_attn_cc_kernel<64><<<grid, 512, 0, st>>>(p);
    cb_count_launch(1);
    CB_CUDA(cudaGetLastError());
    return CB_OK;
}

cb_status cb_attn_launch_combine(cb_ctx* ctx, const CbAttnParams& p, cudaStream_t st) {
    const long rows = (long)p.B * p.Hkv * p.G * p.T;
    const int wpb = 8;
    const unsigned grid = (unsigned)((rows + wpb - 1) / wpb);
    if (p.D == 128) cb_attn_combine_kernel<128><<<grid, wpb * 32, 0, st>>>(p);
    else cb_attn_combine_kernel<64><<<grid, wpb * 32, 0, st>>>(p);
    cb_count_launch(1);
    CB_CUDA(cudaGetLastError());
    return CB_OK;
}

extern "C" cb_status cb_tree_attn(cb_ctx* ctx, const cb_attn_args* a, void* stream) {
    CB_CHECK_ARG(ctx && a);
    CB_CHECK_ARG(a->q && a->k_pool && a->v_pool && a->block_table && a->ctx_len && a->k_tree && a->v_tree &&
                 a->tree_mask && a->n_nodes && a->out);
    CB_CHECK_ARG(a->max_pages >= 1 && a->num_pages >= 1);
    const uintptr_t al = (uintptr_t)a->q | (uintptr_t)a->k_pool | (uintptr_t)a->v_pool | (uintptr_t)a->k_tree |
                         (uintptr_t)a->v_tree | (uintptr_t)a->out;
    CB_CHECK_ARG((al & 15) == 0);
    const cb_config& c = ctx->cfg;
    CbAttnParams p;
    p.q = (const __nv_bfloat16*)a->q; p.k_pool = (const __nv_bfloat16*)a->k_pool; p.v_pool = (const __nv_bfloat16*)a->v_pool;
    p.block_table = a->block_table; p.ctx_len = a->ctx_len;
    p.k_tree = (const __nv_bfloat16*)a->k_tree; p.v_tree = (const __nv_bfloat16*)a->v_tree;
    p.tree_mask = a->tree_mask; p.n_nodes = a->n_nodes;
    p.out = (__nv_bfloat16*)a->out; p.lse = a->lse; p.part = ctx->d_attn_part;
    p.B = c.batch; p.T = c.max_nodes; p.W = (c.max_nodes + 31) / 32; p.Hq = c.n_q_heads; p.Hkv = c.n_kv_heads;
    p.G = c.n_q_heads / c.n_kv_heads; p.D = c.head_dim; p.P = c.page_size;
    p.max_pages = a->max_pages; p.num_pages = a->num_pages;
    p.NPT = CB_MT / p.G;
    p.MT = (p.T + p.NPT - 1) / p.NPT;
    const float scale = a->scale > 0.f ? a->scale : 1.0f / sqrtf((float)c.head_dim);
    p.scale_log2 = scale * 1.4426950408889634f;
    p.status = ctx->d_status;
    // Split the keys of one (sequence, kv head, row tile) over several CTAs when the units alone cannot
    // fill the machine; partials are merged by the combine pass.
    const int max_ctx = a->max_ctx > 0 ? a->max_ctx : a->max_pages * c.page_size;
    const int max_tiles = (max_ctx + CB_KT - 1) / CB_KT + 1;
    const long units = (long)p.B * p.Hkv * p.MT;
    int nsplit = 1;
    if (units < 2L * ctx->num_sms) {
        nsplit = (int)((2L * ctx->num_sms + units - 1) / units);
        nsplit = (int)fminf((float)nsplit, (float)max_tiles);
        nsplit = (int)fminf((float)nsplit, (float)(ctx->attn_max_units / units));
        if (nsplit < 1) nsplit = 1;
    }
    p.nsplit = nsplit;
    cudaStream_t st = (cudaStream_t)stream;
    cb_status s;
    if (c.flags & CB_FLAG_ATTN_CUDA_CORES) s = cb_attn_launch_cuda_cores(ctx, p, st);
    else s = cb_attn_launch_tensor(ctx, p, st);
    if (s != CB_OK) return s;
    if (nsplit > 1) s = cb_attn_launch_combine(ctx, p, st);
    return s;
}
