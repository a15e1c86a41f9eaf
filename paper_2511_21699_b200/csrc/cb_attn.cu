// cb_tree_attn entry point and the plain CUDA-core attention kernel.
//
// The CUDA-core kernel is a debugging aid (CB_FLAG_ATTN_CUDA_CORES): four threads per query row, fp32
// dot products from bf16 tiles staged in shared memory, one online-softmax update per key, one CTA per
// (row tile, sequence, kv head).  The production path is the tensor-core kernel in cb_attn_tc.cu.
#include <math.h>

#include "cb_attn.cuh"

namespace {

// ---------------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(512) cb_attn_cc_kernel(CbAttnParams p) {
    constexpr int DQ = D / 4;
    __shared__ __align__(16) __nv_bfloat16 Ks[32][D];
    __shared__ __align__(16) __nv_bfloat16 Vs[32][D];
    const int mt = blockIdx.y, bk = blockIdx.z;
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

    const int nct = (ctx + CB_KT - 1) / CB_KT;
    for (int tile = 0; tile <= nct; ++tile) {
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

    if (exists) {
        const int io = node, ho = kh * p.G + rl % p.G;
        __nv_bfloat16* op = p.out + (((size_t)b * p.T + io) * p.Hq + ho) * D + qd * DQ;
        const float inv = (valid && l > 0.f) ? 1.f / l : 0.f;
#pragma unroll
        for (int d = 0; d < DQ; ++d) op[d] = __float2bfloat16_rn(acc[d] * inv);
        if (p.lse && qd == 0) p.lse[((size_t)b * p.Hq + ho) * p.T + io] = (valid && l > 0.f) ? (m + log2f(l)) * 0.6931471805599453f : 0.f;
    }
}

}  // namespace

cb_status cb_attn_launch_cuda_cores(cb_ctx* ctx, const CbAttnParams& p, cudaStream_t st) {
    dim3 grid(1, p.MT, p.B * p.Hkv);
    if (p.D == 128) cb_attn_cc_kernel<128><<<grid, 512, 0, st>>>(p);
    else cb_attn_cc_kernel<64><<<grid, 512, 0, st>>>(p);
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
    // The tensor-core kernel is persistent: one CTA per SM, each taking an equal share of all key tiles.
    p.nc = ctx->num_sms < CB_ATTN_MAX_CTAS ? ctx->num_sms : CB_ATTN_MAX_CTAS;
    p.cs = 0;
    {
        const long long cap = (long long)a->max_pages * c.page_size;
        const long long mc = a->max_ctx > 0 && a->max_ctx < cap ? a->max_ctx : cap;
        p.max_tiles = (int)((mc + CB_KT - 1) / CB_KT) + 1;
    }
    cudaStream_t st = (cudaStream_t)stream;
    if (c.flags & CB_FLAG_ATTN_CUDA_CORES) return cb_attn_launch_cuda_cores(ctx, p, st);
    return cb_attn_launch_tensor(ctx, p, st);
}
