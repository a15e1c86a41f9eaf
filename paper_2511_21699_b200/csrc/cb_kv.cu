// KV commit of the accepted path: the root and the accepted draft nodes become cached context.
//
// One CTA per (path position, sequence) copies that node's K row and V row (Hkv * D bf16 each) from the tree tensors
// into the paged pool with 16-byte loads and stores.  The last CTA of a sequence to finish advances ctx_len, so the
// length may be updated in place: every CTA has read the old value before any can have counted in.
#include "cb_common.cuh"

namespace {

__global__ void __launch_bounds__(128) cb_kv_commit_kernel(int T, int Dmax, int row_u4 /* Hkv * D * 2 / 16 */, int P, int max_pages, int num_pages,
                                                           uint4* __restrict__ k_pool, uint4* __restrict__ v_pool,
                                                           const int32_t* __restrict__ block_table, int32_t* ctx_len,
                                                           const uint4* __restrict__ k_tree, const uint4* __restrict__ v_tree,
                                                           const int32_t* __restrict__ n_accept, const int32_t* __restrict__ accept_nodes,
                                                           uint32_t* ticket, uint32_t* status) {
    CB_PDL_ENTRY();
    const int j = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    const int m = min(max(n_accept[b], 0), Dmax);
    const int ctx = ctx_len[b];
    const bool fits = ctx >= 0 && ctx + m + 1 <= max_pages * P;
    __shared__ int s_last;
    if (j <= m && fits) {
        const int node = j == 0 ? 0 : accept_nodes[(size_t)b * Dmax + j - 1];
        const int pos = ctx + j;
        const int page = block_table[(size_t)b * max_pages + pos / P];
        if (node >= 0 && node < T && page >= 0 && page < num_pages) {
            const size_t src = ((size_t)b * T + node) * row_u4, dst = ((size_t)page * P + pos % P) * row_u4;
            for (int k = tid; k < row_u4; k += blockDim.x) {
                k_pool[dst + k] = k_tree[src + k];
                v_pool[dst + k] = v_tree[src + k];
            }
        } else if (tid == 0) {
            atomicCAS(status, 0u, (uint32_t)CB_ERR_INVALID_ARG);     // a node or page index outside its tensor
        }
    } else if (j == 0 && !fits && tid == 0) {
        atomicCAS(status, 0u, (uint32_t)CB_ERR_KV_FULL);
    }
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        s_last = atomicAdd(&ticket[b], 1u) == gridDim.x - 1u ? 1 : 0;
    }
    __syncthreads();
    if (s_last && tid == 0) {
        if (fits) ctx_len[b] = ctx + m + 1;
        ticket[b] = 0u;
    }
}

}  // namespace

extern "C" cb_status cb_kv_commit(cb_ctx* ctx, const cb_kv_commit_args* a, void* stream) {
    CB_CHECK_ARG(ctx && a);
    CB_CHECK_ARG(a->k_pool && a->v_pool && a->block_table && a->ctx_len && a->k_tree && a->v_tree && a->n_accept && a->accept_nodes);
    CB_CHECK_ARG(a->max_pages >= 1 && a->num_pages >= 1);
    const uintptr_t al = (uintptr_t)a->k_pool | (uintptr_t)a->v_pool | (uintptr_t)a->k_tree | (uintptr_t)a->v_tree;
    CB_CHECK_ARG((al & 15) == 0);
    const cb_config& c = ctx->cfg;
    const int row_u4 = c.n_kv_heads * c.head_dim * 2 / 16;
    dim3 grid(c.max_depth + 1, c.batch);
    if (c.batch > 65535) return CB_ERR_UNSUPPORTED;
    CB_CUDA(cb_launch_pdl(cb_kv_commit_kernel, grid, dim3(128), 0, (cudaStream_t)stream, c.max_nodes, c.max_depth, row_u4, c.page_size, a->max_pages,
                          a->num_pages, (uint4*)a->k_pool, (uint4*)a->v_pool, a->block_table, a->ctx_len, (const uint4*)a->k_tree,
                          (const uint4*)a->v_tree, a->n_accept, a->accept_nodes, ctx->d_ticket, ctx->d_status));
    cb_count_launch(1);
    return CB_OK;
}
