// Tree attention: work decomposition shared by the tensor-core kernel, the CUDA-core kernel and the
// split-KV combine pass.
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
    float* part;          // [slot][128][D + 4]: unnormalised O row, running max (log2 domain), sum, 2 pad (rows stay 16-byte aligned)
    int B, T, W, Hq, Hkv, G, D, P, max_pages, num_pages;
    int NPT;              // tree nodes per row tile = 128 / G; a tile holds rows node_local * G + g
    int MT;               // row tiles per (sequence, kv head) = ceil(T / NPT)
    int nsplit;           // key splits per unit; 1 = write the output directly
    float scale_log2;     // softmax scale * log2(e)
    uint32_t* status;
};

// Key tiles of sequence b: ceil(ctx / 128) context tiles followed by one tile holding the tree keys.
// Split s of nsplit covers tiles [lo, hi).
__device__ __forceinline__ void cb_split_range(int ctx, int nsplit, int s, int* lo, int* hi) {
    const int tiles = (ctx + CB_KT - 1) / CB_KT + 1;
    *lo = (int)(((long long)tiles * s) / nsplit);
    *hi = (int)(((long long)tiles * (s + 1)) / nsplit);
}

cb_status cb_attn_launch_cuda_cores(cb_ctx* ctx, const CbAttnParams& p, cudaStream_t st);
cb_status cb_attn_launch_tensor(cb_ctx* ctx, const CbAttnParams& p, cudaStream_t st);
cb_status cb_attn_launch_combine(cb_ctx* ctx, const CbAttnParams& p, cudaStream_t st);
