// Drafts of another speculative-decoding method inserted into the tree as additional branches below the root.
//
// One warp per sequence.  A branch's place in the node order depends on how much of the earlier branches fitted, so lane 0
// first walks the branches in order and fixes each one's first node and length (cut at the size cap, the depth cap and at a
// negative token); the lanes then write the nodes of all branches in parallel.  A node of a chain sees the root, the chain's
// earlier nodes and itself, so its mask row is one bit plus a run of bits.
#include "cb_common.cuh"

namespace {

constexpr int kMaxBranches = 64;

__global__ void __launch_bounds__(32) cb_add_branches_kernel(int T, int max_depth, int K, int Lmax, const int32_t* __restrict__ branches,
                                                             const int32_t* __restrict__ branch_len, int32_t* __restrict__ tok,
                                                             int32_t* __restrict__ par, int32_t* __restrict__ dep, uint32_t* __restrict__ mask,
                                                             int32_t* __restrict__ n_nodes) {
    CB_PDL_ENTRY();
    const int b = blockIdx.x, lane = threadIdx.x;
    const int W = (T + 31) >> 5;
    __shared__ int s_start[kMaxBranches], s_len[kMaxBranches];
    __shared__ int s_n;
    const int n0 = min(max(n_nodes[b], 0), T);
    const int32_t* br = branches + (size_t)b * K * Lmax;
    // usable length of each branch: up to its first negative token, the stated length, the row length and the depth cap
    for (int k = lane; k < K; k += 32) {
        int len = min(min(max(branch_len[(size_t)b * K + k], 0), Lmax), max_depth);
        for (int j = 0; j < len; ++j)
            if (br[(size_t)k * Lmax + j] < 0) { len = j; break; }
        s_len[k] = len;
    }
    __syncwarp();
    if (lane == 0) {
        int n = n0;
        for (int k = 0; k < K; ++k) {
            const int len = n0 >= 1 ? min(s_len[k], T - n) : 0;
            s_start[k] = n; s_len[k] = len;
            n += len;
        }
        s_n = n;
    }
    __syncwarp();
    int32_t* tk = tok + (size_t)b * T;
    int32_t* pr = par + (size_t)b * T;
    int32_t* dp = dep + (size_t)b * T;
    uint32_t* mk = mask + (size_t)b * T * W;
    for (int k = 0; k < K; ++k) {
        const int start = s_start[k], len = s_len[k];
        for (int j = lane; j < len; j += 32) {
            const int node = start + j;
            tk[node] = br[(size_t)k * Lmax + j];
            pr[node] = j == 0 ? 0 : node - 1;
            dp[node] = j + 1;
            for (int w = 0; w < W; ++w) {
                // bits [start, node] that fall into word w, plus the root's bit
                const int lo = max(start, 32 * w), hi = min(node, 32 * w + 31);
                uint32_t m = 0u;
                if (lo <= hi) m = (hi - lo == 31 ? 0xFFFFFFFFu : ((1u << (hi - lo + 1)) - 1u)) << (lo - 32 * w);
                if (w == 0) m |= 1u;
                mk[(size_t)node * W + w] = m;
            }
        }
    }
    if (lane == 0) n_nodes[b] = s_n;
}

}  // namespace

extern "C" cb_status cb_tree_add_branches(cb_ctx* ctx, const int32_t* branches, const int32_t* branch_len, int32_t n_branches, int32_t max_len,
                                          int32_t* tree_tokens, int32_t* tree_parent, int32_t* tree_depth, uint32_t* tree_mask,
                                          int32_t* n_nodes, void* stream) {
    CB_CHECK_ARG(ctx && tree_tokens && tree_parent && tree_depth && tree_mask && n_nodes);
    CB_CHECK_ARG(n_branches >= 0 && n_branches <= kMaxBranches && max_len >= 1);
    CB_CHECK_ARG(n_branches == 0 || (branches && branch_len));
    if (n_branches == 0) return CB_OK;
    const cb_config& c = ctx->cfg;
    CB_CUDA(cb_launch_pdl(cb_add_branches_kernel, dim3(c.batch), dim3(32), 0, (cudaStream_t)stream, c.max_nodes, c.max_depth, n_branches, max_len, branches,
                          branch_len, tree_tokens, tree_parent, tree_depth, tree_mask, n_nodes));
    cb_count_launch(1);
    return CB_OK;
}
