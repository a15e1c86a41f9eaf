// Greedy acceptance: streaming arg-max over the logits of every valid tree node, then a warp-level walk
// that finds the longest verified path.  One launch: CTAs reduce chunks of logit rows into packed
// (value, index) maxima with 64-bit atomic max; the last CTA of a sequence to finish walks its tree.
#include "cb_accept_dev.cuh"

namespace {

template <bool BF16>
__global__ void __launch_bounds__(256) cb_accept_logits_kernel(
    int T, int V, int Dmax, int chunk, int chunks_per_row, const void* __restrict__ logits, int64_t row_stride,
    const int32_t* __restrict__ tok, const int32_t* __restrict__ par, const int32_t* __restrict__ dep,
    const int32_t* __restrict__ n_nodes, unsigned long long* rowmax, uint32_t* ticket,
    int32_t* __restrict__ n_accept, int32_t* __restrict__ accept_nodes, int32_t* __restrict__ out_tokens,
    int32_t* __restrict__ target_out) {
    CB_PDL_ENTRY();
    accept_rows<BF16>(T, V, Dmax, chunk, chunks_per_row, logits, row_stride, tok, par, dep, n_nodes, rowmax, ticket, n_accept, accept_nodes,
                      out_tokens, target_out);
}

__global__ void __launch_bounds__(128) cb_accept_ids_kernel(int B, int T, int Dmax, const int32_t* __restrict__ target_in,
                                                            const int32_t* __restrict__ tok, const int32_t* __restrict__ par,
                                                            const int32_t* __restrict__ dep, const int32_t* __restrict__ n_nodes,
                                                            int32_t* __restrict__ n_accept, int32_t* __restrict__ accept_nodes,
                                                            int32_t* __restrict__ out_tokens, int32_t* __restrict__ target_out) {
    CB_PDL_ENTRY();
    __shared__ int32_t s_target[4][CB_MAX_T];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int b = blockIdx.x * 4 + w;
    if (b >= B) return;
    const int n = min(max(n_nodes[b], 0), T);
    for (int k = lane; k < T; k += 32) {
        const int32_t tg = k < n ? target_in[(size_t)b * T + k] : -1;
        s_target[w][k] = tg;
        if (target_out) target_out[(size_t)b * T + k] = tg;
    }
    __syncwarp();
    accept_walk(b, Dmax, tok + (size_t)b * T, par + (size_t)b * T, dep + (size_t)b * T, n, s_target[w], n_accept, accept_nodes, out_tokens, lane);
}

}  // namespace

extern "C" cb_status cb_accept(cb_ctx* ctx, const int32_t* tree_tokens, const int32_t* tree_parent,
                               const int32_t* tree_depth, const int32_t* n_nodes, const void* logits,
                               int32_t logits_dtype, int64_t logits_row_stride, const int32_t* target_ids_in,
                               int32_t* n_accept, int32_t* accept_nodes, int32_t* out_tokens,
                               int32_t* target_ids_out, void* stream) {
    CB_CHECK_ARG(ctx && tree_tokens && tree_parent && tree_depth && n_nodes && n_accept && accept_nodes && out_tokens);
    CB_CHECK_ARG((logits != nullptr) != (target_ids_in != nullptr));
    const cb_config& c = ctx->cfg;
    const int T = c.max_nodes, Dmax = c.max_depth;
    cudaStream_t st = (cudaStream_t)stream;
    if (target_ids_in) {
        CB_CUDA(cb_launch_pdl(cb_accept_ids_kernel, dim3((c.batch + 3) / 4), dim3(128), 0, st, c.batch, T, Dmax, target_ids_in, tree_tokens,
                              tree_parent, tree_depth, n_nodes, n_accept, accept_nodes, out_tokens, target_ids_out));
    } else {
        CB_CHECK_ARG(logits_dtype == CB_DTYPE_F32 || logits_dtype == CB_DTYPE_BF16);
        CB_CHECK_ARG(logits_row_stride >= c.vocab);
        const int esz = logits_dtype == CB_DTYPE_F32 ? 4 : 2;
        CB_CHECK_ARG(((uintptr_t)logits & (esz - 1)) == 0);
        // chunk: about 32 KB of a row per CTA, fewer chunks when the batch alone fills the machine
        int chunk = 32768 / esz;
        const long rows = (long)c.batch * T;
        if (rows >= 8L * ctx->num_sms) chunk *= 4;
        int cpr = (c.vocab + chunk - 1) / chunk;
        chunk = ((c.vocab + cpr - 1) / cpr + 7) & ~7;
        cpr = (c.vocab + chunk - 1) / chunk;
        dim3 grid(cpr, T, c.batch);
        if (c.batch > 65535) return CB_ERR_UNSUPPORTED;
        if (logits_dtype == CB_DTYPE_F32)
            CB_CUDA(cb_launch_pdl(cb_accept_logits_kernel<false>, grid, dim3(256), 0, st, T, c.vocab, Dmax, chunk, cpr, logits, logits_row_stride,
                                  tree_tokens, tree_parent, tree_depth, n_nodes, ctx->d_rowmax, ctx->d_ticket, n_accept, accept_nodes,
                                  out_tokens, target_ids_out));
        else
            CB_CUDA(cb_launch_pdl(cb_accept_logits_kernel<true>, grid, dim3(256), 0, st, T, c.vocab, Dmax, chunk, cpr, logits, logits_row_stride,
                                  tree_tokens, tree_parent, tree_depth, n_nodes, ctx->d_rowmax, ctx->d_ticket, n_accept, accept_nodes,
                                  out_tokens, target_ids_out));
    }
    cb_count_launch(1);
    return CB_OK;
}

// ---------------------------------------------------------------------------------------------------
// cb_accept_static: the logits form of cb_accept for callers that are not allowed to allocate device
// memory (no workspace, no context).  Its scratch is this file-scope array, part of the library image:
// [0, CB_STATIC_MAX_ROWS) packed row maxima (8 bytes each), then CB_STATIC_MAX_BATCH arrival counters.
// In host code the name g_static_scratch is only a handle for cudaGetSymbolAddress, never a device
// pointer; the per-device address is looked up once and handed to the kernel as an ordinary argument.
#include <mutex>

static __device__ __align__(256) unsigned long long g_static_scratch[CB_STATIC_MAX_ROWS + CB_STATIC_MAX_BATCH / 2];

namespace {
constexpr int kMaxDevices = 64;
struct StaticSetup { unsigned long long* rowmax; uint32_t* ticket; int num_sms; bool ready; };
StaticSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

// One-time set-up for the current device: resolve the array's device address and read the SM count.
cb_status static_setup(int dev, StaticSetup* out) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    StaticSetup& s = g_setup[dev];
    if (!s.ready) {
        void* ptr = nullptr;
        CB_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
        int sms = 0;
        CB_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        s.rowmax = (unsigned long long*)ptr;
        s.ticket = (uint32_t*)(s.rowmax + CB_STATIC_MAX_ROWS);
        s.num_sms = sms;
        s.ready = true;
    }
    *out = s;
    return CB_OK;
}
}  // namespace

extern "C" cb_status cb_accept_static(int32_t batch, int32_t max_nodes, int32_t max_depth, int32_t vocab,
                                      const int32_t* tree_tokens, const int32_t* tree_parent, const int32_t* tree_depth,
                                      const int32_t* n_nodes, const void* logits, int32_t logits_dtype,
                                      int64_t logits_row_stride, int32_t* n_accept, int32_t* accept_nodes,
                                      int32_t* out_tokens, int32_t* target_ids_out, void* stream) {
    CB_CHECK_ARG(tree_tokens && tree_parent && tree_depth && n_nodes && logits && n_accept && accept_nodes && out_tokens);
    CB_CHECK_ARG(batch >= 1 && max_nodes >= 1 && max_nodes <= CB_MAX_T && max_depth >= 0 && vocab >= 1);
    CB_CHECK_ARG(logits_dtype == CB_DTYPE_F32 || logits_dtype == CB_DTYPE_BF16);
    CB_CHECK_ARG(logits_row_stride >= vocab);
    const int esz = logits_dtype == CB_DTYPE_F32 ? 4 : 2;
    CB_CHECK_ARG(((uintptr_t)logits & (esz - 1)) == 0);
    if (batch > CB_STATIC_MAX_BATCH || (long)batch * max_nodes > CB_STATIC_MAX_ROWS) {
        fprintf(stderr, "cacheback: cb_accept_static: batch %d x max_nodes %d exceeds the built-in scratch "
                        "(batch <= %d, batch * max_nodes <= %d)\n", batch, max_nodes, CB_STATIC_MAX_BATCH, CB_STATIC_MAX_ROWS);
        return CB_ERR_STATIC_LIMIT;
    }
    int dev = 0;
    CB_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CB_ERR_UNSUPPORTED;
    StaticSetup su;
    const cb_status ss = static_setup(dev, &su);
    if (ss != CB_OK) return ss;
    cudaStream_t st = (cudaStream_t)stream;
    // The array is shared by every call and keeps what the last one left: clear the part this call uses.
    CB_CUDA(cudaMemsetAsync(su.rowmax, 0, (size_t)batch * max_nodes * sizeof(unsigned long long), st));
    CB_CUDA(cudaMemsetAsync(su.ticket, 0, (size_t)batch * sizeof(uint32_t), st));
    int chunk = 32768 / esz;
    if ((long)batch * max_nodes >= 8L * su.num_sms) chunk *= 4;
    int cpr = (vocab + chunk - 1) / chunk;
    chunk = ((vocab + cpr - 1) / cpr + 7) & ~7;
    cpr = (vocab + chunk - 1) / chunk;
    dim3 grid(cpr, max_nodes, batch);
    if (logits_dtype == CB_DTYPE_F32)
        cb_accept_logits_kernel<false><<<grid, 256, 0, st>>>(max_nodes, vocab, max_depth, chunk, cpr, logits, logits_row_stride,
                                                             tree_tokens, tree_parent, tree_depth, n_nodes, su.rowmax, su.ticket,
                                                             n_accept, accept_nodes, out_tokens, target_ids_out);
    else
        cb_accept_logits_kernel<true><<<grid, 256, 0, st>>>(max_nodes, vocab, max_depth, chunk, cpr, logits, logits_row_stride,
                                                            tree_tokens, tree_parent, tree_depth, n_nodes, su.rowmax, su.ticket,
                                                            n_accept, accept_nodes, out_tokens, target_ids_out);
    cb_count_launch(1);
    CB_CUDA(cudaGetLastError());
    return CB_OK;
}
