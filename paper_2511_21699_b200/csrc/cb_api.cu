// Context management, workspace layout, table dump/load, status polling.
#include <algorithm>
#include <atomic>
#include <new>
#include <vector>

#include "cb_common.cuh"

static std::atomic<uint64_t> g_launches{0};
void cb_count_launch(int n) { g_launches.fetch_add((uint64_t)n); }
extern "C" uint64_t cb_launch_count(void) { return g_launches.load(); }

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static bool config_ok(const cb_config* c) {
    if (!c) return false;
    if (c->batch < 1 || c->batch > (1 << 16)) return false;
    if (c->LL < 1 || c->LL > CB_MAX_LL || c->FL < 1 || c->FL > CB_MAX_FL) return false;
    if (c->LC < 1 || c->LC > (1 << CB_EID_BITS) || c->FC < 1 || c->FC > CB_MAX_FC) return false;
    if (c->max_nodes < 1 || c->max_nodes > CB_MAX_T || c->crt < 0 || c->max_depth < 0) return false;
    if (c->vocab < 1) return false;
    if (c->n_q_heads < 1 || c->n_kv_heads < 1 || c->n_q_heads % c->n_kv_heads != 0) return false;
    if (c->n_q_heads / c->n_kv_heads > 16) return false;
    if (c->head_dim != 64 && c->head_dim != 128) return false;
    if (c->page_size != 16) return false;
    return true;
}

cb_status cb_compute_layout(const cb_config* c, CbLayout* L) {
    if (!config_ok(c)) return CB_ERR_INVALID_ARG;
    uint32_t ns = 32;
    while (ns < 4u * (uint32_t)c->LC) ns <<= 1;
    L->nslots = ns;
    L->E = (uint32_t)align_up((size_t)c->LL + (size_t)c->FC * (1 + c->FL), 4);
    size_t B = (size_t)c->batch, o = 0;
    L->n_guards = 0;
    // a region of `bytes` at the current offset; the checking build puts a guard area behind it
    auto region = [&](size_t bytes) {
        const size_t at = o;
        o = align_up(o + bytes, 256);
        if (CB_DEBUG_BUILD) { L->guard_off[L->n_guards++] = o; o += CB_GUARD_BYTES; }
        return at;
    };
    L->off_hdr = region(B * 4 * 4);
    L->off_index = region(B * ns * 4);
    L->off_lstamp = region(B * (size_t)c->LC * 4);
    L->off_entries = region(B * (size_t)c->LC * L->E * 4);
    L->off_status = region(4 * 4);
    L->off_counters = region(CB_NUM_COUNTERS * 8);
    L->off_rowmax = region(B * (size_t)c->max_nodes * 8);
    L->off_ticket = region(B * 4);
    L->off_bulk_plan = region(B * 16);
    L->attn_max_units = CB_ATTN_MAX_UNITS;
    L->attn_part_floats = (size_t)L->attn_max_units * 128 * ((size_t)c->head_dim + 4);
    L->off_attn_part = region(L->attn_part_floats * 4);
    L->total = o;
    return CB_OK;
}

extern "C" cb_status cb_workspace_bytes(const cb_config* cfg, size_t* bytes) {
    CbLayout L;
    if (!bytes) return CB_ERR_INVALID_ARG;
    cb_status s = cb_compute_layout(cfg, &L);
    if (s != CB_OK) return s;
    *bytes = L.total;
    return CB_OK;
}

extern "C" cb_status cb_create(const cb_config* cfg, void* dev_workspace, size_t bytes, cb_ctx** out) {
    CbLayout L;
    if (!out || !dev_workspace) return CB_ERR_INVALID_ARG;
    cb_status s = cb_compute_layout(cfg, &L);
    if (s != CB_OK) return s;
    if (((uintptr_t)dev_workspace & 255) != 0) return CB_ERR_INVALID_ARG;
    if (bytes < L.total) return CB_ERR_WORKSPACE_TOO_SMALL;
    cb_ctx* c = new (std::nothrow) cb_ctx();
    if (!c) return CB_ERR_CUDA;
    c->cfg = *cfg;
    c->ws = (char*)dev_workspace;
    c->ws_bytes = bytes;
    if (cudaGetDevice(&c->device) != cudaSuccess) { delete c; return CB_ERR_CUDA; }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, c->device) != cudaSuccess) { delete c; return CB_ERR_CUDA; }
    if (prop.major != 10) { delete c; return CB_ERR_UNSUPPORTED; }
    c->num_sms = prop.multiProcessorCount;
    CbTables& t = c->tables;
    t.hdr = (uint32_t*)(c->ws + L.off_hdr);
    t.index = (uint32_t*)(c->ws + L.off_index);
    t.lstamp = (uint32_t*)(c->ws + L.off_lstamp);
    t.entries = (uint32_t*)(c->ws + L.off_entries);
    t.nslots = L.nslots; t.E = L.E;
    t.LL = cfg->LL; t.FL = cfg->FL; t.LC = cfg->LC; t.FC = cfg->FC;
    t.refresh = (cfg->flags & CB_FLAG_NO_FOLLOWER_REFRESH) ? 0u : 1u;
    t.dbg_status = (uint32_t*)(c->ws + L.off_status);
    c->d_status = (uint32_t*)(c->ws + L.off_status);
    c->d_counters = (unsigned long long*)(c->ws + L.off_counters);
    c->d_rowmax = (unsigned long long*)(c->ws + L.off_rowmax);
    c->d_ticket = (uint32_t*)(c->ws + L.off_ticket);
    c->d_bulk_plan = (uint32_t*)(c->ws + L.off_bulk_plan);
    c->d_attn_part = (float*)(c->ws + L.off_attn_part);
    c->attn_part_floats = L.attn_part_floats;
    c->attn_max_units = L.attn_max_units;
    c->n_guards = L.n_guards;
    for (int g = 0; g < L.n_guards; ++g) c->guard_off[g] = L.guard_off[g];
    // Empty tables: header and index zero; entries and stamps need no initialisation (count = 0).
    bool ok = cudaMemset(c->ws + L.off_hdr, 0, L.off_lstamp - L.off_hdr) == cudaSuccess &&
              cudaMemset(c->ws + L.off_status, 0, L.off_attn_part - L.off_status) == cudaSuccess;
    for (int g = 0; g < L.n_guards && ok; ++g) ok = cudaMemset(c->ws + L.guard_off[g], CB_GUARD_BYTE, CB_GUARD_BYTES) == cudaSuccess;
    ok = ok && cudaDeviceSynchronize() == cudaSuccess;
    if (!ok) { delete c; return CB_ERR_CUDA; }
    *out = c;
    return CB_OK;
}

extern "C" void cb_destroy(cb_ctx* ctx) { delete ctx; }

extern "C" int cb_debug_build(void) { return CB_DEBUG_BUILD; }

__global__ void cb_reset_kernel(CbTables t, const int32_t* __restrict__ mask) {
    const int b = blockIdx.y;
    if (mask && mask[b] == 0) return;
    CbSeq s = cb_seq(t, b);
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < t.nslots; i += gridDim.x * blockDim.x) s.index[i] = 0;
    if (blockIdx.x == 0 && threadIdx.x < 4) s.hdr[threadIdx.x] = 0;
}

extern "C" cb_status cb_reset(cb_ctx* ctx, const int32_t* dev_seq_mask, void* stream) {
    CB_CHECK_ARG(ctx);
    uint32_t gx = std::min<uint32_t>(64, (ctx->tables.nslots + 255) / 256);
    cb_reset_kernel<<<dim3(gx, ctx->cfg.batch), 256, 0, (cudaStream_t)stream>>>(ctx->tables, dev_seq_mask);
    cb_count_launch(1);
    CB_CUDA(cudaGetLastError());
    return CB_OK;
}

extern "C" cb_status cb_table_dump(cb_ctx* ctx, int32_t seq, int32_t* n_leaders, int32_t* leaders,
                                   int32_t* n_followers, int32_t* followers) {
    CB_CHECK_ARG(ctx && seq >= 0 && seq < ctx->cfg.batch && n_leaders);
    const CbTables& t = ctx->tables;
    CB_CUDA(cudaDeviceSynchronize());
    uint32_t hdr[4];
    CB_CUDA(cudaMemcpy(hdr, t.hdr + (size_t)seq * 4, sizeof(hdr), cudaMemcpyDeviceToHost));
    const uint32_t n = hdr[1];
    if (n > (uint32_t)t.LC) return CB_ERR_CUDA;
    *n_leaders = (int32_t)n;
    if (n == 0) return CB_OK;
    std::vector<uint32_t> st(n), ent((size_t)n * t.E);
    CB_CUDA(cudaMemcpy(st.data(), t.lstamp + (size_t)seq * t.LC, (size_t)n * 4, cudaMemcpyDeviceToHost));
    CB_CUDA(cudaMemcpy(ent.data(), t.entries + (size_t)seq * t.LC * t.E, (size_t)n * t.E * 4, cudaMemcpyDeviceToHost));
    std::vector<uint32_t> order(n);
    for (uint32_t i = 0; i < n; i++) order[i] = i;
    std::sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) { return st[a] < st[b]; });
    const int LL = t.LL, FL = t.FL, FC = t.FC;
    for (uint32_t r = 0; r < n; r++) {
        const uint32_t* e = ent.data() + (size_t)order[r] * t.E;
        if (leaders) for (int j = 0; j < LL; j++) leaders[(size_t)r * LL + j] = (int32_t)e[j];
        int fo[CB_MAX_FC], nf = 0;
        for (int f = 0; f < FC; f++) if (e[LL + f] != 0) fo[nf++] = f;
        std::sort(fo, fo + nf, [&](int a, int b) { return e[LL + a] < e[LL + b]; });
        if (n_followers) n_followers[r] = nf;
        if (followers) {
            int32_t* dst = followers + (size_t)r * FC * FL;
            for (int k = 0; k < FC * FL; k++) dst[k] = -1;
            for (int k = 0; k < nf; k++)
                for (int j = 0; j < FL; j++) dst[k * FL + j] = (int32_t)e[LL + FC + fo[k] * FL + j];
        }
    }
    return CB_OK;
}

extern "C" cb_status cb_table_load(cb_ctx* ctx, int32_t seq, int32_t n_leaders, const int32_t* leaders,
                                   const int32_t* n_followers, const int32_t* followers) {
    CB_CHECK_ARG(ctx && seq >= 0 && seq < ctx->cfg.batch && n_leaders >= 0 && n_leaders <= ctx->cfg.LC);
    CB_CHECK_ARG(n_leaders == 0 || (leaders && n_followers && followers));
    const CbTables& t = ctx->tables;
    const int LL = t.LL, FL = t.FL, FC = t.FC;
    std::vector<uint32_t> idx(t.nslots, 0u), st(std::max(n_leaders, 1)), ent((size_t)std::max(n_leaders, 1) * t.E, 0u);
    uint32_t clock = 0;
    for (int r = 0; r < n_leaders; r++) {
        uint32_t* e = ent.data() + (size_t)r * t.E;
        int32_t k[4] = {0, 0, 0, 0};
        for (int j = 0; j < LL; j++) { k[j] = leaders[(size_t)r * LL + j]; e[j] = (uint32_t)k[j]; }
        const int nf = n_followers[r];
        if (nf < 1 || nf > FC) return CB_ERR_INVALID_ARG;
        for (int f = 0; f < nf; f++) {
            e[LL + f] = ++clock;
            for (int j = 0; j < FL; j++) e[LL + FC + f * FL + j] = (uint32_t)followers[((size_t)r * FC + f) * FL + j];
        }
        st[r] = ++clock;
        const uint64_t h = cb_hash4(k[0], k[1], k[2], k[3], LL);
        uint32_t bucket = cb_hash_bucket(h, t.nslots);
        const uint32_t word = (cb_hash_tag(h) << CB_EID_BITS) | (uint32_t)r;
        bool placed = false;
        for (uint32_t p = 0; p < (t.nslots >> 5) && !placed; p++) {
            for (uint32_t l = 0; l < 32 && !placed; l++)
                if (idx[bucket * 32 + l] == 0) { idx[bucket * 32 + l] = word; placed = true; }
            bucket = (bucket + 1) & ((t.nslots >> 5) - 1);
        }
        if (!placed) return CB_ERR_PROBE_LIMIT;
    }
    uint32_t hdr[4] = {clock, (uint32_t)n_leaders, 0, 0};
    CB_CUDA(cudaDeviceSynchronize());
    CB_CUDA(cudaMemcpy(t.hdr + (size_t)seq * 4, hdr, sizeof(hdr), cudaMemcpyHostToDevice));
    CB_CUDA(cudaMemcpy(t.index + (size_t)seq * t.nslots, idx.data(), (size_t)t.nslots * 4, cudaMemcpyHostToDevice));
    if (n_leaders > 0) {
        CB_CUDA(cudaMemcpy(t.lstamp + (size_t)seq * t.LC, st.data(), (size_t)n_leaders * 4, cudaMemcpyHostToDevice));
        CB_CUDA(cudaMemcpy(t.entries + (size_t)seq * t.LC * t.E, ent.data(), (size_t)n_leaders * t.E * 4,
                           cudaMemcpyHostToDevice));
    }
    CB_CUDA(cudaDeviceSynchronize());
    return CB_OK;
}

extern "C" cb_status cb_poll_status(cb_ctx* ctx, cb_status* device_status, uint64_t* counters) {
    CB_CHECK_ARG(ctx);
    CB_CUDA(cudaDeviceSynchronize());
    uint32_t st[4];
    CB_CUDA(cudaMemcpy(st, ctx->d_status, sizeof(st), cudaMemcpyDeviceToHost));
    // checking build: the guard areas behind the workspace regions must still hold their fill
    for (int g = 0; g < ctx->n_guards && st[0] == 0; ++g) {
        unsigned char guard[CB_GUARD_BYTES];
        CB_CUDA(cudaMemcpy(guard, ctx->ws + ctx->guard_off[g], CB_GUARD_BYTES, cudaMemcpyDeviceToHost));
        for (int k = 0; k < CB_GUARD_BYTES; ++k)
            if (guard[k] != CB_GUARD_BYTE) { st[0] = (uint32_t)CB_ERR_CANARY; break; }
    }
    if (device_status) *device_status = (cb_status)st[0];
    if (st[0] != 0) CB_CUDA(cudaMemset(ctx->d_status, 0, sizeof(st)));
    if (counters) CB_CUDA(cudaMemcpy(counters, ctx->d_counters, CB_NUM_COUNTERS * 8, cudaMemcpyDeviceToHost));
    return CB_OK;
}

extern "C" const char* cb_status_str(cb_status s) {
    switch (s) {
        case CB_OK: return "ok";
        case CB_ERR_INVALID_ARG: return "invalid argument";
        case CB_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case CB_ERR_CUDA: return "CUDA error";
        case CB_ERR_PROBE_LIMIT: return "hash probe limit reached";
        case CB_ERR_TIMEOUT: return "bounded device wait ran out";
        case CB_ERR_UNSUPPORTED: return "unsupported device or shape";
        case CB_ERR_STATIC_LIMIT: return "problem larger than the built-in static scratch (see cb_accept_static)";
        case CB_ERR_KV_FULL: return "a sequence's pages cannot hold the committed tokens";
        case CB_ERR_CANARY: return "a guard area beside a workspace region was overwritten (checking build)";
    }
    return "unknown status";
}
