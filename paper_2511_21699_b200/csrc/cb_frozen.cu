// Frozen table (Section 3.3): device image, host load / dump, attachment to a context.
#include <algorithm>
#include <vector>

#include "cb_common.cuh"

static size_t fz_align(size_t x, size_t a) { return (x + a - 1) / a * a; }

cb_status cb_frozen_layout(const cb_frozen_config* c, CbFrozenLayout* L) {
    if (!c || !L) return CB_ERR_INVALID_ARG;
    if (c->LL < 1 || c->LL > CB_MAX_LL || c->FL < 1 || c->FL > CB_MAX_FL) return CB_ERR_INVALID_ARG;
    if (c->LC < 1 || c->LC > (1 << CB_EID_BITS) || c->FC < 1 || c->FC > CB_MAX_FC) return CB_ERR_INVALID_ARG;
    uint32_t ns = 32;
    while (ns < 4u * (uint32_t)c->LC) ns <<= 1;
    L->nslots = ns;
    L->E = (uint32_t)fz_align((size_t)c->LL + (size_t)c->FC * (1 + c->FL), 4);
    size_t o = 0;
    L->off_hdr = o;     o = fz_align(o + 4 * 4, 256);
    L->off_index = o;   o = fz_align(o + (size_t)ns * 4, 256);
    L->off_lstamp = o;  o = fz_align(o + (size_t)c->LC * 4, 256);
    L->off_entries = o; o = fz_align(o + (size_t)c->LC * L->E * 4, 256);
    L->total = o;
    return CB_OK;
}

CbTables cb_frozen_view(const cb_frozen_config* c, const CbFrozenLayout& L, void* dev_table) {
    CbTables t;
    char* base = (char*)dev_table;
    t.hdr = (uint32_t*)(base + L.off_hdr);
    t.index = (uint32_t*)(base + L.off_index);
    t.lstamp = (uint32_t*)(base + L.off_lstamp);
    t.entries = (uint32_t*)(base + L.off_entries);
    t.nslots = L.nslots; t.E = L.E;
    t.LL = c->LL; t.FL = c->FL; t.LC = c->LC; t.FC = c->FC;
    t.refresh = 0u;
    t.dbg_status = nullptr;
    return t;
}

extern "C" cb_status cb_frozen_bytes(const cb_frozen_config* cfg, size_t* bytes) {
    CbFrozenLayout L;
    if (!bytes) return CB_ERR_INVALID_ARG;
    cb_status s = cb_frozen_layout(cfg, &L);
    if (s != CB_OK) return s;
    *bytes = L.total;
    return CB_OK;
}

static cb_status fz_check(const cb_frozen_config* cfg, const void* dev_table, size_t bytes, CbFrozenLayout* L) {
    cb_status s = cb_frozen_layout(cfg, L);
    if (s != CB_OK) return s;
    if (!dev_table || ((uintptr_t)dev_table & 255) != 0) return CB_ERR_INVALID_ARG;
    if (bytes < L->total) return CB_ERR_WORKSPACE_TOO_SMALL;
    return CB_OK;
}

extern "C" cb_status cb_frozen_load(const cb_frozen_config* cfg, void* dev_table, size_t bytes, int32_t n_leaders,
                                    const int32_t* leaders, const int32_t* n_followers, const int32_t* followers) {
    CbFrozenLayout L;
    cb_status s = fz_check(cfg, dev_table, bytes, &L);
    if (s != CB_OK) return s;
    CB_CHECK_ARG(n_leaders >= 0 && n_leaders <= cfg->LC);
    CB_CHECK_ARG(n_leaders == 0 || (leaders && n_followers && followers));
    const int LL = cfg->LL, FL = cfg->FL, FC = cfg->FC;
    const uint32_t nb = L.nslots >> 5;
    std::vector<uint32_t> idx(L.nslots, 0u), cnt(std::max(n_leaders, 1), 0u), ent((size_t)std::max(n_leaders, 1) * L.E, 0u);
    for (int r = 0; r < n_leaders; r++) {
        uint32_t* e = ent.data() + (size_t)r * L.E;
        int32_t k[4] = {0, 0, 0, 0};
        for (int j = 0; j < LL; j++) {
            k[j] = leaders[(size_t)r * LL + j];
            if (k[j] < 0) return CB_ERR_INVALID_ARG;
            e[j] = (uint32_t)k[j];
        }
        const int nf = n_followers[r];
        if (nf < 1 || nf > FC) return CB_ERR_INVALID_ARG;
        for (int f = 0; f < nf; f++) {
            e[LL + f] = (uint32_t)(FC - f);                        // larger stamp = more frequent
            for (int j = 0; j < FL; j++) e[LL + FC + f * FL + j] = (uint32_t)followers[((size_t)r * FC + f) * FL + j];
        }
        cnt[r] = (uint32_t)(n_leaders - r);                        // keeps the given order in cb_frozen_dump
        const uint64_t h = cb_hash4(k[0], k[1], k[2], k[3], LL);
        uint32_t bucket = cb_hash_bucket(h, L.nslots);
        const uint32_t word = (cb_hash_tag(h) << CB_EID_BITS) | (uint32_t)r;
        bool placed = false;
        for (uint32_t p = 0; p < nb && !placed; p++) {
            for (uint32_t l = 0; l < 32 && !placed; l++)
                if (idx[bucket * 32 + l] == 0) { idx[bucket * 32 + l] = word; placed = true; }
            bucket = (bucket + 1) & (nb - 1);
        }
        if (!placed) return CB_ERR_PROBE_LIMIT;
    }
    char* base = (char*)dev_table;
    const uint32_t hdr[4] = {0u, (uint32_t)n_leaders, 0u, 0u};
    CB_CUDA(cudaDeviceSynchronize());
    CB_CUDA(cudaMemcpy(base + L.off_hdr, hdr, sizeof(hdr), cudaMemcpyHostToDevice));
    CB_CUDA(cudaMemcpy(base + L.off_index, idx.data(), (size_t)L.nslots * 4, cudaMemcpyHostToDevice));
    if (n_leaders > 0) {
        CB_CUDA(cudaMemcpy(base + L.off_lstamp, cnt.data(), (size_t)n_leaders * 4, cudaMemcpyHostToDevice));
        CB_CUDA(cudaMemcpy(base + L.off_entries, ent.data(), (size_t)n_leaders * L.E * 4, cudaMemcpyHostToDevice));
    }
    CB_CUDA(cudaDeviceSynchronize());
    return CB_OK;
}

extern "C" cb_status cb_frozen_dump(const cb_frozen_config* cfg, const void* dev_table, size_t bytes, int32_t* n_leaders,
                                    int32_t* leaders, int32_t* n_followers, int32_t* followers) {
    CbFrozenLayout L;
    cb_status s = fz_check(cfg, dev_table, bytes, &L);
    if (s != CB_OK) return s;
    CB_CHECK_ARG(n_leaders);
    const char* base = (const char*)dev_table;
    const int LL = cfg->LL, FL = cfg->FL, FC = cfg->FC;
    uint32_t hdr[4];
    CB_CUDA(cudaDeviceSynchronize());
    CB_CUDA(cudaMemcpy(hdr, base + L.off_hdr, sizeof(hdr), cudaMemcpyDeviceToHost));
    const uint32_t n = hdr[1];
    if (n > (uint32_t)cfg->LC) return CB_ERR_INVALID_ARG;        // not a table of this shape
    *n_leaders = (int32_t)n;
    if (n == 0) return CB_OK;
    std::vector<uint32_t> cnt(n), ent((size_t)n * L.E);
    CB_CUDA(cudaMemcpy(cnt.data(), base + L.off_lstamp, (size_t)n * 4, cudaMemcpyDeviceToHost));
    CB_CUDA(cudaMemcpy(ent.data(), base + L.off_entries, (size_t)n * L.E * 4, cudaMemcpyDeviceToHost));
    std::vector<uint32_t> order(n);
    for (uint32_t i = 0; i < n; i++) order[i] = i;
    std::sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) {
        if (cnt[a] != cnt[b]) return cnt[a] > cnt[b];
        const uint32_t* ea = ent.data() + (size_t)a * L.E;
        const uint32_t* eb = ent.data() + (size_t)b * L.E;
        return std::lexicographical_compare(ea, ea + LL, eb, eb + LL);
    });
    for (uint32_t r = 0; r < n; r++) {
        const uint32_t* e = ent.data() + (size_t)order[r] * L.E;
        if (leaders) for (int j = 0; j < LL; j++) leaders[(size_t)r * LL + j] = (int32_t)e[j];
        int fo[CB_MAX_FC], nf = 0;
        for (int f = 0; f < FC; f++) if (e[LL + f] != 0) fo[nf++] = f;
        std::sort(fo, fo + nf, [&](int a, int b) { return e[LL + a] > e[LL + b]; });
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

extern "C" cb_status cb_frozen_attach(cb_ctx* ctx, const cb_frozen_config* cfg, const void* dev_table, size_t bytes) {
    CB_CHECK_ARG(ctx);
    if (!dev_table) {
        ctx->has_frozen = false;
        return CB_OK;
    }
    CbFrozenLayout L;
    cb_status s = fz_check(cfg, dev_table, bytes, &L);
    if (s != CB_OK) return s;
    CB_CHECK_ARG(cfg->LL == ctx->cfg.LL && cfg->FL == ctx->cfg.FL);
    ctx->frozen = cb_frozen_view(cfg, L, const_cast<void*>(dev_table));
    ctx->has_frozen = true;
    return CB_OK;
}
