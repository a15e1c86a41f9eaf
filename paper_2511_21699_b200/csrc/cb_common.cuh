// Shared declarations of the library: context object, workspace layout, table view, hashing.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "cacheback.h"

#define CB_FULL 0xFFFFFFFFu
#define CB_IDX_EMPTY 0u
#define CB_IDX_TOMB 0xFFFFFFFFu
#define CB_EID_BITS 20
#define CB_EID_MASK ((1u << CB_EID_BITS) - 1u)
#define CB_MAX_T 128
#define CB_MAX_LL 4
#define CB_MAX_FL 8
#define CB_MAX_FC 128

// Per-sequence table in the workspace (all 32-bit words):
//   hdr[4]            clock, leader count, unused, unused
//   index[nslots]     open-addressing index over 32-slot buckets: 0 = empty, 0xFFFFFFFF = deleted,
//                     else (tag << 20) | entry id, tag in [1, 4094] taken from the key's hash
//   lstamp[LC]        leader recency stamps (dense, so the LRU scan reads 4 bytes per leader)
//   entries[LC][E]    key[LL], follower stamps[FC] (0 = free), follower tokens[FC][FL]; E padded to 4 words
// Checking build (-DCB_DEBUG): indices taken from memory are range-checked before use.  cb_dbg_in returns whether
// 0 <= i < n; if not it records CB_ERR_INVALID_ARG in the device status and the caller skips the access.  In the regular
// build it is a constant true and costs nothing.
#ifdef CB_DEBUG
#define CB_DEBUG_BUILD 1
__device__ __forceinline__ bool cb_dbg_in(long long i, long long n, uint32_t* status) {
    if (i >= 0 && i < n) return true;
    if (status) atomicCAS(status, 0u, (uint32_t)CB_ERR_INVALID_ARG);
    return false;
}
#else
#define CB_DEBUG_BUILD 0
__device__ __forceinline__ bool cb_dbg_in(long long, long long, uint32_t*) { return true; }
#endif
#define CB_GUARD_BYTES 256      // guard area behind every workspace region of the checking build
#define CB_GUARD_BYTE 0xC5
#define CB_MAX_GUARDS 12

struct CbTables {
    uint32_t* dbg_status;   // device status word for the checking build's range checks (may be null)
    uint32_t* hdr;
    uint32_t* index;
    uint32_t* lstamp;
    uint32_t* entries;
    uint32_t nslots, E;
    int32_t LL, FL, LC, FC;
    uint32_t refresh;  // re-inserting a stored follower refreshes it
};

struct CbSeq {  // one sequence's slice of CbTables
    uint32_t* hdr;
    uint32_t* index;
    uint32_t* lstamp;
    uint32_t* entries;
};

__device__ __forceinline__ CbSeq cb_seq(const CbTables& t, int b) {
    CbSeq s;
    s.hdr = t.hdr + (size_t)b * 4;
    s.index = t.index + (size_t)b * t.nslots;
    s.lstamp = t.lstamp + (size_t)b * t.LC;
    s.entries = t.entries + (size_t)b * t.LC * t.E;
    return s;
}

__host__ __device__ __forceinline__ uint64_t cb_hash4(int32_t k0, int32_t k1, int32_t k2, int32_t k3, int LL) {
    uint64_t h = 0x9E3779B97F4A7C15ull ^ (uint64_t)LL;
    h = (h ^ (uint32_t)k0) * 0xFF51AFD7ED558CCDull; h ^= h >> 32;
    if (LL > 1) { h = (h ^ (uint32_t)k1) * 0xFF51AFD7ED558CCDull; h ^= h >> 32; }
    if (LL > 2) { h = (h ^ (uint32_t)k2) * 0xFF51AFD7ED558CCDull; h ^= h >> 32; }
    if (LL > 3) { h = (h ^ (uint32_t)k3) * 0xFF51AFD7ED558CCDull; h ^= h >> 32; }
    h ^= h >> 33; h *= 0xC4CEB9FE1A85EC53ull; h ^= h >> 33;
    return h;
}
__host__ __device__ __forceinline__ uint32_t cb_hash_tag(uint64_t h) { return (uint32_t)(h & 0xFFFFFFFFull) % 4094u + 1u; }
__host__ __device__ __forceinline__ uint32_t cb_hash_bucket(uint64_t h, uint32_t nslots) {
    return (uint32_t)(h >> 32) & ((nslots >> 5) - 1u);
}

struct cb_ctx {
    cb_config cfg;
    int device;
    char* ws;
    size_t ws_bytes;
    CbTables tables;
    CbTables frozen;        // the read-only table of cb_frozen_attach (one "sequence", shared by the batch)
    bool has_frozen;
    uint32_t* d_status;     // [4]
    unsigned long long* d_counters;  // [CB_NUM_COUNTERS]
    unsigned long long* d_rowmax;    // [batch * max_nodes] packed (value, index) maxima, zero between calls
    uint32_t* d_ticket;     // [batch] CTAs-finished counters, zero between calls
    uint32_t* d_bulk_plan;  // [batch][4] per-sequence plan of cb_update_bulk
    void* bulk_scratch;     // caller's scratch for the order-free path of cb_update_bulk (cb_bulk_scratch_attach), or null
    uint32_t bulk_slots;    // hash slots that fit it (a power of two)
    size_t guard_off[CB_MAX_GUARDS];
    int n_guards;
    float* d_attn_part;     // partial outputs of units shared between CTAs
    size_t attn_part_floats;
    int attn_max_units;     // partial row tiles available
    int num_sms;
};

struct CbLayout {
    uint32_t nslots, E;
    size_t off_hdr, off_index, off_lstamp, off_entries, off_status, off_counters, off_rowmax, off_ticket, off_bulk_plan,
        off_attn_part, attn_part_floats, total;
    int attn_max_units;
    size_t guard_off[CB_MAX_GUARDS];   // checking build: start of the guard area behind each region
    int n_guards;
};

cb_status cb_compute_layout(const cb_config* cfg, CbLayout* L);

// Device image of a frozen table: the single-sequence form of the layout above, in a buffer of its own.  lstamp holds each
// leader's corpus count; a follower's stamp is FC - its rank by count, so the larger stamp is the more frequent follower.
struct CbFrozenLayout {
    uint32_t nslots, E;
    size_t off_hdr, off_index, off_lstamp, off_entries, total;
};
cb_status cb_frozen_layout(const cb_frozen_config* cfg, CbFrozenLayout* L);
CbTables cb_frozen_view(const cb_frozen_config* cfg, const CbFrozenLayout& L, void* dev_table);
void cb_count_launch(int n);

#define CB_ATTN_MAX_UNITS 640   // partial row tiles (128 rows x (D + 4) floats): 2 shared units x 2 row tiles per persistent CTA, 160 CTAs

// Programmatic dependent launch.  Every kernel of the step begins with CB_PDL_ENTRY: it waits until the kernels before
// it in the stream have finished (so nothing they wrote or still read is touched early) and then lets the next kernel's
// blocks be scheduled as SMs become free, which hides launch latency between the microsecond-scale kernels of a step.
#define CB_PDL_ENTRY()                                               \
    do {                                                             \
        asm volatile("griddepcontrol.wait;" ::: "memory");           \
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); \
    } while (0)
#ifdef __CUDACC__
#include <utility>
template <typename... KArgs, typename... Args>
inline cudaError_t cb_launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
#endif

#define CB_CHECK_ARG(cond) do { if (!(cond)) return CB_ERR_INVALID_ARG; } while (0)
#include <stdio.h>
// CUDA failures are exceptional: say where and what on stderr, then report CB_ERR_CUDA.
#define CB_CUDA(call) do { cudaError_t cb_e_ = (call); if (cb_e_ != cudaSuccess) { \
    fprintf(stderr, "cacheback: %s:%d: %s\n", __FILE__, __LINE__, cudaGetErrorString(cb_e_)); return CB_ERR_CUDA; } } while (0)
