"""Loads libcacheback.so and declares the C-ABI prototypes (ctypes). Fails loudly if the library is
missing: there is no fallback path."""
import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
# CACHEBACK_LIBRARY names another build of the library to load, e.g. the checking build libcacheback_debug.so.
SO_PATH = os.environ.get("CACHEBACK_LIBRARY") or os.path.join(HERE, "libcacheback.so")
SO_DEBUG_PATH = os.path.join(HERE, "libcacheback_debug.so")

CB_OK = 0
CB_DTYPE_F32, CB_DTYPE_BF16 = 0, 1
CB_FLAG_NO_FOLLOWER_REFRESH, CB_FLAG_ATTN_CUDA_CORES, CB_FLAG_ATTN_CTA_PAIRS = 1, 2, 4
CB_ERR_STATIC_LIMIT = 7
CB_ERR_KV_FULL = 8
CB_ERR_INVALID_ARG, CB_ERR_CANARY = 1, 9
CB_GUARD_BYTES = 256
CB_STATIC_MAX_BATCH, CB_STATIC_MAX_ROWS = 1024, 8192
CB_NUM_COUNTERS = 8
COUNTER_NAMES = ["inserts", "leader_evictions", "follower_evictions", "queries", "query_hits", "max_probe", "frozen_queries",
                 "frozen_hits"]

EXPORTS = ["cb_workspace_bytes", "cb_create", "cb_destroy", "cb_reset", "cb_update", "cb_draft_tree", "cb_update_draft_tree",
           "cb_tree_attn", "cb_accept", "cb_table_dump", "cb_table_load", "cb_poll_status", "cb_launch_count",
           "cb_status_str", "cb_accept_static", "cb_kv_commit", "cb_frozen_bytes", "cb_frozen_load", "cb_frozen_dump",
           "cb_frozen_attach", "cb_frozen_build_bytes", "cb_frozen_build", "cb_tree_add_branches", "cb_update_bulk", "cb_debug_build",
           "cb_bulk_scratch_bytes", "cb_bulk_scratch_attach", "cb_accept_update_draft_tree"]


class CbConfigC(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("batch", "LL", "FL", "LC", "FC", "max_nodes", "crt", "max_depth", "vocab",
                                          "n_q_heads", "n_kv_heads", "head_dim", "page_size")] + [("flags", C.c_uint32)]


class CbFrozenConfigC(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("LL", "FL", "LC", "FC")]


class CbKvCommitArgsC(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("k_pool", "v_pool", "block_table", "ctx_len", "k_tree", "v_tree", "n_accept",
                                          "accept_nodes")] + [("max_pages", C.c_int32), ("num_pages", C.c_int32)]


class CbAcceptDraftArgsC(C.Structure):
    _fields_ = [("logits", C.c_void_p), ("logits_dtype", C.c_int32), ("logits_row_stride", C.c_int64)] + \
               [(n, C.c_void_p) for n in ("tree_tokens", "tree_parent", "tree_depth", "n_nodes", "n_accept", "accept_nodes", "out_tokens",
                                          "target_ids_out", "tokens")] + [("row_stride", C.c_int64)] + \
               [(n, C.c_void_p) for n in ("seq_len", "next_tokens", "next_parent", "next_depth", "next_mask", "next_n_nodes")]


class CbAttnArgsC(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("q", "k_pool", "v_pool", "block_table", "ctx_len", "k_tree", "v_tree",
                                          "tree_mask", "n_nodes", "out", "lse")] + \
               [("max_pages", C.c_int32), ("num_pages", C.c_int32), ("max_ctx", C.c_int32), ("scale", C.c_float)]


_lib = None


def load():
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(SO_PATH):
        raise RuntimeError("libcacheback.so is not built (%s). Run `python -m paper_2511_21699_b200.build` "
                           "or __graft_entry__.build(); there is no fallback path." % SO_PATH)
    L = C.CDLL(SO_PATH)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    L.cb_workspace_bytes.argtypes = [C.POINTER(CbConfigC), C.POINTER(C.c_size_t)]
    L.cb_create.argtypes = [C.POINTER(CbConfigC), vp, C.c_size_t, C.POINTER(vp)]
    L.cb_destroy.argtypes = [vp]
    L.cb_destroy.restype = None
    L.cb_reset.argtypes = [vp, vp, vp]
    L.cb_update.argtypes = [vp, vp, i64, vp, vp, vp]
    L.cb_update_bulk.argtypes = [vp, vp, i64, vp, vp, vp]
    L.cb_bulk_scratch_bytes.argtypes = [C.POINTER(CbConfigC), i64, C.POINTER(C.c_size_t)]
    L.cb_bulk_scratch_attach.argtypes = [vp, vp, C.c_size_t]
    L.cb_draft_tree.argtypes = [vp, vp, i64, vp, vp, vp, vp, vp, vp, vp]
    L.cb_update_draft_tree.argtypes = [vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, vp]
    L.cb_tree_add_branches.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, vp]
    L.cb_tree_attn.argtypes = [vp, C.POINTER(CbAttnArgsC), vp]
    L.cb_accept_update_draft_tree.argtypes = [vp, C.POINTER(CbAcceptDraftArgsC), vp]
    L.cb_kv_commit.argtypes = [vp, C.POINTER(CbKvCommitArgsC), vp]
    L.cb_accept.argtypes = [vp, vp, vp, vp, vp, vp, i32, i64, vp, vp, vp, vp, vp, vp]
    L.cb_accept_static.argtypes = [i32, i32, i32, i32, vp, vp, vp, vp, vp, i32, i64, vp, vp, vp, vp, vp]
    L.cb_table_dump.argtypes = [vp, i32, C.POINTER(i32), vp, vp, vp]
    L.cb_table_load.argtypes = [vp, i32, i32, vp, vp, vp]
    L.cb_poll_status.argtypes = [vp, C.POINTER(i32), vp]
    L.cb_frozen_bytes.argtypes = [C.POINTER(CbFrozenConfigC), C.POINTER(C.c_size_t)]
    L.cb_frozen_load.argtypes = [C.POINTER(CbFrozenConfigC), vp, C.c_size_t, i32, vp, vp, vp]
    L.cb_frozen_dump.argtypes = [C.POINTER(CbFrozenConfigC), vp, C.c_size_t, C.POINTER(i32), vp, vp, vp]
    L.cb_frozen_attach.argtypes = [vp, C.POINTER(CbFrozenConfigC), vp, C.c_size_t]
    L.cb_frozen_build_bytes.argtypes = [C.POINTER(CbFrozenConfigC), i64, C.POINTER(C.c_size_t)]
    L.cb_frozen_build.argtypes = [C.POINTER(CbFrozenConfigC), vp, i64, vp, C.c_size_t, vp, C.c_size_t, vp]
    L.cb_launch_count.restype = C.c_uint64
    L.cb_launch_count.argtypes = []
    L.cb_status_str.restype = C.c_char_p
    L.cb_status_str.argtypes = [i32]
    L.cb_debug_build.argtypes = []
    for name in EXPORTS:
        if name not in ("cb_destroy", "cb_launch_count", "cb_status_str"):
            getattr(L, name).restype = i32
    _lib = L
    return L
