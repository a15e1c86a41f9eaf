"""Thin Python binding of the C-ABI library: argument marshalling only.

Tensors are torch CUDA tensors (device memory and streams are torch's); every step of the path runs in
the library's kernels.  Method names mirror the C entry points.
"""
import ctypes as C

import numpy as np
import torch

from . import _lib
from ._lib import CbConfigC, CbAttnArgsC, CbKvCommitArgsC, CbFrozenConfigC


class CachebackError(RuntimeError):
    pass


def _check(code, what):
    if code != _lib.CB_OK:
        raise CachebackError("%s failed: %s" % (what, _lib.load().cb_status_str(code).decode()))


def _ptr(t, dtype=None):
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous()):
        raise CachebackError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise CachebackError("expected dtype %s, got %s" % (dtype, t.dtype))
    return t.data_ptr()


def _stream(stream):
    return (stream if stream is not None else torch.cuda.current_stream()).cuda_stream


def cb_accept_static(tree, logits, max_depth, res=None, stream=None):
    """Greedy acceptance from logits without a context and without any device allocation by the library:
    for callers that only have the buffers they were given (a plugin inside someone else's memory pool, a
    fixed memory budget).  The library's built-in scratch array is used instead of a workspace, so batch is
    limited to 1,024 and batch * max_nodes to 8,192; larger shapes raise CachebackError.  Calls on one device
    share that array: do not let two of them overlap on the GPU.  Make the first call on a device outside
    any stream capture.  `res` holds the caller-allocated outputs (n_accept [B], accept_nodes [B, max_depth],
    out_tokens [B, max_depth + 1], target_ids [B, T]); it is created with torch when omitted."""
    lib = _lib.load()
    B, T, V = logits.shape
    if logits.dtype == torch.float32:
        dtype = _lib.CB_DTYPE_F32
    elif logits.dtype == torch.bfloat16:
        dtype = _lib.CB_DTYPE_BF16
    else:
        raise CachebackError("logits must be float32 or bfloat16")
    if not (logits.is_cuda and logits.stride(2) == 1 and logits.stride(0) == T * logits.stride(1)):
        raise CachebackError("logits must be [batch, max_nodes, vocab] with a uniform row stride")
    if res is None:
        i32 = dict(dtype=torch.int32, device=logits.device)
        res = dict(n_accept=torch.empty(B, **i32), accept_nodes=torch.empty(B, max_depth, **i32),
                   out_tokens=torch.empty(B, max_depth + 1, **i32), target_ids=torch.empty(B, T, **i32))
    _check(lib.cb_accept_static(B, T, max_depth, V, _ptr(tree["tokens"], torch.int32), _ptr(tree["parent"], torch.int32),
                                _ptr(tree["depth"], torch.int32), _ptr(tree["n_nodes"], torch.int32), logits.data_ptr(), dtype,
                                logits.stride(1), _ptr(res["n_accept"], torch.int32), _ptr(res["accept_nodes"], torch.int32),
                                _ptr(res["out_tokens"], torch.int32), _ptr(res["target_ids"], torch.int32), _stream(stream)),
           "cb_accept_static")
    return res


class FrozenTable:
    """A frozen table (cb_frozen_*): one device buffer, owned by this object, that contexts attach read-only."""

    def __init__(self, LL, FL, LC, FC, device="cuda:0"):
        self.lib = _lib.load()
        if not torch.cuda.is_available():
            raise CachebackError("no CUDA device: the library has no CPU path")
        self.device = torch.device(device)
        self.cfg = CbFrozenConfigC(LL, FL, LC, FC)
        nbytes = C.c_size_t(0)
        _check(self.lib.cb_frozen_bytes(C.byref(self.cfg), C.byref(nbytes)), "cb_frozen_bytes")
        self.bytes = nbytes.value
        with torch.cuda.device(self.device):
            self.buffer = torch.zeros(nbytes.value + 256, dtype=torch.uint8, device=self.device)
        self.ptr = (self.buffer.data_ptr() + 255) // 256 * 256

    def cb_frozen_load(self, leaders, n_followers, followers):
        """Host arrays: leaders [n, LL], n_followers [n], followers [n, FC, FL], most frequent first."""
        c = self.cfg
        leaders = np.ascontiguousarray(leaders, dtype=np.int32).reshape(-1, c.LL)
        n = leaders.shape[0]
        nfol = np.ascontiguousarray(n_followers, dtype=np.int32).reshape(n)
        fol = np.full((max(n, 1), c.FC, c.FL), -1, dtype=np.int32)
        src = np.asarray(followers, dtype=np.int32).reshape(n, -1, c.FL)
        fol[:n, : src.shape[1]] = src[:, : c.FC]
        with torch.cuda.device(self.device):
            _check(self.lib.cb_frozen_load(C.byref(self.cfg), self.ptr, self.bytes, n, leaders.ctypes.data, nfol.ctypes.data,
                                           fol.ctypes.data), "cb_frozen_load")

    def cb_frozen_build(self, corpus, stream=None):
        """corpus: int32 CUDA tensor [n_tokens].  Counts on the GPU and overwrites this table; the scratch is a temporary
        torch tensor."""
        n = int(corpus.numel())
        nbytes = C.c_size_t(0)
        _check(self.lib.cb_frozen_build_bytes(C.byref(self.cfg), n, C.byref(nbytes)), "cb_frozen_build_bytes")
        with torch.cuda.device(self.device):
            scratch = torch.empty(nbytes.value + 256, dtype=torch.uint8, device=self.device)
            sp = (scratch.data_ptr() + 255) // 256 * 256
            _check(self.lib.cb_frozen_build(C.byref(self.cfg), _ptr(corpus, torch.int32), n, self.ptr, self.bytes, sp, nbytes.value,
                                            _stream(stream)), "cb_frozen_build")
        del scratch

    def cb_frozen_dump(self):
        """(leaders [n, LL], n_followers [n], followers [n, FC, FL]) as host arrays, most frequent first."""
        c = self.cfg
        n = C.c_int32(0)
        leaders = np.empty((c.LC, c.LL), dtype=np.int32)
        nfol = np.empty(c.LC, dtype=np.int32)
        fol = np.empty((c.LC, c.FC, c.FL), dtype=np.int32)
        with torch.cuda.device(self.device):
            _check(self.lib.cb_frozen_dump(C.byref(self.cfg), self.ptr, self.bytes, C.byref(n), leaders.ctypes.data,
                                           nfol.ctypes.data, fol.ctypes.data), "cb_frozen_dump")
        return leaders[: n.value], nfol[: n.value], fol[: n.value]


class Cacheback:
    """One context: per-sequence tables plus scratch, in a workspace tensor owned by this object."""

    def __init__(self, batch, LL, FL, LC, FC, max_nodes, crt, max_depth, vocab, n_q_heads, n_kv_heads, head_dim,
                 page_size=16, flags=0, device="cuda:0"):
        self.lib = _lib.load()
        if not torch.cuda.is_available():
            raise CachebackError("no CUDA device: the library has no CPU path")
        self.device = torch.device(device)
        self.cfg = CbConfigC(batch, LL, FL, LC, FC, max_nodes, crt, max_depth, vocab, n_q_heads, n_kv_heads, head_dim,
                             page_size, flags)
        nbytes = C.c_size_t(0)
        _check(self.lib.cb_workspace_bytes(C.byref(self.cfg), C.byref(nbytes)), "cb_workspace_bytes")
        self.workspace_bytes = nbytes.value
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes.value + 256, dtype=torch.uint8, device=self.device)
            base = (self.workspace.data_ptr() + 255) // 256 * 256
            h = C.c_void_p(None)
            _check(self.lib.cb_create(C.byref(self.cfg), base, nbytes.value, C.byref(h)), "cb_create")
        self._h = h
        self.W = (max_nodes + 31) // 32

    @classmethod
    def from_config(cls, cfg, flags=0, device="cuda:0", batch=None):
        """cfg: a workloads.CbConfig-like object."""
        return cls(batch or cfg.batch, cfg.LL, cfg.FL, cfg.LC, cfg.FC, cfg.max_nodes, cfg.crt, cfg.max_depth, cfg.vocab,
                   cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.page_size, flags, device)

    def close(self):
        if getattr(self, "_h", None):
            self.lib.cb_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the four step calls -----------------------------------------------------------------------
    def cb_reset(self, seq_mask=None, stream=None):
        _check(self.lib.cb_reset(self._h, _ptr(seq_mask, torch.int32), _stream(stream)), "cb_reset")

    def cb_update(self, tokens, n_old, n_new, stream=None):
        _check(self.lib.cb_update(self._h, _ptr(tokens, torch.int32), tokens.stride(0), _ptr(n_old, torch.int32),
                                  _ptr(n_new, torch.int32), _stream(stream)), "cb_update")

    def cb_update_bulk(self, tokens, n_old, n_new, stream=None):
        _check(self.lib.cb_update_bulk(self._h, _ptr(tokens, torch.int32), tokens.stride(0), _ptr(n_old, torch.int32),
                                       _ptr(n_new, torch.int32), _stream(stream)), "cb_update_bulk")

    def cb_bulk_scratch_attach(self, max_windows):
        """Allocates and attaches scratch for the order-free path of cb_update_bulk (runs of up to max_windows windows in
        total per call); 0 or None detaches.  The buffer is kept alive by this object."""
        if not max_windows:
            _check(self.lib.cb_bulk_scratch_attach(self._h, None, 0), "cb_bulk_scratch_attach")
            self._bulk_scratch = None
            return 0
        nbytes = C.c_size_t(0)
        _check(self.lib.cb_bulk_scratch_bytes(C.byref(self.cfg), C.c_int64(int(max_windows)), C.byref(nbytes)), "cb_bulk_scratch_bytes")
        with torch.cuda.device(self.device):
            buf = torch.empty(nbytes.value + 256, dtype=torch.uint8, device=self.device)
        ptr = (buf.data_ptr() + 255) // 256 * 256
        _check(self.lib.cb_bulk_scratch_attach(self._h, C.c_void_p(ptr), C.c_size_t(nbytes.value)), "cb_bulk_scratch_attach")
        self._bulk_scratch = buf
        return nbytes.value

    def alloc_tree(self):
        B, T = self.cfg.batch, self.cfg.max_nodes
        i32 = dict(dtype=torch.int32, device=self.device)
        return dict(tokens=torch.empty(B, T, **i32), parent=torch.empty(B, T, **i32), depth=torch.empty(B, T, **i32),
                    mask=torch.empty(B, T, self.W, **i32), n_nodes=torch.empty(B, **i32))

    def cb_draft_tree(self, tokens, seq_len, tree=None, stream=None):
        tree = tree if tree is not None else self.alloc_tree()
        _check(self.lib.cb_draft_tree(self._h, _ptr(tokens, torch.int32), tokens.stride(0), _ptr(seq_len, torch.int32),
                                      _ptr(tree["tokens"], torch.int32), _ptr(tree["parent"], torch.int32),
                                      _ptr(tree["depth"], torch.int32), _ptr(tree["mask"], torch.int32),
                                      _ptr(tree["n_nodes"], torch.int32), _stream(stream)), "cb_draft_tree")
        return tree

    def cb_update_draft_tree(self, tokens, n_old, n_new, tree=None, stream=None):
        """cb_update(tokens, n_old, n_new) and cb_draft_tree(tokens, n_new) in one launch."""
        tree = tree if tree is not None else self.alloc_tree()
        _check(self.lib.cb_update_draft_tree(self._h, _ptr(tokens, torch.int32), tokens.stride(0), _ptr(n_old, torch.int32),
                                             _ptr(n_new, torch.int32),
                                             _ptr(tree["tokens"], torch.int32), _ptr(tree["parent"], torch.int32),
                                             _ptr(tree["depth"], torch.int32), _ptr(tree["mask"], torch.int32),
                                             _ptr(tree["n_nodes"], torch.int32), _stream(stream)), "cb_update_draft_tree")
        return tree

    def cb_tree_add_branches(self, tree, branches, branch_len, stream=None):
        """branches int32 [batch, K, Lmax], branch_len int32 [batch, K]: extends `tree` in place."""
        K, Lmax = int(branches.shape[1]), int(branches.shape[2])
        _check(self.lib.cb_tree_add_branches(self._h, _ptr(branches, torch.int32), _ptr(branch_len, torch.int32), K, Lmax,
                                             _ptr(tree["tokens"], torch.int32), _ptr(tree["parent"], torch.int32),
                                             _ptr(tree["depth"], torch.int32), _ptr(tree["mask"], torch.int32),
                                             _ptr(tree["n_nodes"], torch.int32), _stream(stream)), "cb_tree_add_branches")
        return tree

    def cb_tree_attn(self, q, k_pool, v_pool, block_table, ctx_len, k_tree, v_tree, tree_mask, n_nodes, out=None,
                     lse=None, max_ctx=0, scale=0.0, stream=None):
        if out is None:
            out = torch.empty_like(q)
        a = CbAttnArgsC(_ptr(q, torch.bfloat16), _ptr(k_pool, torch.bfloat16), _ptr(v_pool, torch.bfloat16),
                        _ptr(block_table, torch.int32), _ptr(ctx_len, torch.int32), _ptr(k_tree, torch.bfloat16),
                        _ptr(v_tree, torch.bfloat16), _ptr(tree_mask, torch.int32), _ptr(n_nodes, torch.int32),
                        _ptr(out, torch.bfloat16), _ptr(lse, torch.float32), block_table.shape[1], k_pool.shape[0],
                        int(max_ctx), float(scale))
        _check(self.lib.cb_tree_attn(self._h, C.byref(a), _stream(stream)), "cb_tree_attn")
        return out

    def cb_kv_commit(self, k_pool, v_pool, block_table, ctx_len, k_tree, v_tree, n_accept, accept_nodes, stream=None):
        a = CbKvCommitArgsC(_ptr(k_pool, torch.bfloat16), _ptr(v_pool, torch.bfloat16), _ptr(block_table, torch.int32),
                            _ptr(ctx_len, torch.int32), _ptr(k_tree, torch.bfloat16), _ptr(v_tree, torch.bfloat16),
                            _ptr(n_accept, torch.int32), _ptr(accept_nodes, torch.int32), block_table.shape[1], k_pool.shape[0])
        _check(self.lib.cb_kv_commit(self._h, C.byref(a), _stream(stream)), "cb_kv_commit")

    def alloc_accept(self):
        B, Dm = self.cfg.batch, self.cfg.max_depth
        i32 = dict(dtype=torch.int32, device=self.device)
        return dict(n_accept=torch.empty(B, **i32), accept_nodes=torch.empty(B, Dm, **i32),
                    out_tokens=torch.empty(B, Dm + 1, **i32), target_ids=torch.empty(B, self.cfg.max_nodes, **i32))

    def cb_accept(self, tree, logits=None, target_ids=None, res=None, stream=None):
        res = res if res is not None else self.alloc_accept()
        dtype, stride, lp = 0, 0, None
        if logits is not None:
            if logits.dtype == torch.float32:
                dtype = _lib.CB_DTYPE_F32
            elif logits.dtype == torch.bfloat16:
                dtype = _lib.CB_DTYPE_BF16
            else:
                raise CachebackError("logits must be float32 or bfloat16")
            if not (logits.is_cuda and logits.dim() == 3 and logits.stride(2) == 1 and
                    logits.stride(0) == logits.shape[1] * logits.stride(1)):
                raise CachebackError("logits must be [batch, max_nodes, vocab] with a uniform row stride")
            stride, lp = logits.stride(1), logits.data_ptr()
        _check(self.lib.cb_accept(self._h, _ptr(tree["tokens"], torch.int32), _ptr(tree["parent"], torch.int32),
                                  _ptr(tree["depth"], torch.int32), _ptr(tree["n_nodes"], torch.int32), lp, dtype, stride,
                                  _ptr(target_ids, torch.int32), _ptr(res["n_accept"], torch.int32),
                                  _ptr(res["accept_nodes"], torch.int32), _ptr(res["out_tokens"], torch.int32),
                                  _ptr(res["target_ids"], torch.int32), _stream(stream)), "cb_accept")
        return res

    def cb_accept_update_draft_tree(self, tree, logits, tokens, seq_len, next_tree=None, res=None, stream=None):
        """cb_accept on `tree` and `logits`, the emitted tokens appended to `tokens` (seq_len advanced in place), then cb_update
        and cb_draft_tree into next_tree (default: the same arrays as `tree`), in one launch."""
        res = res if res is not None else self.alloc_accept()
        next_tree = next_tree if next_tree is not None else tree
        if logits.dtype == torch.float32:
            dtype = _lib.CB_DTYPE_F32
        elif logits.dtype == torch.bfloat16:
            dtype = _lib.CB_DTYPE_BF16
        else:
            raise CachebackError("logits must be float32 or bfloat16")
        if not (logits.is_cuda and logits.dim() == 3 and logits.stride(2) == 1 and logits.stride(0) == logits.shape[1] * logits.stride(1)):
            raise CachebackError("logits must be [batch, max_nodes, vocab] with a uniform row stride")
        a = _lib.CbAcceptDraftArgsC(logits.data_ptr(), dtype, logits.stride(1), _ptr(tree["tokens"], torch.int32),
                                    _ptr(tree["parent"], torch.int32), _ptr(tree["depth"], torch.int32), _ptr(tree["n_nodes"], torch.int32),
                                    _ptr(res["n_accept"], torch.int32), _ptr(res["accept_nodes"], torch.int32),
                                    _ptr(res["out_tokens"], torch.int32), _ptr(res["target_ids"], torch.int32),
                                    _ptr(tokens, torch.int32), tokens.stride(0), _ptr(seq_len, torch.int32),
                                    _ptr(next_tree["tokens"], torch.int32), _ptr(next_tree["parent"], torch.int32),
                                    _ptr(next_tree["depth"], torch.int32), _ptr(next_tree["mask"], torch.int32),
                                    _ptr(next_tree["n_nodes"], torch.int32))
        _check(self.lib.cb_accept_update_draft_tree(self._h, C.byref(a), _stream(stream)), "cb_accept_update_draft_tree")
        return res

    # ---- helpers ------------------------------------------------------------------------------------
    def cb_frozen_attach(self, frozen):
        """frozen: a FrozenTable (kept alive by this object) or None to detach."""
        if frozen is None:
            _check(self.lib.cb_frozen_attach(self._h, None, None, 0), "cb_frozen_attach")
        else:
            _check(self.lib.cb_frozen_attach(self._h, C.byref(frozen.cfg), frozen.ptr, frozen.bytes), "cb_frozen_attach")
        self._frozen = frozen

    def cb_table_dump(self, seq):
        """[(leader tuple, [follower tuples])], least recently used first (host lists)."""
        c = self.cfg
        n = C.c_int32(0)
        leaders = np.empty((c.LC, c.LL), dtype=np.int32)
        nfol = np.empty(c.LC, dtype=np.int32)
        fol = np.empty((c.LC, c.FC, c.FL), dtype=np.int32)
        _check(self.lib.cb_table_dump(self._h, seq, C.byref(n), leaders.ctypes.data, nfol.ctypes.data, fol.ctypes.data),
               "cb_table_dump")
        return [(tuple(int(x) for x in leaders[i]), [tuple(int(x) for x in fol[i, j]) for j in range(nfol[i])])
                for i in range(n.value)]

    def cb_table_dump_arrays(self, seq):
        c = self.cfg
        n = C.c_int32(0)
        leaders = np.empty((c.LC, c.LL), dtype=np.int32)
        nfol = np.empty(c.LC, dtype=np.int32)
        fol = np.empty((c.LC, c.FC, c.FL), dtype=np.int32)
        _check(self.lib.cb_table_dump(self._h, seq, C.byref(n), leaders.ctypes.data, nfol.ctypes.data, fol.ctypes.data),
               "cb_table_dump")
        return leaders[: n.value], nfol[: n.value], fol[: n.value]

    def cb_table_load(self, seq, table):
        c = self.cfg
        n = len(table)
        leaders = np.zeros((max(n, 1), c.LL), dtype=np.int32)
        nfol = np.zeros(max(n, 1), dtype=np.int32)
        fol = np.full((max(n, 1), c.FC, c.FL), -1, dtype=np.int32)
        for i, (L, fs) in enumerate(table):
            leaders[i] = L
            nfol[i] = len(fs)
            for j, f in enumerate(fs):
                fol[i, j] = f
        _check(self.lib.cb_table_load(self._h, seq, n, leaders.ctypes.data, nfol.ctypes.data, fol.ctypes.data),
               "cb_table_load")

    def cb_poll_status(self):
        st = C.c_int32(0)
        cnt = np.zeros(_lib.CB_NUM_COUNTERS, dtype=np.uint64)
        _check(self.lib.cb_poll_status(self._h, C.byref(st), cnt.ctypes.data), "cb_poll_status")
        return st.value, dict(zip(_lib.COUNTER_NAMES, (int(x) for x in cnt)))

    def launch_count(self):
        return int(self.lib.cb_launch_count())
