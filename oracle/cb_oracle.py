"""ctypes binding of the CPU oracle (oracle/cb_oracle.cpp).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's cpu-baseline leg import this module; the CUDA path never
does and shares nothing with it.  The shared object is compiled with g++ on first use.
"""
import ctypes as C
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cb_oracle.cpp")
_SO = os.path.join(_HERE, "libcb_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".tmp%d" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _SO)
    return _SO


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        L = _lib
        L.orc_table_new.restype = C.c_void_p
        L.orc_table_new.argtypes = [C.c_int] * 5
        L.orc_table_free.argtypes = [C.c_void_p]
        L.orc_table_reset.argtypes = [C.c_void_p]
        L.orc_table_clock.restype = C.c_uint64
        L.orc_table_clock.argtypes = [C.c_void_p]
        L.orc_table_num_leaders.restype = C.c_int64
        L.orc_table_num_leaders.argtypes = [C.c_void_p]
        L.orc_insert.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_query.restype = C.c_int
        L.orc_query.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_update.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int]
        L.orc_table_dump.restype = C.c_int64
        L.orc_table_dump.argtypes = [C.c_void_p] * 4
        L.orc_draft_tree.restype = C.c_int
        L.orc_draft_tree.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int] + [C.c_void_p] * 6
        L.orc_frozen_new.restype = C.c_void_p
        L.orc_frozen_new.argtypes = [C.c_int, C.c_int]
        L.orc_frozen_free.argtypes = [C.c_void_p]
        L.orc_frozen_add.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]
        L.orc_draft_tree_dual.restype = C.c_int
        L.orc_draft_tree_dual.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int] + [C.c_void_p] * 8
        L.orc_tree_mask.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p]
        L.orc_argmax_f32.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int, C.c_void_p]
        L.orc_accept.restype = C.c_int
        L.orc_accept.argtypes = [C.c_void_p] * 3 + [C.c_int, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_tree_attn_rows.argtypes = ([C.c_void_p] * 8 + [C.c_int] * 6 + [C.c_double, C.c_void_p, C.c_int,
                                                                               C.c_void_p, C.c_void_p])
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


class OracleTable:
    """One sequence's cache table (Section 3.1)."""

    def __init__(self, LL, FL, LC, FC, refresh_on_reinsert=True):
        self.LL, self.FL, self.LC, self.FC = LL, FL, LC, FC
        self._h = lib().orc_table_new(LL, FL, LC, FC, int(refresh_on_reinsert))

    def __del__(self):
        if getattr(self, "_h", None) and _lib is not None:
            _lib.orc_table_free(self._h)
            self._h = None

    def reset(self):
        lib().orc_table_reset(self._h)

    @property
    def clock(self):
        return int(lib().orc_table_clock(self._h))

    def __len__(self):
        return int(lib().orc_table_num_leaders(self._h))

    def insert(self, leader, follower):
        L, F = _i32(leader), _i32(follower)
        assert L.size == self.LL and F.size == self.FL
        lib().orc_insert(self._h, _p(L), _p(F))

    def query(self, leader):
        L = _i32(leader)
        assert L.size == self.LL
        out = np.empty((self.FC, self.FL), dtype=np.int32)
        n = lib().orc_query(self._h, _p(L), _p(out))
        return [tuple(int(x) for x in out[i]) for i in range(n)]

    def update(self, tokens, n_old, n_new):
        s = _i32(tokens)
        assert n_new <= s.size
        lib().orc_update(self._h, _p(s), int(n_old), int(n_new))

    def dump(self):
        """[(leader tuple, [follower tuples])] — leaders and followers least recently used first."""
        n = len(self)
        leaders = np.empty((n, self.LL), dtype=np.int32)
        nfol = np.empty(n, dtype=np.int32)
        fol = np.empty((n, self.FC, self.FL), dtype=np.int32)
        lib().orc_table_dump(self._h, _p(leaders), _p(nfol), _p(fol))
        return [(tuple(int(x) for x in leaders[i]), [tuple(int(x) for x in fol[i, j]) for j in range(nfol[i])])
                for i in range(n)]

    def dump_arrays(self):
        n = len(self)
        leaders = np.empty((n, self.LL), dtype=np.int32)
        nfol = np.empty(n, dtype=np.int32)
        fol = np.empty((n, self.FC, self.FL), dtype=np.int32)
        lib().orc_table_dump(self._h, _p(leaders), _p(nfol), _p(fol))
        return leaders, nfol, fol

    def draft_tree(self, tokens, seq_len, T, crt, max_depth, with_log=False):
        s = _i32(tokens)
        W = (T + 31) // 32
        tok = np.empty(T, dtype=np.int32)
        par = np.empty(T, dtype=np.int32)
        dep = np.empty(T, dtype=np.int32)
        mask = np.empty((T, W), dtype=np.uint32)
        log = np.full((max(T, 1) * 2, self.LL + 1), -1, dtype=np.int32)
        nq = C.c_int32(0)
        n = lib().orc_draft_tree(self._h, _p(s), int(seq_len), T, crt, max_depth, _p(tok), _p(par), _p(dep),
                                 _p(mask), _p(log), C.addressof(nq))
        if with_log:
            return n, tok, par, dep, mask, [(tuple(int(x) for x in r[:-1]), int(r[-1])) for r in log[: nq.value]]
        return n, tok, par, dep, mask


def frozen_build(corpus, LL, FL, LC, FC):
    """Offline construction of the frozen table (paper Section 4, experimental set-up): the LC most frequent n-grams of
    length LL become the leaders; each leader keeps the FC most frequent n-grams of length FL that follow it.

    readings: the corpus is one token stream; an occurrence counts where LL + FL tokens are available, so every leader
    has at least one follower; equal counts are ordered by the tokens, lexicographically smallest first.
    Returns (leaders int32 [n, LL], n_followers int32 [n], followers int32 [n, FC, FL], -1 in unused places), leaders by
    falling count, each leader's followers by falling count."""
    from collections import Counter
    c = [int(x) for x in np.asarray(corpus).reshape(-1)]
    lead = Counter()
    foll = {}
    for i in range(len(c) - LL - FL + 1):
        lk = tuple(c[i:i + LL])
        lead[lk] += 1
        foll.setdefault(lk, Counter())[tuple(c[i + LL:i + LL + FL])] += 1
    top = sorted(lead.items(), key=lambda kv: (-kv[1], kv[0]))[:LC]
    n = len(top)
    leaders = np.full((n, LL), -1, np.int32)
    nfol = np.zeros(n, np.int32)
    followers = np.full((n, FC, FL), -1, np.int32)
    for r, (lk, _) in enumerate(top):
        leaders[r] = lk
        fs = sorted(foll[lk].items(), key=lambda kv: (-kv[1], kv[0]))[:FC]
        nfol[r] = len(fs)
        for k, (fk, _) in enumerate(fs):
            followers[r, k] = fk
    return leaders, nfol, followers


class OracleFrozen:
    """Read-only table of Section 3.3, filled from frozen_build's arrays (or any arrays of that shape)."""

    def __init__(self, LL, FL, leaders, n_followers, followers):
        self.LL, self.FL = LL, FL
        self._h = lib().orc_frozen_new(LL, FL)
        leaders, n_followers, followers = _i32(leaders), _i32(n_followers), _i32(followers)
        for r in range(leaders.shape[0]):
            lib().orc_frozen_add(self._h, _p(leaders[r]), int(n_followers[r]), _p(np.ascontiguousarray(followers[r])))

    def __del__(self):
        if getattr(self, "_h", None):
            lib().orc_frozen_free(self._h)
            self._h = None


def draft_tree_dual(table, frozen, tokens, seq_len, T, crt, max_depth, with_log=False):
    """Dual-table draft (Section 3.3): `table` (OracleTable) forms the tree, `frozen` (OracleFrozen or None) grows it on."""
    s = _i32(tokens)
    W = (T + 31) // 32
    tok = np.empty(T, dtype=np.int32)
    par = np.empty(T, dtype=np.int32)
    dep = np.empty(T, dtype=np.int32)
    mask = np.empty((T, W), dtype=np.uint32)
    log = np.full((max(T, 1) * 2, table.LL + 1), -1, dtype=np.int32)
    flog = np.full((max(T, 1) * 2, table.LL + 1), -1, dtype=np.int32)
    nq, nfq = C.c_int32(0), C.c_int32(0)
    n = lib().orc_draft_tree_dual(table._h, frozen._h if frozen is not None else None, _p(s), int(seq_len), T, crt, max_depth,
                                  _p(tok), _p(par), _p(dep), _p(mask), _p(log), C.addressof(nq), _p(flog), C.addressof(nfq))
    if with_log:
        unpack = lambda a, k: [(tuple(int(x) for x in r[:-1]), int(r[-1])) for r in a[:k]]
        return n, tok, par, dep, mask, unpack(log, nq.value), unpack(flog, nfq.value)
    return n, tok, par, dep, mask


def tree_mask(par, n, T):
    par = _i32(par)
    mask = np.empty((T, (T + 31) // 32), dtype=np.uint32)
    lib().orc_tree_mask(_p(par), int(n), int(T), _p(mask))
    return mask


def argmax_rows(logits):
    x = np.ascontiguousarray(logits, dtype=np.float32)
    assert x.ndim == 2
    out = np.empty(x.shape[0], dtype=np.int32)
    lib().orc_argmax_f32(_p(x), x.shape[0], x.shape[1], x.shape[1], _p(out))
    return out


def accept(tok, par, dep, n, target, dmax):
    tok, par, dep, target = _i32(tok), _i32(par), _i32(dep), _i32(target)
    nodes = np.empty(dmax, dtype=np.int32)
    out = np.empty(dmax + 1, dtype=np.int32)
    m = lib().orc_accept(_p(tok), _p(par), _p(dep), int(n), _p(target), int(dmax), _p(nodes), _p(out))
    return m, nodes, out


def tree_attn_rows(q, k_pool, v_pool, block_table, ctx_len, k_tree, v_tree, tree_mask_, rows, scale=None):
    """All tensors in the library's layouts, bf16 as uint16 bit patterns. rows: int32 [n, 3] = (b, head, node).
    Returns (out float64 [n, D], lse float64 [n])."""
    q = np.ascontiguousarray(q, dtype=np.uint16)
    k_pool = np.ascontiguousarray(k_pool, dtype=np.uint16)
    v_pool = np.ascontiguousarray(v_pool, dtype=np.uint16)
    k_tree = np.ascontiguousarray(k_tree, dtype=np.uint16)
    v_tree = np.ascontiguousarray(v_tree, dtype=np.uint16)
    bt, cl = _i32(block_table), _i32(ctx_len)
    m = np.ascontiguousarray(tree_mask_, dtype=np.uint32)
    rows = _i32(rows).reshape(-1, 3)
    B, T, Hq, D = q.shape
    _, P, Hkv, _ = k_pool.shape
    assert k_tree.shape == (B, T, Hkv, D) and m.shape == (B, T, (T + 31) // 32)
    out = np.empty((rows.shape[0], D), dtype=np.float64)
    lse = np.empty(rows.shape[0], dtype=np.float64)
    lib().orc_tree_attn_rows(_p(q), _p(k_pool), _p(v_pool), _p(bt), _p(cl), _p(k_tree), _p(v_tree), _p(m),
                             T, Hq, Hkv, D, P, bt.shape[1], float(scale if scale is not None else D ** -0.5),
                             _p(rows), rows.shape[0], _p(out), _p(lse))
    return out, lse


def kv_commit(k_pool, v_pool, block_table, ctx_len, k_tree, v_tree, n_accept, accept_nodes):
    """KV commit of the accepted path (paper Section 3.2: the tokens fed to the verification pass without a cached
    K/V are the non-KV-cached tokens; once a branch is accepted, its tokens are ordinary context for the next step).

    Per sequence b with m = n_accept[b]: the tree root (node 0, the one pending token) and the m accepted nodes
    accept_nodes[b, :m], in path order, become context tokens ctx_len[b] .. ctx_len[b] + m: their K and V rows are
    written into the paged cache at those positions (page block_table[b, pos // P], slot pos % P) and ctx_len[b]
    grows by m + 1.  The bonus token has no K/V yet; it is the next step's root.  A sequence whose new length would
    exceed its pages is left untouched.  Arrays: k_pool, v_pool [num_pages, P, Hkv, D] (any dtype; modified in place),
    k_tree, v_tree [B, T, Hkv, D].  Returns the new ctx_len (int32 [B])."""
    B = block_table.shape[0]
    P = k_pool.shape[1]
    out = np.array(ctx_len, dtype=np.int32, copy=True)
    for b in range(B):
        m = int(n_accept[b])
        ctx = int(ctx_len[b])
        if m < 0 or ctx + m + 1 > block_table.shape[1] * P:
            continue
        path = [0] + [int(x) for x in accept_nodes[b, :m]]
        for j, node in enumerate(path):
            pos = ctx + j
            page = int(block_table[b, pos // P])
            k_pool[page, pos % P] = k_tree[b, node]
            v_pool[page, pos % P] = v_tree[b, node]
        out[b] = ctx + m + 1
    return out


def tree_add_branches(tok, par, dep, mask, n, max_depth, branches, branch_len):
    """Drafts of another speculative-decoding method inserted as additional branches of the tree (paper, Conclusion: the
    tree organisation lets other methods' predicted drafts be added as extra branches).

    readings: a draft is a run of tokens that continues the sequence after the pending token, so it hangs below the root as
    a chain; drafts are taken in the given order; a chain is cut where the tree's size cap T = len(tok) or the depth cap
    would be exceeded (as table followers are) and a negative token ends it; branches are not compared with the nodes
    already present.  A tree without a root (n = 0) takes nothing.
    tok, par, dep: int32 [T]; mask: uint32 [T, W]; branches: int32 [K, Lmax]; branch_len: int32 [K].
    Returns new copies (n, tok, par, dep, mask)."""
    tok, par, dep = (np.array(x, dtype=np.int32, copy=True) for x in (tok, par, dep))
    mask = np.array(mask, dtype=np.uint32, copy=True)
    T = tok.shape[0]
    n = int(n)
    if n < 1:
        return n, tok, par, dep, mask
    branches = np.asarray(branches, dtype=np.int32)
    for k in range(branches.shape[0]):
        p = 0
        for j in range(min(int(branch_len[k]), branches.shape[1])):
            t = int(branches[k, j])
            if t < 0 or n >= T or dep[p] >= max_depth:
                break
            tok[n], par[n], dep[n] = t, p, dep[p] + 1
            mask[n] = mask[p]
            mask[n, n // 32] |= np.uint32(1 << (n % 32))
            p = n
            n += 1
    return n, tok, par, dep, mask
