"""Synthetic tensors of the verify step: paged K/V pool, block tables, context lengths, queries, tree
K/V, logits.  Each tensor has an id; element (flat index i) of tensor t is normal(seed, t, i), so the host
can materialise any slice (for the oracle) while the device fills the whole tensor with the same values.
"""
import numpy as np

from .rng import mix64, normal_f32, normal_bf16_bits, uniform_f64, f32_to_bf16_bits, bf16_bits_to_f32
from .configs import CbConfig


class TID:
    K_POOL, V_POOL, Q, K_TREE, V_TREE, LOGITS, PAGES, CTX, PLANT = 1, 2, 3, 4, 5, 6, 7, 8, 9


def ctx_lens(cfg: CbConfig) -> np.ndarray:
    """int32 [B] context lengths, uniform over cfg.ctx_range (inclusive)."""
    lo, hi = cfg.ctx_range
    u = uniform_f64(cfg.seed, TID.CTX, np.arange(cfg.batch))
    return (lo + np.floor(u * (hi - lo + 1))).astype(np.int32)


def make_block_table(cfg: CbConfig, ctx: np.ndarray):
    """Seeded random placement of every sequence's pages in one pool, so pages are never contiguous.
    Returns (block_table int32 [B, max_pages] padded with -1, num_pages)."""
    P = cfg.page_size
    npg = (ctx.astype(np.int64) + P - 1) // P
    max_pages = int((cfg.max_ctx + P - 1) // P)
    total = int(npg.sum())
    num_pages = total + 3                                  # a few pages no sequence owns
    perm = np.argsort(mix64(cfg.seed, TID.PAGES, np.arange(num_pages)), kind="stable").astype(np.int32)
    bt = np.full((cfg.batch, max_pages), -1, dtype=np.int32)
    o = 0
    for b in range(cfg.batch):
        bt[b, : npg[b]] = perm[o:o + npg[b]]
        o += int(npg[b])
    return bt, num_pages


def _gather(seed, tid, idx, as_f32):
    bits = normal_bf16_bits(seed, tid, idx)
    return bf16_bits_to_f32(bits) if as_f32 else bits


def pool_slice_kv(cfg: CbConfig, pages: np.ndarray, kv_head: int, n_tokens: int, as_f32=True):
    """K and V rows of one kv head for the first n_tokens tokens of the given page list.
    Pool layout [num_pages, page_size, n_kv_heads, head_dim]. Returns (K, V) each [n_tokens, D]."""
    P, H, D = cfg.page_size, cfg.n_kv_heads, cfg.head_dim
    t = np.arange(n_tokens)
    row = (pages[t // P].astype(np.int64) * P + t % P) * H + kv_head
    idx = row[:, None] * D + np.arange(D)[None, :]
    return _gather(cfg.seed, TID.K_POOL, idx, as_f32), _gather(cfg.seed, TID.V_POOL, idx, as_f32)


def pool_full_bits(cfg: CbConfig, num_pages: int):
    """Whole pool as bf16 bit patterns (uint16) [num_pages, P, Hkv, D] for K and V. Small configs only."""
    n = num_pages * cfg.page_size * cfg.n_kv_heads * cfg.head_dim
    shape = (num_pages, cfg.page_size, cfg.n_kv_heads, cfg.head_dim)
    idx = np.arange(n)
    return (normal_bf16_bits(cfg.seed, TID.K_POOL, idx).reshape(shape),
            normal_bf16_bits(cfg.seed, TID.V_POOL, idx).reshape(shape))


def pool_pages_bits(cfg: CbConfig, pages: np.ndarray):
    """The given pages of the pool, all kv heads, as bf16 bit patterns [len(pages), P, Hkv, D] for K and V."""
    P, H, D = cfg.page_size, cfg.n_kv_heads, cfg.head_dim
    per = P * H * D
    idx = np.asarray(pages, dtype=np.int64)[:, None] * per + np.arange(per)[None, :]
    shape = (len(pages), P, H, D)
    return (normal_bf16_bits(cfg.seed, TID.K_POOL, idx).reshape(shape),
            normal_bf16_bits(cfg.seed, TID.V_POOL, idx).reshape(shape))


def seq_bits(cfg: CbConfig, tid: int, b: int, heads: int):
    """One sequence's slice of a [B, T, heads, D] tensor as bf16 bit patterns [T, heads, D]."""
    per = cfg.max_nodes * heads * cfg.head_dim
    return normal_bf16_bits(cfg.seed, tid, b * per + np.arange(per)).reshape(cfg.max_nodes, heads, cfg.head_dim)


def tree_kv(cfg: CbConfig, b: int, kv_head: int, as_f32=True):
    """K and V of the draft-tree tokens of sequence b, one kv head: layout [B, T, Hkv, D] -> [T, D]."""
    T, H, D = cfg.max_nodes, cfg.n_kv_heads, cfg.head_dim
    row = (b * T + np.arange(T)) * H + kv_head
    idx = row[:, None].astype(np.int64) * D + np.arange(D)[None, :]
    return _gather(cfg.seed, TID.K_TREE, idx, as_f32), _gather(cfg.seed, TID.V_TREE, idx, as_f32)


def queries(cfg: CbConfig, b: int, q_head: int, as_f32=True):
    """Queries of sequence b, one q head: layout [B, T, Hq, D] -> [T, D]."""
    T, H, D = cfg.max_nodes, cfg.n_q_heads, cfg.head_dim
    row = (b * T + np.arange(T)) * H + q_head
    idx = row[:, None].astype(np.int64) * D + np.arange(D)[None, :]
    return _gather(cfg.seed, TID.Q, idx, as_f32)


def full_bits(cfg: CbConfig, tid: int, shape):
    """Any whole tensor as bf16 bit patterns. Small configs only."""
    return normal_bf16_bits(cfg.seed, tid, np.arange(int(np.prod(shape)))).reshape(shape)


def logits_rows(cfg: CbConfig, b: int, nodes, dtype="f32") -> np.ndarray:
    """Logit rows [len(nodes), V] of sequence b (layout [B, T, V]); float32 values, rounded through bf16
    when dtype == 'bf16'."""
    nodes = np.asarray(nodes, dtype=np.int64)
    idx = ((b * cfg.max_nodes + nodes)[:, None] * cfg.vocab) + np.arange(cfg.vocab)[None, :]
    x = normal_f32(cfg.seed, TID.LOGITS, idx)
    if dtype == "bf16":
        x = bf16_bits_to_f32(f32_to_bf16_bits(x))
    return x


def plant_logits(cfg: CbConfig, b: int, tok: np.ndarray, par: np.ndarray, dep: np.ndarray, n: int,
                 p_path: float = 0.5):
    """Choose where to plant a winning logit so that about p_path of the root-to-leaf paths carry a run
    of matches: for each chosen leaf, a depth d uniform in [1, depth(leaf)] is drawn and, for every node
    c on the path with depth <= d, (parent(c), token(c)) is planted unless that parent already has a
    plant.  Returns a list of (node, vocab_id); the caller sets logits[b, node, vocab_id] = +32."""
    is_leaf = np.ones(n, dtype=bool)
    for i in range(1, n):
        is_leaf[par[i]] = False
    u = uniform_f64(cfg.seed, TID.PLANT, (b * 4096 + np.arange(max(n, 1))) * 2)
    u2 = uniform_f64(cfg.seed, TID.PLANT, (b * 4096 + np.arange(max(n, 1))) * 2 + 1)
    planted = {}
    for leaf in range(1, n):
        if not is_leaf[leaf] or u[leaf] >= p_path:
            continue
        d = 1 + int(u2[leaf] * dep[leaf])
        path = []
        c = leaf
        while c > 0:
            path.append(c)
            c = int(par[c])
        for c in reversed(path):
            if dep[c] > d:
                break
            planted.setdefault(int(par[c]), int(tok[c]))
    return sorted(planted.items())
