"""Shared set-up for the GPU parity tests: builds the same seeded problem for the CUDA path (device
tensors) and for the oracle (host slices)."""
import numpy as np
import torch

import workloads as W
from workloads import device as wdev
from workloads.tensors import TID


def dev(x, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(x))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def tree_mask_from_parents(par, n, words):
    """uint32 [T, words]: bit j of row i set iff node j is node i or one of its ancestors; rows >= n zero.  Test input for
    attention-only cases (synthetic trees); pinned against the oracle's mask routine in test_oracle_attn.py."""
    T = par.shape[0]
    m = np.zeros((T, words), dtype=np.uint32)
    for i in range(n):
        if par[i] >= 0:
            m[i] = m[par[i]]
        m[i, i // 32] |= np.uint32(1) << np.uint32(i % 32)
    return m


class Problem:
    """Streams, contexts and block tables of one config (host side)."""

    def __init__(self, cfg):
        self.cfg = cfg
        self.ctx = W.ctx_lens(cfg)
        self.toks, self.lens = W.make_streams(cfg, self.ctx)
        self.bt, self.num_pages = W.make_block_table(cfg, self.ctx)
        # prefill = the context: the table has seen exactly the cached tokens plus the pending root
        self.prefill = np.minimum(self.ctx + 1, self.lens).astype(np.int32)


def device_attn_inputs(cfg, prob):
    B, T = cfg.batch, cfg.max_nodes
    bf = torch.bfloat16
    d = {}
    d["k_pool"] = wdev.normal_tensor((prob.num_pages, cfg.page_size, cfg.n_kv_heads, cfg.head_dim), bf, cfg.seed, TID.K_POOL)
    d["v_pool"] = wdev.normal_tensor((prob.num_pages, cfg.page_size, cfg.n_kv_heads, cfg.head_dim), bf, cfg.seed, TID.V_POOL)
    d["q"] = wdev.normal_tensor((B, T, cfg.n_q_heads, cfg.head_dim), bf, cfg.seed, TID.Q)
    d["k_tree"] = wdev.normal_tensor((B, T, cfg.n_kv_heads, cfg.head_dim), bf, cfg.seed, TID.K_TREE)
    d["v_tree"] = wdev.normal_tensor((B, T, cfg.n_kv_heads, cfg.head_dim), bf, cfg.seed, TID.V_TREE)
    d["block_table"] = dev(prob.bt)
    d["ctx_len"] = dev(prob.ctx)
    return d


def synthetic_trees(cfg, full=True):
    """Per-sequence random trees (parents, depths, masks, node counts). full=False varies the size."""
    B, T = cfg.batch, cfg.max_nodes
    Wd = (T + 31) // 32
    par = np.full((B, T), -1, np.int32)
    dep = np.full((B, T), -1, np.int32)
    mask = np.zeros((B, T, Wd), np.uint32)
    n = np.zeros(B, np.int32)
    for b in range(B):
        n[b] = T if full else max(1, T - (b * 7) % T)
        if b == 1 and not full:
            n[b] = 1
        par[b], dep[b] = W.random_tree(cfg.seed, b, int(n[b]), cfg.max_depth, T)
        mask[b] = tree_mask_from_parents(par[b], int(n[b]), Wd)
    return par, dep, mask, n


def oracle_attn_rows(oracle, cfg, prob, mask, b, rows_hi):
    """Oracle outputs for rows (h, i) of sequence b, from a compact host copy of that sequence's inputs."""
    P = cfg.page_size
    npg = (int(prob.ctx[b]) + P - 1) // P
    pages = prob.bt[b, :npg]
    kp, vp = W.pool_pages_bits(cfg, pages)
    q = W.seq_bits(cfg, TID.Q, b, cfg.n_q_heads)[None]
    kt = W.seq_bits(cfg, TID.K_TREE, b, cfg.n_kv_heads)[None]
    vt = W.seq_bits(cfg, TID.V_TREE, b, cfg.n_kv_heads)[None]
    bt = np.arange(max(npg, 1), dtype=np.int32)[None]
    if npg == 0:
        kp = np.zeros((1, P, cfg.n_kv_heads, cfg.head_dim), np.uint16)
        vp = kp
    rows = np.array([(0, h, i) for h, i in rows_hi], dtype=np.int32)
    return oracle.tree_attn_rows(q, kp, vp, bt, prob.ctx[b:b + 1], kt, vt, mask[b:b + 1], rows)


def bf16_to_f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def oracle_attn_rows_by_head(oracle, cfg, prob, mask, rows, threads=None):
    """Oracle outputs for rows (b, h, i) anywhere in the batch.  Rows are grouped by (sequence, kv head); each group gets a
    compact host copy of that head's keys and values only (one kv head, the group's G query heads), so that the full-size
    configurations stay affordable.  The oracle itself is single-threaded; independent groups run on a thread pool.
    Returns (out float64 [n, D], lse float64 [n]) in the order of `rows`."""
    import os
    from concurrent.futures import ThreadPoolExecutor
    rows = np.asarray(rows, dtype=np.int64).reshape(-1, 3)
    P, D, T, G = cfg.page_size, cfg.head_dim, cfg.max_nodes, cfg.gqa
    groups = {}
    for r, (b, h, i) in enumerate(rows):
        groups.setdefault((int(b), int(h) // G), []).append(r)
    out = np.empty((len(rows), D), np.float64)
    lse = np.empty(len(rows), np.float64)

    def work(item):
        (b, kh), idx = item
        ctx = int(prob.ctx[b])
        npg = (ctx + P - 1) // P
        if npg > 0:
            kp, vp = W.pool_slice_kv(cfg, prob.bt[b, :npg], kh, npg * P, as_f32=False)
            kp, vp = kp.reshape(npg, P, 1, D), vp.reshape(npg, P, 1, D)
        else:
            kp = vp = np.zeros((1, P, 1, D), np.uint16)
        q = np.stack([W.queries(cfg, b, kh * G + g, as_f32=False) for g in range(G)], axis=1)[None]   # [1, T, G, D]
        kt, vt = W.tree_kv(cfg, b, kh, as_f32=False)
        sub = np.array([(0, int(rows[r, 1]) % G, int(rows[r, 2])) for r in idx], np.int32)
        # long groups are cut into pieces so that the pool keeps all threads busy
        o, l = oracle.tree_attn_rows(q, kp, vp, np.arange(max(npg, 1), dtype=np.int32)[None], prob.ctx[b:b + 1],
                                     kt[None, :, None, :], vt[None, :, None, :], mask[b:b + 1], sub)
        return idx, o, l

    items = []
    for key, idx in groups.items():
        step = 256
        for k in range(0, len(idx), step):
            items.append((key, idx[k:k + step]))
    nthreads = threads or min(32, os.cpu_count() or 1)
    with ThreadPoolExecutor(max_workers=nthreads) as ex:
        for idx, o, l in ex.map(work, items):
            out[idx] = o
            lse[idx] = l
    return out, lse


def shared_unit_rows(cfg, ctx, n, n_ctas, seed=11):
    """One (b, h, i) row in every unit of tree attention that two persistent CTAs (or CTA pairs) share.

    Restates the decomposition the attention kernel documents: work is counted in 128-key tiles; sequence b has
    ceil(ctx_b / 128) + 1 of them (the last holds the tree's own keys); a row tile packs 128 / G nodes with the G query
    heads of a kv head; a unit is one (sequence, kv head, row group), a row group being a pair of row tiles (one when the
    whole tree cap fits one); every unit is preceded by 3 padding positions when its sequence has two or more row tiles,
    else 2; all units laid end to end in (row group, sequence, kv head) order, row group outermost, are cut into n_ctas
    equal ranges, range c = [total * c // n_ctas, total * (c + 1) // n_ctas)."""
    G, Hkv, T = cfg.gqa, cfg.n_kv_heads, cfg.max_nodes
    npt = 128 // G
    MT = -(-T // npt)
    rng = np.random.default_rng(seed)
    shapes = []
    for b in range(cfg.batch):
        nb = int(min(max(n[b], 0), T))
        tiles = -(-int(ctx[b]) // 128) + 1
        mtn = -(-nb // npt)
        RG = (1 if mtn > 0 else 0) if MT == 1 else (mtn + 1) // 2
        shapes.append((tiles, mtn, RG, 3 if mtn >= 2 else 2))
    units = []                                             # (first position, padding, tiles, b, kh, rg, row tiles)
    pos = 0
    for rg in range(1 if MT == 1 else (MT + 1) // 2):
        for b in range(cfg.batch):
            tiles, mtn, RG, ov = shapes[b]
            if rg >= RG:
                continue
            for kh in range(Hkv):
                nrt = 1 if MT == 1 else min(2, mtn - 2 * rg)
                units.append((pos, ov, tiles, b, kh, rg, nrt))
                pos += ov + tiles
    total = pos
    starts = sorted({total * c // n_ctas for c in range(1, n_ctas)})
    rows, k = [], 0
    for g in starts:
        while k + 1 < len(units) and units[k + 1][0] <= g:
            k += 1
        p0, ov, tiles, b, kh, rg, nrt = units[k]
        first, end = p0 + ov, p0 + ov + tiles
        if first < g < end:                                # key tiles on both sides of the cut
            rt = rg * 2 + int(rng.integers(0, nrt))
            lo, hi = rt * npt, min((rt + 1) * npt, int(n[b]))
            rows.append((b, kh * G + int(rng.integers(0, G)), int(rng.integers(lo, hi))))
    return rows
