"""Pins for the oracle's tree-masked attention: torch CPU softmax on dense masks, the chain tree reducing
to causal attention (library routine), the star tree, closed forms (equal keys -> mean of V, V = 1 -> 1)
and invariance under a permutation of the page pool."""
import numpy as np
import pytest
import torch

import workloads as W
from workloads.tensors import pool_full_bits, full_bits, TID
from workloads.rng import bf16_bits_to_f32
from tests.harness import tree_mask_from_parents


def _setup(cfg, ctx, seed_tree=0, chain=False, star=False):
    B, T = cfg.batch, cfg.max_nodes
    ctx = np.asarray(ctx, dtype=np.int32)
    bt, num_pages = W.make_block_table(cfg, ctx)
    kp, vp = pool_full_bits(cfg, num_pages)
    q = full_bits(cfg, TID.Q, (B, T, cfg.n_q_heads, cfg.head_dim))
    kt = full_bits(cfg, TID.K_TREE, (B, T, cfg.n_kv_heads, cfg.head_dim))
    vt = full_bits(cfg, TID.V_TREE, (B, T, cfg.n_kv_heads, cfg.head_dim))
    masks, ns, pars = [], [], []
    for b in range(B):
        n = T - (b % 3)
        if chain:
            par = np.arange(-1, T - 1, dtype=np.int32)
        elif star:
            par = np.zeros(T, dtype=np.int32); par[0] = -1
        else:
            par, _ = W.random_tree(seed_tree, b, n, cfg.max_depth, T)
        masks.append(tree_mask_from_parents(par, n, (T + 31) // 32))
        ns.append(n); pars.append(par)
    return dict(q=q, kp=kp, vp=vp, bt=bt, ctx=ctx, kt=kt, vt=vt, mask=np.stack(masks), n=ns, par=pars)


def _torch_ref(cfg, d, b, h):
    """Dense-mask softmax attention in torch fp64 for one (sequence, q head): [n, D]."""
    P, G = cfg.page_size, cfg.gqa
    kh = h // G
    ctx, n, T = int(d["ctx"][b]), d["n"][b], cfg.max_nodes
    t = np.arange(ctx)
    pages = d["bt"][b][t // P]
    K = np.concatenate([bf16_bits_to_f32(d["kp"][pages, t % P, kh]), bf16_bits_to_f32(d["kt"][b, :, kh])])
    V = np.concatenate([bf16_bits_to_f32(d["vp"][pages, t % P, kh]), bf16_bits_to_f32(d["vt"][b, :, kh])])
    Q = bf16_bits_to_f32(d["q"][b, :n, h])
    vis = np.ones((n, ctx + T), dtype=bool)
    for i in range(n):
        for j in range(T):
            vis[i, ctx + j] = (int(d["mask"][b, i, j // 32]) >> (j % 32)) & 1
    Qt, Kt, Vt = (torch.from_numpy(x.astype(np.float64)) for x in (Q, K, V))
    s = Qt @ Kt.T * cfg.head_dim ** -0.5
    s = s.masked_fill(~torch.from_numpy(vis), float("-inf"))
    return (torch.softmax(s, dim=-1) @ Vt).numpy(), torch.logsumexp(s, dim=-1).numpy()


def _oracle_rows(oracle, d, rows):
    return oracle.tree_attn_rows(d["q"], d["kp"], d["vp"], d["bt"], d["ctx"], d["kt"], d["vt"], d["mask"], rows)


SMALL = W.CbConfig("attn_small", 3, 2, 2, 64, 2, 12, 4, 0, 4, 2, 64, (5, 70), 100, 1.1, 0.3, (4, 8), 64)


def test_against_torch_dense_mask(oracle):
    d = _setup(SMALL, [37, 70, 5])
    for b in range(3):
        for h in range(4):
            rows = [(b, h, i) for i in range(d["n"][b])]
            out, lse = _oracle_rows(oracle, d, rows)
            ref, ref_lse = _torch_ref(SMALL, d, b, h)
            np.testing.assert_allclose(out, ref, rtol=1e-10, atol=1e-12)
            np.testing.assert_allclose(lse, ref_lse, rtol=1e-10, atol=1e-12)


def test_chain_tree_is_causal_attention(oracle):
    """par[i] = i-1: node i sees the context and tree keys 0..i — ordinary causal attention of T new
    tokens appended to the context, computed here by torch's scaled_dot_product_attention."""
    cfg = SMALL
    d = _setup(cfg, [33, 16, 64], chain=True)
    T, D = cfg.max_nodes, cfg.head_dim
    for b in range(3):
        n, ctx = d["n"][b], int(d["ctx"][b])
        h, kh = 3, 1
        t = np.arange(ctx)
        pages = d["bt"][b][t // cfg.page_size]
        K = np.concatenate([bf16_bits_to_f32(d["kp"][pages, t % 16, kh]), bf16_bits_to_f32(d["kt"][b, :n, kh])])
        V = np.concatenate([bf16_bits_to_f32(d["vp"][pages, t % 16, kh]), bf16_bits_to_f32(d["vt"][b, :n, kh])])
        Q = np.concatenate([np.zeros((ctx, D), np.float32), bf16_bits_to_f32(d["q"][b, :n, h])])
        to = lambda x: torch.from_numpy(x.astype(np.float64))[None, None]
        ref = torch.nn.functional.scaled_dot_product_attention(to(Q), to(K), to(V), is_causal=True)[0, 0, ctx:]
        out, _ = _oracle_rows(oracle, d, [(b, h, i) for i in range(n)])
        np.testing.assert_allclose(out, ref.numpy(), rtol=1e-9, atol=1e-11)


def test_star_tree_rows_are_independent_decodes(oracle):
    """All nodes children of the root: node i sees context + root + itself only."""
    cfg = SMALL
    d = _setup(cfg, [20, 48, 7], star=True)
    b, h, kh = 1, 0, 0
    ctx = int(d["ctx"][b])
    t = np.arange(ctx)
    pages = d["bt"][b][t // 16]
    Kc, Vc = bf16_bits_to_f32(d["kp"][pages, t % 16, kh]), bf16_bits_to_f32(d["vp"][pages, t % 16, kh])
    out, lse = _oracle_rows(oracle, d, [(b, h, i) for i in range(d["n"][b])])
    for i in range(d["n"][b]):
        sel = sorted({0, i})
        K = np.concatenate([Kc, bf16_bits_to_f32(d["kt"][b, sel, kh])]).astype(np.float64)
        V = np.concatenate([Vc, bf16_bits_to_f32(d["vt"][b, sel, kh])]).astype(np.float64)
        q = bf16_bits_to_f32(d["q"][b, i, h]).astype(np.float64)
        s = K @ q / 8.0
        p = np.exp(s - s.max()); p /= p.sum()
        np.testing.assert_allclose(out[i], p @ V, rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(lse[i], np.log(np.exp(s - s.max()).sum()) + s.max(), rtol=1e-12)


def test_closed_forms(oracle):
    cfg = SMALL
    d = _setup(cfg, [37, 70, 5])
    b, h = 0, 2
    rows = [(b, h, i) for i in range(d["n"][b])]
    # V == 1 everywhere -> every output element is exactly the sum of the probabilities = 1
    one = np.uint16(0x3F80)
    d1 = dict(d); d1["vp"] = np.full_like(d["vp"], one); d1["vt"] = np.full_like(d["vt"], one)
    out, _ = _oracle_rows(oracle, d1, rows)
    np.testing.assert_allclose(out, 1.0, rtol=0, atol=1e-14)
    # all keys equal -> uniform weights -> output = mean of the visible V rows; lse = s + log(count)
    d2 = dict(d); d2["kp"] = np.full_like(d["kp"], one); d2["kt"] = np.full_like(d["kt"], one)
    out, lse = _oracle_rows(oracle, d2, rows)
    kh = h // cfg.gqa
    ctx = int(d["ctx"][b]); t = np.arange(ctx); pages = d["bt"][b][t // 16]
    Vc = bf16_bits_to_f32(d["vp"][pages, t % 16, kh]).astype(np.float64)
    Vt = bf16_bits_to_f32(d["vt"][b, :, kh]).astype(np.float64)
    for i in range(d["n"][b]):
        vis = [j for j in range(cfg.max_nodes) if (int(d["mask"][b, i, 0]) >> j) & 1]
        ref = (Vc.sum(0) + Vt[vis].sum(0)) / (ctx + len(vis))
        np.testing.assert_allclose(out[i], ref, rtol=1e-12, atol=1e-14)
        s = bf16_bits_to_f32(d["q"][b, i, h]).astype(np.float64).sum() / 8.0
        np.testing.assert_allclose(lse[i], s + np.log(ctx + len(vis)), rtol=1e-12)


def test_page_permutation_invariance(oracle):
    cfg = SMALL
    d = _setup(cfg, [37, 70, 5])
    rows = [(b, h, i) for b in range(3) for h in (0, 3) for i in (0, d["n"][b] - 1)]
    out, lse = _oracle_rows(oracle, d, rows)
    perm = np.random.default_rng(1).permutation(d["kp"].shape[0])
    inv = np.argsort(perm)
    d2 = dict(d)
    d2["kp"], d2["vp"] = d["kp"][perm], d["vp"][perm]          # page p moves to slot inv[p]
    d2["bt"] = np.where(d["bt"] >= 0, inv[np.maximum(d["bt"], 0)], -1).astype(np.int32)
    out2, lse2 = _oracle_rows(oracle, d2, rows)
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)


def test_mask_from_parents_matches_generator(oracle):
    par, _ = W.random_tree(3, 0, 50, 7, 64)
    assert np.array_equal(oracle.tree_mask(par, 50, 64), tree_mask_from_parents(par, 50, 2))


def test_grouped_row_helper_matches_whole_tensor_call(oracle):
    """The full-size GPU tests call the oracle on one kv head at a time (compact copies of that head's keys); that route
    must give exactly what the whole-tensor call gives."""
    from tests.harness import Problem, synthetic_trees, oracle_attn_rows, oracle_attn_rows_by_head
    cfg = W.CbConfig("attn_small_gqa", 3, 2, 2, 64, 2, 40, 6, 0, 8, 2, 64, (0, 300), 100, 1.1, 0.3, (4, 8), 64)
    prob = Problem(cfg)
    par, dep, mask, n = synthetic_trees(cfg, full=False)
    rng = np.random.default_rng(3)
    rows = [(int(b), int(rng.integers(0, cfg.n_q_heads)), int(rng.integers(0, n[b]))) for b in rng.integers(0, cfg.batch, 40)]
    got, got_lse = oracle_attn_rows_by_head(oracle, cfg, prob, mask, rows, threads=3)
    for k, (b, h, i) in enumerate(rows):
        ref, ref_lse = oracle_attn_rows(oracle, cfg, prob, mask, b, [(h, i)])
        assert np.array_equal(got[k], ref[0]) and got_lse[k] == ref_lse[0]


def test_shared_unit_rows_lie_in_units_cut_by_a_range_boundary():
    from tests.harness import shared_unit_rows
    cfg = W.get_config("c3_8b_gqa")
    ctx = W.ctx_lens(cfg)
    n = np.full(cfg.batch, cfg.max_nodes, np.int32)
    rows = shared_unit_rows(cfg, ctx, n, 148)
    assert 74 <= len(rows) <= 147
    # brute force: label every position of the global sequence with its unit and whether it is a key tile
    G, npt = cfg.gqa, 128 // cfg.gqa
    label = []
    for b in range(cfg.batch):                             # 64 nodes x 4 heads = two row tiles = one row group
        tiles = -(-int(ctx[b]) // 128) + 1
        for kh in range(cfg.n_kv_heads):
            label += [(b, kh, False)] * 3 + [(b, kh, True)] * tiles
    total = len(label)
    cut_units = set()
    for c in range(1, 148):
        g = total * c // 148
        if label[g - 1][:2] == label[g][:2] and label[g - 1][2] and label[g][2]:
            cut_units.add(label[g][:2])
    assert {(b, h // G) for b, h, i in rows} == cut_units
    assert all(0 <= i < cfg.max_nodes for _, _, i in rows)
    # several row groups (128 nodes x 8 heads = 8 row tiles = 4 row groups): the row group is the outermost index
    cfg = W.get_config("c5_70b_long")
    ctx = W.ctx_lens(cfg)
    n = np.full(cfg.batch, cfg.max_nodes, np.int32)
    rows = shared_unit_rows(cfg, ctx, n, 74)
    label = []
    for rg in range(4):
        for b in range(cfg.batch):
            tiles = -(-int(ctx[b]) // 128) + 1
            for kh in range(cfg.n_kv_heads):
                label += [(b, kh, rg, False)] * 3 + [(b, kh, rg, True)] * tiles
    total = len(label)
    cut_units = set()
    for c in range(1, 74):
        g = total * c // 74
        if label[g - 1][:3] == label[g][:3] and label[g - 1][3] and label[g][3]:
            cut_units.add(label[g][:3])
    npt = 128 // cfg.gqa
    assert {(b, h // cfg.gqa, i // (2 * npt)) for b, h, i in rows} == cut_units
