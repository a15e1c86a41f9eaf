"""Pins for the KV-commit oracle (Section 3.2: accepted draft tokens stop being "non-KV-cached" tokens).

The oracle's output is fixed by what committing means: (1) re-rooting — once the path root -> parent(x) is committed,
node x alone, attending to the longer cache plus itself, sees exactly the keys it saw in the tree (context plus
ancestors-or-self), so the attention oracle must give the same row both ways; a wrong position, page, slot, order or
a K/V swap breaks it; (2) a brute-force element loop on a tiny case; (3) nothing outside the written slots changes."""
import numpy as np

import workloads as W
from tests.harness import tree_mask_from_parents
from workloads.tensors import TID


def _case(seed, B=3, T=12, Hq=4, Hkv=2, D=64, P=16, ctxs=(5, 16, 37), max_pages=6):
    rng = np.random.default_rng(seed)
    num_pages = B * max_pages + 2
    perm = rng.permutation(num_pages).astype(np.int32)
    bt = perm[: B * max_pages].reshape(B, max_pages)
    bits = lambda shape, tid: W.normal_bf16_bits(seed, tid, np.arange(int(np.prod(shape)))).reshape(shape)
    kp, vp = bits((num_pages, P, Hkv, D), TID.K_POOL), bits((num_pages, P, Hkv, D), TID.V_POOL)
    kt, vt = bits((B, T, Hkv, D), TID.K_TREE), bits((B, T, Hkv, D), TID.V_TREE)
    q = bits((B, T, Hq, D), TID.Q)
    par = np.full((B, T), -1, np.int32); dep = np.full((B, T), -1, np.int32); mask = np.zeros((B, T, 1), np.uint32)
    for b in range(B):
        par[b], dep[b] = W.random_tree(seed, b, T, 5, T)
        mask[b] = tree_mask_from_parents(par[b], T, 1)
    return dict(bt=bt, ctx=np.array(ctxs, np.int32), kp=kp, vp=vp, kt=kt, vt=vt, q=q, par=par, dep=dep, mask=mask, P=P)


def _path(par, x):
    out = []
    while x > 0:
        out.append(x); x = int(par[x])
    return out[::-1]


def test_rerooting_reproduces_the_tree_attention_row(oracle):
    c = _case(3)
    B, T = c["par"].shape
    for b in range(B):
        x = int(np.argmax(c["dep"][b]))                      # a deepest node
        path = _path(c["par"][b], x)                         # accepted nodes if x were the winner
        rows = np.array([(b, h, x) for h in range(c["q"].shape[2])], np.int32)
        want, want_lse = oracle.tree_attn_rows(c["q"], c["kp"], c["vp"], c["bt"], c["ctx"], c["kt"], c["vt"], c["mask"], rows)
        # commit root -> parent(x); then x, alone, is a one-node tree over the longer cache
        kp, vp = c["kp"].copy(), c["vp"].copy()
        n_acc = np.zeros(B, np.int32); nodes = np.full((B, 8), -1, np.int32)
        n_acc[b] = len(path) - 1; nodes[b, : len(path) - 1] = path[:-1]
        others = [bb for bb in range(B) if bb != b]
        n_acc[others] = -1                                    # left untouched
        ctx2 = oracle.kv_commit(kp, vp, c["bt"], c["ctx"], c["kt"], c["vt"], n_acc, nodes)
        assert ctx2[b] == c["ctx"][b] + len(path) and all(ctx2[o] == c["ctx"][o] for o in others)
        q1 = np.zeros_like(c["q"]); kt1 = np.zeros_like(c["kt"]); vt1 = np.zeros_like(c["vt"])
        q1[b, 0], kt1[b, 0], vt1[b, 0] = c["q"][b, x], c["kt"][b, x], c["vt"][b, x]
        m1 = np.zeros_like(c["mask"]); m1[b, 0, 0] = 1
        rows1 = np.array([(b, h, 0) for h in range(c["q"].shape[2])], np.int32)
        got, got_lse = oracle.tree_attn_rows(q1, kp, vp, c["bt"], ctx2, kt1, vt1, m1, rows1)
        assert np.allclose(got, want, rtol=1e-12, atol=1e-14) and np.allclose(got_lse, want_lse, rtol=1e-12, atol=1e-12)


def test_brute_force_and_untouched_slots(oracle):
    c = _case(11, ctxs=(0, 15, 79))
    B = 3
    n_acc = np.array([2, 0, 3], np.int32)
    nodes = np.full((B, 5), -1, np.int32)
    for b in range(B):
        x = [i for i in range(c["par"].shape[1]) if c["dep"][b, i] == n_acc[b]][0] if n_acc[b] else 0
        nodes[b, : n_acc[b]] = _path(c["par"][b], x)
    kp, vp = c["kp"].copy(), c["vp"].copy()
    ctx2 = oracle.kv_commit(kp, vp, c["bt"], c["ctx"], c["kt"], c["vt"], n_acc, nodes)
    assert ctx2.tolist() == [3, 16, 83]
    written = set()
    P = c["P"]
    for b in range(B):
        for j, node in enumerate([0] + nodes[b, : n_acc[b]].tolist()):
            pos = int(c["ctx"][b]) + j
            page, slot = int(c["bt"][b, pos // P]), pos % P
            written.add((page, slot))
            for hh in range(kp.shape[2]):
                for d in range(kp.shape[3]):
                    assert kp[page, slot, hh, d] == c["kt"][b, node, hh, d] and vp[page, slot, hh, d] == c["vt"][b, node, hh, d]
    keep = np.ones(kp.shape[:2], bool)
    for pg, sl in written:
        keep[pg, sl] = False
    assert np.array_equal(kp[keep], c["kp"][keep]) and np.array_equal(vp[keep], c["vp"][keep])
    assert len(written) == int(n_acc.sum()) + B


def test_full_cache_is_left_alone(oracle):
    c = _case(5, ctxs=(95, 96, 90), max_pages=6)            # capacity 96 tokens
    n_acc = np.array([1, 0, 5], np.int32)
    nodes = np.zeros((3, 5), np.int32)
    nodes[2] = _path(c["par"][2], int(np.argmax(c["dep"][2])))[:5] + [0] * (5 - len(_path(c["par"][2], int(np.argmax(c["dep"][2])))[:5]))
    kp, vp = c["kp"].copy(), c["vp"].copy()
    ctx2 = oracle.kv_commit(kp, vp, c["bt"], c["ctx"], c["kt"], c["vt"], n_acc, nodes)
    assert ctx2.tolist() == [95, 96, 96]                    # 95+2 > 96 and 96+1 > 96 do not fit; 90+6 = 96 does
