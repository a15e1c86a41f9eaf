"""Pins for the oracle's insertion of another drafter's drafts as extra branches: a hand-worked case, the mask against the
separately pinned ancestor-mask routine, the caps, and the consequence for acceptance (a draft that equals the target's own
continuation is accepted whole)."""
import numpy as np

import workloads as W


def _tree(oracle, T=12, dmax=4):
    t = oracle.OracleTable(1, 2, 16, 4)
    t.insert([1], [2, 3])
    return t.draft_tree([9, 1], 2, T, 0, dmax)          # root 1, chain 2 3


def test_by_hand(oracle):
    n, tok, par, dep, mask = _tree(oracle)
    assert n == 3
    br = np.array([[7, 8, 9, 9, 9, 9], [5, -1, 6, 0, 0, 0], [4, 4, 4, 4, 4, 4], [2, 3, 0, 0, 0, 0]], np.int32)
    ln = np.array([6, 3, 0, 2], np.int32)
    n2, tok2, par2, dep2, mask2 = oracle.tree_add_branches(tok, par, dep, mask, n, 4, br, ln)
    # branch 0 is cut at depth 4; branch 1 ends at its negative token; branch 2 is empty; branch 3 repeats the table's chain
    assert n2 == 10
    assert tok2[:n2].tolist() == [1, 2, 3, 7, 8, 9, 9, 5, 2, 3]
    assert par2[:n2].tolist() == [-1, 0, 1, 0, 3, 4, 5, 0, 0, 8]
    assert dep2[:n2].tolist() == [0, 1, 2, 1, 2, 3, 4, 1, 1, 2]
    assert mask2[6, 0] == 0b1111001 and mask2[7, 0] == 0b10000001 and mask2[9, 0] == 0b1100000001
    assert (tok2[n2:] == -1).all() and (mask2[n2:] == 0).all()
    assert np.array_equal(tok[:3], tok2[:3]) and tok[3] == -1             # inputs are not modified


def test_mask_is_the_ancestor_mask_and_caps_hold(oracle):
    rng = np.random.default_rng(2)
    cfg = W.get_config("c1_tiny")
    s = W.make_stream(cfg, 0, 600).tolist()
    t = oracle.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC)
    t.update(s, 0, 300)
    T = cfg.max_nodes
    for pos in range(300, 500, 9):
        n, tok, par, dep, mask = t.draft_tree(s, pos, T, cfg.crt, cfg.max_depth)
        K, Lm = int(rng.integers(0, 5)), 7
        br = rng.integers(0, 50, (K, Lm)).astype(np.int32)
        ln = rng.integers(0, Lm + 3, K).astype(np.int32)
        n2, tok2, par2, dep2, mask2 = oracle.tree_add_branches(tok, par, dep, mask, n, cfg.max_depth, br, ln)
        assert n <= n2 <= T and np.array_equal(tok2[:n], tok[:n]) and np.array_equal(par2[:n], par[:n])
        assert np.array_equal(mask2, oracle.tree_mask(par2, n2, T))
        assert n2 - n == min(T - n, sum(min(int(l), Lm, cfg.max_depth) for l in ln)) or n2 == T
        for i in range(n, n2):
            assert dep2[i] == dep2[par2[i]] + 1 <= cfg.max_depth and (par2[i] == 0 or par2[i] == i - 1)
        t.update(s, pos, pos + 9)
    n0, *_ = oracle.tree_add_branches(np.full(4, -1), np.full(4, -1), np.full(4, -1), np.zeros((4, 1)), 0, 4, [[1, 2]], [2])
    assert n0 == 0


def test_a_correct_draft_is_accepted_whole(oracle):
    n, tok, par, dep, mask = _tree(oracle, T=16, dmax=8)
    truth = [2, 3, 30, 31, 32, 33]                                        # what the target will say after the root
    n2, tok2, par2, dep2, mask2 = oracle.tree_add_branches(tok, par, dep, mask, n, 8, [truth[:5]], [5])
    target = np.full(16, 99, np.int32)
    for i in range(n2):                                                    # the target's choice after a node on the true path
        d = dep2[i]
        path = []
        c = i
        while c > 0:
            path.append(tok2[c]); c = par2[c]
        if path[::-1] == truth[:d]:
            target[i] = truth[d]
    m, nodes, out = oracle.accept(tok2, par2, dep2, n2, target, 8)
    assert m == 5 and out[:6].tolist() == truth
    m0, _, out0 = oracle.accept(tok, par, dep, n, target, 8)
    assert m0 == 2 and out0[:3].tolist() == truth[:3]                      # the table's own chain alone gets two tokens
