"""Pins for the oracle's frozen table (Section 3.3) and its offline builder (Section 4): a corpus counted by hand,
counts re-derived with vectorised window comparisons and numpy's bincount, a dual-table draft worked by hand, and the
special cases in which the dual draft must reduce to the single-table one."""
import numpy as np
import pytest

import workloads as W


# ------------------------------------------------------------------------------------------------ builder
def test_builder_hand_counted(oracle):
    # corpus: 1 2 3 1 2 4 1 2 3 5 ; LL = 1, FL = 2 -> windows at i = 0..7
    #   leader 1: (2,3) x2, (2,4) x1      count 3
    #   leader 2: (3,1), (4,1), (3,5)     count 3
    #   leader 3: (1,2) x1                count 1   (the 3 at i = 8 has only one token after it)
    #   leader 4: (1,2) x1                count 1
    corpus = [1, 2, 3, 1, 2, 4, 1, 2, 3, 5]
    L, nf, F = oracle.frozen_build(corpus, 1, 2, 3, 2)
    assert L.tolist() == [[1], [2], [3]]                      # 1 and 2 tie at 3: smaller token first; 3 beats 4 on a tie at 1
    assert nf.tolist() == [2, 2, 1]
    assert F[0].tolist() == [[2, 3], [2, 4]]
    assert F[1].tolist() == [[3, 1], [3, 5]]                  # three followers tie at 1: the two smallest stay
    assert F[2].tolist() == [[1, 2], [-1, -1]]
    L, nf, F = oracle.frozen_build(corpus, 2, 1, 8, 4)
    #   (1,2): 3,4,3 -> count 3; (2,3): 1,5 ; (3,1): 2 ; (2,4): 1 ; (4,1): 2
    assert L.tolist() == [[1, 2], [2, 3], [2, 4], [3, 1], [4, 1]]
    assert nf.tolist() == [2, 2, 1, 1, 1]
    assert F[0, :2].tolist() == [[3], [4]] and F[1, :2].tolist() == [[1], [5]]


def _count(c, key, at):
    """occurrences of key in c at the offsets `at` (vectorised comparison, no hashing)."""
    ok = np.ones(len(at), bool)
    for j, k in enumerate(key):
        ok &= c[at + j] == k
    return int(ok.sum())


@pytest.mark.parametrize("LL,FL,LC,FC,vocab", [(1, 3, 12, 4, 20), (2, 2, 40, 3, 6), (3, 1, 25, 5, 4)])
def test_builder_counts_and_order(oracle, LL, FL, LC, FC, vocab):
    rng = np.random.default_rng(5 + LL)
    c = (rng.zipf(1.6, 3000) % vocab).astype(np.int32)
    L, nf, F = oracle.frozen_build(c, LL, FL, LC, FC)
    at = np.arange(len(c) - LL - FL + 1)
    lcount = [_count(c, L[r], at) for r in range(len(L))]
    keys = [(-lcount[r], tuple(L[r])) for r in range(len(L))]
    assert keys == sorted(keys) and len(set(keys)) == len(keys)
    # nothing outside the table beats the last leader inside it
    seen = {tuple(c[i:i + LL]) for i in at}
    assert len(L) == min(LC, len(seen))
    inside = {tuple(x) for x in L.tolist()}
    for k in seen - inside:
        assert (-_count(c, k, at), k) > keys[-1]
    for r in range(len(L)):
        fk = [(-_count(c, list(L[r]) + list(F[r, k]), at), tuple(F[r, k])) for k in range(nf[r])]
        assert fk == sorted(fk) and len(set(fk)) == len(fk) and fk[0][0] < 0
        assert (F[r, nf[r]:] == -1).all()
        after = {tuple(c[i + LL:i + LL + FL]) for i in at if tuple(c[i:i + LL]) == tuple(L[r])}
        assert nf[r] == min(FC, len(after))
        for k in after - {tuple(x) for x in F[r, :nf[r]].tolist()}:
            assert (-_count(c, list(L[r]) + list(k), at), k) > fk[-1]
        assert sum(-x[0] for x in fk) <= lcount[r]


def test_builder_unigram_leaders_are_a_bincount(oracle):
    rng = np.random.default_rng(11)
    c = rng.integers(0, 50, 5000).astype(np.int32)
    FL = 2
    L, nf, F = oracle.frozen_build(c, 1, FL, 16, 1)
    cnt = np.bincount(c[: len(c) - FL], minlength=50)
    order = np.lexsort((np.arange(50), -cnt))[:16]
    assert L[:, 0].tolist() == order.tolist()


# ------------------------------------------------------------------------------------------------ dual-table draft
FROZEN = {(1,): [(4, 5), (2, 3)], (3,): [(6, 7)], (5,): [(8, 8)], (7,): [(1, 1)]}


def _frozen(oracle, d, LL, FL):
    keys = list(d.keys())
    FC = max(len(v) for v in d.values())
    L = np.array(keys, np.int32).reshape(len(keys), LL)
    nf = np.array([len(d[k]) for k in keys], np.int32)
    F = np.full((len(keys), FC, FL), -1, np.int32)
    for r, k in enumerate(keys):
        for j, f in enumerate(d[k]):
            F[r, j] = f
    return oracle.OracleFrozen(LL, FL, L, nf, F)


def test_dual_draft_by_hand(oracle):
    """dynamic: 1 -> (2,3).  Sequence ... 1.  The dynamic pass gives root 1 with the branch 2 3 and misses on 3; the frozen pass
    then walks root, node 2 and the ends it adds itself."""
    t = oracle.OracleTable(1, 2, 16, 4)
    t.insert([1], [2, 3])
    fz = _frozen(oracle, FROZEN, 1, 2)
    n, tok, par, dep, mask, log, flog = oracle.draft_tree_dual(t, fz, [9, 1], 2, 12, 0, 8, with_log=True)
    assert n == 12
    assert tok.tolist() == [1, 2, 3, 4, 5, 2, 3, 6, 7, 8, 8, 6]
    assert par.tolist() == [-1, 0, 1, 0, 3, 0, 5, 2, 7, 4, 9, 6]
    assert dep.tolist() == [0, 1, 2, 1, 2, 1, 2, 3, 4, 3, 4, 3]
    assert log == [((1,), 1), ((3,), 0)]
    assert flog == [((1,), 2), ((3,), 1), ((5,), 1), ((3,), 1)]
    assert mask[11, 0] == (1 << 11) | (1 << 6) | (1 << 5) | 1
    assert t.clock == 3                                        # one insert, two dynamic queries; frozen queries do not tick
    # the reserve for deeper levels also binds the frozen followers of the root: with crt = 9 the root may hold 3 nodes
    t = oracle.OracleTable(1, 2, 16, 4)
    t.insert([1], [2, 3])
    n, tok, par, dep, mask, log, flog = oracle.draft_tree_dual(t, fz, [9, 1], 2, 12, 9, 8, with_log=True)
    assert n == 11
    assert tok[:n].tolist() == [1, 2, 3, 6, 7, 1, 1, 4, 5, 2, 3]
    assert par[:n].tolist() == [-1, 0, 1, 2, 3, 4, 5, 6, 7, 6, 9]
    assert dep[:n].tolist() == [0, 1, 2, 3, 4, 5, 6, 7, 8, 7, 8]   # nodes at depth 8 = max_depth are not queried
    assert flog == [((3,), 1), ((7,), 1), ((1,), 2)]


@pytest.mark.parametrize("name", ["c1_tiny", "c2_7b"])
def test_without_frozen_table_it_is_the_single_table_draft(oracle, name):
    cfg = W.get_config(name)
    s = W.make_stream(cfg, 0, 900).tolist()
    a = oracle.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC)
    b = oracle.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC)
    a.update(s, 0, 400)
    b.update(s, 0, 400)
    for pos in range(400, 880, 7):
        ra = a.draft_tree(s, pos, cfg.max_nodes, cfg.crt, cfg.max_depth)
        rb = oracle.draft_tree_dual(b, None, s, pos, cfg.max_nodes, cfg.crt, cfg.max_depth)
        assert ra[0] == rb[0] and all(np.array_equal(x, y) for x, y in zip(ra[1:], rb[1:]))
        a.update(s, pos, pos + 7)
        b.update(s, pos, pos + 7)
    assert a.clock == b.clock and a.dump() == b.dump()


@pytest.mark.parametrize("crt", [0, 5, 14])
@pytest.mark.parametrize("LL,FL", [(1, 3), (2, 2)])
def test_only_frozen_equals_a_dynamic_table_with_the_same_content(oracle, LL, FL, crt):
    """With an empty dynamic table, the frozen pass alone builds the tree (the 'Only Frozen' row of Table 1).  A dynamic
    table that holds the same leaders, with the followers inserted least frequent first so that the most frequent is the
    most recent, must give the same tree through the ordinary single-table draft."""
    rng = np.random.default_rng(3)
    vocab = 12
    c = rng.integers(0, vocab, 4000).astype(np.int32)
    FC = 3
    L, nf, F = oracle.frozen_build(c, LL, FL, 256, FC)
    fz = oracle.OracleFrozen(LL, FL, L, nf, F)
    dyn = oracle.OracleTable(LL, FL, 256, FC)
    for r in range(len(L)):
        for k in reversed(range(nf[r])):
            dyn.insert(L[r], F[r, k])
    T, dmax = 24, 9
    grown = 0
    for trial in range(40):
        s = rng.integers(0, vocab, 6).tolist()
        empty = oracle.OracleTable(LL, FL, 256, FC)
        n2, tok2, par2, dep2, mask2, log2, flog2 = oracle.draft_tree_dual(empty, fz, s, len(s), T, crt, dmax, with_log=True)
        n1, tok1, par1, dep1, mask1, log1 = dyn.draft_tree(s, len(s), T, crt, dmax, with_log=True)
        assert n1 == n2 and np.array_equal(tok1, tok2) and np.array_equal(par1, par2) and np.array_equal(dep1, dep2)
        assert np.array_equal(mask1, mask2)
        assert flog2 == log1 and log2 == [(tuple(s[-LL:]), 0)]
        grown += n2 > 1
    assert grown > 20


def test_full_tree_leaves_nothing_to_the_frozen_table(oracle):
    t = oracle.OracleTable(1, 2, 16, 4)
    for f in ([2, 3], [4, 5], [6, 7]):
        t.insert([1], f)
    fz = _frozen(oracle, FROZEN, 1, 2)
    n, tok, par, dep, mask, log, flog = oracle.draft_tree_dual(t, fz, [1], 1, 7, 0, 8, with_log=True)
    assert n == 7 and flog == [] and tok.tolist() == [1, 6, 7, 4, 5, 2, 3]


def test_frozen_pass_leaves_the_dynamic_table_alone(oracle):
    cfg = W.get_config("c1_tiny")
    s = W.make_stream(cfg, 1, 700).tolist()
    L, nf, F = oracle.frozen_build(W.make_stream(cfg, 7, 3000), cfg.LL, cfg.FL, 256, cfg.FC)
    fz = oracle.OracleFrozen(cfg.LL, cfg.FL, L, nf, F)
    a = oracle.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC)
    b = oracle.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC)
    a.update(s, 0, 300)
    b.update(s, 0, 300)
    bigger = 0
    for pos in range(300, 690, 5):
        n1, tok1, par1, *_ = a.draft_tree(s, pos, cfg.max_nodes, cfg.crt, cfg.max_depth)
        n2, tok2, par2, dep2, mask2, log2, flog2 = oracle.draft_tree_dual(b, fz, s, pos, cfg.max_nodes, cfg.crt, cfg.max_depth, with_log=True)
        # the dynamic pass comes first, untouched: its tree is a prefix of the dual tree
        assert n2 >= n1 and np.array_equal(tok1[:n1], tok2[:n1]) and np.array_equal(par1[:n1], par2[:n1])
        for i in range(1, n2):
            assert 0 <= par2[i] < i and dep2[i] == dep2[par2[i]] + 1 <= cfg.max_depth
        bigger += n2 > n1
        a.update(s, pos, pos + 5)
        b.update(s, pos, pos + 5)
    assert a.clock == b.clock and a.dump() == b.dump()
    assert bigger > 5
