"""Pins for the oracle's draft-tree growth and tree mask (Section 3.2): the paper's Figure 2 example made
concrete and worked by hand, structural properties checked against an OrderedDict table model, and the
stop rule."""
import numpy as np
import pytest

from tests.conftest import golden
from tests.od_model import ODTable
import workloads as W


def _fresh(oracle, g):
    t = oracle.OracleTable(**g["params"])
    for L, F in g["inserts"]:
        t.insert(L, F)
    return t


@pytest.mark.parametrize("case", [0, 1, 2])
def test_figure2_trace(oracle, case):
    g = golden("trace_c_tree.json")
    c = g["cases"][case]
    t = _fresh(oracle, g)
    s = g["sequence"]
    n, tok, par, dep, mask, log = t.draft_tree(s, len(s), c["T"], c["crt"], c["max_depth"], with_log=True)
    assert n == c["n"]
    assert tok[:n].tolist() == c["tok"] and par[:n].tolist() == c["par"] and dep[:n].tolist() == c["dep"]
    assert mask[:n, 0].tolist() == c["mask"]
    assert (tok[n:] == -1).all() and (par[n:] == -1).all() and (dep[n:] == -1).all() and (mask[n:] == 0).all()
    assert log == [(tuple(k), h) for k, h in c["queries"]]
    assert [d[0] for d in t.dump()] == [tuple(k) for k in c["leader_order_after"]]


def test_first_level_is_the_papers_example(oracle):
    """'the fox' returns three followers; each becomes a branch below the root."""
    g = golden("trace_c_tree.json")
    t = _fresh(oracle, g)
    fs = t.query([12, 13])
    assert sorted(fs) == [(20, 21), (22, 23), (24, 25)]


def test_short_sequences(oracle):
    t = oracle.OracleTable(2, 2, 16, 2)
    t.insert([5, 6], [7, 8])
    n, tok, par, dep, mask = t.draft_tree([6], 1, 8, 0, 8)          # fewer than LL tokens: root only
    assert n == 1 and tok[0] == 6 and mask[0, 0] == 1
    assert t.clock == 1                                             # no query was issued
    n, tok, *_ = t.draft_tree([5, 6], 2, 8, 0, 8)
    assert n == 3 and tok[:3].tolist() == [6, 7, 8]
    n, *_ = t.draft_tree([], 0, 8, 0, 8)
    assert n == 0


def test_depth_cap_truncates_chains(oracle):
    t = oracle.OracleTable(1, 3, 16, 2)
    t.insert([1], [2, 3, 4])
    t.insert([4], [5, 6, 7])
    n, tok, par, dep, _ = t.draft_tree([1], 1, 16, 0, 5)
    assert tok[:n].tolist() == [1, 2, 3, 4, 5, 6] and dep[:n].tolist() == [0, 1, 2, 3, 4, 5]
    n, tok, par, dep, _ = t.draft_tree([1], 1, 16, 0, 2)
    assert tok[:n].tolist() == [1, 2, 3]                            # cut chain is never grown further


@pytest.mark.parametrize("name", ["c1_tiny", "c2_7b", "c4_13b_turns", "c1_evict256"])
def test_tree_properties_on_streams(oracle, name):
    cfg = W.get_config(name)
    n_tok = 1500
    s = W.make_stream(cfg, 0, n_tok).tolist()
    t = oracle.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC)
    m = ODTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC)
    pos = 300
    t.update(s, 0, pos)
    m.update(s, 0, pos)
    sizes = []
    while pos < n_tok - 20:
        n, tok, par, dep, mask, log = t.draft_tree(s, pos, cfg.max_nodes, cfg.crt, cfg.max_depth, with_log=True)
        T = cfg.max_nodes
        assert 1 <= n <= T and tok[0] == s[pos - 1] and par[0] == -1 and dep[0] == 0
        for i in range(1, n):
            assert 0 <= par[i] < i and dep[i] == dep[par[i]] + 1 <= cfg.max_depth
        # replay the logged queries on the model: same hit counts, and the tree is exactly the logged
        # followers laid out breadth first
        for key, hits in log:
            assert len(m.peek(key)) == hits
            m.query(key)
        assert t.dump() == m.dump()
        # stop rule: if the tree is not full, every complete leaf below the depth cap was queried and missed
        def key_of(i):
            out = []
            while i >= 0:
                out.append(int(tok[i])); i = par[i]
            full = s[:pos - 1] + out[::-1]
            return tuple(full[-cfg.LL:])
        if n < T:
            has_child = set(int(p) for p in par[1:n])
            for i in range(n):
                if i in has_child or dep[i] >= cfg.max_depth:
                    continue
                if dep[i] % cfg.FL != 0:
                    continue                                  # inside a cut chain: never queried
                assert m.peek(key_of(i)) == [], (i, key_of(i))
        # every child chain below node p is a stored follower of p's key, most recent first
        kids = {}
        for i in range(1, n):
            kids.setdefault(int(par[i]), []).append(i)
        for p, cs in kids.items():
            if dep[p] % cfg.FL != 0:
                assert len(cs) == 1                           # chain interior
                continue
            fol = m.peek(key_of(p))
            assert len(cs) <= len(fol)
            for rank, c in enumerate(cs):
                chain = [int(tok[c])]
                x = c
                while x in kids and dep[x] % cfg.FL != 0:
                    x = kids[x][0]
                    chain.append(int(tok[x]))
                assert tuple(chain) == fol[rank][:len(chain)]
        # level 1 (chains hanging off the root, depths 1..FL) leaves crt nodes for deeper levels
        assert sum(1 for i in range(1, n) if dep[i] <= cfg.FL) <= max(1, T - cfg.crt) - 1
        for i in range(n):                                    # mask = ancestors-or-self
            anc, c = set(), i
            while c >= 0:
                anc.add(c); c = int(par[c])
            assert {j for j in range(T) if (int(mask[i, j // 32]) >> (j % 32)) & 1} == anc
        sizes.append(n)
        step = 1 + (n % 5)
        t.update(s, pos, pos + step)
        m.update(s, pos, pos + step)
        pos += step
    assert max(sizes) > 1
