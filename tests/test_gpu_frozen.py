"""GPU parity: the dual-table draft (frozen table attached) against the oracle, bit-exact: a hand trace, cold-start
closed loops on the workloads' streams with a frozen table built from a separate synthetic corpus, the frozen-only
case, detaching, and the load / dump round trip of the frozen table's device image."""
import numpy as np
import pytest
import torch

import workloads as W
from tests.harness import Problem, dev
from tests.test_gpu_table import _assert_tables_equal, _stream_targets

pytestmark = pytest.mark.gpu


def _corpus(cfg, n_tok):
    """Synthetic stand-in for the paper's corpus sample: streams of the config's own token distribution, other seeds."""
    return np.concatenate([W.make_stream(cfg, 1000 + k, n_tok // 4) for k in range(4)]).astype(np.int32)


def _frozen_pair(oracle, LL, FL, LC, FC, arrays):
    from paper_2511_21699_b200 import FrozenTable
    L, nf, F = arrays
    ft = FrozenTable(LL, FL, LC, FC)
    ft.cb_frozen_load(L, nf, F)
    return ft, oracle.OracleFrozen(LL, FL, L, nf, F)


def test_load_dump_round_trip(oracle):
    cfg = W.get_config("c1_tiny")
    arrays = oracle.frozen_build(_corpus(cfg, 8000), cfg.LL, cfg.FL, 512, 6)
    ft, _ = _frozen_pair(oracle, cfg.LL, cfg.FL, 512, 6, arrays)
    L, nf, F = ft.cb_frozen_dump()
    assert np.array_equal(L, arrays[0]) and np.array_equal(nf, arrays[1]) and np.array_equal(F, arrays[2])
    assert len(L) > 50


def test_dual_draft_hand_trace_on_gpu(oracle):
    """The example worked by hand in the oracle's pins: dynamic 1 -> (2,3); frozen 1 -> (4,5),(2,3); 3 -> (6,7); ..."""
    from paper_2511_21699_b200 import Cacheback, FrozenTable
    cb = Cacheback(1, 1, 2, 16, 4, 12, 0, 8, 100, 1, 1, 64)
    s = dev(np.array([[1, 2, 3]], np.int32))
    cb.cb_update(s, dev(np.array([0], np.int32)), dev(np.array([3], np.int32)))
    ft = FrozenTable(1, 2, 8, 2)
    ft.cb_frozen_load([[1], [3], [5], [7]], [2, 1, 1, 1],
                      [[[4, 5], [2, 3]], [[6, 7], [-1, -1]], [[8, 8], [-1, -1]], [[1, 1], [-1, -1]]])
    cb.cb_frozen_attach(ft)
    tree = cb.cb_draft_tree(dev(np.array([[9, 1]], np.int32)), dev(np.array([2], np.int32)))
    assert int(tree["n_nodes"][0]) == 12
    assert tree["tokens"][0].cpu().tolist() == [1, 2, 3, 4, 5, 2, 3, 6, 7, 8, 8, 6]
    assert tree["parent"][0].cpu().tolist() == [-1, 0, 1, 0, 3, 0, 5, 2, 7, 4, 9, 6]
    assert tree["depth"][0].cpu().tolist() == [0, 1, 2, 1, 2, 1, 2, 3, 4, 3, 4, 3]
    assert int(tree["mask"][0, 11, 0]) == (1 << 11) | (1 << 6) | (1 << 5) | 1
    st, cnt = cb.cb_poll_status()
    assert st == 0 and cnt["queries"] == 2 and cnt["query_hits"] == 1 and cnt["frozen_queries"] == 4 and cnt["frozen_hits"] == 4
    cb.cb_frozen_attach(None)
    tree = cb.cb_draft_tree(dev(np.array([[9, 1]], np.int32)), dev(np.array([2], np.int32)))
    assert int(tree["n_nodes"][0]) == 3 and tree["tokens"][0, :3].cpu().tolist() == [1, 2, 3]


@pytest.mark.parametrize("name,steps,prompt,fLC,fFC", [("c1_tiny", 30, 8, 512, 8), ("c2_7b", 24, 48, 4096, 6),
                                                       ("c3_8b_gqa", 8, 32, 4096, 16), ("c4_13b_turns", 8, 64, 2048, 2),
                                                       ("c1_evict256", 20, 300, 1024, 4), ("p_tuned", 12, 64, 8192, 128),
                                                       ("p_fc40_evict", 12, 600, 2048, 70)])
def test_dual_draft_closed_loop(oracle, name, steps, prompt, fLC, fFC):
    """Cold start: a short prompt in the dynamic table, so that the frozen pass supplies much of each tree."""
    from paper_2511_21699_b200 import Cacheback
    cfg = W.get_config(name)
    prob = Problem(cfg)
    B, T = cfg.batch, cfg.max_nodes
    cb = Cacheback.from_config(cfg)
    ft, ofz = _frozen_pair(oracle, cfg.LL, cfg.FL, fLC, fFC, oracle.frozen_build(_corpus(cfg, 20000), cfg.LL, cfg.FL, fLC, fFC))
    cb.cb_frozen_attach(ft)
    otabs = [oracle.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC) for _ in range(B)]
    toks_d = dev(prob.toks)
    pos = np.full(B, prompt, np.int32)
    cb.cb_update(toks_d, torch.zeros(B, dtype=torch.int32, device="cuda"), dev(pos))
    for b in range(B):
        otabs[b].update(prob.toks[b], 0, int(pos[b]))
    tree, res = cb.alloc_tree(), cb.alloc_accept()
    fq = fh = grew = 0
    for step in range(steps):
        cb.cb_draft_tree(toks_d, dev(pos), tree)
        g = {k: v.cpu().numpy() for k, v in tree.items()}
        tgt = np.full((B, T), -1, np.int32)
        exp = []
        for b in range(B):
            n, tok, par, dep, mask, log, flog = oracle.draft_tree_dual(otabs[b], ofz, prob.toks[b], int(pos[b]), T, cfg.crt,
                                                                     cfg.max_depth, with_log=True)
            assert g["n_nodes"][b] == n, (step, b, g["n_nodes"][b], n)
            assert np.array_equal(g["tokens"][b], tok) and np.array_equal(g["parent"][b], par), (step, b)
            assert np.array_equal(g["depth"][b], dep), (step, b)
            assert np.array_equal(g["mask"][b].view(np.uint32), mask), (step, b)
            fq += len(flog)
            fh += sum(1 for _, h in flog if h > 0)
            grew += any(h > 0 for _, h in flog)
            tgt[b] = _stream_targets(prob.toks[b], int(pos[b]), n, tok, par, T, b, step)
            exp.append(oracle.accept(tok, par, dep, n, tgt[b], cfg.max_depth))
        cb.cb_accept(tree, target_ids=dev(tgt), res=res)
        r = {k: v.cpu().numpy() for k, v in res.items()}
        new_pos = pos.copy()
        for b in range(B):
            m, nodes, out = exp[b]
            assert r["n_accept"][b] == m and np.array_equal(r["out_tokens"][b], out), (step, b)
            new_pos[b] = min(pos[b] + m + 1, prob.lens[b] - T - 2)
        cb.cb_update(toks_d, dev(pos), dev(new_pos))
        for b in range(B):
            otabs[b].update(prob.toks[b], int(pos[b]), int(new_pos[b]))
        pos = new_pos
    _assert_tables_equal(cb, otabs, range(B) if B <= 8 else [0, 1, B // 2, B - 1])
    st, cnt = cb.cb_poll_status()
    assert st == 0, st
    assert cnt["frozen_queries"] == fq and cnt["frozen_hits"] == fh
    assert grew > 0


def test_only_frozen(oracle):
    """Empty dynamic tables: every tree comes from the frozen table alone (the 'Only Frozen' row of Table 1)."""
    from paper_2511_21699_b200 import Cacheback
    cfg = W.get_config("c1_tiny")
    prob = Problem(cfg)
    B, T = cfg.batch, cfg.max_nodes
    cb = Cacheback.from_config(cfg)
    ft, ofz = _frozen_pair(oracle, cfg.LL, cfg.FL, 512, 8, oracle.frozen_build(_corpus(cfg, 20000), cfg.LL, cfg.FL, 512, 8))
    cb.cb_frozen_attach(ft)
    toks_d = dev(prob.toks)
    sizes = []
    for pos0 in (5, 40, 90):
        pos = np.full(B, pos0, np.int32)
        tree = cb.cb_draft_tree(toks_d, dev(pos))
        g = {k: v.cpu().numpy() for k, v in tree.items()}
        for b in range(B):
            empty = oracle.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC)
            n, tok, par, dep, mask = oracle.draft_tree_dual(empty, ofz, prob.toks[b], pos0, T, cfg.crt, cfg.max_depth)
            assert g["n_nodes"][b] == n and np.array_equal(g["tokens"][b], tok) and np.array_equal(g["parent"][b], par)
            assert np.array_equal(g["mask"][b].view(np.uint32), mask)
            sizes.append(n)
        assert cb.cb_table_dump(0) == []
    assert max(sizes) > 1
    assert cb.cb_poll_status()[0] == 0


# ------------------------------------------------------------------------------------------------ builder on the GPU
def _build_and_compare(oracle, corpus, LL, FL, LC, FC):
    from paper_2511_21699_b200 import FrozenTable
    ft = FrozenTable(LL, FL, LC, FC)
    ft.cb_frozen_build(dev(np.asarray(corpus, np.int32)))
    L, nf, F = ft.cb_frozen_dump()
    oL, onf, oF = oracle.frozen_build(corpus, LL, FL, LC, FC)
    assert L.shape == oL.shape, (L.shape, oL.shape)
    assert np.array_equal(L, oL) and np.array_equal(nf, onf) and np.array_equal(F, oF)
    return ft, len(L)


@pytest.mark.parametrize("LL,FL,LC,FC,vocab,n", [(1, 3, 64, 4, 300, 20000),      # more distinct leaders than LC
                                                 (1, 3, 1024, 16, 300, 20000),   # all leaders fit; FC at its maximum
                                                 (2, 2, 500, 3, 12, 30000),      # tiny vocabulary: many equal counts
                                                 (3, 1, 777, 5, 6, 9000),
                                                 (4, 8, 2048, 2, 40, 15000),     # longest leader and follower
                                                 (2, 3, 16, 1, 1000, 5000),      # nearly every count is 1: ties decide
                                                 (1, 3, 4096, 128, 2000, 60000)])  # the paper's follower capacity
def test_builder_matches_the_oracle(oracle, LL, FL, LC, FC, vocab, n):
    rng = np.random.default_rng(LL * 100 + FL)
    corpus = (rng.zipf(1.3, n) % vocab).astype(np.int32)
    _, got = _build_and_compare(oracle, corpus, LL, FL, LC, FC)
    assert got > 0


def test_builder_on_the_workload_corpus_and_reuse(oracle):
    """The table the closed-loop tests load from the oracle's builder, built on the GPU instead; building twice into the
    same buffers gives the same table."""
    from paper_2511_21699_b200 import Cacheback
    cfg = W.get_config("c2_7b")
    corpus = _corpus(cfg, 60000)
    ft, n = _build_and_compare(oracle, corpus, cfg.LL, cfg.FL, 4096, 6)
    first = ft.cb_frozen_dump()
    ft.cb_frozen_build(dev(corpus))
    again = ft.cb_frozen_dump()
    assert all(np.array_equal(a, b) for a, b in zip(first, again))
    # the built table drives the draft like the loaded one
    ofz = oracle.OracleFrozen(cfg.LL, cfg.FL, *first)
    cb = Cacheback.from_config(cfg)
    cb.cb_frozen_attach(ft)
    prob = Problem(cfg)
    pos = np.full(cfg.batch, 40, np.int32)
    tree = cb.cb_draft_tree(dev(prob.toks), dev(pos))
    for b in range(cfg.batch):
        empty = oracle.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC)
        nn, tok, par, dep, mask = oracle.draft_tree_dual(empty, ofz, prob.toks[b], 40, cfg.max_nodes, cfg.crt, cfg.max_depth)
        assert int(tree["n_nodes"][b]) == nn and np.array_equal(tree["tokens"][b].cpu().numpy(), tok)


def test_builder_edge_cases(oracle):
    from paper_2511_21699_b200 import FrozenTable, CachebackError
    for corpus in ([], [5], [1, 2, 3], [1, 2, 3, 4], [7] * 50):
        _build_and_compare(oracle, np.array(corpus, np.int32), 1, 3, 8, 2)
    ft = FrozenTable(1, 2, 8, 2)
    with pytest.raises(CachebackError):
        ft.cb_frozen_build(dev(np.array([1, 2, -1, 3, 4, 5], np.int32)))     # negative ids are rejected
