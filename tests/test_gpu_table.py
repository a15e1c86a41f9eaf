"""GPU parity: cb_update, cb_draft_tree and cb_accept (ids form) against the oracle, bit-exact, including a
closed-loop replay in which the token stream itself plays the target model (losslessness)."""
import numpy as np
import pytest
import torch

import workloads as W
from tests.conftest import golden
from tests.harness import Problem, dev

pytestmark = pytest.mark.gpu


def _mk(cfg, flags=0):
    from paper_2511_21699_b200 import Cacheback
    return Cacheback.from_config(cfg, flags=flags)


def _assert_tables_equal(cb, otabs, seqs):
    for b in seqs:
        gl, gn, gf = cb.cb_table_dump_arrays(b)
        ol, on, of = otabs[b].dump_arrays()
        assert gl.shape == ol.shape, (b, gl.shape, ol.shape)
        assert np.array_equal(gl, ol), b
        assert np.array_equal(gn, on), b
        assert np.array_equal(gf, of), b


def _stream_targets(s, pos, n, tok, par, T, b, step):
    """Mode-B target: the stream continuation along matching paths, junk elsewhere."""
    tgt = np.full(T, -1, np.int32)
    on_path = np.zeros(T, bool)
    on_path[0] = True
    for i in range(n):
        if i > 0:
            p = par[i]
            d = 0
            c = i
            while c > 0:
                d += 1; c = par[c]
            on_path[i] = on_path[p] and tok[i] == s[pos - 1 + d]
        if on_path[i]:
            d = 0
            c = i
            while c > 0:
                d += 1; c = par[c]
            tgt[i] = s[pos + d]
        else:
            tgt[i] = int(W.mix64(7, 300 + step, b * 1024 + i) % np.uint64(1000)) + 200000
    return tgt


@pytest.mark.parametrize("name,steps", [("c1_tiny", 24), ("c2_7b", 24), ("c3_8b_gqa", 10), ("c4_13b_turns", 10),
                                        ("c5_70b_long", 4), ("c1_evict256", 24), ("c1_evict1024", 12),
                                        ("c3_evict256", 10), ("c3_evict1024", 10), ("p_tuned", 16),
                                        ("p_fc40_evict", 16)])
def test_update_draft_accept_closed_loop(oracle, name, steps):
    cfg = W.get_config(name)
    prob = Problem(cfg)
    B, T = cfg.batch, cfg.max_nodes
    cb = _mk(cfg)
    otabs = [oracle.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC) for _ in range(B)]
    toks_d = dev(prob.toks)
    zero = torch.zeros(B, dtype=torch.int32, device="cuda")
    pos = prob.prefill.copy()
    if "evict" in name:                          # long prompts, so that the shrunk tables overflow
        pos = (prob.lens - T - 2 - 8 * steps).astype(np.int32)
    # prompt initialisation (Section 3.3): one bulk update from an empty table
    cb.cb_update(toks_d, zero, dev(pos))
    for b in range(B):
        otabs[b].update(prob.toks[b], 0, int(pos[b]))
    check = range(B) if B <= 8 else [0, 1, B // 2, B - 1]
    _assert_tables_equal(cb, otabs, check)
    tree = cb.alloc_tree()
    res = cb.alloc_accept()
    total_accept = 0
    for step in range(steps):
        cb.cb_draft_tree(toks_d, dev(pos), tree)
        g = {k: v.cpu().numpy() for k, v in tree.items()}
        tgt = np.full((B, T), -1, np.int32)
        exp = []
        for b in range(B):
            n, tok, par, dep, mask = otabs[b].draft_tree(prob.toks[b], int(pos[b]), T, cfg.crt, cfg.max_depth)
            assert g["n_nodes"][b] == n, (step, b)
            assert np.array_equal(g["tokens"][b], tok) and np.array_equal(g["parent"][b], par), (step, b)
            assert np.array_equal(g["depth"][b], dep), (step, b)
            assert np.array_equal(g["mask"][b].view(np.uint32), mask), (step, b)
            tgt[b] = _stream_targets(prob.toks[b], int(pos[b]), n, tok, par, T, b, step)
            exp.append(oracle.accept(tok, par, dep, n, tgt[b], cfg.max_depth))
        cb.cb_accept(tree, target_ids=dev(tgt), res=res)
        r = {k: v.cpu().numpy() for k, v in res.items()}
        new_pos = pos.copy()
        for b in range(B):
            m, nodes, out = exp[b]
            assert r["n_accept"][b] == m and np.array_equal(r["accept_nodes"][b], nodes), (step, b)
            assert np.array_equal(r["out_tokens"][b], out), (step, b)
            # losslessness: the emitted tokens are the stream's own continuation
            assert np.array_equal(out[:m + 1], prob.toks[b, pos[b]:pos[b] + m + 1]), (step, b)
            new_pos[b] = min(pos[b] + m + 1, prob.lens[b] - T - 2)
            total_accept += m
        cb.cb_update(toks_d, dev(pos), dev(new_pos))
        for b in range(B):
            otabs[b].update(prob.toks[b], int(pos[b]), int(new_pos[b]))
        pos = new_pos
    _assert_tables_equal(cb, otabs, check)
    st, cnt = cb.cb_poll_status()
    assert st == 0, st
    assert cnt["inserts"] > 0 and cnt["queries"] > 0
    if "evict" in name:
        assert cnt["leader_evictions"] > 0
    if name.startswith("p_"):
        assert cnt["follower_evictions"] > 0     # hot unigram leaders overflow even 128 followers
    if name in ("c1_tiny", "c3_8b_gqa", "c4_13b_turns", "c5_70b_long"):
        assert total_accept > 0                  # the drafter does get tokens accepted on these streams


@pytest.mark.parametrize("name,steps", [("c1_tiny", 16), ("c2_7b", 16), ("c3_8b_gqa", 6), ("c1_evict256", 16),
                                        ("p_tuned", 10), ("p_fc40_evict", 10)])
def test_update_draft_in_one_launch(oracle, name, steps):
    """cb_update_draft_tree = cb_update then cb_draft_tree: same trees every step and the same table at the end as the
    oracle's update followed by its draft."""
    cfg = W.get_config(name)
    prob = Problem(cfg)
    B, T = cfg.batch, cfg.max_nodes
    cb = _mk(cfg)
    otabs = [oracle.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC) for _ in range(B)]
    toks_d = dev(prob.toks)
    zero = torch.zeros(B, dtype=torch.int32, device="cuda")
    pos = prob.prefill.copy()
    if "evict" in name:
        pos = (prob.lens - T - 2 - 8 * steps).astype(np.int32)
    cb.cb_update(toks_d, zero, dev(pos))
    for b in range(B):
        otabs[b].update(prob.toks[b], 0, int(pos[b]))
    prev = pos.copy()
    tree = cb.alloc_tree()
    for step in range(steps):
        cb.cb_update_draft_tree(toks_d, dev(prev), dev(pos), tree)
        g = {k: v.cpu().numpy() for k, v in tree.items()}
        new_pos = pos.copy()
        for b in range(B):
            otabs[b].update(prob.toks[b], int(prev[b]), int(pos[b]))
            n, tok, par, dep, mask = otabs[b].draft_tree(prob.toks[b], int(pos[b]), T, cfg.crt, cfg.max_depth)
            assert g["n_nodes"][b] == n, (step, b)
            assert np.array_equal(g["tokens"][b], tok) and np.array_equal(g["parent"][b], par), (step, b)
            assert np.array_equal(g["depth"][b], dep), (step, b)
            assert np.array_equal(g["mask"][b].view(np.uint32), mask), (step, b)
            # the stream is the target: accept the matching path, plus the bonus token
            m = oracle.accept(tok, par, dep, n, _stream_targets(prob.toks[b], int(pos[b]), n, tok, par, T, b, step), cfg.max_depth)[0]
            new_pos[b] = min(pos[b] + m + 1 + (step % 3), prob.lens[b] - T - 2)
        prev, pos = pos, new_pos
    check = range(B) if B <= 8 else [0, 1, B // 2, B - 1]
    _assert_tables_equal(cb, otabs, check)
    st, cnt = cb.cb_poll_status()
    assert st == 0, st
    assert cnt["inserts"] > 0 and cnt["queries"] > 0


@pytest.mark.parametrize("fixture", ["trace_a_lru.json", "trace_b_follower_refresh.json"])
def test_hand_traces_on_gpu(fixture):
    g = golden(fixture)
    ids = g["ids"]
    p = g["params"]
    from paper_2511_21699_b200 import Cacheback
    cb = Cacheback(1, p["LL"], p["FL"], p["LC"], p["FC"], 4, 0, 1, 100, 1, 1, 64)   # depth cap 1: one query per call
    # inserts are fed as two-token streams; queries as one-node draft calls
    for k, step in enumerate(g["steps"]):
        L = ids[step["leader"]]
        if step["op"] == "ins":
            s = dev(np.array([[L, ids[step["follower"]]]], np.int32))
            cb.cb_update(s, dev(np.array([0], np.int32)), dev(np.array([2], np.int32)))
        else:
            s = dev(np.array([[L]], np.int32))
            tree = cb.cb_draft_tree(s, dev(np.array([1], np.int32)))
            n = int(tree["n_nodes"][0])
            got = tree["tokens"][0, 1:n].cpu().tolist()
            assert got == [ids[f] for f in step["returns"]][: len(got)] and len(got) == min(3, len(step["returns"]))
        want = [((ids[l],), [(ids[f],) for f in fs]) for l, fs in step["state"]]
        assert cb.cb_table_dump(0) == want, (fixture, k)


def test_figure2_tree_on_gpu():
    g = golden("trace_c_tree.json")
    p = g["params"]
    from paper_2511_21699_b200 import Cacheback
    for c in g["cases"]:
        cb = Cacheback(1, p["LL"], p["FL"], p["LC"], p["FC"], c["T"], c["crt"], c["max_depth"], 100, 1, 1, 64)
        for L, F in g["inserts"]:
            s = dev(np.array([L + F], np.int32))
            cb.cb_update(s, dev(np.array([0], np.int32)), dev(np.array([4], np.int32)))
        s = dev(np.array([g["sequence"]], np.int32))
        tree = cb.cb_draft_tree(s, dev(np.array([4], np.int32)))
        n = int(tree["n_nodes"][0])
        assert n == c["n"]
        assert tree["tokens"][0, :n].cpu().tolist() == c["tok"]
        assert tree["parent"][0, :n].cpu().tolist() == c["par"]
        assert tree["depth"][0, :n].cpu().tolist() == c["dep"]
        assert tree["mask"][0, :n, 0].cpu().tolist() == c["mask"]
        assert [d[0] for d in cb.cb_table_dump(0)] == [tuple(k) for k in c["leader_order_after"]]


def test_no_refresh_flag_and_reset_and_load(oracle):
    from paper_2511_21699_b200 import Cacheback, _lib
    cfg = W.get_config("c1_tiny")
    s = W.make_stream(cfg, 0, 700)
    cb = Cacheback(2, cfg.LL, cfg.FL, 64, 2, 8, 0, 4, 100, 1, 1, 64, flags=_lib.CB_FLAG_NO_FOLLOWER_REFRESH)
    ot = oracle.OracleTable(cfg.LL, cfg.FL, 64, 2, refresh_on_reinsert=False)
    ot.update(s, 0, 700)
    toks = dev(np.stack([s, s[::-1]]))
    cb.cb_update(toks, dev(np.array([0, 0], np.int32)), dev(np.array([700, 300], np.int32)))
    assert cb.cb_table_dump(0) == ot.dump()
    assert len(cb.cb_table_dump(1)) > 0
    # reset only sequence 1
    cb.cb_reset(dev(np.array([0, 1], np.int32)))
    assert cb.cb_table_dump(0) == ot.dump() and cb.cb_table_dump(1) == []
    # load sequence 0's table into sequence 1: same canonical content, and it keeps working
    cb.cb_table_load(1, ot.dump())
    assert cb.cb_table_dump(1) == ot.dump()
    extra = np.concatenate([s[:10], s[300:320]]).astype(np.int32)
    ot.update(extra, 0, 30)
    cb.cb_update(dev(np.stack([extra, extra])), dev(np.array([0, 0], np.int32)), dev(np.array([30, 30], np.int32)))
    assert cb.cb_table_dump(1) == ot.dump() and cb.cb_table_dump(0) == ot.dump()
    cb.cb_reset()
    assert cb.cb_table_dump(0) == [] and cb.cb_table_dump(1) == []
    assert cb.cb_poll_status()[0] == 0


def test_argument_errors():
    from paper_2511_21699_b200 import Cacheback, CachebackError
    with pytest.raises(CachebackError):
        Cacheback(1, 9, 2, 16, 2, 8, 0, 4, 100, 1, 1, 64)           # LL too large
    with pytest.raises(CachebackError):
        Cacheback(1, 2, 2, 16, 2, 8, 0, 4, 100, 3, 2, 64)           # heads do not divide
    cb = Cacheback(1, 2, 2, 16, 2, 8, 0, 4, 100, 1, 1, 64)
    tree = cb.alloc_tree()
    with pytest.raises(CachebackError):
        cb.cb_accept(tree)                                          # neither logits nor ids
