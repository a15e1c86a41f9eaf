"""GPU parity: cb_accept_update_draft_tree (one step's acceptance, the emitted tokens appended to the history, the next
step's update and draft, in one launch) against the oracle's sequence of the same calls, in a generation loop: the logits
decide what is emitted: for every node whose path follows the synthetic stream the stream's next token is planted as the row's
maximum (the stream plays the target model), every other row keeps the arg-max of its random logits."""
import numpy as np
import pytest
import torch

import workloads as W
from workloads import device as wdev
from workloads.tensors import TID
from tests.harness import Problem, dev
from tests.test_gpu_table import _assert_tables_equal, _stream_targets

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,dtype,steps", [("c1_tiny", "f32", 8), ("c1_tiny", "bf16", 8), ("c2_7b", "f32", 6), ("c4_13b_turns", "f32", 4),
                                              ("p_tuned", "f32", 5)])
def test_accept_update_draft_in_one_launch(oracle, name, dtype, steps):
    from paper_2511_21699_b200 import Cacheback
    cfg = W.get_config(name)
    prob = Problem(cfg)
    B, T, V = cfg.batch, cfg.max_nodes, cfg.vocab
    cb = Cacheback.from_config(cfg)
    check = list(range(B)) if B <= 8 else [0, 1, B // 2, B - 1]
    otabs = {b: oracle.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC) for b in check}
    hist = prob.toks.copy()                                   # the host copy of every checked sequence's history
    toks_d = dev(prob.toks)
    pos = prob.prefill.copy().astype(np.int32)
    zero = torch.zeros(B, dtype=torch.int32, device="cuda")
    seq_len = dev(pos)
    cb.cb_update_bulk(toks_d, zero, seq_len)
    tree = cb.alloc_tree()
    cb.cb_draft_tree(toks_d, seq_len, tree)
    otree = {}
    for b in check:
        otabs[b].update(hist[b], 0, int(pos[b]))
        otree[b] = otabs[b].draft_tree(hist[b], int(pos[b]), T, cfg.crt, cfg.max_depth)
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    logits = wdev.normal_tensor((B, T, V), tdt, cfg.seed, TID.LOGITS)
    res = cb.alloc_accept()
    emitted = 0
    for step in range(steps):
        g = {k: v.cpu().numpy() for k, v in tree.items()}
        for b in check:
            n, tok, par, dep, mask = otree[b]
            assert g["n_nodes"][b] == n and np.array_equal(g["tokens"][b], tok) and np.array_equal(g["parent"][b], par), (step, b)
            assert np.array_equal(g["depth"][b], dep) and np.array_equal(g["mask"][b].view(np.uint32), mask), (step, b)
        # plant matches in the device logits for every sequence (restored after the call)
        plants = {}
        for b in range(B):
            nb = int(g["n_nodes"][b])
            st_t = _stream_targets(prob.toks[b], int(pos[b]), nb, g["tokens"][b], g["parent"][b], T, b, step)
            plants[b] = [(i, int(st_t[i])) for i in range(nb) if 0 <= st_t[i] < min(V, 200000)]
        idx = [(b, node, vid) for b in range(B) for node, vid in plants[b]]
        if idx:
            ib, inode, iv = (torch.tensor([t[k] for t in idx], device="cuda") for k in range(3))
            saved = logits[ib, inode, iv].clone()
            logits[ib, inode, iv] = 32.0
        cb.cb_accept_update_draft_tree(tree, logits, toks_d, seq_len, res=res)
        torch.cuda.synchronize()
        if idx:
            logits[ib, inode, iv] = saved
        r = {k: v.cpu().numpy() for k, v in res.items()}
        new_len = seq_len.cpu().numpy()
        toks_h = toks_d.cpu().numpy()
        for b in check:
            n, tok, par, dep, mask = otree[b]
            rows = W.logits_rows(cfg, b, np.arange(n), dtype)
            for node, vid in plants[b]:
                rows[node, vid] = 32.0
            tgt = np.full(T, -1, np.int32)
            tgt[:n] = oracle.argmax_rows(rows)
            m, nodes, out = oracle.accept(tok, par, dep, n, tgt, cfg.max_depth)
            assert r["n_accept"][b] == m and np.array_equal(r["accept_nodes"][b], nodes) and np.array_equal(r["out_tokens"][b], out), (step, b)
            assert np.array_equal(r["target_ids"][b], tgt), (step, b)
            old = int(pos[b])
            hist[b, old:old + m + 1] = out[:m + 1]
            assert new_len[b] == old + m + 1, (step, b)
            assert np.array_equal(toks_h[b, :old + m + 1], hist[b, :old + m + 1]), (step, b)
            otabs[b].update(hist[b], old, old + m + 1)
            otree[b] = otabs[b].draft_tree(hist[b], old + m + 1, T, cfg.crt, cfg.max_depth)
            emitted += m + 1
        pos = new_len.copy()
    g = {k: v.cpu().numpy() for k, v in tree.items()}
    for b in check:
        n, tok, par, dep, mask = otree[b]
        assert g["n_nodes"][b] == n and np.array_equal(g["tokens"][b], tok) and np.array_equal(g["parent"][b], par), ("last", b)
    _assert_tables_equal(cb, otabs, check)
    assert cb.cb_poll_status()[0] == 0
    assert emitted >= steps * len(check)
    if name in ("c1_tiny", "p_tuned"):
        assert emitted > steps * len(check)                   # draft tokens were accepted, not only bonus tokens


def test_fused_step_without_room_in_the_history(oracle):
    """A history that cannot take the emitted tokens: nothing is appended, the length stays, the status says so, and the next
    tree is the draft of the unchanged sequence."""
    from paper_2511_21699_b200 import Cacheback, _lib
    cfg = W.get_config("c1_tiny")
    prob = Problem(cfg)
    B, T, V = cfg.batch, cfg.max_nodes, cfg.vocab
    cb = Cacheback.from_config(cfg)
    L = 200
    toks_d = dev(prob.toks[:, :L].copy())                     # row stride = L: full
    seq_len = torch.full((B,), L, dtype=torch.int32, device="cuda")
    zero = torch.zeros(B, dtype=torch.int32, device="cuda")
    cb.cb_update(toks_d, zero, seq_len)
    tree, ref = cb.alloc_tree(), cb.alloc_tree()
    cb.cb_draft_tree(toks_d, seq_len, tree)
    logits = wdev.normal_tensor((B, T, V), torch.float32, cfg.seed, TID.LOGITS)
    cb.cb_accept_update_draft_tree(tree, logits, toks_d, seq_len, next_tree=ref)
    torch.cuda.synchronize()
    st, _ = cb.cb_poll_status()
    assert st == _lib.CB_ERR_INVALID_ARG
    assert (seq_len.cpu().numpy() == L).all()
    assert np.array_equal(toks_d.cpu().numpy(), prob.toks[:, :L])
    again = cb.alloc_tree()
    cb.cb_draft_tree(toks_d, seq_len, again)
    for k in ("tokens", "parent", "depth", "n_nodes"):
        assert torch.equal(ref[k], again[k]), k
