"""GPU parity: cb_tree_add_branches against the oracle, bit-exact, in a closed loop in which a second drafter supplies
branches (for some sequences the stream's true continuation, for others noise, of varying lengths); acceptance then has to
take the true branch, and tree attention over the extended tree stays within tolerance of the oracle."""
import numpy as np
import pytest
import torch

import workloads as W
from tests.harness import Problem, dev, device_attn_inputs, oracle_attn_rows, bf16_to_f64
from tests.test_gpu_attn import _check_rows
from tests.test_gpu_table import _stream_targets

pytestmark = pytest.mark.gpu


def _other_drafter(prob, pos, B, K, Lmax, step):
    """K branches per sequence: branch b % K of every other sequence is the stream's continuation; the rest is noise with an
    occasional negative token.  Lengths 0 .. Lmax + 1 (one beyond the row)."""
    rng = np.random.default_rng(100 + step)
    br = rng.integers(0, 30000, (B, K, Lmax)).astype(np.int32)
    ln = rng.integers(0, Lmax + 2, (B, K)).astype(np.int32)
    br[rng.random((B, K, Lmax)) < 0.03] = -1
    good = np.zeros(B, np.int32)
    for b in range(0, B, 2):
        k = b % K
        br[b, k] = prob.toks[b, pos[b]:pos[b] + Lmax]
        ln[b, k] = Lmax
        good[b] = 1
    return br, ln, good


@pytest.mark.parametrize("name,steps,K,Lmax", [("c1_tiny", 16, 3, 6), ("c3_8b_gqa", 6, 5, 9), ("c4_13b_turns", 6, 64, 4),
                                               ("p_tuned", 4, 2, 30)])
def test_branches_closed_loop(oracle, name, steps, K, Lmax):
    from paper_2511_21699_b200 import Cacheback
    cfg = W.get_config(name)
    prob = Problem(cfg)
    B, T = cfg.batch, cfg.max_nodes
    cb = Cacheback.from_config(cfg)
    otabs = [oracle.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC) for _ in range(B)]
    toks_d = dev(prob.toks)
    pos = np.full(B, 40, np.int32)                        # short prompt: the table alone drafts little
    cb.cb_update(toks_d, torch.zeros(B, dtype=torch.int32, device="cuda"), dev(pos))
    for b in range(B):
        otabs[b].update(prob.toks[b], 0, 40)
    tree, res = cb.alloc_tree(), cb.alloc_accept()
    added = 0
    for step in range(steps):
        br, ln, good = _other_drafter(prob, pos, B, K, Lmax, step)
        cb.cb_draft_tree(toks_d, dev(pos), tree)
        n_before = tree["n_nodes"].cpu().numpy().copy()
        cb.cb_tree_add_branches(tree, dev(br), dev(ln))
        g = {k: v.cpu().numpy() for k, v in tree.items()}
        tgt = np.full((B, T), -1, np.int32)
        exp = []
        for b in range(B):
            n, tok, par, dep, mask = otabs[b].draft_tree(prob.toks[b], int(pos[b]), T, cfg.crt, cfg.max_depth)
            assert n_before[b] == n
            n, tok, par, dep, mask = oracle.tree_add_branches(tok, par, dep, mask, n, cfg.max_depth, br[b], ln[b])
            assert g["n_nodes"][b] == n, (step, b, g["n_nodes"][b], n)
            assert np.array_equal(g["tokens"][b], tok) and np.array_equal(g["parent"][b], par), (step, b)
            assert np.array_equal(g["depth"][b], dep) and np.array_equal(g["mask"][b].view(np.uint32), mask), (step, b)
            added += n - n_before[b]
            tgt[b] = _stream_targets(prob.toks[b], int(pos[b]), n, tok, par, T, b, step)
            exp.append(oracle.accept(tok, par, dep, n, tgt[b], cfg.max_depth))
        cb.cb_accept(tree, target_ids=dev(tgt), res=res)
        r = {k: v.cpu().numpy() for k, v in res.items()}
        new_pos = pos.copy()
        for b in range(B):
            m, nodes, out = exp[b]
            assert r["n_accept"][b] == m and np.array_equal(r["out_tokens"][b], out), (step, b)
            assert np.array_equal(out[:m + 1], prob.toks[b, pos[b]:pos[b] + m + 1]), (step, b)
            room = T - n_before[b]
            if good[b] and room > 0:                          # the true branch is taken as far as it fitted
                assert m >= min(Lmax, cfg.max_depth, room - sum(min(max(int(l), 0), Lmax, cfg.max_depth) for l in ln[b, :b % K])), (step, b)
            new_pos[b] = min(pos[b] + m + 1, prob.lens[b] - T - 2)
        cb.cb_update(toks_d, dev(pos), dev(new_pos))
        for b in range(B):
            otabs[b].update(prob.toks[b], int(pos[b]), int(new_pos[b]))
        pos = new_pos
    assert cb.cb_poll_status()[0] == 0
    assert added > 0 or name == "p_tuned"


def test_attention_over_an_extended_tree(oracle):
    from paper_2511_21699_b200 import Cacheback
    cfg = W.get_config("c1_tiny")
    prob = Problem(cfg)
    B, T = cfg.batch, cfg.max_nodes
    cb = Cacheback.from_config(cfg)
    pos = np.full(B, 60, np.int32)
    cb.cb_update(dev(prob.toks), torch.zeros(B, dtype=torch.int32, device="cuda"), dev(pos))
    tree = cb.cb_draft_tree(dev(prob.toks), dev(pos))
    br = np.arange(B * 2 * 5, dtype=np.int32).reshape(B, 2, 5)
    cb.cb_tree_add_branches(tree, dev(br), dev(np.array([[5, 3]] * B, np.int32)))
    n = tree["n_nodes"].cpu().numpy()
    mask = tree["mask"].cpu().numpy().view(np.uint32)
    assert np.array_equal(mask[0], oracle.tree_mask(tree["parent"][0].cpu().numpy(), int(n[0]), T))
    d = device_attn_inputs(cfg, prob)
    lse = torch.zeros((B, cfg.n_q_heads, T), dtype=torch.float32, device="cuda")
    out = cb.cb_tree_attn(d["q"], d["k_pool"], d["v_pool"], d["block_table"], d["ctx_len"], d["k_tree"], d["v_tree"],
                          tree["mask"], tree["n_nodes"], lse=lse)
    rows = [(h, i) for h in range(cfg.n_q_heads) for i in range(int(n[0]))]
    ref, ref_lse = oracle_attn_rows(oracle, cfg, prob, mask, 0, rows)
    hh = torch.tensor([r[0] for r in rows], device="cuda")
    ii = torch.tensor([r[1] for r in rows], device="cuda")
    _check_rows(bf16_to_f64(out[0, ii, hh]), lse[0, hh, ii].cpu().numpy().astype(np.float64), ref, ref_lse, "extended")
    assert n[0] >= 9


def test_argument_checks():
    from paper_2511_21699_b200 import Cacheback, CachebackError
    cfg = W.get_config("c1_tiny")
    cb = Cacheback.from_config(cfg)
    tree = cb.alloc_tree()
    with pytest.raises(CachebackError):
        cb.cb_tree_add_branches(tree, torch.zeros((1, 65, 2), dtype=torch.int32, device="cuda"),
                                torch.zeros((1, 65), dtype=torch.int32, device="cuda"))
