"""GPU parity: cb_kv_commit against the oracle, bit-exact (pools and context lengths), then tree attention over the
grown cache against the attention oracle (the committed rows must be where the next step looks for them)."""
import numpy as np
import pytest
import torch

import workloads as W
from tests.harness import Problem, dev, device_attn_inputs, synthetic_trees, bf16_to_f64

pytestmark = pytest.mark.gpu


def _u16(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def _accepted_paths(cfg, par, dep, n, rng):
    B, Dm = cfg.batch, cfg.max_depth
    n_acc = np.zeros(B, np.int32)
    nodes = np.full((B, Dm), -1, np.int32)
    for b in range(B):
        x = int(rng.integers(0, n[b]))
        path = []
        while x > 0:
            path.append(x); x = int(par[b, x])
        path = path[::-1]
        n_acc[b] = len(path)
        nodes[b, : len(path)] = path
    return n_acc, nodes


@pytest.mark.parametrize("name", ["c1_tiny", "c3_8b_gqa"])
def test_kv_commit_matches_oracle_and_feeds_attention(oracle, name):
    from paper_2511_21699_b200 import Cacheback
    cfg = W.get_config(name)
    prob = Problem(cfg)
    B, T, P = cfg.batch, cfg.max_nodes, cfg.page_size
    # leave room in every sequence's last page(s): shorten the contexts a little, keep the block table
    ctx = np.maximum(prob.ctx - (cfg.max_depth + 2), 0).astype(np.int32)
    par, dep, mask, n = synthetic_trees(cfg, full=False)
    n_acc, nodes = _accepted_paths(cfg, par, dep, n, np.random.default_rng(3))
    d = device_attn_inputs(cfg, prob)
    cb = Cacheback.from_config(cfg)
    ctx_d = dev(ctx)
    # oracle on host copies
    kp_h, vp_h = _u16(d["k_pool"]).copy(), _u16(d["v_pool"]).copy()
    want_ctx = oracle.kv_commit(kp_h, vp_h, prob.bt, ctx, _u16(d["k_tree"]), _u16(d["v_tree"]), n_acc, nodes)
    cb.cb_kv_commit(d["k_pool"], d["v_pool"], d["block_table"], ctx_d, d["k_tree"], d["v_tree"], dev(n_acc), dev(nodes))
    torch.cuda.synchronize()
    assert cb.cb_poll_status()[0] == 0
    assert np.array_equal(ctx_d.cpu().numpy(), want_ctx) and np.array_equal(want_ctx, ctx + n_acc + 1)
    assert np.array_equal(_u16(d["k_pool"]), kp_h) and np.array_equal(_u16(d["v_pool"]), vp_h)
    # a second commit right after (ticket scratch must be clean): commit only the root of each sequence
    zero = np.zeros(B, np.int32)
    want_ctx2 = oracle.kv_commit(kp_h, vp_h, prob.bt, want_ctx, _u16(d["k_tree"]), _u16(d["v_tree"]), zero, nodes)
    cb.cb_kv_commit(d["k_pool"], d["v_pool"], d["block_table"], ctx_d, d["k_tree"], d["v_tree"], dev(zero), dev(nodes))
    torch.cuda.synchronize()
    assert np.array_equal(ctx_d.cpu().numpy(), want_ctx2)
    assert np.array_equal(_u16(d["k_pool"]), kp_h) and np.array_equal(_u16(d["v_pool"]), vp_h)
    # attention over the grown cache agrees with the oracle on the same (committed) inputs
    out = cb.cb_tree_attn(d["q"], d["k_pool"], d["v_pool"], d["block_table"], ctx_d, d["k_tree"], d["v_tree"], dev(mask.view(np.int32)), dev(n))
    torch.cuda.synchronize()
    for b in sorted({0, B - 1}):
        rows = np.array([(b, h, i) for h in (0, cfg.n_q_heads - 1) for i in (0, int(n[b]) - 1)], np.int32)
        npg = (int(want_ctx2[b]) + P - 1) // P
        ref, _ = oracle.tree_attn_rows(_u16(d["q"]), kp_h, vp_h, prob.bt, want_ctx2, _u16(d["k_tree"]), _u16(d["v_tree"]), mask, rows)
        got = bf16_to_f64(out[b, torch.tensor(rows[:, 2]).cuda(), torch.tensor(rows[:, 1]).cuda()])
        assert (np.abs(got - ref) <= 2e-2 + 1e-2 * np.abs(ref)).all(), (name, b)


def test_kv_commit_full_cache_reports_and_skips(oracle):
    from paper_2511_21699_b200 import Cacheback, _lib
    cfg = W.get_config("c1_tiny")
    prob = Problem(cfg)
    d = device_attn_inputs(cfg, prob)
    cb = Cacheback.from_config(cfg)
    cap = prob.bt.shape[1] * cfg.page_size
    ctx_d = dev(np.array([cap - 1], np.int32))
    before = _u16(d["k_pool"]).copy()
    nodes = np.full((1, cfg.max_depth), -1, np.int32); nodes[0, 0] = 1
    cb.cb_kv_commit(d["k_pool"], d["v_pool"], d["block_table"], ctx_d, d["k_tree"], d["v_tree"], dev(np.array([1], np.int32)), dev(nodes))
    st, _ = cb.cb_poll_status()
    assert st == _lib.CB_ERR_KV_FULL
    assert int(ctx_d[0]) == cap - 1 and np.array_equal(_u16(d["k_pool"]), before)
