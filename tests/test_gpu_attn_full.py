"""GPU parity of cb_tree_attn at the full size of the batched configurations, in the launch shape the benchmark times
(full synthetic trees).  Checked rows per configuration: every row of two whole sequences (all kv heads, all nodes),
4,096 seeded random (sequence, head, node) rows, and one row in every unit that two persistent CTAs share (a wrong
partial at one hand-over point would otherwise hide among a million rows).  Same tolerances as test_gpu_attn.py."""
import numpy as np
import pytest
import torch

import workloads as W
from tests.harness import Problem, dev, device_attn_inputs, synthetic_trees, oracle_attn_rows_by_head, shared_unit_rows, bf16_to_f64
from tests.test_gpu_attn import _check_rows

pytestmark = pytest.mark.gpu

N_RANDOM = 4096


def _rows(cfg, prob, n, n_ctas):
    G = cfg.gqa
    whole = [(b, h, i) for b in (0, cfg.batch - 1) for h in range(cfg.n_q_heads) for i in range(int(n[b]))]
    # random rows come in groups that share a (sequence, kv head), so that the host copy of that head's keys serves many
    rng = np.random.default_rng(7)
    per = 64
    rand = []
    for _ in range(N_RANDOM // per):
        b, kh = int(rng.integers(0, cfg.batch)), int(rng.integers(0, cfg.n_kv_heads))
        for _ in range(per):
            rand.append((b, kh * G + int(rng.integers(0, G)), int(rng.integers(0, int(n[b])))))
    seams = shared_unit_rows(cfg, prob.ctx, n, n_ctas)
    return whole, rand, seams


@pytest.mark.parametrize("name", ["c3_8b_gqa", "c4_13b_turns", "c5_70b_long"])
def test_attn_full_size_whole_sequences_random_rows_and_seams(oracle, name):
    from paper_2511_21699_b200 import Cacheback
    cfg = W.get_config(name)
    prob = Problem(cfg)
    B, T = cfg.batch, cfg.max_nodes
    par, dep, mask, n = synthetic_trees(cfg, full=True)
    d = device_attn_inputs(cfg, prob)
    cb = Cacheback.from_config(cfg)
    lse = torch.full((B, cfg.n_q_heads, T), 7.0, dtype=torch.float32, device="cuda")
    out = torch.full((B, T, cfg.n_q_heads, cfg.head_dim), 3.0, dtype=torch.bfloat16, device="cuda")
    cb.cb_tree_attn(d["q"], d["k_pool"], d["v_pool"], d["block_table"], d["ctx_len"], d["k_tree"], d["v_tree"],
                    dev(mask.view(np.int32)), dev(n), out=out, lse=lse, max_ctx=int(prob.ctx.max()))
    torch.cuda.synchronize()
    assert cb.cb_poll_status()[0] == 0
    n_ctas = min(torch.cuda.get_device_properties(0).multi_processor_count, 160)   # ranges of the stream-K split: one per SM
    whole, rand, seams = _rows(cfg, prob, n, n_ctas)
    assert len(whole) == 2 * cfg.n_q_heads * T and len(rand) >= 4096 and len(seams) >= n_ctas // 2, (len(whole), len(rand), len(seams))
    rows = np.array(whole + rand + seams, np.int64)
    ref, ref_lse = oracle_attn_rows_by_head(oracle, cfg, prob, mask, rows)
    bb, hh, ii = (torch.from_numpy(rows[:, k]).cuda() for k in range(3))
    got = bf16_to_f64(out[bb, ii, hh])
    got_lse = lse[bb, hh, ii].cpu().numpy().astype(np.float64)
    k0, k1 = len(whole), len(whole) + len(rand)
    _check_rows(got[:k0], got_lse[:k0], ref[:k0], ref_lse[:k0], (name, "whole sequences", k0))
    _check_rows(got[k0:k1], got_lse[k0:k1], ref[k0:k1], ref_lse[k0:k1], (name, "random rows", k1 - k0))
    _check_rows(got[k1:], got_lse[k1:], ref[k1:], ref_lse[k1:], (name, "shared units", len(rows) - k1))
