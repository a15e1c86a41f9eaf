"""GPU parity: cb_update_bulk (prompt initialisation spread over many warps per sequence) against the oracle's plain
sequential update: table contents, recency order and clock, for empty and non-empty tables, for runs that qualify for the
parallel path and runs that must fall back (possible leader eviction, short runs), then drafting from the result."""
import numpy as np
import pytest
import torch

import workloads as W
from tests.harness import Problem, dev
from tests.test_gpu_table import _assert_tables_equal

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,flags", [("c1_tiny", 0), ("c2_7b", 0), ("c2_7b", 1), ("c3_8b_gqa", 0), ("c4_13b_turns", 0),
                                        ("p_tuned", 0), ("p_fc40_evict", 0), ("c1_evict256", 0), ("c5_70b_long", 0)])
@pytest.mark.parametrize("scratch", ["none", "all", "some"])
def test_bulk_prompt_then_incremental_then_draft(oracle, name, flags, scratch):
    """scratch: "all" attaches scratch that holds every sequence's run (the order-free path where a run qualifies), "some"
    scratch for about half of the batch's windows (the rest takes the other paths in the same call)."""
    from paper_2511_21699_b200 import Cacheback
    cfg = W.get_config(name)
    prob = Problem(cfg)
    B, T = cfg.batch, cfg.max_nodes
    if scratch == "some" and B < 4:
        pytest.skip("one sequence: nothing to split")
    cb = Cacheback.from_config(cfg, flags=flags)
    if scratch != "none":
        total = int(np.sum(prob.prefill))
        cb.cb_bulk_scratch_attach(total if scratch == "all" else max(total // 2, 1024))
    check = list(range(B)) if B <= 8 else [0, 1, B // 2, B - 1]
    otabs = {b: oracle.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC, refresh_on_reinsert=not (flags & 1)) for b in check}
    toks_d = dev(prob.toks)
    room = int((prob.lens - T - 2).min())
    p1 = np.minimum(prob.prefill, room - 400).astype(np.int32)              # the prompt
    p2 = (p1 + 300).astype(np.int32)                                        # a long run appended to a filled table
    p2[::2] += 37
    p3 = (p2 + 20).astype(np.int32)                                         # a short run: below the parallel threshold
    zero = torch.zeros(B, dtype=torch.int32, device="cuda")
    cb.cb_update_bulk(toks_d, zero, dev(p1))
    for b in check:
        otabs[b].update(prob.toks[b], 0, int(p1[b]))
    _assert_tables_equal(cb, otabs, check)
    cb.cb_update_bulk(toks_d, dev(p1), dev(p2))
    cb.cb_update_bulk(toks_d, dev(p2), dev(p3))
    for b in check:
        otabs[b].update(prob.toks[b], int(p1[b]), int(p2[b]))
        otabs[b].update(prob.toks[b], int(p2[b]), int(p3[b]))
    _assert_tables_equal(cb, otabs, check)
    st, cnt = cb.cb_poll_status()
    assert st == 0, st
    w = cfg.LL + cfg.FL
    assert cnt["inserts"] == int(np.sum(np.maximum(p3 - w + 1, 0)))
    if "evict" in name:
        assert cnt["leader_evictions"] > 0
    # drafting and the per-step update carry on from the bulk-built state exactly as from a sequentially built one
    pos = p3.copy()
    tree = cb.alloc_tree()
    for step in range(3):
        cb.cb_draft_tree(toks_d, dev(pos), tree)
        g = {k: v.cpu().numpy() for k, v in tree.items()}
        for b in check:
            n, tok, par, dep, mask = otabs[b].draft_tree(prob.toks[b], int(pos[b]), T, cfg.crt, cfg.max_depth)
            assert g["n_nodes"][b] == n and np.array_equal(g["tokens"][b], tok) and np.array_equal(g["parent"][b], par), (step, b)
        new_pos = (pos + 3).astype(np.int32)
        cb.cb_update(toks_d, dev(pos), dev(new_pos))
        for b in check:
            otabs[b].update(prob.toks[b], int(pos[b]), int(new_pos[b]))
        pos = new_pos
    _assert_tables_equal(cb, otabs, check)
    assert cb.cb_poll_status()[0] == 0


def test_bulk_equals_sequential_call_on_a_prompt():
    """The same prompt through cb_update, cb_update_bulk and cb_update_bulk with scratch: identical dumps (the times are printed; the benchmark reports them)."""
    from paper_2511_21699_b200 import Cacheback
    cfg = W.get_config("c2_7b")
    prob = Problem(cfg)
    toks_d = dev(prob.toks)
    zero = torch.zeros(1, dtype=torch.int32, device="cuda")
    n = dev(prob.prefill)
    times = {}
    dumps = {}
    for kind in ("seq", "bulk", "bulk_scratch"):
        best = 1e9
        for rep in range(3):
            cb = Cacheback.from_config(cfg)
            if kind == "bulk_scratch":
                cb.cb_bulk_scratch_attach(int(prob.prefill[0]))
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            (cb.cb_update if kind == "seq" else cb.cb_update_bulk)(toks_d, zero, n)
            e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        times[kind] = best
        dumps[kind] = cb.cb_table_dump(0)
    assert dumps["seq"] == dumps["bulk"] == dumps["bulk_scratch"]
    print("prompt of %d tokens: sequential %.3f ms, bulk %.3f ms, bulk with scratch %.3f ms" % (int(prob.prefill[0]), times["seq"], times["bulk"], times["bulk_scratch"]))
