"""GPU parity: cb_accept with logits (fp32 and bf16) against the oracle's first-maximum argmax and greedy
acceptance, bit-exact, with planted matches on about half of the tree paths."""
import numpy as np
import pytest
import torch

import workloads as W
from workloads import device as wdev
from workloads.tensors import TID
from tests.harness import Problem, dev, synthetic_trees

pytestmark = pytest.mark.gpu


def _trees(cfg, full):
    B, T = cfg.batch, cfg.max_nodes
    par, dep, mask, n = synthetic_trees(cfg, full=full)
    tok = np.full((B, T), -1, np.int32)
    for b in range(B):
        tok[b, :n[b]] = (W.mix64(cfg.seed, 77, b * 4096 + np.arange(n[b])) % np.uint64(cfg.vocab)).astype(np.int32)
    return tok, par, dep, n


def _run(cfg, dtype, full, sample_b, oracle, stride_pad=0):
    from paper_2511_21699_b200 import Cacheback
    B, T, V = cfg.batch, cfg.max_nodes, cfg.vocab
    tok, par, dep, n = _trees(cfg, full)
    cb = Cacheback.from_config(cfg)
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    if stride_pad:
        store = torch.zeros(B, T, V + stride_pad, dtype=tdt, device="cuda")
        base = wdev.normal_tensor((B, T, V), tdt, cfg.seed, TID.LOGITS)
        store[:, :, :V] = base
        logits = store[:, :, :V]
        del base
    else:
        logits = wdev.normal_tensor((B, T, V), tdt, cfg.seed, TID.LOGITS)
    plants = {}
    for b in range(B):
        plants[b] = W.plant_logits(cfg, b, tok[b], par[b], dep[b], int(n[b]))
        for node, vid in plants[b]:
            logits[b, node, vid] = 32.0
    tree = dict(tokens=dev(tok), parent=dev(par), depth=dev(dep), n_nodes=dev(n))
    for rep in range(2):                                   # twice: the scratch must come back clean
        res = cb.cb_accept(tree, logits=logits)
        r = {k: v.cpu().numpy() for k, v in res.items()}
        assert (r["target_ids"][np.arange(T)[None, :] >= n[:, None]] == -1).all()
        for b in sample_b:
            nb = int(n[b])
            rows = W.logits_rows(cfg, b, np.arange(nb), dtype)
            for node, vid in plants[b]:
                rows[node, vid] = 32.0
            tgt = oracle.argmax_rows(rows)
            assert np.array_equal(r["target_ids"][b, :nb], tgt), (b, rep)
            full_t = np.full(T, -1, np.int32); full_t[:nb] = tgt
            m, nodes, out = oracle.accept(tok[b], par[b], dep[b], nb, full_t, cfg.max_depth)
            assert r["n_accept"][b] == m and np.array_equal(r["accept_nodes"][b], nodes), (b, rep)
            assert np.array_equal(r["out_tokens"][b], out), (b, rep)
    # the same targets through the ids form give the same result
    res2 = cb.cb_accept(tree, target_ids=res["target_ids"].clone())
    for k in ("n_accept", "accept_nodes", "out_tokens"):
        assert torch.equal(res[k], res2[k])
    return r


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("name,full", [("c1_tiny", True), ("c1_tiny", False), ("c2_7b", True), ("c4_13b_turns", False), ("p_tuned", True)])
def test_accept_logits_small(oracle, name, full, dtype):
    cfg = W.get_config(name)
    sample = range(cfg.batch) if cfg.batch <= 4 else [0, 1, 2, 31, 63]
    r = _run(cfg, dtype, full, sample, oracle)
    assert r["n_accept"].max() >= 1                      # planted matches are found


@pytest.mark.parametrize("name,dtype", [("c3_8b_gqa", "f32"), ("c3_8b_gqa", "bf16"), ("c5_70b_long", "bf16"), ("c5_70b_long", "f32")])
def test_accept_logits_full_size_sampled(oracle, name, dtype):
    cfg = W.get_config(name)
    _run(cfg, dtype, False, [0, 1, cfg.batch // 2, cfg.batch - 1], oracle)


def test_accept_ties_and_odd_strides(oracle):
    """bf16 logits tie at the maximum in many rows: the lowest index must win. Rows start at odd offsets."""
    cfg = W.CbConfig("ties", 3, 2, 2, 64, 2, 8, 4, 0, 1, 1, 64, (16, 16), 5003, 1.1, 0.3, (4, 8), 64)
    _run(cfg, "bf16", True, range(3), oracle, stride_pad=3)
    _run(cfg, "f32", True, range(3), oracle, stride_pad=1)
    from paper_2511_21699_b200 import Cacheback
    cb = Cacheback.from_config(cfg)
    tok, par, dep, n = _trees(cfg, True)
    x = torch.zeros(3, 8, 5003, dtype=torch.float32, device="cuda")     # every element ties; -0.0 == +0.0
    x[:, :, 0] = -0.0
    res = cb.cb_accept(dict(tokens=dev(tok), parent=dev(par), depth=dev(dep), n_nodes=dev(n)), logits=x)
    assert (res["target_ids"] == 0).all()
    x[:, :, 4999] = 1.0
    x[:, :, 5001] = 1.0
    res = cb.cb_accept(dict(tokens=dev(tok), parent=dev(par), depth=dev(dep), n_nodes=dev(n)), logits=x)
    assert (res["target_ids"] == 4999).all()
