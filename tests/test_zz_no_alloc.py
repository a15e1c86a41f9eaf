"""cb_accept_static: acceptance from logits for callers that may not allocate device memory (code living
inside another owner's memory pool, or under a budget fixed before the library loads).  It runs on the
library's built-in scratch array instead of a workspace.  Checked here against the regular cb_accept on
the same inputs and against the CPU oracle, bit for bit, on two calls in a row (the shared array must come
back clean), plus the size limit.  Collected last so that a failure here cannot hide the other tests."""
import numpy as np
import pytest
import torch

import workloads as W
from workloads import device as wdev
from workloads.tensors import TID

pytestmark = pytest.mark.gpu


def _problem(cfg, dtype):
    B, T, V = cfg.batch, cfg.max_nodes, cfg.vocab
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    par = np.full((B, T), -1, np.int32)
    dep = np.full((B, T), -1, np.int32)
    tok = np.full((B, T), -1, np.int32)
    n = np.zeros(B, np.int32)
    for b in range(B):
        n[b] = max(1, T - (b * 5) % T)
        par[b], dep[b] = W.random_tree(cfg.seed, b, int(n[b]), cfg.max_depth, T)
        tok[b, :n[b]] = (W.mix64(cfg.seed, 78, b * 4096 + np.arange(n[b])) % np.uint64(V)).astype(np.int32)
    logits = wdev.normal_tensor((B, T, V), dtype, cfg.seed, TID.LOGITS)
    for b in range(B):
        for node, vid in W.plant_logits(cfg, b, tok[b], par[b], dep[b], int(n[b])):
            logits[b, node, vid] = 32.0
    tree = dict(tokens=dev(tok), parent=dev(par), depth=dev(dep), n_nodes=dev(n))
    return tree, logits, (tok, par, dep, n)


def _oracle_accept(oracle, cfg, logits, host_tree):
    """Arg-max and acceptance of every sequence by the CPU oracle, from the same logits (read back from the device)."""
    tok, par, dep, n = host_tree
    B, T = cfg.batch, cfg.max_nodes
    lg = logits.float().cpu().numpy()
    out = dict(n_accept=np.zeros(B, np.int32), accept_nodes=np.full((B, cfg.max_depth), -1, np.int32),
               out_tokens=np.full((B, cfg.max_depth + 1), -1, np.int32), target_ids=np.full((B, T), -1, np.int32))
    for b in range(B):
        nb = int(n[b])
        out["target_ids"][b, :nb] = oracle.argmax_rows(lg[b, :nb])
        m, nodes, toks = oracle.accept(tok[b], par[b], dep[b], nb, out["target_ids"][b], cfg.max_depth)
        out["n_accept"][b], out["accept_nodes"][b], out["out_tokens"][b] = m, nodes, toks
    return out


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_static_matches_regular_twice(oracle, dtype):
    from paper_2511_21699_b200 import Cacheback, cb_accept_static
    cfg = W.CbConfig("noalloc", 6, 2, 3, 64, 2, 48, 6, 0, 1, 1, 64, (16, 16), 9001, 1.1, 0.3, (4, 8), 64)
    tree, logits, host_tree = _problem(cfg, dtype)
    want = Cacheback.from_config(cfg).cb_accept(tree, logits=logits)
    ref = _oracle_accept(oracle, cfg, logits, host_tree)
    for call in range(2):
        got = cb_accept_static(tree, logits, cfg.max_depth)
        torch.cuda.synchronize()
        for k in ("n_accept", "accept_nodes", "out_tokens", "target_ids"):
            assert torch.equal(got[k], want[k]), (k, call)
            assert np.array_equal(got[k].cpu().numpy(), ref[k]), (k, call, "oracle")
    assert int(want["n_accept"].max()) >= 1
    # a second, differently shaped problem right after: the shared array carries nothing over
    cfg2 = W.CbConfig("noalloc2", 3, 2, 3, 64, 2, 16, 4, 0, 1, 1, 64, (16, 16), 777, 1.1, 0.3, (4, 8), 64)
    tree2, logits2, _ = _problem(cfg2, dtype)
    want2 = Cacheback.from_config(cfg2).cb_accept(tree2, logits=logits2)
    got2 = cb_accept_static(tree2, logits2, cfg2.max_depth)
    for k in ("n_accept", "accept_nodes", "out_tokens", "target_ids"):
        assert torch.equal(got2[k], want2[k]), k


def test_static_rejects_oversize():
    from paper_2511_21699_b200 import cb_accept_static, CachebackError, _lib
    B, T, V = 128, 128, 8                                   # 16,384 rows > CB_STATIC_MAX_ROWS
    z = lambda *s: torch.zeros(*s, dtype=torch.int32, device="cuda")
    tree = dict(tokens=z(B, T), parent=z(B, T), depth=z(B, T), n_nodes=z(B))
    with pytest.raises(CachebackError, match="static scratch"):
        cb_accept_static(tree, torch.zeros(B, T, V, device="cuda"), 4)
    assert B * T > _lib.CB_STATIC_MAX_ROWS
