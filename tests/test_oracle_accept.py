"""Pins for the oracle's target argmax and greedy acceptance (Section 3.2): the Figure 2 caption worked by
hand, brute force over all root-to-node paths, and the losslessness / tokens-per-step invariants."""
import numpy as np
import pytest

from tests.conftest import golden
import workloads as W


def test_trace_d(oracle):
    g = golden("trace_d_accept.json")
    tr = g["tree"]
    m, nodes, out = oracle.accept(tr["tok"], tr["par"], tr["dep"], tr["n"], g["target"], 8)
    assert m == g["n_accept"]
    assert nodes[:m].tolist() == g["accept_nodes"] and (nodes[m:] == -1).all()
    assert out[:m + 1].tolist() == g["out_tokens"] and (out[m + 1:] == -1).all()


def test_no_match_emits_one_token(oracle):
    g = golden("trace_d_accept.json")["tree"]
    target = [77] * g["n"]
    m, nodes, out = oracle.accept(g["tok"], g["par"], g["dep"], g["n"], target, 8)
    assert m == 0 and out[0] == 77 and (out[1:] == -1).all() and (nodes == -1).all()


def test_argmax_first_maximum(oracle):
    x = np.array([[0.5, 2.0, 2.0, -1.0], [-3.0, -3.0, -5.0, -3.0], [0.0, -0.0, 0.0, -1.0]], dtype=np.float32)
    assert oracle.argmax_rows(x).tolist() == [1, 0, 0]
    rng = np.random.default_rng(0)
    y = np.round(rng.normal(size=(50, 999)).astype(np.float32) * 4) / 4          # many exact ties
    assert oracle.argmax_rows(y).tolist() == np.argmax(y, axis=1).tolist()       # numpy: first occurrence


@pytest.mark.parametrize("seed", range(6))
def test_brute_force_longest_matching_path(oracle, seed):
    """Enumerate every node's root path; the accepted path must be a longest fully matching one, the
    smallest-index node among those of that depth, and the emitted tokens must be the target's own
    greedy continuation along it (losslessness)."""
    rng = np.random.default_rng(seed)
    T = 24
    par, dep = W.random_tree(seed, 0, T, 6)
    tok = rng.integers(0, 4, size=T).astype(np.int32)
    target = rng.integers(0, 4, size=T).astype(np.int32)
    m, nodes, out = oracle.accept(tok, par, dep, T, target, 6)
    best, best_len = 0, 0
    for i in range(T):
        path, c = [], i
        while c > 0:
            path.append(c); c = int(par[c])
        path = path[::-1]
        if all(tok[c] == target[par[c]] for c in path) and len(path) > best_len:
            best, best_len = i, len(path)
    assert m == best_len
    assert (nodes[m - 1] if m else 0) == best
    assert 1 <= m + 1 <= 1 + int(dep.max())                   # tokens emitted per step
    prev = 0
    for k in range(m):                                        # each emitted token is the target's choice
        assert out[k] == target[prev] and par[nodes[k]] == prev
        prev = int(nodes[k])
    assert out[m] == target[prev]
