"""Pins for the oracle's cache table and sliding-window update (Section 3.1; Section 3.2/3.3 last
paragraphs).  None of these re-use the oracle's own formulas: hand traces, an OrderedDict model,
brute-force closed forms and capacity invariants."""
import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from tests.conftest import golden
from tests.od_model import ODTable
import workloads as W


def _name_state(state, ids):
    return [((ids[l],), [(ids[f],) for f in fs]) for l, fs in state]


@pytest.mark.parametrize("fixture", ["trace_a_lru.json", "trace_b_follower_refresh.json"])
def test_hand_traces(oracle, fixture):
    g = golden(fixture)
    ids = g["ids"]
    t = oracle.OracleTable(**g["params"])
    for k, step in enumerate(g["steps"]):
        if step["op"] == "ins":
            t.insert([ids[step["leader"]]], [ids[step["follower"]]])
        else:
            got = t.query([ids[step["leader"]]])
            assert got == [(ids[f],) for f in step["returns"]], (fixture, k)
        assert t.dump() == _name_state(step["state"], ids), (fixture, k)


def test_trace_b_distinguishes_no_refresh_reading(oracle):
    g = golden("trace_b_follower_refresh.json")
    ids = g["ids"]
    t = oracle.OracleTable(**g["params"], refresh_on_reinsert=False)
    for step in g["steps"][:-1]:
        t.insert([ids[step["leader"]]], [ids[step["follower"]]])
    assert t.query([ids["a"]]) == [(ids["d"],), (ids["c"],)]


def test_trace_a_is_the_sliding_window_of_its_stream(oracle):
    g = golden("trace_a_lru.json")
    ids = g["ids"]
    s = [ids[c] for c in "abacad"]
    t = oracle.OracleTable(**g["params"])
    t.update(s, 0, len(s))
    assert t.dump() == _name_state(g["steps"][4]["state"], ids)
    assert t.clock == 5


def test_update_windows_match_trace_d(oracle):
    g = golden("trace_d_accept.json")["update"]
    s = g["sequence"]
    t1 = oracle.OracleTable(g["params"]["LL"], g["params"]["FL"], 64, 4)
    t2 = oracle.OracleTable(g["params"]["LL"], g["params"]["FL"], 64, 4)
    t1.update(s, g["n_old"], g["n_new"])
    for L, F in g["windows"]:
        t2.insert(L, F)
    assert t1.dump() == t2.dump() and t1.clock == len(g["windows"])


def test_update_is_incremental(oracle):
    """Ingesting a stream in pieces inserts exactly the windows of ingesting it whole; partial windows
    at the end wait for a later call."""
    cfg = W.get_config("c1_tiny")
    s = W.make_stream(cfg, 0, 600)
    whole = oracle.OracleTable(cfg.LL, cfg.FL, 128, cfg.FC)
    parts = oracle.OracleTable(cfg.LL, cfg.FL, 128, cfg.FC)
    whole.update(s, 0, 600)
    cuts = [0, 1, 3, 4, 5, 9, 200, 201, 207, 600]
    for a, b in zip(cuts[:-1], cuts[1:]):
        parts.update(s, a, b)
    assert whole.dump() == parts.dump()
    assert whole.clock == parts.clock == 600 - (cfg.LL + cfg.FL) + 1


ops = st.lists(st.tuples(st.sampled_from(["ins", "ins", "ins", "query"]),
                         st.lists(st.integers(0, 3), min_size=2, max_size=2),
                         st.lists(st.integers(0, 2), min_size=2, max_size=2)), max_size=120)


@settings(max_examples=300, deadline=None)
@given(ops=ops, LL=st.integers(1, 2), FL=st.integers(1, 2), LC=st.integers(1, 5), FC=st.integers(1, 3),
       refresh=st.booleans())
def test_against_ordered_dict_model(oracle, ops, LL, FL, LC, FC, refresh):
    t = oracle.OracleTable(LL, FL, LC, FC, refresh_on_reinsert=refresh)
    m = ODTable(LL, FL, LC, FC, refresh_on_reinsert=refresh)
    for op, L, F in ops:
        L, F = L[:LL], F[:FL]
        if op == "ins":
            t.insert(L, F)
            m.insert(L, F)
        else:
            assert t.query(L) == m.query(L)
        d = t.dump()
        assert d == m.dump()
        assert len(d) <= LC and all(1 <= len(fs) <= FC for _, fs in d)      # capacity invariants


@pytest.mark.parametrize("name,n", [("c1_tiny", 2048), ("c2_7b", 3000), ("c4_13b_turns", 4096)])
def test_closed_form_without_leader_eviction(oracle, name, n):
    """With LC above the number of distinct leaders the state is order-free: a leader's recency is the
    index of its last window and its followers are the FC distinct followers observed last."""
    cfg = W.get_config(name)
    s = W.make_stream(cfg, 0, n).tolist()
    t = oracle.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC)
    t.update(s, 0, n)
    w = cfg.LL + cfg.FL
    last_window = {}
    last_seen = {}
    for i in range(n - w + 1):
        L, F = tuple(s[i:i + cfg.LL]), tuple(s[i + cfg.LL:i + w])
        last_window[L] = i
        last_seen.setdefault(L, {})[F] = i
    expect = []
    for L in sorted(last_window, key=last_window.get):
        fs = sorted(last_seen[L], key=last_seen[L].get)[-cfg.FC:]
        expect.append((L, fs))
    assert len(expect) <= cfg.LC
    assert t.dump() == expect


@pytest.mark.parametrize("LC", [16, 256])
def test_leader_set_is_most_recently_touched(oracle, LC):
    cfg = W.get_config("c1_tiny")
    n = 2048
    s = W.make_stream(cfg, 0, n).tolist()
    t = oracle.OracleTable(cfg.LL, cfg.FL, LC, cfg.FC)
    w = cfg.LL + cfg.FL
    touched = []
    for i in range(n - w + 1):
        L = tuple(s[i:i + cfg.LL])
        t.insert(L, s[i + cfg.LL:i + w])
        touched.append(L)
        if i % 7 == 3:                       # a hit refreshes the leader; a miss changes nothing
            Lq = tuple(s[(i * 13) % (n - w):][:cfg.LL])
            if t.query(Lq):
                touched.append(Lq)
        assert len(t) <= LC
    recent = []
    for L in reversed(touched):
        if L not in recent:
            recent.append(L)
        if len(recent) == LC:
            break
    assert [d[0] for d in t.dump()] == list(reversed(recent))


def test_eviction_drops_followers_with_the_leader(oracle):
    t = oracle.OracleTable(1, 1, 2, 3)
    t.insert([1], [10]); t.insert([1], [11]); t.insert([2], [20]); t.insert([3], [30])   # evicts leader 1
    assert t.query([1]) == []
    t.insert([1], [12])                                                                  # evicts leader 2
    assert t.dump() == [((3,), [(30,)]), ((1,), [(12,)])]
