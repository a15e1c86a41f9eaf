"""The C-ABI library loads without a GPU and exports every function the public header declares."""
import ctypes
import os
import re

from tests.conftest import ROOT


def _declared():
    with open(os.path.join(ROOT, "include", "cacheback.h")) as f:
        src = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    return sorted(set(re.findall(r"\b(cb_[a-z_0-9]+)\s*\(", src)))


def test_header_symbols_are_exported():
    import __graft_entry__
    __graft_entry__.build()
    from paper_2511_21699_b200 import _lib
    lib = _lib.load()
    names = _declared()
    assert {"cb_update", "cb_draft_tree", "cb_tree_attn", "cb_accept"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(_lib.EXPORTS) == set(names)


def test_host_side_argument_checks_need_no_gpu():
    from paper_2511_21699_b200 import _lib
    lib = _lib.load()
    cfg = _lib.CbConfigC(1, 2, 3, 4096, 4, 16, 4, 5, 32000, 8, 8, 64, 16, 0)
    n = ctypes.c_size_t(0)
    assert lib.cb_workspace_bytes(ctypes.byref(cfg), ctypes.byref(n)) == 0 and n.value > 4096 * 4
    bad = _lib.CbConfigC(1, 2, 3, 4096, 4, 16, 4, 5, 32000, 8, 3, 64, 16, 0)      # heads do not divide
    assert lib.cb_workspace_bytes(ctypes.byref(bad), ctypes.byref(n)) == 1
    bad = _lib.CbConfigC(1, 2, 3, 4096, 4, 256, 4, 5, 32000, 8, 8, 64, 16, 0)     # tree cap above 128
    assert lib.cb_workspace_bytes(ctypes.byref(bad), ctypes.byref(n)) == 1
    assert lib.cb_status_str(4).decode().startswith("hash probe")
    assert lib.cb_accept_static(4096, 16, 4, 100, 1, 1, 1, 1, 8, 0, 100, 1, 1, 1, None, None) == _lib.CB_ERR_STATIC_LIMIT


def test_frozen_table_sizes_and_argument_checks_need_no_gpu():
    from paper_2511_21699_b200 import _lib
    lib = _lib.load()
    n, m = ctypes.c_size_t(0), ctypes.c_size_t(0)
    cfg = _lib.CbFrozenConfigC(1, 3, 1 << 16, 128)
    assert lib.cb_frozen_bytes(ctypes.byref(cfg), ctypes.byref(n)) == 0
    assert n.value >= (1 << 16) * (1 + 128 * 4) * 4                               # entries: key + FC * (stamp + FL tokens)
    assert lib.cb_frozen_build_bytes(ctypes.byref(cfg), 1 << 20, ctypes.byref(m)) == 0 and m.value > (1 << 20) * 32
    assert lib.cb_frozen_build_bytes(ctypes.byref(cfg), (1 << 30) + 1, ctypes.byref(m)) == 1   # corpus above the stated limit
    for bad in (_lib.CbFrozenConfigC(0, 3, 16, 4), _lib.CbFrozenConfigC(1, 9, 16, 4), _lib.CbFrozenConfigC(1, 3, 16, 129),
                _lib.CbFrozenConfigC(1, 3, (1 << 20) + 1, 4)):
        assert lib.cb_frozen_bytes(ctypes.byref(bad), ctypes.byref(n)) == 1
    assert lib.cb_frozen_attach(None, ctypes.byref(cfg), None, 0) == 1            # no context


def test_bulk_scratch_sizes_and_argument_checks_need_no_gpu():
    """Two hash tables of the next power of two >= 2 * windows slots at 40 bytes a slot, plus 4 bytes per window place."""
    from paper_2511_21699_b200 import _lib
    lib = _lib.load()
    cfg = _lib.CbConfigC(128, 3, 5, 65536, 8, 128, 32, 16, 32000, 64, 8, 128, 16, 0)
    n = ctypes.c_size_t(0)
    last = 0
    for windows in (1, 1000, 4096, 4097, 127459, 4193536):
        assert lib.cb_bulk_scratch_bytes(ctypes.byref(cfg), windows, ctypes.byref(n)) == 0
        slots = 2048
        while slots < 2 * windows:
            slots *= 2
        assert 42 * slots <= n.value <= 42 * slots + 16 * 256 + (cfg.batch + 1) * 4 + 64, (windows, n.value)
        assert n.value >= last
        last = n.value
    assert lib.cb_bulk_scratch_bytes(ctypes.byref(cfg), 0, ctypes.byref(n)) == 1
    assert lib.cb_bulk_scratch_bytes(ctypes.byref(cfg), (1 << 29) + 1, ctypes.byref(n)) == 1
    assert lib.cb_bulk_scratch_bytes(None, 16, ctypes.byref(n)) == 1
    assert lib.cb_bulk_scratch_attach(None, None, 0) == 1                           # no context
