"""The checking build of the library (-DCB_DEBUG): the stand-in for a memory checker.  Without a GPU: it builds, exports
the same symbols and asks for a larger workspace (the guard areas).  On a GPU, in a process of its own that loads it in
place of the regular library: the tiny draft-and-verify step gives the oracle's results with a clean status, and a guard
byte overwritten from the host is reported by cb_poll_status."""
import ctypes
import os
import subprocess
import sys

import pytest

from tests.conftest import ROOT


def test_checking_build_exports_and_guards_need_no_gpu():
    import __graft_entry__
    __graft_entry__.build()
    from paper_2511_21699_b200 import _lib
    regular, checking = ctypes.CDLL(os.path.join(ROOT, "paper_2511_21699_b200", "libcacheback.so")), ctypes.CDLL(_lib.SO_DEBUG_PATH)
    for name in _lib.EXPORTS:
        assert hasattr(checking, name), name
    assert regular.cb_debug_build() == 0 and checking.cb_debug_build() == 1
    cfg = _lib.CbConfigC(1, 2, 3, 4096, 4, 16, 4, 5, 32000, 8, 8, 64, 16, 0)
    a, b = ctypes.c_size_t(0), ctypes.c_size_t(0)
    for lib in (regular, checking):
        lib.cb_workspace_bytes.argtypes = [ctypes.POINTER(_lib.CbConfigC), ctypes.POINTER(ctypes.c_size_t)]
    assert regular.cb_workspace_bytes(ctypes.byref(cfg), ctypes.byref(a)) == 0
    assert checking.cb_workspace_bytes(ctypes.byref(cfg), ctypes.byref(b)) == 0
    assert b.value == a.value + 10 * _lib.CB_GUARD_BYTES          # one guard area behind each of the ten regions


_CHILD = r"""
import sys
sys.path.insert(0, %r)
import numpy as np, torch
import __graft_entry__
from paper_2511_21699_b200 import _lib, Cacheback
assert _lib.load().cb_debug_build() == 1
__graft_entry__.smoke()                                  # update, draft, attention, acceptance on the tiny config against the oracle
import workloads as W
cfg = W.get_config("c1_tiny")
cb = Cacheback.from_config(cfg)
st, _ = cb.cb_poll_status()
assert st == 0, st
# a stray write just behind the first workspace region (the table headers: batch * 16 bytes, rounded up to 256), made from the host
base = (cb.workspace.data_ptr() + 255) // 256 * 256 - cb.workspace.data_ptr()
cb.workspace[base + 256 + 7] = 0
st, _ = cb.cb_poll_status()
assert st == _lib.CB_ERR_CANARY, st
cb.workspace[base + 256 + 7] = 0xC5
st, _ = cb.cb_poll_status()
assert st == 0, st
# a page id outside the pool in the block table: recorded, the tile reads as zeros, nothing faults
from workloads import device as wdev
from workloads.tensors import TID
ctx = W.ctx_lens(cfg)
bt, num_pages = W.make_block_table(cfg, ctx)
bt = bt.copy(); bt[0, 3] = num_pages + 1000
bf = torch.bfloat16
dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
B, T = cfg.batch, cfg.max_nodes
kp = wdev.normal_tensor((num_pages, cfg.page_size, cfg.n_kv_heads, cfg.head_dim), bf, 0, TID.K_POOL)
vp = wdev.normal_tensor((num_pages, cfg.page_size, cfg.n_kv_heads, cfg.head_dim), bf, 0, TID.V_POOL)
q = wdev.normal_tensor((B, T, cfg.n_q_heads, cfg.head_dim), bf, 0, TID.Q)
kt = wdev.normal_tensor((B, T, cfg.n_kv_heads, cfg.head_dim), bf, 0, TID.K_TREE)
vt = wdev.normal_tensor((B, T, cfg.n_kv_heads, cfg.head_dim), bf, 0, TID.V_TREE)
mask = torch.zeros(B, T, 1, dtype=torch.int32, device="cuda"); mask[:, 0, 0] = 1
out = cb.cb_tree_attn(q, kp, vp, dev(bt), dev(ctx), kt, vt, mask, torch.ones(B, dtype=torch.int32, device="cuda"))
torch.cuda.synchronize()
st, _ = cb.cb_poll_status()
assert st == _lib.CB_ERR_INVALID_ARG, st
assert torch.isfinite(out.float()).all()
print("checking build ok")
"""


@pytest.mark.gpu
def test_checking_build_runs_the_tiny_step_and_reports_planted_errors():
    from paper_2511_21699_b200 import _lib
    env = dict(os.environ, CACHEBACK_LIBRARY=_lib.SO_DEBUG_PATH)
    r = subprocess.run([sys.executable, "-c", _CHILD % ROOT], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "checking build ok" in r.stdout, (r.stdout[-2000:], r.stderr[-3000:])
