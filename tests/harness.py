"""Shared set-up for the GPU parity tests: builds the same seeded problem for the CUDA path (device
tensors) and for the oracle (host slices)."""
import numpy as np
import torch

import workloads as W
from workloads import device as wdev
from workloads.tensors import TID


def dev(x, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(x))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


class Problem:
    """Streams, contexts and block tables of one config (host side)."""

    def __init__(self, cfg):
        self.cfg = cfg
        self.ctx = W.ctx_lens(cfg)
        self.toks, self.lens = W.make_streams(cfg, self.ctx)
        self.bt, self.num_pages = W.make_block_table(cfg, self.ctx)
        # prefill = the context: the table has seen exactly the cached tokens plus the pending root
        self.prefill = np.minimum(self.ctx + 1, self.lens).astype(np.int32)


def device_attn_inputs(cfg, prob):
    B, T = cfg.batch, cfg.max_nodes
    bf = torch.bfloat16
    d = {}
    d["k_pool"] = wdev.normal_tensor((prob.num_pages, cfg.page_size, cfg.n_kv_heads, cfg.head_dim), bf, cfg.seed, TID.K_POOL)
    d["v_pool"] = wdev.normal_tensor((prob.num_pages, cfg.page_size, cfg.n_kv_heads, cfg.head_dim), bf, cfg.seed, TID.V_POOL)
    d["q"] = wdev.normal_tensor((B, T, cfg.n_q_heads, cfg.head_dim), bf, cfg.seed, TID.Q)
    d["k_tree"] = wdev.normal_tensor((B, T, cfg.n_kv_heads, cfg.head_dim), bf, cfg.seed, TID.K_TREE)
    d["v_tree"] = wdev.normal_tensor((B, T, cfg.n_kv_heads, cfg.head_dim), bf, cfg.seed, TID.V_TREE)
    d["block_table"] = dev(prob.bt)
    d["ctx_len"] = dev(prob.ctx)
    return d


def synthetic_trees(cfg, full=True):
    """Per-sequence random trees (parents, depths, masks, node counts). full=False varies the size."""
    B, T = cfg.batch, cfg.max_nodes
    Wd = (T + 31) // 32
    par = np.full((B, T), -1, np.int32)
    dep = np.full((B, T), -1, np.int32)
    mask = np.zeros((B, T, Wd), np.uint32)
    n = np.zeros(B, np.int32)
    for b in range(B):
        n[b] = T if full else max(1, T - (b * 7) % T)
        if b == 1 and not full:
            n[b] = 1
        par[b], dep[b] = W.random_tree(cfg.seed, b, int(n[b]), cfg.max_depth, T)
        mask[b] = W.tree_mask_from_parents(par[b], int(n[b]), Wd)
    return par, dep, mask, n


def oracle_attn_rows(oracle, cfg, prob, mask, b, rows_hi):
    """Oracle outputs for rows (h, i) of sequence b, from a compact host copy of that sequence's inputs."""
    P = cfg.page_size
    npg = (int(prob.ctx[b]) + P - 1) // P
    pages = prob.bt[b, :npg]
    kp, vp = W.pool_pages_bits(cfg, pages)
    q = W.seq_bits(cfg, TID.Q, b, cfg.n_q_heads)[None]
    kt = W.seq_bits(cfg, TID.K_TREE, b, cfg.n_kv_heads)[None]
    vt = W.seq_bits(cfg, TID.V_TREE, b, cfg.n_kv_heads)[None]
    bt = np.arange(max(npg, 1), dtype=np.int32)[None]
    if npg == 0:
        kp = np.zeros((1, P, cfg.n_kv_heads, cfg.head_dim), np.uint16)
        vp = kp
    rows = np.array([(0, h, i) for h, i in rows_hi], dtype=np.int32)
    return oracle.tree_attn_rows(q, kp, vp, bt, prob.ctx[b:b + 1], kt, vt, mask[b:b + 1], rows)


def bf16_to_f64(t):
    return t.float().cpu().numpy().astype(np.float64)
