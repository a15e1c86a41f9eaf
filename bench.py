#!/usr/bin/env python
"""Benchmark of the Cacheback draft-and-verify step on B200.

A step is one pass of the whole hot path over one batch: cb_update (sliding window over the tokens accepted by the
previous step) -> cb_draft_tree -> cb_tree_attn -> cb_accept (fp32 logits); the first two are issued as the library's
one-launch form cb_update_draft_tree unless --separate-calls is given.  Inputs are synthetic (seeded generators in
workloads/).  Prints ONE JSON line.

With no --config the headline is the largest configuration (70B-shaped: batch 128, 64/8 heads, context 32,768, trees of
128 nodes) with synthetic full trees, so that the attention shape is the stated one; the figure with the drafter's own
trees stands beside it, and `per_config` holds one record for each of the four full-size configurations (7B-shaped
batch 1, 8B GQA batch 32, 13B batch 64, 70B batch 128).  With --config NAME only that configuration is run.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

--gpus N > 1 outside a torchrun launch starts N ranks itself (one process per GPU); ranks are independent replicas.
"""
import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "draft_tree_tokens_verified_per_s"
UNIT = "tokens/s"
ADVANCE = 4            # tokens each sequence advances per step (a typical accepted run plus the bonus token)
HEADLINE = "c5_70b_long"
FULL_SIZE = ["c2_7b", "c3_8b_gqa", "c4_13b_turns", "c5_70b_long"]


def parse(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default=None, help="one workload only (default: headline %s plus per_config records)" % HEADLINE)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-closed-loop", action="store_true")
    ap.add_argument("--drafted-headline", action="store_true", help="headline value from the drafter's own trees instead of full ones")
    ap.add_argument("--separate-calls", action="store_true", help="cb_update and cb_draft_tree as two launches")
    ap.add_argument("--frozen", type=int, default=0, metavar="TOKENS",
                    help="attach a frozen table built on the GPU from a synthetic corpus of this many tokens (0 = none)")
    ap.add_argument("--flags", type=int, default=0, help="cb_config.flags for the context (4 = tree attention as pairs of CTAs)")
    ap.add_argument("--rank-plumbing-only", action="store_true", help=argparse.SUPPRESS)
    return ap.parse_args(argv)


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one cb_attn_tc_kernel launch with full trees, from the ncu
# captures summarised under profiles/.  Reported only while the kernel sources still hash to the captured ones; after any
# change to them the figure is stale and `traffic` is null until the capture is redone.
ATTN_TRAFFIC = {"sources_sha1": "631ae1a4edeb073d1c842aef25b5ff4467c347b4",
                "bytes_per_launch": {"c2_7b": 70.2e6, "c3_8b_gqa": 557.6e6, "c4_13b_turns": 2767.4e6},
                "source": {k: "profiles/cb_attn_tc_kernel_c2_c3_c4_c5b8.md" for k in ("c2_7b", "c3_8b_gqa", "c4_13b_turns")},
                # config 5 holds 25 GB and runs 20 ms per launch: too large to capture.  The same shape at batch 8 was captured
                # (1,405.0 + 8.4 and 1,432.1 + 8.4 MB per launch); keys and values are streamed per sequence, so the traffic is taken
                # to grow with the batch: mean x 128 / 8.
                "scaled": {"c5_70b_long": (1427.0e6 * 16.0,
                                           "profiles/cb_attn_tc_kernel_c2_c3_c4_c5b8.md: c5_70b_b8 (same shape, batch 8), mean of two captures "
                                           "x 16 sequences' worth; not a capture of this workload")}}
ATTN_SOURCES = ("cb_attn_tc.cu", "cb_tc_dev.cuh", "cb_attn_pair.cuh", "cb_attn.cuh", "cb_attn.cu")


def attn_sources_sha1():
    import hashlib
    h = hashlib.sha1()
    for f in ATTN_SOURCES:
        with open(os.path.join(ROOT, "paper_2511_21699_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "tflops": float(d["bf16_tflops"]),
                "tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "kind": "measured (MEASURED_PEAKS.json)"}
    return {"hbm_gbs": 6650.0, "tflops": 1590.0, "tflops_sustained": 1400.0, "kind": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
                for k, nm in enumerate(names):
                    if r[3 + k].lower().startswith("active"):
                        reasons.add(nm)
            except Exception:
                pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def reduce_over_ranks(seconds, units, device):
    """Whole-job figures of a replicated run: the slowest rank's time and the units of all ranks together.
    (No collective is on the data path: ranks are independent replicas; these two all-reduces only gather the result.)"""
    import torch
    import torch.distributed as dist
    t = torch.tensor([seconds], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    u = torch.tensor([units], device=device, dtype=torch.float64)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(n, argv):
    """Starts this script as n ranks of one node (one process per GPU) and passes their output through; used when
    --gpus n > 1 is given outside a torchrun launch."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n), "--master-addr", "127.0.0.1",
           "--master-port", str(free_port()), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def ancestor_masks(par):
    """Bit-packed ancestor-or-self rows for synthetic full trees given as parent arrays [B, T] (an input of the
    attention-only shape; drafted trees get their masks from cb_draft_tree)."""
    B, T = par.shape
    m = np.zeros((B, T, (T + 31) // 32), np.uint32)
    for b in range(B):
        for i in range(T):
            if par[b, i] >= 0:
                m[b, i] = m[b, par[b, i]]
            m[b, i, i // 32] |= np.uint32(1) << np.uint32(i % 32)
    return m


def attn_bytes(cfg, ctx, n_nodes):
    """Algorithmic HBM bytes of one cb_tree_attn launch: cached K and V once, tree K/V, Q in, O out."""
    D, Hkv, Hq = cfg.head_dim, cfg.n_kv_heads, cfg.n_q_heads
    return float(np.sum(ctx.astype(np.float64) * Hkv * D * 2 * 2 + n_nodes * Hkv * D * 4 + n_nodes * Hq * D * 4))


def attn_flops(cfg, ctx, n_nodes, pairs):
    """4 * Hq * D * (node-context pairs + node-ancestor pairs): the two products of attention."""
    return float(4.0 * cfg.n_q_heads * cfg.head_dim * (np.sum(n_nodes * ctx.astype(np.float64)) + pairs))


def attn_roofline(cfg, ctx, n_nodes, pairs, ms, pk):
    """Roofline record of one cb_tree_attn launch (attention kernel plus its merge pass): the slower of bytes over the
    measured copy bandwidth and flops over the measured bf16 matmul rate."""
    a_bytes, fl = attn_bytes(cfg, ctx, n_nodes), attn_flops(cfg, ctx, n_nodes, pairs)
    t_mem, t_cmp = a_bytes / (pk["hbm_gbs"] * 1e9), fl / (pk["tflops"] * 1e12)
    if t_mem >= t_cmp:
        r = {"bound": "hbm", "achieved": a_bytes / (ms * 1e-3) / 1e9, "peak": pk["hbm_gbs"], "unit": "GB/s"}
    else:
        r = {"bound": "tensor", "achieved": fl / (ms * 1e-3) / 1e12, "peak": pk["tflops"], "unit": "TFLOP/s"}
        r["frac_of_sustained"] = r["achieved"] / pk["tflops_sustained"]
        r["peak_sustained"] = pk["tflops_sustained"]
    r["frac"] = r["achieved"] / r["peak"]
    r.update({"ms_per_launch": ms, "algorithmic_bytes": a_bytes, "flops": fl, "gbs": a_bytes / (ms * 1e-3) / 1e9,
              "tflops": fl / (ms * 1e-3) / 1e12, "roofline_ms": 1e3 * max(t_mem, t_cmp), "peak_source": pk["kind"]})
    return r


# --------------------------------------------------------------------------------------------------------
def oracle_sample(cfg, ctx, toks, lens, bt, steps, full_trees, nb=2, nh=2, nn=16):
    """The oracle, as it stands, timed single-threaded on a bounded sample of the step: nb sequences; table update,
    drafting, arg-max and acceptance whole; attention on nh query heads and (with full trees) nn of the tree's nodes,
    its time scaled to all heads and nodes.  Returns (tokens per step of the whole batch, seconds per step of the whole
    batch, words describing the sample)."""
    import workloads as W
    from oracle import cb_oracle as orc
    B, T = cfg.batch, cfg.max_nodes
    nb, nh = min(B, nb), min(cfg.n_q_heads, nh)
    G = cfg.gqa
    t_total, tok_total = 0.0, 0.0
    for b in range(nb):
        tab = orc.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC)
        pos = int(min(ctx[b] + 1, lens[b]))
        tab.update(toks[b], 0, pos)
        npg = (int(ctx[b]) + cfg.page_size - 1) // cfg.page_size
        heads = list(range(nh))
        kvs = {}
        for kh in sorted({h // G for h in heads}):          # the sampled heads' kv heads only: one compact copy per kv head
            kp, vp = W.pool_slice_kv(cfg, bt[b, :npg], kh, npg * cfg.page_size, as_f32=False)
            kt, vt = W.tree_kv(cfg, b, kh, as_f32=False)
            kvs[kh] = (kp.reshape(npg, cfg.page_size, 1, cfg.head_dim), vp.reshape(npg, cfg.page_size, 1, cfg.head_dim),
                       kt[None, :, None, :], vt[None, :, None, :])
        qh = {h: W.queries(cfg, b, h, as_f32=False)[None, :, None, :] for h in heads}
        if full_trees:
            fpar, fdep = W.random_tree(cfg.seed, b, T, cfg.max_depth, T)
            fmask = orc.tree_mask(fpar, T, T)
        for rep in range(steps):
            t0 = time.perf_counter()
            tab.update(toks[b], pos, pos + ADVANCE)
            pos += ADVANCE
            n, tok, par, dep, mask = tab.draft_tree(toks[b], pos, T, cfg.crt, cfg.max_depth)
            t1 = time.perf_counter()
            if full_trees:
                n, par, dep, mask, tok = T, fpar, fdep, fmask, np.maximum(fpar, 0).astype(np.int32)
            nodes = list(range(n))
            if full_trees and n > nn:
                nodes = sorted(set(range(0, n, n // nn)))[:nn]
            rows = np.array([(0, 0, i) for i in nodes], np.int32)
            t2 = time.perf_counter()
            for h in heads:
                kp, vp, kt, vt = kvs[h // G]
                orc.tree_attn_rows(qh[h], kp, vp, np.arange(npg, dtype=np.int32)[None], ctx[b:b + 1], kt, vt, mask[None], rows)
            t3 = time.perf_counter()
            lr = W.logits_rows(cfg, b, np.arange(n))        # input preparation, not counted
            t4 = time.perf_counter()
            tgt = np.full(T, -1, np.int32)
            tgt[:n] = orc.argmax_rows(lr)
            orc.accept(tok, par, dep, n, tgt, cfg.max_depth)
            t5 = time.perf_counter()
            t_total += (t1 - t0) + (t3 - t2) * (cfg.n_q_heads / nh) * (n / len(nodes)) + (t5 - t4)
            tok_total += n
    per_step_tokens = tok_total / (nb * steps) * B
    per_step_seconds = t_total / (nb * steps) * B          # one thread walks the batch sequence by sequence
    sample = ("%d of %d sequences x %d steps; update, draft, arg-max and acceptance whole; attention on %d of %d q heads%s, "
              "its time scaled by heads%s (an extrapolation by flop count); step time scaled by sequences; single thread"
              % (nb, B, steps, nh, cfg.n_q_heads, (" and %d of %d nodes" % (min(nn, T), T)) if full_trees else "",
                 " and nodes" if full_trees else ""))
    return per_step_tokens, per_step_seconds, sample


def run_reference(args, rank, world):
    """The oracle, as it stands, timed on the host cores (single thread) on a bounded sample of the step."""
    if rank != 0:
        return
    import workloads as W
    cfg = W.get_config(args.config or HEADLINE)
    ctx = W.ctx_lens(cfg)
    toks, lens = W.make_streams(cfg, ctx)
    bt, num_pages = W.make_block_table(cfg, ctx)
    steps = max(1, min(args.steps, 3))
    full = not args.drafted_headline
    tokens, seconds, sample = oracle_sample(cfg, ctx, toks, lens, bt, steps, full)
    val = tokens / seconds
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps, "warmup": 0,
        "ms_per_step": 1e3 * seconds, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "batch": cfg.batch, "tree_cap": cfg.max_nodes, "trees": "synthetic full" if full else "drafted"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


# --------------------------------------------------------------------------------------------------------
def closed_loop(args, cfg, ctx, toks, lens, tensors, device, frozen):
    """The decoding loop with the token stream as the target model, wholly on the device: every step is cb_update_draft_tree
    -> cb_tree_attn -> (target ids: the stream's continuation along matching paths) -> cb_accept -> cb_kv_commit, and the
    sequences advance by what was accepted plus the bonus token.  32 steps in one CUDA graph.  Returns mean accepted tokens
    per step (bonus token included), whether every emitted token equals the stream (speculative decoding is lossless), and
    the step time."""
    import torch
    import workloads as W
    from workloads import device as wdev
    from workloads.tensors import TID
    from paper_2511_21699_b200 import Cacheback
    q, kt, vt, toks_d, out, logits = tensors
    B, T, Dm = cfg.batch, cfg.max_nodes, cfg.max_depth
    KC = 32
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device)
    margin = 4 * KC * (Dm + 1) + 16                         # room for the cache to grow (up to four replays of the graph)
    prefill = np.minimum(ctx + 1, lens).astype(np.int32)
    assert int((lens - prefill).min()) > KC * (Dm + 1) + Dm + 2, "stream too short for the closed loop"
    from dataclasses import replace
    bt, num_pages = W.make_block_table(replace(cfg, ctx_range=(cfg.ctx_range[0], cfg.ctx_range[1] + margin)), ctx + margin)
    pshape = (num_pages, cfg.page_size, cfg.n_kv_heads, cfg.head_dim)
    kp = wdev.fill_normal(torch.empty(pshape, dtype=torch.bfloat16, device=device), cfg.seed + 5, TID.K_POOL)
    vp = wdev.fill_normal(torch.empty(pshape, dtype=torch.bfloat16, device=device), cfg.seed + 5, TID.V_POOL)
    bt_d, ctx0, pre_d, zeros_d = dev(bt), dev(ctx), dev(prefill), dev(np.zeros(B, np.int32))
    cb = Cacheback.from_config(cfg, device=device, flags=args.flags)
    if frozen is not None:
        cb.cb_frozen_attach(frozen)
    tree, res = cb.alloc_tree(), cb.alloc_accept()
    i32 = dict(dtype=torch.int32, device=device)
    tgt = torch.empty(B, T, **i32)
    pos_old, pos, ctx_d = torch.empty(B, **i32), torch.empty(B, **i32), torch.empty(B, **i32)
    log_acc, log_tok, log_n = torch.zeros(KC, B, **i32), torch.zeros(KC, B, Dm + 1, **i32), torch.zeros(KC, B, **i32)
    max_ctx = int(ctx.max()) + margin

    def reset():
        cb.cb_reset()
        cb.cb_update_bulk(toks_d, zeros_d, pre_d)          # prompt initialisation
        pos_old.copy_(pre_d); pos.copy_(pre_d); ctx_d.copy_(ctx0)

    def step(s):
        cb.cb_update_draft_tree(toks_d, pos_old, pos, tree)
        cb.cb_tree_attn(q, kp, vp, bt_d, ctx_d, kt, vt, tree["mask"], tree["n_nodes"], out=out, max_ctx=max_ctx)
        wdev.stream_targets(toks_d, pos, tree, cfg.vocab, tgt)
        cb.cb_accept(tree, target_ids=tgt, res=res)
        cb.cb_kv_commit(kp, vp, bt_d, ctx_d, kt, vt, res["n_accept"], res["accept_nodes"])
        log_acc[s].copy_(res["n_accept"]); log_tok[s].copy_(res["out_tokens"]); log_n[s].copy_(tree["n_nodes"])
        pos_old.copy_(pos)
        pos.add_(res["n_accept"]).add_(1)

    # The same loop with the target's choice handed over as logits (its arg-max planted in the rows, the stand-in for an LM
    # head): once with the calls of the loop above, once with cb_accept_update_draft_tree, which takes acceptance, the
    # append to the history, the update and the next draft in one launch.  Both read the logits; only the launches differ.
    saved = torch.empty(B, T, dtype=torch.float32, device=device)
    seq_len = torch.empty(B, **i32)

    def reset_logits_loop():
        reset()
        seq_len.copy_(pre_d)
        cb.cb_draft_tree(toks_d, seq_len, tree)

    def step_logits(fused):
        cb.cb_tree_attn(q, kp, vp, bt_d, ctx_d, kt, vt, tree["mask"], tree["n_nodes"], out=out, max_ctx=max_ctx)
        wdev.stream_targets(toks_d, seq_len, tree, cfg.vocab, tgt)
        wdev.plant_logits(logits, tgt, tree["n_nodes"], saved)
        if fused:
            log_n_one.copy_(tree["n_nodes"])                 # the verified tree's sizes are overwritten by the next draft
            cb.cb_accept_update_draft_tree(tree, logits, toks_d, seq_len, res=res)
            wdev.plant_logits(logits, tgt, log_n_one, saved, restore=True)
        else:
            cb.cb_accept(tree, logits=logits, res=res)
            wdev.plant_logits(logits, tgt, tree["n_nodes"], saved, restore=True)
        cb.cb_kv_commit(kp, vp, bt_d, ctx_d, kt, vt, res["n_accept"], res["accept_nodes"])
        log_emit.add_(res["n_accept"]).add_(1)
        if not fused:
            pos_old.copy_(seq_len)
            seq_len.add_(res["n_accept"]).add_(1)
            cb.cb_update_draft_tree(toks_d, pos_old, seq_len, tree)

    log_n_one, log_emit = torch.empty(B, **i32), torch.zeros(B, **i32)

    def time_logits_loop(fused):
        reset_logits_loop()
        step_logits(fused)
        stream.synchronize()
        gl = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gl, stream=stream):
            for s in range(KC):
                step_logits(fused)
        reset_logits_loop()
        gl.replay()
        reset_logits_loop()
        log_emit.zero_()
        stream.synchronize()
        e0.record(stream)
        gl.replay()
        e1.record(stream)
        stream.synchronize()
        emitted = log_emit.cpu().numpy().astype(np.int64)
        ok = bool(np.array_equal(seq_len.cpu().numpy().astype(np.int64), prefill.astype(np.int64) + emitted))
        return e0.elapsed_time(e1) / KC, float(emitted.sum()) / (KC * B), ok

    stream = torch.cuda.Stream(device=device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        reset()
        step(0)                                             # eager, so that every kernel is loaded before the capture
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for s in range(KC):
                step(s)
        room = int((lens - prefill).min()) - Dm - 2
        replays = int(max(1, min(4, room // (KC * (Dm + 1)))))   # the loop goes on from where the last replay left it
        reset()
        g.replay()                                          # warms the graph up
        reset()
        stream.synchronize()
        ms, accs, toks_out, nns = 0.0, [], [], []
        for rep_ in range(replays):
            e0.record(stream)
            g.replay()
            e1.record(stream)
            stream.synchronize()
            ms += e0.elapsed_time(e1)
            accs.append(log_acc.cpu().numpy()); toks_out.append(log_tok.cpu().numpy()); nns.append(log_n.cpu().numpy())
        ms_sep, mat_sep, ok_sep = time_logits_loop(False)
        ms_fused, mat_fused, ok_fused = time_logits_loop(True)
    st, _ = cb.cb_poll_status()
    assert st == 0, "device status %d in the closed loop" % st
    acc, tok, nn = np.concatenate(accs), np.concatenate(toks_out), np.concatenate(nns)
    steps = KC * replays
    lossless = True
    for b in range(B):
        p0 = int(prefill[b])
        emitted = np.concatenate([tok[s, b, :acc[s, b] + 1] for s in range(steps)])
        lossless = lossless and bool(np.array_equal(emitted, toks[b, p0:p0 + len(emitted)]))
    steps_tokens = float((acc + 1).sum())
    return {"steps": steps, "steps_per_graph": KC, "ms_per_step": ms / steps, "mat": steps_tokens / (steps * B), "lossless": lossless,
            "mat_definition": "tokens emitted per step and sequence: accepted draft tokens plus the bonus token",
            "mean_tree_nodes": float(nn.mean()), "tree_tokens_per_s": float(nn.sum()) / (ms * 1e-3),
            "emitted_tokens_per_s": steps_tokens / (ms * 1e-3),
            "calls": "cb_update_draft_tree, cb_tree_attn, stream targets (workloads), cb_accept (ids), cb_kv_commit; positions advance on the device",
            "paper_mat_context": {"no_frozen": 1.96, "dual": 2.42, "source": "Table 1, Vicuna 7B on SpecBench, 1x RTX 4090 (context only: other model, other data)"},
            "frozen_table": frozen is not None,
            "with_logits": {"steps": KC, "ms_per_step_separate_calls": ms_sep, "ms_per_step_fused_call": ms_fused, "mat_separate": mat_sep,
                            "mat_fused": mat_fused, "lengths_consistent": ok_sep and ok_fused,
                            "separate_calls": "cb_tree_attn, stream targets + planting (workloads), cb_accept (logits), cb_kv_commit, cb_update_draft_tree",
                            "fused_call": "cb_tree_attn, stream targets + planting (workloads), cb_accept_update_draft_tree, cb_kv_commit"}}


def measure(args, cfg_name, rank, world, device, headline):
    """Everything measured on one configuration.  Returns the record; a headline record also carries the pieces of the
    top-level line (keys that start with an underscore: whole-job value, end-to-end figure, launch count)."""
    import torch
    import workloads as W
    from workloads import device as wdev
    from workloads.tensors import TID
    from paper_2511_21699_b200 import Cacheback
    from dataclasses import replace

    if world > 1:
        import torch.distributed as dist
    cfg = replace(W.get_config(cfg_name), seed=rank)        # every rank has its own batch of sequences
    B, T = cfg.batch, cfg.max_nodes
    ctx = W.ctx_lens(cfg)
    toks, lens = W.make_streams(cfg, ctx)
    bt, num_pages = W.make_block_table(cfg, ctx)
    K, Wm = args.steps, max(args.warmup, 3)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device)
    bf = torch.bfloat16
    pk = peaks()

    # Rotate through R copies of the streamed tensors so that no step finds its inputs in the 126 MB L2.
    pool_bytes = num_pages * cfg.page_size * cfg.n_kv_heads * cfg.head_dim * 2 * 2
    logit_bytes = B * T * cfg.vocab * 4
    R = int(min(8, max(1, -(-3 * 126e6 // (pool_bytes + logit_bytes)))))
    pshape = (num_pages, cfg.page_size, cfg.n_kv_heads, cfg.head_dim)
    kps = [wdev.fill_normal(torch.empty(pshape, dtype=bf, device=device), cfg.seed + 17 * r, TID.K_POOL) for r in range(R)]
    vps = [wdev.fill_normal(torch.empty(pshape, dtype=bf, device=device), cfg.seed + 17 * r, TID.V_POOL) for r in range(R)]
    lgs = [wdev.fill_normal(torch.empty((B, T, cfg.vocab), dtype=torch.float32, device=device), cfg.seed + 17 * r, TID.LOGITS)
           for r in range(R)]
    q = wdev.fill_normal(torch.empty((B, T, cfg.n_q_heads, cfg.head_dim), dtype=bf, device=device), cfg.seed, TID.Q)
    kt = wdev.fill_normal(torch.empty((B, T, cfg.n_kv_heads, cfg.head_dim), dtype=bf, device=device), cfg.seed, TID.K_TREE)
    vt = wdev.fill_normal(torch.empty((B, T, cfg.n_kv_heads, cfg.head_dim), dtype=bf, device=device), cfg.seed, TID.V_TREE)
    bt_d, ctx_d, toks_d = dev(bt), dev(ctx), dev(toks)
    out = torch.empty_like(q)
    max_ctx = int(ctx.max())

    cb = Cacheback.from_config(cfg, device=device, flags=args.flags)
    prefill = np.minimum(ctx + 1, lens).astype(np.int32)
    total = 3 * (Wm + K) + 8
    assert int((lens - prefill).min()) > ADVANCE * total + T, "stream too short for this many steps"
    n_old = dev(np.stack([prefill + ADVANCE * s for s in range(total)]).astype(np.int32))
    n_new = dev(np.stack([prefill + ADVANCE * (s + 1) for s in range(total)]).astype(np.int32))
    zeros_d, prefill_d = dev(np.zeros(B, np.int32)), dev(prefill)

    stream = torch.cuda.Stream(device=device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn, reps=3):
        tt = []
        for _ in range(reps):
            e0.record(stream)
            fn()
            e1.record(stream)
            stream.synchronize()
            tt.append(e0.elapsed_time(e1))
        return float(np.median(tt))

    with torch.cuda.stream(stream):
        # ---- prompt initialisation (the bulk form of cb_update), timed on its own: the tables start empty each time
        # with scratch attached (the order-free path) and without (warps by leader); the last run leaves the tables filled
        windows = float(np.sum(np.maximum(prefill.astype(np.int64) - cfg.LL - cfg.FL + 1, 0)))
        bulk_ms, bulk_plain_ms = [], []
        for with_scratch, acc in ((False, bulk_plain_ms), (True, bulk_ms)):
            scratch_bytes = cb.cb_bulk_scratch_attach(int(windows) if with_scratch else 0)
            for rep in range(3):
                cb.cb_reset()
                stream.synchronize()
                e0.record(stream)
                cb.cb_update_bulk(toks_d, zeros_d, prefill_d)
                e1.record(stream)
                stream.synchronize()
                acc.append(e0.elapsed_time(e1))
        cb.cb_bulk_scratch_attach(0)
    entry_bytes = (cfg.LL + 1 + cfg.FC * (cfg.FL + 1)) * 4
    bulk_bytes = windows * (entry_bytes + (cfg.FL + 2) * 4)
    bulk_t = float(np.median(bulk_ms)) * 1e-3
    bulk = {"ms": 1e3 * bulk_t, "windows": windows, "windows_per_s": windows / bulk_t, "algorithmic_bytes": bulk_bytes,
            "bytes_per_window": entry_bytes + (cfg.FL + 2) * 4, "gbs": bulk_bytes / bulk_t / 1e9,
            "frac_of_hbm": bulk_bytes / bulk_t / 1e9 / pk["hbm_gbs"], "scratch_bytes": scratch_bytes,
            "path": "order-free (scratch attached: one thread per window, one warp per distinct leader)",
            "ms_without_scratch": float(np.median(bulk_plain_ms))}

    frozen_info, ft = None, None
    if args.frozen > 0:
        # Stand-in for the paper's corpus sample: streams of the workload's own token distribution under other seeds.
        from paper_2511_21699_b200 import FrozenTable
        nseg = max(1, args.frozen // (1 << 20))
        corpus = dev(np.concatenate([W.make_stream(cfg, 1000 + k, args.frozen // nseg) for k in range(nseg)]).astype(np.int32))
        ft = FrozenTable(cfg.LL, cfg.FL, 1 << 16, min(16, 2 * cfg.FC), device=device)
        ft.cb_frozen_build(corpus)                            # warm-up build
        fe0, fe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        fe0.record()
        ft.cb_frozen_build(corpus)
        fe1.record()
        torch.cuda.synchronize()
        cb.cb_frozen_attach(ft)
        frozen_info = {"corpus_tokens": int(corpus.numel()), "LC": 1 << 16, "FC": min(16, 2 * cfg.FC),
                       "leaders": int(len(ft.cb_frozen_dump()[0])), "build_ms": fe0.elapsed_time(fe1)}

    trees = [cb.alloc_tree() for _ in range(total)]         # every step keeps its own tree, so later passes can reuse it
    res = cb.alloc_accept()
    rtrees = [W.random_tree(cfg.seed, b, T, cfg.max_depth, T) for b in range(B)]
    fpar, fdep = np.stack([t[0] for t in rtrees]), np.stack([t[1] for t in rtrees])
    ftree = dict(tokens=dev(np.maximum(fpar, 0)), parent=dev(fpar), depth=dev(fdep), mask=dev(ancestor_masks(fpar).view(np.int32)),
                 n_nodes=dev(np.full(B, T, np.int32)))
    full_pairs = float(np.sum(fdep + 1))                    # node-ancestor pairs of the synthetic full trees (self included)

    def front(s):
        if args.separate_calls:
            cb.cb_update(toks_d, n_old[s], n_new[s])
            cb.cb_draft_tree(toks_d, n_new[s], trees[s])
        else:
            cb.cb_update_draft_tree(toks_d, n_old[s], n_new[s], trees[s])

    def step(s, full):
        r = s % R
        front(s)
        at = ftree if full else trees[s]
        cb.cb_tree_attn(q, kps[r], vps[r], bt_d, ctx_d, kt, vt, at["mask"], at["n_nodes"], out=out, max_ctx=max_ctx)
        cb.cb_accept(at, logits=lgs[r], res=res)

    def one_call(which, s):
        r = s % R
        tr = trees[s]
        if which == "cb_update":
            cb.cb_update(toks_d, n_old[s], n_new[s])
        elif which == "cb_draft_tree":
            cb.cb_draft_tree(toks_d, n_new[s], tr)
        elif which == "cb_update_draft_tree":
            cb.cb_update_draft_tree(toks_d, n_old[s], n_new[s], tr)
        elif which == "cb_tree_attn":
            cb.cb_tree_attn(q, kps[r], vps[r], bt_d, ctx_d, kt, vt, ftree["mask"], ftree["n_nodes"], out=out, max_ctx=max_ctx)
        elif which == "cb_tree_attn_drafted":
            cb.cb_tree_attn(q, kps[r], vps[r], bt_d, ctx_d, kt, vt, tr["mask"], tr["n_nodes"], out=out, max_ctx=max_ctx)
        elif which == "cb_accept":
            cb.cb_accept(ftree, logits=lgs[r], res=res)
        else:
            cb.cb_accept(tr, logits=lgs[r], res=res)

    rec = {"workload": cfg_name}
    with torch.cuda.stream(stream):
        for s in range(Wm):                                  # eager warm-up (also sets kernel attributes)
            step(s, s % 2 == 0)
        stream.synchronize()
        # The K timed steps are captured once into a CUDA graph: at batch 1 a step is a handful of microsecond-scale
        # kernels and host launch cost would otherwise dominate.  The two graphs (full trees, drafted trees) walk
        # disjoint step indices of the token streams.
        graphs = {}
        for full, base in ((True, Wm), (False, Wm + K)):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for s in range(base, base + K):
                    step(s, full)
            graphs[full] = g
        launches0 = cb.launch_count()
        for s in range(Wm, Wm + K):                          # same sequence eagerly, to count launches
            step(s, True)
        launches = cb.launch_count() - launches0
        stream.synchronize()
        if world > 1:
            dist.barrier()
        sampler = ClockSampler(device.index or 0)
        sampler.start()
        torch.cuda.synchronize()
        step_ms, reps_used = {}, {}
        for full in (True, False):
            times = []
            reps = 3
            while len(times) < reps:
                e0.record(stream)
                graphs[full].replay()
                e1.record(stream)
                stream.synchronize()
                times.append(e0.elapsed_time(e1))
                if len(times) == 3:
                    # keep replaying until the timed region spans about 0.4 s, so that the clock sampler sees it
                    reps = int(min(400, max(3, 400.0 / max(float(np.median(times)), 1e-3))))
            step_ms[full] = float(np.median(times)) / K
            reps_used[full] = reps
        nn_drafted = torch.stack([t["n_nodes"] for t in trees[Wm + K:Wm + 2 * K]]).cpu().numpy().astype(np.float64)
        # Per-call times, for the roofline of the dominant kernel: each call is captured K times back to back in a graph of
        # its own (inputs rotating as in the step) and the replay is timed with events on this stream.  Eager launches
        # would measure the host's enqueue cost at batch 1, not the kernels.
        base = 2 * (Wm + K)
        for s in range(base, base + K):                      # one eager pass leaves valid trees for every step index
            step(s, False)
        stream.synchronize()
        per_call = {}
        for which in ("cb_update", "cb_draft_tree", "cb_update_draft_tree", "cb_tree_attn", "cb_tree_attn_drafted", "cb_accept",
                      "cb_accept_drafted"):
            gc = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gc, stream=stream):
                for s in range(base, base + K):
                    one_call(which, s)
            per_call[which] = timed(gc.replay) / K
            del gc
        nn_percall = torch.stack([t["n_nodes"] for t in trees[base:base + K]]).cpu().numpy().astype(np.float64)
        clocks = sampler.stop()
    del graphs

    nn_full = np.full(B, float(T))
    nn_mean = nn_percall.mean(axis=0)                        # trees of the steps the per-call graphs ran
    roof_full = attn_roofline(cfg, ctx, nn_full, full_pairs, per_call["cb_tree_attn"], pk)
    # the drafter reports no depths here: 4 ancestors per node stand in for the drafted trees' mean
    roof_drafted = attn_roofline(cfg, ctx, nn_mean, float(np.sum(nn_mean * 4)), per_call["cb_tree_attn_drafted"], pk)
    traffic, traffic_source = None, "none: no ncu capture of the kernel sources as they are now"
    if ATTN_TRAFFIC["sources_sha1"] == attn_sources_sha1() and cfg_name in ATTN_TRAFFIC["bytes_per_launch"]:
        traffic = ATTN_TRAFFIC["bytes_per_launch"][cfg_name]
        traffic_source = ATTN_TRAFFIC["source"][cfg_name] + " (ncu dram__bytes_read.sum + dram__bytes_write.sum; kernel sources hash-matched)"
    elif ATTN_TRAFFIC["sources_sha1"] == attn_sources_sha1() and cfg_name in ATTN_TRAFFIC["scaled"]:
        traffic, traffic_source = ATTN_TRAFFIC["scaled"][cfg_name]
    roof_full.update({"traffic": traffic, "traffic_source": traffic_source,
                      "kernel": "cb_tree_attn (attention kernel, plus its merge pass where the launch is not in cluster mode)"})
    acc_bytes_full, acc_bytes_dr = float(B * T) * cfg.vocab * 4, float(np.sum(nn_mean)) * cfg.vocab * 4
    accept = {"gbs": acc_bytes_full / (per_call["cb_accept"] * 1e-3) / 1e9, "algorithmic_bytes": acc_bytes_full,
              "ms_per_launch": per_call["cb_accept"],
              "gbs_drafted_trees": acc_bytes_dr / (per_call["cb_accept_drafted"] * 1e-3) / 1e9}
    accept["frac_of_hbm"] = accept["gbs"] / pk["hbm_gbs"]
    accept["frac_of_hbm_drafted_trees"] = accept["gbs_drafted_trees"] / pk["hbm_gbs"]
    tok_full, tok_dr = float(B * T), float(nn_drafted.sum()) / K
    rec.update({
        "batch": B, "tree_cap": T, "context": [int(ctx.min()), int(ctx.max())],
        "ms_per_step": step_ms[True], "ms_per_step_drafted_trees": step_ms[False],
        "value_full_trees": tok_full / (step_ms[True] * 1e-3), "value_drafted_trees": tok_dr / (step_ms[False] * 1e-3),
        "mean_tree_nodes_drafted": float(nn_drafted.mean()),
        "per_call_ms": per_call, "roofline": roof_full, "roofline_drafted_trees": roof_drafted, "accept": accept,
        "prompt_ingest": bulk, "clocks": clocks,
        "l2": "rotating %d copies of K/V pool and logits (%.0f MB)" % (R, R * (pool_bytes + logit_bytes) / 1e6),
        "replays": reps_used[True]})
    if B == 1:
        rec["latency_bound"] = ("at batch 1 cb_update, cb_draft_tree and cb_accept move a few KB to a few MB per call through chains "
                                "of dependent memory round trips: their time is launch plus round trips, not bandwidth")

    def run_closed_loop():
        if args.no_closed_loop or world > 1:
            return
        lg0 = lgs[0]
        kps.clear(); vps.clear(); lgs.clear()              # the loop brings its own pool (with room to grow) and keeps one copy of the logits
        torch.cuda.empty_cache()
        rec["closed_loop"] = closed_loop(args, cfg, ctx, toks, lens, (q, kt, vt, toks_d, out, lg0), device, ft)

    if not headline:
        st, counters = cb.cb_poll_status()
        assert st == 0, "device status %d" % st
        run_closed_loop()
        return rec

    # ---- whole-job figures over ranks
    full = not args.drafted_headline
    seconds, tokens = step_ms[full] * 1e-3, (tok_full if full else tok_dr)
    if world > 1:
        seconds, tokens = reduce_over_ranks(seconds, tokens, device)
    rec["_value"], rec["_ms_per_step"], rec["_launches"], rec["_frozen"] = tokens / seconds, seconds * 1e3, int(launches), frozen_info

    # ---- end to end through the public API with host buffers: H2D of the step's inputs, D2H of its result
    if not args.no_e2e:
        pin = lambda t: t.cpu().pin_memory()
        hq, hkt, hvt, hlg = pin(q), pin(kt), pin(vt), pin(lgs[0])
        h_old, h_new = pin(n_old), pin(n_new)
        dq, dkt, dvt, dlg = torch.empty_like(q), torch.empty_like(kt), torch.empty_like(vt), lgs[0]
        d_old, d_new = torch.empty(B, dtype=torch.int32, device=device), torch.empty(B, dtype=torch.int32, device=device)
        h_acc = torch.empty(B, dtype=torch.int32).pin_memory()
        h_out = torch.empty(B, cfg.max_depth + 1, dtype=torch.int32).pin_memory()
        h_nn = torch.empty(B, dtype=torch.int32).pin_memory()
        h2d = sum(t.numel() * t.element_size() for t in (hq, hkt, hvt, hlg)) + 2 * B * 4
        d2h = (h_acc.numel() + h_out.numel() + h_nn.numel()) * 4
        s0 = 2 * (Wm + K) + K
        ke = int(max(3, min(K, total - s0 - 2, 2000.0 / max(step_ms[full] + h2d / 20e6, 1e-3))))     # a couple of seconds of steps
        e2e_tokens = 0.0
        with torch.cuda.stream(stream):
            def e2e_step(s):
                r = s % R
                dq.copy_(hq, non_blocking=True); dkt.copy_(hkt, non_blocking=True); dvt.copy_(hvt, non_blocking=True)
                dlg.copy_(hlg, non_blocking=True)
                d_old.copy_(h_old[s], non_blocking=True); d_new.copy_(h_new[s], non_blocking=True)
                tr = trees[s]
                if args.separate_calls:
                    cb.cb_update(toks_d, d_old, d_new)
                    cb.cb_draft_tree(toks_d, d_new, tr)
                else:
                    cb.cb_update_draft_tree(toks_d, d_old, d_new, tr)
                at = ftree if full else tr
                cb.cb_tree_attn(dq, kps[r], vps[r], bt_d, ctx_d, dkt, dvt, at["mask"], at["n_nodes"], out=out, max_ctx=max_ctx)
                cb.cb_accept(at, logits=dlg, res=res)
                h_acc.copy_(res["n_accept"], non_blocking=True); h_out.copy_(res["out_tokens"], non_blocking=True)
                h_nn.copy_(at["n_nodes"], non_blocking=True)
                stream.synchronize()
                return float(h_nn.sum())                     # the tree nodes this step verified
            for s in range(s0, s0 + 2):
                e2e_step(s)
            t0 = time.perf_counter()
            for s in range(s0 + 2, s0 + 2 + ke):
                e2e_tokens += e2e_step(s)
            e2e_s = time.perf_counter() - t0
        if world > 1:
            e2e_s, e2e_tokens = reduce_over_ranks(e2e_s, e2e_tokens, device)
        rec["_e2e"] = {"value": e2e_tokens / e2e_s, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                       "ms_per_step": 1e3 * e2e_s / ke, "steps": ke}
        del hq, hkt, hvt, hlg, dq, dkt, dvt
    st, counters = cb.cb_poll_status()
    assert st == 0, "device status %d" % st
    rec["_counters"] = counters
    if not args.no_e2e:
        del dlg
    run_closed_loop()
    if world == 1 and rank == 0 and not args.no_cpu_baseline:
        tokens_c, seconds_c, sample = oracle_sample(cfg, ctx, toks, lens, bt, 2, full)
        rec["_cpu"] = {"value": tokens_c / seconds_c, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample}
    return rec


def run_ours(args, rank, world, local_rank):
    import torch
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    head_name = args.config or HEADLINE
    names = [args.config] if args.config else (FULL_SIZE if world == 1 else [HEADLINE])
    per_config, head = [], None
    for name in names:
        rec = measure(args, name, rank, world, device, name == head_name)
        torch.cuda.empty_cache()
        if name == head_name:
            head = rec
        per_config.append({k: v for k, v in rec.items() if not k.startswith("_")})
    if rank == 0:
        full = not args.drafted_headline
        line = {
            "metric": METRIC, "value": head["_value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": head["_ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": head_name, "batch": head["batch"], "tree_cap": head["tree_cap"],
                       "trees": "synthetic full (%d nodes each)" % head["tree_cap"] if full else "drafted",
                       "value_drafted_trees": head["value_drafted_trees"], "ms_per_step_drafted_trees": head["ms_per_step_drafted_trees"],
                       "mean_tree_nodes_drafted": head["mean_tree_nodes_drafted"], "context": head["context"], "l2": head["l2"],
                       "launch": "CUDA graph of the timed steps, replayed %d times, median" % head["replays"],
                       "frozen_table": head["_frozen"],
                       "calls": ("cb_update, cb_draft_tree" if args.separate_calls else "cb_update_draft_tree") + ", cb_tree_attn, cb_accept",
                       "parallelism": "replicas x%d" % world},
            "clocks": head["clocks"], "gpu_launches": head["_launches"],
            "roofline": head["roofline"], "per_call_ms": head["per_call_ms"], "accept": head["accept"],
            "prompt_ingest": head["prompt_ingest"], "closed_loop": head.get("closed_loop"), "per_config": per_config,
            "counters": head["_counters"],
        }
        if "_e2e" in head:
            line["e2e"] = head["_e2e"]
        if "_cpu" in head:
            line["cpu_baseline"] = head["_cpu"]
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def rank_plumbing_only(rank, world):
    """The rank start-up and result gathering alone, on CPU (gloo): what a test of the multi-rank launch can run without a GPU."""
    import torch
    import torch.distributed as dist
    dist.init_process_group("gloo")
    seconds, units = reduce_over_ranks(0.010 * (rank + 1), 1000.0 + rank, torch.device("cpu"))
    if rank == 0:
        print(json.dumps({"n_gpus": world, "seconds": seconds, "units": units}))
    dist.destroy_process_group()


def main():
    args = parse()
    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.rank_plumbing_only:
        rank_plumbing_only(rank, world)
        return
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if not os.path.exists(os.path.join(ROOT, "paper_2511_21699_b200", "libcacheback.so")):
        import __graft_entry__
        __graft_entry__.build()
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
