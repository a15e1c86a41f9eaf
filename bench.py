#!/usr/bin/env python
"""Benchmark of the Cacheback draft-and-verify step on B200.

A step is one pass of the whole hot path over one batch: cb_update (sliding window over the tokens
accepted by the previous step) -> cb_draft_tree -> cb_tree_attn -> cb_accept (fp32 logits); the first two are
issued as the library's one-launch form cb_update_draft_tree unless --separate-calls is given.  The default
workload is the Llama-2-7B-shaped configuration (batch 1, 32 heads, head_dim 128, context 4,096 in 16-token
pages, tree cap 64).  Inputs are synthetic (seeded generators in workloads/).  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]
"""
import argparse
import json
import os
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


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=48)
    ap.add_argument("--warmup", type=int, default=6)
    ap.add_argument("--config", default="c2_7b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--full-trees", action="store_true", help="attention/acceptance on synthetic full-size trees")
    ap.add_argument("--separate-calls", action="store_true", help="cb_update and cb_draft_tree as two launches")
    ap.add_argument("--frozen", type=int, default=0, metavar="TOKENS",
                    help="attach a frozen table built on the GPU from a synthetic corpus of this many tokens (0 = none)")
    return ap.parse_args()


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one cb_attn_tc_kernel launch, from the ncu capture
# summarised in profiles/cb_attn_tc_kernel_<workload>.md.  It is reported only while the kernel sources still hash to the
# captured ones; after any change to them the figure is stale and `traffic` is null until the capture is redone.
ATTN_TRAFFIC = {"sources_sha1": "940d4a8002e5bcb4876bd7445ef665e14f2a13aa",
                "bytes_per_launch": {"c2_7b": 70.37e6, "c3_8b_gqa": 558.2e6, "c4_13b_turns": 2768.5e6}}


def attn_sources_sha1():
    import hashlib
    h = hashlib.sha1()
    for f in ("cb_attn_tc.cu", "cb_attn.cuh", "cb_attn.cu"):
        with open(os.path.join(ROOT, "paper_2511_21699_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), "measured"
    return 6650.0, 1590.0, "fallback"


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
    return float(4.0 * cfg.n_q_heads * cfg.head_dim * (np.sum(n_nodes * ctx.astype(np.float64)) + pairs))


# --------------------------------------------------------------------------------------------------------
def run_reference(args, rank, world):
    """The oracle, as it stands, timed on the host cores (single thread) on a bounded sample of the step."""
    if rank != 0:
        return
    import workloads as W
    from workloads.tensors import TID
    from oracle import cb_oracle as orc
    cfg = W.get_config(args.config)
    ctx = W.ctx_lens(cfg)
    toks, lens = W.make_streams(cfg, ctx)
    bt, num_pages = W.make_block_table(cfg, ctx)
    B, T = cfg.batch, cfg.max_nodes
    nb = min(B, 2)                                         # sequences per sampled step
    nh = min(cfg.n_q_heads, 4)                             # attention heads per sampled step
    tabs = [orc.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC) for _ in range(nb)]
    pos = np.minimum(ctx + 1, lens)[:nb].astype(np.int64)
    for b in range(nb):
        tabs[b].update(toks[b], 0, int(pos[b]))
    kv = {}
    for b in range(nb):
        npg = (int(ctx[b]) + cfg.page_size - 1) // cfg.page_size
        kp, vp = W.pool_pages_bits(cfg, bt[b, :npg])
        kv[b] = (kp, vp, W.seq_bits(cfg, TID.Q, b, cfg.n_q_heads)[None], W.seq_bits(cfg, TID.K_TREE, b, cfg.n_kv_heads)[None],
                 W.seq_bits(cfg, TID.V_TREE, b, cfg.n_kv_heads)[None], np.arange(npg, dtype=np.int32)[None])
    steps = max(1, min(args.steps, 8))
    warm = min(args.warmup, 1)
    t_total, tok_total = 0.0, 0
    for s in range(warm + steps):
        t_step, n_step = 0.0, 0
        for b in range(nb):
            t0 = time.perf_counter()
            tabs[b].update(toks[b], int(pos[b]), int(pos[b]) + ADVANCE)
            pos[b] += ADVANCE
            n, tok, par, dep, mask = tabs[b].draft_tree(toks[b], int(pos[b]), T, cfg.crt, cfg.max_depth)
            t1 = time.perf_counter()
            kp, vp, q, kt, vt, btl = kv[b]
            rows = np.array([(0, h, i) for h in range(nh) for i in range(n)], np.int32)
            orc.tree_attn_rows(q, kp, vp, btl, ctx[b:b + 1], kt, vt, mask[None], rows)
            t2 = time.perf_counter()
            lr = W.logits_rows(cfg, b, np.arange(n))
            t3 = time.perf_counter()
            tgt = np.full(T, -1, np.int32)
            tgt[:n] = orc.argmax_rows(lr)
            orc.accept(tok, par, dep, n, tgt, cfg.max_depth)
            t4 = time.perf_counter()
            # attention is sampled on nh of Hq heads: scale its time to all heads; logits generation (t2..t3) is input
            # preparation and is not counted
            t_step += (t1 - t0) + (t2 - t1) * (cfg.n_q_heads / nh) + (t4 - t3)
            n_step += n
        if s >= warm:
            t_total += t_step * (B / nb)                   # one thread walks the batch sequence by sequence
            tok_total += n_step * (B / nb)
    val = tok_total / t_total
    sample = ("%d of %d sequences, %d of %d q heads per step (attention time scaled by heads, step time by sequences), "
              "%d steps, single thread" % (nb, B, nh, cfg.n_q_heads, steps))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps, "warmup": warm,
        "ms_per_step": 1e3 * t_total / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": cfg.name, "batch": B, "tree_cap": T},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


# --------------------------------------------------------------------------------------------------------
def cpu_baseline(cfg, prob_host, tree_host):
    """Oracle timed on this machine's host cores on a bounded sample of the same workload (rank 0, N = 1)."""
    import workloads as W
    from workloads.tensors import TID
    from oracle import cb_oracle as orc
    ctx, toks, lens, bt = prob_host
    B, T = cfg.batch, cfg.max_nodes
    nb, nh = min(B, 2), min(cfg.n_q_heads, 4)
    t_step, n_tok = 0.0, 0
    for b in range(nb):
        tab = orc.OracleTable(cfg.LL, cfg.FL, cfg.LC, cfg.FC)
        pos = int(min(ctx[b] + 1, lens[b]))
        tab.update(toks[b], 0, pos)
        npg = (int(ctx[b]) + cfg.page_size - 1) // cfg.page_size
        kp, vp = W.pool_pages_bits(cfg, bt[b, :npg])
        q = W.seq_bits(cfg, TID.Q, b, cfg.n_q_heads)[None]
        kt = W.seq_bits(cfg, TID.K_TREE, b, cfg.n_kv_heads)[None]
        vt = W.seq_bits(cfg, TID.V_TREE, b, cfg.n_kv_heads)[None]
        for rep in range(2):
            t0 = time.perf_counter()
            tab.update(toks[b], pos, pos + ADVANCE)
            pos += ADVANCE
            n, tok, par, dep, mask = tab.draft_tree(toks[b], pos, T, cfg.crt, cfg.max_depth)
            t1 = time.perf_counter()
            rows = np.array([(0, h, i) for h in range(nh) for i in range(n)], np.int32)
            orc.tree_attn_rows(q, kp, vp, np.arange(npg, dtype=np.int32)[None], ctx[b:b + 1], kt, vt, mask[None], rows)
            t2 = time.perf_counter()
            lr = W.logits_rows(cfg, b, np.arange(n))
            t3 = time.perf_counter()
            tgt = np.full(T, -1, np.int32)
            tgt[:n] = orc.argmax_rows(lr)
            orc.accept(tok, par, dep, n, tgt, cfg.max_depth)
            t4 = time.perf_counter()
            t_step += (t1 - t0) + (t2 - t1) * (cfg.n_q_heads / nh) + (t4 - t3)
            n_tok += n
    return {"value": n_tok / t_step, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": "%d of %d sequences x 2 steps, %d of %d q heads (attention time scaled by heads); single thread"
                      % (nb, B, nh, cfg.n_q_heads)}


def run_ours(args, rank, world, local_rank):
    import torch
    import workloads as W
    from workloads import device as wdev
    from workloads.tensors import TID
    from paper_2511_21699_b200 import Cacheback

    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    from dataclasses import replace
    cfg = replace(W.get_config(args.config), seed=rank)        # every rank has its own batch of sequences
    B, T = cfg.batch, cfg.max_nodes
    ctx = W.ctx_lens(cfg)
    toks, lens = W.make_streams(cfg, ctx)
    bt, num_pages = W.make_block_table(cfg, ctx)
    K, Wm = args.steps, max(args.warmup, 3)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device)
    bf = torch.bfloat16

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

    cb = Cacheback.from_config(cfg, device=device)
    prefill = np.minimum(ctx + 1, lens).astype(np.int32)
    total = 2 * (Wm + K) + 4
    assert int((lens - prefill).min()) > ADVANCE * total + T, "stream too short for this many steps"
    n_old = dev(np.stack([prefill + ADVANCE * s for s in range(total)]).astype(np.int32))
    n_new = dev(np.stack([prefill + ADVANCE * (s + 1) for s in range(total)]).astype(np.int32))
    cb.cb_update_bulk(toks_d, dev(np.zeros(B, np.int32)), dev(prefill))     # prompt initialisation, untimed
    frozen_info = None
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
    if args.full_trees:
        rtrees = [W.random_tree(cfg.seed, b, T, cfg.max_depth, T) for b in range(B)]
        par, dep = np.stack([t[0] for t in rtrees]), np.stack([t[1] for t in rtrees])
        mask = ancestor_masks(par)
        nn = np.full(B, T, np.int32)
        ftree = dict(tokens=dev(np.maximum(par, 0)), parent=dev(par), depth=dev(dep), mask=dev(mask.view(np.int32)),
                     n_nodes=dev(nn))

    def step(s):
        r = s % R
        tr = trees[s]
        if args.separate_calls:
            cb.cb_update(toks_d, n_old[s], n_new[s])
            cb.cb_draft_tree(toks_d, n_new[s], tr)
        else:
            cb.cb_update_draft_tree(toks_d, n_old[s], n_new[s], tr)
        at = ftree if args.full_trees else tr
        cb.cb_tree_attn(q, kps[r], vps[r], bt_d, ctx_d, kt, vt, at["mask"], at["n_nodes"], out=out, max_ctx=int(ctx.max()))
        cb.cb_accept(at, logits=lgs[r], res=res)

    stream = torch.cuda.Stream(device=device)
    with torch.cuda.stream(stream):
        for s in range(Wm):                                  # eager warm-up (also sets kernel attributes)
            step(s)
        stream.synchronize()
        # The K timed steps are captured once into a CUDA graph: at batch 1 a step is a handful of
        # microsecond-scale kernels and host launch cost would otherwise dominate.
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for s in range(Wm, Wm + K):
                step(s)
        launches0 = cb.launch_count()
        for s in range(Wm, Wm + K):                          # same sequence eagerly, to count launches
            step(s)
        launches = cb.launch_count() - launches0
        stream.synchronize()
        if world > 1:
            dist.barrier()
        sampler = ClockSampler(local_rank)
        sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        times = []
        reps = 3
        while len(times) < reps:
            e0.record(stream)
            g.replay()
            e1.record(stream)
            stream.synchronize()
            times.append(e0.elapsed_time(e1))
            if len(times) == 3:
                # keep replaying until the timed region spans about 0.4 s, so that the clock sampler sees it
                reps = int(min(400, max(3, 400.0 / max(float(np.median(times)), 1e-3))))
        ms_total = float(np.median(times))
        nn_timed = torch.stack([t["n_nodes"] for t in trees[Wm:Wm + K]]).cpu().numpy().astype(np.float64)
        # Per-call times, for the roofline of the dominant kernel: each of the four calls is captured K times back to
        # back in a graph of its own (inputs rotating as in the step) and the replay is timed with events on this stream.
        # Eager launches would measure the host's enqueue cost at batch 1, not the kernels.
        base = Wm + K

        def one_call(which, s):
            r = s % R
            tr = trees[s]
            at = ftree if args.full_trees else tr
            if which == 0:
                cb.cb_update(toks_d, n_old[s], n_new[s])
            elif which == 1:
                cb.cb_draft_tree(toks_d, n_new[s], tr)
            elif which == 2:
                cb.cb_tree_attn(q, kps[r], vps[r], bt_d, ctx_d, kt, vt, at["mask"], at["n_nodes"], out=out, max_ctx=int(ctx.max()))
            elif which == 3:
                cb.cb_accept(at, logits=lgs[r], res=res)
            else:
                cb.cb_update_draft_tree(toks_d, n_old[s], n_new[s], tr)

        for s in range(base, base + K):                      # one eager pass leaves valid trees for every step index
            step(s)
        stream.synchronize()
        per_med = np.zeros(5)
        for which in range(5):
            gc = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gc, stream=stream):
                for s in range(base, base + K):
                    one_call(which, s)
            tt = []
            for _ in range(3):
                e0.record(stream)
                gc.replay()
                e1.record(stream)
                stream.synchronize()
                tt.append(e0.elapsed_time(e1) / K)
            per_med[which] = float(np.median(tt))
            del gc
        nn_percall = torch.stack([t["n_nodes"] for t in trees[base:base + K]]).cpu().numpy().astype(np.float64)
        clocks = sampler.stop()
    nn_attn = (np.full((K, B), float(T)) if args.full_trees else nn_timed)
    if args.full_trees:
        nn_percall = np.full((K, B), float(T))
    tokens = float(nn_attn.sum())
    local_tokens = tokens
    if world > 1:
        ms_total, tokens = reduce_over_ranks(ms_total, tokens, device)
    value = tokens / (ms_total * 1e-3)

    # end to end through the public API with host buffers: H2D of the step's inputs, D2H of its result
    pin = lambda t: t.cpu().pin_memory()
    hq, hkt, hvt, hlg = pin(q), pin(kt), pin(vt), pin(lgs[0])
    h_old, h_new = pin(n_old), pin(n_new)
    dq, dkt, dvt, dlg = torch.empty_like(q), torch.empty_like(kt), torch.empty_like(vt), torch.empty_like(lgs[0])
    d_old, d_new = torch.empty(B, dtype=torch.int32, device=device), torch.empty(B, dtype=torch.int32, device=device)
    h_acc = torch.empty(B, dtype=torch.int32).pin_memory()
    h_out = torch.empty(B, cfg.max_depth + 1, dtype=torch.int32).pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in (hq, hkt, hvt, hlg)) + 2 * B * 4
    d2h = h_acc.numel() * 4 + h_out.numel() * 4
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
            at = ftree if args.full_trees else tr
            cb.cb_tree_attn(dq, kps[r], vps[r], bt_d, ctx_d, dkt, dvt, at["mask"], at["n_nodes"], out=out, max_ctx=int(ctx.max()))
            cb.cb_accept(at, logits=dlg, res=res)
            h_acc.copy_(res["n_accept"], non_blocking=True); h_out.copy_(res["out_tokens"], non_blocking=True)
            stream.synchronize()
        for s in range(Wm, Wm + 3):
            e2e_step(s)
        t0 = time.perf_counter()
        for s in range(Wm, Wm + K):
            e2e_step(s)
        e2e_s = time.perf_counter() - t0
    e2e_tokens = local_tokens
    if world > 1:
        e2e_s, e2e_tokens = reduce_over_ranks(e2e_s, local_tokens, device)
    e2e_val = e2e_tokens / e2e_s

    st, counters = cb.cb_poll_status()
    assert st == 0, "device status %d" % st
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    hbm_peak, tf_peak, peak_kind = peaks()
    nn_mean = nn_percall.mean(axis=0)                       # trees of the steps the per-call graphs ran
    a_bytes = attn_bytes(cfg, ctx, nn_mean)
    attn_ms = float(per_med[2])
    t_mem, t_cmp = a_bytes / (hbm_peak * 1e9), attn_flops(cfg, ctx, nn_mean, float(np.sum(nn_mean * 4))) / (tf_peak * 1e12)
    traffic = ATTN_TRAFFIC["bytes_per_launch"].get(cfg.name) if ATTN_TRAFFIC["sources_sha1"] == attn_sources_sha1() else None
    if t_mem >= t_cmp:
        roof = {"bound": "hbm", "achieved": a_bytes / (attn_ms * 1e-3) / 1e9, "peak": hbm_peak, "unit": "GB/s"}
    else:
        fl = attn_flops(cfg, ctx, nn_mean, float(np.sum(nn_mean * 4)))
        roof = {"bound": "tensor", "achieved": fl / (attn_ms * 1e-3) / 1e12, "peak": tf_peak, "unit": "TFLOP/s"}
    roof.update({"frac": roof["achieved"] / roof["peak"], "traffic": traffic, "kernel": "cb_tree_attn (attention kernel, plus its merge pass where the launch is not in cluster mode)",
                 "ms_per_launch": attn_ms, "peak_source": peak_kind + " (MEASURED_PEAKS.json)" if peak_kind == "measured" else "fallback",
                 "algorithmic_bytes": a_bytes})
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms_total / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "batch": B, "tree_cap": T, "mean_tree_nodes": float(nn_attn.mean()),
                   "context": [int(ctx.min()), int(ctx.max())], "l2": "rotating %d copies of K/V pool and logits (%.0f MB)" %
                   (R, R * (pool_bytes + logit_bytes) / 1e6), "launch": "CUDA graph of the timed steps, replayed %d times, median" % reps,
                   "trees": "synthetic full" if args.full_trees else "drafted", "frozen_table": frozen_info,
                   "calls": ("cb_update, cb_draft_tree" if args.separate_calls else "cb_update_draft_tree") + ", cb_tree_attn, cb_accept",
                   "parallelism": "replicas x%d" % world},
        "clocks": clocks, "gpu_launches": int(launches),
        "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                "ms_per_step": 1e3 * e2e_s / K},
        "roofline": roof,
        "per_call_ms": {"cb_update": float(per_med[0]), "cb_draft_tree": float(per_med[1]), "cb_tree_attn": float(per_med[2]),
                        "cb_accept": float(per_med[3]), "cb_update_draft_tree": float(per_med[4])},
        "accept_gbs": (float(np.sum(nn_mean)) * cfg.vocab * 4) / (float(per_med[3]) * 1e-3) / 1e9,
        "counters": counters,
    }
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(cfg, (ctx, toks, lens, bt), None)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if not os.path.exists(os.path.join(ROOT, "paper_2511_21699_b200", "libcacheback.so")):
        import __graft_entry__
        __graft_entry__.build()
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
