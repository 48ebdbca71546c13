#!/usr/bin/env python
"""Benchmark of the TriSpec verify pass on B200.

One "step" is one whole verify pass (tree mask -> tree-masked GQA attention -> LM-head softmax
statistics -> acceptance scan) over one batch of seeded synthetic input, launched through the
fused C-ABI call. The metric is verified draft tokens per second per verify pass.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints one JSON line (rank 0). With N > 1 (torchrun) every rank runs its own batch of the same
shape (independent sequences, no data-path collective): weak scaling.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "verified_draft_tokens_per_s"
UNIT = "draft tokens/s"
NOMINAL = {"hbm_gbs": 7700.0, "bf16_tflops": 2250.0}     # data-sheet figures, for context beside the measured peaks


def dram_traffic(kernel: str, workload: str):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of `kernel` on `workload`, from the
    tracked record of the last profiler capture, or None when there is no capture or when the kernel's
    sources have changed since it was taken (the record carries their digest)."""
    from paper_2601_23180_b200 import profile_traffic as pt
    return pt.lookup(kernel, workload)


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        for r in self.rows:
            if len(r) < 6:
                continue
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ---------------------------------------------------------------------------------------------
# CPU baseline: the oracle, as it stands, on a bounded sample of the workload
# ---------------------------------------------------------------------------------------------
def oracle_sample(cfg, inp, n_attn_rows: int, n_lm_rows: int, w64_cache=None):
    """Times the oracle on a sample of one verify pass and scales to the whole pass.
    Returns (draft tokens/s, description, threads)."""
    import numpy as np
    from oracle import trispec_oracle as orc
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    seqs = list(range(cfg.B)) if inp.get("seq_index") is None else [int(s) for s in inp["seq_index"]]
    T = cfg.T
    t0 = time.perf_counter()
    mask, _ = orc.build_tree_mask(inp["parent"])
    t_mask = time.perf_counter() - t0
    # attention rows of one (sequence, KV head) group, so that the context is converted once
    G = cfg.Hq // cfg.Hkv
    # whole (sequence, KV head) groups in order, T * G rows each, until n_attn_rows are taken
    samples = []
    for grp in range((n_attn_rows + T * G - 1) // (T * G)):
        b, kvh = seqs[(grp // cfg.Hkv) % len(seqs)], grp % cfg.Hkv
        for i in range(min(T * G, n_attn_rows - len(samples))):
            samples.append((b, i % T, kvh * G + (i // T) % G))
    t0 = time.perf_counter()
    orc.verify_attn(inp["q"], inp["k_tree"], inp["v_tree"], mask, inp["k_cache"], inp["v_cache"], inp["ctx_len"],
                    1.0 / math.sqrt(cfg.D), block_table=inp.get("block_table"), block_size=cfg.block_size,
                    samples=samples)
    t_attn = time.perf_counter() - t0
    total_attn_rows = len(seqs) * T * cfg.Hq
    # LM-head rows: the fp64 copy of W is made once per pass, then one matrix-vector product per row
    # the fp64 copy of W is part of every oracle pass; a caller that times many samples of one
    # workload passes a cache so that the copy is made (and timed) once and its time counted each time
    if w64_cache is not None and "W64" in w64_cache:
        W64, t_w = w64_cache["W64"], w64_cache["t_w"]
    else:
        t0 = time.perf_counter()
        W64 = orc.bf16_to_f64(inp["W"])
        t_w = time.perf_counter() - t0
        if w64_cache is not None:
            w64_cache["W64"], w64_cache["t_w"] = W64, t_w
    t_lm, left = 0.0, n_lm_rows
    for b in seqs:                                  # whole sequences, then a prefix of the next one
        n = min(T, left)
        if n <= 0:
            break
        t0 = time.perf_counter()
        st = orc.lmhead_stats(inp["h"][b:b + 1, :n], inp["W"], inp["parent"][b:b + 1, :n], inp["tok"][b:b + 1, :n],
                              cfg.logit_scale, W64=W64)
        t_lm += time.perf_counter() - t0
        left -= n
    del W64
    t0 = time.perf_counter()
    p1 = np.tile(st["p_top1"][:, :1], (cfg.B, T))
    orc.accept_scan(p1, p1 * 0.1, np.zeros((cfg.B, T), dtype=np.int64), inp["parent"], inp["tok"], cfg.lam, cfg.mode)
    t_scan = time.perf_counter() - t0
    t_pass = (t_mask + t_attn * total_attn_rows / n_attn_rows + t_w + t_lm * (len(seqs) * T) / n_lm_rows + t_scan)
    desc = (f"{n_attn_rows} of {total_attn_rows} attention rows and {n_lm_rows} of {len(seqs) * T} LM-head rows "
            f"(+ full mask, scan, one fp64 copy of W), scaled to one pass; measured {t_mask + t_attn + t_w + t_lm + t_scan:.1f} s")
    return len(seqs) * cfg.k / t_pass, desc, threads


def oracle_timed(cfg, inp, budget_s: float, w64_cache=None):
    """Probe the oracle's per-row cost, then time a sample sized for about `budget_s` seconds
    (the whole pass if it fits)."""
    n_seq = cfg.B if cfg.n_active is None else cfg.n_active
    tot_a, tot_l = n_seq * cfg.T * cfg.Hq, n_seq * cfg.T
    v, _, _ = oracle_sample(cfg, inp, n_attn_rows=min(cfg.T * (cfg.Hq // cfg.Hkv), tot_a), n_lm_rows=min(2, tot_l),
                            w64_cache=w64_cache)
    est_full = n_seq * cfg.k / v
    f = min(1.0, budget_s / est_full)
    G = cfg.Hq // cfg.Hkv
    # whole (sequence, KV head) groups only: the oracle converts a group's context once, so a part of a
    # group would be charged the whole conversion and scale to too slow a pass
    grp = cfg.T * G
    na = max(grp, min(int(f * tot_a) // grp * grp, tot_a))
    nl = max(1, min(int(f * tot_l), tot_l))
    return oracle_sample(cfg, inp, n_attn_rows=na, n_lm_rows=nl, w64_cache=w64_cache)


def run_reference(args, cfg, rank):
    if rank != 0:
        return
    from paper_2601_23180_b200 import inputs as gen
    inp = gen.make_inputs(cfg)
    # The whole run is bounded to about two minutes whatever K and W are: every step times a fresh
    # sample of the pass, sized to its share of that budget (at least a few rows), and scales it to
    # the whole pass. The fp64 copy of W is made and timed once and counted in every step.
    n_steps = args.warmup + args.steps
    cache = {}
    t_start = time.perf_counter()
    per_step = max(0.05, min(8.0, 110.0 / max(n_steps, 1)))
    vals = []
    for step in range(n_steps):
        left = 150.0 - (time.perf_counter() - t_start)
        budget = per_step if left > per_step * (n_steps - step) else max(0.02, left / max(n_steps - step, 1))
        v, desc, threads = oracle_timed(cfg, inp, budget_s=budget, w64_cache=cache)
        if step >= args.warmup:
            vals.append(v)
    value = len(vals) / sum(1.0 / v for v in vals)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * cfg_tokens(cfg) / value,
        # every step times a bounded sample of the pass and scales it to the whole pass: ms_per_step is
        # what one whole pass of the oracle would take, not a time this run spent
        "extrapolated": True, "seconds_measured": time.perf_counter() - t_start,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(cfg),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle (numpy/BLAS)", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
# One kernel alone, L2 flushed before every launch (--only attention | lmhead | scan)
# ---------------------------------------------------------------------------------------------
def _roof(peaks, flops, byts, ms):
    """Roofline record of one launch: the bound is the larger of the two lower-bound times."""
    tensor_bound = flops / (peaks["bf16_tflops"] * 1e12) > byts / (peaks["hbm_gbs"] * 1e9)
    r = ({"bound": "tensor", "achieved": flops / ms / 1e9, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
          "work_per_launch": flops} if tensor_bound else
         {"bound": "hbm", "achieved": byts / ms / 1e6, "peak": peaks["hbm_gbs"], "unit": "GB/s",
          "work_per_launch": byts})
    r.update({"frac": r["achieved"] / r["peak"], "ms_per_launch": ms, "traffic": None,
              "hbm_gbs": byts / ms / 1e6, "tflops": flops / ms / 1e9,
              "peak_source": f"{peaks['source']} (burst: the kernel is timed alone)"})
    return r


def _scan_stress_inputs(cfg, B):
    """2^20-sequence input of the scan kernels: the workload's tree generator (1024 distinct
    trees, tiled), statistics synthesised on the device: the top-1 of a node is the token of
    its first child (so that walks go on) or a random token; about a quarter of the nodes
    fail the margin test."""
    import numpy as np
    import torch
    from paper_2601_23180_b200 import inputs as gen
    T = cfg.T
    trees = np.stack([gen.make_tree(cfg, b) for b in range(1024)])
    toks = np.stack([gen.make_tokens(cfg, b, trees[b]) for b in range(1024)])
    parent = torch.from_numpy(trees).cuda().repeat(B // 1024, 1).contiguous()
    tok = torch.from_numpy(toks.astype(np.int32)).cuda().repeat(B // 1024, 1).contiguous()
    g = torch.Generator(device="cuda").manual_seed(cfg.seed)
    first_child = np.full((1024, T), -1, dtype=np.int64)
    for b in range(1024):
        for c in range(T - 1, 0, -1):
            first_child[b, trees[b, c]] = c
    fc = torch.from_numpy(first_child).cuda().repeat(B // 1024, 1)
    rnd = torch.randint(0, cfg.V, (B, T), generator=g, device="cuda", dtype=torch.int32)
    top1 = torch.where(fc >= 0, torch.gather(tok, 1, fc.clamp(min=0)), rnd).to(torch.int32).contiguous()
    p1 = 0.5 + 0.5 * torch.rand((B, T), generator=g, device="cuda")
    p1 = torch.where(torch.rand((B, T), generator=g, device="cuda") < 0.15, p1 * 0.5, p1).contiguous()
    p2 = (0.1 * torch.rand((B, T), generator=g, device="cuda")).contiguous()
    return parent, tok, {"p_top1": p1, "p_top2": p2, "top1_idx": top1}


def run_only(args, cfg):
    """Times one entry point by itself: every call bracketed by CUDA events on its stream, a
    buffer larger than L2 zeroed before each call; prints one JSON line with that kernel's
    roofline. `scan` runs the scan-only stress input (2^20 sequences), where HBM, not launch
    latency, bounds the integer kernels."""
    import dataclasses
    import numpy as np
    import torch
    from paper_2601_23180_b200 import binding as ts
    from paper_2601_23180_b200 import inputs as gen
    from paper_2601_23180_b200 import runner
    torch.cuda.set_device(0)
    peaks = _peaks()
    stream = torch.cuda.current_stream()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    n = max(3, min(args.steps, 200))

    out = {"only": args.only, "metric": METRIC, "unit": UNIT, "n_gpus": 1, "steps": n, "data": "synthetic",
           "config": {"workload": cfg.name, "l2": "256 MB buffer zeroed before every timed call"}}

    def timed(fn, bytes_touched=0.0):
        """Median time of one call. A call that streams more than twice the L2 capacity evicts its
        own data: such calls are timed back to back inside one pair of events; smaller ones are
        bracketed one by one with the flush buffer zeroed before each."""
        for _ in range(max(args.warmup, 3)):
            fn()
        if bytes_touched > 2 * 126e6:
            out["config"]["l2"] = "inputs larger than L2; calls back to back inside one pair of events"
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record(stream)
            for _ in range(n):
                fn()
            e1.record(stream)
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / n
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        for s_, e_ in evs:
            flush.zero_()
            s_.record(stream)
            fn()
            e_.record(stream)
        torch.cuda.synchronize()
        return statistics.median(s_.elapsed_time(e_) for s_, e_ in evs)

    n_seq = cfg.B if cfg.n_active is None else cfg.n_active
    if args.only == "scan":
        B, T = 1 << 20, cfg.T
        parent, tok, stats = _scan_stress_inputs(cfg, B)
        so = ts.alloc_scan_out(B, T)
        sa = ts.scan_args(stats, parent, tok, cfg.lam, gen.MODE_PROXY, so)
        so_nc = {k: v for k, v in so.items() if k not in ("esc_index", "n_escalated")}
        sa_nc = ts.scan_args(stats, parent, tok, cfg.lam, gen.MODE_PROXY, so_nc)
        mask = torch.zeros((B, T), dtype=torch.int64, device="cuda")
        depth = torch.zeros((B, T), dtype=torch.int32, device="cuda")
        ta = ts.tree_args(parent, mask, depth)
        ms_both = timed(lambda: ts.trispec_accept_scan(sa), B * (T * 24 + 22))
        ms_scan = timed(lambda: ts.trispec_accept_scan(sa_nc), B * (T * 24 + 17))
        ms_mask = timed(lambda: ts.trispec_build_tree_mask(ta), B * T * 16)
        # per sequence: parent, tok, top1_idx, p_top1, p_top2 (4 B per node, each read once); outputs: path
        # (4 B per node), accept_len, bonus, last_node, near_thr (4 B each), escalate (1 B); the compaction
        # adds 1 B read and 4 B written per sequence; the mask kernel reads 4 B and writes 12 B per node
        scan_bytes, compact_bytes, mask_bytes = B * (T * 24 + 17), B * 5, B * T * 16
        hb = peaks["hbm_gbs"]
        out.update({
            "config": {"workload": f"scan stress: 2^20 sequences of the {cfg.name} tree shape", "T": T,
                       "mean_accept_len": so["accept_len"].float().mean().item(),
                       "escalated": int(so["n_escalated"].item()),
                       "l2": "inputs larger than L2; calls back to back inside one pair of events"},
            "value": B * cfg.k / (ms_scan * 1e-3), "ms_per_step": ms_scan, "dtype": "int32",
            "roofline": {"kernel": "accept_scan_kernel", "bound": "hbm", "achieved": scan_bytes / ms_scan / 1e6,
                         "peak": hb, "unit": "GB/s", "frac": scan_bytes / ms_scan / 1e6 / hb,
                         "work_per_launch": scan_bytes, "ms_per_launch": ms_scan, "traffic": None},
            "scan_with_compaction": {"kernel": "accept_scan_kernel + esc_count_kernel + esc_compact_kernel (one block per 65536 flags)", "ms": ms_both,
                                     "achieved": (scan_bytes + compact_bytes) / ms_both / 1e6, "unit": "GB/s",
                                     "frac": (scan_bytes + compact_bytes) / ms_both / 1e6 / hb},
            "tree_mask_roofline": {"kernel": "tree_mask_block_kernel", "bound": "hbm", "achieved": mask_bytes / ms_mask / 1e6,
                                   "peak": hb, "unit": "GB/s", "frac": mask_bytes / ms_mask / 1e6 / hb,
                                   "work_per_launch": mask_bytes, "ms_per_launch": ms_mask}})
        print(json.dumps(out), flush=True)
        return
    if args.only == "prune":
        # token pruning on the scan stress trees: every sequence pruned at a random node of depth <= 2
        B, T = 1 << 20, cfg.T
        parent, tok, _ = _scan_stress_inputs(cfg, B)
        mask = torch.zeros((B, T), dtype=torch.int64, device="cuda")
        ts.trispec_build_tree_mask(ts.tree_args(parent, mask, None))
        g = torch.Generator(device="cuda").manual_seed(cfg.seed)
        root = torch.randint(0, 8, (B,), generator=g, device="cuda", dtype=torch.int32)
        po = ts.alloc_prune_out(B, T)
        pa = ts.prune_args(parent, tok, mask, root, po)
        byts = B * (T * 40 + 8)       # in: parent, tok (4 B), mask (8 B) per node; out: 24 B per node
        ms = timed(lambda: ts.trispec_prune_tree(pa), byts)
        out.update({"config": {"workload": f"prune stress: 2^20 sequences of the {cfg.name} tree shape", "T": T,
                               "mean_kept_nodes": po["n_keep"].float().mean().item(), "l2": out["config"]["l2"]},
                    "value": B * cfg.k / (ms * 1e-3), "ms_per_step": ms, "dtype": "int32",
                    "roofline": {"kernel": "prune_tree_kernel", "bound": "hbm", "achieved": byts / ms / 1e6,
                                 "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": byts / ms / 1e6 / peaks["hbm_gbs"],
                                 "work_per_launch": byts, "ms_per_launch": ms, "traffic": None}})
        print(json.dumps(out), flush=True)
        return
    if args.only == "commit":
        # KV commit stress: 32768 sequences with the workload's KV heads, 7 rows appended each
        B, T, Hkv, D = 32768, cfg.T, cfg.Hkv, cfg.D
        kt = torch.randn((B, T, Hkv, D), device="cuda").to(torch.bfloat16)
        vt = torch.randn((B, T, Hkv, D), device="cuda").to(torch.bfloat16)
        Lcap = 8
        kc = torch.zeros((B, Lcap, Hkv, D), dtype=torch.bfloat16, device="cuda")
        vc = torch.zeros_like(kc)
        ctx = torch.zeros(B, dtype=torch.int32, device="cuda")
        ctx_out = torch.zeros_like(ctx)
        path = torch.arange(1, T + 1, dtype=torch.int32, device="cuda").clamp(max=T - 1).repeat(B, 1).contiguous()
        acc = torch.full((B,), 6, dtype=torch.int32, device="cuda")
        ca = ts.commit_args(kt, vt, kc, vc, ctx, path, acc, ctx_out)
        byts = B * 7 * Hkv * D * 2 * 2 * 2          # 7 rows of K and V read and written
        ms = timed(lambda: ts.trispec_commit_kv(ca), byts)
        out.update({"config": {"workload": f"commit stress: {B} sequences x 7 appended rows, Hkv {Hkv}", "l2": out["config"]["l2"]},
                    "value": B * 6 / (ms * 1e-3), "ms_per_step": ms, "dtype": "u8",
                    "roofline": {"kernel": "kv_commit_kernel", "bound": "hbm", "achieved": byts / ms / 1e6,
                                 "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": byts / ms / 1e6 / peaks["hbm_gbs"],
                                 "work_per_launch": byts, "ms_per_launch": ms, "traffic": None}})
        print(json.dumps(out), flush=True)
        return
    if args.only == "sample":
        # bonus sampling for every sequence of the workload: one more pass over W
        inp = gen.make_inputs(cfg, with_attention=False)
        pas = runner.VerifyPass(cfg, inp, with_attention=False)
        last = torch.zeros(cfg.B, dtype=torch.int32, device="cuda")
        bonus = torch.full((cfg.B,), -2, dtype=torch.int32, device="cuda")
        sa = ts.sample_args(pas.dev["h"], pas.dev["W"], last, bonus, cfg.logit_scale, 1234, 0, dev_status=pas.status)
        ws = ts.alloc_workspace(ts.trispec_sample_bonus_workspace(sa))
        sa.workspace, sa.workspace_bytes = ws.data_ptr(), ws.numel()

        def call():
            bonus.fill_(-2)
            ts.trispec_sample_bonus(sa)
        byts = 2.0 * cfg.V * cfg.d + 2.0 * cfg.B * cfg.d
        ms = timed(call, byts)
        roof = _roof(peaks, 2.0 * cfg.B * cfg.d * cfg.V, byts, ms)
        roof["kernel"] = "sample_gemm_kernel (+ gather, finalize, flag reset)"
        assert int(pas.status.item()) == 0
        out.update({"value": cfg.B / (ms * 1e-3), "unit": "sampled tokens/s", "ms_per_step": ms, "dtype": "bf16",
                    "roofline": roof})
        print(json.dumps(out), flush=True)
        return
    if args.only == "attention":
        inp = gen.make_inputs(cfg, with_lm_head=False)
        small = dataclasses.replace(cfg, V=4096, d=64)      # the LM head is not run: a token-sized stand-in
        inp.update({k: v for k, v in gen.make_inputs(small, with_attention=False).items() if k in ("h", "W")})
        pas = runner.VerifyPass(small, inp)
        Lsum = float(np.asarray(inp["ctx_len"])[pas.seqs].sum())
        rows = cfg.T
        if args.tree_nodes is not None:          # pruned trees: fewer query rows per sequence
            rows = max(0, min(cfg.T, args.tree_nodes))
            n_nodes = torch.full((cfg.B,), rows, dtype=torch.int32, device="cuda")
            pas.attn_args.n_nodes = n_nodes.data_ptr()
            out["config"]["tree_nodes"] = rows
        byts = (Lsum + n_seq * cfg.T) * cfg.Hkv * cfg.D * 4 + 2 * n_seq * rows * cfg.Hq * cfg.D * 2
        ms = timed(lambda: ts.trispec_verify_attn(pas.attn_args), byts)
        flops = 4.0 * rows * cfg.Hq * cfg.D * (Lsum + n_seq * cfg.T)
        roof = _roof(peaks, flops, byts, ms)
        roof["kernel"] = ("verify_attn_pieces_kernel" if ts.trispec_verify_attn_plan(pas.attn_args) == "pieces"
                          else "verify_attn_split_kernel")
        roof["traffic"] = dram_traffic(roof["kernel"], cfg.name)
    else:
        inp = gen.make_inputs(cfg, with_attention=False)
        pas = runner.VerifyPass(cfg, inp, with_attention=False)
        M = n_seq * cfg.T
        lm_bytes = 2.0 * cfg.V * cfg.d + 2.0 * M * cfg.d + 40.0 * M
        ms = timed(lambda: ts.trispec_lmhead_stats(pas.lm_args), lm_bytes)
        roof = _roof(peaks, 2.0 * M * cfg.d * cfg.V, lm_bytes, ms)
        roof["kernel"] = "lmhead_gemm_kernel (+ finalize)"
        roof["traffic"] = dram_traffic("lmhead_gemm_kernel", cfg.name)
    assert int(pas.status.item()) == 0, "a device-side wait timed out"
    out.update({"value": n_seq * cfg.k / (ms * 1e-3), "ms_per_step": ms, "dtype": "bf16", "roofline": roof})
    print(json.dumps(out), flush=True)


# ---------------------------------------------------------------------------------------------
# Multi-rank host logic (replicas only: sequences are independent, there is no data-path exchange)
# ---------------------------------------------------------------------------------------------
def rank_config(cfg, rank: int):
    """Every rank verifies its own batch of the workload's shape: same config, seed offset by rank."""
    import dataclasses
    return dataclasses.replace(cfg, seed=cfg.seed + rank)


def max_over_ranks(values, world: int, device="cpu"):
    """Element-wise maximum of per-rank timings over all ranks (identity for one rank)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def aggregate_throughput(cfg, world: int, ms_per_step: float) -> float:
    """Whole-job draft tokens per second: every rank processed one batch per step (weak scaling)."""
    return cfg_tokens(cfg) * world / (ms_per_step * 1e-3)


def cfg_tokens(cfg):
    n = cfg.B if cfg.n_active is None else cfg.n_active
    return n * cfg.k


def config_dict(cfg):
    """The workload as both arms of the benchmark print it (same keys, same values)."""
    n_seq = cfg.B if cfg.n_active is None else cfg.n_active
    return {"workload": cfg.name, "B": cfg.B, "active_sequences": n_seq, "draft_tokens": cfg.k,
            "tree_nodes": cfg.T, "context": cfg.L, "context_min": cfg.L if cfg.L_min is None else cfg.L_min,
            "Hq": cfg.Hq, "Hkv": cfg.Hkv, "head_dim": cfg.D, "hidden": cfg.d, "vocab": cfg.V,
            "kv": "paged" if cfg.paged else "contiguous", "mode": "target" if cfg.mode else "proxy",
            "l2": "inputs larger than L2 (LM-head weights + KV cache are streamed every pass)",
            "parallelism": "independent replicas, one batch per GPU"}


# ---------------------------------------------------------------------------------------------
# One workload measured through the fused call
# ---------------------------------------------------------------------------------------------
def _roofline(kind, peaks, flops, byts, ms, loop_ms, kernel, workload, timed):
    """Roofline record of one entry point: the bound is the larger of the two lower-bound times at the
    measured peaks. `frac` is against the measured peak (the sustained bf16 figure when the timed loop
    ran long enough for the power cap to bite, else the burst figure); the burst and the data-sheet
    fractions stand beside it."""
    sustained = kind == "lmhead" and peaks.get("bf16_tflops_sustained") and loop_ms >= 200.0
    tc_peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    tflops, gbs = flops / (ms * 1e-3) / 1e12, byts / (ms * 1e-3) / 1e9
    if flops / (tc_peak * 1e12) >= byts / (peaks["hbm_gbs"] * 1e9):
        r = {"kernel": kernel, "bound": "tensor", "achieved": tflops, "peak": tc_peak, "unit": "TFLOP/s",
             "frac": tflops / tc_peak, "work_per_launch": flops,
             "peak_source": f"{peaks['source']} {'sustained' if sustained else 'burst'} bf16 GEMM",
             "frac_of_burst_peak": tflops / peaks["bf16_tflops"], "frac_of_nominal": tflops / NOMINAL["bf16_tflops"]}
    else:
        r = {"kernel": kernel, "bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
             "frac": gbs / peaks["hbm_gbs"], "work_per_launch": byts,
             "peak_source": f"{peaks['source']} copy bandwidth", "frac_of_nominal": gbs / NOMINAL["hbm_gbs"]}
    r.update({"traffic": dram_traffic(kernel, workload), "ms_per_launch": ms, "timed": timed})
    return r


def measure_workload(cfg, inp, steps, warmup, peaks, world=1, dist=None, clock_index=0, sample_clocks=True):
    """Times one workload on the current device: K passes back to back (the metric), single-pass
    latency, the LM head and the attention in situ, and the pass through the host-buffer entry point.
    Returns a dict; `total_ms` and `e2e_ms` are this rank's (the caller takes the maximum over ranks)."""
    import numpy as np
    import torch
    from paper_2601_23180_b200 import binding as ts
    from paper_2601_23180_b200 import runner
    pas = runner.VerifyPass(cfg, inp)
    pas.prepare_host(inp)
    stream = torch.cuda.current_stream()

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(warmup):
        pas.run()
    sync_all()
    assert int(pas.status.item()) == 0, "a device-side wait timed out"

    # ---- device-resident timing: K passes, CUDA events on the launching stream
    sampler = ClockSampler(clock_index)
    if sample_clocks:
        sampler.start()
    e_start, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n0 = ts.launch_count()
    sync_all()
    t_host0 = time.perf_counter()
    e_start.record(stream)
    for _ in range(steps):
        pas.run()
    e_end.record(stream)
    host_us_per_call = (time.perf_counter() - t_host0) / steps * 1e6   # launch cost, GPU running behind
    sync_all()
    launches = ts.launch_count() - n0
    total_ms = e_start.elapsed_time(e_end)      # K passes back to back, one bracket
    # latency of a single pass (each bracketed by its own events; clocks recover between them)
    n_lat = min(steps, 100)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_lat)]
    for s_, e_ in ev:
        s_.record(stream)
        pas.run()
        e_.record(stream)
    torch.cuda.synchronize()
    pass_latency_ms = statistics.median(s_.elapsed_time(e_) for s_, e_ in ev)

    # ---- per-step breakdown, measured in situ with the launch queue kept full:
    #   lmhead    = K back-to-back calls of trispec_lmhead_stats (W, 0.6 GB or more, evicts itself from L2)
    #   attention = event-bracketed attention calls, each preceded by an LM-head call (W streaming
    #               flushes the KV cache from L2, as in the real pass); the marginal cost
    #               (K full passes) - (K passes without attention) is reported beside it
    def timed_loop(fn):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    def bracketed(fn, before):
        """Mean device time of `fn` alone, each call preceded (untimed) by `before`, which streams the
        LM-head weights through L2 exactly as the full pass does, so the timed call sees the cache
        state it has inside a pass."""
        n = min(steps, 200)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        for s_, e_ in evs:
            before()
            s_.record(stream)
            fn()
            e_.record(stream)
        torch.cuda.synchronize()
        return sum(s_.elapsed_time(e_) for s_, e_ in evs) / n

    lm_call = lambda: ts.trispec_lmhead_stats(pas.lm_args)
    attn_call = lambda: ts.trispec_verify_attn(pas.attn_args)
    ms_lmhead = timed_loop(lm_call)
    ms_full = timed_loop(pas.run)
    ms_no_attn = timed_loop(lambda: ts.trispec_verify(pas.tree_args, None, pas.lm_args, pas.scan_args))
    ms_attn = bracketed(attn_call, lm_call)
    ms_lmhead_single = bracketed(lm_call, attn_call)
    part_ms = {"lmhead": ms_lmhead, "lmhead_single_call": ms_lmhead_single, "attention": ms_attn,
               "attention_marginal_in_pass": ms_full - ms_no_attn,
               "tree_mask_and_scan": max(ms_no_attn - ms_lmhead, 0.0), "full_pass_back_to_back": ms_full}

    # ---- end to end through the host-buffer entry point: H2D inputs + pass + D2H results per step
    for _ in range(3):
        pas.run_host()
    sync_all()
    t0 = time.perf_counter()
    for _ in range(steps):
        pas.run_host()
        torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3
    clocks = sampler.stop() if sample_clocks else None
    assert int(pas.status.item()) == 0, "a device-side wait timed out"

    n_seq = cfg.B if cfg.n_active is None else cfg.n_active
    M = n_seq * cfg.T
    lm_flops = 2.0 * M * cfg.d * cfg.V
    lm_bytes = 2.0 * cfg.V * cfg.d + 2.0 * M * cfg.d + 40.0 * M
    lm_kernel = "lmhead_rows_kernel" if n_seq == 1 else "lmhead_gemm_kernel"
    lm_roof = _roofline("lmhead", peaks, lm_flops, lm_bytes, ms_lmhead, ms_lmhead * steps, lm_kernel, cfg.name,
                        "trispec_lmhead_stats back to back (GEMM + finalize kernel; CUDA events on the stream)")
    Lsum = float(np.asarray(inp["ctx_len"])[pas.seqs].sum())
    attn_bytes = (Lsum + n_seq * cfg.T) * cfg.Hkv * cfg.D * 2 * 2 + 2 * n_seq * cfg.T * cfg.Hq * cfg.D * 2
    attn_flops = 4.0 * cfg.T * cfg.Hq * cfg.D * (Lsum + n_seq * cfg.T)
    attn_kernel = "verify_attn_pieces_kernel" if ts.trispec_verify_attn_plan(pas.attn_args) == "pieces" \
        else "verify_attn_split_kernel"
    attn_roof = _roofline("attention", peaks, attn_flops, attn_bytes, ms_attn, 0.0, attn_kernel,
                          cfg.name, "trispec_verify_attn bracketed by CUDA events right after an LM-head call "
                          "(the cache state it meets inside a pass)")
    out = {"total_ms": total_ms, "e2e_ms": e2e_ms, "launches": launches, "host_us_per_call": host_us_per_call,
           "pass_latency_ms_median": pass_latency_ms, "kernels_ms": part_ms, "clocks": clocks,
           "roofline": lm_roof, "attention_roofline": attn_roof, "h2d_bytes": pas.h2d_bytes,
           "d2h_bytes": pas.d2h_bytes}
    del pas
    torch.cuda.empty_cache()
    return out


# ---------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="long_paged",
                    help="the workload of the headline figures (default: the largest single-GPU configuration)")
    ap.add_argument("--impl", default="trispec", choices=["trispec", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-workload", action="store_true",
                    help="skip the per_workload block (the other four configurations)")
    ap.add_argument("--only", default=None, choices=["attention", "lmhead", "scan", "prune", "commit", "sample"],
                    help="time one entry point alone (L2 flushed before each call) instead of the pass")
    ap.add_argument("--tree-nodes", type=int, default=None,
                    help="with --only attention: every tree keeps only its first N nodes (a pruned tree)")
    ap.add_argument("--batch", type=int, default=None,
                    help="override the number of sequences of the workload (reduced copies for profiler captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "trispec" else args.warmup

    from paper_2601_23180_b200 import inputs as gen
    cfg = gen.CONFIGS[args.workload]
    if args.batch is not None:
        import dataclasses as _dc
        cfg = _dc.replace(cfg, B=args.batch, name=f"{cfg.name}[B={args.batch}]",
                          n_active=None if cfg.n_active is None else min(cfg.n_active, args.batch))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, cfg, rank)
        return
    if args.only is not None:
        if rank == 0:
            run_only(args, cfg)
        return

    import torch
    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the verify pass has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    from paper_2601_23180_b200 import build as tbuild
    if rank == 0:
        tbuild.build()
    if world > 1:
        dist.barrier()
    peaks = _peaks()

    # every rank verifies its own batch of the same shape (seed offset by rank); the inputs are
    # generated once, before anything is timed
    rcfg = rank_config(cfg, rank)
    inp = gen.make_inputs(rcfg)
    m = measure_workload(rcfg, inp, args.steps, args.warmup, peaks, world=world, dist=dist, clock_index=local_rank,
                         sample_clocks=(rank == 0))
    total_ms, e2e_ms = max_over_ranks([m["total_ms"], m["e2e_ms"]], world, device="cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    tokens = cfg_tokens(cfg) * world
    ms_per_step = total_ms / args.steps
    line = {
        "metric": METRIC, "value": aggregate_throughput(cfg, world, ms_per_step), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config_dict(cfg),
        "e2e": {"value": tokens / (e2e_ms * 1e-3 / args.steps), "unit": UNIT,
                "h2d_bytes_per_step": m["h2d_bytes"], "d2h_bytes_per_step": m["d2h_bytes"]},
        "gpu_launches": m["launches"], "host_us_per_call": m["host_us_per_call"],
        "pass_latency_ms_median": m["pass_latency_ms_median"], "clocks": m["clocks"],
        "roofline": m["roofline"], "kernels_ms": m["kernels_ms"], "attention_roofline": m["attention_roofline"],
    }
    if not args.no_cpu_baseline and world == 1:
        v, desc, threads = oracle_timed(cfg, inp, budget_s=20.0)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle (numpy/BLAS)",
                                "sample": desc}
    del inp

    # ---- the other configurations, same measurements with fewer steps (one GPU only: with N > 1 all
    # GPUs would be held meanwhile)
    if world == 1 and not args.no_per_workload and args.batch is None:
        per = {}
        n_steps = min(args.steps, 200)
        for name in gen.CONFIG_ORDER:
            if name == cfg.name:
                mm, k_steps = m, args.steps
            else:
                wcfg = gen.CONFIGS[name]
                winp = gen.make_inputs(wcfg)
                mm, k_steps = measure_workload(wcfg, winp, n_steps, args.warmup, peaks, clock_index=local_rank), n_steps
                del winp
            wc = gen.CONFIGS[name]
            ms = mm["total_ms"] / k_steps
            per[name] = {"config": config_dict(wc), "steps": k_steps, "pass_ms_back_to_back": ms,
                         "pass_latency_ms_median": mm["pass_latency_ms_median"],
                         "value": cfg_tokens(wc) / (ms * 1e-3),
                         "e2e_value": cfg_tokens(wc) / (mm["e2e_ms"] * 1e-3 / k_steps),
                         "lmhead_roofline": mm["roofline"], "attention_roofline": mm["attention_roofline"],
                         "kernels_ms": mm["kernels_ms"], "gpu_launches": mm["launches"],
                         "sm_mhz": None if mm["clocks"] is None else mm["clocks"]["sm_mhz"],
                         "clock_reasons": None if mm["clocks"] is None else mm["clocks"]["reasons"]}
        line["per_workload"] = per
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
