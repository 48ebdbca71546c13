"""Parity at the full sizes of the five workload configs, in the launch configuration the
benchmark times (the fused pass through `runner.VerifyPass`).

The oracle cannot redo a whole pass at these sizes in reasonable time, so it recomputes
sampled outputs one by one: a set of attention rows (sequence, node, head), the LM-head
statistics of three nodes in each of three sequences (all rows, and the scan decided by the oracle
alone, for the two smallest workloads), the whole tree mask, and the acceptance scan
of every sequence from the statistics the GPU produced (the rule is exact integer work on
given statistics, so it must agree everywhere except where a margin sits on the threshold).
Tolerances are those of the small-size parity tests.
"""
import math

import numpy as np
import pytest

from oracle import trispec_oracle as orc
from paper_2601_23180_b200 import inputs as gen

pytestmark = pytest.mark.gpu

N_ATTN_SAMPLES = 24


@pytest.mark.parametrize("name", gen.CONFIG_ORDER)
def test_full_size_pass_sampled_against_oracle(name):
    import torch
    import tests.gpu_helpers as H
    from paper_2601_23180_b200 import runner
    cfg = gen.CONFIGS[name]
    inp = gen.make_inputs(cfg)
    pas = runner.VerifyPass(cfg, inp)
    pas.run()
    torch.cuda.synchronize()
    got = pas.results()
    assert got["status"] == 0
    seqs = pas.seqs
    B, T = cfg.B, cfg.T

    # ---- tree mask: whole output
    ref_mask, ref_depth = orc.build_tree_mask(inp["parent"])
    assert np.array_equal(got["mask"].view(np.uint64), ref_mask)
    assert np.array_equal(got["depth"], ref_depth)

    # ---- attention: sampled rows, among them the root and the last node, the shortest and
    # the longest context
    g = np.random.default_rng(1234)
    ctx = np.asarray(inp["ctx_len"])
    b_short = min(seqs, key=lambda b: ctx[b])
    b_long = max(seqs, key=lambda b: ctx[b])
    samples = [(b_short, 0, 0), (b_short, T - 1, cfg.Hq - 1), (b_long, 0, cfg.Hq - 1), (b_long, T - 1, 0)]
    while len(samples) < N_ATTN_SAMPLES:
        samples.append((int(g.choice(seqs)), int(g.integers(T)), int(g.integers(cfg.Hq))))
    ref_o, ref_lse = orc.verify_attn(inp["q"], inp["k_tree"], inp["v_tree"], ref_mask, inp["k_cache"],
                                     inp["v_cache"], inp["ctx_len"], 1.0 / math.sqrt(cfg.D),
                                     block_table=inp.get("block_table"), block_size=cfg.block_size,
                                     samples=samples)
    for (b, i, h) in samples:
        err = np.abs(got["o"][b, i, h] - ref_o[b, i, h]).max()
        assert err <= 2e-2, (b, i, h, err)                    # bf16 in, fp32 accumulate, bf16 out
        assert abs(got["attn_lse"][b, h, i] - ref_lse[b, h, i]) <= 1e-3 * max(1.0, abs(ref_lse[b, h, i]))
    untouched = [b for b in range(B) if b not in seqs]
    for b in untouched:
        assert np.isnan(got["o"][b]).all()

    # ---- LM-head statistics: the root, an inner node and the last node of the first, the middle and
    # the last verified sequence, so that the first and last rows of an M tile and both CTAs of a
    # pair are compared. The oracle gets each node as the second row of a two-row chain whose first
    # row is the node's parent (the drafted-token probability is read in the parent's row).
    W64 = orc.bf16_to_f64(inp["W"])
    lm_seqs = sorted({seqs[0], seqs[len(seqs) // 2], seqs[-1]})
    lm_nodes = sorted({0, min(12, T - 1), T - 1})
    for b0 in lm_seqs:
        for node in lm_nodes:
            par = int(inp["parent"][b0, node])
            rows = [node] if par < 0 else [par, node]
            sub_parent = np.array([[-1, 0][:len(rows)]], dtype=np.int32)
            ref = orc.lmhead_stats(inp["h"][b0:b0 + 1, rows], inp["W"], sub_parent, inp["tok"][b0:b0 + 1, rows],
                                   cfg.logit_scale, W64=W64)
            j = len(rows) - 1
            sub = {k: v[b0:b0 + 1, node:node + 1] for k, v in got["stats"].items()}
            one = {k: v[:, j:j + 1] for k, v in ref.items()}
            n_tie = H.check_stats(sub, one, [0], 1)
            assert n_tie <= 1

    # ---- the two smallest workloads: the oracle's whole LM head, and the scan decided by the oracle alone
    if name in ("tiny_chain", "proxy_tree"):
        ref_st = orc.lmhead_stats(inp["h"], inp["W"], inp["parent"], inp["tok"], cfg.logit_scale, seqs=seqs, W64=W64)
        H.check_stats(got["stats"], ref_st, seqs, T)
        ref_only = orc.accept_scan(ref_st["p_top1"], ref_st["p_top2"], ref_st["top1_idx"], inp["parent"], inp["tok"],
                                   cfg.lam, mode=cfg.mode)
        gap = ref_st["top1_val"] - ref_st["top2_val"]
        near_tie = gap < 1e-3 * np.maximum(1.0, np.abs(ref_st["top1_val"]))
        n_cmp = 0
        for b in seqs:
            visited = [0] + [int(x) for x in ref_only["path"][b] if x >= 0]
            if ref_only["near_thr"][b] > 0 or got["scan"]["near_thr"][b] > 0 or near_tie[b, visited].any():
                continue
            for k in ("accept_len", "escalate", "bonus_tok", "last_node"):
                assert got["scan"][k][b] == ref_only[k][b], (k, b)
            assert np.array_equal(got["scan"]["path"][b], ref_only["path"][b])
            n_cmp += 1
        assert n_cmp >= len(seqs) - max(1, len(seqs) // 4)
    del W64

    # ---- acceptance scan: every sequence, from the GPU's own statistics
    st = got["stats"]
    ref_scan = orc.accept_scan(st["p_top1"].astype(np.float64), st["p_top2"].astype(np.float64),
                               st["top1_idx"].astype(np.int64), inp["parent"], inp["tok"], cfg.lam, mode=cfg.mode)
    n_checked = 0
    for b in seqs:
        if ref_scan["near_thr"][b] > 0 or got["scan"]["near_thr"][b] > 0:
            continue
        for k in ("accept_len", "escalate", "bonus_tok", "last_node"):
            assert got["scan"][k][b] == ref_scan[k][b], (k, b)
        assert np.array_equal(got["scan"]["path"][b], ref_scan["path"][b])
        n_checked += 1
    assert n_checked >= len(seqs) - max(1, len(seqs) // 4)
    for b in untouched:
        assert got["scan"]["accept_len"][b] == 0 and got["scan"]["last_node"][b] == -1
