"""Parity at the full sizes of the five workload configs, in the launch configuration the
benchmark times (the fused pass through `runner.VerifyPass`).

The oracle cannot redo a whole pass at these sizes in reasonable time, so it recomputes
sampled outputs one by one: a set of attention rows (sequence, node, head), the LM-head
statistics of the first nodes of one sequence, the whole tree mask, and the acceptance scan
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
N_LM_NODES = 12


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

    # ---- LM-head statistics: the first nodes of one sequence (parents precede children, so a
    # prefix of the node list is a tree of its own)
    b0 = seqs[len(seqs) // 2]
    n = min(N_LM_NODES, T)
    ref = orc.lmhead_stats(inp["h"][b0:b0 + 1, :n], inp["W"], inp["parent"][b0:b0 + 1, :n],
                           inp["tok"][b0:b0 + 1, :n], cfg.logit_scale)
    sub = {k: v[b0:b0 + 1, :n] for k, v in got["stats"].items()}
    n_tie = H.check_stats(sub, ref, [0], n)
    assert n_tie <= 1

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
