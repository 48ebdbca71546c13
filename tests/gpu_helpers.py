"""Helpers for the GPU parity tests: move generator output to the device, call the library
through its C ABI binding and bring results back as numpy."""
from __future__ import annotations

import math
from typing import Dict, Optional

import numpy as np
import torch

from paper_2601_23180_b200 import inputs as gen


def bf16_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> CUDA tensor of dtype bfloat16 (bits preserved)."""
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def i32_dev(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).cuda()


def to_device(inp: Dict[str, np.ndarray]) -> Dict[str, Optional[torch.Tensor]]:
    dev: Dict[str, Optional[torch.Tensor]] = {}
    for k in ("q", "k_tree", "v_tree", "k_cache", "v_cache", "h", "W"):
        if k in inp and inp[k] is not None:
            dev[k] = bf16_dev(inp[k])
    for k in ("parent", "tok", "ctx_len", "block_table", "seq_index"):
        dev[k] = None if inp.get(k) is None else i32_dev(inp[k])
    return dev


def run_tree_mask(parent_dev: torch.Tensor, status: Optional[torch.Tensor] = None):
    from paper_2601_23180_b200 import binding as ts
    B, T = parent_dev.shape
    mask = torch.zeros((B, T), dtype=torch.int64, device="cuda")
    depth = torch.zeros((B, T), dtype=torch.int32, device="cuda")
    ts.trispec_build_tree_mask(ts.tree_args(parent_dev, mask, depth, dev_status=status))
    torch.cuda.synchronize()
    return mask, depth


def run_lmhead(dev, cfg: gen.VerifyConfig, logit_scale=None):
    from paper_2601_23180_b200 import binding as ts
    B, T = dev["parent"].shape
    st = ts.alloc_stats(B, T)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    a = ts.lmhead_args(dev["h"], dev["W"], dev["parent"], dev["tok"],
                       cfg.logit_scale if logit_scale is None else logit_scale, st,
                       seq_index=dev.get("seq_index"), dev_status=status)
    ws = ts.alloc_workspace(ts.trispec_lmhead_stats_workspace(a))
    a.workspace, a.workspace_bytes = ws.data_ptr(), ws.numel()
    ts.trispec_lmhead_stats(a)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "device-side wait timed out"
    return {k: v.cpu().numpy() for k, v in st.items()}


def run_scan(stats_np, parent, tok, lam, mode, active=None, start_node=None, criterion=0, q_draft=None,
             u_accept=None, accept_rule=0, alpha=0.0):
    from paper_2601_23180_b200 import binding as ts
    B, T = parent.shape
    st = {
        "p_top1": torch.from_numpy(np.asarray(stats_np["p_top1"], dtype=np.float32)).cuda(),
        "p_top2": torch.from_numpy(np.asarray(stats_np["p_top2"], dtype=np.float32)).cuda(),
        "top1_idx": i32_dev(stats_np["top1_idx"]),
    }
    f32 = lambda x: None if x is None else torch.from_numpy(np.asarray(x, dtype=np.float32)).cuda()
    if "p_draft" in stats_np:
        st["p_draft"] = f32(stats_np["p_draft"])
    if "entropy" in stats_np:
        st["entropy"] = torch.from_numpy(np.asarray(stats_np["entropy"], dtype=np.float32)).cuda()
    out = ts.alloc_scan_out(B, T)
    act = None if active is None else torch.from_numpy(np.asarray(active, dtype=np.uint8)).cuda()
    sn = None if start_node is None else i32_dev(start_node)
    a = ts.scan_args(st, i32_dev(parent), i32_dev(tok), lam, mode, out, active=act, start_node=sn,
                     criterion=criterion, q_draft=f32(q_draft), u_accept=f32(u_accept), accept_rule=accept_rule,
                     alpha=alpha)
    ts.trispec_accept_scan(a)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def run_attn(dev, cfg: gen.VerifyConfig, mask_dev, want_lse=True, n_nodes=None, expect_status=0):
    from paper_2601_23180_b200 import binding as ts
    B, T, Hq, D = dev["q"].shape
    o = torch.full((B, T, Hq, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, Hq, T), float("nan"), dtype=torch.float32, device="cuda") if want_lse else None
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    a = ts.attn_args(dev["q"], dev["k_tree"], dev["v_tree"], mask_dev, dev["k_cache"], dev["v_cache"],
                     dev["ctx_len"], 1.0 / math.sqrt(D), o, block_table=dev.get("block_table"),
                     block_size=cfg.block_size, seq_index=dev.get("seq_index"), lse=lse, dev_status=status,
                     n_nodes=None if n_nodes is None else i32_dev(n_nodes))
    ws = ts.alloc_workspace(ts.trispec_verify_attn_workspace(a))
    a.workspace, a.workspace_bytes = ws.data_ptr(), ws.numel()
    ts.trispec_verify_attn(a)
    torch.cuda.synchronize()
    assert int(status.item()) == expect_status, f"device status {int(status.item())}"
    return o.float().cpu().numpy(), (None if lse is None else lse.cpu().numpy())


def check_stats(gpu, ref, seqs, T, near_tie=1e-3, nodes=None):
    """LM-head statistics against the oracle: lse / probabilities within 1e-3 relative
    (probabilities below 1e-6: 1e-9 absolute); top1_idx exact unless the oracle's top-1/top-2
    logits are within `near_tie` relative, which is counted and returned; top2_idx exact unless
    that holds or the oracle's second and third largest logits are that close."""
    n_tie = 0
    for b in seqs:
        for r in (range(T) if nodes is None else nodes):
            for k in ("lse", "max", "top1_val"):
                assert abs(gpu[k][b, r] - ref[k][b, r]) <= 1e-3 * max(1.0, abs(ref[k][b, r])), (k, b, r)
            gap12 = ref["top1_val"][b, r] - ref["top2_val"][b, r]
            tie = gap12 < near_tie * max(1.0, abs(ref["top1_val"][b, r]))
            if tie:
                n_tie += 1
            else:
                assert gpu["top1_idx"][b, r] == ref["top1_idx"][b, r], (b, r)
            if not tie:
                gap23 = ref["top2_val"][b, r] - ref["top3_val"][b, r]
                if not gap23 < near_tie * max(1.0, abs(ref["top2_val"][b, r])):   # a NaN gap (V = 2) compares exactly
                    assert gpu["top2_idx"][b, r] == ref["top2_idx"][b, r], ("top2_idx", b, r)
            assert gpu["top2_idx"][b, r] != gpu["top1_idx"][b, r], ("top2_idx == top1_idx", b, r)
            for k in ("p_top1", "p_top2"):
                g, e = float(gpu[k][b, r]), float(ref[k][b, r])
                assert abs(g - e) <= max(1e-3 * e, 1e-9), (k, b, r, g, e)
            assert abs(gpu["top2_val"][b, r] - ref["top2_val"][b, r]) <= 1e-3 * max(1.0, abs(ref["top2_val"][b, r]))
            if "entropy" in gpu and "entropy" in ref:
                # H = lse - E_p[z]: the difference of two O(10) fp32 quantities, hence an absolute bound
                assert abs(gpu["entropy"][b, r] - ref["entropy"][b, r]) <= 1e-3 * max(1.0, ref["entropy"][b, r]), \
                    ("entropy", b, r, gpu["entropy"][b, r], ref["entropy"][b, r])
            # the drafted token's probability: defined for child nodes (the oracle has NaN at a root)
            e = float(ref["p_draft"][b, r])
            if np.isnan(e):
                assert np.isnan(gpu["p_draft"][b, r])
            else:
                g = float(gpu["p_draft"][b, r])
                assert abs(g - e) <= max(1e-3 * e, 1e-9), ("p_draft", b, r, g, e)
                assert abs(gpu["draft_logit"][b, r] - ref["draft_logit"][b, r]) <= 1e-3 * max(1.0, abs(ref["draft_logit"][b, r]))
    return n_tie
