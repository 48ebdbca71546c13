"""Device-resident state of one verify-pass workload and the calls that run it.

Holds the torch tensors (device memory only) and the C-ABI argument structs for one config,
so that tests, the smoke check and the benchmark launch exactly the same thing. No arithmetic
happens here: `run()` is one call of `trispec_verify`, `run_host()` one call of
`trispec_verify_host`.
"""
from __future__ import annotations

import math
from typing import Dict, Optional

import numpy as np
import torch

from . import binding as ts
from . import inputs as gen


def _bf16_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def _i32_dev(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).cuda()


def _pack_round_inputs(inp: Dict[str, np.ndarray], names):
    """One flat byte tensor (CPU) holding the named arrays back to back, and the (name, shape, dtype)
    list that carves it: int32 for the tree arrays, bf16 for the activations (stored as bit patterns)."""
    arrays, specs = {}, []
    for k in names:
        if k in ("parent", "tok"):
            arrays[k] = np.ascontiguousarray(inp[k], dtype=np.int32)
            specs.append((k, arrays[k].shape, torch.int32))
        else:
            arrays[k] = np.ascontiguousarray(inp[k]).view(np.uint16)
            specs.append((k, arrays[k].shape, torch.bfloat16))
    flat = torch.zeros(ts._carve_bytes(specs), dtype=torch.uint8)
    for k, view in ts._carve(flat, specs).items():
        view.view(torch.uint8).copy_(torch.from_numpy(arrays[k].view(np.uint8).reshape(-1)).view(view.view(torch.uint8).shape))
    return flat, specs


class VerifyPass:
    def __init__(self, cfg: gen.VerifyConfig, inp: Dict[str, np.ndarray], with_attention: bool = True,
                 criterion: int = ts.CRIT_MARGIN):
        self.cfg = cfg
        B, T = cfg.B, cfg.T
        d: Dict[str, Optional[torch.Tensor]] = {}
        for k in ("W",) + (("k_cache", "v_cache") if with_attention else ()):
            d[k] = _bf16_dev(inp[k])
        for k in ("ctx_len", "block_table", "seq_index"):
            d[k] = None if inp.get(k) is None else _i32_dev(inp[k])
        # the per-round inputs sit back to back in two device buffers, in the order the host-buffer
        # entry point copies them, so that each group arrives in one transfer
        self._round_groups = [("parent", "tok", "h")] + ([("q", "k_tree", "v_tree")] if with_attention else [])
        for group in self._round_groups:
            flat, specs = _pack_round_inputs(inp, group)
            d.update(ts._carve(flat.cuda(), specs))
        self.dev = d
        seqs = list(range(B)) if inp.get("seq_index") is None else [int(s) for s in inp["seq_index"]]
        self.seqs = seqs
        active = np.zeros(B, dtype=np.uint8)
        active[seqs] = 1
        self.active = torch.from_numpy(active).cuda()
        self.mask = torch.zeros((B, T), dtype=torch.int64, device="cuda")
        self.depth = torch.zeros((B, T), dtype=torch.int32, device="cuda")
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")
        # the entropy is computed only for the routing criterion that reads it (the margin rule of Eq. 8 does not)
        self.stats = ts.alloc_stats(B, T, entropy=(criterion == ts.CRIT_ENTROPY))
        self.scan_out = ts.alloc_scan_out(B, T)
        self.tree_args = ts.tree_args(d["parent"], self.mask, self.depth, dev_status=self.status)
        self.attn_args = None
        self.o = self.attn_lse = None
        if with_attention:
            self.o = torch.full((B, T, cfg.Hq, cfg.D), float("nan"), dtype=torch.bfloat16, device="cuda")
            self.attn_lse = torch.full((B, cfg.Hq, T), float("nan"), dtype=torch.float32, device="cuda")
            a = ts.attn_args(d["q"], d["k_tree"], d["v_tree"], self.mask, d["k_cache"], d["v_cache"], d["ctx_len"],
                             1.0 / math.sqrt(cfg.D), self.o, block_table=d["block_table"],
                             block_size=cfg.block_size, seq_index=d["seq_index"], lse=self.attn_lse,
                             dev_status=self.status)
            self.attn_ws = ts.alloc_workspace(ts.trispec_verify_attn_workspace(a))
            a.workspace, a.workspace_bytes = self.attn_ws.data_ptr(), self.attn_ws.numel()
            self.attn_args = a
        l = ts.lmhead_args(d["h"], d["W"], d["parent"], d["tok"], cfg.logit_scale, self.stats,
                           seq_index=d["seq_index"], dev_status=self.status)
        self.lm_ws = ts.alloc_workspace(ts.trispec_lmhead_stats_workspace(l))
        l.workspace, l.workspace_bytes = self.lm_ws.data_ptr(), self.lm_ws.numel()
        self.lm_args = l
        self.scan_args = ts.scan_args(self.stats, d["parent"], d["tok"], cfg.lam, cfg.mode, self.scan_out,
                                      active=self.active, criterion=criterion)
        self._host = None

    # one verify pass, inputs resident on the device
    def run(self, stream=None):
        ts.trispec_verify(self.tree_args, self.attn_args, self.lm_args, self.scan_args, stream)

    # ---- the same pass with the per-round inputs and results in pinned host memory
    def prepare_host(self, inp: Dict[str, np.ndarray]):
        """Pinned host copies of the per-round inputs and of the results, each group in one buffer
        laid out like its device counterpart."""
        B, T = self.cfg.B, self.cfg.T
        h: Dict[str, torch.Tensor] = {}
        self._host_flat = []
        for group in self._round_groups:
            flat, specs = _pack_round_inputs(inp, group)
            flat = flat.pin_memory()
            self._host_flat.append(flat)
            h.update(ts._carve(flat, specs))
        specs = ts.scan_out_specs(B, T)
        out_flat = torch.zeros(ts._carve_bytes(specs), dtype=torch.uint8).pin_memory()
        self._host_flat.append(out_flat)
        h.update(ts._carve(out_flat, specs))
        self._host = h
        self._host_io = ts.host_io(**h)
        ins = ("parent", "tok", "h", "q", "k_tree", "v_tree")
        self.h2d_bytes = sum(h[k].numel() * h[k].element_size() for k in ins if k in h)
        self.d2h_bytes = sum(h[k].numel() * h[k].element_size()
                             for k in ("accept_len", "bonus_tok", "last_node", "path", "escalate"))
        return h

    def run_host(self, stream=None):
        ts.trispec_verify_host(self._host_io, self.tree_args, self.attn_args, self.lm_args, self.scan_args, stream)

    def results(self) -> Dict[str, object]:
        out: Dict[str, object] = {
            "mask": self.mask.cpu().numpy(), "depth": self.depth.cpu().numpy(),
            "stats": {k: v.cpu().numpy() for k, v in self.stats.items()},
            "scan": {k: v.cpu().numpy() for k, v in self.scan_out.items()},
            "status": int(self.status.item()),
        }
        if self.o is not None:
            out["o"] = self.o.float().cpu().numpy()
            out["attn_lse"] = self.attn_lse.cpu().numpy()
        return out
