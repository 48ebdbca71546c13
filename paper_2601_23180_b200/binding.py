"""ctypes binding of libtrispec.so: same names as the C ABI, argument marshalling only.

Tensors are torch CUDA tensors (torch is used for device memory and streams, nothing else);
every step of the verify pass runs inside the library's kernels. Importing this module
fails loudly when the library has not been built: there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libtrispec.so")

MODE_PROXY = 0
MODE_TARGET = 1
KV_CONTIGUOUS = 0
KV_PAGED = 1

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2601_23180_b200.build` "
                      "(there is no CPU or PyTorch fallback for the verify pass)")
_lib = C.CDLL(LIB_PATH)

_vp, _i, _f, _sz = C.c_void_p, C.c_int, C.c_float, C.c_size_t


class TreeArgs(C.Structure):
    _fields_ = [("B", _i), ("T", _i), ("parent", _vp), ("mask", _vp), ("depth", _vp), ("dev_status", _vp)]


class AttnArgs(C.Structure):
    _fields_ = [("B", _i), ("T", _i), ("Hq", _i), ("Hkv", _i), ("D", _i), ("scale", _f),
                ("q", _vp), ("k_tree", _vp), ("v_tree", _vp), ("kv_layout", _i),
                ("k_cache", _vp), ("v_cache", _vp), ("Lmax", _i), ("num_blocks", _i),
                ("block_size", _i), ("max_blocks_per_seq", _i), ("block_table", _vp),
                ("ctx_len", _vp), ("mask", _vp), ("seq_index", _vp), ("B_active", _i),
                ("o", _vp), ("lse", _vp), ("workspace", _vp), ("workspace_bytes", _sz),
                ("dev_status", _vp), ("n_nodes", _vp)]


class Stats(C.Structure):
    _fields_ = [(n, _vp) for n in ("max", "lse", "top1_val", "top2_val", "p_top1", "p_top2",
                                   "top1_idx", "top2_idx", "draft_logit", "p_draft", "entropy")]


class LmheadArgs(C.Structure):
    _fields_ = [("B", _i), ("T", _i), ("d", _i), ("V", _i), ("logit_scale", _f), ("h", _vp), ("W", _vp),
                ("parent", _vp), ("tok", _vp), ("seq_index", _vp), ("B_active", _i), ("out", Stats),
                ("workspace", _vp), ("workspace_bytes", _sz), ("dev_status", _vp)]


class ScanArgs(C.Structure):
    _fields_ = [("B", _i), ("T", _i), ("lam", _f), ("mode", _i), ("criterion", _i), ("parent", _vp), ("tok", _vp),
                ("stats", Stats), ("active", _vp), ("start_node", _vp), ("q_draft", _vp), ("u_accept", _vp),
                ("accept_rule", _i), ("alpha", _f), ("accept_len", _vp),
                ("bonus_tok", _vp), ("path", _vp), ("last_node", _vp), ("near_thr", _vp),
                ("n_escalated", _vp), ("esc_index", _vp), ("escalate", _vp), ("compact_scratch", _vp)]


class PruneArgs(C.Structure):
    _fields_ = [("B", _i), ("T", _i), ("parent", _vp), ("tok", _vp), ("mask", _vp), ("root", _vp),
                ("n_keep", _vp), ("node_map", _vp), ("parent_out", _vp), ("tok_out", _vp),
                ("mask_out", _vp), ("depth_out", _vp)]


class CommitArgs(C.Structure):
    _fields_ = [("B", _i), ("T", _i), ("Hkv", _i), ("D", _i), ("k_tree", _vp), ("v_tree", _vp),
                ("kv_layout", _i), ("k_cache", _vp), ("v_cache", _vp), ("Lmax", _i), ("num_blocks", _i),
                ("block_size", _i), ("max_blocks_per_seq", _i), ("block_table", _vp), ("ctx_len", _vp),
                ("path", _vp), ("accept_len", _vp), ("active", _vp), ("ctx_len_out", _vp), ("dev_status", _vp)]


class SampleArgs(C.Structure):
    _fields_ = [("B", _i), ("T", _i), ("d", _i), ("V", _i), ("logit_scale", _f), ("h", _vp), ("W", _vp),
                ("last_node", _vp), ("bonus_tok", _vp), ("sample_value", _vp), ("seed", C.c_ulonglong),
                ("step", C.c_ulonglong), ("workspace", _vp), ("workspace_bytes", _sz), ("dev_status", _vp)]


class HostIO(C.Structure):
    _fields_ = [(n, _vp) for n in ("parent", "tok", "q", "k_tree", "v_tree", "h", "accept_len", "bonus_tok",
                                   "last_node", "path", "escalate")]


_lib.trispec_status_string.restype = C.c_char_p
_lib.trispec_status_string.argtypes = [_i]
_lib.trispec_launch_count.restype = C.c_longlong
_lib.trispec_build_tree_mask.argtypes = [C.POINTER(TreeArgs), _vp]
_lib.trispec_verify_attn_workspace.restype = _sz
_lib.trispec_verify_attn_workspace.argtypes = [C.POINTER(AttnArgs)]
_lib.trispec_verify_attn.argtypes = [C.POINTER(AttnArgs), _vp]
_lib.trispec_verify_plan.restype = C.c_char_p
_lib.trispec_verify_plan.argtypes = [C.POINTER(AttnArgs), C.POINTER(LmheadArgs), C.POINTER(ScanArgs)]
_lib.trispec_verify_attn_plan.restype = C.c_char_p
_lib.trispec_verify_attn_plan.argtypes = [C.POINTER(AttnArgs)]
_lib.trispec_lmhead_stats_workspace.restype = _sz
_lib.trispec_lmhead_stats_workspace.argtypes = [C.POINTER(LmheadArgs)]
_lib.trispec_lmhead_stats.argtypes = [C.POINTER(LmheadArgs), _vp]
_lib.trispec_lmhead_stats_noalloc.argtypes = [C.POINTER(LmheadArgs), _vp]
_lib.trispec_accept_scan.argtypes = [C.POINTER(ScanArgs), _vp]
_lib.trispec_prune_tree.argtypes = [C.POINTER(PruneArgs), _vp]
_lib.trispec_commit_kv.argtypes = [C.POINTER(CommitArgs), _vp]
_lib.trispec_sample_bonus_workspace.restype = _sz
_lib.trispec_sample_bonus_workspace.argtypes = [C.POINTER(SampleArgs)]
_lib.trispec_sample_bonus.argtypes = [C.POINTER(SampleArgs), _vp]
_lib.trispec_verify.argtypes = [C.POINTER(TreeArgs), C.POINTER(AttnArgs), C.POINTER(LmheadArgs),
                                C.POINTER(ScanArgs), _vp]

_lib.trispec_verify_host.argtypes = [C.POINTER(HostIO), C.POINTER(TreeArgs), C.POINTER(AttnArgs),
                                     C.POINTER(LmheadArgs), C.POINTER(ScanArgs), _vp]

EXPORTS = ["trispec_verify_host", "trispec_verify_plan", "trispec_verify_attn_plan", "trispec_status_string", "trispec_launch_count", "trispec_build_tree_mask",
           "trispec_verify_attn_workspace", "trispec_verify_attn", "trispec_lmhead_stats_workspace",
           "trispec_lmhead_stats", "trispec_lmhead_stats_noalloc", "trispec_accept_scan", "trispec_verify",
           "trispec_prune_tree", "trispec_commit_kv", "trispec_sample_bonus_workspace", "trispec_sample_bonus"]


class TrispecError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__(f"trispec error {code}: {_lib.trispec_status_string(code).decode()}")


def _check(code: int):
    if code != 0:
        raise TrispecError(code)


def _p(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous(), "tensors passed to the library must be contiguous"
    return t.data_ptr()


def _hold(a, *objs):
    """Keeps the tensors whose addresses went into the argument struct alive as long as the struct is:
    a temporary passed to a builder would otherwise be freed, and its memory handed out again (for
    instance as the workspace), before the kernels have run."""
    held = []
    for o in objs:
        if isinstance(o, dict):
            held.extend(v for v in o.values() if v is not None)
        elif o is not None:
            held.append(o)
    a._held = tuple(held)
    return a


def _stream(stream: Optional[torch.cuda.Stream]) -> Optional[int]:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def status_string(code: int) -> str:
    return _lib.trispec_status_string(code).decode()


def launch_count() -> int:
    return int(_lib.trispec_launch_count())


STAT_F32 = ("max", "lse", "top1_val", "top2_val", "p_top1", "p_top2", "draft_logit", "p_draft", "entropy")
STAT_I32 = ("top1_idx", "top2_idx")


def alloc_stats(B: int, T: int, device="cuda", entropy: bool = True) -> Dict[str, torch.Tensor]:
    """Output buffers of the LM-head statistics. The entropy is optional in the C ABI (a null pointer
    skips its computation, which saves two instructions per logit in the GEMM's epilogue)."""
    st = {k: torch.full((B, T), float("nan"), dtype=torch.float32, device=device)
          for k in STAT_F32 if entropy or k != "entropy"}
    st.update({k: torch.full((B, T), -1, dtype=torch.int32, device=device) for k in STAT_I32})
    return st


def _stats_struct(st: Dict[str, torch.Tensor]) -> Stats:
    s = Stats()
    for name, _ in Stats._fields_:
        setattr(s, name, _p(st.get(name)))
    return s


# ------------------------------------------------------------------------------ argument builders
def tree_args(parent: torch.Tensor, mask: torch.Tensor, depth: Optional[torch.Tensor],
              dev_status: Optional[torch.Tensor] = None) -> TreeArgs:
    B, T = parent.shape
    return _hold(TreeArgs(B, T, _p(parent), _p(mask), _p(depth), _p(dev_status)), parent, mask, depth, dev_status)


def attn_args(q, k_tree, v_tree, mask, k_cache, v_cache, ctx_len, scale, o, workspace=None,
              block_table=None, block_size=64, seq_index=None, lse=None, dev_status=None, n_nodes=None) -> AttnArgs:
    B, T, Hq, D = q.shape
    Hkv = k_tree.shape[2]
    a = AttnArgs()
    a.B, a.T, a.Hq, a.Hkv, a.D, a.scale = B, T, Hq, Hkv, D, float(scale)
    a.q, a.k_tree, a.v_tree = _p(q), _p(k_tree), _p(v_tree)
    a.k_cache, a.v_cache = _p(k_cache), _p(v_cache)
    if block_table is None:
        a.kv_layout, a.Lmax = KV_CONTIGUOUS, k_cache.shape[1]
        a.num_blocks, a.block_size, a.max_blocks_per_seq = 0, 0, 0
    else:
        a.kv_layout, a.num_blocks = KV_PAGED, k_cache.shape[0]
        a.block_size, a.max_blocks_per_seq = int(block_size), block_table.shape[1]
        a.Lmax = a.block_size * a.max_blocks_per_seq
    a.block_table, a.ctx_len, a.mask = _p(block_table), _p(ctx_len), _p(mask)
    a.seq_index = _p(seq_index)
    a.B_active = 0 if seq_index is None else int(seq_index.numel())
    a.o, a.lse = _p(o), _p(lse)
    a.workspace = _p(workspace)
    a.workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    a.dev_status = _p(dev_status)
    a.n_nodes = _p(n_nodes)
    return _hold(a, q, k_tree, v_tree, mask, k_cache, v_cache, ctx_len, o, workspace, block_table, seq_index, lse,
                 dev_status, n_nodes)


def lmhead_args(h, W, parent, tok, logit_scale, stats, workspace=None, seq_index=None,
                dev_status=None) -> LmheadArgs:
    B, T = parent.shape
    a = LmheadArgs()
    a.B, a.T, a.d, a.V, a.logit_scale = B, T, h.shape[-1], W.shape[0], float(logit_scale)
    a.h, a.W, a.parent, a.tok = _p(h), _p(W), _p(parent), _p(tok)
    a.seq_index = _p(seq_index)
    a.B_active = 0 if seq_index is None else int(seq_index.numel())
    a.out = _stats_struct(stats)
    a.workspace = _p(workspace)
    a.workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    a.dev_status = _p(dev_status)
    return _hold(a, h, W, parent, tok, stats, workspace, seq_index, dev_status)


CRIT_MARGIN, CRIT_TOP1, CRIT_ENTROPY = 0, 1, 2
ACCEPT_GREEDY, ACCEPT_STOCHASTIC, ACCEPT_TOKEN_SPECIFIC = 0, 1, 2


def scan_args(stats, parent, tok, lam, mode, out: Dict[str, torch.Tensor], active=None,
              start_node=None, criterion=CRIT_MARGIN, q_draft=None, u_accept=None,
              accept_rule=ACCEPT_GREEDY, alpha=0.0) -> ScanArgs:
    B, T = parent.shape
    a = ScanArgs()
    a.B, a.T, a.lam, a.mode, a.criterion = B, T, float(lam), int(mode), int(criterion)
    a.parent, a.tok = _p(parent), _p(tok)
    a.stats = _stats_struct(stats)
    a.active, a.start_node = _p(active), _p(start_node)
    a.q_draft, a.u_accept = _p(q_draft), _p(u_accept)
    a.accept_rule, a.alpha = int(accept_rule), float(alpha)
    for k in ("accept_len", "bonus_tok", "path", "last_node", "near_thr", "n_escalated", "esc_index", "escalate",
              "compact_scratch"):
        setattr(a, k, _p(out.get(k)))
    return _hold(a, stats, parent, tok, out, active, start_node, q_draft, u_accept)


def _nbytes(shape, dtype) -> int:
    return int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()


def _carve(buf: torch.Tensor, specs, align: int = 16):
    """Views into one flat uint8 buffer in the given order: (name, shape, dtype). Every array starts
    on a multiple of `align` bytes (the kernels want 16); where the sizes are multiples of it the arrays
    follow each other without gaps, which is what lets the host-buffer entry point merge their copies."""
    out, off = {}, 0
    for name, shape, dtype in specs:
        off = (off + align - 1) // align * align
        n = _nbytes(shape, dtype)
        out[name] = buf[off:off + n].view(dtype).view(*shape)
        off += n
    return out


def _carve_bytes(specs, align: int = 16) -> int:
    off = 0
    for _, shape, dtype in specs:
        off = (off + align - 1) // align * align + _nbytes(shape, dtype)
    return off


def scan_out_specs(B: int, T: int):
    """The scan's outputs in the order `trispec_verify_host` copies them back (accept_len, bonus_tok,
    last_node, path, escalate), then the ones that stay on the device."""
    i32 = torch.int32
    return [("accept_len", (B,), i32), ("bonus_tok", (B,), i32), ("last_node", (B,), i32), ("path", (B, T), i32),
            ("escalate", (B,), torch.uint8)]


def alloc_scan_out(B: int, T: int, device="cuda") -> Dict[str, torch.Tensor]:
    """Output buffers of the scan. The five arrays a decode loop reads back are carved out of one
    allocation, back to back, so that their device-to-host copies can be merged into one."""
    specs = scan_out_specs(B, T)
    out = _carve(torch.empty(_carve_bytes(specs), dtype=torch.uint8, device=device), specs)
    for k, v in out.items():
        v.fill_(9 if k == "escalate" else -7)
    i32 = dict(dtype=torch.int32, device=device)
    out.update({"near_thr": torch.full((B,), -7, **i32), "n_escalated": torch.full((1,), -7, **i32),
                "esc_index": torch.full((B,), -7, **i32)})
    if B > 65536:     # scratch that lets the escalation list be built by one block per 65536 sequences
        out["compact_scratch"] = torch.full(((B + 65535) // 65536,), -7, **i32)
    return out


def prune_args(parent, tok, mask, root, out: Dict[str, torch.Tensor]) -> PruneArgs:
    B, T = parent.shape
    a = PruneArgs()
    a.B, a.T = B, T
    a.parent, a.tok, a.mask, a.root = _p(parent), _p(tok), _p(mask), _p(root)
    a.n_keep, a.node_map = _p(out["n_keep"]), _p(out["node_map"])
    a.parent_out, a.tok_out = _p(out["parent"]), _p(out["tok"])
    a.mask_out, a.depth_out = _p(out.get("mask")), _p(out.get("depth"))
    return _hold(a, parent, tok, mask, root, out)


def alloc_prune_out(B: int, T: int, device="cuda") -> Dict[str, torch.Tensor]:
    i32 = dict(dtype=torch.int32, device=device)
    return {"n_keep": torch.full((B,), -7, **i32), "node_map": torch.full((B, T), -7, **i32),
            "parent": torch.full((B, T), -7, **i32), "tok": torch.full((B, T), -7, **i32),
            "mask": torch.full((B, T), -7, dtype=torch.int64, device=device), "depth": torch.full((B, T), -7, **i32)}


def commit_args(k_tree, v_tree, k_cache, v_cache, ctx_len, path, accept_len, ctx_len_out, block_table=None,
                block_size=64, active=None, dev_status=None) -> CommitArgs:
    B, T, Hkv, D = k_tree.shape
    a = CommitArgs()
    a.B, a.T, a.Hkv, a.D = B, T, Hkv, D
    a.k_tree, a.v_tree, a.k_cache, a.v_cache = _p(k_tree), _p(v_tree), _p(k_cache), _p(v_cache)
    if block_table is None:
        a.kv_layout, a.Lmax = KV_CONTIGUOUS, k_cache.shape[1]
        a.num_blocks, a.block_size, a.max_blocks_per_seq = 0, 0, 0
    else:
        a.kv_layout, a.Lmax = KV_PAGED, 0
        a.num_blocks, a.block_size, a.max_blocks_per_seq = k_cache.shape[0], block_size, block_table.shape[1]
    a.block_table, a.ctx_len, a.path, a.accept_len = _p(block_table), _p(ctx_len), _p(path), _p(accept_len)
    a.active, a.ctx_len_out, a.dev_status = _p(active), _p(ctx_len_out), _p(dev_status)
    return _hold(a, k_tree, v_tree, k_cache, v_cache, ctx_len, path, accept_len, ctx_len_out, block_table, active,
                 dev_status)


def alloc_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    return torch.empty(max(256, (nbytes + 255) // 256 * 256), dtype=torch.uint8, device=device)


# ------------------------------------------------------------------------------ entry points
def trispec_build_tree_mask(args: TreeArgs, stream=None):
    _check(_lib.trispec_build_tree_mask(C.byref(args), _stream(stream)))


def trispec_verify_attn_workspace(args: AttnArgs) -> int:
    return int(_lib.trispec_verify_attn_workspace(C.byref(args)))


def trispec_verify_attn_plan(args: AttnArgs) -> str:
    return _lib.trispec_verify_attn_plan(C.byref(args)).decode()


def trispec_verify_plan(attn: Optional[AttnArgs], lm: LmheadArgs, scan: Optional[ScanArgs] = None) -> str:
    return _lib.trispec_verify_plan(C.byref(attn) if attn is not None else None, C.byref(lm),
                                    C.byref(scan) if scan is not None else None).decode()


def trispec_verify_attn(args: AttnArgs, stream=None):
    _check(_lib.trispec_verify_attn(C.byref(args), _stream(stream)))


def trispec_prune_tree(args: PruneArgs, stream=None):
    _check(_lib.trispec_prune_tree(C.byref(args), _stream(stream)))


def sample_args(h, W, last_node, bonus_tok, logit_scale, seed, step, sample_value=None, workspace=None,
                dev_status=None) -> SampleArgs:
    B, T = last_node.shape[0], h.numel() // (last_node.shape[0] * h.shape[-1])
    a = SampleArgs()
    a.B, a.T, a.d, a.V, a.logit_scale = B, T, h.shape[-1], W.shape[0], float(logit_scale)
    a.h, a.W, a.last_node, a.bonus_tok, a.sample_value = _p(h), _p(W), _p(last_node), _p(bonus_tok), _p(sample_value)
    a.seed, a.step = int(seed), int(step)
    a.workspace = _p(workspace)
    a.workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    a.dev_status = _p(dev_status)
    return _hold(a, h, W, last_node, bonus_tok, sample_value, workspace, dev_status)


def trispec_sample_bonus_workspace(args: SampleArgs) -> int:
    return int(_lib.trispec_sample_bonus_workspace(C.byref(args)))


def trispec_sample_bonus(args: SampleArgs, stream=None):
    _check(_lib.trispec_sample_bonus(C.byref(args), _stream(stream)))


def trispec_commit_kv(args: CommitArgs, stream=None):
    _check(_lib.trispec_commit_kv(C.byref(args), _stream(stream)))


def trispec_lmhead_stats_workspace(args: LmheadArgs) -> int:
    return int(_lib.trispec_lmhead_stats_workspace(C.byref(args)))


def trispec_lmhead_stats(args: LmheadArgs, stream=None):
    _check(_lib.trispec_lmhead_stats(C.byref(args), _stream(stream)))


NOALLOC_SCRATCH_BYTES = 1 << 20


def trispec_lmhead_stats_noalloc(args: LmheadArgs, stream=None):
    """LM-head statistics without a caller workspace (the library's built-in 1 MiB scratch is
    used; `args.workspace` is ignored). For callers that must not allocate device memory."""
    _check(_lib.trispec_lmhead_stats_noalloc(C.byref(args), _stream(stream)))


def trispec_accept_scan(args: ScanArgs, stream=None):
    _check(_lib.trispec_accept_scan(C.byref(args), _stream(stream)))


def trispec_verify(tree: TreeArgs, attn: Optional[AttnArgs], lm: LmheadArgs, scan: ScanArgs, stream=None):
    _check(_lib.trispec_verify(C.byref(tree), None if attn is None else C.byref(attn), C.byref(lm),
                               C.byref(scan), _stream(stream)))


def host_io(**host_tensors) -> HostIO:
    """HostIO from (pinned) CPU tensors; names as in the C struct, missing ones stay NULL."""
    io = HostIO()
    for name, _ in HostIO._fields_:
        t = host_tensors.get(name)
        setattr(io, name, None if t is None else _p(t))
    return io


def trispec_verify_host(io: HostIO, tree: TreeArgs, attn: Optional[AttnArgs], lm: LmheadArgs, scan: ScanArgs,
                        stream=None):
    _check(_lib.trispec_verify_host(C.byref(io), C.byref(tree), None if attn is None else C.byref(attn),
                                    C.byref(lm), C.byref(scan), _stream(stream)))
