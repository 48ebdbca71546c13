"""Seeded synthetic inputs for the TriSpec verify pass.

This module only *draws* inputs (draft trees, tokens, bf16 tensors); it holds none of the
method's arithmetic (no mask, no attention, no softmax statistics, no acceptance rule), so
it can feed both the CUDA path and the CPU oracle without coupling them.

All floating-point tensors are produced as bf16 bit patterns (``uint16``), rounded once here
(round-to-nearest-even), so every consumer sees identical bits.

Randomness: numpy Philox streams keyed by (seed, tensor tag, sequence index), so any tensor
can be regenerated alone and sequences are independent of the batch size.

Workload shapes follow the paper's setup (EAGLE-2 style draft tree: depth 6, 60 draft tokens,
margin threshold 0.5; Section 4.1 "Setup") and the model families it evaluates.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, Optional

import numpy as np

MODE_PROXY = 0
MODE_TARGET = 1

_TAGS = {
    "tree": 1, "tok": 2, "q": 3, "k_tree": 4, "v_tree": 5, "k_cache": 6, "v_cache": 7,
    "W": 8, "h_noise": 9, "h_plan": 10, "ctx_len": 11, "block_perm": 12, "active": 13,
}


def _rng(seed: int, tag: str, idx: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), (_TAGS[tag] << 40) | int(idx)]))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclasses.dataclass(frozen=True)
class VerifyConfig:
    """One verify-pass workload. k draft tokens per sequence, T = k + 1 tree nodes (node 0 is
    the last committed token, whose distribution is the paper's p_1; Eq. 2 / Eq. 5)."""
    name: str
    B: int
    k: int
    tree: str            # "chain" or "random"
    max_depth: int       # depth of the deepest draft node (random trees)
    L: int               # maximum committed context length
    Hq: int
    Hkv: int
    d: int               # hidden size
    V: int               # vocabulary size
    logit_scale: float
    p_conf: float = 0.7  # weight of the confident (alpha = 8) mixture component
    L_min: Optional[int] = None   # ragged context lengths uniform in [L_min, L]
    paged: bool = False
    block_size: int = 64
    mode: int = MODE_PROXY
    n_active: Optional[int] = None  # verify only this many (seed-chosen) sequences
    rho: float = 0.0     # prob. that a confident non-leaf node favours a non-child token
    lam: float = 0.5     # margin threshold lambda
    D: int = 128
    seed: int = 0

    @property
    def T(self) -> int:
        return self.k + 1


CONFIGS: Dict[str, VerifyConfig] = {
    # 1: tiny chain verify
    "tiny_chain": VerifyConfig("tiny_chain", B=1, k=8, tree="chain", max_depth=8, L=512,
                               Hq=16, Hkv=8, d=2048, V=32000, logit_scale=4.0),
    # 2: proxy-shaped tree verify (the headline workload)
    "proxy_tree": VerifyConfig("proxy_tree", B=8, k=60, tree="random", max_depth=6, L=4096,
                               Hq=16, Hkv=8, d=2048, V=151936, logit_scale=4.0),
    # 3: target-scale verify for escalated sequences
    "target_escalated": VerifyConfig("target_escalated", B=8, k=60, tree="random", max_depth=6,
                                     L=16384, Hq=64, Hkv=8, d=5120, V=151936, logit_scale=2.5,
                                     mode=MODE_TARGET, n_active=3),
    # 4: LLaMA-family shape
    "llama_tree": VerifyConfig("llama_tree", B=16, k=48, tree="random", max_depth=8, L=8192,
                               Hq=32, Hkv=8, d=4096, V=128256, logit_scale=3.0, p_conf=0.6),
    # 5: long-reasoning, memory-bound stress (ragged, paged)
    "long_paged": VerifyConfig("long_paged", B=64, k=60, tree="random", max_depth=6, L=32768,
                               L_min=8192, Hq=16, Hkv=8, d=2048, V=151936, logit_scale=4.0,
                               paged=True),
}
CONFIG_ORDER = ["tiny_chain", "proxy_tree", "target_escalated", "llama_tree", "long_paged"]


def small_variant(cfg: VerifyConfig, **over) -> VerifyConfig:
    """A reduced copy of a config for element-by-element parity tests (same structure)."""
    return dataclasses.replace(cfg, **over)


# --------------------------------------------------------------------------------------
# draft trees and tokens
# --------------------------------------------------------------------------------------
def make_tree(cfg: VerifyConfig, b: int) -> np.ndarray:
    """Parent-index array of one draft tree: parent[0] = -1, parent[i] < i, siblings adjacent.

    "random": a spine 0 -> 1 -> ... -> max_depth fixes the depth, the remaining nodes are
    attached one at a time under a uniformly chosen node that is not at max depth and has
    fewer than 4 children; nodes are then relabelled in (depth, parent) order.
    """
    T = cfg.T
    if cfg.tree == "chain":
        return np.arange(-1, T - 1, dtype=np.int32)
    g = _rng(cfg.seed, "tree", b)
    Dm = min(cfg.max_depth, T - 1)
    par = [-1] + list(range(Dm))
    dep = list(range(Dm + 1))
    nch = [1] * Dm + [0]
    while len(par) < T:
        cand = [i for i in range(len(par)) if dep[i] < Dm and nch[i] < 4]
        p = cand[int(g.integers(len(cand)))]
        par.append(p)
        dep.append(dep[p] + 1)
        nch.append(0)
        nch[p] += 1
    # relabel breadth-first so that parent[i] < i and the children of a node are contiguous
    order = [0]
    children = [[] for _ in range(T)]
    for i in range(1, T):
        children[par[i]].append(i)
    head = 0
    while head < len(order):
        order.extend(children[order[head]])
        head += 1
    new_id = {old: new for new, old in enumerate(order)}
    out = np.full(T, -1, dtype=np.int32)
    for old in range(1, T):
        out[new_id[old]] = new_id[par[old]]
    return out


def make_tokens(cfg: VerifyConfig, b: int, parent: np.ndarray) -> np.ndarray:
    """Draft tokens, uniform over the vocabulary, distinct among siblings."""
    g = _rng(cfg.seed, "tok", b)
    T = cfg.T
    tok = g.integers(0, cfg.V, size=T).astype(np.int32)
    for p in range(T):
        kids = np.nonzero(parent == p)[0]
        seen = set()
        for c in kids:
            while int(tok[c]) in seen:
                tok[c] = int(g.integers(0, cfg.V))
            seen.add(int(tok[c]))
    return tok


# --------------------------------------------------------------------------------------
# bf16 tensors
# --------------------------------------------------------------------------------------
def _normal_bf16(g: np.random.Generator, shape, std: float = 1.0) -> np.ndarray:
    x = g.standard_normal(shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return f32_to_bf16_bits(x)


def _parallel_fill(out: np.ndarray, seed: int, tag: str, std: float = 1.0, threads: int = 8):
    """Fill out[i] (first axis) with N(0, std^2) bf16 bits, one keyed stream per index."""
    def job(i):
        out[i] = _normal_bf16(_rng(seed, tag, i), out.shape[1:], std)
    n = out.shape[0]
    if n <= 1 or out[0].size < (1 << 16):
        for i in range(n):
            job(i)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(job, range(n)))


def make_lm_head(cfg: VerifyConfig) -> np.ndarray:
    """LM-head weights W ~ N(0, 0.02^2), bf16 bits, [V][d]; generated in slabs of 4096 rows."""
    W = np.empty((cfg.V, cfg.d), dtype=np.uint16)
    slab = 4096
    n = (cfg.V + slab - 1) // slab

    def job(i):
        r0, r1 = i * slab, min(cfg.V, (i + 1) * slab)
        W[r0:r1] = _normal_bf16(_rng(cfg.seed, "W", i), (r1 - r0, cfg.d), 0.02)
    with ThreadPoolExecutor(max_workers=8) as ex:
        list(ex.map(job, range(n)))
    return W


def make_hidden(cfg: VerifyConfig, W: np.ndarray, parent: np.ndarray, tok: np.ndarray) -> Dict[str, np.ndarray]:
    """Final hidden states h[b][node] = alpha * W[y] / ||W[y]|| + N(0, I), bf16 bits.

    y is the token of one favoured child (uniformly chosen) for a non-leaf node and a uniform
    random token for a leaf; with probability rho a confident non-leaf node favours a random
    non-child token instead (exercises the "confident rejection" branch). alpha is 8 with
    probability p_conf and 1 otherwise.
    """
    B, T, d = cfg.B, cfg.T, cfg.d
    h = np.empty((B, T, d), dtype=np.uint16)
    alpha = np.empty((B, T), dtype=np.float32)
    fav = np.empty((B, T), dtype=np.int32)
    for b in range(B):
        g = _rng(cfg.seed, "h_plan", b)
        for r in range(T):
            kids = np.nonzero(parent[b] == r)[0]
            a = 8.0 if g.random() < cfg.p_conf else 1.0
            stray = g.random() < cfg.rho
            rnd_tok = int(g.integers(0, cfg.V))
            pick = int(g.integers(0, max(1, len(kids))))
            if len(kids) == 0 or (stray and a == 8.0):
                y = rnd_tok
            else:
                y = int(tok[b, kids[pick]])
            alpha[b, r] = a
            fav[b, r] = y
        w = bf16_bits_to_f32(W[fav[b]]).astype(np.float64)           # [T][d]
        w /= np.linalg.norm(w, axis=1, keepdims=True)
        noise = _rng(cfg.seed, "h_noise", b).standard_normal((T, d), dtype=np.float32)
        h[b] = f32_to_bf16_bits((alpha[b][:, None] * w + noise).astype(np.float32))
    return {"h": h, "alpha": alpha, "favoured_tok": fav}


def make_inputs(cfg: VerifyConfig, with_lm_head: bool = True, with_attention: bool = True,
                W: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """All inputs of one verify pass as numpy arrays (bf16 tensors as uint16 bit patterns).

    Layouts: q [B][T][Hq][D]; k_tree, v_tree [B][T][Hkv][D]; contiguous cache
    k_cache, v_cache [B][L][Hkv][D]; paged cache pool [num_blocks][block][Hkv][D] with
    block_table int32 [B][max_blocks] (a seeded permutation of the pool) and ctx_len int32 [B];
    h [B][T][d]; W [V][d]; parent, tok int32 [B][T]; seq_index int32 [n_active] or None.
    """
    B, T = cfg.B, cfg.T
    out: Dict[str, np.ndarray] = {}
    parent = np.stack([make_tree(cfg, b) for b in range(B)])
    tok = np.stack([make_tokens(cfg, b, parent[b]) for b in range(B)])
    out["parent"], out["tok"] = parent, tok

    if cfg.L_min is None:
        ctx_len = np.full(B, cfg.L, dtype=np.int32)
    else:
        ctx_len = _rng(cfg.seed, "ctx_len").integers(cfg.L_min, cfg.L + 1, size=B).astype(np.int32)
    out["ctx_len"] = ctx_len

    if cfg.n_active is not None:
        perm = _rng(cfg.seed, "active").permutation(B)
        out["seq_index"] = np.sort(perm[:cfg.n_active]).astype(np.int32)
    else:
        out["seq_index"] = None

    if with_attention:
        q = np.empty((B, T, cfg.Hq, cfg.D), dtype=np.uint16)
        kt = np.empty((B, T, cfg.Hkv, cfg.D), dtype=np.uint16)
        vt = np.empty_like(kt)
        _parallel_fill(q, cfg.seed, "q")
        _parallel_fill(kt, cfg.seed, "k_tree")
        _parallel_fill(vt, cfg.seed, "v_tree")
        out["q"], out["k_tree"], out["v_tree"] = q, kt, vt
        if cfg.paged:
            bs = cfg.block_size
            max_blocks = (cfg.L + bs - 1) // bs
            need = (ctx_len.astype(np.int64) + bs - 1) // bs
            num_blocks = int(need.sum())
            perm = _rng(cfg.seed, "block_perm").permutation(num_blocks).astype(np.int32)
            table = np.full((B, max_blocks), -1, dtype=np.int32)
            o = 0
            for b in range(B):
                table[b, :need[b]] = perm[o:o + need[b]]
                o += int(need[b])
            kc = np.empty((num_blocks, bs, cfg.Hkv, cfg.D), dtype=np.uint16)
            vc = np.empty_like(kc)
            # fill in chunks of 256 blocks so that the streams do not depend on thread count
            ch = 256
            kcv = [kc[i:i + ch] for i in range(0, num_blocks, ch)]
            vcv = [vc[i:i + ch] for i in range(0, num_blocks, ch)]

            def job(i):
                kcv[i][...] = _normal_bf16(_rng(cfg.seed, "k_cache", i), kcv[i].shape)
                vcv[i][...] = _normal_bf16(_rng(cfg.seed, "v_cache", i), vcv[i].shape)
            with ThreadPoolExecutor(max_workers=8) as ex:
                list(ex.map(job, range(len(kcv))))
            out["block_table"] = table
        else:
            kc = np.empty((B, cfg.L, cfg.Hkv, cfg.D), dtype=np.uint16)
            vc = np.empty_like(kc)
            _parallel_fill(kc, cfg.seed, "k_cache")
            _parallel_fill(vc, cfg.seed, "v_cache")
            out["block_table"] = None
        out["k_cache"], out["v_cache"] = kc, vc

    if with_lm_head:
        if W is None:
            W = make_lm_head(cfg)
        out["W"] = W
        out.update(make_hidden(cfg, W, parent, tok))
    return out
