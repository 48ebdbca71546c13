"""CPU oracle for the TriSpec verify pass — TEST INFRASTRUCTURE, not a product path.

Plain, slow, fp64 numpy restatement of what the verification pass computes, written from
the paper's definitions. It shares no code with the CUDA path and must only be used by the
tests, the smoke check and the benchmark's CPU-baseline leg.

What each function follows:
  build_tree_mask  tree attention mask of a draft tree (Figure 4, "attention mask updates";
                   tree configuration of Section 4.1): a node sees its ancestors and itself.
  verify_attn      the attention of one parallel verification pass (Eq. 2 / Eq. 5): every
                   tree node attends to the whole committed context plus the tree keys its
                   mask row allows; plain softmax(q k / sqrt(D)) v.
  lmhead_stats     per-position softmax distribution p_i in R^V (Eq. 5) reduced to the
                   quantities the rule needs: top_1(p), top_2(p) (Eq. 8), argmax token x_i^(p)
                   (greedy form of Eq. 6) and p_i(x_i^(d)) for each drafted child.
  accept_scan      greedy acceptance s_i (Eq. 6), acceptance length tau_a (Eq. 7), margin
                   predicate g (Eq. 8), trusted prefix tau_m (Eq. 9) and the routing cases
                   (i)/(ii) of "Adaptive Verification Routing" / Algorithm 1; TARGET mode is
                   the "standard left-to-right acceptance rule" applied after Eq. 10.
  prune_tree       token pruning of routing case (ii) ("prune these tokens from the draft tree
                   and pass the remaining branches to the target"; ablation on token pruning).
  accept_scan_token_specific
                   the token-specific deferral rule of the SpecCascade baselines (appendix
                   "Baseline Implementation Details: SpecCascade") as an acceptance rule.
  accept_scan_stochastic, sample_bonus
                   Eq. 6 at temperature 1 and the bonus draw of Algorithm 1 (Gumbel-max with
                   counter-based Philox noise).
  commit_kv        X <- X + Y of Algorithm 1 as the KV cache sees it: the keys/values of the
                   last committed token and of the accepted draft tokens are appended.

Readings of the paper taken here (the paper states the rule for a chain of k tokens):
  * Tree rule = the chain rule applied along the path the greedy matches select; the margin
    test at a node precedes the child match (if g = 0 at depth j then tau_m = j and, all
    earlier tokens having matched, tau_a >= j: case (ii)).
  * top_2 is the largest entry among indices other than the arg-max (two equal maxima give
    margin 0). Ties resolve to the lowest vocabulary index; duplicate sibling tokens resolve
    to the lowest node index.
  * Parity of the tree rule is pinned by brute force over all root-to-leaf paths in the tests;
    the end-to-end behaviour of the paper's models (acceptance lengths, speedups) is
    "parity unpinned": it needs the paper's models and datasets.
"""
from __future__ import annotations

from typing import Dict, Iterable, Optional, Sequence, Tuple

import numpy as np

MODE_PROXY = 0
MODE_TARGET = 1
# routing criteria of the "Routing Criteria" study: which proxy feature decides trust at a position
CRIT_MARGIN = 0    # top_1(p) - top_2(p) >= lambda   (Eq. 8, the default)
CRIT_TOP1 = 1      # top_1(p) >= lambda
CRIT_ENTROPY = 2   # H(p) <= lambda


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float64 values (exact)."""
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


# ----------------------------------------------------------------------------------------
# tree mask (Figure 4; Section 4.1 tree configuration)
# ----------------------------------------------------------------------------------------
def build_tree_mask(parent: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """mask[b][i] has bit j set iff j is an ancestor of i or j == i; depth[b][i] = number of
    edges from the root. parent[b][0] = -1 and parent[b][i] < i; T <= 64."""
    parent = np.asarray(parent)
    B, T = parent.shape
    assert T <= 64
    mask = np.zeros((B, T), dtype=np.uint64)
    depth = np.zeros((B, T), dtype=np.int32)
    for b in range(B):
        for i in range(T):
            bits = 0
            steps = 0
            p = i
            while p >= 0:
                bits |= (1 << p)
                p = int(parent[b, p])
                steps += 1
            mask[b, i] = np.uint64(bits)
            depth[b, i] = steps - 1
    return mask, depth


# ----------------------------------------------------------------------------------------
# verification attention (Eq. 2 / Eq. 5: one parallel pass over the drafted tokens)
# ----------------------------------------------------------------------------------------
def _context_kv(cache_bits: np.ndarray, b: int, kvh: int, L: int,
                block_table: Optional[np.ndarray], block_size: int) -> np.ndarray:
    """[L][D] fp64 keys or values of sequence b, KV head kvh. Contiguous cache is
    [B][Lmax][Hkv][D]; a paged pool is [num_blocks][block][Hkv][D] and token t lives in block
    block_table[b][t // block], slot t % block."""
    if block_table is None:
        return bf16_to_f64(cache_bits[b, :L, kvh, :])
    t = np.arange(L)
    blk = block_table[b, t // block_size]
    return bf16_to_f64(cache_bits[blk, t % block_size, kvh, :])


def verify_attn(q: np.ndarray, k_tree: np.ndarray, v_tree: np.ndarray, mask: np.ndarray,
                k_cache: np.ndarray, v_cache: np.ndarray, ctx_len: np.ndarray, scale: float,
                block_table: Optional[np.ndarray] = None, block_size: int = 64,
                seqs: Optional[Iterable[int]] = None,
                samples: Optional[Sequence[Tuple[int, int, int]]] = None):
    """o[b][i][h] = sum_j softmax_j(scale * q[b][i][h] . k_j) v_j over the visible keys j:
    all ctx_len[b] context positions and the tree nodes whose bit is set in mask[b][i].
    KV head of query head h is h // (Hq // Hkv).

    Returns (o float64 [B][T][Hq][D], lse float64 [B][Hq][T]); entries that were not asked for
    (seqs / samples restrict the work) are NaN. `samples` is a list of (b, i, h)."""
    B, T, Hq, D = q.shape
    Hkv = k_tree.shape[2]
    G = Hq // Hkv
    o = np.full((B, T, Hq, D), np.nan)
    lse = np.full((B, Hq, T), np.nan)
    if samples is None:
        bs = range(B) if seqs is None else list(seqs)
        todo = {}
        for b in bs:
            for g in range(Hkv):
                todo[(b, g)] = [(i, h) for h in range(g * G, (g + 1) * G) for i in range(T)]
    else:
        todo = {}
        for (b, i, h) in samples:
            todo.setdefault((int(b), int(h) // G), []).append((int(i), int(h)))
    for (b, g), items in todo.items():
        L = int(ctx_len[b])
        Kc = _context_kv(k_cache, b, g, L, block_table, block_size)
        Vc = _context_kv(v_cache, b, g, L, block_table, block_size)
        Kt = bf16_to_f64(k_tree[b, :, g, :])
        Vt = bf16_to_f64(v_tree[b, :, g, :])
        for (i, h) in items:
            qi = bf16_to_f64(q[b, i, h, :])
            vis = [j for j in range(T) if (int(mask[b, i]) >> j) & 1]
            s = np.concatenate([Kc @ qi, Kt[vis] @ qi]) * scale
            m = s.max()
            e = np.exp(s - m)
            den = e.sum()
            p = e / den
            o[b, i, h, :] = p[:L] @ Vc + p[L:] @ Vt[vis]
            lse[b, h, i] = m + np.log(den)
    return o, lse


# ----------------------------------------------------------------------------------------
# LM-head softmax statistics (Eq. 5 distributions; top_1/top_2 of Eq. 8)
# ----------------------------------------------------------------------------------------
STAT_F = ("max", "lse", "top1_val", "top2_val", "top3_val", "p_top1", "p_top2", "draft_logit", "p_draft",
          "entropy")
STAT_I = ("top1_idx", "top2_idx")


def row_logits(h_row_bits: np.ndarray, W64: np.ndarray, logit_scale: float) -> np.ndarray:
    """z_v = logit_scale * <h, W_v> for every vocabulary entry v (fp64)."""
    return logit_scale * (W64 @ bf16_to_f64(h_row_bits))


def lmhead_stats(h: np.ndarray, W: np.ndarray, parent: np.ndarray, tok: np.ndarray,
                 logit_scale: float, seqs: Optional[Iterable[int]] = None,
                 W64: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Per row r = (b, node): p = softmax(z) over the vocabulary, reduced to
    max z, lse = log sum exp z, the largest entry (top1_val, top1_idx; ties -> lowest index),
    the largest entry among the other indices (top2_val, top2_idx), the largest entry among the
    rest (top3_val; reported so that a comparison can tell when top2_idx sits on a tie), p_top1,
    p_top2; and for
    each child node c the logit of its drafted token in its parent's row (draft_logit[b][c])
    and the probability p_draft[b][c] = p_{parent(c)}(tok[c]). Entries of node 0 in
    draft_logit / p_draft are NaN. entropy = -sum_v p ln p (nats), the feature of the entropy
    routing criterion of the "Routing Criteria" study. h is [B][T][d] bf16 bits, W is [V][d] bf16 bits.
    All outputs are [B][T]; rows of sequences not in `seqs` are NaN / -1."""
    B, T, d = h.shape
    if W64 is None:
        W64 = bf16_to_f64(W)
    out = {k: np.full((B, T), np.nan) for k in STAT_F}
    out.update({k: np.full((B, T), -1, dtype=np.int64) for k in STAT_I})
    for b in (range(B) if seqs is None else seqs):
        for r in range(T):
            z = row_logits(h[b, r], W64, logit_scale)
            m = z.max()
            lse = m + np.log(np.exp(z - m).sum())
            i1 = int(np.argmax(z))                 # first occurrence = lowest index
            z_wo = z.copy()
            z_wo[i1] = -np.inf
            i2 = int(np.argmax(z_wo))
            z_wo[i2] = -np.inf
            # third largest entry: only for the parity tests' accounting of near-ties behind top_2
            out["top3_val"][b, r] = z_wo.max() if len(z) > 2 else np.nan
            out["max"][b, r] = m
            out["lse"][b, r] = lse
            out["top1_val"][b, r] = z[i1]
            out["top2_val"][b, r] = z[i2]
            out["top1_idx"][b, r] = i1
            out["top2_idx"][b, r] = i2
            out["p_top1"][b, r] = np.exp(z[i1] - lse)
            out["p_top2"][b, r] = np.exp(z[i2] - lse)
            p = np.exp(z - lse)
            nz = p > 0
            out["entropy"][b, r] = -(p[nz] * (z[nz] - lse)).sum()     # -sum p ln p, in nats
            for c in range(1, T):
                if int(parent[b, c]) == r:
                    out["draft_logit"][b, c] = z[int(tok[b, c])]
                    out["p_draft"][b, c] = np.exp(z[int(tok[b, c])] - lse)
    return out


# ----------------------------------------------------------------------------------------
# acceptance scan (Eq. 6-9, routing cases (i)/(ii), Algorithm 1)
# ----------------------------------------------------------------------------------------
def accept_scan(p_top1: np.ndarray, p_top2: np.ndarray, top1_idx: np.ndarray,
                parent: np.ndarray, tok: np.ndarray, lam: float, mode: int = MODE_PROXY,
                active: Optional[np.ndarray] = None,
                start_node: Optional[np.ndarray] = None,
                near_eps: float = 1e-3, criterion: int = CRIT_MARGIN,
                entropy: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Greedy walk of each draft tree.

    At the current node (position i+1 of the chain formulas, i = tokens accepted so far):
      PROXY mode: if top_1(p) - top_2(p) < lambda the position is untrusted: tau_m = i, and as
        every earlier token matched tau_a >= tau_m: case (ii), accept x_{1:tau_m}, escalate.
      Otherwise look for the child whose drafted token equals the arg-max token (s_{i+1} = 1):
        none -> tau_a = i < tau_m: case (i), approve, bonus = arg-max token of this node;
        found -> accept it and move there.
      TARGET mode: the same without the margin test (never escalates).
    `criterion` replaces the margin by another proxy feature (the paper's routing-criteria
    study): CRIT_TOP1 trusts a position iff top_1(p) >= lambda, CRIT_ENTROPY iff the entropy of
    p is <= lambda (reading: plain Shannon entropy in nats; the paper cites a "composite"
    entropy criterion without defining it).

    Outputs per sequence: accept_len, escalate (0/1), bonus_tok (-1 if escalated), path
    [B][T] (accepted node ids in order, -1 padded), last_node, near_thr (number of visited
    positions with |feature - lambda| < near_eps; PROXY mode only); plus n_escalated and
    esc_index (ascending sequence ids that escalated, -1 padded). Inactive sequences get
    accept_len 0, escalate 0, bonus -1, last_node -1.
    """
    parent = np.asarray(parent)
    B, T = parent.shape
    res = {
        "accept_len": np.zeros(B, dtype=np.int32),
        "escalate": np.zeros(B, dtype=np.uint8),
        "bonus_tok": np.full(B, -1, dtype=np.int32),
        "path": np.full((B, T), -1, dtype=np.int32),
        "last_node": np.full(B, -1, dtype=np.int32),
        "near_thr": np.zeros(B, dtype=np.int32),
    }
    for b in range(B):
        if active is not None and not active[b]:
            continue
        cur = 0 if start_node is None else int(start_node[b])
        n = 0
        while True:
            if mode == MODE_PROXY:
                if criterion == CRIT_MARGIN:
                    feature = float(p_top1[b, cur]) - float(p_top2[b, cur])
                    trusted = feature >= lam
                elif criterion == CRIT_TOP1:
                    feature = float(p_top1[b, cur])
                    trusted = feature >= lam
                else:
                    feature = float(entropy[b, cur])
                    trusted = feature <= lam
                if abs(feature - lam) < near_eps:
                    res["near_thr"][b] += 1
                if not trusted:
                    res["escalate"][b] = 1
                    break
            nxt = -1
            for c in range(cur + 1, T):
                if int(parent[b, c]) == cur and int(tok[b, c]) == int(top1_idx[b, cur]):
                    nxt = c
                    break
            if nxt < 0:
                res["bonus_tok"][b] = int(top1_idx[b, cur])
                break
            res["path"][b, n] = nxt
            n += 1
            cur = nxt
        res["accept_len"][b] = n
        res["last_node"][b] = cur
    esc = np.nonzero(res["escalate"])[0].astype(np.int32)
    res["n_escalated"] = np.int32(len(esc))
    res["esc_index"] = np.full(B, -1, dtype=np.int32)
    res["esc_index"][:len(esc)] = esc
    return res


# ----------------------------------------------------------------------------------------
# the whole pass
# ----------------------------------------------------------------------------------------
def verify(inp: Dict[str, np.ndarray], scale: float, logit_scale: float, lam: float,
           mode: int = MODE_PROXY, block_size: int = 64, with_attention: bool = True):
    """Mask -> attention -> LM-head statistics -> acceptance scan, on the arrays produced by
    the input generator. Only sequences listed in inp["seq_index"] (all if None) are verified."""
    parent, tok = inp["parent"], inp["tok"]
    B = parent.shape[0]
    seqs = list(range(B)) if inp.get("seq_index") is None else [int(s) for s in inp["seq_index"]]
    active = np.zeros(B, dtype=np.uint8)
    active[seqs] = 1
    mask, depth = build_tree_mask(parent)
    out = {"mask": mask, "depth": depth}
    if with_attention:
        o, lse = verify_attn(inp["q"], inp["k_tree"], inp["v_tree"], mask, inp["k_cache"],
                             inp["v_cache"], inp["ctx_len"], scale,
                             block_table=inp.get("block_table"), block_size=block_size, seqs=seqs)
        out["o"], out["attn_lse"] = o, lse
    st = lmhead_stats(inp["h"], inp["W"], parent, tok, logit_scale, seqs=seqs)
    out["stats"] = st
    out["scan"] = accept_scan(st["p_top1"], st["p_top2"], st["top1_idx"], parent, tok, lam,
                              mode=mode, active=active)
    return out


# ----------------------------------------------------------------------------------------
# token pruning (routing case (ii): "prune these tokens from the draft tree and pass the
# remaining branches to the target"; ablation "Token pruning strategies")
# ----------------------------------------------------------------------------------------
def prune_tree(parent: np.ndarray, tok: np.ndarray, root: np.ndarray) -> Dict[str, np.ndarray]:
    """The branches that remain after the proxy accepted a prefix: the subtree below the last
    accepted node root[b] (that node becomes node 0 of the new tree: it is the last committed
    token of the next verifier). Nodes keep their relative order, so parent'[i] < i still holds.

    Outputs, all padded to the input width T: n_keep [B]; node_map [B][T] (new index -> old
    index, -1 beyond n_keep); parent' and tok' [B][T] (-1 beyond n_keep; parent'[0] = -1).
    root[b] < 0 (sequence not escalated) gives n_keep 0 and all -1.
    Reading: "remaining branches" = descendants of the last accepted node; every other branch
    contradicts the accepted prefix."""
    parent = np.asarray(parent)
    B, T = parent.shape
    out = {"n_keep": np.zeros(B, dtype=np.int32), "node_map": np.full((B, T), -1, dtype=np.int32),
           "parent": np.full((B, T), -1, dtype=np.int32), "tok": np.full((B, T), -1, dtype=np.int32)}
    for b in range(B):
        r = int(root[b])
        if r < 0:
            continue
        new_of = {}
        for i in range(T):
            # i is kept iff walking up from i meets r
            p = i
            while p >= 0 and p != r:
                p = int(parent[b, p])
            if p == r:
                new_of[i] = len(new_of)
        for i, j in new_of.items():
            out["node_map"][b, j] = i
            out["tok"][b, j] = tok[b, i]
            out["parent"][b, j] = -1 if i == r else new_of[int(parent[b, i])]
        out["n_keep"][b] = len(new_of)
    return out


# ----------------------------------------------------------------------------------------
# KV commit of the accepted path (the step after a verification round in the decode loop:
# X <- X + Y of Algorithm 1 seen from the KV cache)
# ----------------------------------------------------------------------------------------
def commit_kv(k_cache: np.ndarray, v_cache: np.ndarray, ctx_len: np.ndarray, k_tree: np.ndarray,
              v_tree: np.ndarray, path: np.ndarray, accept_len: np.ndarray,
              block_table: Optional[np.ndarray] = None, block_size: int = 64,
              active: Optional[np.ndarray] = None):
    """Appends to each sequence's cache the keys/values of tree node 0 (the last committed token,
    whose K/V were not in the cache yet) and of the accept_len[b] accepted nodes path[b][:n], in
    that order, at positions ctx_len[b], ctx_len[b] + 1, ...; returns (k_cache', v_cache',
    ctx_len') as new arrays. Layouts as in verify_attn (contiguous [B][L][Hkv][D] or paged pool
    + block_table). A sequence whose new length would exceed its capacity is left unchanged."""
    kc, vc = np.array(k_cache, copy=True), np.array(v_cache, copy=True)
    new_len = np.array(ctx_len, dtype=np.int32, copy=True)
    B = k_tree.shape[0]
    for b in range(B):
        if active is not None and not active[b]:
            continue
        n = int(accept_len[b])
        nodes = [0] + [int(path[b, j]) for j in range(n)]
        L = int(ctx_len[b])
        cap = kc.shape[1] if block_table is None else int((np.asarray(block_table[b]) >= 0).sum()) * block_size
        if L + len(nodes) > cap:
            continue
        for j, node in enumerate(nodes):
            t = L + j
            if block_table is None:
                kc[b, t] = k_tree[b, node]
                vc[b, t] = v_tree[b, node]
            else:
                blk = int(block_table[b, t // block_size])
                kc[blk, t % block_size] = k_tree[b, node]
                vc[blk, t % block_size] = v_tree[b, node]
        new_len[b] = L + len(nodes)
    return kc, vc, new_len


# ----------------------------------------------------------------------------------------
# stochastic acceptance (Eq. 6 at temperature 1) and bonus sampling (Algorithm 1:
# x_bonus ~ p_{tau_a + 1})
# ----------------------------------------------------------------------------------------
def accept_scan_stochastic(p_top1: np.ndarray, p_top2: np.ndarray, p_draft: np.ndarray,
                           q_draft: np.ndarray, u: np.ndarray, parent: np.ndarray, tok: np.ndarray,
                           lam: float, mode: int = MODE_PROXY, active: Optional[np.ndarray] = None,
                           near_eps: float = 1e-3, near_accept_eps: float = 1e-6) -> Dict[str, np.ndarray]:
    """The walk of accept_scan with the Bernoulli acceptance of Eq. 6 in place of the arg-max
    match: a drafted child c is accepted iff u[c] < min(1, p_draft[c] / q_draft[c]), where
    p_draft[c] is the verifier's probability of tok[c] at c's parent, q_draft[c] the drafter's,
    and u[c] a uniform number in [0, 1) supplied by the caller. The decision is taken in fp64
    whatever the precision of the arrays; a drafter probability of 0 counts as ratio 1.
    Readings: the paper states the rule for a chain; on a tree the children of the current node
    are tried in node order and the first accepted one is taken. When no child is accepted the
    round ends in case (i) and the bonus token has to be SAMPLED from the current node's
    distribution (Algorithm 1), which this function cannot do from statistics: it returns
    bonus_tok = -2 for "sample at last_node". The margin test precedes the children as in
    accept_scan. Outputs as accept_scan (without the escalation list), plus near_accept [B]: the
    number of children tested along the walk whose uniform number lies within near_accept_eps of
    the acceptance ratio (a decision that an implementation dividing in lower precision may
    take the other way; such sequences are counted, not compared)."""
    parent = np.asarray(parent)
    B, T = parent.shape
    res = {"accept_len": np.zeros(B, dtype=np.int32), "escalate": np.zeros(B, dtype=np.uint8),
           "bonus_tok": np.full(B, -1, dtype=np.int32), "path": np.full((B, T), -1, dtype=np.int32),
           "last_node": np.full(B, -1, dtype=np.int32), "near_thr": np.zeros(B, dtype=np.int32),
           "near_accept": np.zeros(B, dtype=np.int32)}
    for b in range(B):
        if active is not None and not active[b]:
            continue
        cur, n = 0, 0
        while True:
            if mode == MODE_PROXY:
                margin = float(p_top1[b, cur]) - float(p_top2[b, cur])
                if abs(margin - lam) < near_eps:
                    res["near_thr"][b] += 1
                if not (margin >= lam):
                    res["escalate"][b] = 1
                    break
            nxt = -1
            for c in range(cur + 1, T):
                if int(parent[b, c]) != cur:
                    continue
                qc = float(q_draft[b, c])
                ratio = min(1.0, float(p_draft[b, c]) / qc) if qc > 0.0 else 1.0
                if abs(float(u[b, c]) - ratio) < near_accept_eps:
                    res["near_accept"][b] += 1
                if float(u[b, c]) < ratio:
                    nxt = c
                    break
            if nxt < 0:
                res["bonus_tok"][b] = -2
                break
            res["path"][b, n] = nxt
            n += 1
            cur = nxt
        res["accept_len"][b] = n
        res["last_node"][b] = cur
    return res


# ----------------------------------------------------------------------------------------
# token-specific deferral rule (appendix "Baseline Implementation Details: SpecCascade")
# ----------------------------------------------------------------------------------------
def accept_scan_token_specific(p_top1: np.ndarray, p_top2: np.ndarray, top1_idx: np.ndarray,
                               p_draft: np.ndarray, parent: np.ndarray, tok: np.ndarray, lam: float,
                               alpha: float, mode: int = MODE_PROXY, active: Optional[np.ndarray] = None,
                               near_eps: float = 1e-3, near_accept_eps: float = 1e-6) -> Dict[str, np.ndarray]:
    """The walk of accept_scan with the token-specific deferral rule in place of the arg-max
    match: the rule compares the verifier's probability of the candidate token with the
    verifier's maximum probability and never looks at the drafter's distribution. A drafted
    child c of the current node is accepted iff
        p_draft[c] >= (1 - alpha) * p_top1[current node],
    p_draft[c] being the verifier's probability of tok[c] at c's parent (the paper runs the rule
    with alpha = 0.2). alpha = 0 accepts only a token as probable as the arg-max (greedy
    acceptance); alpha = 1 accepts any drafted token.
    Readings: on a tree the children of the current node are tried in node order and the first
    that passes is taken (as for duplicate siblings and for the stochastic rule); when none
    passes the round ends in case (i) with the verifier's arg-max token as the bonus token, as in
    greedy acceptance. In PROXY mode the margin test of Eq. 8 precedes the children as in
    accept_scan. The comparison is made in fp64; near_accept [B] counts the tested children with
    |p_draft - (1 - alpha) p_top1| < near_accept_eps. Outputs as accept_scan, without the
    escalation list."""
    parent = np.asarray(parent)
    B, T = parent.shape
    res = {"accept_len": np.zeros(B, dtype=np.int32), "escalate": np.zeros(B, dtype=np.uint8),
           "bonus_tok": np.full(B, -1, dtype=np.int32), "path": np.full((B, T), -1, dtype=np.int32),
           "last_node": np.full(B, -1, dtype=np.int32), "near_thr": np.zeros(B, dtype=np.int32),
           "near_accept": np.zeros(B, dtype=np.int32)}
    for b in range(B):
        if active is not None and not active[b]:
            continue
        cur, n = 0, 0
        while True:
            if mode == MODE_PROXY:
                margin = float(p_top1[b, cur]) - float(p_top2[b, cur])
                if abs(margin - lam) < near_eps:
                    res["near_thr"][b] += 1
                if not (margin >= lam):
                    res["escalate"][b] = 1
                    break
            bar = (1.0 - float(alpha)) * float(p_top1[b, cur])
            nxt = -1
            for c in range(cur + 1, T):
                if int(parent[b, c]) != cur:
                    continue
                if abs(float(p_draft[b, c]) - bar) < near_accept_eps:
                    res["near_accept"][b] += 1
                if float(p_draft[b, c]) >= bar:
                    nxt = c
                    break
            if nxt < 0:
                res["bonus_tok"][b] = int(top1_idx[b, cur])
                break
            res["path"][b, n] = nxt
            n += 1
            cur = nxt
        res["accept_len"][b] = n
        res["last_node"][b] = cur
    return res


_PHILOX_M0, _PHILOX_M1 = 0xD2511F53, 0xCD9E8D57
_PHILOX_W0, _PHILOX_W1 = 0x9E3779B9, 0xBB67AE85


def philox4x32_10(counter: Sequence[int], key: Sequence[int]) -> Tuple[int, int, int, int]:
    """Philox-4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy
    as 1, 2, 3", SC'11): a counter-based generator, 128-bit counter and 64-bit key -> four 32-bit
    words. Written from the published definition."""
    c0, c1, c2, c3 = (int(x) & 0xFFFFFFFF for x in counter)
    k0, k1 = (int(x) & 0xFFFFFFFF for x in key)
    for _ in range(10):
        p0 = _PHILOX_M0 * c0
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> 32, p0 & 0xFFFFFFFF
        hi1, lo1 = p1 >> 32, p1 & 0xFFFFFFFF
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & 0xFFFFFFFF, lo1, (hi0 ^ c3 ^ k1) & 0xFFFFFFFF, lo0
        k0 = (k0 + _PHILOX_W0) & 0xFFFFFFFF
        k1 = (k1 + _PHILOX_W1) & 0xFFFFFFFF
    return c0, c1, c2, c3


def gumbel_from_word(w: int) -> float:
    """Standard Gumbel variate from one 32-bit word of the generator: the word's upper 23 bits
    give u = ((w >> 9) + 0.5) / 2^23, a point strictly inside (0, 1) that a single-precision
    float holds exactly, and G = -ln(-ln u). Dropping the lower 9 bits bounds the variate:
    G lies in [-ln(-ln(2^-24)), -ln(-ln(1 - 2^-24))] = [-2.812, 16.636], so an entry more than
    19.45 below the largest logit can never be drawn (its probability is below 4e-9)."""
    uu = ((int(w) >> 9) + 0.5) / 8388608.0
    return float(-np.log(-np.log(uu)))


def gumbel_noise(seed: int, step: int, b: int, v: int) -> float:
    """Standard Gumbel variate of vocabulary entry v of sequence b in round `step`:
    word (v mod 4) of philox4x32_10(counter = (v div 4, b, step low, step high), key = seed),
    turned into a variate by gumbel_from_word."""
    w = philox4x32_10((v >> 2, b, step & 0xFFFFFFFF, (step >> 32) & 0xFFFFFFFF),
                      (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF))[v & 3]
    return gumbel_from_word(w)


def gumbel_noise_row(seed: int, step: int, b: int, V: int) -> np.ndarray:
    """gumbel_noise(seed, step, b, v) for v = 0..V-1, with the same rounds written on numpy
    arrays (checked against the scalar form in the tests)."""
    nblk = (V + 3) // 4
    m32 = np.uint64(0xFFFFFFFF)
    c0 = np.arange(nblk, dtype=np.uint64)
    c1 = np.full(nblk, b & 0xFFFFFFFF, dtype=np.uint64)
    c2 = np.full(nblk, step & 0xFFFFFFFF, dtype=np.uint64)
    c3 = np.full(nblk, (step >> 32) & 0xFFFFFFFF, dtype=np.uint64)
    k0, k1 = seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF
    for _ in range(10):
        p0 = np.uint64(_PHILOX_M0) * c0
        p1 = np.uint64(_PHILOX_M1) * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & m32
        hi1, lo1 = p1 >> np.uint64(32), p1 & m32
        c0, c1, c2, c3 = (hi1 ^ c1 ^ np.uint64(k0)) & m32, lo1, (hi0 ^ c3 ^ np.uint64(k1)) & m32, lo0
        k0 = (k0 + _PHILOX_W0) & 0xFFFFFFFF
        k1 = (k1 + _PHILOX_W1) & 0xFFFFFFFF
    words = (np.stack([c0, c1, c2, c3], axis=1).reshape(-1)[:V] >> np.uint64(9)).astype(np.float64)
    uu = (words + 0.5) / 8388608.0
    return -np.log(-np.log(uu))


def sample_bonus(h: np.ndarray, W: np.ndarray, logit_scale: float, node: np.ndarray, seed: int, step: int,
                 W64: Optional[np.ndarray] = None):
    """x_bonus ~ softmax(z) at row (b, node[b]) by the Gumbel-max identity: argmax_v (z_v + G_v)
    with independent standard Gumbel G_v is a sample of softmax(z). node[b] < 0 skips the
    sequence (-1 returned). Also returns the winning perturbed value and its margin over the
    runner-up (for the near-tie accounting of the parity tests). h is [B][T][d], W [V][d] bf16 bits."""
    B = h.shape[0]
    if W64 is None:
        W64 = bf16_to_f64(W)
    V = W64.shape[0]
    tok = np.full(B, -1, dtype=np.int64)
    best = np.full(B, np.nan)
    gap = np.full(B, np.nan)
    for b in range(B):
        if int(node[b]) < 0:
            continue
        z = row_logits(h[b, int(node[b])], W64, logit_scale)
        g = gumbel_noise_row(seed, step, b, V)
        y = z + g
        i1 = int(np.argmax(y))
        tok[b], best[b] = i1, y[i1]
        y2 = y.copy()
        y2[i1] = -np.inf
        gap[b] = y[i1] - y2.max()
    return tok, best, gap
