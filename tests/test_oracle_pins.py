"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU).

Each test compares the oracle with something other than itself: hand-derived fixtures,
closed forms, textbook routines written independently here, exact rational arithmetic, or
brute force on tiny inputs.
"""
import itertools
import json
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import trispec_oracle as orc
from paper_2601_23180_b200 import inputs as gen

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _load(name):
    with open(os.path.join(GOLD, name)) as f:
        return json.load(f)


def bf16(x):
    return gen.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


# ------------------------------------------------------------------------------- mask
def test_mask_golden():
    for case in _load("tree_mask_cases.json")["cases"]:
        parent = np.array([case["parent"]], dtype=np.int32)
        mask, depth = orc.build_tree_mask(parent)
        for i, vis in enumerate(case["visible"]):
            assert int(mask[0, i]) == sum(1 << j for j in vis)
        assert depth[0].tolist() == case["depth"]


def test_mask_transitive_closure_and_invariants():
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=6)
    parent = np.stack([gen.make_tree(cfg, b) for b in range(cfg.B)])
    mask, depth = orc.build_tree_mask(parent)
    for b in range(cfg.B):
        closure = [0] * cfg.T
        for i in range(cfg.T):                      # independent recursion
            closure[i] = (closure[parent[b, i]] if parent[b, i] >= 0 else 0) | (1 << i)
            assert int(mask[b, i]) == closure[i]
            assert bin(closure[i]).count("1") == depth[b, i] + 1
            assert closure[i] >> (i + 1) == 0       # never sees a later node
        assert depth[b].max() == cfg.max_depth


def test_mask_chain_is_lower_triangular_and_star():
    T = 9
    chain = np.arange(-1, T - 1, dtype=np.int32)[None]
    m, d = orc.build_tree_mask(chain)
    assert [int(x) for x in m[0]] == [(1 << (i + 1)) - 1 for i in range(T)]
    star = np.array([[-1] + [0] * (T - 1)], dtype=np.int32)
    m, d = orc.build_tree_mask(star)
    assert [int(x) for x in m[0]] == [1] + [1 | (1 << i) for i in range(1, T)]


# -------------------------------------------------------------------------- attention
def _attn_inputs(B=2, T=5, Hq=4, Hkv=2, D=16, L=11, seed=0, tree="chain"):
    g = np.random.default_rng(seed)
    q = bf16(g.standard_normal((B, T, Hq, D)))
    kt = bf16(g.standard_normal((B, T, Hkv, D)))
    vt = bf16(g.standard_normal((B, T, Hkv, D)))
    kc = bf16(g.standard_normal((B, L, Hkv, D)))
    vc = bf16(g.standard_normal((B, L, Hkv, D)))
    if tree == "chain":
        parent = np.tile(np.arange(-1, T - 1, dtype=np.int32), (B, 1))
    else:
        parent = np.stack([np.array([-1] + [int(g.integers(0, i)) for i in range(1, T)], dtype=np.int32)
                           for _ in range(B)])
    ctx = np.full(B, L, dtype=np.int32)
    return q, kt, vt, kc, vc, parent, ctx


def _dense_causal_attention(q64, k64, v64, scale):
    """Textbook causal attention of a full sequence: softmax(tril(Q K^T) * scale) V."""
    n = q64.shape[0]
    s = (q64 @ k64.T) * scale
    s = np.where(np.tril(np.ones((n, n), dtype=bool)), s, -np.inf)
    s = s - s.max(axis=1, keepdims=True)
    p = np.exp(s)
    p /= p.sum(axis=1, keepdims=True)
    return p @ v64


def test_attention_chain_equals_causal_attention():
    B, T, Hq, Hkv, D, L = 2, 5, 4, 2, 16, 11
    q, kt, vt, kc, vc, parent, ctx = _attn_inputs(B, T, Hq, Hkv, D, L)
    mask, _ = orc.build_tree_mask(parent)
    scale = 1.0 / math.sqrt(D)
    o, lse = orc.verify_attn(q, kt, vt, mask, kc, vc, ctx, scale)
    f = lambda x: gen.bf16_bits_to_f32(x).astype(np.float64)
    G = Hq // Hkv
    for b in range(B):
        for h in range(Hq):
            g = h // G
            K = np.concatenate([f(kc[b, :, g]), f(kt[b, :, g])])
            V = np.concatenate([f(vc[b, :, g]), f(vt[b, :, g])])
            # queries of the context rows are irrelevant: use zeros there, keep the last T rows
            Q = np.concatenate([np.zeros((L, D)), f(q[b, :, h])])
            ref = _dense_causal_attention(Q, K, V, scale)[L:]
            np.testing.assert_allclose(o[b, :, h], ref, rtol=1e-12, atol=1e-12)


def test_attention_weights_sum_to_one_and_mean_of_values():
    q, kt, vt, kc, vc, parent, ctx = _attn_inputs(tree="random", seed=3)
    mask, _ = orc.build_tree_mask(parent)
    B, T, Hq, D = q.shape
    # constant values: the output must be that constant (weights sum to one)
    vconst_t = np.broadcast_to(bf16(np.float32(1.5)), vt.shape)
    vconst_c = np.broadcast_to(bf16(np.float32(1.5)), vc.shape)
    o, _ = orc.verify_attn(q, kt, vconst_t, mask, kc, vconst_c, ctx, 0.25)
    np.testing.assert_allclose(o, 1.5, rtol=1e-13)
    # zero keys: uniform weights over the visible set -> mean of the visible values
    o, lse = orc.verify_attn(q, np.zeros_like(kt), vt, mask, np.zeros_like(kc), vc, ctx, 0.25)
    f = lambda x: gen.bf16_bits_to_f32(x).astype(np.float64)
    G = Hq // kt.shape[2]
    for b in range(B):
        for i in range(T):
            vis = [j for j in range(T) if (int(mask[b, i]) >> j) & 1]
            for h in range(Hq):
                vals = np.concatenate([f(vc[b, :, h // G]), f(vt[b, vis, h // G])])
                np.testing.assert_allclose(o[b, i, h], vals.mean(axis=0), rtol=1e-12, atol=1e-13)
                assert abs(lse[b, h, i] - math.log(len(vals))) < 1e-12


def test_attention_two_key_closed_form():
    # one context key with q.k = 1, the root's own key with q.k = 0, scale = ln 3:
    # weights 3/4 and 1/4 (Eq. 5 softmax; visible set = context + self)
    D = 8
    q = bf16(np.eye(1, D, 0)).reshape(1, 1, 1, D)
    kc = bf16(np.eye(1, D, 0)).reshape(1, 1, 1, D)
    kt = bf16(np.zeros((1, 1, 1, D)))
    vc = bf16(np.full((1, 1, 1, D), 4.0))
    vt = bf16(np.full((1, 1, 1, D), -4.0))
    mask, _ = orc.build_tree_mask(np.array([[-1]], dtype=np.int32))
    o, lse = orc.verify_attn(q, kt, vt, mask, kc, vc, np.array([1], dtype=np.int32), math.log(3.0))
    np.testing.assert_allclose(o[0, 0, 0], 0.75 * 4.0 + 0.25 * -4.0, rtol=1e-14)
    assert abs(lse[0, 0, 0] - math.log(4.0)) < 1e-14


def test_attention_paged_equals_contiguous_and_gqa_equals_mha():
    B, T, Hq, Hkv, D, L = 2, 6, 4, 2, 16, 37
    q, kt, vt, kc, vc, parent, _ = _attn_inputs(B, T, Hq, Hkv, D, L, seed=5, tree="random")
    ctx = np.array([37, 20], dtype=np.int32)
    mask, _ = orc.build_tree_mask(parent)
    o_ref, lse_ref = orc.verify_attn(q, kt, vt, mask, kc, vc, ctx, 0.3)
    # paged copy with 8-token blocks in shuffled order
    bs = 8
    nblk_seq = (L + bs - 1) // bs
    rng = np.random.default_rng(1)
    perm = rng.permutation(B * nblk_seq)
    table = perm.reshape(B, nblk_seq).astype(np.int32)
    pool_k = np.zeros((B * nblk_seq, bs, Hkv, D), dtype=np.uint16)
    pool_v = np.zeros_like(pool_k)
    for b in range(B):
        for t in range(L):
            pool_k[table[b, t // bs], t % bs] = kc[b, t]
            pool_v[table[b, t // bs], t % bs] = vc[b, t]
    o_p, lse_p = orc.verify_attn(q, kt, vt, mask, pool_k, pool_v, ctx, 0.3, block_table=table, block_size=bs)
    assert np.array_equal(o_p, o_ref) and np.array_equal(lse_p, lse_ref)
    # GQA == MHA with every KV head repeated G times
    G = Hq // Hkv
    rep = lambda x: np.repeat(x, G, axis=2)
    o_m, _ = orc.verify_attn(q, rep(kt), rep(vt), mask, rep(kc), rep(vc), ctx, 0.3)
    assert np.array_equal(o_m, o_ref)


def test_attention_empty_context_and_permutation_invariance():
    q, kt, vt, kc, vc, parent, ctx = _attn_inputs(B=1, T=4, L=9, seed=7, tree="random")
    mask, _ = orc.build_tree_mask(parent)
    # L = 0: tree-only attention; the root sees only itself -> o = v_tree[root]
    o, _ = orc.verify_attn(q, kt, vt, mask, kc, vc, np.zeros(1, dtype=np.int32), 0.2)
    f = lambda x: gen.bf16_bits_to_f32(x).astype(np.float64)
    G = q.shape[2] // kt.shape[2]
    for h in range(q.shape[2]):
        np.testing.assert_allclose(o[0, 0, h], f(vt[0, 0, h // G]), rtol=1e-15)
    # context keys are all visible, so their order cannot matter
    perm = np.random.default_rng(2).permutation(9)
    o1, _ = orc.verify_attn(q, kt, vt, mask, kc, vc, ctx, 0.2)
    o2, _ = orc.verify_attn(q, kt, vt, mask, kc[:, perm], vc[:, perm], ctx, 0.2)
    np.testing.assert_allclose(o1, o2, rtol=1e-12, atol=1e-13)
    # samples interface returns the same numbers
    o3, _ = orc.verify_attn(q, kt, vt, mask, kc, vc, ctx, 0.2, samples=[(0, 2, 1)])
    assert np.array_equal(o3[0, 2, 1], o1[0, 2, 1]) and np.isnan(o3[0, 0, 0]).all()


# ---------------------------------------------------------------------- LM-head stats
def _one_row_stats(h_bits, W_bits, scale, parent=None, tok=None):
    T = h_bits.shape[0]
    if parent is None:
        parent = np.arange(-1, T - 1, dtype=np.int32)
    if tok is None:
        tok = np.zeros(T, dtype=np.int32)
    return orc.lmhead_stats(h_bits[None], W_bits, parent[None], tok[None], scale)


def test_stats_closed_forms_golden():
    for case in _load("softmax_closed_forms.json")["cases"]:
        c = np.array(case["c"], dtype=np.float32)
        V, d = len(c), 4
        W = np.zeros((V, d), dtype=np.float32)
        W[:, 0] = c
        W[:, 1] = 7.0                      # must be ignored by the one-hot hidden state
        h = np.zeros((1, d), dtype=np.float32)
        h[0, 0] = 1.0
        st = _one_row_stats(bf16(h), bf16(W), math.log(case["base"]))
        frac = lambda nd: nd[0] / nd[1]
        assert abs(st["p_top1"][0, 0] - frac(case["p_top1"])) < 1e-14
        assert abs(st["p_top2"][0, 0] - frac(case["p_top2"])) < 1e-14
        assert abs((st["p_top1"][0, 0] - st["p_top2"][0, 0]) - frac(case["margin"])) < 1e-14
        assert st["top1_idx"][0, 0] == case["top1_idx"]
        assert st["top2_idx"][0, 0] == case["top2_idx"]
        assert abs(st["lse"][0, 0] - math.log(case["lse_exp"])) < 1e-14


def test_stats_against_exact_rational_logits_and_full_sort():
    g = np.random.default_rng(11)
    V, d, T = 13, 6, 4
    Wb, hb = bf16(g.standard_normal((V, d))), bf16(g.standard_normal((T, d)))
    parent = np.array([-1, 0, 0, 1], dtype=np.int32)
    tok = np.array([0, 5, 9, 2], dtype=np.int32)
    scale = 1.75
    st = _one_row_stats(hb, Wb, scale, parent, tok)
    Wf, hf = gen.bf16_bits_to_f32(Wb), gen.bf16_bits_to_f32(hb)
    for r in range(T):
        # exact logits by rational arithmetic (bf16 values are dyadic rationals)
        z = [float(Fraction(scale) * sum(Fraction(float(Wf[v, j])) * Fraction(float(hf[r, j]))
                                          for j in range(d))) for v in range(V)]
        m = max(z)
        lse = m + math.log(math.fsum(math.exp(x - m) for x in z))
        order = sorted(range(V), key=lambda v: (-z[v], v))     # full sort, ties -> low index
        assert st["top1_idx"][0, r] == order[0] and st["top2_idx"][0, r] == order[1]
        assert abs(st["max"][0, r] - m) < 1e-13
        assert abs(st["lse"][0, r] - lse) < 1e-13
        assert abs(st["p_top1"][0, r] - math.exp(z[order[0]] - lse)) < 1e-13
        assert abs(st["p_top2"][0, r] - math.exp(z[order[1]] - lse)) < 1e-13
        assert abs(st["top3_val"][0, r] - z[order[2]]) < 1e-13
        # probabilities over the vocabulary sum to one
        assert abs(math.fsum(math.exp(x - st["lse"][0, r]) for x in z) - 1.0) < 1e-12
    # drafted-token probability is read in the PARENT's row
    for c in range(1, T):
        r = parent[c]
        z = float(Fraction(scale) * sum(Fraction(float(Wf[tok[c], j])) * Fraction(float(hf[r, j]))
                                        for j in range(d)))
        assert abs(st["draft_logit"][0, c] - z) < 1e-13
        assert abs(st["p_draft"][0, c] - math.exp(z - st["lse"][0, r])) < 1e-13
    assert np.isnan(st["p_draft"][0, 0])


def test_stats_shift_invariance_and_ties():
    g = np.random.default_rng(12)
    V, d = 17, 5
    W, h = g.standard_normal((V, d)).astype(np.float32), g.standard_normal((1, d)).astype(np.float32)
    st0 = _one_row_stats(bf16(h), bf16(W), 2.0)
    # add a constant logit c*scale through an extra coordinate: p unchanged, lse shifted
    W1 = np.concatenate([W, np.full((V, 1), 3.0, dtype=np.float32)], axis=1)
    h1 = np.concatenate([h, np.ones((1, 1), dtype=np.float32)], axis=1)
    st1 = _one_row_stats(bf16(h1), bf16(W1), 2.0)
    assert abs(st1["lse"][0, 0] - st0["lse"][0, 0] - 6.0) < 1e-12
    assert abs(st1["p_top1"][0, 0] - st0["p_top1"][0, 0]) < 1e-13
    assert abs(st1["p_top2"][0, 0] - st0["p_top2"][0, 0]) < 1e-13
    assert st1["top1_idx"][0, 0] == st0["top1_idx"][0, 0]
    # duplicate the arg-max row at a LOWER and a HIGHER index: equal maxima -> margin 0,
    # top-1 is the lowest index, top-2 the next one
    i1 = int(st0["top1_idx"][0, 0])
    W2 = np.concatenate([W[i1:i1 + 1], W, W[i1:i1 + 1]])
    st2 = _one_row_stats(bf16(h), bf16(W2), 2.0)
    assert st2["top1_idx"][0, 0] == 0 and st2["top2_idx"][0, 0] == i1 + 1
    assert st2["p_top1"][0, 0] == st2["p_top2"][0, 0]


def test_stats_generator_straddles_threshold():
    """The synthetic hidden-state recipe must produce both trusted and untrusted positions
    at lambda = 0.5 with the configured logit scale (otherwise the scan is never exercised)."""
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=1, V=4096)
    inp = gen.make_inputs(cfg, with_attention=False)
    st = orc.lmhead_stats(inp["h"], inp["W"], inp["parent"], inp["tok"], cfg.logit_scale)
    margin = st["p_top1"][0] - st["p_top2"][0]
    conf = inp["alpha"][0] == 8.0
    assert (margin[conf] >= 0.5).mean() > 0.9
    assert (margin[~conf] >= 0.5).mean() < 0.1
    assert (st["top1_idx"][0][conf] == inp["favoured_tok"][0][conf]).all()


# ------------------------------------------------------------------------ accept scan
def _chain_case_arrays(k, s, g, V=50):
    """Chain tree whose stats realise the given acceptance bits s and margin bits g."""
    T = k + 1
    parent = np.arange(-1, T - 1, dtype=np.int32)[None]
    tok = (np.arange(T, dtype=np.int32) + 10)[None]
    top1 = np.zeros((1, T), dtype=np.int64)
    for i in range(k):
        top1[0, i] = tok[0, i + 1] if s[i] else 5      # token 5 is never drafted
    top1[0, k] = 7
    p1 = np.where(np.array(g) == 1, 0.9, 0.5)[None]
    p2 = np.where(np.array(g) == 1, 0.05, 0.3)[None]
    return parent, tok, top1, p1, p2


def test_scan_golden_chain_cases():
    for case in _load("scan_chain_cases.json")["cases"]:
        k, s, g = case["k"], case["s"], case["g"]
        # the fixture's tau_a / tau_m follow Eq. 7 / Eq. 9 literally (checked here too)
        tau_a = min([i for i in range(k) if s[i] == 0] + [k])
        tau_m = min([i for i in range(k + 1) if g[i] == 0] + [k + 1])
        assert (tau_a, tau_m) == (case["tau_a"], case["tau_m"])
        parent, tok, top1, p1, p2 = _chain_case_arrays(k, s, g)
        r = orc.accept_scan(p1, p2, top1, parent, tok, lam=0.5)
        assert r["escalate"][0] == case["escalate"]
        assert r["accept_len"][0] == case["n_accepted"]
        assert r["path"][0, :case["n_accepted"]].tolist() == list(range(1, case["n_accepted"] + 1))
        assert (r["path"][0, case["n_accepted"]:] == -1).all()
        if case["bonus_pos"] is None:
            assert r["bonus_tok"][0] == -1
        else:
            assert r["bonus_tok"][0] == top1[0, case["bonus_pos"] - 1]
        assert r["last_node"][0] == case["n_accepted"]


def _brute_force_tree(parent, tok, top1, margin, lam, target_mode=False):
    """Every root-to-leaf path evaluated with the chain formulas (Eq. 6-9 and the routing
    rule); the tree result is the best path. Independent of the oracle's walk."""
    T = len(parent)
    leaves = [i for i in range(T) if not any(parent[c] == i for c in range(T))]
    best = None
    for leaf in leaves:
        path = []
        p = leaf
        while p >= 0:
            path.append(p)
            p = parent[p]
        path.reverse()
        k = len(path) - 1
        s = [1 if tok[path[i + 1]] == top1[path[i]] else 0 for i in range(k)]
        g = [1 if (target_mode or margin[path[i]] >= lam) else 0 for i in range(k + 1)]
        tau_a = min([i for i in range(k) if s[i] == 0] + [k])
        tau_m = min([i for i in range(k + 1) if g[i] == 0] + [k + 1])
        if tau_a < tau_m:
            res = (tau_a, 0, int(top1[path[tau_a]]), tuple(path[1:tau_a + 1]))
        else:
            res = (tau_m, 1, -1, tuple(path[1:tau_m + 1]))
        if best is None or res[0] > best[0]:
            best = res
        elif res[0] == best[0]:
            assert res == best, "maximising paths disagree"
    return best


@pytest.mark.parametrize("seed", range(40))
def test_scan_equals_brute_force_over_paths(seed):
    g = np.random.default_rng(seed)
    T = int(g.integers(1, 11))
    V = int(g.integers(3, 17))
    parent = np.array([-1] + [int(g.integers(0, i)) for i in range(1, T)], dtype=np.int32)
    tok = np.zeros(T, dtype=np.int32)
    for p in range(T):                                   # distinct sibling tokens
        kids = [c for c in range(T) if parent[c] == p]
        tok[kids] = g.permutation(V)[:len(kids)] if len(kids) <= V else g.integers(0, V, len(kids))
    tok[0] = int(g.integers(0, V))
    top1 = np.zeros(T, dtype=np.int64)
    for r in range(T):
        kids = [c for c in range(T) if parent[c] == r]
        top1[r] = tok[kids[int(g.integers(len(kids)))]] if kids and g.random() < 0.7 else int(g.integers(0, V))
    p1 = g.uniform(0.3, 1.0, T)
    p2 = p1 * g.uniform(0.0, 0.6, T)
    for lam, mode in ((0.5, orc.MODE_PROXY), (0.2, orc.MODE_PROXY), (0.5, orc.MODE_TARGET)):
        r = orc.accept_scan(p1[None], p2[None], top1[None], parent[None], tok[None], lam, mode=mode)
        n, esc, bonus, path = _brute_force_tree(parent.tolist(), tok.tolist(), top1.tolist(),
                                                (p1 - p2).tolist(), lam, mode == orc.MODE_TARGET)
        assert r["accept_len"][0] == n and r["escalate"][0] == esc and r["bonus_tok"][0] == bonus
        assert tuple(r["path"][0, :n].tolist()) == path
        assert r["last_node"][0] == (path[-1] if n else 0)


def test_scan_lambda_limits_and_target_mode():
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=12, V=512, rho=0.3)
    inp = gen.make_inputs(cfg, with_attention=False)
    st = orc.lmhead_stats(inp["h"], inp["W"], inp["parent"], inp["tok"], cfg.logit_scale)
    args = (st["p_top1"], st["p_top2"], st["top1_idx"], inp["parent"], inp["tok"])
    never = orc.accept_scan(*args, lam=0.0)                       # g == 1 everywhere
    target = orc.accept_scan(*args, lam=0.5, mode=orc.MODE_TARGET)
    minus_inf = orc.accept_scan(*args, lam=-np.inf)
    for key in ("accept_len", "escalate", "bonus_tok", "path", "last_node"):
        assert np.array_equal(never[key], target[key]) and np.array_equal(minus_inf[key], target[key])
    assert never["escalate"].sum() == 0 and (never["bonus_tok"] >= 0).all()
    always = orc.accept_scan(*args, lam=1.0 + 1e-9)               # g == 0 everywhere
    assert always["escalate"].all() and (always["accept_len"] == 0).all()
    assert (always["bonus_tok"] == -1).all() and always["n_escalated"] == cfg.B
    assert always["esc_index"].tolist() == list(range(cfg.B))
    proxy = orc.accept_scan(*args, lam=0.5)
    _, depth = orc.build_tree_mask(inp["parent"])
    assert (proxy["accept_len"] <= depth.max(axis=1)).all()
    assert (proxy["bonus_tok"][proxy["escalate"] == 1] == -1).all()
    assert (proxy["accept_len"] <= target["accept_len"]).all()    # the margin test only stops earlier
    # both outcomes occur with the synthetic mixture, and rho > 0 produces mid-path approvals
    assert 0 < proxy["escalate"].sum() < cfg.B
    # inactive sequences are left untouched
    active = np.zeros(cfg.B, dtype=np.uint8)
    active[[1, 4]] = 1
    part = orc.accept_scan(*args, lam=0.5, active=active)
    for b in range(cfg.B):
        if active[b]:
            assert part["accept_len"][b] == proxy["accept_len"][b] and part["escalate"][b] == proxy["escalate"][b]
        else:
            assert part["accept_len"][b] == 0 and part["escalate"][b] == 0 and part["last_node"][b] == -1


def test_scan_all_confident_all_match_chain_emits_k_plus_one_tokens():
    # if g = 1 everywhere then tau_m = k + 1 and the proxy produces the (k+1)-th token (Eq. 9)
    k = 8
    parent, tok, top1, p1, p2 = _chain_case_arrays(k, [1] * k, [1] * (k + 1))
    r = orc.accept_scan(p1, p2, top1, parent, tok, lam=0.5)
    assert r["accept_len"][0] == k and r["escalate"][0] == 0 and r["bonus_tok"][0] == 7
    # near-threshold positions are counted
    p1b = p1.copy()
    p1b[0, 3] = p2[0, 3] + 0.5 + 5e-4
    r = orc.accept_scan(p1b, p2, top1, parent, tok, lam=0.5)
    assert r["near_thr"][0] == 1 and r["accept_len"][0] == k


def test_scan_start_node():
    # TARGET-mode re-verification may resume from the proxy's last accepted node
    parent = np.array([[-1, 0, 0, 1, 1, 3]], dtype=np.int32)
    tok = np.array([[0, 11, 12, 13, 14, 15]], dtype=np.int32)
    top1 = np.array([[11, 13, 0, 15, 0, 99]], dtype=np.int64)
    p = np.full((1, 6), 0.5)
    full = orc.accept_scan(p, p, top1, parent, tok, 0.5, mode=orc.MODE_TARGET)
    assert full["path"][0, :3].tolist() == [1, 3, 5] and full["bonus_tok"][0] == 99
    part = orc.accept_scan(p, p, top1, parent, tok, 0.5, mode=orc.MODE_TARGET,
                           start_node=np.array([1], dtype=np.int32))
    assert part["accept_len"][0] == 2 and part["path"][0, :2].tolist() == [3, 5]


# ------------------------------------------------------------------------- whole pass
def test_verify_end_to_end_small():
    cfg = gen.small_variant(gen.CONFIGS["target_escalated"], B=4, n_active=2, L=96, V=1024, d=64,
                            Hq=8, Hkv=2, logit_scale=3.6 / (0.02 * 8.0))
    inp = gen.make_inputs(cfg)
    out = orc.verify(inp, 1.0 / math.sqrt(cfg.D), cfg.logit_scale, cfg.lam, mode=cfg.mode)
    act = set(int(s) for s in inp["seq_index"])
    for b in range(cfg.B):
        if b in act:
            assert np.isfinite(out["o"][b]).all() and out["scan"]["last_node"][b] >= 0
        else:
            assert np.isnan(out["o"][b]).all() and out["scan"]["last_node"][b] == -1
    assert out["scan"]["escalate"].sum() == 0     # TARGET mode never escalates


def test_verify_hands_the_four_steps_the_right_arrays():
    """The whole-pass function against its four steps called by hand on a batch where only a
    subset of the sequences is verified (seq_index): the subset must reach the attention and the
    LM head as `seqs`, the scan as the `active` flags, and the scan must read the statistics the
    LM head produced; a sequence outside the subset yields NaN / -1 everywhere."""
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=5, n_active=3, k=12, max_depth=4, L=70, V=300, d=64,
                            Hq=4, Hkv=2, rho=0.3, logit_scale=3.6 / (0.02 * 8.0), seed=21)
    inp = gen.make_inputs(cfg)
    seqs = [int(s) for s in inp["seq_index"]]
    assert 0 < len(seqs) < cfg.B
    scale = 1.0 / math.sqrt(cfg.D)
    out = orc.verify(inp, scale, cfg.logit_scale, cfg.lam, mode=orc.MODE_PROXY)
    mask, depth = orc.build_tree_mask(inp["parent"])
    assert np.array_equal(out["mask"], mask) and np.array_equal(out["depth"], depth)
    o, lse = orc.verify_attn(inp["q"], inp["k_tree"], inp["v_tree"], mask, inp["k_cache"], inp["v_cache"],
                             inp["ctx_len"], scale, seqs=seqs)
    assert np.array_equal(out["o"], o, equal_nan=True) and np.array_equal(out["attn_lse"], lse, equal_nan=True)
    st = orc.lmhead_stats(inp["h"], inp["W"], inp["parent"], inp["tok"], cfg.logit_scale, seqs=seqs)
    for k in st:
        assert np.array_equal(out["stats"][k], st[k], equal_nan=True), k
    active = np.zeros(cfg.B, dtype=np.uint8)
    active[seqs] = 1
    sc = orc.accept_scan(st["p_top1"], st["p_top2"], st["top1_idx"], inp["parent"], inp["tok"], cfg.lam,
                         mode=orc.MODE_PROXY, active=active)
    for k in sc:
        assert np.array_equal(out["scan"][k], sc[k]), k
    # the subset matters: a verified sequence has finite outputs and a walk, the others have neither
    for b in range(cfg.B):
        if b in seqs:
            assert np.isfinite(out["o"][b]).all() and np.isfinite(out["stats"]["lse"][b]).all()
            assert out["scan"]["last_node"][b] >= 0
        else:
            assert np.isnan(out["o"][b]).all() and np.isnan(out["stats"]["lse"][b]).all()
            assert out["scan"]["last_node"][b] == -1 and out["scan"]["accept_len"][b] == 0
    # and the outcome is not degenerate: both routing cases occur, something is accepted
    assert out["scan"]["escalate"][seqs].sum() + (out["scan"]["bonus_tok"][seqs] >= 0).sum() == len(seqs)
    # TARGET mode of the same call never escalates and accepts at least as much on every sequence
    tgt = orc.verify(inp, scale, cfg.logit_scale, cfg.lam, mode=orc.MODE_TARGET, with_attention=False)
    assert "o" not in tgt and tgt["scan"]["escalate"].sum() == 0
    assert (tgt["scan"]["accept_len"][seqs] >= out["scan"]["accept_len"][seqs]).all()
