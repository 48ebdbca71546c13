"""Pins of the oracle's token pruning and KV commit (CPU only): hand-derived cases, special
cases that reduce to the identity or to a plain slice, invariants that tie them to the tree mask
and to the attention oracle, and brute force on small random trees."""
import itertools
import math

import numpy as np
import pytest

from oracle import trispec_oracle as orc
from paper_2601_23180_b200 import inputs as gen


def _cfg(**kw):
    return gen.small_variant(gen.CONFIGS["proxy_tree"], **kw)


# ------------------------------------------------------------------------------ pruning
def test_prune_hand_case():
    # routing case (ii): the subtree below the last accepted node remains. Tree (node: parent)
    # 0:-1 1:0 2:0 3:1 4:1 5:2 6:3 ; accepted up to node 1 -> nodes {1,3,4,6} remain, relabelled 0..3
    parent = np.array([[-1, 0, 0, 1, 1, 2, 3]], dtype=np.int32)
    tok = np.array([[10, 11, 12, 13, 14, 15, 16]], dtype=np.int32)
    r = orc.prune_tree(parent, tok, np.array([1]))
    assert r["n_keep"][0] == 4
    assert r["node_map"][0].tolist() == [1, 3, 4, 6, -1, -1, -1]
    assert r["parent"][0].tolist() == [-1, 0, 0, 1, -1, -1, -1]
    assert r["tok"][0].tolist() == [11, 13, 14, 16, -1, -1, -1]


def test_prune_at_root_is_identity_at_leaf_is_single_node_and_skip():
    cfg = _cfg(B=3)
    parent = np.stack([gen.make_tree(cfg, b) for b in range(3)])
    tok = np.stack([gen.make_tokens(cfg, b, parent[b]) for b in range(3)])
    T = cfg.T
    leaf = max(i for i in range(T) if not (parent[1] == i).any())
    r = orc.prune_tree(parent, tok, np.array([0, leaf, -1]))
    assert r["n_keep"].tolist() == [T, 1, 0]
    assert np.array_equal(r["parent"][0], parent[0]) and np.array_equal(r["tok"][0], tok[0])
    assert np.array_equal(r["node_map"][0], np.arange(T))
    assert r["node_map"][1, 0] == leaf and r["parent"][1, 0] == -1 and (r["node_map"][1, 1:] == -1).all()
    assert (r["node_map"][2] == -1).all() and (r["parent"][2] == -1).all()


def test_prune_chain_is_a_suffix():
    T = 9
    parent = np.arange(-1, T - 1, dtype=np.int32)[None]
    tok = np.arange(100, 100 + T, dtype=np.int32)[None]
    for j in range(T):
        r = orc.prune_tree(parent, tok, np.array([j]))
        n = T - j
        assert r["n_keep"][0] == n
        assert r["tok"][0, :n].tolist() == list(range(100 + j, 100 + T))
        assert r["parent"][0, :n].tolist() == list(range(-1, n - 1))


@pytest.mark.parametrize("seed", range(6))
def test_prune_agrees_with_tree_mask_and_subtree_counts(seed):
    """Independent route: membership through the mask bits (bit r of mask[i]), sizes through a
    bottom-up child count; the pruned tree's own mask is the old mask with the kept bits packed."""
    cfg = _cfg(B=4, seed=seed)
    parent = np.stack([gen.make_tree(cfg, b) for b in range(4)])
    tok = np.stack([gen.make_tokens(cfg, b, parent[b]) for b in range(4)])
    T = cfg.T
    mask, depth = orc.build_tree_mask(parent)
    g = np.random.default_rng(seed)
    root = g.integers(0, T, size=4)
    r = orc.prune_tree(parent, tok, root)
    for b in range(4):
        size = np.ones(T, dtype=int)
        for i in range(T - 1, 0, -1):
            size[parent[b, i]] += size[i]
        keep = [i for i in range(T) if (int(mask[b, i]) >> int(root[b])) & 1]
        assert r["n_keep"][b] == size[root[b]] == len(keep)
        assert r["node_map"][b, :len(keep)].tolist() == keep
        # valid tree: parents precede children, one root
        pp = r["parent"][b, :len(keep)]
        assert pp[0] == -1 and all(0 <= pp[j] < j for j in range(1, len(keep)))
        # mask of the pruned tree = packed bits of the old mask restricted to kept nodes
        new_mask, new_depth = orc.build_tree_mask(pp[None])
        for j, i in enumerate(keep):
            packed = 0
            for jj, ii in enumerate(keep):
                if (int(mask[b, i]) >> ii) & 1:
                    packed |= 1 << jj
            assert int(new_mask[0, j]) == packed
            assert new_depth[0, j] == depth[b, i] - depth[b, root[b]]


def test_prune_then_target_scan_continues_the_proxy_walk():
    """A TARGET-mode scan of the pruned tree from its node 0 accepts exactly what a TARGET-mode
    scan of the unpruned tree accepts from start_node = last accepted node (the w/ and w/o token
    pruning variants verify the same remaining tokens)."""
    cfg = _cfg(B=6, seed=3)
    parent = np.stack([gen.make_tree(cfg, b) for b in range(6)])
    tok = np.stack([gen.make_tokens(cfg, b, parent[b]) for b in range(6)])
    T = cfg.T
    g = np.random.default_rng(5)
    root = g.integers(0, T // 3, size=6).astype(np.int32)
    # target top-1: first child's token on most nodes, so that walks go on
    top1 = g.integers(0, cfg.V, size=(6, T))
    for b in range(6):
        for i in range(T):
            kids = np.nonzero(parent[b] == i)[0]
            if len(kids) and g.random() < 0.8:
                top1[b, i] = tok[b, kids[0]]
    full = orc.accept_scan(np.ones((6, T)), np.zeros((6, T)), top1, parent, tok, 0.5, mode=orc.MODE_TARGET,
                           start_node=root)
    pr = orc.prune_tree(parent, tok, root)
    top1_p = np.zeros((6, T), dtype=np.int64)
    for b in range(6):
        n = pr["n_keep"][b]
        top1_p[b, :n] = top1[b, pr["node_map"][b, :n]]
    pruned = orc.accept_scan(np.ones((6, T)), np.zeros((6, T)), top1_p, pr["parent"], pr["tok"], 0.5,
                             mode=orc.MODE_TARGET)
    for b in range(6):
        n = full["accept_len"][b]
        assert pruned["accept_len"][b] == n and pruned["bonus_tok"][b] == full["bonus_tok"][b]
        assert [pr["node_map"][b, j] for j in pruned["path"][b, :n]] == full["path"][b, :n].tolist()


# ------------------------------------------------------------------------------ KV commit
def _kv_case(paged: bool, B=3, L=100, seed=0):
    name = "long_paged" if paged else "proxy_tree"
    cfg = gen.small_variant(gen.CONFIGS[name], B=B, L=L + 64, L_min=(L + 64) if paged else None, Hq=4, Hkv=2, seed=seed)
    inp = gen.make_inputs(cfg, with_lm_head=False)
    inp["ctx_len"] = np.array([L, L - 37, 5][:B], dtype=np.int32)
    return cfg, inp


@pytest.mark.parametrize("paged", [False, True])
def test_commit_appends_root_and_path_rows_and_touches_nothing_else(paged):
    cfg, inp = _kv_case(paged)
    B, T = cfg.B, cfg.T
    path = np.full((B, T), -1, dtype=np.int32)
    path[0, :3] = [2, 7, 19]
    path[1, :1] = [1]
    acc = np.array([3, 1, 0], dtype=np.int32)
    kc, vc, nl = orc.commit_kv(inp["k_cache"], inp["v_cache"], inp["ctx_len"], inp["k_tree"], inp["v_tree"], path,
                               acc, block_table=inp.get("block_table"), block_size=cfg.block_size)
    assert nl.tolist() == [int(inp["ctx_len"][b]) + int(acc[b]) + 1 for b in range(B)]

    def row(cache, b, t):
        if not paged:
            return cache[b, t]
        return cache[inp["block_table"][b, t // cfg.block_size], t % cfg.block_size]
    changed = np.zeros(kc.shape[:2], dtype=bool)
    for b in range(B):
        L = int(inp["ctx_len"][b])
        nodes = [0] + path[b, :acc[b]].tolist()
        for j, node in enumerate(nodes):
            assert np.array_equal(row(kc, b, L + j), inp["k_tree"][b, node])
            assert np.array_equal(row(vc, b, L + j), inp["v_tree"][b, node])
            if paged:
                changed[inp["block_table"][b, (L + j) // cfg.block_size], (L + j) % cfg.block_size] = True
            else:
                changed[b, L + j] = True
    assert np.array_equal(kc[~changed], inp["k_cache"][~changed])
    assert np.array_equal(vc[~changed], inp["v_cache"][~changed])


def test_commit_paged_equals_contiguous_through_attention():
    """After a commit, attention of a fresh one-node tree over the longer context must equal
    attention over [old context + committed rows] assembled by hand (ties commit_kv to verify_attn)."""
    cfg, inp = _kv_case(False, B=2, L=70, seed=2)
    B, T = cfg.B, cfg.T
    inp["ctx_len"] = np.array([70, 33], dtype=np.int32)
    path = np.full((B, T), -1, dtype=np.int32)
    path[0, :2] = [1, 5]
    acc = np.array([2, 0], dtype=np.int32)
    kc, vc, nl = orc.commit_kv(inp["k_cache"], inp["v_cache"], inp["ctx_len"], inp["k_tree"], inp["v_tree"], path, acc)
    # by hand: concatenate
    for b in range(B):
        L = int(inp["ctx_len"][b])
        nodes = [0] + path[b, :acc[b]].tolist()
        hand_k = np.concatenate([inp["k_cache"][b, :L], inp["k_tree"][b, nodes]], axis=0)
        hand_v = np.concatenate([inp["v_cache"][b, :L], inp["v_tree"][b, nodes]], axis=0)
        assert np.array_equal(kc[b, :nl[b]], hand_k) and np.array_equal(vc[b, :nl[b]], hand_v)
    q1 = inp["q"][:, :1]
    kt1, vt1 = inp["k_tree"][:, :1], inp["v_tree"][:, :1]
    m1 = np.ones((B, 1), dtype=np.uint64)
    o_new, _ = orc.verify_attn(q1, kt1, vt1, m1, kc, vc, nl, 0.1)
    # the same keys presented as [context | tree chain]: a chain tree whose last node is the query
    for b in range(B):
        n = int(acc[b]) + 1
        nodes = [0] + path[b, :acc[b]].tolist()
        ktc = np.concatenate([inp["k_tree"][b, nodes], kt1[b]], axis=0)[None]
        vtc = np.concatenate([inp["v_tree"][b, nodes], vt1[b]], axis=0)[None]
        qc = np.concatenate([inp["q"][b, nodes], q1[b]], axis=0)[None]
        chain_parent = np.arange(-1, n, dtype=np.int32)[None]
        mc, _ = orc.build_tree_mask(chain_parent)
        o_chain, _ = orc.verify_attn(qc, ktc, vtc, mc, inp["k_cache"][b:b + 1], inp["v_cache"][b:b + 1],
                                     inp["ctx_len"][b:b + 1], 0.1)
        assert np.allclose(o_new[b, 0], o_chain[0, n], rtol=0, atol=1e-12)


def test_commit_respects_capacity_and_active():
    cfg, inp = _kv_case(False, B=3, L=100)
    B, T = cfg.B, cfg.T
    Lcap = inp["k_cache"].shape[1]
    inp["ctx_len"] = np.array([Lcap - 1, Lcap - 2, 10], dtype=np.int32)
    path = np.full((B, T), -1, dtype=np.int32)
    path[:, 0] = 1
    acc = np.array([1, 1, 1], dtype=np.int32)          # needs 2 rows each
    kc, vc, nl = orc.commit_kv(inp["k_cache"], inp["v_cache"], inp["ctx_len"], inp["k_tree"], inp["v_tree"], path,
                               acc, active=np.array([1, 1, 0], dtype=np.uint8))
    assert nl.tolist() == [Lcap - 1, Lcap, 10]          # 0: no room, 1: fits exactly, 2: inactive
    assert np.array_equal(kc[0], inp["k_cache"][0]) and np.array_equal(kc[2], inp["k_cache"][2])


# ------------------------------------------------------------------------------ entropy, routing criteria
def _stats_from_logits(z):
    """Runs lmhead_stats on a [rows][V] logit table by making W the identity-like basis: h = one-hot
    rows are not needed - instead build h, W with W = I (V x V) and h = the logits (bf16-exact values)."""
    rows, V = z.shape
    d = ((V + 63) // 64) * 64
    W = np.zeros((V, d), dtype=np.float32)
    W[np.arange(V), np.arange(V)] = 1.0
    h = np.zeros((1, rows, d), dtype=np.float32)
    h[0, :, :V] = z
    to_bits = lambda x: (x.view(np.uint32) >> 16).astype(np.uint16)
    parent = np.arange(-1, rows - 1, dtype=np.int32)[None]
    tok = np.zeros((1, rows), dtype=np.int32)
    return orc.lmhead_stats(to_bits(h), to_bits(W), parent, tok, 1.0)


def test_entropy_closed_forms():
    import math
    V = 8
    z = np.zeros((4, V), dtype=np.float32)
    z[1, 0] = 64.0                      # one-hot in the limit: H -> 0
    z[2, :2] = 1.0                      # two maxima and six entries lower by 1
    z[3, 0] = 2.0                       # logits {2, 0 x 7}: p1 = e^2 / (e^2 + 7)
    st = _stats_from_logits(z)
    assert abs(st["entropy"][0, 0] - math.log(V)) < 1e-12              # uniform: ln V
    assert 0 <= st["entropy"][0, 1] < 1e-20
    a = 2 * math.e / (2 * math.e + 6)
    h2 = -(a * math.log(a / 2) + (1 - a) * math.log((1 - a) / 6))
    assert abs(st["entropy"][0, 2] - h2) < 1e-12
    p1 = math.exp(2) / (math.exp(2) + 7)
    h3 = -(p1 * math.log(p1) + (1 - p1) * math.log((1 - p1) / 7))
    assert abs(st["entropy"][0, 3] - h3) < 1e-12
    assert (st["entropy"][0] <= math.log(V) + 1e-12).all()
    # H = lse - E_p[z]
    for r in range(4):
        p = np.exp(z[r].astype(np.float64) - st["lse"][0, r])
        assert abs(st["entropy"][0, r] - (st["lse"][0, r] - (p * z[r]).sum())) < 1e-12


@pytest.mark.parametrize("crit", [orc.CRIT_TOP1, orc.CRIT_ENTROPY])
def test_scan_criteria_reduce_to_known_cases(crit):
    cfg = _cfg(B=5, seed=9)
    B, T = 5, cfg.T
    parent = np.stack([gen.make_tree(cfg, b) for b in range(B)])
    tok = np.stack([gen.make_tokens(cfg, b, parent[b]) for b in range(B)])
    g = np.random.default_rng(1)
    top1 = g.integers(0, cfg.V, size=(B, T))
    for b in range(B):
        for i in range(T):
            kids = np.nonzero(parent[b] == i)[0]
            if len(kids) and g.random() < 0.8:
                top1[b, i] = tok[b, kids[0]]
    p1 = g.uniform(0.2, 1.0, size=(B, T))
    p2 = g.uniform(0.0, 0.2, size=(B, T))
    ent = g.uniform(0.0, 3.0, size=(B, T))
    kw = dict(criterion=crit, entropy=ent)
    target = orc.accept_scan(p1, p2, top1, parent, tok, 0.5, mode=orc.MODE_TARGET)
    # a threshold nothing fails -> never escalates and equals plain greedy acceptance
    always = orc.accept_scan(p1, p2, top1, parent, tok, -1.0 if crit == orc.CRIT_TOP1 else 10.0, **kw)
    assert not always["escalate"].any()
    for k in ("accept_len", "bonus_tok", "path"):
        assert np.array_equal(always[k], target[k])
    # a threshold everything fails -> escalates at the root with nothing accepted
    never = orc.accept_scan(p1, p2, top1, parent, tok, 2.0 if crit == orc.CRIT_TOP1 else -1.0, **kw)
    assert never["escalate"].all() and (never["accept_len"] == 0).all() and (never["bonus_tok"] == -1).all()
    # general threshold: the walk stops at the first visited node whose feature fails
    lam = 0.6 if crit == orc.CRIT_TOP1 else 1.5
    r = orc.accept_scan(p1, p2, top1, parent, tok, lam, **kw)
    for b in range(B):
        nodes = [0] + target["path"][b, :target["accept_len"][b]].tolist()
        ok = [(p1[b, n] >= lam) if crit == orc.CRIT_TOP1 else (ent[b, n] <= lam) for n in nodes]
        if all(ok):
            assert r["escalate"][b] == 0 and r["accept_len"][b] == target["accept_len"][b]
        else:
            j = ok.index(False)
            assert r["escalate"][b] == 1 and r["accept_len"][b] == j and r["last_node"][b] == nodes[j]
    # top-1 criterion with p2 = 0 is the margin criterion
    if crit == orc.CRIT_TOP1:
        m = orc.accept_scan(p1, np.zeros_like(p2), top1, parent, tok, lam)
        for k in ("accept_len", "escalate", "bonus_tok", "path"):
            assert np.array_equal(m[k], r[k])


# ------------------------------------------------------------------------------ stochastic acceptance, sampling
def test_philox_known_answers_and_vector_form():
    # known-answer vectors of Philox-4x32-10 (Random123 distribution, kat_vectors)
    kat = [((0, 0, 0, 0), (0, 0), "6627e8d5 e169c58d bc57ac4c 9b00dbd8"),
           ((0xffffffff,) * 4, (0xffffffff,) * 2, "408f276d 41c83b0e a20bc7c6 6d5451fd"),
           ((0x243f6a88, 0x85a308d3, 0x13198a2e, 0x03707344), (0xa4093822, 0x299f31d0),
            "d16cfe09 94fdcceb 5001e420 24126ea1")]
    for c, k, want in kat:
        assert " ".join("%08x" % x for x in orc.philox4x32_10(c, k)) == want
    row = orc.gumbel_noise_row(0x1234567890abcdef, 5, 3, 37)
    for v in (0, 1, 2, 3, 4, 17, 36):
        assert row[v] == orc.gumbel_noise(0x1234567890abcdef, 5, 3, v)
    assert np.isfinite(row).all()


def test_gumbel_max_samples_the_softmax():
    """Over many rounds the sampled tokens follow softmax(z) (Gumbel-max identity): 5 tokens,
    20000 draws, every frequency within 4 standard deviations."""
    z = np.array([1.0, 0.0, -1.0, 2.0, 0.5])
    p = np.exp(z) / np.exp(z).sum()
    n = 20000
    counts = np.zeros(5)
    for step in range(n // 8):
        for b in range(8):
            counts[np.argmax(z + orc.gumbel_noise_row(99, step, b, 5))] += 1
    assert np.all(np.abs(counts / n - p) < 4 * np.sqrt(p * (1 - p) / n))


def test_stochastic_scan_special_cases_and_acceptance_probability():
    cfg = _cfg(B=4, seed=12)
    B, T = 4, cfg.T
    parent = np.stack([gen.make_tree(cfg, b) for b in range(B)])
    tok = np.stack([gen.make_tokens(cfg, b, parent[b]) for b in range(B)])
    g = np.random.default_rng(3)
    p1, p2 = np.ones((B, T)), np.zeros((B, T))                       # always trusted
    pd = g.uniform(0.05, 0.9, size=(B, T))
    u = g.uniform(0, 1, size=(B, T))
    # q = p: ratio 1, every first child is accepted down to a leaf; bonus has to be sampled
    r = orc.accept_scan_stochastic(p1, p2, pd, pd, u, parent, tok, 0.5)
    for b in range(B):
        cur, want = 0, []
        while (parent[b] == cur).any():
            cur = int(np.nonzero(parent[b] == cur)[0][0])
            want.append(cur)
        assert r["path"][b, :len(want)].tolist() == want and r["accept_len"][b] == len(want)
        assert r["bonus_tok"][b] == -2 and r["escalate"][b] == 0
    # p = 0: nothing is accepted; u = 0 with p > 0: same as q = p
    r0 = orc.accept_scan_stochastic(p1, p2, np.zeros((B, T)), pd, u, parent, tok, 0.5)
    assert (r0["accept_len"] == 0).all() and (r0["bonus_tok"] == -2).all()
    ru = orc.accept_scan_stochastic(p1, p2, pd, 5 * pd, np.zeros((B, T)), parent, tok, 0.5)
    assert np.array_equal(ru["path"], r["path"])
    # untrusted root escalates before any Bernoulli test
    re = orc.accept_scan_stochastic(np.full((B, T), 0.3), p2, pd, pd, u, parent, tok, 0.5)
    assert re["escalate"].all() and (re["accept_len"] == 0).all() and (re["bonus_tok"] == -1).all()
    # chain: P(tau_a >= j) = prod_{i<=j} min(1, p_i / q_i) (Eq. 6, Eq. 7), by Monte Carlo
    Tc = 6
    cp = np.arange(-1, Tc - 1, dtype=np.int32)[None]
    ct = np.arange(Tc, dtype=np.int32)[None]
    ratio = np.array([1.0, 0.9, 0.5, 1.0, 0.8, 0.3])                  # entry 0 unused (root)
    pdc, qdc = np.minimum(ratio, 1.0)[None] * 0.5, np.full((1, Tc), 0.5)
    n = 20000
    lens = np.zeros(Tc, dtype=int)
    uu = np.random.default_rng(8).uniform(0, 1, size=(n, Tc))
    for t in range(n):
        rr = orc.accept_scan_stochastic(np.ones((1, Tc)), np.zeros((1, Tc)), pdc, qdc, uu[t:t + 1], cp, ct, 0.5)
        lens[rr["accept_len"][0]] += 1
    surv = np.cumprod(ratio[1:])                                      # P(tau_a >= j), j = 1..5
    for j in range(1, Tc):
        pj = surv[j - 1]
        assert abs(lens[j:].sum() / n - pj) < 4 * np.sqrt(pj * (1 - pj) / n) + 1e-9


def test_stochastic_scan_decides_in_double_precision_and_counts_near_ties():
    """Eq. 6 compares u with min(1, p/q). A single-precision division rounds 0.1f/0.3f up to
    0.33333334; a uniform number just below that but above the exact quotient must be REJECTED,
    and counted as lying on the boundary (near_accept), whatever precision the arrays have."""
    parent = np.array([[-1, 0]], dtype=np.int32)
    tok = np.array([[0, 7]], dtype=np.int32)
    one, zero = np.ones((1, 2), dtype=np.float32), np.zeros((1, 2), dtype=np.float32)
    p = np.array([[0.0, 0.1]], dtype=np.float32)
    q = np.array([[0.0, 0.3]], dtype=np.float32)
    exact = float(p[0, 1]) / float(q[0, 1])
    rounded = float(np.float32(p[0, 1]) / np.float32(q[0, 1]))
    assert rounded != exact
    lo, hi = min(exact, rounded), max(exact, rounded)
    u_between = np.array([[0.0, (lo + hi) / 2]], dtype=np.float64)
    r = orc.accept_scan_stochastic(one, zero, p, q, u_between, parent, tok, 0.5)
    assert r["accept_len"][0] == (1 if u_between[0, 1] < exact else 0)
    assert r["near_accept"][0] == 1
    # far from the ratio on either side: decided, not counted
    for uu, want in ((0.2, 1), (0.5, 0)):
        r = orc.accept_scan_stochastic(one, zero, p, q, np.array([[0.0, uu]]), parent, tok, 0.5)
        assert r["accept_len"][0] == want and r["near_accept"][0] == 0
    # only children that are actually tested count: after the first accepted child the siblings are not
    parent3 = np.array([[-1, 0, 0]], dtype=np.int32)
    tok3 = np.array([[0, 7, 8]], dtype=np.int32)
    p3 = np.array([[0.0, 0.5, 0.1]]); q3 = np.array([[0.0, 0.5, 0.3]])
    u3 = np.array([[0.0, 0.9, exact]])
    r = orc.accept_scan_stochastic(np.ones((1, 3)), np.zeros((1, 3)), p3, q3, u3, parent3, tok3, 0.5)
    assert r["path"][0, 0] == 1 and r["near_accept"][0] == 0


def test_gumbel_variate_range_is_bounded_by_the_23_bit_uniform():
    """The uniform number keeps the upper 23 bits of a word, so the variate cannot leave
    [-ln(-ln 2^-24), -ln(-ln(1 - 2^-24))]; an entry 19.45 below the best logit is out of reach."""
    g_min, g_max = orc.gumbel_from_word(0), orc.gumbel_from_word(0xFFFFFFFF)
    assert abs(g_min - (-math.log(24 * math.log(2)))) < 1e-12
    assert abs(g_max - (-math.log(-math.log1p(-2.0 ** -24)))) < 1e-9
    assert -2.813 < g_min < -2.811 and 16.63 < g_max < 16.64
    assert g_max - g_min < 19.45
    for w in (1, 0x1FF, 0x200, 0x7FFFFFFF, 0x80000000, 0xFFFFFE00):
        assert g_min <= orc.gumbel_from_word(w) <= g_max
    # words that differ only in the dropped 9 bits give the same variate; the next one up differs
    assert orc.gumbel_from_word(0x200) == orc.gumbel_from_word(0x3FF) != orc.gumbel_from_word(0x400)
    # monotone in the word
    ws = [0, 0x200, 0x12345600, 0x80000000, 0xFFFFFFFF]
    gs = [orc.gumbel_from_word(w) for w in ws]
    assert all(a < b for a, b in zip(gs, gs[1:]))


def _one_hot_rows(B, T, d, hot):
    """bf16 hidden states that are unit vectors: row (b, i) = e_{hot[b][i]}."""
    h = np.zeros((B, T, d), dtype=np.float32)
    for b in range(B):
        for i in range(T):
            h[b, i, hot[b][i]] = 1.0
    return gen.f32_to_bf16_bits(h)


def test_sample_bonus_on_hand_set_logits():
    """Algorithm 1's x_bonus ~ p: with one-hot hidden states the logits of row (b, node) are a
    column of W, set by hand to bf16-exact values; the expected token is the arg-max of
    z + noise with the noise taken from the scalar generator (counter (v div 4, b, step))."""
    V, d, B, T = 7, 4, 4, 3
    Wf = np.array([[0.0, 2.0, -1.0, 0.5],
                   [1.0, 0.0, -1.0, 0.5],
                   [0.5, -2.0, 3.0, 0.5],
                   [0.0, 0.0, 0.0, 0.5],
                   [-1.0, 1.0, 0.0, 0.5],
                   [2.0, 1.5, 0.25, 0.5],
                   [0.0, -0.5, 1.0, 0.5]], dtype=np.float32)
    W = gen.f32_to_bf16_bits(Wf)
    hot = [[0, 1, 2], [1, 2, 3], [2, 0, 1], [3, 3, 0]]
    h = _one_hot_rows(B, T, d, hot)
    scale = 1.5
    node = np.array([2, 0, -1, 1])                 # sequence 2 is skipped
    seed, step = 0xDEADBEEF12345678, (1 << 33) + 5  # both halves of the 64-bit step are used
    tok, best, gap = orc.sample_bonus(h, W, scale, node, seed, step)
    flipped = 0
    for b in range(B):
        if node[b] < 0:
            assert tok[b] == -1 and np.isnan(best[b]) and np.isnan(gap[b])
            continue
        z = scale * Wf[:, hot[b][node[b]]].astype(np.float64)
        y = np.array([z[v] + orc.gumbel_noise(seed, step, b, v) for v in range(V)])
        order = np.argsort(-y, kind="stable")
        assert tok[b] == order[0]
        assert abs(best[b] - y[order[0]]) < 1e-12 and abs(gap[b] - (y[order[0]] - y[order[1]])) < 1e-12
        flipped += int(order[0] != int(np.argmax(z)))
    # sequence 3, node 1 has all logits equal (column 3): the winner is the arg-max of the noise alone
    noise3 = [orc.gumbel_noise(seed, step, 3, v) for v in range(V)]
    assert tok[3] == int(np.argmax(noise3))
    # the noise must be able to overturn the arg-max of the logits: over rounds, it does, and the
    # round index, the sequence index and the seed all change the draw
    n_flip, draws = 0, set()
    for st in range(200):
        t2, _, _ = orc.sample_bonus(h, W, scale, node, seed, st)
        n_flip += int(t2[0] != int(np.argmax(Wf[:, hot[0][2]])))
        draws.add(tuple(int(x) for x in t2))
    assert 5 < n_flip < 195 and len(draws) > 20
    same_rows = _one_hot_rows(2, 1, d, [[0], [0]])
    t3 = [tuple(orc.sample_bonus(same_rows, W, scale, np.array([0, 0]), seed, st)[0]) for st in range(50)]
    assert any(a != b for a, b in t3)              # sequence index enters the counter
    t4 = [orc.sample_bonus(same_rows, W, scale, np.array([0, 0]), seed + 1, st)[0][0] for st in range(50)]
    assert [a for a, _ in t3] != t4                # so does the seed


def test_sample_bonus_draws_follow_the_softmax():
    """20 000 draws through sample_bonus itself (8 sequences x 2500 rounds, the same row in every
    sequence): every frequency within 4 standard deviations of softmax(z)."""
    V, d, B = 6, 2, 8
    Wf = np.array([[1.0, 0.0], [0.0, 0.0], [-1.0, 0.0], [2.0, 0.0], [0.5, 0.0], [-3.0, 0.0]], dtype=np.float32)
    W = gen.f32_to_bf16_bits(Wf)
    h = _one_hot_rows(B, 1, d, [[0]] * B)
    z = Wf[:, 0].astype(np.float64)
    p = np.exp(z) / np.exp(z).sum()
    W64 = orc.bf16_to_f64(W)
    counts = np.zeros(V)
    rounds = 2500
    node = np.zeros(B, dtype=np.int64)
    for step in range(rounds):
        tok, _, _ = orc.sample_bonus(h, W, 1.0, node, 7, step, W64=W64)
        counts += np.bincount(tok, minlength=V)
    n = rounds * B
    assert counts.sum() == n
    assert np.all(np.abs(counts / n - p) < 4 * np.sqrt(p * (1 - p) / n))


# ------------------------------------------------------------------------------ token-specific deferral rule
def test_token_specific_rule_hand_chain():
    """Chain 0 -> 1 -> 2 -> 3, alpha = 0.2 (the paper's setting): a drafted token is accepted iff
    its probability is at least 0.8 of the verifier's maximum at that position."""
    parent = np.array([[-1, 0, 1, 2]], dtype=np.int32)
    tok = np.array([[0, 5, 6, 7]], dtype=np.int32)
    p1 = np.array([[0.50, 0.60, 0.90, 0.70]])
    p2 = np.zeros((1, 4))
    top1 = np.array([[9, 6, 8, 4]], dtype=np.int64)      # only node 1's arg-max is the drafted token
    # child probabilities at the parent's position: 0.45 >= 0.8*0.50 (accepted though not the arg-max),
    # 0.60 >= 0.8*0.60 (the arg-max itself), 0.70 < 0.8*0.90 = 0.72 (deferred)
    pd = np.array([[np.nan, 0.45, 0.60, 0.70]])
    r = orc.accept_scan_token_specific(p1, p2, top1, pd, parent, tok, 0.0, 0.2, mode=orc.MODE_TARGET)
    assert r["accept_len"][0] == 2 and r["path"][0, :3].tolist() == [1, 2, -1]
    assert r["last_node"][0] == 2 and r["bonus_tok"][0] == 8 and r["escalate"][0] == 0
    # greedy acceptance on the same statistics stops at the root: token 5 is not the arg-max 9
    g = orc.accept_scan(p1, p2, top1, parent, tok, 0.0, mode=orc.MODE_TARGET)
    assert g["accept_len"][0] == 0 and g["bonus_tok"][0] == 9
    # the threshold itself: 0.72 exactly passes (>=), and is counted as lying on the boundary
    pd_edge = np.array([[np.nan, 0.45, 0.60, 0.8 * 0.90]])
    e = orc.accept_scan_token_specific(p1, p2, top1, pd_edge, parent, tok, 0.0, 0.2, mode=orc.MODE_TARGET)
    assert e["accept_len"][0] == 3 and e["bonus_tok"][0] == 4 and e["near_accept"][0] == 1
    # PROXY mode: the margin test comes first; node 2 untrusted (0.9 - 0.5 < 0.45) -> escalate with 2 accepted
    p2m = np.array([[0.0, 0.0, 0.5, 0.0]])
    m = orc.accept_scan_token_specific(p1, p2m, top1, pd, parent, tok, 0.45, 0.2, mode=orc.MODE_PROXY)
    assert m["escalate"][0] == 1 and m["accept_len"][0] == 2 and m["bonus_tok"][0] == -1


def test_token_specific_rule_limits_reduce_to_greedy_and_to_accept_everything():
    """alpha = 0 on real softmax statistics is greedy acceptance (a token reaches the maximum
    probability only by being the arg-max); alpha = 1 accepts the first child at every node
    down to a leaf; the accepted length on a chain never shrinks as alpha grows."""
    cfg = _cfg(B=6, k=14, max_depth=5, V=200, d=64, rho=0.3, logit_scale=3.6 / (0.02 * 8.0), seed=31)
    inp = gen.make_inputs(cfg, with_attention=False)
    st = orc.lmhead_stats(inp["h"], inp["W"], inp["parent"], inp["tok"], cfg.logit_scale)
    parent, tok = inp["parent"], inp["tok"]
    for mode in (orc.MODE_PROXY, orc.MODE_TARGET):
        g = orc.accept_scan(st["p_top1"], st["p_top2"], st["top1_idx"], parent, tok, cfg.lam, mode=mode)
        r0 = orc.accept_scan_token_specific(st["p_top1"], st["p_top2"], st["top1_idx"], st["p_draft"], parent, tok,
                                            cfg.lam, 0.0, mode=mode)
        for k in ("accept_len", "escalate", "bonus_tok", "path", "last_node", "near_thr"):
            assert np.array_equal(g[k], r0[k]), (k, mode)
    assert (g["accept_len"] > 0).any()
    r1 = orc.accept_scan_token_specific(st["p_top1"], st["p_top2"], st["top1_idx"], st["p_draft"], parent, tok,
                                        cfg.lam, 1.0, mode=orc.MODE_TARGET)
    for b in range(cfg.B):
        cur, want = 0, []
        while (parent[b] == cur).any():
            cur = int(np.nonzero(parent[b] == cur)[0][0])
            want.append(cur)
        assert r1["path"][b, :len(want)].tolist() == want and r1["accept_len"][b] == len(want)
        assert r1["bonus_tok"][b] == st["top1_idx"][b, cur]
    # chain: monotone in alpha
    ccfg = gen.small_variant(gen.CONFIGS["tiny_chain"], B=5, V=200, d=64, logit_scale=3.6 / (0.02 * 8.0), seed=32)
    cin = gen.make_inputs(ccfg, with_attention=False)
    cst = orc.lmhead_stats(cin["h"], cin["W"], cin["parent"], cin["tok"], ccfg.logit_scale)
    prev = None
    for alpha in (0.0, 0.2, 0.5, 0.9, 1.0):
        r = orc.accept_scan_token_specific(cst["p_top1"], cst["p_top2"], cst["top1_idx"], cst["p_draft"],
                                           cin["parent"], cin["tok"], 0.5, alpha, mode=orc.MODE_TARGET)
        if prev is not None:
            assert (r["accept_len"] >= prev).all()
        prev = r["accept_len"].copy()
    assert (prev == ccfg.k).all()
