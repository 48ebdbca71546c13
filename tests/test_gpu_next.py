"""GPU parity of token pruning and KV commit against the oracle (bit-exact: integer and byte work),
through the C ABI, plus a proxy round -> prune -> commit composition on one stream."""
import dataclasses
import math

import numpy as np
import pytest

from oracle import trispec_oracle as orc
from paper_2601_23180_b200 import inputs as gen

pytestmark = pytest.mark.gpu


def _trees(name, B, seed=0):
    cfg = gen.small_variant(gen.CONFIGS[name], B=B, seed=seed)
    parent = np.stack([gen.make_tree(cfg, b) for b in range(B)])
    tok = np.stack([gen.make_tokens(cfg, b, parent[b]) for b in range(B)])
    return cfg, parent, tok


def _run_prune(parent, tok, root):
    import torch
    import tests.gpu_helpers as H
    from paper_2601_23180_b200 import binding as ts
    B, T = parent.shape
    pd, td = H.i32_dev(parent), H.i32_dev(tok)
    mask, _ = H.run_tree_mask(pd)
    out = ts.alloc_prune_out(B, T)
    ts.trispec_prune_tree(ts.prune_args(pd, td, mask, H.i32_dev(root), out))
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


@pytest.mark.parametrize("name,B", [("proxy_tree", 37), ("llama_tree", 9), ("tiny_chain", 5)])
def test_prune_bit_exact(name, B):
    cfg, parent, tok = _trees(name, B, seed=3)
    T = cfg.T
    g = np.random.default_rng(7)
    root = g.integers(-1, T, size=B).astype(np.int32)      # -1 = sequence skipped
    root[0] = 0                                            # identity
    root[-1] = T - 1                                       # a leaf
    got = _run_prune(parent, tok, root)
    ref = orc.prune_tree(parent, tok, root)
    for k in ("n_keep", "node_map", "parent", "tok"):
        assert np.array_equal(got[k], ref[k]), k
    # mask / depth of the pruned tree = what the mask oracle gives for the pruned parents
    for b in range(B):
        n = int(ref["n_keep"][b])
        if n:
            m, d = orc.build_tree_mask(ref["parent"][b:b + 1, :n])
            assert np.array_equal(got["mask"][b, :n].view(np.uint64), m[0])
            assert np.array_equal(got["depth"][b, :n], d[0])
        assert (got["mask"][b, n:] == 0).all() and (got["depth"][b, n:] == -1).all()


def test_prune_large_batch_and_argument_errors():
    import torch
    from paper_2601_23180_b200 import binding as ts
    cfg, parent, tok = _trees("proxy_tree", 64, seed=1)
    reps = 47                                              # 3008 sequences: many blocks, ragged last block
    parent, tok = np.tile(parent, (reps, 1)), np.tile(tok, (reps, 1))
    root = np.random.default_rng(0).integers(-1, cfg.T, size=parent.shape[0]).astype(np.int32)
    got = _run_prune(parent, tok, root)
    ref = orc.prune_tree(parent, tok, root)
    for k in ("n_keep", "node_map", "parent", "tok"):
        assert np.array_equal(got[k], ref[k]), k
    a = ts.PruneArgs()
    a.B, a.T = 4, 65
    n0 = ts.launch_count()
    with pytest.raises(ts.TrispecError) as e:
        ts.trispec_prune_tree(a)
    assert e.value.code == 2 and ts.launch_count() == n0   # T > 64
    a.T = 9
    with pytest.raises(ts.TrispecError) as e:
        ts.trispec_prune_tree(a)
    assert e.value.code == 1 and ts.launch_count() == n0   # null pointers


def _run_commit(cfg, inp, path, acc, active=None, in_place=False):
    import torch
    import tests.gpu_helpers as H
    from paper_2601_23180_b200 import binding as ts
    dev = H.to_device(inp)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx_out = dev["ctx_len"] if in_place else torch.full_like(dev["ctx_len"], -7)
    act = None if active is None else torch.from_numpy(active).cuda()
    a = ts.commit_args(dev["k_tree"], dev["v_tree"], dev["k_cache"], dev["v_cache"], dev["ctx_len"], H.i32_dev(path),
                       H.i32_dev(acc), ctx_out, block_table=dev.get("block_table"), block_size=cfg.block_size,
                       active=act, dev_status=status)
    ts.trispec_commit_kv(a)
    torch.cuda.synchronize()
    bits = lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16)
    return bits(dev["k_cache"]), bits(dev["v_cache"]), ctx_out.cpu().numpy(), int(status.item())


@pytest.mark.parametrize("name,in_place", [("proxy_tree", False), ("long_paged", True), ("target_escalated", False)])
def test_commit_bit_exact(name, in_place):
    paged = name == "long_paged"
    cfg = gen.small_variant(gen.CONFIGS[name], B=6, L=300, L_min=300 if paged else None, n_active=None, seed=4)
    inp = gen.make_inputs(cfg, with_lm_head=False)
    B, T = cfg.B, cfg.T
    g = np.random.default_rng(11)
    inp["ctx_len"] = np.array([0, 63, 64, 200, 299 - 7, 128], dtype=np.int32)
    # accepted paths: descending chains of real tree nodes
    path = np.full((B, T), -1, dtype=np.int32)
    acc = np.zeros(B, dtype=np.int32)
    for b in range(B):
        cur, n = 0, 0
        while n < [0, 3, 6, 2, 6, 1][b]:
            kids = np.nonzero(inp["parent"][b] == cur)[0]
            if not len(kids):
                break
            cur = int(g.choice(kids))
            path[b, n] = cur
            n += 1
        acc[b] = n
    active = np.array([1, 1, 1, 0, 1, 1], dtype=np.uint8)
    ref_k, ref_v, ref_len = orc.commit_kv(inp["k_cache"], inp["v_cache"], inp["ctx_len"], inp["k_tree"], inp["v_tree"],
                                          path, acc, block_table=inp.get("block_table"), block_size=cfg.block_size,
                                          active=active)
    got_k, got_v, got_len, status = _run_commit(cfg, inp, path, acc, active=active, in_place=in_place)
    assert status == 0
    assert np.array_equal(got_len, ref_len)
    assert np.array_equal(got_k, ref_k) and np.array_equal(got_v, ref_v)


def test_commit_without_room_flags_and_leaves_the_sequence_alone():
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=2, L=128, seed=2)
    inp = gen.make_inputs(cfg, with_lm_head=False)
    inp["ctx_len"] = np.array([127, 126], dtype=np.int32)
    path = np.full((2, cfg.T), -1, dtype=np.int32)
    path[:, 0] = 1
    acc = np.array([1, 1], dtype=np.int32)                 # two rows each: only sequence 1 fits
    ref_k, ref_v, ref_len = orc.commit_kv(inp["k_cache"], inp["v_cache"], inp["ctx_len"], inp["k_tree"], inp["v_tree"],
                                          path, acc)
    got_k, got_v, got_len, status = _run_commit(cfg, inp, path, acc)
    assert status == 9
    assert got_len.tolist() == ref_len.tolist() == [127, 128]
    assert np.array_equal(got_k, ref_k) and np.array_equal(got_v, ref_v)


def test_round_then_prune_and_commit_on_one_stream():
    """One proxy round of the decode loop: verify pass -> (escalated sequences) prune at the
    last accepted node, and commit the accepted path, launched back to back; compared with the
    oracle run on the GPU's own scan outputs (so only the new steps are under test here)."""
    import torch
    import tests.gpu_helpers as H
    from paper_2601_23180_b200 import binding as ts
    from paper_2601_23180_b200 import runner
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=6, L=200, V=8000, d=256, rho=0.3,
                            logit_scale=3.6 / (0.02 * 16.0), seed=5)
    inp = gen.make_inputs(cfg)
    inp["ctx_len"] = np.full(cfg.B, 130, dtype=np.int32)   # room for the appended rows
    pas = runner.VerifyPass(cfg, inp)
    B, T = cfg.B, cfg.T
    pout = ts.alloc_prune_out(B, T)
    # prune where the proxy escalated: root = last_node for escalated sequences, else -1
    pas.run()
    esc = pas.scan_out["escalate"].to(torch.bool)
    root = torch.where(esc, pas.scan_out["last_node"], torch.full_like(pas.scan_out["last_node"], -1))
    ts.trispec_prune_tree(ts.prune_args(pas.dev["parent"], pas.dev["tok"], pas.mask, root, pout))
    ctx_out = torch.zeros_like(pas.dev["ctx_len"])
    ts.trispec_commit_kv(ts.commit_args(pas.dev["k_tree"], pas.dev["v_tree"], pas.dev["k_cache"], pas.dev["v_cache"],
                                        pas.dev["ctx_len"], pas.scan_out["path"], pas.scan_out["accept_len"], ctx_out,
                                        dev_status=pas.status))
    torch.cuda.synchronize()
    assert int(pas.status.item()) == 0
    scan = {k: v.cpu().numpy() for k, v in pas.scan_out.items()}
    ref_p = orc.prune_tree(inp["parent"], inp["tok"], root.cpu().numpy())
    for k in ("n_keep", "node_map", "parent", "tok"):
        assert np.array_equal(pout[k].cpu().numpy(), ref_p[k]), k
    ref_k, ref_v, ref_len = orc.commit_kv(inp["k_cache"], inp["v_cache"], inp["ctx_len"], inp["k_tree"], inp["v_tree"],
                                          scan["path"], scan["accept_len"])
    bits = lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(ctx_out.cpu().numpy(), ref_len)
    assert np.array_equal(bits(pas.dev["k_cache"]), ref_k) and np.array_equal(bits(pas.dev["v_cache"]), ref_v)
    assert scan["escalate"].sum() >= 1 and (scan["accept_len"] > 0).any()


def _with_duplicate_siblings(parent, tok):
    """Gives the first two children of every node that has two the same token (the generator makes
    siblings distinct): the acceptance rules must then take the one with the lower node index."""
    tok = tok.copy()
    n = 0
    for b in range(parent.shape[0]):
        for i in range(parent.shape[1]):
            kids = np.nonzero(parent[b] == i)[0]
            if len(kids) >= 2:
                tok[b, kids[1]] = tok[b, kids[0]]
                n += 1
    assert n > 0
    return tok


@pytest.mark.parametrize("mode", [gen.MODE_PROXY, gen.MODE_TARGET])
def test_greedy_scan_with_duplicate_sibling_tokens(mode):
    """Two children of a node carrying the same token: the lower node index is accepted."""
    import tests.gpu_helpers as H
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=45, seed=9)
    B, T = cfg.B, cfg.T
    parent = np.stack([gen.make_tree(cfg, b) for b in range(B)])
    tok = _with_duplicate_siblings(parent, np.stack([gen.make_tokens(cfg, b, parent[b]) for b in range(B)]))
    g = np.random.default_rng(5)
    top1 = g.integers(0, cfg.V, size=(B, T))
    hit_second = 0
    for b in range(B):
        for i in range(T):
            kids = np.nonzero(parent[b] == i)[0]
            if len(kids) and g.random() < 0.9:
                top1[b, i] = tok[b, kids[min(1, len(kids) - 1)]]      # the duplicated token where there is one
    st = {"p_top1": g.uniform(0.45, 1.0, size=(B, T)).astype(np.float32),
          "p_top2": g.uniform(0.0, 0.1, size=(B, T)).astype(np.float32), "top1_idx": top1}
    ref = orc.accept_scan(st["p_top1"].astype(np.float64), st["p_top2"].astype(np.float64), top1, parent, tok, 0.5,
                          mode=mode)
    got = H.run_scan(st, parent, tok, 0.5, mode)
    clean = ref["near_thr"] == 0
    assert clean.sum() >= B - 3
    for k in ("accept_len", "escalate", "bonus_tok", "last_node", "path"):
        assert np.array_equal(got[k][clean], ref[k][clean]), k
    # the case under test occurred: an accepted node whose next sibling carries the same token
    for b in range(B):
        for c in ref["path"][b]:
            if c >= 0 and c + 1 < T and parent[b, c + 1] == parent[b, c] and tok[b, c + 1] == tok[b, c]:
                hit_second += 1
    assert hit_second >= 10


@pytest.mark.parametrize("mode", [gen.MODE_PROXY, gen.MODE_TARGET])
@pytest.mark.parametrize("dup", [False, True])
def test_stochastic_acceptance_bit_exact(mode, dup):
    """Eq. 6 at temperature 1 on fp32 inputs given to both sides. The oracle decides in fp64, the
    kernel in fp32: sequences whose walk tests a uniform number within 1e-6 of the acceptance ratio
    are counted and set aside (as are near-threshold margins); every other sequence must agree."""
    import tests.gpu_helpers as H
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=53, seed=8)
    B, T = cfg.B, cfg.T
    parent = np.stack([gen.make_tree(cfg, b) for b in range(B)])
    tok = np.stack([gen.make_tokens(cfg, b, parent[b]) for b in range(B)])
    if dup:
        tok = _with_duplicate_siblings(parent, tok)
    g = np.random.default_rng(4)
    st = {"p_top1": g.uniform(0.4, 1.0, size=(B, T)).astype(np.float32),
          "p_top2": g.uniform(0.0, 0.2, size=(B, T)).astype(np.float32),
          "p_draft": g.uniform(0.0, 0.8, size=(B, T)).astype(np.float32),
          "top1_idx": g.integers(0, cfg.V, size=(B, T))}
    q = g.uniform(0.05, 0.9, size=(B, T)).astype(np.float32)
    q[:, 5] = 0.0                                             # drafter probability 0: ratio taken as 1
    u = g.uniform(0, 1, size=(B, T)).astype(np.float32)
    # plant boundary draws: u equal to the fp32 quotient, which the fp64 ratio may fall on either side of
    for b in (3, 11, 29):
        c = 1
        u[b, c] = np.float32(st["p_draft"][b, c]) / np.float32(q[b, c]) if q[b, c] > st["p_draft"][b, c] else u[b, c]
    ref = orc.accept_scan_stochastic(st["p_top1"], st["p_top2"], st["p_draft"], q, u, parent, tok, 0.5, mode=mode)
    got = H.run_scan(st, parent, tok, 0.5, mode, q_draft=q, u_accept=u)
    clean = (ref["near_thr"] == 0) & (ref["near_accept"] == 0)
    assert clean.sum() >= B - 6 and (ref["near_accept"] > 0).sum() <= 3
    for k in ("accept_len", "escalate", "bonus_tok", "last_node", "path"):
        assert np.array_equal(got[k][clean], ref[k][clean]), k
    assert (ref["accept_len"] > 0).any() and (ref["bonus_tok"] == -2).any()
    if mode == gen.MODE_PROXY:
        assert ref["escalate"].any()


@pytest.mark.parametrize("mode", [gen.MODE_PROXY, gen.MODE_TARGET])
@pytest.mark.parametrize("alpha", [0.2, 0.0, 1.0])
def test_token_specific_rule_bit_exact(mode, alpha):
    """The token-specific deferral rule (accept iff p(drafted token) >= (1 - alpha) max p) on fp32
    statistics given to both sides: bit-exact except sequences that test a probability within 1e-6
    of the bar (the kernel multiplies in fp32) or meet a near-threshold margin."""
    import tests.gpu_helpers as H
    from paper_2601_23180_b200 import binding as ts
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=47, seed=10)
    B, T = cfg.B, cfg.T
    parent = np.stack([gen.make_tree(cfg, b) for b in range(B)])
    tok = np.stack([gen.make_tokens(cfg, b, parent[b]) for b in range(B)])
    g = np.random.default_rng(6)
    p1 = g.uniform(0.35, 1.0, size=(B, T)).astype(np.float32)
    # a drafted token's probability at its parent: sometimes the maximum itself, mostly a fraction of it
    pd = np.full((B, T), np.nan, dtype=np.float32)
    for b in range(B):
        for c in range(1, T):
            f = 1.0 if g.random() < 0.3 else g.uniform(0.3, 1.0)
            pd[b, c] = np.float32(f) * p1[b, parent[b, c]]
    st = {"p_top1": p1, "p_top2": g.uniform(0.0, 0.1, size=(B, T)).astype(np.float32), "p_draft": pd,
          "top1_idx": g.integers(0, cfg.V, size=(B, T))}
    ref = orc.accept_scan_token_specific(p1.astype(np.float64), st["p_top2"].astype(np.float64), st["top1_idx"],
                                         pd.astype(np.float64), parent, tok, 0.5, alpha, mode=mode)
    got = H.run_scan(st, parent, tok, 0.5, mode, accept_rule=ts.ACCEPT_TOKEN_SPECIFIC, alpha=alpha)
    clean = (ref["near_thr"] == 0) & (ref["near_accept"] == 0)
    if alpha == 0.0:
        # the bar is the maximum itself and many drafted tokens sit exactly on it: exact in both precisions
        clean = ref["near_thr"] == 0
    assert clean.sum() >= B - 6
    for k in ("accept_len", "escalate", "bonus_tok", "last_node", "path"):
        assert np.array_equal(got[k][clean], ref[k][clean]), (k, alpha)
    if alpha == 1.0:
        assert (ref["accept_len"][ref["escalate"] == 0] > 0).all()
    if alpha == 0.2:
        assert 0 < (ref["accept_len"] > 0).sum() and (ref["bonus_tok"] >= 0).any()


def _run_sample(dev, cfg, last_node, bonus_in, seed, step):
    import torch
    import tests.gpu_helpers as H
    from paper_2601_23180_b200 import binding as ts
    bonus = H.i32_dev(bonus_in)
    val = torch.full((cfg.B,), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    a = ts.sample_args(dev["h"], dev["W"], H.i32_dev(last_node), bonus, cfg.logit_scale, seed, step,
                       sample_value=val, dev_status=status)
    ws = ts.alloc_workspace(ts.trispec_sample_bonus_workspace(a))
    a.workspace, a.workspace_bytes = ws.data_ptr(), ws.numel()
    ts.trispec_sample_bonus(a)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return bonus.cpu().numpy(), val.cpu().numpy()


@pytest.mark.parametrize("name,over", [("proxy_tree", dict(B=5, V=20011, d=256)),        # few sequences: W on the M side
                                       ("llama_tree", dict(B=19, V=128256 // 8, d=512)),  # 32 sequence columns
                                       ("proxy_tree", dict(B=40, V=9000, d=128)),         # 64 sequence columns, two epilogue groups
                                       ("proxy_tree", dict(B=33, V=5000, d=64)),          # one sequence in the second group
                                       ("proxy_tree", dict(B=64, V=7000, d=128)),         # both groups full
                                       ("proxy_tree", dict(B=70, V=6000, d=64))])         # sequences on the M side
def test_bonus_sampling_matches_gumbel_max_oracle(name, over):
    """The sampled token is argmax_v (z_v + G_v) with the oracle's counter-based noise. fp32 logits
    can flip the arg-max only where the two best perturbed logits are closer than the LM-head
    tolerance (1e-3 relative); those sequences are counted, the rest must agree exactly."""
    import tests.gpu_helpers as H
    cfg = gen.small_variant(gen.CONFIGS[name], logit_scale=3.6 / (0.02 * math.sqrt(over["d"])), **over)
    inp = gen.make_inputs(cfg, with_attention=False)
    dev = H.to_device(inp)
    B, T = cfg.B, cfg.T
    g = np.random.default_rng(3)
    last = g.integers(0, T, size=B).astype(np.int32)
    bonus_in = np.full(B, -2, dtype=np.int32)
    bonus_in[1] = 777                                   # not asked for: left alone
    seed, step = 0x9e3779b97f4a7c15, 41
    node = np.where(bonus_in == -2, last, -1)
    ref_tok, ref_best, ref_gap = orc.sample_bonus(inp["h"], inp["W"], cfg.logit_scale, node, seed, step)
    got, val = _run_sample(dev, cfg, last, bonus_in, seed, step)
    assert got[1] == 777 and np.isnan(val[1])
    n_tie = 0
    for b in range(B):
        if bonus_in[b] != -2:
            continue
        assert abs(val[b] - ref_best[b]) <= 1e-3 * max(1.0, abs(ref_best[b]))
        if ref_gap[b] < 1e-3 * max(1.0, abs(ref_best[b])):
            n_tie += 1
        else:
            assert got[b] == ref_tok[b], (b, got[b], ref_tok[b])
    assert n_tie <= 1
    # the same (seed, step) reproduces the draw; another step draws afresh
    # (peaked rows can draw the same token again, so the winning perturbed logits are compared)
    again, val_again = _run_sample(dev, cfg, last, bonus_in, seed, step)
    _, val_other = _run_sample(dev, cfg, last, bonus_in, seed, step + 1)
    live = bonus_in == -2
    assert np.array_equal(again, got) and np.array_equal(val_again[live], val[live])
    assert not np.any(val_other[live] == val[live])


def test_bonus_sampling_follows_the_softmax_on_a_small_vocabulary():
    """V = 64, one row with a known distribution sampled over many steps and sequences: every
    frequency within 4.5 standard deviations of softmax(z) (computed by the oracle's lmhead_stats)."""
    import torch
    import tests.gpu_helpers as H
    from paper_2601_23180_b200 import binding as ts
    cfg = gen.small_variant(gen.CONFIGS["tiny_chain"], B=128, V=64, d=64, logit_scale=3.0)
    inp = gen.make_inputs(gen.small_variant(cfg, B=1), with_attention=False)
    T = cfg.T
    h = np.repeat(inp["h"], cfg.B, axis=0)              # every sequence holds the same rows
    dev = {"h": H.bf16_dev(h), "W": H.bf16_dev(inp["W"])}
    W64 = orc.bf16_to_f64(inp["W"])
    z = orc.row_logits(inp["h"][0, 3], W64, cfg.logit_scale)
    p = np.exp(z - z.max())
    p /= p.sum()
    last = np.full(cfg.B, 3, dtype=np.int32)
    counts = np.zeros(cfg.V)
    n_steps = 60
    for step in range(n_steps):
        got, _ = _run_sample(dev, cfg, last, np.full(cfg.B, -2, dtype=np.int32), 12345, step)
        counts += np.bincount(got, minlength=cfg.V)
    n = n_steps * cfg.B
    assert counts.sum() == n
    # counts are integers: allow two draws on top of 4.5 standard deviations (rare tokens)
    assert np.all(np.abs(counts - n * p) <= 4.5 * np.sqrt(n * p * (1 - p)) + 2.0)


def test_fused_pass_with_entropy_routing():
    """The fused pass asks the LM head for the entropy only when the routing criterion reads it. Here
    it does: the entropies must match the oracle's, and the scan must be the oracle's entropy-routed
    walk on the statistics the GPU produced (sequences with a feature on the threshold excepted)."""
    import torch
    import tests.gpu_helpers as H
    from paper_2601_23180_b200 import binding as ts
    from paper_2601_23180_b200 import runner
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=6, L=130, V=12000, d=256, lam=1.2,
                            logit_scale=3.6 / (0.02 * 16.0), seed=11)
    inp = gen.make_inputs(cfg)
    margin_pass = runner.VerifyPass(cfg, inp)
    assert "entropy" not in margin_pass.stats            # the margin rule does not pay for it
    pas = runner.VerifyPass(cfg, inp, criterion=ts.CRIT_ENTROPY)
    pas.run()
    torch.cuda.synchronize()
    got = pas.results()
    assert got["status"] == 0
    ref_st = orc.lmhead_stats(inp["h"], inp["W"], inp["parent"], inp["tok"], cfg.logit_scale)
    H.check_stats(got["stats"], ref_st, pas.seqs, cfg.T)
    st = got["stats"]
    ref = orc.accept_scan(st["p_top1"].astype(np.float64), st["p_top2"].astype(np.float64),
                          st["top1_idx"].astype(np.int64), inp["parent"], inp["tok"], cfg.lam, mode=cfg.mode,
                          criterion=orc.CRIT_ENTROPY, entropy=st["entropy"].astype(np.float64))
    clean = (ref["near_thr"] == 0) & (got["scan"]["near_thr"] == 0)
    assert clean.sum() >= cfg.B - 2
    for k in ("accept_len", "escalate", "bonus_tok", "last_node", "path"):
        assert np.array_equal(got["scan"][k][clean], ref[k][clean]), k
    # the entropy criterion must route both ways on this input, or the test says nothing
    assert 0 < ref["escalate"].sum() < cfg.B


@pytest.mark.parametrize("name,over,n_nodes", [
    # G = 8: four M tiles of 16 nodes; whole tiles, part of a tile and nothing at all are left out
    ("target_escalated", dict(B=5, n_active=5, L=700), [61, 30, 16, 5, 0]),
    # one M tile, cluster merge over several splits
    ("proxy_tree", dict(B=3, L=2000), [61, 1, 40]),
    # more than 8 splits: the workspace merge kernel skips the rows too
    ("proxy_tree", dict(B=2, L=9300, Hq=4, Hkv=2), [7, 61]),
])
def test_attention_of_pruned_trees(name, over, n_nodes):
    """With n_nodes, a sequence's tree ends after its first n_nodes[b] nodes (parents precede children, so
    a prefix of the nodes is a tree): those rows equal the oracle's, the others are never written."""
    import tests.gpu_helpers as H
    cfg = gen.small_variant(gen.CONFIGS[name], **over)
    inp = gen.make_inputs(cfg, with_lm_head=False)
    dev = H.to_device(inp)
    mask_dev, _ = H.run_tree_mask(dev["parent"])
    o, lse = H.run_attn(dev, cfg, mask_dev, n_nodes=np.array(n_nodes, dtype=np.int32))
    ref_mask, _ = orc.build_tree_mask(inp["parent"])
    ref_o, ref_lse = orc.verify_attn(inp["q"], inp["k_tree"], inp["v_tree"], ref_mask, inp["k_cache"],
                                     inp["v_cache"], inp["ctx_len"], 1.0 / math.sqrt(cfg.D),
                                     block_table=inp.get("block_table"), block_size=cfg.block_size)
    for b in range(cfg.B):
        n = n_nodes[b]
        if n:
            assert np.abs(o[b, :n] - ref_o[b, :n]).max() <= 2e-2, b
            assert np.abs(lse[b, :, :n] - ref_lse[b, :, :n]).max() <= 1e-3 * max(1.0, np.abs(ref_lse[b, :, :n]).max())
        assert np.isnan(o[b, n:]).all() and np.isnan(lse[b, :, n:]).all(), b


def test_tree_mask_large_batch_matches_oracle():
    """Batches of 2048 sequences and more take the thread-per-sequence mask kernel: bit-exact against the
    oracle on the workload's trees, on a chain of 64 nodes, and with malformed parents flagged as in the
    warp-per-sequence kernel (mask 0, depth -1, for the node and everything below it)."""
    import tests.gpu_helpers as H
    cfg = gen.CONFIGS["proxy_tree"]
    distinct = np.stack([gen.make_tree(dataclasses.replace(cfg, seed=cfg.seed + s), 0) for s in range(300)])
    ref_mask, ref_depth = orc.build_tree_mask(distinct)
    B = 2048 + 37                                             # a ragged last block
    idx = np.arange(B) % len(distinct)
    parent = distinct[idx].copy()
    bad_rows = [5, 64, 2000, B - 1]
    for b in bad_rows:
        parent[b, 7] = 9                                      # parent after the child
    mask, depth = H.run_tree_mask(H.i32_dev(parent))
    mask, depth = mask.cpu().numpy().view(np.uint64), depth.cpu().numpy()
    good = np.ones(B, dtype=bool); good[bad_rows] = False
    assert np.array_equal(mask[good], ref_mask[idx][good]) and np.array_equal(depth[good], ref_depth[idx][good])
    for b in bad_rows:
        below = [i for i in range(cfg.T) if (int(ref_mask[idx[b], i]) >> 7) & 1]   # node 7 and its descendants
        assert len(below) >= 1
        for i in range(cfg.T):
            if i in below:
                assert mask[b, i] == 0 and depth[b, i] == -1
            else:
                assert mask[b, i] == ref_mask[idx[b], i] and depth[b, i] == ref_depth[idx[b], i]
    # other node counts (49: copy loops that wrap a sequence boundary at odd offsets; 9: several sequences per step)
    for name, nb in (("llama_tree", 2048 + 5), ("tiny_chain", 4096 + 2)):
        c2 = gen.CONFIGS[name]
        d2 = np.stack([gen.make_tree(dataclasses.replace(c2, seed=c2.seed + s), 0) for s in range(100)])
        i2 = (np.arange(nb) * 7) % len(d2)
        m2, dp2 = H.run_tree_mask(H.i32_dev(d2[i2].copy()))
        rm2, rd2 = orc.build_tree_mask(d2)
        assert np.array_equal(m2.cpu().numpy().view(np.uint64), rm2[i2]) and np.array_equal(dp2.cpu().numpy(), rd2[i2])
    chain = np.tile(np.arange(-1, 63, dtype=np.int32), (2048, 1))
    m, d = H.run_tree_mask(H.i32_dev(chain))
    cm, cd = orc.build_tree_mask(chain[:1])
    assert np.array_equal(m.cpu().numpy().view(np.uint64), np.tile(cm, (2048, 1)))
    assert np.array_equal(d.cpu().numpy(), np.tile(cd, (2048, 1)))


def test_host_pass_with_separately_allocated_host_buffers():
    """The host-buffer entry point merges copies only where host and device addresses both follow each
    other; with every host array in an allocation of its own it must fall back to one transfer per array
    and give the same results as the device-resident pass."""
    import torch
    from paper_2601_23180_b200 import binding as ts
    from paper_2601_23180_b200 import runner
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=3, L=300, V=6000, d=128, logit_scale=3.6 / (0.02 * math.sqrt(128)))
    inp = gen.make_inputs(cfg)
    pas = runner.VerifyPass(cfg, inp)
    pas.run()
    torch.cuda.synchronize()
    want = {k: v.clone() for k, v in pas.scan_out.items()}
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    B, T = cfg.B, cfg.T
    host = {"parent": pin(inp["parent"]), "tok": pin(inp["tok"])}
    for k in ("h", "q", "k_tree", "v_tree"):
        host[k] = pin(inp[k].view(np.int16))
    for k in ("accept_len", "bonus_tok", "last_node"):
        host[k] = torch.full((B,), -9, dtype=torch.int32).pin_memory()
    host["path"] = torch.full((B, T), -9, dtype=torch.int32).pin_memory()
    host["escalate"] = torch.full((B,), 7, dtype=torch.uint8).pin_memory()
    for k in ("q", "k_tree", "v_tree", "h"):
        pas.dev[k].zero_()                                   # the pass must bring them from the host
    pas.dev["parent"].fill_(-1)
    pas.dev["tok"].zero_()
    ts.trispec_verify_host(ts.host_io(**host), pas.tree_args, pas.attn_args, pas.lm_args, pas.scan_args)
    torch.cuda.synchronize()
    assert int(pas.status.item()) == 0
    for k in ("accept_len", "bonus_tok", "last_node", "path", "escalate"):
        assert torch.equal(host[k], want[k].cpu()), k


def test_escalation_list_of_a_very_large_batch():
    """More than 65536 sequences: with the optional scratch the ordered list of escalated ids is built by
    one block per 65536 flags (two launches), without it by one block; both must give the ascending ids
    of the sequences the scan flagged, -1 beyond them, and the scan itself must match the oracle."""
    import torch
    import tests.gpu_helpers as H
    from paper_2601_23180_b200 import binding as ts
    cfg, parent64, tok64 = _trees("proxy_tree", 64, seed=21)
    B, T = 3 * 65536 + 4321, cfg.T                      # four blocks, the last one ragged
    reps = (B + 63) // 64
    parent, tok = np.tile(parent64, (reps, 1))[:B], np.tile(tok64, (reps, 1))[:B]
    g = np.random.default_rng(12)
    first_child = np.full((64, T), -1)
    for b in range(64):
        for c in range(T - 1, 0, -1):
            first_child[b, parent64[b, c]] = c
    fc = np.tile(first_child, (reps, 1))[:B]
    top1 = np.where(fc >= 0, np.take_along_axis(tok, np.maximum(fc, 0), axis=1), 7).astype(np.int64)
    p1 = g.uniform(0.52, 1.0, size=(B, T)).astype(np.float32)
    p1[g.uniform(size=(B, T)) < 0.1] = 0.3              # about a tenth of the nodes is untrusted
    p1[1000:70000] = 0.9                                # a long stretch without any escalation
    p2 = np.zeros((B, T), dtype=np.float32)
    st = {"p_top1": torch.from_numpy(p1).cuda(), "p_top2": torch.from_numpy(p2).cuda(),
          "top1_idx": H.i32_dev(top1)}
    pd, td = H.i32_dev(parent), H.i32_dev(tok)
    results = []
    for with_scratch in (True, False):
        out = ts.alloc_scan_out(B, T)
        assert "compact_scratch" in out
        if not with_scratch:
            del out["compact_scratch"]
        n0 = ts.launch_count()
        ts.trispec_accept_scan(ts.scan_args(st, pd, td, 0.5, gen.MODE_PROXY, out))
        torch.cuda.synchronize()
        assert ts.launch_count() - n0 == (3 if with_scratch else 2)
        got = {k: v.cpu().numpy() for k, v in out.items()}
        esc = np.nonzero(got["escalate"])[0]
        assert 1000 < len(esc) < B - 1000 and not ((esc >= 1000) & (esc < 70000)).any()
        assert got["n_escalated"][0] == len(esc)
        assert np.array_equal(got["esc_index"][:len(esc)], esc) and (got["esc_index"][len(esc):] == -1).all()
        results.append(got)
    for k in ("accept_len", "escalate", "bonus_tok", "last_node", "esc_index"):
        assert np.array_equal(results[0][k], results[1][k]), k
    # the walk itself against the oracle, on a sample that spans the block boundaries
    pick = np.concatenate([np.arange(0, 40), np.arange(65536 - 20, 65536 + 20), np.arange(B - 40, B)])
    ref = orc.accept_scan(p1[pick].astype(np.float64), p2[pick].astype(np.float64), top1[pick], parent[pick], tok[pick], 0.5)
    for k in ("accept_len", "escalate", "bonus_tok", "last_node"):
        assert np.array_equal(results[0][k][pick], ref[k]), k
