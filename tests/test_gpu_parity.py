"""GPU parity tests: the CUDA path, called through the C ABI, against the CPU oracle on the
same seeded inputs, element by element at sizes that span several tiles and ragged tails."""
import math

import numpy as np
import pytest

from oracle import trispec_oracle as orc
from paper_2601_23180_b200 import inputs as gen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def H():
    import tests.gpu_helpers as h
    return h


# ------------------------------------------------------------------------------ tree mask
@pytest.mark.parametrize("name", gen.CONFIG_ORDER)
def test_tree_mask_bit_exact(H, name):
    cfg = gen.CONFIGS[name]
    parent = np.stack([gen.make_tree(cfg, b) for b in range(cfg.B)])
    mask, depth = H.run_tree_mask(H.i32_dev(parent))
    ref_mask, ref_depth = orc.build_tree_mask(parent)
    assert np.array_equal(mask.cpu().numpy().view(np.uint64), ref_mask)
    assert np.array_equal(depth.cpu().numpy(), ref_depth)


def test_tree_mask_edge_cases(H):
    # single node; T = 64 chain (bit 63 set); malformed parents are flagged, not followed
    for parent in (np.array([[-1]], dtype=np.int32), np.arange(-1, 63, dtype=np.int32)[None]):
        mask, depth = H.run_tree_mask(H.i32_dev(parent))
        ref_mask, ref_depth = orc.build_tree_mask(parent)
        assert np.array_equal(mask.cpu().numpy().view(np.uint64), ref_mask)
        assert np.array_equal(depth.cpu().numpy(), ref_depth)
    bad = np.array([[-1, 0, 2, 1], [-1, 0, 0, 7]], dtype=np.int32)
    mask, depth = H.run_tree_mask(H.i32_dev(bad))
    m = mask.cpu().numpy()
    assert m[0, 2] == 0 and depth[0, 2].item() == -1 and m[0, 1] == 3
    assert m[1, 3] == 0 and depth[1, 3].item() == -1


# ------------------------------------------------------------------------------ accept scan
@pytest.mark.parametrize("mode", [gen.MODE_PROXY, gen.MODE_TARGET])
@pytest.mark.parametrize("name,B", [("proxy_tree", 37), ("llama_tree", 16), ("tiny_chain", 5)])
def test_scan_bit_exact_on_oracle_stats(H, name, B, mode):
    cfg = gen.small_variant(gen.CONFIGS[name], B=B, V=2048, d=128, rho=0.3,
                            logit_scale=3.6 / (0.02 * math.sqrt(128)))
    inp = gen.make_inputs(cfg, with_attention=False)
    st = orc.lmhead_stats(inp["h"], inp["W"], inp["parent"], inp["tok"], cfg.logit_scale)
    # the scan decides in fp32: give both sides the same fp32 probabilities
    st32 = {"p_top1": st["p_top1"].astype(np.float32), "p_top2": st["p_top2"].astype(np.float32),
            "top1_idx": st["top1_idx"]}
    active = (np.arange(B) % 5 != 3).astype(np.uint8)
    for lam in (0.5, 0.0, 1.5):
        ref = orc.accept_scan(st32["p_top1"].astype(np.float64), st32["p_top2"].astype(np.float64),
                              st32["top1_idx"], inp["parent"], inp["tok"], lam, mode=mode, active=active)
        got = H.run_scan(st32, inp["parent"], inp["tok"], lam, mode, active=active)
        clean = ref["near_thr"] == 0
        for k in ("accept_len", "escalate", "bonus_tok", "last_node", "path"):
            assert np.array_equal(got[k][clean], ref[k][clean]), (k, lam)
        assert np.array_equal(got["near_thr"], ref["near_thr"])
        if clean.all():
            assert got["n_escalated"][0] == ref["n_escalated"]
            assert np.array_equal(got["esc_index"], ref["esc_index"])


@pytest.mark.parametrize("crit,lam", [(1, 0.6), (2, 1.5)])
def test_scan_routing_criteria_bit_exact(H, crit, lam):
    """Top-1-probability and entropy routing (the routing-criteria study) on fp32 statistics given to
    both sides: bit-exact except sequences that visit a feature within 1e-3 of the threshold."""
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=41, seed=6)
    B, T = cfg.B, cfg.T
    parent = np.stack([gen.make_tree(cfg, b) for b in range(B)])
    tok = np.stack([gen.make_tokens(cfg, b, parent[b]) for b in range(B)])
    g = np.random.default_rng(2)
    top1 = g.integers(0, cfg.V, size=(B, T))
    for b in range(B):
        for i in range(T):
            kids = np.nonzero(parent[b] == i)[0]
            if len(kids) and g.random() < 0.85:
                top1[b, i] = tok[b, g.choice(kids)]
    st = {"p_top1": g.uniform(0.3, 1.0, size=(B, T)).astype(np.float32),
          "p_top2": g.uniform(0.0, 0.3, size=(B, T)).astype(np.float32),
          "entropy": g.uniform(0.0, 3.0, size=(B, T)).astype(np.float32), "top1_idx": top1}
    ref = orc.accept_scan(st["p_top1"].astype(np.float64), st["p_top2"].astype(np.float64), top1, parent, tok, lam,
                          criterion=crit, entropy=st["entropy"].astype(np.float64))
    got = H.run_scan(st, parent, tok, lam, gen.MODE_PROXY, criterion=crit)
    clean = ref["near_thr"] == 0
    assert clean.sum() >= B - 3 and ref["escalate"].any() and not ref["escalate"].all()
    for k in ("accept_len", "escalate", "bonus_tok", "last_node", "path"):
        assert np.array_equal(got[k][clean], ref[k][clean]), k
    assert np.array_equal(got["near_thr"], ref["near_thr"])


def test_scan_start_node_and_large_batch(H):
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=3000, V=512, d=64, rho=0.2,
                            logit_scale=3.6 / (0.02 * 8.0))
    parent = np.stack([gen.make_tree(cfg, b) for b in range(cfg.B)])
    tok = np.stack([gen.make_tokens(cfg, b, parent[b]) for b in range(cfg.B)])
    g = np.random.default_rng(0)
    # synthetic statistics: top-1 is a child's token with probability 0.7
    top1 = np.zeros((cfg.B, cfg.T), dtype=np.int64)
    for b in range(cfg.B):
        for r in range(cfg.T):
            kids = np.nonzero(parent[b] == r)[0]
            top1[b, r] = tok[b, g.choice(kids)] if len(kids) and g.random() < 0.7 else g.integers(0, cfg.V)
    p1 = g.uniform(0.4, 1.0, (cfg.B, cfg.T)).astype(np.float32)
    p2 = (p1 * g.uniform(0.0, 0.5, (cfg.B, cfg.T))).astype(np.float32)
    st = {"p_top1": p1, "p_top2": p2, "top1_idx": top1}
    start = g.integers(0, 3, cfg.B).astype(np.int32)
    for mode, sn in ((gen.MODE_PROXY, None), (gen.MODE_TARGET, start)):
        ref = orc.accept_scan(p1.astype(np.float64), p2.astype(np.float64), top1, parent, tok, 0.5, mode=mode,
                              start_node=sn)
        got = H.run_scan(st, parent, tok, 0.5, mode, start_node=sn)
        clean = ref["near_thr"] == 0
        for k in ("accept_len", "escalate", "bonus_tok", "last_node", "path"):
            assert np.array_equal(got[k][clean], ref[k][clean]), k
        esc = np.nonzero(got["escalate"])[0]
        assert got["n_escalated"][0] == len(esc)
        assert np.array_equal(got["esc_index"][:len(esc)], esc) and (got["esc_index"][len(esc):] == -1).all()


# ------------------------------------------------------------------------------ LM-head stats
LM_CASES = [
    # name, overrides: several M tiles, several vocabulary tiles per CTA, ragged vocabulary tail
    ("tiny_chain", dict(V=5000, d=256)),
    ("proxy_tree", dict(B=3, V=40011, d=512)),
    ("proxy_tree", dict(B=5, V=151936 // 8, d=192, logit_scale=3.6 / (0.02 * math.sqrt(192)))),
    ("target_escalated", dict(B=7, n_active=3, V=9000, d=320, logit_scale=3.6 / (0.02 * math.sqrt(320)))),
    ("llama_tree", dict(B=2, V=128256 // 4, d=1024, logit_scale=3.6 / (0.02 * 32.0))),
    # M tiles that do not divide the chip's CTA pairs: the pairs left over sweep all M tiles over a tail of the vocabulary
    ("proxy_tree", dict(B=20, V=40011, d=256)),                                  # 5 M tiles: 14 ranges + 4 tail pairs
    ("llama_tree", dict(B=31, V=21000, d=128)),                                  # 8 M tiles (the last one ragged): 9 + 2
    ("target_escalated", dict(B=40, n_active=37, V=3000, d=64)),                 # 10 M tiles picked by seq_index: 7 + 4
    # one active sequence: the kernel with W on the M side and the tree's nodes as columns
    ("proxy_tree", dict(B=1, V=40011, d=512)),                                   # 61 nodes: two column chunks
    ("llama_tree", dict(B=1, V=9000, d=256)),                                    # 49 nodes
    ("target_escalated", dict(B=4, n_active=1, V=7000, d=320)),                  # the one sequence is picked by seq_index
    ("tiny_chain", dict(k=15, V=3000, d=128)),                                   # 16 nodes: exactly one 16-column block
    ("tiny_chain", dict(k=31, V=200, d=64)),                                     # 32 nodes, fewer vocabulary units than SMs
    ("proxy_tree", dict(B=1, V=151936 // 8, d=192)),                             # ranges of 128 + 16 rows: the low second box
    ("llama_tree", dict(B=1, V=128256 // 8 + 4, d=256)),                         # vocabulary not a multiple of 8: the 2-D view of W
]


@pytest.mark.parametrize("name,over", LM_CASES)
def test_lmhead_stats_against_oracle(H, name, over):
    over = dict(over)
    if "logit_scale" not in over:
        over["logit_scale"] = 3.6 / (0.02 * math.sqrt(over["d"]))
    cfg = gen.small_variant(gen.CONFIGS[name], rho=0.2, **over)
    inp = gen.make_inputs(cfg, with_attention=False)
    dev = H.to_device(inp)
    got = H.run_lmhead(dev, cfg)
    seqs = list(range(cfg.B)) if inp["seq_index"] is None else [int(s) for s in inp["seq_index"]]
    ref = orc.lmhead_stats(inp["h"], inp["W"], inp["parent"], inp["tok"], cfg.logit_scale, seqs=seqs)
    n_tie = H.check_stats(got, ref, seqs, cfg.T)
    assert n_tie <= 0.02 * len(seqs) * cfg.T + 2
    # rows of sequences that were not asked for stay untouched
    for b in range(cfg.B):
        if b not in seqs:
            assert np.isnan(got["lse"][b]).all() and (got["top1_idx"][b] == -1).all()


def test_lmhead_tiny_vocab_and_argument_errors(H):
    import torch
    from paper_2601_23180_b200 import binding as ts
    # V = 19 (one 32-wide tile with 13 masked columns), duplicated maximum -> margin exactly 0
    cfg = gen.small_variant(gen.CONFIGS["tiny_chain"], V=19, d=64, logit_scale=2.0)
    inp = gen.make_inputs(cfg, with_attention=False)
    inp["W"][7] = inp["W"][3]
    dev = H.to_device(inp)
    got = H.run_lmhead(dev, cfg)
    ref = orc.lmhead_stats(inp["h"], inp["W"], inp["parent"], inp["tok"], cfg.logit_scale)
    for r in range(cfg.T):
        assert abs(got["lse"][0, r] - ref["lse"][0, r]) < 1e-3
        if ref["top1_idx"][0, r] == 3:
            assert got["top1_idx"][0, r] == 3 and got["top2_idx"][0, r] == 7
            assert got["p_top1"][0, r] == got["p_top2"][0, r]
    # argument errors are reported before any launch
    st = ts.alloc_stats(cfg.B, cfg.T)
    a = ts.lmhead_args(dev["h"], dev["W"], dev["parent"], dev["tok"], cfg.logit_scale, st)
    n0 = ts.launch_count()
    with pytest.raises(ts.TrispecError) as e:
        ts.trispec_lmhead_stats(a)            # no workspace
    assert e.value.code == 1 and ts.launch_count() == n0
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    a.workspace, a.workspace_bytes = ws.data_ptr(), 256
    with pytest.raises(ts.TrispecError) as e:
        ts.trispec_lmhead_stats(a)            # workspace too small
    assert e.value.code == 3 and ts.launch_count() == n0


# ------------------------------------------------------------------------------ attention
ATTN_CASES = [
    # (name, overrides, ctx_len override)
    ("tiny_chain", dict(), None),                                              # config 1 at full size
    ("proxy_tree", dict(B=3, L=1000), None),                                   # ragged last tile
    ("proxy_tree", dict(B=1, L=4096), None),                                   # several KV splits
    ("target_escalated", dict(B=4, n_active=2, L=700), None),                  # G = 8: 4 M tiles, subset
    ("llama_tree", dict(B=2, L=520), None),                                    # G = 4, T = 49
    ("long_paged", dict(B=5, L=2100, L_min=70), None),                         # paged, ragged
    ("long_paged", dict(B=4, L=300, L_min=1), [0, 1, 64, 65]),                 # empty / one-key contexts
    ("proxy_tree", dict(B=2, L=64, Hq=8, Hkv=8), [64, 0]),                     # G = 1 (MHA)
    ("proxy_tree", dict(B=1, L=9300, Hq=4, Hkv=2), None),                      # > 8 KV splits: workspace merge
    ("long_paged", dict(B=3, L=5000, L_min=5000, Hq=4, Hkv=2), [5000, 40, 2300]),  # 8-CTA clusters with idle splits
    # cluster sizes that do not divide 128: uneven row shares in the merge
    ("tiny_chain", dict(B=1, L=900, Hq=4, Hkv=2), None),                       # 3 splits
    ("tiny_chain", dict(B=1, L=1300, Hq=4, Hkv=2), None),                      # 5 splits
    ("tiny_chain", dict(B=6, L=1800, Hq=16, Hkv=8), None),                     # 6 splits
    ("proxy_tree", dict(B=1, L=1800, Hq=4, Hkv=2), None),                      # 7 splits, T = 61
    ("tiny_chain", dict(B=5, L=2500, Hq=16, Hkv=8), [2500, 1000, 64, 2499, 7]),  # 7 splits, ragged
]


@pytest.mark.parametrize("name,over,ctx", ATTN_CASES)
def test_attention_against_oracle(H, name, over, ctx):
    cfg = gen.small_variant(gen.CONFIGS[name], **over)
    inp = gen.make_inputs(cfg, with_lm_head=False)
    if ctx is not None:
        inp["ctx_len"] = np.array(ctx, dtype=np.int32)
    dev = H.to_device(inp)
    mask_dev, _ = H.run_tree_mask(dev["parent"])
    o, lse = H.run_attn(dev, cfg, mask_dev)
    seqs = list(range(cfg.B)) if inp["seq_index"] is None else [int(s) for s in inp["seq_index"]]
    ref_mask, _ = orc.build_tree_mask(inp["parent"])
    ref_o, ref_lse = orc.verify_attn(inp["q"], inp["k_tree"], inp["v_tree"], ref_mask, inp["k_cache"],
                                     inp["v_cache"], inp["ctx_len"], 1.0 / math.sqrt(cfg.D),
                                     block_table=inp["block_table"], block_size=cfg.block_size, seqs=seqs)
    for b in range(cfg.B):
        if b in seqs:
            err = np.abs(o[b] - ref_o[b]).max()
            assert err <= 2e-2, (b, err)                      # bf16 in, fp32 accumulate, bf16 out
            assert np.abs(lse[b] - ref_lse[b]).max() <= 1e-3 * max(1.0, np.abs(ref_lse[b]).max())
        else:
            assert np.isnan(o[b]).all()                       # untouched


PIECES_CASES = [c for c in ATTN_CASES if c[0] != "tiny_chain" or c[1]] + [
    ("long_paged", dict(B=9, L=3000, L_min=200), None),                        # ragged lengths: pieces of very different items
    ("target_escalated", dict(B=5, n_active=3, L=1500), None),                 # 4 M tiles: groups of four CTAs share K/V
    ("proxy_tree", dict(B=130, L=64), None),                                   # more than 128 sequences: falls back to the split plan
]


@pytest.mark.parametrize("name,over,ctx", PIECES_CASES)
def test_attention_persistent_kernel_against_oracle(H, monkeypatch, name, over, ctx):
    """The persistent kernel (balanced pieces, partials merged by a second kernel), forced through the
    planner's override, on the cases of the split kernels and a few of its own."""
    monkeypatch.setenv("TRISPEC_ATTN_PLAN", "pieces")
    test_attention_against_oracle(H, name, over, ctx)


def test_attention_argument_errors(H):
    import torch
    from paper_2601_23180_b200 import binding as ts
    # one sequence with a long context is cut into more than 8 KV splits, which are merged
    # through a caller-provided workspace
    cfg = gen.small_variant(gen.CONFIGS["tiny_chain"], L=9300, Hq=2, Hkv=2)
    inp = gen.make_inputs(cfg, with_lm_head=False)
    dev = H.to_device(inp)
    mask_dev, _ = H.run_tree_mask(dev["parent"])
    o = torch.zeros((cfg.B, cfg.T, cfg.Hq, cfg.D), dtype=torch.bfloat16, device="cuda")
    a = ts.attn_args(dev["q"], dev["k_tree"], dev["v_tree"], mask_dev, dev["k_cache"], dev["v_cache"],
                     dev["ctx_len"], 0.1, o)
    assert ts.trispec_verify_attn_workspace(a) > 0
    n0 = ts.launch_count()
    with pytest.raises(ts.TrispecError) as e:
        ts.trispec_verify_attn(a)                              # no workspace
    assert e.value.code == 1
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    a.workspace, a.workspace_bytes = ws.data_ptr(), 256
    with pytest.raises(ts.TrispecError) as e:
        ts.trispec_verify_attn(a)                              # workspace too small
    assert e.value.code == 3 and ts.launch_count() == n0
    a.D = 64
    with pytest.raises(ts.TrispecError) as e:
        ts.trispec_verify_attn(a)                              # unsupported head dim
    assert e.value.code == 2 and ts.launch_count() == n0


# ------------------------------------------------------------------------------ the whole pass
def _check_pass(H, cfg, inp, got, ref, seqs):
    assert got["status"] == 0
    assert np.array_equal(got["mask"].view(np.uint64), ref["mask"])
    assert np.array_equal(got["depth"], ref["depth"])
    if "o" in ref:
        for b in seqs:
            assert np.abs(got["o"][b] - ref["o"][b]).max() <= 2e-2
    H.check_stats(got["stats"], ref["stats"], seqs, cfg.T)
    # decisions: bit-exact except sequences whose walk meets a margin within 1e-3 of lambda
    # (PROXY) or a top-1/top-2 logit gap below 1e-3 relative (TARGET); those are counted
    st = ref["stats"]
    gap = st["top1_val"] - st["top2_val"]
    near_tie = gap < 1e-3 * np.maximum(1.0, np.abs(st["top1_val"]))
    n_skipped = 0
    for b in range(cfg.B):
        if b not in seqs:
            assert got["scan"]["accept_len"][b] == 0 and got["scan"]["last_node"][b] == -1
            continue
        visited = [0] + [int(x) for x in ref["scan"]["path"][b] if x >= 0]
        if ref["scan"]["near_thr"][b] > 0 or got["scan"]["near_thr"][b] > 0 or near_tie[b, visited].any():
            n_skipped += 1
            continue
        for k in ("accept_len", "escalate", "bonus_tok", "last_node"):
            assert got["scan"][k][b] == ref["scan"][k][b], (k, b)
        assert np.array_equal(got["scan"]["path"][b], ref["scan"]["path"][b])
    assert n_skipped <= max(1, len(seqs) // 4)
    return n_skipped


PASS_CASES = [
    ("tiny_chain", dict(V=4000, d=256)),
    ("proxy_tree", dict(B=4, L=500, V=20000, d=256, rho=0.3)),
    ("target_escalated", dict(B=5, n_active=2, L=300, V=6000, d=320, Hq=32, rho=0.3)),
    ("llama_tree", dict(B=3, L=260, V=9000, d=128, rho=0.3)),
    ("long_paged", dict(B=6, L=900, L_min=100, V=5000, d=192, rho=0.3)),
    # one active sequence: a short context (mask + attention beside the LM head on the library's second
    # stream; the sequence picked through seq_index) and a long one (LM head first, then the attention)
    ("target_escalated", dict(B=4, n_active=1, L=300, V=6000, d=320, Hq=32, rho=0.3)),
    ("proxy_tree", dict(B=1, L=4096, V=20000, d=256, rho=0.3)),
]


@pytest.mark.parametrize("name,over", PASS_CASES)
@pytest.mark.parametrize("host", [False, True])
def test_fused_verify_pass(H, name, over, host):
    from paper_2601_23180_b200 import runner
    import torch
    over = dict(over)
    over["logit_scale"] = 3.6 / (0.02 * math.sqrt(over["d"]))
    cfg = gen.small_variant(gen.CONFIGS[name], **over)
    inp = gen.make_inputs(cfg)
    pas = runner.VerifyPass(cfg, inp)
    if host:
        # per-round inputs come from pinned host memory; device copies start out as garbage
        hb = pas.prepare_host(inp)
        for k in ("q", "k_tree", "v_tree", "h"):
            pas.dev[k].zero_()
        pas.dev["parent"].fill_(-1)
        pas.dev["tok"].zero_()
        pas.run_host()
    else:
        pas.run()
    torch.cuda.synchronize()
    got = pas.results()
    seqs = pas.seqs
    ref = orc.verify(inp, 1.0 / math.sqrt(cfg.D), cfg.logit_scale, cfg.lam, mode=cfg.mode)
    _check_pass(H, cfg, inp, got, ref, seqs)
    if host:
        for k in ("accept_len", "bonus_tok", "last_node", "path", "escalate"):
            assert np.array_equal(hb[k].numpy(), got["scan"][k]), k
    # both routing outcomes must be exercised somewhere in PROXY mode
    if cfg.mode == gen.MODE_PROXY and cfg.B >= 4:
        assert 0 < ref["scan"]["escalate"][seqs].sum() < len(seqs) or cfg.B < 4


def test_run_to_run_determinism(H):
    from paper_2601_23180_b200 import runner
    import torch
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=3, L=700, V=30000, d=256, logit_scale=3.6 / 0.32)
    inp = gen.make_inputs(cfg)
    pas = runner.VerifyPass(cfg, inp)
    pas.run(); torch.cuda.synchronize()
    a = pas.results()
    pas.run(); torch.cuda.synchronize()
    b = pas.results()
    assert np.array_equal(a["o"], b["o"])
    for k in a["stats"]:
        assert np.array_equal(a["stats"][k], b["stats"][k], equal_nan=True)


# ------------------------------------------------------------------------------ size limits and degenerate shapes
EDGE_CASES = [
    # the largest tree the library takes (T = 64: mask bit 63, both halves of every warp full), a chain of
    # that length (depth 63), a single node (T = 1: the root alone), 16 query heads per KV head, MHA
    ("proxy_tree", dict(B=3, k=63, L=200, V=6000, d=128, rho=0.3)),
    ("tiny_chain", dict(B=2, k=63, max_depth=63, L=130, V=5000, d=128)),
    ("proxy_tree", dict(B=4, k=0, max_depth=0, L=100, V=4096, d=64)),
    ("proxy_tree", dict(B=2, k=20, L=300, Hq=16, Hkv=1, V=4000, d=128, rho=0.3)),
    ("proxy_tree", dict(B=2, k=60, L=70, Hq=4, Hkv=4, V=4000, d=128, rho=0.3)),
]


@pytest.mark.parametrize("name,over", EDGE_CASES)
def test_fused_pass_at_size_limits(H, name, over):
    over = dict(over)
    over.setdefault("logit_scale", 3.6 / (0.02 * math.sqrt(over["d"])))
    cfg = gen.small_variant(gen.CONFIGS[name], **over)
    inp = gen.make_inputs(cfg)
    from paper_2601_23180_b200 import runner
    import torch
    pas = runner.VerifyPass(cfg, inp)
    pas.run()
    torch.cuda.synchronize()
    got = pas.results()
    ref = orc.verify(inp, 1.0 / math.sqrt(cfg.D), cfg.logit_scale, cfg.lam, mode=cfg.mode)
    _check_pass(H, cfg, inp, got, ref, list(range(cfg.B)))
    assert got["mask"].view(np.uint64).max() == ref["mask"].max()


@pytest.mark.parametrize("plan", ["splits", "pieces"])
def test_attention_with_one_dominant_split_and_large_values(H, monkeypatch, plan):
    """Eight KV splits of one sequence, one of which holds every key that matters (scores about 20
    above the rest) while the values are eight times larger than usual: the splits' partials differ by
    e^20 in weight, which is where a partial kept in low precision, or merged with the wrong reference
    maximum, would show. The outputs reach several units here, where half a bf16 step of the result alone is
    1.6e-2: the bound is the usual 2e-2 plus one bf16 step (2^-8 relative) of the reference value."""
    monkeypatch.setenv("TRISPEC_ATTN_PLAN", plan)
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=1, L=2048, seed=23)
    inp = gen.make_inputs(cfg, with_lm_head=False)
    q = gen.bf16_bits_to_f32(inp["q"])
    k = gen.bf16_bits_to_f32(inp["k_cache"])
    q[..., 0] = 8.0                                           # every query row looks along dimension 0
    k[0, 768:1024, :, 0] = 28.25                              # keys of tiles 12-15 (split 3 of 8): +20 after scaling
    inp["q"], inp["k_cache"] = gen.f32_to_bf16_bits(q), gen.f32_to_bf16_bits(k)
    for name in ("v_cache", "v_tree"):
        inp[name] = gen.f32_to_bf16_bits(gen.bf16_bits_to_f32(inp[name]) * 8.0)
    dev = H.to_device(inp)
    mask_dev, _ = H.run_tree_mask(dev["parent"])
    o, lse = H.run_attn(dev, cfg, mask_dev)
    ref_mask, _ = orc.build_tree_mask(inp["parent"])
    ref_o, ref_lse = orc.verify_attn(inp["q"], inp["k_tree"], inp["v_tree"], ref_mask, inp["k_cache"], inp["v_cache"],
                                     inp["ctx_len"], 1.0 / math.sqrt(cfg.D))
    assert np.abs(ref_lse).min() > 18.0                       # the dominant split decides every row
    assert 0.3 < np.abs(ref_o).max() < 8.0
    assert (np.abs(o - ref_o) <= 2e-2 + np.abs(ref_o) / 256.0).all()
    small = np.abs(ref_o) < 1.0
    assert small.mean() > 0.3 and np.abs(o - ref_o)[small].max() <= 2e-2
    assert np.abs(lse - ref_lse).max() <= 1e-3 * np.abs(ref_lse).max()
