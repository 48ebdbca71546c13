"""GPU tests of what a decode loop relies on besides the arithmetic: calls of the library issued
back to back on one stream see each other's results (a KV commit, a pruning step or the scan's
escalation list feeding the next verification), and out-of-range lengths, dead rows of a pruned
tree and malformed trees are worked around and reported through the status word, never by a
fault. Everything here is a wrong-value check: no input makes a kernel leave its arrays."""
import math

import numpy as np
import pytest

from oracle import trispec_oracle as orc
from paper_2601_23180_b200 import inputs as gen

pytestmark = pytest.mark.gpu


def _attn_call(ts, torch, dev, cfg, mask_dev, o, lse, status, n_nodes=None, seq_index=None):
    a = ts.attn_args(dev["q"], dev["k_tree"], dev["v_tree"], mask_dev, dev["k_cache"], dev["v_cache"],
                     dev["ctx_len"], 1.0 / math.sqrt(cfg.D), o, block_table=dev.get("block_table"),
                     block_size=cfg.block_size, seq_index=seq_index, lse=lse, dev_status=status, n_nodes=n_nodes)
    ws = ts.alloc_workspace(ts.trispec_verify_attn_workspace(a))
    a.workspace, a.workspace_bytes = ws.data_ptr(), ws.numel()
    return a, ws


@pytest.mark.parametrize("paged", [False, True])
def test_commit_then_attention_on_one_stream_sees_the_new_cache(paged):
    """trispec_commit_kv (lengths updated in place) followed at once by trispec_verify_attn: the
    attention must run over the longer cache, including the rows the commit just wrote."""
    import torch
    import tests.gpu_helpers as H
    from paper_2601_23180_b200 import binding as ts
    name = "long_paged" if paged else "proxy_tree"
    cfg = gen.small_variant(gen.CONFIGS[name], B=6, L=1280, L_min=1280 if paged else None, seed=13)
    inp = gen.make_inputs(cfg, with_lm_head=False)
    B, T = cfg.B, cfg.T
    # lengths that end inside a 64-key tile and at a tile boundary; room for up to 7 appended rows
    inp["ctx_len"] = np.array([1000, 1023, 1024, 63, 0, 1200], dtype=np.int32)
    g = np.random.default_rng(2)
    path = np.full((B, T), -1, dtype=np.int32)
    acc = np.zeros(B, dtype=np.int32)
    for b in range(B):
        cur, n = 0, 0
        while n < 6:
            kids = np.nonzero(inp["parent"][b] == cur)[0]
            if not len(kids):
                break
            cur = int(g.choice(kids))
            path[b, n] = cur
            n += 1
        acc[b] = n
    dev = H.to_device(inp)
    mask_dev, _ = H.run_tree_mask(dev["parent"])
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    o = torch.full((B, T, cfg.Hq, cfg.D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, cfg.Hq, T), float("nan"), dtype=torch.float32, device="cuda")
    ca = ts.commit_args(dev["k_tree"], dev["v_tree"], dev["k_cache"], dev["v_cache"], dev["ctx_len"], H.i32_dev(path),
                        H.i32_dev(acc), dev["ctx_len"], block_table=dev.get("block_table"),
                        block_size=cfg.block_size, dev_status=status)
    aa, ws = _attn_call(ts, torch, dev, cfg, mask_dev, o, lse, status)
    torch.cuda.synchronize()
    for _ in range(2):                     # the second round commits on top of the first
        ts.trispec_commit_kv(ca)
        ts.trispec_verify_attn(aa)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    kc, vc, ln = inp["k_cache"], inp["v_cache"], inp["ctx_len"]
    for _ in range(2):
        kc, vc, ln = orc.commit_kv(kc, vc, ln, inp["k_tree"], inp["v_tree"], path, acc,
                                   block_table=inp.get("block_table"), block_size=cfg.block_size)
    assert np.array_equal(dev["ctx_len"].cpu().numpy(), ln) and (ln > inp["ctx_len"]).all()
    ref_mask, _ = orc.build_tree_mask(inp["parent"])
    ref_o, ref_lse = orc.verify_attn(inp["q"], inp["k_tree"], inp["v_tree"], ref_mask, kc, vc, ln,
                                     1.0 / math.sqrt(cfg.D), block_table=inp.get("block_table"),
                                     block_size=cfg.block_size)
    got_o, got_lse = o.float().cpu().numpy(), lse.cpu().numpy()
    assert np.abs(got_o - ref_o).max() <= 2e-2
    assert np.abs(got_lse - ref_lse).max() <= 1e-3 * max(1.0, np.abs(ref_lse).max())
    # the appended rows matter: attention over the old lengths differs visibly for the short sequences
    old_o, _ = orc.verify_attn(inp["q"], inp["k_tree"], inp["v_tree"], ref_mask, inp["k_cache"], inp["v_cache"],
                               inp["ctx_len"], 1.0 / math.sqrt(cfg.D), block_table=inp.get("block_table"),
                               block_size=cfg.block_size, seqs=[3, 4])
    assert np.abs(old_o[4] - ref_o[4]).max() > 0.1


def test_prune_then_attention_on_one_stream_uses_the_new_node_counts():
    """trispec_prune_tree followed at once by trispec_verify_attn with n_nodes = its n_keep and the
    pruned mask: rows of the pruned tree equal the oracle's, the rest is never written."""
    import torch
    import tests.gpu_helpers as H
    from paper_2601_23180_b200 import binding as ts
    cfg = gen.small_variant(gen.CONFIGS["target_escalated"], B=5, n_active=None, L=700, seed=14)
    inp = gen.make_inputs(cfg, with_lm_head=False)
    B, T = cfg.B, cfg.T
    dev = H.to_device(inp)
    mask_dev, _ = H.run_tree_mask(dev["parent"])
    root = np.array([0, 1, 2, -1, 5], dtype=np.int32)
    ref_p = orc.prune_tree(inp["parent"], inp["tok"], root)
    # the caller gathers the per-node activations of the kept nodes (node_map) before the target pass;
    # here the gather is done on the host from the oracle's map, the counts and masks come from the GPU
    for k in ("q", "k_tree", "v_tree"):
        new = np.zeros_like(inp[k])
        for b in range(B):
            n = int(ref_p["n_keep"][b])
            new[b, :n] = inp[k][b, ref_p["node_map"][b, :n]]
        inp[k] = new
        dev[k] = H.bf16_dev(new)
    pout = ts.alloc_prune_out(B, T)
    pout["n_keep"].fill_(T)                       # stale counts: a premature read would compute every row
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    o = torch.full((B, T, cfg.Hq, cfg.D), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, cfg.Hq, T), float("nan"), dtype=torch.float32, device="cuda")
    pa = ts.prune_args(dev["parent"], H.i32_dev(inp["tok"]), mask_dev, H.i32_dev(root), pout)
    aa, ws = _attn_call(ts, torch, dev, cfg, pout["mask"], o, lse, status, n_nodes=pout["n_keep"])
    torch.cuda.synchronize()
    ts.trispec_prune_tree(pa)
    ts.trispec_verify_attn(aa)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(pout["n_keep"].cpu().numpy(), ref_p["n_keep"])
    got_o = o.float().cpu().numpy()
    for b in range(B):
        n = int(ref_p["n_keep"][b])
        if n:
            m, _ = orc.build_tree_mask(ref_p["parent"][b:b + 1, :n])
            sub = {k: inp[k][b:b + 1, :n] for k in ("q", "k_tree", "v_tree")}
            ro, _ = orc.verify_attn(sub["q"], sub["k_tree"], sub["v_tree"], m, inp["k_cache"][b:b + 1],
                                    inp["v_cache"][b:b + 1], inp["ctx_len"][b:b + 1], 1.0 / math.sqrt(cfg.D))
            assert np.abs(got_o[b, :n] - ro[0]).max() <= 2e-2, b
        assert np.isnan(got_o[b, n:]).all(), b


def test_escalation_list_of_a_proxy_round_drives_the_target_round_on_one_stream():
    """Proxy pass, then at once a target pass whose seq_index is the proxy scan's esc_index buffer
    (first n entries valid): the target pass must verify exactly the escalated sequences."""
    import torch
    import tests.gpu_helpers as H
    from paper_2601_23180_b200 import binding as ts
    from paper_2601_23180_b200 import runner
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=8, L=200, V=6000, d=128, rho=0.3,
                            logit_scale=3.6 / (0.02 * math.sqrt(128)), seed=15)
    inp = gen.make_inputs(cfg)
    ref = orc.verify(inp, 1.0 / math.sqrt(cfg.D), cfg.logit_scale, cfg.lam, mode=orc.MODE_PROXY)
    esc = [int(b) for b in np.nonzero(ref["scan"]["escalate"])[0]]
    assert 0 < len(esc) < cfg.B and (ref["scan"]["near_thr"] == 0).all()
    pas = runner.VerifyPass(cfg, inp)
    # the target round: same tensors (a stand-in for the target model's), its own outputs
    B, T = cfg.B, cfg.T
    st2 = ts.alloc_stats(B, T)
    so2 = ts.alloc_scan_out(B, T)
    esc_buf = pas.scan_out["esc_index"]
    esc_buf.copy_(torch.arange(B - 1, -1, -1, dtype=torch.int32, device="cuda"))   # stale: the reverse order
    la = ts.lmhead_args(pas.dev["h"], pas.dev["W"], pas.dev["parent"], pas.dev["tok"], cfg.logit_scale, st2,
                        seq_index=esc_buf[:len(esc)], dev_status=pas.status)
    ws = ts.alloc_workspace(ts.trispec_lmhead_stats_workspace(la))
    la.workspace, la.workspace_bytes = ws.data_ptr(), ws.numel()
    torch.cuda.synchronize()
    pas.run()
    ts.trispec_lmhead_stats(la)
    torch.cuda.synchronize()
    assert int(pas.status.item()) == 0
    assert pas.scan_out["esc_index"].cpu().numpy()[:len(esc)].tolist() == esc
    got = {k: v.cpu().numpy() for k, v in st2.items()}
    H.check_stats(got, ref["stats"], esc, T)
    for b in range(B):
        if b not in esc:
            assert np.isnan(got["lse"][b]).all()        # not verified by the target round


def test_oversize_context_length_is_clamped_and_flagged():
    """ctx_len beyond the capacity (a stale or corrupt entry): the kernel attends over the capacity,
    never past the block-table row or the cache, and reports TRISPEC_ERR_BAD_LENGTH (10)."""
    import torch
    import tests.gpu_helpers as H
    for paged in (False, True):
        name = "long_paged" if paged else "proxy_tree"
        cfg = gen.small_variant(gen.CONFIGS[name], B=3, L=640, L_min=640 if paged else None, seed=16)
        inp = gen.make_inputs(cfg, with_lm_head=False)
        good = inp["ctx_len"].copy()
        assert (good == 640).all()
        bad = good.copy()
        bad[1] = 640 + 1000                          # past the capacity of 640
        bad[2] = -5                                  # negative: read as 0
        dev = H.to_device(dict(inp, ctx_len=bad))
        mask_dev, _ = H.run_tree_mask(dev["parent"])
        o, lse = H.run_attn(dev, cfg, mask_dev, expect_status=10)
        ref_mask, _ = orc.build_tree_mask(inp["parent"])
        clamped = np.array([640, 640, 0], dtype=np.int32)
        ref_o, ref_lse = orc.verify_attn(inp["q"], inp["k_tree"], inp["v_tree"], ref_mask, inp["k_cache"],
                                         inp["v_cache"], clamped, 1.0 / math.sqrt(cfg.D),
                                         block_table=inp.get("block_table"), block_size=cfg.block_size)
        assert np.abs(o - ref_o).max() <= 2e-2
        assert np.abs(lse - ref_lse).max() <= 1e-3 * max(1.0, np.abs(ref_lse).max())


def test_dead_rows_of_a_pruned_tree_may_hold_nan():
    """With n_nodes the rows of q, k_tree and v_tree past a sequence's count are never used: NaN bit
    patterns there (an uninitialised gather buffer) must not reach any output row."""
    import tests.gpu_helpers as H
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=3, L=300, seed=17)
    inp = gen.make_inputs(cfg, with_lm_head=False)
    n_nodes = np.array([61, 20, 1], dtype=np.int32)
    poisoned = dict(inp)
    for k in ("q", "k_tree", "v_tree"):
        a = inp[k].copy()
        for b in range(cfg.B):
            a[b, n_nodes[b]:] = 0x7FC0              # bf16 quiet NaN
        poisoned[k] = a
    dev = H.to_device(poisoned)
    mask_dev, _ = H.run_tree_mask(dev["parent"])
    o, lse = H.run_attn(dev, cfg, mask_dev, n_nodes=n_nodes)
    ref_mask, _ = orc.build_tree_mask(inp["parent"])
    ref_o, ref_lse = orc.verify_attn(inp["q"], inp["k_tree"], inp["v_tree"], ref_mask, inp["k_cache"], inp["v_cache"],
                                     inp["ctx_len"], 1.0 / math.sqrt(cfg.D))
    for b in range(cfg.B):
        n = int(n_nodes[b])
        assert np.isfinite(o[b, :n]).all(), b
        assert np.abs(o[b, :n] - ref_o[b, :n]).max() <= 2e-2, b
        assert np.abs(lse[b, :, :n] - ref_lse[b, :, :n]).max() <= 1e-3 * max(1.0, np.abs(ref_lse[b, :, :n]).max())
        assert np.isnan(o[b, n:]).all()


def test_malformed_tree_is_reported_through_the_status_word():
    """Both mask kernels (warp per sequence, thread per sequence) report a parent array that is not a
    tree as TRISPEC_ERR_BAD_TREE (11); a well-formed batch leaves the status word at zero. The fused
    pass hands the same word to the mask step, so its caller learns of the tree after the pass."""
    import torch
    import tests.gpu_helpers as H
    from paper_2601_23180_b200 import runner
    cfg = gen.CONFIGS["proxy_tree"]
    for B in (5, 2048 + 3):
        parent = np.stack([gen.make_tree(cfg, b % 7) for b in range(B)])
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        H.run_tree_mask(H.i32_dev(parent), status)
        assert int(status.item()) == 0
        for bad_row, node, value in ((B - 1, 7, 9), (2, 5, -3), (0, 0, 0), (1, 9, -1)):
            p2 = parent.copy()
            p2[bad_row, node] = value                # after the child / below -1 / a rooted root / a second root
            status.zero_()
            H.run_tree_mask(H.i32_dev(p2), status)
            assert int(status.item()) == 11, (B, bad_row, node, value)
    scfg = gen.small_variant(cfg, B=3, L=100, V=4000, d=64, logit_scale=3.6 / (0.02 * 8.0))
    inp = gen.make_inputs(scfg)
    inp["parent"][1, 4] = 30
    pas = runner.VerifyPass(scfg, inp)
    pas.run()
    torch.cuda.synchronize()
    assert int(pas.status.item()) == 11


def test_host_pass_rejects_argument_structs_of_different_passes():
    import torch
    from paper_2601_23180_b200 import binding as ts
    from paper_2601_23180_b200 import runner
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=2, L=64, V=4000, d=64, logit_scale=3.6 / (0.02 * 8.0))
    inp = gen.make_inputs(cfg)
    pas = runner.VerifyPass(cfg, inp)
    pas.prepare_host(inp)
    other = pas.dev["parent"].clone()
    keep = pas.scan_args.parent
    pas.scan_args.parent = other.data_ptr()
    n0 = ts.launch_count()
    with pytest.raises(ts.TrispecError) as e:
        pas.run_host()
    assert e.value.code == 1 and ts.launch_count() == n0
    pas.scan_args.parent = keep
    pas.run_host()
    torch.cuda.synchronize()
    assert int(pas.status.item()) == 0


def test_single_sequence_pass_with_its_attention_on_the_second_stream_stays_one_ordered_unit():
    """One active sequence with a short context: the fused pass runs mask + attention on the library's
    second stream beside the LM head. Inputs written on the caller's stream just before the call must be
    seen by both sides, and work enqueued on that stream right after the call must see every output."""
    import torch
    from paper_2601_23180_b200 import binding as ts, runner
    cfg = gen.small_variant(gen.CONFIGS["tiny_chain"], V=4096, d=256, L=700, seed=31,
                            logit_scale=3.6 / (0.02 * math.sqrt(256)))
    inp = gen.make_inputs(cfg)
    pas = runner.VerifyPass(cfg, inp)
    assert ts.trispec_verify_attn_plan(pas.attn_args) in ("cluster", "splits")
    # reference: the four steps one after the other, synchronised
    ts.trispec_build_tree_mask(pas.tree_args)
    ts.trispec_verify_attn(pas.attn_args)
    ts.trispec_lmhead_stats(pas.lm_args)
    ts.trispec_accept_scan(pas.scan_args)
    torch.cuda.synchronize()
    want = {"o": pas.o.clone(), "mask": pas.mask.clone(), "top1": pas.stats["top1_idx"].clone(),
            "lse": pas.stats["lse"].clone(), "acc": pas.scan_out["accept_len"].clone(),
            "path": pas.scan_out["path"].clone()}
    ref_o, _ = orc.verify_attn(inp["q"], inp["k_tree"], inp["v_tree"], orc.build_tree_mask(inp["parent"])[0],
                               inp["k_cache"], inp["v_cache"], inp["ctx_len"], 1.0 / math.sqrt(cfg.D))
    assert np.abs(want["o"].float().cpu().numpy() - ref_o).max() <= 2e-2
    q_good, h_good, parent_good = pas.dev["q"].clone(), pas.dev["h"].clone(), pas.dev["parent"].clone()
    side = torch.cuda.Stream()
    for rep in range(20):
        with torch.cuda.stream(side):
            # spoil the inputs and the outputs, then restore the inputs on the same stream right before the call
            pas.dev["q"].zero_(); pas.dev["h"].zero_(); pas.dev["parent"].fill_(-1)
            pas.o.fill_(float("nan")); pas.mask.zero_(); pas.stats["top1_idx"].fill_(-7)
            pas.scan_out["accept_len"].fill_(-9)
            big = torch.empty(64 << 20, dtype=torch.uint8, device="cuda"); big.zero_()   # keeps the stream busy
            pas.dev["q"].copy_(q_good); pas.dev["h"].copy_(h_good); pas.dev["parent"].copy_(parent_good)
            pas.run(side)
            got = {"o": pas.o.clone(), "mask": pas.mask.clone(), "top1": pas.stats["top1_idx"].clone(),
                   "lse": pas.stats["lse"].clone(), "acc": pas.scan_out["accept_len"].clone(),
                   "path": pas.scan_out["path"].clone()}
        side.synchronize()
        for k in want:
            a, b = got[k], want[k]
            if a.dtype.is_floating_point:
                assert torch.equal(torch.nan_to_num(a.float(), nan=-1.0), torch.nan_to_num(b.float(), nan=-1.0)), (k, rep)
            else:
                assert torch.equal(a, b), (k, rep)
    assert int(pas.status.item()) == 0
