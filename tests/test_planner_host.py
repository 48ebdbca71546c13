"""Host-side planning that can be observed without a GPU: the workspace queries.

`trispec_verify_attn_workspace` returns 0 when the KV splits of a sequence are merged inside a thread-block
cluster, and the size of the fp32 partials when plain CTAs and the merge kernel are used instead;
`trispec_lmhead_stats_workspace` shows which LM-head kernel a call takes. Without a device the planners
assume 148 SMs."""
from paper_2601_23180_b200 import binding as ts
from paper_2601_23180_b200 import inputs as gen


def _attn_args(cfg, n_active=None):
    a = ts.AttnArgs()
    a.B, a.T, a.Hq, a.Hkv, a.D, a.scale = cfg.B, cfg.T, cfg.Hq, cfg.Hkv, cfg.D, 1.0
    a.kv_layout, a.Lmax = ts.KV_CONTIGUOUS, cfg.L
    a.B_active = 0 if n_active is None else n_active
    a.seq_index = None if n_active is None else 1     # any non-null value: only its presence is looked at
    return a


def test_attention_workspace_follows_the_split_plan():
    # proxy_tree: 64 (sequence, KV head) items x 4 splits in clusters: merged on chip, no workspace
    assert ts.trispec_verify_attn_workspace(_attn_args(gen.CONFIGS["proxy_tree"])) == 0
    # llama_tree: 256 items, no split
    assert ts.trispec_verify_attn_workspace(_attn_args(gen.CONFIGS["llama_tree"])) == 0
    # target_escalated: 3 active sequences x 8 KV heads x 4 M tiles = 96 items; 4 clustered splits would be 384
    # CTAs (two waves), 3 plain splits are 288 CTAs (one wave of the 296 slots): partials go to the workspace
    cfg = gen.CONFIGS["target_escalated"]
    ws = ts.trispec_verify_attn_workspace(_attn_args(cfg, n_active=3))
    assert ws == 96 * 3 * 128 * (128 + 2) * 4
    # one sequence with a very long context: more than 8 splits, workspace as well
    long1 = gen.small_variant(gen.CONFIGS["proxy_tree"], B=1, L=65536, Hq=4, Hkv=2)
    assert ts.trispec_verify_attn_workspace(_attn_args(long1)) > 0
    # long_paged: 512 (sequence, head) items of up to 513 steps would fill two waves of 296 slots to 86 %:
    # the persistent kernel takes it, two partial slots for each of its 296 CTAs
    cfg = gen.CONFIGS["long_paged"]
    a = _attn_args(cfg)
    a.kv_layout, a.block_size, a.max_blocks_per_seq, a.num_blocks = ts.KV_PAGED, 64, cfg.L // 64, 1000
    assert ts.trispec_verify_attn_workspace(a) == 2 * 296 * 128 * (128 + 2) * 4
    assert ts.trispec_verify_attn_plan(a) == "pieces"
    assert ts.trispec_verify_attn_plan(_attn_args(gen.CONFIGS["proxy_tree"])) == "cluster"
    assert ts.trispec_verify_attn_plan(_attn_args(gen.CONFIGS["target_escalated"], n_active=3)) == "splits"


def test_lmhead_workspace_shows_the_kernel_choice():
    def args(B, T, d, V, n_active=None):
        a = ts.LmheadArgs()
        a.B, a.T, a.d, a.V, a.logit_scale = B, T, d, V, 1.0
        a.B_active = 0 if n_active is None else n_active
        a.seq_index = None if n_active is None else 1
        return a
    # batches: CTA pairs, 74 // n_mt vocabulary ranges x n_mt M tiles x 256 rows x 32 bytes
    assert ts.trispec_lmhead_stats_workspace(args(8, 61, 2048, 151936)) == 37 * 2 * 256 * 32
    # 16 M tiles leave 10 of the 74 pairs over: they become tail pairs (one more block of partial rows each)
    assert ts.trispec_lmhead_stats_workspace(args(64, 61, 2048, 151936)) == (4 + 10) * 16 * 256 * 32
    assert ts.trispec_lmhead_stats_workspace(args(32, 61, 2048, 151936)) == (9 + 2) * 8 * 256 * 32
    # no tail where it would not shorten the longest pair (llama_tree: 28 tiles either way)
    assert ts.trispec_lmhead_stats_workspace(args(16, 49, 4096, 128256)) == 18 * 4 * 256 * 32
    # one active sequence: one range per SM x 64 rows x 32 bytes
    assert ts.trispec_lmhead_stats_workspace(args(1, 9, 2048, 32000)) == 148 * 64 * 32
    assert ts.trispec_lmhead_stats_workspace(args(8, 61, 5120, 151936, n_active=1)) == 148 * 64 * 32
    # fewer 16-row vocabulary units than SMs
    assert ts.trispec_lmhead_stats_workspace(args(1, 9, 64, 200)) == 13 * 64 * 32
    # unsupported shapes plan nothing
    assert ts.trispec_lmhead_stats_workspace(args(1, 65, 2048, 32000)) == 0


def test_pass_form_follows_the_active_sequences_and_the_size_of_the_attention():
    def lm_args(B, n_active=None):
        a = ts.LmheadArgs()
        a.B, a.T, a.d, a.V, a.logit_scale = B, 61, 2048, 151936, 1.0
        a.B_active = 0 if n_active is None else n_active
        a.seq_index = None if n_active is None else 1
        return a
    one = gen.small_variant
    # batches: attention, then LM head
    assert ts.trispec_verify_plan(_attn_args(gen.CONFIGS["proxy_tree"]), lm_args(8)) == "attention_first"
    assert ts.trispec_verify_plan(None, lm_args(1)) == "attention_first"
    # one sequence, 512 context tokens: 8 KV heads x 2 splits = 16 CTAs: the LM head can spare their SMs
    assert ts.trispec_verify_plan(_attn_args(gen.CONFIGS["tiny_chain"]), lm_args(1)) == "side_by_side"
    # one sequence, 4096 context tokens: 64 CTAs would cost the LM head (151936 x 2048 weights) too many SMs
    assert ts.trispec_verify_plan(_attn_args(one(gen.CONFIGS["proxy_tree"], B=1)), lm_args(1)) == "lm_first"
    # one ACTIVE sequence of several, picked through an index list
    a = _attn_args(one(gen.CONFIGS["tiny_chain"], B=4), n_active=1)
    assert ts.trispec_verify_plan(a, lm_args(4, n_active=1)) == "side_by_side"
    # ... unless the scan writes its escalation list over that index list: then in stream order
    s = ts.ScanArgs()
    s.esc_index = 1
    assert ts.trispec_verify_plan(a, lm_args(4, n_active=1), s) == "lm_first"
    s.esc_index = 2
    assert ts.trispec_verify_plan(a, lm_args(4, n_active=1), s) == "side_by_side"
