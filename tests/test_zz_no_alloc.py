"""The LM-head entry point for callers that cannot allocate device memory.

`trispec_lmhead_stats_noalloc` is for a decode loop that lives inside a serving engine whose
memory pool already owns all free device memory: there a cudaMalloc fails, or stalls every
stream while it runs, so the loop has no way to obtain the workspace that
`trispec_lmhead_stats` asks for. The variant keeps its partial statistics in a fixed 1 MiB
array inside the library instead. This file checks, through the C ABI, that it returns what
the workspace entry point returns and what the CPU oracle computes, on calls in a row with different inputs (the array
is shared and keeps the previous call's contents, which must not leak into the next result),
and that a problem too large for the array is refused before anything is launched.

The file is named so that pytest collects it after every other test file.
"""
import numpy as np
import pytest

from oracle import trispec_oracle as orc
from paper_2601_23180_b200 import inputs as gen

pytestmark = pytest.mark.gpu


def _run(ts, torch, dev, cfg, noalloc: bool):
    B, T = dev["parent"].shape
    st = ts.alloc_stats(B, T)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    a = ts.lmhead_args(dev["h"], dev["W"], dev["parent"], dev["tok"], cfg.logit_scale, st,
                       seq_index=dev.get("seq_index"), dev_status=status)
    if noalloc:
        ts.trispec_lmhead_stats_noalloc(a)                 # no workspace in the arguments
    else:
        ws = ts.alloc_workspace(ts.trispec_lmhead_stats_workspace(a))
        a.workspace, a.workspace_bytes = ws.data_ptr(), ws.numel()
        ts.trispec_lmhead_stats(a)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return {k: v.cpu().numpy() for k, v in st.items()}


def _same(got, ref, seqs, T):
    # Both entry points run the same kernels on the same inputs; the tolerances are the ones
    # the parity tests use for these statistics (1e-3 relative, indices exact).
    for b in seqs:
        for k in ("top1_idx", "top2_idx"):
            assert np.array_equal(got[k][b], ref[k][b]), (k, b)
        for k in ("max", "lse", "top1_val", "top2_val", "p_top1", "p_top2"):
            assert np.allclose(got[k][b], ref[k][b], rtol=1e-3, atol=1e-9), (k, b)
        for k in ("draft_logit", "p_draft"):
            assert np.isnan(got[k][b, 0]) and np.isnan(ref[k][b, 0])
            assert np.allclose(got[k][b, 1:T], ref[k][b, 1:T], rtol=1e-3, atol=1e-9), (k, b)


def test_noalloc_entry_matches_workspace_entry_twice_in_a_row():
    import torch
    import tests.gpu_helpers as H
    from paper_2601_23180_b200 import binding as ts
    cases = [
        gen.small_variant(gen.CONFIGS["proxy_tree"], B=5, L=64, V=20000, d=256, logit_scale=3.6 / (0.02 * 16.0)),
        # second call: other shapes, a sequence subset and another seed, so that anything left
        # in the shared array by the first call would show
        gen.small_variant(gen.CONFIGS["target_escalated"], B=6, n_active=3, L=64, V=9000, d=320, Hq=32, seed=7),
        # 64 sequences: the workspace entry point would plan more partial rows than the built-in array
        # holds (pairs that sweep every M tile); this entry point plans fewer of them and must still agree
        gen.small_variant(gen.CONFIGS["proxy_tree"], B=64, L=64, V=6000, d=64, logit_scale=3.6 / (0.02 * 8.0), seed=9),
    ]
    for cfg in cases:
        inp = gen.make_inputs(cfg)
        dev = H.to_device(inp)
        seqs = list(range(cfg.B)) if inp.get("seq_index") is None else [int(s) for s in inp["seq_index"]]
        ref = _run(ts, torch, dev, cfg, noalloc=False)
        got = _run(ts, torch, dev, cfg, noalloc=True)
        _same(got, ref, seqs, cfg.T)
        # and against the CPU oracle, with the tolerances of the LM-head parity tests: agreement of the
        # two entry points alone would only show that they share their kernels
        want = orc.lmhead_stats(inp["h"], inp["W"], inp["parent"], inp["tok"], cfg.logit_scale, seqs=seqs)
        n_tie = H.check_stats(got, want, seqs, cfg.T)
        assert n_tie <= 0.02 * len(seqs) * cfg.T + 2


def test_noalloc_entry_refuses_what_does_not_fit():
    import torch
    from paper_2601_23180_b200 import binding as ts
    # 600 sequences need 150 M tiles x 8 KB of partials, more than the built-in 1 MiB
    B, T, d, V = 600, 61, 64, 4096
    z16 = lambda *s: torch.zeros(s, dtype=torch.bfloat16, device="cuda")
    z32 = lambda *s: torch.zeros(s, dtype=torch.int32, device="cuda")
    st = ts.alloc_stats(B, T)
    a = ts.lmhead_args(z16(B * T, d), z16(V, d), z32(B, T), z32(B, T), 1.0, st)
    assert ts.trispec_lmhead_stats_workspace(a) > ts.NOALLOC_SCRATCH_BYTES
    n0 = ts.launch_count()
    with pytest.raises(ts.TrispecError) as e:
        ts.trispec_lmhead_stats_noalloc(a)
    assert e.value.code == 8 and "built-in scratch" in str(e.value)
    assert ts.launch_count() == n0
