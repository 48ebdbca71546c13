"""The C-ABI library builds, loads without a GPU and exports every function the header declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "trispec.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(trispec_[a-z_]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    from paper_2601_23180_b200 import build
    lib_path = build.build()
    lib = ctypes.CDLL(lib_path)
    names = _declared()
    assert {"trispec_build_tree_mask", "trispec_verify_attn", "trispec_lmhead_stats", "trispec_accept_scan",
            "trispec_verify", "trispec_verify_host"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/trispec.h but not exported"
    lib.trispec_status_string.restype = ctypes.c_char_p
    assert lib.trispec_status_string(0) == b"ok"
    assert lib.trispec_status_string(3) == b"workspace too small"


def test_binding_names_match_header():
    from paper_2601_23180_b200 import build
    build.build()
    from paper_2601_23180_b200 import binding
    for n in _declared():
        assert n in binding.EXPORTS
        assert hasattr(binding, n) or n in ("trispec_status_string", "trispec_launch_count")


def test_host_side_argument_validation_without_gpu():
    """Argument errors are found on the host before any CUDA call."""
    from paper_2601_23180_b200 import build
    lib = ctypes.CDLL(build.build())
    from paper_2601_23180_b200 import binding as ts
    assert lib.trispec_build_tree_mask(None, None) == 1
    t = ts.TreeArgs(4, 65, 16, 16, None)
    assert lib.trispec_build_tree_mask(ctypes.byref(t), None) == 2      # T > 64
    a = ts.AttnArgs()
    a.B, a.T, a.Hq, a.Hkv, a.D = 2, 9, 16, 8, 64
    assert lib.trispec_verify_attn(ctypes.byref(a), None) == 2          # head dim
    a.D, a.Hq = 128, 24
    assert lib.trispec_verify_attn(ctypes.byref(a), None) == 2          # group size 3
    s = ts.ScanArgs()
    s.B, s.T = 3, 9
    assert lib.trispec_accept_scan(ctypes.byref(s), None) == 1          # null pointers
    l = ts.LmheadArgs()
    l.B, l.T, l.d, l.V = 1, 9, 100, 32000
    assert lib.trispec_lmhead_stats(ctypes.byref(l), None) == 2         # d % 64


def test_status_strings_and_host_pass_struct_check_without_gpu():
    """Every status code has its own text, and the host-buffer pass refuses argument structs that do
    not describe one pass (different parent / token buffers) before any CUDA call."""
    from paper_2601_23180_b200 import build
    lib = ctypes.CDLL(build.build())
    lib.trispec_status_string.restype = ctypes.c_char_p
    texts = [lib.trispec_status_string(c) for c in range(0, 12)]
    assert len(set(texts)) == 12 and b"unknown status" not in texts
    assert lib.trispec_status_string(99) == b"unknown status"
    from paper_2601_23180_b200 import binding as ts
    io, t, l, s = ts.HostIO(), ts.TreeArgs(), ts.LmheadArgs(), ts.ScanArgs()
    t.parent, l.parent, s.parent = 4096, 8192, 4096
    assert lib.trispec_verify_host(ctypes.byref(io), ctypes.byref(t), None, ctypes.byref(l), ctypes.byref(s), None) == 1
    l.parent = 4096
    l.tok, s.tok = 256, 512
    assert lib.trispec_verify_host(ctypes.byref(io), ctypes.byref(t), None, ctypes.byref(l), ctypes.byref(s), None) == 1
    # the scan refuses an unknown acceptance rule or a slack outside [0, 1] before anything is launched
    sc = ts.ScanArgs()
    sc.B, sc.T = 2, 9
    for f in ("parent", "tok", "accept_len", "bonus_tok", "path", "last_node", "escalate"):
        setattr(sc, f, 4096)
    sc.stats.top1_idx = sc.stats.p_top1 = sc.stats.p_top2 = sc.stats.p_draft = 4096
    sc.accept_rule = 7
    assert lib.trispec_accept_scan(ctypes.byref(sc), None) == 1
    sc.accept_rule, sc.alpha = ts.ACCEPT_TOKEN_SPECIFIC, 1.5
    assert lib.trispec_accept_scan(ctypes.byref(sc), None) == 1
