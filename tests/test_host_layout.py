"""Host-side layout helpers: the per-round arrays and the results are carved out of single buffers
so that the host-buffer entry point can merge their copies. No GPU needed."""
import numpy as np
import torch

from paper_2601_23180_b200 import binding as ts
from paper_2601_23180_b200 import inputs as gen
from paper_2601_23180_b200 import runner


def test_carve_is_gapless_when_sizes_allow_and_aligned_otherwise():
    # sizes that are multiples of 16 bytes: the views follow each other without gaps
    specs = [("a", (8,), torch.int32), ("b", (8, 4), torch.int32), ("c", (16,), torch.uint8)]
    flat = torch.zeros(ts._carve_bytes(specs), dtype=torch.uint8)
    v = ts._carve(flat, specs)
    assert ts._carve_bytes(specs) == 32 + 128 + 16
    assert v["b"].data_ptr() == v["a"].data_ptr() + 32 and v["c"].data_ptr() == v["b"].data_ptr() + 128
    # an odd size: the next array starts on the next multiple of 16 bytes
    specs = [("a", (3,), torch.int32), ("b", (5,), torch.bfloat16)]
    flat = torch.zeros(ts._carve_bytes(specs), dtype=torch.uint8)
    v = ts._carve(flat, specs)
    assert v["b"].data_ptr() == v["a"].data_ptr() + 16 and ts._carve_bytes(specs) == 16 + 10
    # views alias the flat buffer
    v["a"].fill_(-1)
    assert flat[:12].eq(255).all() and flat[12:].eq(0).all()


def test_scan_outputs_are_laid_out_in_copy_order():
    B, T = 8, 61
    specs = ts.scan_out_specs(B, T)
    assert [s[0] for s in specs] == ["accept_len", "bonus_tok", "last_node", "path", "escalate"]
    flat = torch.zeros(ts._carve_bytes(specs), dtype=torch.uint8)
    v = ts._carve(flat, specs)
    off = 0
    for name, shape, dtype in specs:
        assert v[name].data_ptr() == flat.data_ptr() + off, name    # B * 4 is a multiple of 16 here: no gaps
        off += v[name].numel() * v[name].element_size()
    assert off == 3 * B * 4 + B * T * 4 + B


def test_round_inputs_pack_and_unpack_bit_exactly():
    cfg = gen.small_variant(gen.CONFIGS["proxy_tree"], B=3, L=64, V=4096, d=64)
    inp = gen.make_inputs(cfg)
    for names in (("parent", "tok", "h"), ("q", "k_tree", "v_tree")):
        flat, specs = runner._pack_round_inputs(inp, names)
        v = ts._carve(flat, specs)
        for k in names:
            if k in ("parent", "tok"):
                assert np.array_equal(v[k].numpy(), inp[k])
            else:
                assert np.array_equal(v[k].view(torch.int16).numpy().view(np.uint16), inp[k].view(np.uint16))
            assert v[k].data_ptr() % 16 == 0
