"""CPU-side checks of the C-ABI library: it builds, loads, exports every entry
point the header declares, and rejects bad arguments on the host before any
CUDA call (so these run without a GPU)."""
import ctypes
import os
import re

import paper_2602_04929_b200 as tb
from paper_2602_04929_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(tb_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    lib = tb.load()
    declared = _declared()
    assert len(declared) >= 14
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(tb.exported_symbols())


def test_status_strings():
    assert tb.status_string(0) == "ok"
    for st in range(1, 7):
        assert tb.status_string(st) not in ("ok", "unknown status")
    assert tb.status_string(99) == "unknown status"


def test_descriptor_layout_matches_header():
    assert ctypes.sizeof(binding.LayerDesc) == 11 * 4
    assert ctypes.sizeof(binding.Stats) == 64


def test_workspace_queries_and_growth():
    d = tb.layer_desc(256, 256, 1, 256, 4, 0, 8, flags=3)
    a = tb.tb_quantize_layer_workspace(d, False, False)
    b = tb.tb_quantize_layer_workspace(d, True, True)
    assert 0 < a < b
    lib = tb.load()
    assert lib.tb_factor_workspace(1, 256) > 2 * 256 * 256 * 8
    assert lib.tb_factor_workspace(0, 256) == 0
    assert lib.tb_prepare_correction_workspace(1, 128) >= 2 * 128 * 128 * 8
    assert lib.tb_build_hout_workspace(4, 64, 256) >= 4 * 64 * 256 * 8
    assert tb.tb_quantize_from_host_workspace(d, 2048, 1) > b


def test_bad_descriptions_are_rejected_on_the_host():
    lib = tb.load()
    one = ctypes.c_void_p(256)  # never dereferenced: validation fails first

    def call(desc, ws=one, ws_bytes=1 << 40, H_out=None, U_out=None):
        return lib.tb_quantize_layer(ctypes.byref(desc), one, one, one, H_out, U_out, None, None, None,
                                     one, one, one, None, None, None, None, None, ws, ws_bytes, None)

    ok = dict(d_out=256, d_in=256, n_heads=2, d_head=128, bits=4, quant_group=128, out_block=8)
    bad = [dict(ok, n_heads=3), dict(ok, bits=1), dict(ok, bits=9), dict(ok, quant_group=100),
           dict(ok, out_block=7), dict(ok, out_block=0), dict(ok, n_cand=0), dict(ok, n_cand=33),
           dict(ok, n_hin=3), dict(ok, cd_iters=-1)]
    for kw in bad:
        assert call(tb.layer_desc(**kw)) == 1, kw
    assert call(tb.layer_desc(**dict(ok, d_in=192, quant_group=0))) == 2      # d_in not a multiple of 128
    assert call(tb.layer_desc(**dict(ok, quant_group=16))) == 2               # group not a multiple of 32
    assert call(tb.layer_desc(**ok), H_out=one, U_out=None) == 1              # H_out without U_out
    assert call(tb.layer_desc(**ok), ws=None) == 3
    assert call(tb.layer_desc(**ok), ws_bytes=1024) == 3
    assert call(tb.layer_desc(**ok), ws=ctypes.c_void_p(8)) == 3               # misaligned workspace
    # other entry points
    assert lib.tb_accumulate_hessian(None, one, 0, 10, 64, None) == 1
    assert lib.tb_accumulate_hessian(one, one, 7, 10, 64, None) == 1
    assert lib.tb_accumulate_hessian(one, one, 0, 10, 60, None) == 1
    assert lib.tb_finalize_hessian(one, None, None, 64, 0, 0.01, None) == 1
    assert lib.tb_factor(one, 1, 64, one, None, one, None, 0, None) == 3
    assert lib.tb_factor(one, 0, 64, one, None, one, one, 1 << 40, None) == 1
    assert lib.tb_prepare_correction(one, one, 1, 64, one, one, one, 16, None) == 3
    assert lib.tb_build_hout(one, one, None, 3, 2, 64, 128, 0.0, one, 1 << 40, None) == 1


def test_host_entry_point_validates_the_whole_description_first():
    """tb_quantize_from_host must reject everything tb_quantize_layer would reject before it
    enqueues a copy (the pointers below are never dereferenced)."""
    lib = tb.load()
    one = ctypes.c_void_p(256)

    def call(desc, n_tok=4096, g_heads=2, G=one, ws=one, ws_bytes=1 << 40):
        return lib.tb_quantize_from_host(ctypes.byref(desc), one, one, n_tok, G, g_heads, 0.01, 0.01,
                                         one, one, one, None, None, ws, ws_bytes, None)

    ok = dict(d_out=256, d_in=256, n_heads=2, d_head=128, bits=4, quant_group=128, out_block=8)
    for kw in [dict(ok, bits=1), dict(ok, bits=9), dict(ok, out_block=7), dict(ok, out_block=0),
               dict(ok, n_cand=0), dict(ok, n_cand=33), dict(ok, cd_iters=-1), dict(ok, n_heads=3),
               dict(ok, quant_group=100)]:
        assert call(tb.layer_desc(**kw)) == 1, kw
    assert call(tb.layer_desc(**dict(ok, quant_group=16))) == 2
    assert call(tb.layer_desc(**dict(ok, d_in=192, quant_group=0))) == 2
    assert call(tb.layer_desc(**dict(ok, n_hin=2))) == 2
    assert call(tb.layer_desc(**ok), n_tok=0) == 1
    assert call(tb.layer_desc(**ok), g_heads=3) == 1
    assert call(tb.layer_desc(**ok), ws=None) == 3
    assert call(tb.layer_desc(**ok), ws_bytes=4096) == 3
    assert lib.tb_selftest_bounded_wait(-1, None, None) == 1
    assert lib.tb_selftest_bounded_wait(10 ** 10, None, None) == 1
