"""CPU-side checks of the boundary: the library loads and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = []
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            names += re.findall(r"PUZZLE_API[^;(]*?\b(puzzle_\w+)\s*\(", text)
    return names


def test_library_exports_every_declared_symbol():
    from paper_2602_11937_b200 import binding, build
    build.build()
    lib = ctypes.CDLL(binding.library_path())
    declared = _declared()
    assert len(declared) >= 8
    for name in declared:
        assert hasattr(lib, name), name
    assert set(declared) == set(binding.EXPORTS)


def test_status_strings_and_workspace_size_need_no_gpu():
    import paper_2602_11937_b200 as P
    assert P.puzzle_status_string(0) == "ok"
    for code in range(1, 6):
        assert P.puzzle_status_string(code) not in ("ok", "unknown status")
    d = P.layer_desc()
    a = P.puzzle_decode_attn_workspace_bytes(d, 16, 0)
    b = P.puzzle_decode_attn_workspace_bytes(d, 16, 8)
    partials = 16 * 64 * 8 * 65 * 4                     # 8 splits of (o, lse) per (sequence, query head)
    head = b - partials                                 # CTA-speed words (these grow with the SM count) + arrival counters
    assert a > 0 and head % 256 == 0 and head >= 256 + 16384 * 4
    big = P.puzzle_decode_attn_workspace_bytes(d, 4096, 1) - 4096 * 64 * 65 * 4
    assert big - head == (4096 * 8 - 16384) * 4         # the counter block grows with the batch only beyond its floor
    bad = P.layer_desc(head_dim=128)
    assert P.puzzle_decode_attn_workspace_bytes(bad, 16, 0) == 0


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2602_11937_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", "/nonexistent/libpuzzle_attn.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.puzzle_launch_count()


def test_static_entry_point_reports_argument_errors_before_touching_the_device():
    """A NULL q (or out) is an argument error of puzzle_decode_attn_static that the host sees: it returns
    PUZZLE_ERR_NULL without a CUDA call, so this runs without a GPU.  The cache pointers are never followed."""
    from paper_2602_11937_b200 import binding
    lib = binding._load()
    desc = binding.layer_desc()
    kv = binding.KVView()
    kv.k_cache, kv.v_cache, kv.seq_lens = 0x1000, 0x2000, 0x3000
    kv.num_blocks, kv.max_blocks_per_seq = 64, 16
    kv.block_table, kv.k_scale, kv.v_scale = None, None, None
    call = lambda q, out: lib.puzzle_decode_attn_static(ctypes.byref(desc), ctypes.byref(kv), q, None, out, None, 4, 0,
                                                        None, None)
    assert call(None, ctypes.c_void_p(0x5000)) == 1      # PUZZLE_ERR_NULL
    assert call(ctypes.c_void_p(0x4000), None) == 1
    assert call(ctypes.c_void_p(0x4004), ctypes.c_void_p(0x5000)) == 2   # q not 8-byte aligned: PUZZLE_ERR_SHAPE
