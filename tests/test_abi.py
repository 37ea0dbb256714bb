"""The C-ABI library loads and exports every symbol include/ppd.h declares (no GPU needed)."""
import ctypes
import os
import re

import paper_2307_05908_b200 as ppd

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ppd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ppd_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    lib = ppd.load()
    names = declared_symbols()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(ppd.SIGNATURES)


def test_host_side_argument_checks_need_no_gpu():
    lib = ppd.load()
    import ppd_inputs
    cfg = ppd.make_config(ppd_inputs.TINY, max_seq=64, max_k=3)
    n = lib.ppd_device_bytes(ctypes.byref(cfg))
    assert 8_000_000 < n < 200_000_000
    bad = ppd.make_config(ppd_inputs.TINY, max_seq=64, max_k=9)
    assert lib.ppd_device_bytes(ctypes.byref(bad)) == 0
    bad = ppd.make_config(ppd_inputs.TINY, max_seq=64)
    bad.head_dim = 48
    assert lib.ppd_device_bytes(ctypes.byref(bad)) == 0
    assert lib.ppd_packed_bytes(32, 256) == 16384 and lib.ppd_packed_bytes(33, 257) == 4 * 16384
    assert lib.ppd_packed_bytes(0, 5) == 0
    assert lib.ppd_strerror(-2).decode().startswith("KV cache")
    h = ctypes.c_void_p()
    assert lib.ppd_create(ctypes.byref(cfg), None, n, None, None, ctypes.byref(h)) == -1
    assert lib.ppd_op_gemv(None, 1, 1, None, 1, 256, None, 0.0, 0, None, None, 1, None) == -1
    assert lib.ppd_position(None) == -1
    # 7B arena: packed weights + KV for 1024 positions + workspaces
    cfg7 = ppd.make_config(ppd_inputs.LLAMA_7B, max_seq=1024, max_k=3)
    n7 = lib.ppd_device_bytes(ctypes.byref(cfg7))
    assert 13.4e9 < n7 < 15.5e9
