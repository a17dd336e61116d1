"""The C-ABI library loads and exports every symbol the header declares; argument validation
works without a GPU (no compute call is made here)."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2602_02071_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return binding.load()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "baps.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(baps_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = _declared_functions()
    assert "baps_attention_fwd" in names and "baps_hif8_encode" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_status_strings(lib):
    assert binding.status_string(0) == "BAPS_OK"
    assert binding.status_string(-2) == "BAPS_ERR_UNSUPPORTED"
    assert binding.status_string(-5) == "BAPS_ERR_TIMEOUT"
    assert binding.status_string(-99) == "BAPS_ERR_UNKNOWN"


def test_argument_validation_needs_no_device(lib):
    # null pointers / bad sizes are rejected before any CUDA call
    assert lib.baps_hif8_encode(None, None, 16, None) == -1
    assert lib.baps_hif8_encode(None, None, 0, None) == 0
    assert lib.baps_hif8_decode(ctypes.c_void_p(8), ctypes.c_void_p(16), 16, None) == -3
    assert lib.baps_softmax_rows(ctypes.c_void_p(16), ctypes.c_void_p(32), 4, 100, 128, None) == -2
    assert lib.baps_softmax_rows(ctypes.c_void_p(16), ctypes.c_void_p(32), 4, 1 << 17, 128, None) == -2
    assert lib.baps_softmax_rows(ctypes.c_void_p(16), ctypes.c_void_p(32), 4, 1024, 32, None) == -2
    # block_k = 64 still needs a multiple of 128 columns (the header says so)
    assert lib.baps_softmax_rows(ctypes.c_void_p(16), ctypes.c_void_p(32), 4, 192, 64, None) == -2
    assert lib.baps_softmax_rows(ctypes.c_void_p(16), ctypes.c_void_p(32), -1, 1024, 128, None) == -1
    p16 = ctypes.c_void_p(256)
    assert lib.baps_softmax_rows_codes(p16, p16, p16, None, 4, 1024, 128, None) == -1
    assert lib.baps_softmax_rows_codes(p16, p16, p16, p16, 4, 192, 64, None) == -2
    assert lib.baps_softmax_rows_codes(p16, ctypes.c_void_p(8), p16, p16, 4, 1024, 128, None) == -3
    assert lib.baps_softmax_rows_codes(p16, p16, ctypes.c_void_p(2), p16, 4, 1024, 128, None) == -3
    p = ctypes.c_void_p(256)
    # H % Hkv != 0
    assert lib.baps_attention_fwd(p, p, p, p, 1, 3, 2, 128, 128, 0, 128, 128, None) == -1
    # unsupported head dim / tile / sequence length
    assert lib.baps_attention_fwd(p, p, p, p, 1, 2, 2, 128, 96, 0, 128, 128, None) == -2
    assert lib.baps_attention_fwd(p, p, p, p, 1, 2, 2, 128, 128, 0, 64, 64, None) == -2
    assert lib.baps_attention_fwd(p, p, p, p, 1, 2, 2, 192, 128, 0, 128, 128, None) == -2
    assert lib.baps_attention_fwd_f32(p, p, p, p, 1, 2, 2, 128, 64, 0, 64, 128, None) == -2
    assert lib.baps_attention_fwd(p, p, p, None, 1, 2, 2, 128, 128, 0, 128, 128, None) == -1
    assert lib.baps_attention_fwd(ctypes.c_void_p(8), p, p, p, 1, 2, 2, 128, 128, 0, 128, 128, None) == -3
    # statistics buffers: out_f32 is written with 16-byte stores, the others with 4-byte ones
    for bad in (binding._Stats(None, None, None, 264), binding._Stats(258, None, None, None),
                binding._Stats(None, 257, None, None), binding._Stats(None, None, 2, None)):
        assert lib.baps_attention_fwd_ex(p, p, p, p, 1, 2, 2, 128, 128, 0, 128, 128, 0, None,
                                         ctypes.byref(bad), None) == -3
    opts = binding._Opts(7, 0, 0.0, 0)
    assert lib.baps_attention_fwd_ex(p, p, p, p, 1, 2, 2, 128, 128, 0, 128, 128, 0,
                                     ctypes.byref(opts), None, None) == -2


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(FileNotFoundError):
        binding.load()
