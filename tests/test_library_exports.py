"""Host-side checks that need no GPU: the built library exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "iv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(iv_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_four_path_calls():
    names = _declared_symbols()
    for must in ("iv_hash_chunks", "iv_merkle_root", "iv_verify_manifest", "iv_hash_ragged"):
        assert must in names


def test_library_loads_and_exports_every_declared_symbol():
    from paper_2510_23938_b200 import build
    build.build()                                  # nvcc cross-compiles without a GPU
    lib = ctypes.CDLL(build.LIB)
    for name in _declared_symbols():
        assert hasattr(lib, name), f"{name} is declared in include/iv.h but not exported"


def test_binding_lists_the_same_entry_points():
    from paper_2510_23938_b200 import binding
    assert sorted(binding.EXPORTS) == _declared_symbols()


def test_struct_layouts_match_the_header():
    from paper_2510_23938_b200 import binding
    assert ctypes.sizeof(binding.VerifyResult) == 48
    assert binding.VerifyResult.root.offset == 16
    assert ctypes.sizeof(binding.Manifest) == 64
    assert binding.Manifest.root.offset == 32
    assert ctypes.sizeof(binding.VerifyResult384) == 64 and ctypes.sizeof(binding.VerifyResult512) == 80
    assert ctypes.sizeof(binding.Manifest384) == 80 and ctypes.sizeof(binding.Manifest512) == 96


def test_create_fails_loudly_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2510_23938_b200 import binding
    with pytest.raises(binding.IvError) as err:
        binding.Context(0)
    assert err.value.code == binding.IV_ERR_NO_DEVICE


def test_strerror_texts():
    from paper_2510_23938_b200 import binding
    lib = binding.load_library()
    assert lib.iv_strerror(0) == b"ok"
    assert b"invalid" in lib.iv_strerror(binding.IV_ERR_INVALID_ARG)
