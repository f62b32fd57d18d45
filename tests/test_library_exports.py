"""CPU check of the boundary: the shared library loads and exports every entry point the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "tabed.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tabed_[a-z_]+)\s*\(", text)))


def test_header_declares_the_four_core_calls():
    syms = declared_symbols()
    for name in ("tabed_init", "tabed_draft_round", "tabed_verify", "tabed_update_weights"):
        assert name in syms


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2601_20357_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    for name in declared_symbols():
        assert hasattr(lib, name), name
    lib.tabed_strerror.restype = ctypes.c_char_p
    assert lib.tabed_strerror(0) == b"ok"
    assert b"order" in lib.tabed_strerror(-3)


def test_binding_lists_every_declared_symbol():
    from paper_2601_20357_b200 import binding
    assert sorted(binding.EXPORTS) == declared_symbols()


def test_null_arguments_are_rejected_without_a_gpu():
    from paper_2601_20357_b200 import binding
    L = binding.lib()
    assert L.tabed_init(None, None, None) == -2
    assert L.tabed_draft_round(None, None, None, None) == -2
    assert L.tabed_verify(None, None, None, None, None, None) == -2
    assert L.tabed_update_weights(None, None, None) == -2
    assert L.tabed_launch_count(None) == 0
    L.tabed_destroy(None)
