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


def test_weight_pointers_must_be_16_byte_aligned():
    """The projection kernels read the drafter with 128-bit loads: tabed_init refuses a weight pointer that is
    not 16-byte aligned, before it touches the device (the addresses here are never dereferenced)."""
    import ctypes as C
    from paper_2601_20357_b200 import binding
    L = binding.lib()
    n_layers = 2

    def attempt(bad_field, bad_layer=0):
        cfg = binding.TabedConfig()
        cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.n_kv_heads, cfg.d_ffn, cfg.vocab, cfg.dtype = n_layers, 128, 2, 2, 256, 1000, 1
        cfg.rms_eps, cfg.rope_theta = 1e-5, 10000.0
        cfg.n_inputs, cfg.n_requests, cfg.gamma, cfg.window_h, cfg.policy, cfg.distance, cfg.sample_mode = 2, 1, 3, 4, 0, 0, 0
        cfg.tau, cfg.kv_capacity, cfg.device, cfg.stream = 1.0, 64, 63, None      # a device no machine has: nothing can run
        w = binding.TabedWeights()
        keep = []
        for nm in ("embed", "lm_head", "final_norm"):
            setattr(w, nm, 0x10000 + (4 if nm == bad_field else 0))
        for nm in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "norm1", "norm2"):
            arr = (C.c_void_p * n_layers)(*[0x20000 + 256 * l + (2 if (nm == bad_field and l == bad_layer) else 0) for l in range(n_layers)])
            keep.append(arr)
            setattr(w, nm, C.cast(arr, binding._PP))
        h = C.c_void_p()
        return L.tabed_init(C.byref(cfg), C.byref(w), C.byref(h))

    for field in ("embed", "lm_head", "final_norm", "wq", "w_down", "norm2"):
        assert attempt(field, 1 if field in ("w_down", "norm2") else 0) == -1, field
    assert attempt(None) == -5          # aligned pointers pass this check (and then fail for want of that device)
