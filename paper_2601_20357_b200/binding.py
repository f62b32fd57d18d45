"""ctypes binding of libtabed_b200.so: the same entry points as include/tabed.h.

Argument marshalling only: every step of the round runs in the CUDA library.  torch tensors are
used as device (or host) buffers; each wrapper checks dtype, device, contiguity and element count,
passes raw pointers, and raises TabedError on a negative return code.  There is no fallback: if the
shared library has not been built, loading fails with an error.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import torch

from . import build as _build

OK = 0
ERR_INVALID_ARG, ERR_NULL_PTR, ERR_BAD_STATE, ERR_KV_OVERFLOW, ERR_CUDA, ERR_TIMEOUT, ERR_UNSUPPORTED, ERR_NUMERIC = range(-1, -9, -1)
DTYPE_FP32, DTYPE_BF16 = 0, 1
POLICY_STATIC, POLICY_GRID_MT, POLICY_SOFTMAX_INV_ERR, POLICY_RANDOM, POLICY_GRID_HARD, POLICY_ADABOOST = range(6)
DIST_KL, DIST_TVD = 0, 1
MODE_SAMPLE, MODE_GREEDY = 0, 1
(VIEW_QK, VIEW_Q, VIEW_P, VIEW_LOGITS, VIEW_KV_LEN, VIEW_WEIGHTS, VIEW_WINDOW_SUM, VIEW_PENDING,
 VIEW_GRID_J, VIEW_ERROR_FLAG, VIEW_TRACE, VIEW_ACC_PRIMARY, VIEW_SIBLING) = range(13)
PATH_AUTO, PATH_PER_OP, PATH_PERSISTENT, PATH_TENSOR_CORE = 0, 1, 2, 3
MAX_DEV = 11
(PROF_QKV, PROF_ATTENTION, PROF_OPROJ, PROF_GATEUP, PROF_DOWN, PROF_LM_HEAD, PROF_ENSEMBLE, PROF_VERIFY,
 PROF_UPDATE, PROF_DRAFT_ROUND) = range(10)

EXPORTS = [
    "tabed_init", "tabed_destroy", "tabed_strerror", "tabed_load_prefix_kv", "tabed_prefill_tokens",
    "tabed_prefill_embeds", "tabed_pool_embeds", "tabed_set_pending", "tabed_decode_step", "tabed_ensemble_step",
    "tabed_draft_round", "tabed_draft_round_logits", "tabed_verify", "tabed_update_weights",
    "tabed_round_host", "tabed_debug_view", "tabed_debug_override_logits", "tabed_state_export", "tabed_state_import",
    "tabed_launch_count", "tabed_profile_begin", "tabed_profile_end", "tabed_ensemble_step_static",
    "tabed_select_path", "tabed_current_path", "tabed_debug_trace", "tabed_debug_gemm_tc",
    "tabed_last_device_error", "tabed_sync_lengths", "tabed_debug_barrier_timeout", "tabed_static_last_error",
    "tabed_set_policy_uniforms",
]


class TabedError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().tabed_strerror(code).decode()
        super().__init__(f"{where}: {msg} ({code})")


class TabedConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "d_ffn", "vocab", "dtype")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float)] + \
               [(n, C.c_int32) for n in ("n_inputs", "n_requests", "gamma", "window_h", "policy", "distance", "sample_mode")] + \
               [("tau", C.c_float), ("kv_capacity", C.c_int32), ("device", C.c_int32), ("stream", C.c_void_p),
                ("tree_width", C.c_int32)]


_PP = C.POINTER(C.c_void_p)


class TabedWeights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p)] + \
               [(n, _PP) for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "norm1", "norm2")]


_LIB = None


def lib_path() -> str:
    return _build.LIB_PATH


def lib() -> C.CDLL:
    """Load the CUDA library (raises if it has not been built)."""
    global _LIB
    if _LIB is None:
        path = lib_path()
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: run `python -m paper_2601_20357_b200.build` "
                               "(there is no CPU or eager fallback)")
        L = C.CDLL(path)
        vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
        L.tabed_strerror.restype = C.c_char_p
        L.tabed_strerror.argtypes = [C.c_int]
        L.tabed_init.argtypes = [C.POINTER(TabedConfig), C.POINTER(TabedWeights), C.POINTER(vp)]
        L.tabed_destroy.argtypes = [vp]
        L.tabed_destroy.restype = None
        L.tabed_load_prefix_kv.argtypes = [vp, i32, vp, vp, i32]
        L.tabed_prefill_tokens.argtypes = [vp, i32, vp, i32]
        L.tabed_prefill_embeds.argtypes = [vp, i32, vp, i32]
        L.tabed_pool_embeds.argtypes = [vp, vp, i32, i32, i32, vp]
        L.tabed_set_pending.argtypes = [vp, vp, vp]
        L.tabed_decode_step.argtypes = [vp, vp, vp]
        L.tabed_ensemble_step.argtypes = [vp] + [vp] * 6
        L.tabed_draft_round.argtypes = [vp, vp, vp, vp]
        L.tabed_draft_round_logits.argtypes = [vp, vp, vp, vp, vp]
        L.tabed_verify.argtypes = [vp] + [vp] * 5
        L.tabed_update_weights.argtypes = [vp, vp, vp]
        L.tabed_round_host.argtypes = [vp] + [vp] * 9
        L.tabed_debug_view.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(sz)]
        L.tabed_debug_override_logits.argtypes = [vp, vp]
        L.tabed_state_export.argtypes = [vp, vp, C.POINTER(sz)]
        L.tabed_state_import.argtypes = [vp, vp, sz]
        L.tabed_profile_begin.argtypes = [vp, i32]
        L.tabed_profile_end.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
        L.tabed_ensemble_step_static.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp]
        L.tabed_select_path.argtypes = [vp, i32]
        L.tabed_current_path.argtypes = [vp]
        L.tabed_debug_trace.argtypes = [vp, i32]
        L.tabed_debug_gemm_tc.argtypes = [vp, vp, i32, i32, i32, i32, vp, i32, vp]
        L.tabed_set_policy_uniforms.argtypes = [vp, vp]
        L.tabed_last_device_error.argtypes = [vp]
        L.tabed_sync_lengths.argtypes = [vp]
        L.tabed_debug_barrier_timeout.argtypes = [vp]
        L.tabed_static_last_error.argtypes = [i32, vp]
        L.tabed_launch_count.argtypes = [vp]
        L.tabed_launch_count.restype = C.c_int64
        for name in EXPORTS:
            if name not in ("tabed_strerror", "tabed_destroy", "tabed_launch_count"):
                getattr(L, name).restype = C.c_int
        _LIB = L
    return _LIB


def _check(code: int, where: str) -> None:
    if code != OK:
        raise TabedError(code, where)


def _ptr(t: Optional[torch.Tensor], dtype, numel: Optional[int], name: str, device: Optional[torch.device]) -> Optional[int]:
    if t is None:
        return None
    if t.dtype != dtype:
        raise TypeError(f"{name}: expected {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name}: must be contiguous")
    if numel is not None and t.numel() != numel:
        raise ValueError(f"{name}: expected {numel} elements, got {t.numel()}")
    if device is not None and t.device != device:
        raise ValueError(f"{name}: expected device {device}, got {t.device}")
    return t.data_ptr()


class _DeviceView:
    """Exposes a library-owned device buffer through __cuda_array_interface__."""

    def __init__(self, ptr: int, shape, typestr: str):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (ptr, False), "version": 3,
                                         "strides": None}


class Tabed:
    """One handle of the library; method names follow the C entry points (tabed_<name>)."""

    def __init__(self, *, n_inputs: int, n_requests: int, gamma: int, window_h: int, policy: int, vocab: int,
                 distance: int = DIST_KL, sample_mode: int = MODE_SAMPLE, tau: float = 1.0,
                 drafter=None, weights: Optional[Dict[str, object]] = None, kv_capacity: int = 0,
                 device: int = 0, stream: Optional[torch.cuda.Stream] = None, tree_width: int = 1):
        self._h = C.c_void_p()
        self.D = max(1, tree_width)                     # candidates per depth of the token tree
        self.device = torch.device("cuda", device)
        self.m, self.B, self.G, self.V = n_inputs, n_requests, gamma, vocab
        self.R = n_inputs * n_requests
        self.Rt = gamma + 1 + gamma * (self.D - 1)      # rows of target logits per request
        self.policy = policy
        cfg = TabedConfig()
        cfg.n_inputs, cfg.n_requests, cfg.gamma, cfg.window_h = n_inputs, n_requests, gamma, window_h
        cfg.policy, cfg.distance, cfg.sample_mode, cfg.tau = policy, distance, sample_mode, tau
        cfg.vocab, cfg.device = vocab, device
        cfg.stream = stream.cuda_stream if stream is not None else None
        cfg.kv_capacity = kv_capacity
        cfg.tree_width = tree_width
        self.drafter = drafter
        self._keep = []
        wptr = None
        if drafter is not None:
            cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.n_kv_heads = drafter.n_layers, drafter.d_model, drafter.n_heads, drafter.n_kv_heads
            cfg.d_ffn, cfg.dtype = drafter.d_ffn, DTYPE_FP32 if drafter.dtype == "fp32" else DTYPE_BF16
            cfg.rms_eps, cfg.rope_theta = drafter.rms_eps, drafter.rope_theta
            tdt = torch.float32 if drafter.dtype == "fp32" else torch.bfloat16
            self.wdtype = tdt
            w = TabedWeights()
            for nm in ("embed", "lm_head", "final_norm"):
                _ptr(weights[nm], tdt, None, nm, self.device)
                setattr(w, nm, weights[nm].data_ptr())
            for nm in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "norm1", "norm2"):
                arr = (C.c_void_p * drafter.n_layers)(*[_ptr(t, tdt, None, nm, self.device) for t in weights[nm]])
                self._keep.append(arr)
                setattr(w, nm, C.cast(arr, _PP))
            self._keep.append(weights)
            wptr = C.byref(w)
        self.cfg = cfg
        with torch.cuda.device(self.device):
            _check(lib().tabed_init(C.byref(cfg), wptr, C.byref(self._h)), "tabed_init")

    # -- lifetime ---------------------------------------------------------------------------------
    def destroy(self) -> None:
        if self._h:
            lib().tabed_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    # -- drafter-side ---------------------------------------------------------------------------------
    def load_prefix_kv(self, row: int, k: torch.Tensor, v: torch.Tensor) -> None:
        length = k.shape[2]
        _check(lib().tabed_load_prefix_kv(self._h, row, _ptr(k, self.wdtype, None, "k", self.device),
                                          _ptr(v, self.wdtype, k.numel(), "v", self.device), length), "tabed_load_prefix_kv")

    def prefill_tokens(self, row: int, tokens: torch.Tensor) -> None:
        _check(lib().tabed_prefill_tokens(self._h, row, _ptr(tokens, torch.int32, None, "tokens", self.device),
                                          tokens.numel()), "tabed_prefill_tokens")

    def prefill_embeds(self, row: int, embeds: torch.Tensor) -> None:
        _check(lib().tabed_prefill_embeds(self._h, row, _ptr(embeds, torch.float32, None, "embeds", self.device),
                                          embeds.shape[0]), "tabed_prefill_embeds")

    def pool_embeds(self, tokens: torch.Tensor, grid_h: int, grid_w: int, out: torch.Tensor) -> None:
        d = tokens.shape[1]
        _check(lib().tabed_pool_embeds(self._h, _ptr(tokens, torch.float32, grid_h * grid_w * d, "tokens", self.device), grid_h, grid_w, d,
                                       _ptr(out, torch.float32, (grid_h // 2) * (grid_w // 2) * d, "out", self.device)), "tabed_pool_embeds")

    def set_pending(self, tok: torch.Tensor, cnt: torch.Tensor) -> None:
        _check(lib().tabed_set_pending(self._h, _ptr(tok, torch.int32, self.B * 2, "tok", self.device),
                                       _ptr(cnt, torch.int32, self.B, "cnt", self.device)), "tabed_set_pending")

    def decode_step(self, tok: torch.Tensor, out_logits: Optional[torch.Tensor]) -> None:
        _check(lib().tabed_decode_step(self._h, _ptr(tok, torch.int32, self.B, "tok", self.device),
                                       _ptr(out_logits, torch.float32, self.R * self.V, "out_logits", self.device)),
               "tabed_decode_step")

    # -- round ------------------------------------------------------------------------------------------
    def ensemble_step(self, logits, w, u, y, q=None, qk=None) -> None:
        d = self.device
        _check(lib().tabed_ensemble_step(self._h, _ptr(logits, torch.float32, self.R * self.V, "logits", d),
                                         _ptr(w, torch.float32, self.R, "w", d), _ptr(u, torch.float32, self.B, "u", d),
                                         _ptr(y, torch.int32, self.B, "y", d), _ptr(q, torch.float32, self.B * self.V, "q", d),
                                         _ptr(qk, torch.float32, self.R * self.V, "qk", d)), "tabed_ensemble_step")

    def draft_round(self, u_draft, out_tokens, out_q=None) -> None:
        d = self.device
        _check(lib().tabed_draft_round(self._h, _ptr(u_draft, torch.float32, self.B * self.G * self.D, "u_draft", d),
                                       _ptr(out_tokens, torch.int32, self.B * self.G * self.D, "out_tokens", d),
                                       _ptr(out_q, torch.float32, self.B * self.G * self.V, "out_q", d)), "tabed_draft_round")

    def draft_round_logits(self, drafter_logits, u_draft, out_tokens, out_q=None) -> None:
        d = self.device
        _check(lib().tabed_draft_round_logits(
            self._h, _ptr(drafter_logits, torch.float32, self.G * self.R * self.V, "drafter_logits", d),
            _ptr(u_draft, torch.float32, self.B * self.G * self.D, "u_draft", d),
            _ptr(out_tokens, torch.int32, self.B * self.G * self.D, "out_tokens", d),
            _ptr(out_q, torch.float32, self.B * self.G * self.V, "out_q", d)), "tabed_draft_round_logits")

    def verify(self, target_logits, u_accept, u_resid, out_n_accept, out_next_token) -> None:
        d = self.device
        _check(lib().tabed_verify(self._h, _ptr(target_logits, torch.float32, self.B * self.Rt * self.V, "target_logits", d),
                                  _ptr(u_accept, torch.float32, self.B * self.G * self.D, "u_accept", d),
                                  _ptr(u_resid, torch.float32, self.B, "u_resid", d),
                                  _ptr(out_n_accept, torch.int32, self.B, "out_n_accept", d),
                                  _ptr(out_next_token, torch.int32, self.B, "out_next_token", d)), "tabed_verify")

    def set_policy_uniforms(self, u_policy: Optional[torch.Tensor]) -> None:
        self._keep_u_policy = u_policy
        _check(lib().tabed_set_policy_uniforms(self._h, _ptr(u_policy, torch.float32, self.R, "u_policy", self.device)),
               "tabed_set_policy_uniforms")

    def update_weights(self, out_w=None, out_w_argmax=None) -> None:
        d = self.device
        _check(lib().tabed_update_weights(self._h, _ptr(out_w, torch.float32, self.R, "out_w", d),
                                          _ptr(out_w_argmax, torch.int32, self.B, "out_w_argmax", d)), "tabed_update_weights")

    def round_host(self, u_draft, u_accept, u_resid, target_logits, out_tokens, out_n_accept, out_next_token,
                   out_w=None, out_w_argmax=None) -> None:
        cpu = torch.device("cpu")
        _check(lib().tabed_round_host(
            self._h, _ptr(u_draft, torch.float32, self.B * self.G * self.D, "u_draft", cpu),
            _ptr(u_accept, torch.float32, self.B * self.G * self.D, "u_accept", cpu), _ptr(u_resid, torch.float32, self.B, "u_resid", cpu),
            _ptr(target_logits, torch.float32, self.B * self.Rt * self.V, "target_logits", cpu),
            _ptr(out_tokens, torch.int32, self.B * self.G * self.D, "out_tokens", cpu),
            _ptr(out_n_accept, torch.int32, self.B, "out_n_accept", cpu),
            _ptr(out_next_token, torch.int32, self.B, "out_next_token", cpu),
            _ptr(out_w, torch.float32, self.R, "out_w", cpu), _ptr(out_w_argmax, torch.int32, self.B, "out_w_argmax", cpu)),
            "tabed_round_host")

    # -- views / state -----------------------------------------------------------------------------------
    def debug_view(self, what: int) -> torch.Tensor:
        """A torch tensor aliasing a library-owned device buffer (no copy)."""
        ptr, nbytes = C.c_void_p(), C.c_size_t()
        _check(lib().tabed_debug_view(self._h, what, C.byref(ptr), C.byref(nbytes)), "tabed_debug_view")
        B, G, m, V, R = self.B, self.G, self.m, self.V, self.R
        shape, ts = {
            VIEW_QK: ((B, G, m, V), "<f4"), VIEW_Q: ((B, G, V), "<f4"), VIEW_P: ((B, self.Rt, V), "<f4"),
            VIEW_ACC_PRIMARY: ((B,), "<i4"), VIEW_SIBLING: ((B,), "<i4"),
            VIEW_LOGITS: ((G, B, m, V), "<f4"), VIEW_KV_LEN: ((R,), "<i4"), VIEW_WEIGHTS: ((B, m), "<f4"),
            VIEW_WINDOW_SUM: ((B, MAX_DEV), "<i8"), VIEW_PENDING: ((B, 3), "<i4"), VIEW_GRID_J: ((B,), "<i4"),
            VIEW_ERROR_FLAG: ((1,), "<i4"),
            VIEW_TRACE: ((G, 5 * (self.drafter.n_layers if self.drafter is not None else 0) + 8, 8), "<u8")}[what]
        return torch.as_tensor(_DeviceView(ptr.value, shape, ts), device=self.device)

    def debug_override_logits(self, drafter_logits: Optional[torch.Tensor]) -> None:
        self._keep_override = drafter_logits
        _check(lib().tabed_debug_override_logits(
            self._h, _ptr(drafter_logits, torch.float32, self.G * self.R * self.V, "drafter_logits", self.device)),
            "tabed_debug_override_logits")

    def state_export(self) -> bytes:
        n = C.c_size_t()
        _check(lib().tabed_state_export(self._h, None, C.byref(n)), "tabed_state_export")
        buf = C.create_string_buffer(n.value)
        _check(lib().tabed_state_export(self._h, buf, C.byref(n)), "tabed_state_export")
        return buf.raw[:n.value]

    def state_import(self, blob: bytes) -> None:
        _check(lib().tabed_state_import(self._h, blob, len(blob)), "tabed_state_import")

    def profile_begin(self, kernel_class: int) -> None:
        _check(lib().tabed_profile_begin(self._h, kernel_class), "tabed_profile_begin")

    def profile_end(self):
        """(total milliseconds, number of timed intervals) of the class given to profile_begin."""
        ms, n = C.c_double(), C.c_int64()
        _check(lib().tabed_profile_end(self._h, C.byref(ms), C.byref(n)), "tabed_profile_end")
        return ms.value, n.value

    def select_path(self, path: int) -> None:
        _check(lib().tabed_select_path(self._h, path), "tabed_select_path")

    def current_path(self) -> int:
        rc = lib().tabed_current_path(self._h)
        if rc < 0:
            raise TabedError(rc, "tabed_current_path")
        return rc

    def debug_trace(self, on: bool, cta: int = 0) -> None:
        _check(lib().tabed_debug_trace(self._h, 1 + int(cta) if on else 0), "tabed_debug_trace")

    def last_device_error(self) -> int:
        """Return code of the device-side failures recorded since the last call (0 if none); clears the record."""
        return int(lib().tabed_last_device_error(self._h))

    def sync_lengths(self) -> None:
        _check(lib().tabed_sync_lengths(self._h), "tabed_sync_lengths")

    def debug_barrier_timeout(self) -> int:
        return int(lib().tabed_debug_barrier_timeout(self._h))

    def launch_count(self) -> int:
        return int(lib().tabed_launch_count(self._h))


def weights_to_device(drafter, weights_np: Dict[str, object], device: torch.device) -> Dict[str, object]:
    """numpy float32 weights (bf16-representable for a bf16 drafter) -> device tensors of the drafter's dtype."""
    tdt = torch.float32 if drafter.dtype == "fp32" else torch.bfloat16
    conv = lambda a: torch.from_numpy(a).to(device=device, dtype=tdt).contiguous()
    out: Dict[str, object] = {}
    for k, v in weights_np.items():
        out[k] = [conv(a) for a in v] if isinstance(v, list) else conv(v)
    return out


def debug_gemm_tc(w: torch.Tensor, act: torch.Tensor, ks: int = 1) -> torch.Tensor:
    """tabed_debug_gemm_tc: out[s][o] = sum_k w[o][k] * bf16(act[s][k]) on the tcgen05 path.  w bf16 [rows][K], act float [n][K]."""
    rows, K = w.shape
    n = act.shape[0]
    out = torch.empty((n, rows), dtype=torch.float32, device=w.device)
    _check(lib().tabed_debug_gemm_tc(_ptr(w, torch.bfloat16, rows * K, "w", w.device), _ptr(act, torch.float32, n * K, "act", w.device),
                                     rows, K, n, ks, out.data_ptr(), w.device.index or 0, None), "tabed_debug_gemm_tc")
    return out


def static_last_error(device: int = 0, stream: Optional[torch.cuda.Stream] = None) -> int:
    """tabed_static_last_error: code of a failure recorded by tabed_ensemble_step_static on `device` (0 if none)."""
    return int(lib().tabed_static_last_error(device, stream.cuda_stream if stream is not None else None))


def ensemble_step_static(logits: torch.Tensor, w: torch.Tensor, u: torch.Tensor, y: torch.Tensor, q: torch.Tensor,
                         qk: Optional[torch.Tensor] = None, sample_mode: int = MODE_SAMPLE,
                         stream: Optional[torch.cuda.Stream] = None) -> None:
    """tabed_ensemble_step_static: the ensemble step without a handle and without any allocation.

    For callers that cannot allocate device memory where they draft (all memory already owned by a
    serving pool, fixed budgets, paths that must not hit cudaMalloc): scratch is a fixed array inside
    the library.  logits [B][m][V], w [B][m], u [B] -> y [B], q [B][V], optional qk [B][m][V].
    Calls on one device share that scratch, so they must not overlap on the GPU."""
    B, m, V = logits.shape
    d = logits.device
    _check(lib().tabed_ensemble_step_static(
        _ptr(logits, torch.float32, B * m * V, "logits", d), _ptr(w, torch.float32, B * m, "w", d),
        _ptr(u, torch.float32, B, "u", d), B, m, V, sample_mode, d.index if d.index is not None else 0,
        stream.cuda_stream if stream is not None else None,
        _ptr(y, torch.int32, B, "y", d), _ptr(q, torch.float32, B * V, "q", d),
        _ptr(qk, torch.float32, B * m * V, "qk", d)), "tabed_ensemble_step_static")
