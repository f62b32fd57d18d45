"""Shared set-up for the GPU parity tests: builds the CUDA handle and the CPU checker on the same
seeded inputs and runs them round by round.  Values only ever flow from the seeded generators and
the checker into the CUDA library, never the other way."""
from __future__ import annotations

import dataclasses
from typing import Optional

import numpy as np
import torch

from oracle.drafter import OracleDrafter
from oracle.tabed import TabedOracle
from paper_2601_20357_b200 import binding as TB
from paper_2601_20357_b200 import workloads as W

DEV = torch.device("cuda", 0)

# |logit_gpu - logit_oracle| in the lock-step rounds, where each side builds its own caches.
# fp32 drafter: fp32 accumulation against fp64, ~1e-6 relative.  bf16 drafter: every matmul input is rounded to
# bf16; a value that the two sides compute ~1e-7 apart can fall on different sides of a rounding boundary (one
# step = 2^-8 relative), and the caches hold ~10^6 such roundings, so the two forward passes differ like two runs
# of the checker with a 1e-7 relative perturbation before every rounding (tests/test_oracle_drafter.py measures
# that on a small model).  How far depends on depth and width, so the bound is per workload: three times the
# largest (max, mean) of |dlogit| observed on a B200 over all rounds of all tests of that workload.
# tests/test_gpu_forward_tight.py has the sharper check (identical caches, one step).
LOCKSTEP_OBSERVED = {
    "tiny": (2.1e-7, 3.3e-8),               # 2 layers, d = 128, fp32
    "llava_small": (1.7e-2, 2.1e-3),        # 4 layers, d = 768
    "large_vocab": (4.0e-2, 4.0e-3),        # 12 layers, d = 896
    "long_context": (1.6e-2, 1.9e-3),       # 4 layers, d = 768, 8192 cached positions
    "batched_serving": (1.9e-2, 2.2e-3),    # 4 layers, d = 768, 96 rows
}
LOCKSTEP_OBSERVED_OTHER = {"fp32": (2.1e-7, 3.3e-8), "bf16": (1.2e-2, 1.6e-3)}     # the tests' two-layer drafters (d <= 896)


def logit_tols(wl):
    """(max, mean) bound on |dlogit| of a lock-step round of this workload."""
    obs = LOCKSTEP_OBSERVED.get(wl.name.split("[")[0], LOCKSTEP_OBSERVED_OTHER[wl.drafter.dtype])
    return 3.0 * obs[0], 3.0 * obs[1]


PROB_TOL = 1e-5           # tolerance on probabilities (the bar the library is built to)


def t(a: np.ndarray, dtype=None) -> torch.Tensor:
    x = torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    return x if dtype is None else x.to(dtype)


def make_oracle(wl: W.Workload, drafter: Optional[OracleDrafter]) -> TabedOracle:
    return TabedOracle(n_inputs=wl.n_inputs, n_requests=wl.n_requests, gamma=wl.gamma, window_h=wl.window_h,
                       policy=wl.policy, vocab=wl.drafter.vocab, distance=wl.distance, sample_mode=wl.sample_mode,
                       tau=wl.tau, drafter=drafter, kv_capacity=wl.kv_capacity, tree_width=wl.tree_width)


def make_gpu(wl: W.Workload, weights_dev=None) -> TB.Tabed:
    return TB.Tabed(n_inputs=wl.n_inputs, n_requests=wl.n_requests, gamma=wl.gamma, window_h=wl.window_h,
                    policy=wl.policy, vocab=wl.drafter.vocab, distance=wl.distance, sample_mode=wl.sample_mode,
                    tau=wl.tau, drafter=wl.drafter if weights_dev is not None else None, weights=weights_dev,
                    kv_capacity=wl.kv_capacity, tree_width=wl.tree_width)


@dataclasses.dataclass
class Pair:
    wl: W.Workload
    gpu: TB.Tabed
    orc: TabedOracle


def build_pair(wl: W.Workload, kv_lengths: Optional[np.ndarray] = None, prefill_path: Optional[int] = None) -> Pair:
    """Drafter-backed handle and checker with identical weights, prefixes / synthetic caches, pending tokens.
    prefill_path: path selected while the prompts are fed (None = the library's choice: chunks of positions
    through the tensor-core kernels for a bf16 drafter); the automatic choice is restored afterwards."""
    weights = W.make_weights(wl)
    orc = make_oracle(wl, OracleDrafter(wl.drafter, weights))
    wdev = TB.weights_to_device(wl.drafter, weights, DEV)
    gpu = make_gpu(wl, wdev)
    if prefill_path is not None:
        gpu.select_path(prefill_path)
    tdt = torch.float32 if wl.drafter.dtype == "fp32" else torch.bfloat16
    if wl.synthetic_kv_len is not None:
        lens = kv_lengths if kv_lengths is not None else W.synthetic_kv_lengths(wl)
        for row in range(wl.n_rows):
            k, v = W.make_synthetic_kv(wl, row, int(lens[row]))
            orc.load_kv(row, k, v)
            gpu.load_prefix_kv(row, t(k, tdt), t(v, tdt))
    else:
        for b in range(wl.n_requests):
            for k, segs in enumerate(W.make_prefixes(wl, b)):
                row = b * wl.n_inputs + k
                orc.prefill(row, segs)
                for seg in segs:
                    if seg.kind == "tokens":
                        gpu.prefill_tokens(row, t(seg.data))
                    else:
                        gpu.prefill_embeds(row, t(seg.data))
    if prefill_path is not None:
        gpu.select_path(TB.PATH_AUTO)
    pend = W.initial_pending(wl)
    orc.set_pending(pend)
    tok = np.zeros((wl.n_requests, 2), np.int32)
    tok[:, 0] = pend
    gpu.set_pending(t(tok), t(np.ones(wl.n_requests, np.int32)))
    return Pair(wl, gpu, orc)


def gpu_state(gpu: TB.Tabed):
    torch.cuda.synchronize()
    pend = gpu.debug_view(TB.VIEW_PENDING).cpu().numpy()
    return pend


def check_error_flag(gpu: TB.Tabed):
    assert int(gpu.debug_view(TB.VIEW_ERROR_FLAG).cpu()[0]) == 0


def assert_decisions_equal(p: Pair, toks_g, a_g, z_g, w_g, am_g, bit_exact_floats: bool):
    """Compare one finished round of the CUDA handle with the checker's round."""
    o, g = p.orc, p.gpu
    torch.cuda.synchronize()
    assert np.array_equal(toks_g.cpu().numpy().reshape(o.cands.shape), o.cands), "drafted tokens (all candidates)"
    assert np.array_equal(a_g.cpu().numpy(), o.n_accept), "accept counts"
    assert np.array_equal(g.debug_view(TB.VIEW_ACC_PRIMARY).cpu().numpy(), o.acc_prim), "accepted tokens of the primary chain"
    assert np.array_equal(g.debug_view(TB.VIEW_SIBLING).cpu().numpy(), o.sib_tok), "accepted sibling"
    assert np.array_equal(z_g.cpu().numpy(), o.next_token), "replacement / bonus token"
    assert np.array_equal(am_g.cpu().numpy(), np.argmax(o.w, axis=1)), "weight argmax"
    wg = w_g.cpu().numpy()
    if bit_exact_floats:
        assert np.array_equal(wg, o.w), "ensemble weights (bitwise)"
        n_dev = o.n_dev
        assert np.array_equal(g.debug_view(TB.VIEW_WINDOW_SUM).cpu().numpy()[:, :n_dev], o.running), "window sums"
    else:
        assert np.max(np.abs(wg - o.w)) <= 1e-5, "ensemble weights"
    if o.policy in (W.POLICY_GRID_MT, W.POLICY_GRID_HARD):
        assert np.array_equal(g.debug_view(TB.VIEW_GRID_J).cpu().numpy(), o.j_star), "grid j*"
    pend = g.debug_view(TB.VIEW_PENDING).cpu().numpy()
    for b in range(o.B):
        assert pend[b, 0] == len(o.pending[b]) and list(pend[b, 1:1 + pend[b, 0]]) == o.pending[b], "pending tokens"
    if o.caches is not None:
        assert np.array_equal(g.debug_view(TB.VIEW_KV_LEN).cpu().numpy(), o.kv_lengths()), "committed cache lengths"
    check_error_flag(g)


def assert_p_equal(p: Pair):
    """Target distributions, bitwise: the chain's positions and, with a token tree, the one leaf that was used."""
    o, g = p.orc, p.gpu
    G, d = o.gamma, o.d
    gp = g.debug_view(TB.VIEW_P).cpu().numpy()
    assert np.array_equal(gp[:, :G + 1], o.p[:, :G + 1]), "target p (bitwise)"
    for b in range(o.B):
        if o.sib_tok[b] >= 0:
            row = G + 1 + int(o.acc_prim[b]) * (d - 1) + (list(o.cands[b, o.acc_prim[b]]).index(int(o.sib_tok[b])) - 1)
            assert np.array_equal(gp[b, row], o.p[b, row]), "target p at the accepted leaf (bitwise)"


def logits_round(p: Pair, rnd: int, logits: np.ndarray, target: Optional[np.ndarray] = None):
    """One round on supplied drafter logits through tabed_draft_round_logits; everything bit-exact."""
    wl, o, g = p.wl, p.orc, p.gpu
    ud, ua, ur = W.round_uniforms(wl, rnd)
    o.draft_round_logits(logits, ud)
    tl = target if target is not None else W.target_logits(wl, rnd, logits)
    o.verify(tl, ua, ur)
    up = W.policy_uniforms(wl, rnd) if wl.policy == W.POLICY_RANDOM else None
    o_w, o_am = o.update_weights(up)
    if up is not None:
        g.set_policy_uniforms(t(up))
    toks = torch.empty((wl.n_requests, wl.gamma, wl.tree_width), dtype=torch.int32, device=DEV)
    out_q = torch.empty((wl.n_requests, wl.gamma, wl.drafter.vocab), dtype=torch.float32, device=DEV)
    a = torch.empty(wl.n_requests, dtype=torch.int32, device=DEV)
    z = torch.empty_like(a)
    am = torch.empty_like(a)
    w = torch.empty((wl.n_requests, wl.n_inputs), dtype=torch.float32, device=DEV)
    g.draft_round_logits(t(logits), t(ud), toks, out_q)
    g.verify(t(tl), t(ua), t(ur), a, z)
    torch.cuda.synchronize()
    assert np.array_equal(out_q.cpu().numpy(), o.q), "ensembled q (bitwise)"
    assert np.array_equal(g.debug_view(TB.VIEW_QK).cpu().numpy(), o.qk), "per-drafter q^(k) (bitwise)"
    assert_p_equal(p)
    g.update_weights(w, am)
    assert_decisions_equal(p, toks, a, z, w, am, bit_exact_floats=True)


def lockstep_round(p: Pair, rnd: int, override: bool = True):
    """One full round with the drafter's own forward pass.

    The checker runs first on its own trajectory.  With `override` its fp32 logits are handed to the
    CUDA round for the ensemble decisions, so both follow the same trajectory exactly and the CUDA
    forward pass can be compared with the checker's at every step; without it the CUDA round runs
    free and integer results are still required to match."""
    wl, o, g = p.wl, p.orc, p.gpu
    B, G, m, V = wl.n_requests, wl.gamma, wl.n_inputs, wl.drafter.vocab
    ud, ua, ur = W.round_uniforms(wl, rnd)
    o.draft_round(ud)
    logits_o = o.logits.copy()
    tl = W.target_logits(wl, rnd, logits_o)
    o.verify(tl, ua, ur)
    up = W.policy_uniforms(wl, rnd) if wl.policy == W.POLICY_RANDOM else None
    o.update_weights(up)
    if up is not None:
        g.set_policy_uniforms(t(up))
    toks = torch.empty((B, G, wl.tree_width), dtype=torch.int32, device=DEV)
    a = torch.empty(B, dtype=torch.int32, device=DEV)
    z = torch.empty_like(a)
    am = torch.empty_like(a)
    w = torch.empty((B, m), dtype=torch.float32, device=DEV)
    if override:
        g.debug_override_logits(t(logits_o))
    g.draft_round(t(ud), toks)
    g.verify(t(tl), t(ua), t(ur), a, z)
    torch.cuda.synchronize()
    # forward parity: logits within the derived bound, probabilities within 1e-5
    own = g.debug_view(TB.VIEW_LOGITS).clone()
    diff = (own.cpu().numpy().astype(np.float64) - logits_o.astype(np.float64))
    dt = wl.drafter.dtype
    print(f"LOCKSTEP {wl.name} {dt} round {rnd}: max |dlogit| {np.max(np.abs(diff)):.3e} mean {np.mean(np.abs(diff)):.3e}")
    tol_max, tol_mean = logit_tols(wl)
    assert np.max(np.abs(diff)) <= tol_max, f"logits max err {np.max(np.abs(diff))} > {tol_max}"
    assert np.mean(np.abs(diff)) <= tol_mean, f"logits mean err {np.mean(np.abs(diff))} > {tol_mean}"
    qk_own = torch.empty((B, m, V), dtype=torch.float32, device=DEV)
    y_tmp = torch.empty(B, dtype=torch.int32, device=DEV)
    for i in range(G):
        g.ensemble_step(own[i].contiguous(), None, t(ud.reshape(B, G, -1)[:, i, 0].copy()), y_tmp, None, qk_own)
        err = np.max(np.abs(qk_own.cpu().numpy().astype(np.float64) - o.qk[:, i].astype(np.float64)))
        assert err <= PROB_TOL, f"probabilities step {i}: {err}"
    if override:
        assert np.array_equal(g.debug_view(TB.VIEW_QK).cpu().numpy(), o.qk)
        assert_p_equal(p)
    g.update_weights(w, am)
    assert_decisions_equal(p, toks, a, z, w, am, bit_exact_floats=override)
    if override:
        g.debug_override_logits(None)
    return float(np.max(np.abs(diff)))
