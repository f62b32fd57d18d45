"""One TABED speculative-decoding round on the CPU: Algorithm 1, verification, weight update.

TEST INFRASTRUCTURE ONLY.

State per request: the ensemble weight w* chosen at the end of the previous
round (Algorithm 1 steps 2-3 run before the drafting loop and w* is held for the
whole block, Sec. 4.1), a window of the last h verified positions' deviations
(Sec. 4.1 "cache and reuse"), the m row caches of the shared drafter, and the
pending token(s): the verified tokens the drafter has not consumed yet (one after
a rejection, two after a fully accepted block).

Readings taken where the paper is silent are listed with the library's design
notes; the ones that shape this file: the window holds only positions with a
verified prefix and a drafted q^(k) (i <= min(a, gamma-1)); before any history
exists the weights are equal (the paper's Static baseline); the grid has 11
candidates j = 0..10; deviations are summed, not averaged, over the window.
"""
from __future__ import annotations

from collections import deque
from typing import List, Optional

import numpy as np

from . import exact32 as x32

F = np.float32

POLICY_STATIC, POLICY_GRID_MT, POLICY_SOFTMAX_INV_ERR, POLICY_RANDOM, POLICY_GRID_HARD, POLICY_ADABOOST = 0, 1, 2, 3, 4, 5
DIST_KL, DIST_TVD = 0, 1
MODE_SAMPLE, MODE_GREEDY = 0, 1
N_GRID = 10


class TabedOracle:
    def __init__(self, *, n_inputs: int, n_requests: int, gamma: int, window_h: int,
                 policy: int, vocab: int, distance: int = DIST_KL, sample_mode: int = MODE_SAMPLE,
                 tau: float = 1.0, drafter=None, kv_capacity: int = 0, tree_width: int = 1):
        self.m, self.B, self.gamma, self.h = n_inputs, n_requests, gamma, window_h
        self.d = tree_width            # candidates per depth of the token tree (1: a plain chain)
        self.policy, self.V = policy, vocab
        self.distance, self.mode, self.tau = distance, sample_mode, tau
        if policy in (POLICY_GRID_MT, POLICY_GRID_HARD) and n_inputs != 2:
            raise ValueError("the grid policies are defined for two drafting methods")
        self.w = np.tile(x32.policy_static(n_inputs), (n_requests, 1))          # [B][m]
        self.j_star = np.full(n_requests, -1, np.int32)
        n_dev = (N_GRID + 1) if policy in (POLICY_GRID_MT, POLICY_GRID_HARD) else n_inputs
        self.n_dev = n_dev
        self.window = [deque() for _ in range(n_requests)]      # entries: int64 [n_dev]
        self.running = np.zeros((n_requests, n_dev), np.int64)  # h == 0: all history
        self.count = np.zeros(n_requests, np.int64)
        self.drafter = drafter
        self.caches = ([drafter.new_cache(kv_capacity) for _ in range(self.m * self.B)]
                       if drafter is not None else None)
        self.pending: List[List[int]] = [[] for _ in range(n_requests)]
        # results of the round in flight
        self.tokens = None      # [B][gamma] int32
        self.q = None           # [B][gamma][V] fp32
        self.qk = None          # [B][gamma][m][V] fp32
        self.logits = None      # [gamma][B][m][V] fp32
        self.p = None           # [B][gamma+1][V] fp32
        self.n_accept = None
        self.next_token = None
        self.cands = None       # [B][gamma][d] int32 candidates of every depth (column 0: the primary chain)
        self.acc_prim = None    # [B] accepted primaries;  sib_tok [B]: the accepted sibling's token or -1
        self.sib_tok = None

    def n_target_rows(self) -> int:
        """Rows of target logits per request: the primary chain's gamma + 1 positions, then one leaf per sibling
        candidate, depth-major: row gamma + 1 + i * (d - 1) + (c - 1) follows sibling c of depth i."""
        return self.gamma + 1 + self.gamma * (self.d - 1)

    # ---- drafter-side helpers -------------------------------------------------
    def prefill(self, row: int, segments) -> None:
        """Consume a row's prompt prefix (token ids or embeddings) into its cache."""
        for seg in segments:
            x = (self.drafter.embed_tokens(seg.data) if seg.kind == "tokens"
                 else np.asarray(seg.data, np.float64))
            self.drafter.forward(self.caches[row], x, want_logits=False)

    def load_kv(self, row: int, k: np.ndarray, v: np.ndarray) -> None:
        self.caches[row].load(k, v)

    def set_pending(self, tokens) -> None:
        self.pending = [[int(t)] for t in tokens]

    def kv_lengths(self) -> np.ndarray:
        return np.array([c.length for c in self.caches], np.int32)

    def _decode(self, b: int, token: int, want_logits: bool):
        """Feed one token to all m rows of request b (the same continuation, Algorithm 1 input)."""
        out = []
        for k in range(self.m):
            lg = self.drafter.forward(self.caches[b * self.m + k],
                                      self.drafter.embed_tokens([token]), want_logits)
            out.append(None if lg is None else lg[0])
        return out

    # ---- Algorithm 1, steps 4-8 ------------------------------------------------
    def _ensemble_step(self, b: int, i: int, logits_bk: np.ndarray, u) -> int:
        qk = x32.softmax_exact(logits_bk)                      # [m][V]
        q = x32.ensemble_exact(qk, self.w[b])
        self.qk[b, i], self.q[b, i] = qk, q
        self.cands[b, i] = x32.draw_candidates(q, np.atleast_1d(u), self.mode == MODE_GREEDY)
        return int(self.cands[b, i, 0])

    def _begin_round(self):
        B, G, m, V = self.B, self.gamma, self.m, self.V
        self.tokens = np.zeros((B, G), np.int32)
        self.q = np.zeros((B, G, V), F)
        self.qk = np.zeros((B, G, m, V), F)
        self.logits = np.zeros((G, B, m, V), F)
        self.cands = np.full((B, G, self.d), -1, np.int32)

    def draft_round(self, u_draft: np.ndarray):
        """gamma batched drafter steps; returns (tokens [B][gamma], q [B][gamma][V]).  u_draft [B][gamma] (or
        [B][gamma][d] with a token tree: one uniform per candidate)."""
        self._begin_round()
        u_draft = np.asarray(u_draft).reshape(self.B, self.gamma, self.d)
        for b in range(self.B):
            pend = self.pending[b]
            assert 1 <= len(pend) <= 2
            for t in pend[:-1]:
                self._decode(b, t, want_logits=False)          # catch-up: cache only
            tok = pend[-1]
            for i in range(self.gamma):
                lg = np.stack(self._decode(b, tok, True)).astype(F)     # [m][V]
                self.logits[i, b] = lg
                tok = self._ensemble_step(b, i, lg, u_draft[b, i])
                self.tokens[b, i] = tok
        return self.tokens, self.q

    def draft_round_logits(self, logits: np.ndarray, u_draft: np.ndarray):
        """Steps 6-7 on caller-supplied drafter logits [gamma][B][m][V]; no forward pass."""
        self._begin_round()
        u_draft = np.asarray(u_draft).reshape(self.B, self.gamma, self.d)
        self.logits = np.asarray(logits, F)
        for b in range(self.B):
            for i in range(self.gamma):
                self.tokens[b, i] = self._ensemble_step(b, i, self.logits[i, b], u_draft[b, i])
        return self.tokens, self.q

    # ---- Sec. 3, item 3 ---------------------------------------------------------
    def verify(self, target_logits: np.ndarray, u_accept: np.ndarray, u_resid: np.ndarray):
        """Sequential acceptance and the replacement / bonus token.
        target_logits [B][n_target_rows()][V] fp32; u_accept [B][gamma] ([B][gamma][d] with a tree).
        Returns (n_accept [B], next_token [B]); n_accept counts every accepted draft token (an accepted sibling too)."""
        B, G, d = self.B, self.gamma, self.d
        tl = np.asarray(target_logits, F)
        u_accept = np.asarray(u_accept).reshape(B, G, d)
        self.p = np.zeros((B, self.n_target_rows(), self.V), F)
        self.p[:, :G + 1] = x32.softmax_exact(tl[:, :G + 1])              # the primary chain's positions
        self.n_accept = np.zeros(B, np.int32)
        self.next_token = np.zeros(B, np.int32)
        self.acc_prim = np.zeros(B, np.int32)
        self.sib_tok = np.full(B, -1, np.int32)
        for b in range(B):
            i, z, sib = 0, None, -1
            while i < G and z is None and sib < 0:
                P, Q = self.p[b, i], self.q[b, i]
                if self.mode == MODE_GREEDY:
                    t = x32.argmax_lowest(P)
                    hit = [c for c in range(d) if int(self.cands[b, i, c]) == t]
                    if hit and hit[0] == 0:
                        i += 1
                    elif hit:
                        sib = hit[0]
                    else:
                        z = t
                    continue
                for c in range(d):
                    x = int(self.cands[b, i, c])
                    if x32.accept(P[x], Q[x], u_accept[b, i, c]):
                        if c > 0:
                            sib = c
                        break
                    # rejected: the replacement comes from the residual unless another candidate can be tried
                    more = c + 1 < d and int(self.cands[b, i, c + 1]) >= 0
                    P2, Q2, ok = x32.tree_after_rejection(P, Q, x) if more else (None, None, False)
                    if not ok:
                        mass = x32.residual_masses(P, Q)
                        if int(mass.sum(dtype=np.uint64)) == 0:
                            mass = x32.masses(P)
                        z = x32.draw(mass, u_resid[b])
                        break
                    P, Q = P2, Q2
                else:
                    raise AssertionError("unreachable: the last candidate either is accepted or ends the depth")
                if z is None and sib < 0:
                    i += 1                                            # the primary was accepted
            self.acc_prim[b] = i
            if sib >= 0:
                # an accepted sibling is a leaf: the next token comes from the target's distribution after it
                row = G + 1 + i * (d - 1) + (sib - 1)
                self.p[b, row] = x32.softmax_exact(tl[b, row])
                self.sib_tok[b] = self.cands[b, i, sib]
                z = x32.argmax_lowest(self.p[b, row]) if self.mode == MODE_GREEDY else x32.draw(x32.masses(self.p[b, row]), u_resid[b])
                self.n_accept[b] = i + 1
            else:
                if z is None:                                         # every primary accepted: bonus token from p_gamma
                    z = x32.argmax_lowest(self.p[b, G]) if self.mode == MODE_GREEDY else x32.draw(x32.masses(self.p[b, G]), u_resid[b])
                self.n_accept[b] = i
            self.next_token[b] = z
        return self.n_accept, self.next_token

    # ---- Sec. 4.1 deviation; App. B policies; Algorithm 1 steps 2-3 --------------
    def _deviation(self, p: np.ndarray, qk: np.ndarray, label: int) -> np.ndarray:
        """What one verified position contributes to the window: soft labels -> the distance of every drafter (or grid
        candidate) from p; hard labels -> whether each grid candidate's most likely token is the verified token
        (Sec. 4.1), or, for the AdaBoost variant, whether each drafter's most likely token is NOT it (its error)."""
        if self.policy == POLICY_GRID_HARD:
            return x32.grid_hard_matches(qk, label, N_GRID)
        if self.policy == POLICY_ADABOOST:
            return x32.drafter_errors(qk, label)
        dist = x32.tvd_fixed if self.distance == DIST_TVD else x32.kl_fixed
        if self.policy == POLICY_GRID_MT:
            return np.array([dist(p, x32.ensemble_exact(qk, x32.grid_weight(j, N_GRID)))
                             for j in range(N_GRID + 1)], np.int64)
        return np.array([dist(p, qk[k]) for k in range(self.m)], np.int64)

    def update_weights(self, u_policy=None):
        """Push the round's verified positions into the window, choose w* for the next block,
        and advance the caches / pending tokens.  u_policy [B][m]: uniforms of the Random policy.
        Returns (w [B][m], w_argmax [B])."""
        G = self.gamma
        self.u_policy = u_policy
        for b in range(self.B):
            a = int(self.acc_prim[b])                # accepted tokens of the primary chain (the drafter consumed those)
            sib = int(self.sib_tok[b])
            for i in range(min(a, G - 1) + 1):
                # the verified token of position i: the accepted draft, or what was emitted at the first other position
                label = int(self.tokens[b, i]) if i < a else (sib if sib >= 0 else int(self.next_token[b]))
                dev = self._deviation(self.p[b, i], self.qk[b, i], label)
                self.running[b] += dev
                self.count[b] += 1
                if self.h > 0:
                    self.window[b].append(dev)
                    if len(self.window[b]) > self.h:
                        self.running[b] -= self.window[b].popleft()
            self.w[b] = self._policy(b)
            # bookkeeping of the drafter rows
            if self.caches is not None:
                n_pend = len(self.pending[b])
                keep = n_pend + (a if a < G else G - 1)
                for k in range(self.m):
                    c = self.caches[b * self.m + k]
                    c.length = c.length - (n_pend + G - 1) + keep
            z = int(self.next_token[b])
            if a == G:
                self.pending[b] = [int(self.tokens[b, G - 1]), z]
            else:
                self.pending[b] = [sib, z] if sib >= 0 else [z]
        return self.w.copy(), np.argmax(self.w, axis=1).astype(np.int32)

    def _policy(self, b: int) -> np.ndarray:
        if self.policy == POLICY_RANDOM:
            return x32.policy_random(self.u_policy[b])
        if self.policy == POLICY_STATIC or self.count[b] == 0:
            return x32.policy_static(self.m)
        if self.policy == POLICY_GRID_HARD:
            self.j_star[b] = int(np.argmax(self.running[b]))            # most matches, lowest j on ties
            return x32.grid_weight(int(self.j_star[b]), N_GRID)
        if self.policy == POLICY_ADABOOST:
            n = len(self.window[b]) if self.h > 0 else int(self.count[b])
            return x32.policy_adaboost(self.running[b], n, self.V, self.tau)   # tau holds the constant C
        tvd = self.distance == DIST_TVD
        if self.policy == POLICY_GRID_MT:
            self.j_star[b] = int(np.argmin(self.running[b]))            # lowest j on ties
            return x32.grid_weight(int(self.j_star[b]), N_GRID)
        e = np.array([x32.fixed_to_float(int(t), tvd) for t in self.running[b]], F)
        return x32.policy_softmax_inv_err(e, self.tau)

    def window_error(self, b: int) -> np.ndarray:
        """Accumulated deviation over the window as float64, [n_dev]."""
        return self.running[b].astype(np.float64) * 2.0 ** -(40 + (1 if self.distance == DIST_TVD else 0))
