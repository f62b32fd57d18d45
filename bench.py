#!/usr/bin/env python
"""Benchmark of one TABED speculative-decoding round on B200.

A step is one round of the whole hot path on one batch of synthetic input:
tabed_draft_round (gamma batched shared-weight drafter steps with ensemble + draw at each) ->
tabed_verify -> tabed_update_weights.  The stand-in for the target model (it only has to produce
target logits) is outside the path: its logits are prepared by an untimed rehearsal of exactly the
rounds that are then timed (the library is deterministic, so the replay sees the same rounds).

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU checker instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2601_20357_b200 import workloads as W  # noqa: E402

METRIC = "sd_rounds_per_sec"
UNIT = "rounds/s"
PAPER_CONTEXT = ("paper (A100 80GB, fp16): expected walltime speedup 1.74x over autoregressive decoding, "
                 "~5% block-efficiency gain over single drafting; no rounds/s published")


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of ONE launch of the dominant kernel, from the ncu
# captures summarised under profiles/ ; keyed by (workload, kernel class).  Entries are removed when the kernel changes.
NCU_TRAFFIC = {("llava_small", "draft_round"): {"bytes": 690.13e6, "algorithmic_bytes_of_that_launch": 698.0e6,
                                                "source": "profiles/k_draft_round_llava_small_ncu_full.md"},
               ("large_vocab", "draft_round"): {"bytes": 3303.0e6, "algorithmic_bytes_of_that_launch": 3290.5e6,
                                                "source": "profiles/k_draft_round_llava_small_ncu_full.md (third part)"},
               ("long_context", "draft_round"): {"bytes": 3016.1e6, "algorithmic_bytes_of_that_launch": 3006.5e6,
                                                 "source": "profiles/k_draft_round_llava_small_ncu_full.md (second part)"},
               # captured on 16 of the 32 requests (capture-size rule) and scaled by the rows: 366.3 MB x 2
               ("batched_serving", "attention"): {"bytes": 732.6e6, "algorithmic_bytes_of_that_launch": 707.5e6,
                                                  "source": "profiles/k_attn_tc_bf16_batched_serving_ncu_full.md "
                                                            "(16 requests captured, scaled x2 to the 32 of the workload)"}}


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# --------------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------------
class ClockSampler:
    """nvidia-smi in a loop (every 20 ms); only samples stamped inside [mark_begin, mark_end] are used."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.path = tempfile.mktemp(suffix=".csv")
        self.proc = None
        self.gpu_index = gpu_index
        self.t0 = self.t1 = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
            time.sleep(0.5)                      # let the first samples arrive before the timed region opens
        except OSError:
            self.proc = None

    def mark_begin(self):
        self.t0 = time.time()

    def mark_end(self):
        self.t1 = time.time()

    def stop(self):
        import datetime
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons, all_sm = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                f_sm, f_mx = float(parts[1]), float(parts[2])
            except ValueError:
                continue
            all_sm.append(f_sm)
            if self.t0 is not None and not (self.t0 - 0.02 <= ts <= self.t1 + 0.02):
                continue
            sm.append(f_sm); mx.append(f_mx)
            for nm, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        os.unlink(self.path)
        return {"sm_mhz": float(np.median(sm)) if sm else (float(np.median(all_sm)) if all_sm else None),
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm), "samples_total": len(all_sm),
                "reasons": sorted(reasons)}


# --------------------------------------------------------------------------------------------------
# CPU checker as baseline / reference arm
# --------------------------------------------------------------------------------------------------
def oracle_setup(wl):
    from oracle.drafter import OracleDrafter
    from oracle.tabed import TabedOracle
    weights = W.make_weights(wl)
    orc = TabedOracle(n_inputs=wl.n_inputs, n_requests=wl.n_requests, gamma=wl.gamma, window_h=wl.window_h,
                      policy=wl.policy, vocab=wl.drafter.vocab, distance=wl.distance, sample_mode=wl.sample_mode,
                      tau=wl.tau, drafter=OracleDrafter(wl.drafter, weights), kv_capacity=wl.kv_capacity,
                      tree_width=wl.tree_width)
    if wl.synthetic_kv_len is not None:
        lens = W.synthetic_kv_lengths(wl)
        for row in range(wl.n_rows):
            k, v = W.make_synthetic_kv(wl, row, int(lens[row]))
            orc.load_kv(row, k, v)
    else:
        for b in range(wl.n_requests):
            for k, segs in enumerate(W.make_prefixes(wl, b)):
                orc.prefill(b * wl.n_inputs + k, segs)
    orc.set_pending(W.initial_pending(wl))
    return orc


def oracle_round(orc, wl, rnd):
    ud, ua, ur = W.round_uniforms(wl, rnd)
    orc.draft_round(ud)
    a, _ = orc.verify(W.target_logits(wl, rnd, orc.logits), ua, ur)
    orc.update_weights()
    return int(a.sum())


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def oracle_sample(wl):
    """The part of the workload one CPU step covers: whole rounds of the first requests, as many as keep a round
    of the plain checker to a few seconds (rows x layers x width is what a round costs)."""
    c = wl.drafter
    cost_row = c.n_params_layers + c.n_params_head                   # multiply-accumulates per row and step
    rows_max = max(wl.n_inputs, int(2.0e8 / cost_row) * wl.n_inputs)  # ~1-2 s of fp64 matrix-vector work per round
    n_req = max(1, min(wl.n_requests, rows_max // wl.n_inputs))
    return wl if n_req == wl.n_requests else wl.replace(n_requests=n_req)


def time_oracle(wl, rounds, warmup=0, budget_s=None):
    """Times `rounds` rounds (after `warmup`) of the checker; with a budget, stops early once it is used up.
    Returns (request-rounds per second, seconds, rounds actually timed)."""
    orc = oracle_setup(wl)
    for r in range(warmup):
        oracle_round(orc, wl, r)
    t0 = time.perf_counter()
    done = 0
    for r in range(warmup, warmup + rounds):
        oracle_round(orc, wl, r)
        done += 1
        if budget_s is not None and time.perf_counter() - t0 > budget_s:
            break
    dt = time.perf_counter() - t0
    return wl.n_requests * done / dt, dt, done


def config_of(wl):
    """The `config` object both arms print (identical keys and values for one workload)."""
    return {"workload": wl.name, "n_inputs": wl.n_inputs, "n_requests": wl.n_requests, "rows": wl.n_rows, "gamma": wl.gamma,
            "window_h": wl.window_h, "vocab": wl.drafter.vocab, "layers": wl.drafter.n_layers, "d_model": wl.drafter.d_model,
            "tree_width": wl.tree_width}


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sub = oracle_sample(wl)
    warm = min(args.warmup, 2)
    value, dt, done = time_oracle(sub, args.steps, warm, budget_s=150.0)
    cores = blas_threads()
    what = (f"each step = one whole round of the first {sub.n_requests} of {wl.n_requests} requests ({sub.n_rows} rows, their full caches); "
            f"{done} of {args.steps} steps timed after {warm} warm-up steps ({dt:.1f} s); value = requests x steps / time")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1000.0 * dt / max(done, 1), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(wl),
        "drafted_tokens_per_sec": value * wl.gamma,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------------
# CUDA arm
# --------------------------------------------------------------------------------------------------
def run_prefill(args, wl):
    """Feeding the prompts (not part of a round; the caches it leaves are what the rounds read): one JSON line with
    the tokens per second of both ways of feeding them, on a fresh handle each."""
    import torch
    from paper_2601_20357_b200 import binding as TB
    if wl.synthetic_kv_len is not None or wl.drafter.dtype != "bf16":
        print(json.dumps({"metric": "prefill_tokens_per_sec", "unavailable": "the workload's caches are loaded, not computed, "
                          "or its drafter is fp32 (fed one position at a time only)"}), flush=True)
        return
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    res = {}
    for name, path in (("chunks_of_256_positions_tcgen05", None), ("one_position_at_a_time", TB.PATH_PER_OP)):
        best = None
        for rep in range(3):
            tms = []
            g = gpu_setup(wl, device, prefill_path=path, prefill_times=tms)
            g.destroy()
            best = tms[0] if best is None or tms[0][1] < best[1] else best
        res[name] = {"tokens": best[0], "ms": best[1], "tokens_per_sec": best[0] / (best[1] / 1000.0)}
    # the pooled image prefix (2 x 2 average of a 24 x 24 token grid in the drafter's embedding width)
    g = gpu_setup(wl, device)
    x = torch.randn((576, wl.drafter.d_model), device=device)
    y = torch.empty((144, wl.drafter.d_model), device=device)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=device)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(20)]
    for i in range(23):
        flush.zero_()
        if i >= 3:
            evs[i - 3][0].record()
        g.pool_embeds(x, 24, 24, y)
        if i >= 3:
            evs[i - 3][1].record()
    torch.cuda.synchronize(device)
    pool_us = 1000.0 * float(np.mean([a.elapsed_time(b) for a, b in evs]))
    pool_bytes = (576 + 144) * wl.drafter.d_model * 4
    g.destroy()
    c = wl.drafter
    layer_w = c.n_layers * (c.d_model * (c.n_heads + 2 * c.n_kv_heads) * (c.d_model // c.n_heads) + c.n_heads * (c.d_model // c.n_heads) * c.d_model
                            + 3 * c.d_model * c.d_ffn) * 2
    print(json.dumps({"metric": "prefill_tokens_per_sec", "value": res["chunks_of_256_positions_tcgen05"]["tokens_per_sec"],
                      "unit": "tokens/s", "n_gpus": 1, "higher_is_better": True, "data": "synthetic",
                      "config": {"workload": wl.name, "rows": wl.n_rows, "prompt_tokens": res["chunks_of_256_positions_tcgen05"]["tokens"]},
                      "ways": res, "layer_weight_bytes_per_chunk": int(layer_w),
                      "pool_2x2": {"tokens_in": 576, "tokens_out": 144, "avg_us": pool_us, "bytes": int(pool_bytes),
                                   "gbs": pool_bytes / (pool_us * 1e-6) / 1e9, "note": "k_pool2x2, 20 launches, L2 flushed before each"},
                      "note": "best of 3 fresh handles each, CUDA events around the feeding calls; a chunk reads the layers' "
                              "weights once for 256 positions"}), flush=True)


def gpu_setup(wl, device, prefill_path=None, prefill_times=None):
    """prefill_path: path forced while the prompts are fed (None: the library's choice); prefill_times: a list that
    receives (tokens, milliseconds) of the prompt feeding, timed with CUDA events."""
    import torch
    from paper_2601_20357_b200 import binding as TB
    weights = TB.weights_to_device(wl.drafter, W.make_weights(wl), device)
    g = TB.Tabed(n_inputs=wl.n_inputs, n_requests=wl.n_requests, gamma=wl.gamma, window_h=wl.window_h,
                 policy=wl.policy, vocab=wl.drafter.vocab, distance=wl.distance, sample_mode=wl.sample_mode,
                 tau=wl.tau, drafter=wl.drafter, weights=weights, kv_capacity=wl.kv_capacity, device=device.index,
                 tree_width=wl.tree_width)
    tdt = torch.float32 if wl.drafter.dtype == "fp32" else torch.bfloat16
    dev = lambda a, dt=None: (torch.from_numpy(np.ascontiguousarray(a)).to(device) if dt is None
                              else torch.from_numpy(np.ascontiguousarray(a)).to(device).to(dt))
    if wl.synthetic_kv_len is not None:
        lens = W.synthetic_kv_lengths(wl)
        for row in range(wl.n_rows):
            k, v = W.make_synthetic_kv(wl, row, int(lens[row]))
            g.load_prefix_kv(row, dev(k, tdt), dev(v, tdt))
    else:
        if prefill_path is not None:
            g.select_path(prefill_path)
        feed = [(b * wl.n_inputs + k, seg.kind, dev(seg.data)) for b in range(wl.n_requests)
                for k, segs in enumerate(W.make_prefixes(wl, b)) for seg in segs]
        torch.cuda.synchronize(device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for row, kind, data in feed:
            if kind == "tokens":
                g.prefill_tokens(row, data)
            else:
                g.prefill_embeds(row, data)
        e1.record()
        torch.cuda.synchronize(device)
        if prefill_times is not None:
            prefill_times.append((int(sum(x[2].shape[0] for x in feed)), float(e0.elapsed_time(e1))))
        if prefill_path is not None:
            g.select_path(TB.PATH_AUTO)
    tok = np.zeros((wl.n_requests, 2), np.int32)
    tok[:, 0] = W.initial_pending(wl)
    g.set_pending(dev(tok), dev(np.ones(wl.n_requests, np.int32)))
    torch.cuda.synchronize(device)
    return g


def class_bytes(wl, kv_tokens_total, mean_accept):
    """Algorithmic bytes one timed interval of each kernel class has to move."""
    c = wl.drafter
    e = 4 if c.dtype == "fp32" else 2
    R, B, m, G, V, d, F = wl.n_rows, wl.n_requests, wl.n_inputs, wl.gamma, c.vocab, c.d_model, c.d_ffn
    kvd = c.n_kv_heads * c.head_dim
    valid = min(mean_accept, G - 1) + 1
    cb = {
        "qkv": (d * d + 2 * kvd * d) * e + R * d * 4 + R * (d + 2 * kvd) * 4,
        "attention": kv_tokens_total * 2 * kvd * e + R * (d + 2 * kvd) * 4 + R * d * 4,
        "oproj": d * d * e + 2 * R * d * 4,
        "gateup": 2 * F * d * e + R * d * 4 + R * F * 4,
        "down": d * F * e + R * F * 4 + 2 * R * d * 4,
        "lm_head": V * d * e + R * d * 4 + R * V * 4,
        "ensemble": R * V * 4 + B * V * 4 + R * V * 4,
        "verify": (G + 1) * B * V * 4 * 2 + G * B * V * 4,
        "update": valid * (m + 1) * B * V * 4,
    }
    # the persistent kernel runs the whole drafting round: gamma x (all layers + LM head + ensemble)
    cb["draft_round"] = G * (c.n_layers * (cb["qkv"] + cb["attention"] + cb["oproj"] + cb["gateup"] + cb["down"])
                             + cb["lm_head"] + cb["ensemble"])
    return cb


def measure(wl, device, K, Wm, *, rank=0, dist=None, path="auto", breakdown=False, e2e_steps=0, trace=None, trace_cta=0,
            clock_index=None):
    """Sets the workload up on `device`, rehearses the rounds (to have the target stand-in's logits), then times K
    rounds after Wm warm-up rounds, one CUDA-event pair per round, 256 MB written between rounds.  Returns a dict."""
    import torch
    from paper_2601_20357_b200 import binding as TB
    from paper_2601_20357_b200.replicas import whole_job
    total = K + Wm
    B, G, m, V = wl.n_requests, wl.gamma, wl.n_inputs, wl.drafter.vocab
    if wl.kv_capacity and wl.synthetic_kv_len is None:
        need = max(sum(l for _, l in pre) for pre in wl.prefixes) + (total + e2e_steps + 24) * (G + 1) + 8
        if need > wl.kv_capacity:
            wl = wl.replace(kv_capacity=need)
    g = gpu_setup(wl, device)
    if path == "per-op":
        g.select_path(TB.PATH_PER_OP)
    elif path == "tensor-core":
        g.select_path(TB.PATH_TENSOR_CORE)
    snap = g.state_export()
    alpha = torch.from_numpy(W.request_alpha(wl)).to(device)
    gen = torch.Generator(device=device)
    gen.manual_seed(W.MASTER_SEED + rank)

    # uniforms for every round, resident on the device
    u = [tuple(torch.from_numpy(x).to(device) for x in W.round_uniforms(wl, r)) for r in range(total)]
    toks = torch.empty((B, G, wl.tree_width), dtype=torch.int32, device=device)
    a = torch.empty(B, dtype=torch.int32, device=device)
    z = torch.empty_like(a)
    am = torch.empty_like(a)
    w = torch.empty((B, m), dtype=torch.float32, device=device)

    def synth_target(rnd):
        lg = g.debug_view(TB.VIEW_LOGITS)                               # [G][B][m][V]
        mix = torch.einsum("gbnv,bn->bgv", lg, alpha)
        tl = torch.empty((B, wl.n_target_rows, V), dtype=torch.float32, device=device)
        tl[:, :G] = mix
        tl[:, G] = mix[:, G - 1]
        if wl.tree_width > 1:               # leaves of the token tree: the mix of the next step (the last step's for the deepest)
            nxt = torch.clamp(torch.arange(G, device=device) + 1, max=G - 1)
            tl[:, G + 1:] = mix[:, nxt].repeat_interleave(wl.tree_width - 1, dim=1)
        tl += wl.sigma(rnd) * torch.randn(tl.shape, generator=gen, device=device)
        return tl

    # ---- rehearsal: produce the target logits of every round (untimed) ----
    targets, accepted = [], 0
    for r in range(total):
        g.draft_round(u[r][0], toks)
        tl = synth_target(r)
        g.verify(tl, u[r][1], u[r][2], a, z)
        g.update_weights(w, am)
        targets.append(tl)
        accepted += int(a.sum())
    torch.cuda.synchronize(device)
    mean_accept = accepted / (total * B)
    kv_mean = float(g.debug_view(TB.VIEW_KV_LEN).float().sum())       # tokens cached at the end of the rehearsal
    g.state_import(snap)
    kv_start = float(g.debug_view(TB.VIEW_KV_LEN).float().sum())
    kv_tokens_total = 0.5 * (kv_start + kv_mean) + wl.n_rows * (1 + G / 2)

    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=device)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]

    def one_round(r):
        g.draft_round(u[r][0], toks)
        g.verify(targets[r], u[r][1], u[r][2], a, z)
        g.update_weights(w, am)

    sampler = ClockSampler(clock_index) if clock_index is not None else None
    if sampler:
        sampler.start()
    for r in range(Wm):
        flush.zero_()
        one_round(r)
    torch.cuda.synchronize(device)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize(device)
    launches0 = g.launch_count()
    cur_path = g.current_path()
    persistent = cur_path == TB.PATH_PERSISTENT
    if persistent:
        top_cls, top_name, top_kernel = TB.PROF_DRAFT_ROUND, "draft_round", "k_draft_round (persistent: gamma decoder steps + ensemble)"
    elif cur_path == TB.PATH_TENSOR_CORE:
        top_cls, top_name, top_kernel = TB.PROF_ATTENTION, "attention", "k_attn_tc_bf16 (decode attention of all rows over their bf16 K,V caches)"
    else:
        top_cls, top_name, top_kernel = TB.PROF_LM_HEAD, "lm_head", "k_gemv (LM head)"
    g.profile_begin(top_cls)
    if sampler:
        sampler.mark_begin()
    wall0 = time.perf_counter()
    for i in range(K):
        flush.zero_()                       # the target model's pass between rounds evicts L2 in deployment
        ev[i][0].record()
        one_round(Wm + i)
        ev[i][1].record()
    head_ms, head_n = g.profile_end()       # synchronises the stream
    torch.cuda.synchronize(device)
    wall = time.perf_counter() - wall0
    if sampler:
        sampler.mark_end()
    dev_err = g.last_device_error()
    if dev_err != 0:                        # a bounded wait ran out or a cache overflowed: the timing means nothing
        raise RuntimeError(f"device-side error {dev_err} after the timed rounds of {wl.name}")
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize(device)
    clocks = sampler.stop() if sampler else None
    launches = g.launch_count() - launches0
    per_round = np.array([s.elapsed_time(e) for s, e in ev])
    dev_ms, _, value = whole_job(float(per_round.sum()), B * K, dist, device)     # slowest rank's time, all ranks' rounds

    peak, peak_kind = read_peaks()
    cb = class_bytes(wl, kv_tokens_total, mean_accept)
    head_dur = head_ms / max(head_n, 1)
    head_gbs = cb[top_name] / (head_dur * 1e-3) / 1e9
    round_bytes = int(cb["draft_round"] + cb["verify"] + cb["update"])
    res = {
        "wl": wl, "value": value, "dev_ms": dev_ms, "ms_per_step": dev_ms / K, "mean_accept": mean_accept, "wall": wall,
        "launches": int(launches), "clocks": clocks, "path": {TB.PATH_PERSISTENT: "persistent", TB.PATH_TENSOR_CORE: "tensor-core projections",
                                                            TB.PATH_PER_OP: "per-operation"}[cur_path],
        "roofline": {"kernel": top_kernel, "bound": "hbm", "achieved": head_gbs, "peak": peak, "unit": "GB/s",
                     "frac": head_gbs / peak, "peak_kind": peak_kind,
                     "traffic": (NCU_TRAFFIC.get((wl.name, top_name)) or {}).get("bytes"),
                     "traffic_note": NCU_TRAFFIC.get((wl.name, top_name)),
                     "avg_us": 1000.0 * head_dur, "launches_timed": head_n, "bytes_per_launch": int(cb[top_name]),
                     "share_of_round": head_ms / K / (dev_ms / K)},
        "round_roofline": {"bytes_per_round": round_bytes, "achieved_gbs": round_bytes / (dev_ms / K * 1e-3) / 1e9,
                           "frac": round_bytes / (dev_ms / K * 1e-3) / 1e9 / peak,
                           "note": "algorithmic bytes of one round / measured round time / peak"},
        "kernels": {}, "e2e": None,
    }

    # ---- per-class breakdown (separate untimed-for-the-headline passes over the same rounds) ----
    if rank == 0 and breakdown:
        names = ["qkv", "attention", "oproj", "gateup", "down", "lm_head", "ensemble", "verify", "update", "draft_round"]
        nb = min(K, 12)
        for cls, nm in enumerate(names):
            if (nm == "draft_round") != persistent and nm not in ("verify", "update"):
                continue
            g.state_import(snap)
            for r in range(Wm):
                one_round(r)
            g.profile_begin(cls)
            for i in range(nb):
                flush.zero_()
                one_round(Wm + i)
            ms, n = g.profile_end()
            dur = ms / max(n, 1)
            res["kernels"][nm] = {"intervals_per_round": n / nb, "avg_us": 1000.0 * dur, "bytes": int(cb[nm]),
                                  "gbs": cb[nm] / (dur * 1e-3) / 1e9 if dur > 0 else None,
                                  "frac_of_peak": cb[nm] / (dur * 1e-3) / 1e9 / peak if dur > 0 else None,
                                  "share_of_round": ms / nb / float(per_round.mean())}

    # ---- end to end through the host-buffer entry point ----
    if rank == 0 and e2e_steps > 0:
        ne = min(e2e_steps, K)
        g.state_import(snap)
        for r in range(Wm):
            one_round(r)
        torch.cuda.synchronize(device)
        pin = lambda x: x.cpu().pin_memory()
        hu = [(pin(u[Wm + i][0]), pin(u[Wm + i][1]), pin(u[Wm + i][2]), pin(targets[Wm + i])) for i in range(ne)]
        h_toks = torch.empty((B, G, wl.tree_width), dtype=torch.int32).pin_memory()
        h_a = torch.empty(B, dtype=torch.int32).pin_memory()
        h_z = torch.empty(B, dtype=torch.int32).pin_memory()
        h_am = torch.empty(B, dtype=torch.int32).pin_memory()
        h_w = torch.empty((B, m), dtype=torch.float32).pin_memory()
        t0 = time.perf_counter()
        for i in range(ne):
            g.round_host(hu[i][0], hu[i][1], hu[i][2], hu[i][3], h_toks, h_a, h_z, h_w, h_am)
        dt = time.perf_counter() - t0
        h2d = sum(x.numel() * x.element_size() for x in hu[0])
        d2h = sum(x.numel() * x.element_size() for x in (h_toks, h_a, h_z, h_am, h_w)) + 4
        res["e2e"] = {"value": B * ne / dt, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                      "steps": ne, "note": "tabed_round_host, pinned host buffers, L2 not flushed between rounds; the device-side "
                                           "error word is read back with the results"}

    if rank == 0 and trace and persistent:
        g.state_import(snap)
        for r in range(Wm):
            one_round(r)
        g.debug_trace(True, trace_cta)
        flush.zero_()
        g.draft_round(u[Wm][0], toks)
        torch.cuda.synchronize(device)
        g.debug_trace(False)
        tr = g.debug_view(TB.VIEW_TRACE).cpu().numpy().astype(np.int64)
        g.verify(targets[Wm], u[Wm][1], u[Wm][2], a, z)
        g.update_weights(w, am)
        write_trace(trace, trace_cta, wl, tr, float((clocks or {}).get("sm_mhz") or 1965.0))
    g.destroy()
    del targets, flush
    torch.cuda.empty_cache()
    return res


def write_trace(path, cta, wl, tr, mhz):
    L, G = wl.drafter.n_layers, wl.gamma
    nb_step = 5 * L + 3
    names_b = [f"L{l}.{nm}" for l in range(L) for nm in ("qkv", "attn", "o", "gateup", "down")] + ["lm_head", "expsum", "mix"]
    with open(path, "w") as f:
        f.write("# made by: python " + " ".join(a if a != path else "<this file>" for a in sys.argv) + "\n")
        f.write(f"# phase timeline of k_draft_round, workload {wl.name} (CTA {cta}): us from the end of the previous phase to the end of this one,\n"
                f"# then that CTA's share of it in us (cycles / {mhz:.0f} MHz): waiting for + staging activations, waiting for weight tiles, products,\n"
                f"# epilogue + refill, rest, (unused)\n"
                f"# (attention phases: waiting for + staging q/k/v, scores+softmax, PV+write, split merge, rest, -;\n"
                f"#  a phase in which the CTA owns no tile shows only the time it took to walk through it)\n")
        prev = None
        for st in range(G):
            for j in range(nb_step):
                tcur = int(tr[st, j, 0])
                secs = " ".join(f"{int(c) / mhz:7.2f}" for c in tr[st, j, 1:7])
                f.write(f"step {st} {names_b[j]:>12s} {((tcur - prev) / 1000.0 if prev is not None else 0.0):8.2f}   {secs}\n")
                prev = tcur
        f.write(f"# first barrier to last barrier: {(int(tr[G - 1, nb_step - 1, 0]) - int(tr[0, 0, 0])) / 1000.0:.1f} us\n")


def run_ours(args, wl):
    import torch
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=device)
    K, Wm = args.steps, args.warmup
    r = measure(wl, device, K, Wm, rank=rank, dist=dist, path=args.path, breakdown=not args.no_breakdown, e2e_steps=args.e2e_steps,
                trace=args.trace, trace_cta=args.trace_cta, clock_index=local)
    wl = r["wl"]
    # ---- the other workloads of the paper's shape, a few dozen rounds each (one GPU only) ----
    per_config = {}
    if rank == 0 and world == 1 and not args.no_per_config and args.path == "auto":
        for name in ("tiny", "llava_small", "large_vocab", "long_context", "batched_serving"):
            if name == wl.name:
                o = r
            else:
                o = measure(W.WORKLOADS[name], device, min(K, 30), 3)
            per_config[name] = {
                "ms_per_step": o["ms_per_step"], "rounds_per_sec": o["value"], "drafted_tokens_per_sec": o["value"] * o["wl"].gamma,
                "block_efficiency": o["mean_accept"] + 1.0, "path": o["path"], "rows": o["wl"].n_rows,
                "dominant_kernel": o["roofline"]["kernel"].split(" ")[0], "dominant_kernel_frac": o["roofline"]["frac"],
                "dominant_kernel_us": o["roofline"]["avg_us"], "dominant_kernel_share_of_round": o["roofline"]["share_of_round"],
                "round_frac": o["round_roofline"]["frac"], "bytes_per_round": o["round_roofline"]["bytes_per_round"]}
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    cpu = None
    if not args.no_cpu_baseline and world == 1:
        sub = oracle_sample(wl)
        v, dt, done = time_oracle(sub, args.cpu_rounds, 0, budget_s=25.0)
        cpu = {"value": v, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
               "sample": f"first {done} whole rounds of the first {sub.n_requests} of {wl.n_requests} requests of {wl.name} "
                         f"({sub.n_rows} rows, their full caches; prompt feeding / cache loading untimed), {dt:.1f} s; "
                         "value = requests x rounds / time"}
    G = wl.gamma
    line = {
        "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": r["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if wl.drafter.dtype == "bf16" else "f32",
        "dtype_note": ("bf16 weights, KV caches and matmul inputs with fp32 accumulation; decisions (softmax, mix, draw, accept, "
                       "deviations) in exactly rounded fp32 and integer arithmetic"),
        "data": "synthetic",
        "config": config_of(wl),
        "details": {"l2": "256 MB written between rounds (stands for the target model's pass); rounds timed one by one "
                          "with CUDA events", "parallelism": f"replicas x{world}", "path": r["path"]},
        "drafted_tokens_per_sec": r["value"] * G,
        "block_efficiency": r["mean_accept"] + 1.0,
        "wall_ms_per_step_incl_flush": 1000.0 * r["wall"] / K,
        "roofline": r["roofline"],
        "round_roofline": r["round_roofline"],
        "kernels": r["kernels"],
        "per_config": per_config,
        "cpu_baseline": cpu,
        "e2e": r["e2e"],
        "gpu_launches": r["launches"],
        "clocks": r["clocks"],
        "context": PAPER_CONTEXT,
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="batched_serving", choices=sorted(W.WORKLOADS),
                    help="workload of the headline line (default: the largest single-GPU one, 32 requests x 3 inputs)")
    ap.add_argument("--e2e-steps", type=int, default=50)
    ap.add_argument("--cpu-rounds", type=int, default=60, help="at most this many rounds of the CPU checker (and at most ~25 s)")
    ap.add_argument("--no-per-config", action="store_true", help="skip the short runs of the other four workloads")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-breakdown", action="store_true")
    ap.add_argument("--trace", default=None, help="write the persistent kernel's phase timeline of one round to this file")
    ap.add_argument("--trace-cta", type=int, default=0, help="the CTA whose phase timeline --trace records")
    ap.add_argument("--tree-width", type=int, default=1, help="candidates per depth of the token tree (Sec. 5); 1 = a plain chain")
    ap.add_argument("--requests", type=int, default=0, help="override the workload's number of concurrent requests (profiling aid)")
    ap.add_argument("--prefill", action="store_true",
                    help="time the feeding of the workload's prompts instead of rounds: chunks of positions through the "
                         "tensor-core kernels (the library's choice for bf16) and one position at a time")
    ap.add_argument("--path", default="auto", choices=["auto", "per-op", "tensor-core"],
                    help="drafting path (per-op forces one kernel per operation, tensor-core the tcgen05 projections)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    wl = W.WORKLOADS[args.config]
    if args.tree_width > 1:
        wl = wl.replace(tree_width=args.tree_width)
    if args.requests > 0:
        wl = wl.replace(n_requests=args.requests, name=f"{wl.name}[B={args.requests}]")
    if args.impl == "reference":
        run_reference(args, wl)
    elif args.prefill:
        run_prefill(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
