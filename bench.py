#!/usr/bin/env python
"""Benchmark of the RazorAttention hot path on B200: compress -> (append, decode attention) x steps.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3] [--impl reference]

One "step" is one pass of the whole hot path over one synthetic batch of the workload:
prefill-end compression of every layer (from a dense layer buffer resident in HBM), then the
workload's decode steps, each a razor_append + razor_decode_attention on every layer.

metric/value: compressed-cache decode attention GB/s = compressed K+V bytes the pass's decode calls
attend over, divided by the time of the WHOLE pass (compression and appends included).
`decode` in the JSON line isolates the decode-attention kernel; `roofline` is that kernel against
the measured HBM copy bandwidth.  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "compressed_cache_decode_attention_GBps"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0        # the "~8 TB/s" the target is quoted against
FALLBACK_HBM_GBS = 6650.0       # used only when MEASURED_PEAKS.json is absent
# DRAM traffic of the decode kernel per algorithmic byte comes from an ncu capture summarised under profiles/.
# The summary names the sources it was taken on by their SHA-256; the ratio is used only while those
# sources are unchanged, otherwise roofline.traffic is null.
DECODE_TRAFFIC_PROFILE = os.path.join("profiles", "decode_kernel_cfg3_half_scale_and_cfg4_ncu_full.md")
DECODE_SOURCES = ["razor_decode.cu", "razor_sync.cuh", "razor_common.cuh", "razor_internal.h"]


def decode_sources_sha256() -> str:
    import hashlib
    h = hashlib.sha256()
    for name in DECODE_SOURCES:
        with open(os.path.join(ROOT, "paper_2407_15891_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def decode_traffic_per_alg_byte():
    """(ratio, where it comes from) or (None, why not)."""
    import re
    path = os.path.join(ROOT, DECODE_TRAFFIC_PROFILE)
    try:
        text = open(path).read()
    except OSError:
        return None, "no capture summary"
    sha = re.search(r"decode_sources_sha256:\s*([0-9a-f]{64})", text)
    ratio = re.search(r"dram_bytes_per_algorithmic_byte:\s*([0-9.]+)", text)
    if not sha or not ratio:
        return None, "capture summary carries no source hash"
    if sha.group(1) != decode_sources_sha256():
        return None, "the decode kernel's sources changed since the capture in " + DECODE_TRAFFIC_PROFILE
    return float(ratio.group(1)), DECODE_TRAFFIC_PROFILE


# ---------------------------------------------------------------------------------------------- byte accounting
def kept_tokens(w, layer: int, extra: int = 0) -> int:
    """Tokens the compressed cache of one layer holds, summed over (sequence, KV head), after `extra` appended
    tokens: a retrieval head holds its whole context, any other head at most n_sink + window tokens."""
    r = w.retrieval(layer)
    n_retr, n_other = int(r.sum()), int((1 - r).sum())
    tot = 0
    for b in range(w.batch):
        n = w.ctx_len[b] + extra
        tot += n_retr * n + n_other * min(n, w.n_sink + w.window[b])
    return tot


def compressed_bytes(w, layer: int, extra: int = 0) -> int:
    """Algorithmic bytes of one decode launch: every kept K and V row once."""
    return kept_tokens(w, layer, extra) * 2 * w.head_dim * w.esz()


def dense_bytes(w, extra: int = 0) -> int:
    """K + V bytes of one layer's uncompressed cache."""
    return sum(n + extra for n in w.ctx_len) * w.n_kv_heads * 2 * w.head_dim * w.esz()


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="razor", choices=["razor", "reference"])
    ap.add_argument("--workload", default="cfg3", choices=["cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--layers", type=int, default=0, help="use only the first LAYERS layers (profiling; not a valid bench number)")
    ap.add_argument("--decode-steps", type=int, default=0, help="override the workload's decode steps (profiling)")
    ap.add_argument("--scale", type=float, default=1.0, help="shrink contexts and windows (profiling captures; not a valid bench number)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-dense", action="store_true")
    ap.add_argument("--only-round", type=int, default=0, metavar="TOKENS",
                    help="run only the long-round leg with TOKENS new tokens per sequence and print its line (profiling; not the bench line)")
    ap.add_argument("--only-head-scores", type=int, default=0, metavar="HEADS",
                    help="run only the head-score leg on HEADS heads and print its line (profiling; not the bench line)")
    return ap.parse_args()


def max_over_ranks(ms: float, dist, device) -> float:
    """The slowest rank's time (every rank runs an independent replica; the job is as slow as that one)."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(world: int, bytes_per_rank: float, ms: float) -> float:
    """Whole-job GB/s of `world` replicas that each moved bytes_per_rank in ms (the max over ranks)."""
    return world * bytes_per_rank / (ms * 1e-3) / 1e9


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx, self.proc, self.lines = gpu_index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.idx)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); pw.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"], f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "power_w_max": max(pw), "samples": len(sm),
                "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------- oracle leg
def oracle_sample(w, budget_s=12.0):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: layer 0, sequence 0,
    KV heads taken in order until the budget is spent (at least one retrieval and one other head);
    per head one compression and the workload's decode steps (one query each, no appends: the oracle
    would recompress the whole history at every append).
    Returns (GB/s = compressed K+V bytes attended / (compress + decode time), description, threads, raw)."""
    import numpy as np
    from oracle import razor_oracle as orc
    from paper_2407_15891_b200 import synth
    try:
        cores = len(os.sched_getaffinity(0))        # host cores this process may run on
    except AttributeError:
        cores = os.cpu_count() or 1
    try:
        from threadpoolctl import threadpool_info
        blas = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        blas = 1
    threads = cores
    retr = w.retrieval(0)
    order = [g for g in range(w.n_kv_heads) if retr[g]][:1] + [g for g in range(w.n_kv_heads) if not retr[g]][:1]
    order += [g for g in range(w.n_kv_heads) if g not in order]
    b = 0
    n, win, T = w.ctx_len[b], w.window[b], w.decode_steps
    qs = [synth.make_queries(w, 0, t).double().numpy() for t in range(T)]
    scale = 1.0 / math.sqrt(w.head_dim)
    t_comp = t_dec = 0.0
    bytes_attended = 0
    heads = n_retr = 0
    t_start = time.perf_counter()
    for g in order:
        K, V = synth.make_dense_head(w, 0, b, g)
        K, V = K.double().numpy()[:n], V.double().numpy()[:n]
        t0 = time.perf_counter()
        hc = orc.compress_head(K, V, n, w.n_sink, win, bool(retr[g]))
        t1 = time.perf_counter()
        for t in range(T):
            for j in range(w.group):
                orc.decode_head(qs[t][b, g * w.group + j], hc, scale)
        t2 = time.perf_counter()
        t_comp += t1 - t0
        t_dec += t2 - t1
        bytes_attended += T * len(hc.kept_pos) * 2 * w.head_dim * w.esz()
        heads += 1
        n_retr += int(retr[g])
        if time.perf_counter() - t_start > budget_s and heads >= 2:
            break
    desc = (f"layer 0, sequence 0, {heads} of {w.n_kv_heads} KV heads ({n_retr} retrieval): one compression + {T} "
            f"decode steps each (no appends); compress {t_comp:.3f}s, decode {t_dec:.3f}s "
            f"(decode alone: {bytes_attended / t_dec / 1e9:.2f} GB/s); inputs generated per head outside the timing; "
            f"plain numpy fp64: the compression (row gather + sum) runs on one thread, the decode's matrix-vector "
            f"products in a BLAS pool of {blas} threads; {cores} host cores available")
    return bytes_attended / (t_comp + t_dec) / 1e9, desc, threads, dict(decode_s=t_dec, compress_s=t_comp, heads=heads)


def run_reference(args):
    """--impl reference: the CPU oracle timed on the host cores, same metric / unit / config."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2407_15891_b200 import synth
    w = synth.workload(args.workload)
    vals, times = [], []
    desc, threads = "", 1
    budget = max(2.0, min(12.0, 90.0 / max(1, args.steps + args.warmup)))
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        v, desc, threads, _ = oracle_sample(w, budget_s=budget)
        if i >= args.warmup:
            vals.append(v)
            times.append(time.perf_counter() - t0)
    value = statistics.mean(vals)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * statistics.mean(times), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(w, args):
    cfg = _workload_config(w, args)
    if args.layers or args.decode_steps or args.scale != 1.0:
        cfg["reduced_for_profiling"] = True      # not the benchmark workload: numbers are not bench values
    return cfg


def _workload_config(w, args):
    return {"workload": f"{w.name}: batch {w.batch}, {w.n_layers} layers, {w.n_q_heads}/{w.n_kv_heads} heads, "
                        f"head_dim {w.head_dim}, context {min(w.ctx_len)}..{max(w.ctx_len)}, {w.dtype} K/V, "
                        f"{w.n_retrieval_kv} retrieval KV heads per layer, n_sink {w.n_sink}, window "
                        f"{min(w.window)}..{max(w.window)}, {w.decode_steps} decode steps per pass",
            "step": "compress all layers + decode_steps x layers x razor_decode_step (append + decode attention in one launch)",
            "l2": "inputs larger than L2 (every launch streams > 126 MB of distinct cache pages)",
            "dense_input": "one seeded dense layer buffer resident in HBM, reused for every layer"}


# ---------------------------------------------------------------------------------------------- GPU legs
def decode_only(rz, synth, name, n_layers, dev, peak, reps=60, n_tok=1, alibi=False, with_append=False):
    """Decode attention alone on the first n_layers layers of another workload (each layer compressed from
    one seeded dense buffer): back-to-back razor_decode_attention calls cycling over the layers, so that
    every call streams pages that the L2 no longer holds."""
    import numpy as np
    import torch
    w = synth.workload(name)
    w.n_layers = n_layers
    retr = [w.retrieval(l) for l in range(n_layers)]
    cfg = rz.make_config(w.batch, n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, 0 if alibi else w.n_sink,
                         max(w.ctx_len), max(4, n_tok), use_compensation=0 if alibi else 1)
    cache = rz.RazorCache(cfg, w.ctx_len, w.window, np.stack(retr), device=dev)
    if alibi:   # the ALiBi variant: distance penalty on every logit, recent tokens only, no compensation token
        slopes = np.array([2.0 ** (-8.0 * (i + 1) / w.n_q_heads) for i in range(w.n_q_heads)], dtype=np.float32)
        rz.razor_cache_set_alibi(cache.handle, np.tile(slopes, n_layers))
        w = synth.Workload(w.name, w.batch, w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, w.ctx_len,
                           w.window, 0, w.n_retrieval_kv, w.decode_steps, w.seed)
    w0 = synth.Workload(w.name, w.batch, 1, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, w.ctx_len, w.window,
                        w.n_sink, w.n_retrieval_kv, 1, w.seed)
    K, V = synth.make_dense_kv(w0, 0, dev)
    for l in range(n_layers):
        cache.compress(l, K, V, w.ctx_len, retr[l], w.window)
    del K, V
    if n_tok > 1:     # a round of n_tok new tokens per sequence: bulk append, then all their queries in one call
        kv_shape = (w.batch, n_tok, w.n_kv_heads, w.head_dim)
        k_new = synth.normal_bf16(w.seed, synth.TAG_KNEW, kv_shape, dev, sub=77)
        v_new = synth.normal_bf16(w.seed, synth.TAG_VNEW, kv_shape, dev, sub=77)
        q = synth.normal_bf16(w.seed, synth.TAG_Q, (w.batch, n_tok, w.n_q_heads, w.head_dim), dev, sub=77)
        out = torch.empty(q.shape, dtype=torch.float32, device=dev)
        for l in range(n_layers):
            cache.append_many(l, k_new, v_new)
        call = cache.decode_multi
    else:
        q = synth.make_queries(w, 0, 0, dev)
        out = torch.empty((w.batch, w.n_q_heads, w.head_dim), dtype=torch.float32, device=dev)
        call = cache.decode
    for l in range(n_layers):
        call(l, q, out)
    torch.cuda.synchronize()
    reps = max(reps, n_layers)
    a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(reps):
        call(i % n_layers, q, out)
    b.record()
    torch.cuda.synchronize()
    us = a.elapsed_time(b) * 1e3 / reps
    kept = compressed_bytes(w, 0, extra=n_tok if n_tok > 1 else 0)
    gbs = kept / (us * 1e-6) / 1e9
    res = {"workload": f"{name}: batch {w.batch}, {w.n_q_heads}/{w.n_kv_heads} heads, context {max(w.ctx_len)}, "
                       f"{n_layers} layers cycled ({n_layers * kept / 1e9:.2f} GB of pages)",
           "us_per_layer": us, "gbs": gbs, "frac_of_measured": gbs / peak, "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS,
           "compressed_mb_per_layer": kept / 1e6, "launches_timed": reps,
           "query_tokens_per_call": n_tok, "alibi": bool(alibi)}
    if with_append and n_tok == 1:
        # the workload's decode step as a pass runs it: razor_append + razor_decode_attention on every layer
        k_new, v_new = synth.make_new_kv(w, 0, 0, dev)
        steps = 3
        for l in range(n_layers):                      # (max_new_tokens of this cache is steps + 1)
            cache.decode_step(l, k_new, v_new, q, out)
        torch.cuda.synchronize()
        a.record()
        for _ in range(steps - 1):
            for l in range(n_layers):
                cache.decode_step(l, k_new, v_new, q, out)
        b.record()
        torch.cuda.synchronize()
        us_p = a.elapsed_time(b) * 1e3 / ((steps - 1) * n_layers)
        kept_p = compressed_bytes(w, 0, extra=2)
        res["with_append"] = {"us_per_layer": us_p, "us_per_decode_step": us_p * n_layers,
                              "gbs": kept_p / (us_p * 1e-6) / 1e9,
                              "frac_of_measured": kept_p / (us_p * 1e-6) / 1e9 / peak,
                              "frac_of_nominal_8TBs": kept_p / (us_p * 1e-6) / 1e9 / NOMINAL_HBM_GBS,
                              "launches_timed": (steps - 1) * n_layers,
                              "note": "per layer: one razor_decode_step call (append + decode attention), all layers "
                                      "of the configuration, CUDA events at the ends of the run only"}
    res["device_status"] = cache.device_status()
    cache.close()
    return res


def long_round_leg(rz, synth, dev, n_tok=512, n_layers=2, reps=6):
    """A prompt-sized round on the 32K MHA shape: n_tok new tokens per sequence appended in bulk, then all their
    queries in one razor_decode_attention_multi call (the query-tiled tensor-core kernel: the cache is streamed
    once per 128 query rows).  A dense contraction: 4 * D flops per (query row, visible kept token)."""
    import numpy as np
    import torch
    w = synth.workload("cfg2")
    w.n_layers = n_layers
    retr = [w.retrieval(l) for l in range(n_layers)]
    cfg = rz.make_config(w.batch, n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, w.n_sink, max(w.ctx_len), n_tok)
    cache = rz.RazorCache(cfg, w.ctx_len, w.window, np.stack(retr), device=dev)
    w0 = synth.Workload(w.name, w.batch, 1, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, w.ctx_len, w.window,
                        w.n_sink, w.n_retrieval_kv, 1, w.seed)
    K, V = synth.make_dense_kv(w0, 0, dev)
    for l in range(n_layers):
        cache.compress(l, K, V, w.ctx_len, retr[l], w.window)
    del K, V
    kv_shape = (w.batch, n_tok, w.n_kv_heads, w.head_dim)
    k_new = synth.normal_bf16(w.seed, synth.TAG_KNEW, kv_shape, dev, sub=78)
    v_new = synth.normal_bf16(w.seed, synth.TAG_VNEW, kv_shape, dev, sub=78)
    q = synth.normal_bf16(w.seed, synth.TAG_Q, (w.batch, n_tok, w.n_q_heads, w.head_dim), dev, sub=78)
    out = torch.empty(q.shape, dtype=torch.float32, device=dev)
    for l in range(n_layers):
        cache.append_many(l, k_new, v_new)
        cache.decode_multi(l, q, out)
    torch.cuda.synchronize()
    a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(reps):
        cache.decode_multi(i % n_layers, q, out)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / reps
    # visible (query row, kept token) pairs: every kept token from before the round for every row, the round's own
    # tokens causally
    G = w.group
    pairs = 0
    for bb in range(w.batch):
        for g in range(w.n_kv_heads):
            n = w.ctx_len[bb] + n_tok
            kept = n if retr[0][g] else min(n, w.n_sink + w.window[bb])
            pairs += G * (n_tok * (kept - n_tok) + n_tok * (n_tok + 1) // 2)
    flops = 4.0 * w.head_dim * pairs
    try:
        peak = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["bf16_tflops"])
        kind = "measured (cuBLAS bf16 burst)"
    except Exception:
        peak, kind = 1590.0, "fallback"
    status = cache.device_status()
    cache.close()
    return {"workload": f"cfg2 shape: batch {w.batch}, {w.n_q_heads} heads, context {max(w.ctx_len)}, round of {n_tok} tokens",
            "ms_per_layer": ms, "tflops": flops / (ms * 1e-3) / 1e12, "bound": "tensor", "peak_tflops": peak,
            "peak_kind": kind, "frac": flops / (ms * 1e-3) / 1e12 / peak, "device_status": status,
            "note": "tcgen05 S = Q K^T and O = P V (P as a bf16 head plus a bf16 remainder: three matrix products per "
                    "block where the flop count above has two), one exponential per score"}


def chunked_prefill_leg(rz, synth, dev, peak, chunk=8192, reps=3):
    """One cfg3-shaped layer (batch 4, 40 heads, 65536 tokens) built chunk by chunk from an empty layer with
    razor_append_many, as a chunked prefill hands its K/V over: no dense cache of the whole context exists.
    Bytes: every chunk row is read once; a row that stays is written once; an evicted row is read once more."""
    import numpy as np
    import torch
    w = synth.workload("cfg3")
    N = max(w.ctx_len)
    retr = w.retrieval(0)
    cfg = rz.make_config(w.batch, 1, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, w.n_sink, 0, N)
    cache = rz.RazorCache(cfg, [0] * w.batch, w.window, np.stack([retr]), device=dev)
    shp = (w.batch, chunk, w.n_kv_heads, w.head_dim)
    k = synth.normal_bf16(w.seed, synth.TAG_KNEW, shp, dev, sub=5)
    v = synth.normal_bf16(w.seed, synth.TAG_VNEW, shp, dev, sub=6)
    n_chunks = N // chunk

    def build():
        cache.start_empty(0, retr, w.window)
        for _ in range(n_chunks):
            cache.append_many(0, k, v)

    build()
    torch.cuda.synchronize()
    a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        build()
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / reps
    row = w.head_dim * 2 * 2                                    # K and V row, bf16
    # Algorithmic bytes: every chunk row read once, and written once when it is stored (with chunk <= window every
    # row is in the cache after its chunk: the cache is usable for attention after every chunk).  With chunks of
    # at least the window length the evicted rows are not read back (their sum is on record).
    read = w.batch * w.n_kv_heads * N * row
    written = w.batch * row * w.n_kv_heads * N
    status = cache.device_status()
    cache.close()
    total = read + written
    return {"workload": f"cfg3 layer: {n_chunks} chunks of {chunk} tokens, batch {w.batch}, {w.n_kv_heads} heads",
            "ms_per_layer": ms, "us_per_chunk": ms * 1e3 / n_chunks, "gbs": total / (ms * 1e-3) / 1e9,
            "frac_of_measured": total / (ms * 1e-3) / 1e9 / peak, "read_gb": read / 1e9,
            "write_gb": written / 1e9, "device_status": status,
            "note": "bytes = chunk rows read once + rows stored once" + ("; evicted rows are not read back (chunk >= window)"
                    if chunk >= max(w.window) else "; chunks shorter than the window read the rows they evict once more")}


def head_scores_leg(rz, synth, dev, reps=5, heads=32):
    """Section 3.3's score reduction on its own input shape: 2500 random tokens repeated 4 times, 32 heads of
    dimension 128 (one layer of a 7B-class model).  A dense contraction (causal Q.K^T), so it is reported
    against the tensor peak; it runs once per model, offline."""
    import torch
    H, period, D = heads, 2500, 128
    n = 4 * period
    Q = synth.normal_bf16(7, synth.TAG_Q, (H, n, D), dev)
    K = synth.normal_bf16(7, synth.TAG_K, (H, n, D), dev)
    rz.razor_head_scores(Q, K, period)
    torch.cuda.synchronize()
    a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        rz.razor_head_scores(Q, K, period)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / reps
    tiles = sum(t + 1 for t in range((n + 127) // 128) if (t + 1) * 128 > period)   # 128 x 128 score tiles computed
    flops = H * tiles * 2.0 * 128 * 128 * D
    try:
        peak = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["bf16_tflops"])
        kind = "measured (cuBLAS bf16 burst)"
    except Exception:
        peak, kind = 1590.0, "fallback"
    return {"workload": f"{H} heads x {n} tokens x {D}, period {period}", "ms": ms, "tflops": flops / (ms * 1e-3) / 1e12,
            "bound": "tensor", "peak_tflops": peak, "peak_kind": kind, "frac": flops / (ms * 1e-3) / 1e12 / peak,
            "note": "tcgen05 score tiles in tensor memory, exp-bound (one ex2 per score); an offline, once-per-model step"}


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import numpy as np
    import torch
    from paper_2407_15891_b200 import binding as rz
    from paper_2407_15891_b200 import build as rz_build
    from paper_2407_15891_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if args.only_round > 0:
        if rank == 0:
            print(json.dumps(long_round_leg(rz, synth, dev, n_tok=args.only_round, reps=max(1, args.steps))))
        return
    if args.only_head_scores > 0:
        if rank == 0:
            print(json.dumps(head_scores_leg(rz, synth, dev, reps=max(1, args.steps), heads=args.only_head_scores)))
        return
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        rz_build.build()
    if dist is not None:
        dist.barrier()
    rz.load()

    w = synth.workload(args.workload, args.scale)
    if args.layers:
        w.n_layers = min(w.n_layers, args.layers)
    if args.decode_steps:
        w.decode_steps = args.decode_steps
    L, T = w.n_layers, w.decode_steps
    tdt = synth.torch_dtype(w)
    per_seq = w.name == "cfg5"

    retr = [w.retrieval(l) for l in range(L)]
    cfg = rz.make_config(w.batch, L, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, w.n_sink, max(w.ctx_len), T + 4)
    cache = rz.RazorCache(cfg, w.ctx_len, w.window, np.stack(retr), device=dev)

    # inputs, resident in HBM before the timed region
    if per_seq:
        dense = []
        for b in range(w.batch):
            wb = synth.Workload(w.name, 1, 1, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, [w.ctx_len[b]],
                                [w.window[b]], w.n_sink, w.n_retrieval_kv, T, w.seed * 131 + b)
            K, V = synth.make_dense_kv(wb, 0, dev)
            dense.append((K[0], V[0]))
    else:
        w0 = synth.Workload(w.name, w.batch, 1, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, w.ctx_len, w.window,
                            w.n_sink, w.n_retrieval_kv, T, w.seed)
        Kd, Vd = synth.make_dense_kv(w0, 0, dev)
    n_q = 4   # distinct per-step inputs, cycled
    qs = [synth.make_queries(w, 0, i, dev) for i in range(n_q)]
    kvs = [synth.make_new_kv(w, 0, i, dev) for i in range(n_q)]
    out = torch.empty((w.batch, w.n_q_heads, w.head_dim), dtype=torch.float32, device=dev)
    torch.cuda.synchronize()

    launches = {"n": 0}

    def compress_all():
        for l in range(L):
            if per_seq:
                for b in range(w.batch):
                    cache.compress_seq(l, b, dense[b][0], dense[b][1], w.ctx_len[b], retr[l], w.window[b])
                    launches["n"] += 3    # plan, streaming compression kernel, finalize
            else:
                cache.compress(l, Kd, Vd, w.ctx_len, retr[l], w.window)
                launches["n"] += 3

    def one_pass(ev=None):
        compress_all()
        if ev is not None:
            ev["compress_end"].record()
        for t in range(T):
            k_new, v_new = kvs[t % n_q]
            q = qs[t % n_q]
            for l in range(L):
                cache.decode_step(l, k_new, v_new, q, out)      # append + decode attention, one launch
                launches["n"] += 1 + combine_launched(l)        # streaming kernel (+ combine kernel for heads in many parts)

    combine_cache = {}

    def combine_launched(l):
        """1 when the layer's schedule has a head in more parts than the streaming kernel folds itself."""
        if l not in combine_cache:
            combine_cache[l] = int(len(rz.razor_schedule_combine_heads(cache.handle, l)) > 0)
        return combine_cache[l]

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # algorithmic bytes of the pass
    def decode_alg_bytes(l, t):
        kv = compressed_bytes(w, l, extra=t + 1)
        n_nonretr = int((1 - retr[l]).sum()) * w.batch
        small = w.batch * w.n_q_heads * w.head_dim * (w.esz() + 4) + n_nonretr * 2 * w.head_dim * 4
        return kv, kv + small
    attended = sum(decode_alg_bytes(l, t)[0] for l in range(L) for t in range(T))
    compress_read = dense_bytes(w) * L
    compress_write = sum(compressed_bytes(w, l) for l in range(L))

    for _ in range(args.warmup):
        one_pass()
    sync_all()

    sampler = ClockSampler(local)
    sampler.start()
    ev = {"compress_end": torch.cuda.Event(enable_timing=True)}
    starts, ends, comp_ends = [], [], []
    launches["n"] = 0
    sync_all()
    for _ in range(args.steps):
        s = torch.cuda.Event(enable_timing=True); e = torch.cuda.Event(enable_timing=True)
        ev["compress_end"] = torch.cuda.Event(enable_timing=True)
        s.record()
        one_pass(ev)
        e.record()
        starts.append(s); ends.append(e); comp_ends.append(ev["compress_end"])
    sync_all()
    clocks = sampler.stop()
    n_launches = launches["n"]

    total_ms = max_over_ranks(starts[0].elapsed_time(ends[-1]), dist, dev)
    ms_per_step = total_ms / args.steps
    value = replica_throughput(world, attended, ms_per_step)

    comp_ms = statistics.mean(s.elapsed_time(c) for s, c in zip(starts, comp_ends))
    dec_phase_ms = statistics.mean(c.elapsed_time(e) for c, e in zip(comp_ends, ends))
    # The decode launches are timed as they run in the pass: no event sits between two launches (an event record
    # between an append and its decode kernel would undo the overlap of their programmatic launches), so the
    # duration of one launch is the decode phase of the pass divided by its launches.  That phase also holds the
    # append kernels, which makes the figure an upper bound on the decode launch itself.
    n_dec = T * L
    us_per_launch = dec_phase_ms * 1e3 / n_dec
    alg_total = sum(decode_alg_bytes(l, t)[1] for l in range(L) for t in range(T))
    alg_per_launch = alg_total / n_dec
    dec_gbs = alg_total / (dec_phase_ms * 1e-3) / 1e9
    peak, peak_kind = measured_peak()
    ratio, ratio_src = decode_traffic_per_alg_byte()
    roofline = {"bound": "hbm", "kernel": "decode_kernel (+ its dependent combine_kernel): one razor_decode_attention call",
                "achieved": dec_gbs, "peak": peak, "unit": "GB/s",
                "frac": dec_gbs / peak, "peak_kind": f"of {peak_kind} (sustained copy bandwidth)",
                "frac_of_nominal_8TBs": dec_gbs / NOMINAL_HBM_GBS,
                "alg_bytes_per_launch": alg_per_launch, "us_per_launch": us_per_launch,
                "launches_timed": n_dec * args.steps,
                "how": "decode phase of the timed passes / its razor_decode_step calls (append + decode attention in one "
                       "launch), CUDA events at the ends of the phase only",
                "traffic": (ratio * alg_per_launch) if ratio else None, "traffic_source": ratio_src}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": w.dtype if w.dtype != "bf16" else "bf16", "data": "synthetic", "config": workload_config(w, args),
        "clocks": clocks, "gpu_launches": n_launches, "roofline": roofline,
        "decode": {"gbs_kernel": dec_gbs, "us_per_layer": us_per_launch,
                   "us_per_decode_step": dec_phase_ms * 1e3 / T,
                   "gbs_phase_incl_append": attended / (dec_phase_ms * 1e-3) / 1e9,
                   "compressed_gb_per_decode_step": attended / T / 1e9},
        "compress": {"ms_per_pass": comp_ms, "gbs": (compress_read + compress_write) / (comp_ms * 1e-3) / 1e9,
                     "read_gb": compress_read / 1e9, "write_gb": compress_write / 1e9},
    }

    # ------------------------------------------------------------------ append alone: latency-bound, reported in us
    compress_all()
    sync_all()
    a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
    a.record()
    for t in range(T):
        k_new, v_new = kvs[t % n_q]
        for l in range(L):
            cache.append(l, k_new, v_new)
    b.record()
    sync_all()
    app_us = a.elapsed_time(b) * 1e3 / (T * L)
    # decode attention alone, back to back over the layers (every call streams pages the L2 no longer holds)
    reps = max(1, 80 // L)
    for l in range(L):
        cache.decode(l, qs[0], out)
    sync_all()
    a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(reps * L):
        cache.decode(i % L, qs[i % n_q], out)
    b.record()
    sync_all()
    dec_alone_us = a.elapsed_time(b) * 1e3 / (reps * L)
    kept_now = statistics.mean(compressed_bytes(w, l, extra=T) for l in range(L))
    line["decode"]["us_per_layer_back_to_back_no_append"] = dec_alone_us
    line["decode"]["gbs_back_to_back_no_append"] = kept_now / (dec_alone_us * 1e-6) / 1e9
    # the same step as two calls (razor_append, then razor_decode_attention)
    a.record()
    for t in range(2):
        for l in range(L):
            cache.append(l, kvs[t % n_q][0], kvs[t % n_q][1])
            cache.decode(l, qs[t % n_q], out)
    b.record()
    sync_all()
    line["decode"]["us_per_layer_as_two_calls"] = a.elapsed_time(b) * 1e3 / (2 * L)
    line["append"] = {"us_per_layer_in_pass": us_per_launch - dec_alone_us,
                      "us_per_call_back_to_back": app_us, "launches_timed": T * L,
                      "note": "in the pass: a razor_decode_step call minus a razor_decode_attention call timed back to back "
                              "without appends; back to back: razor_append calls alone, one token per (sequence, KV "
                              "head), bound by the host's launch rate"}

    # ------------------------------------------------------------------ dense full-cache decode, same GPU
    if not args.no_dense and rank == 0 and not per_seq:
        try:
            cfg_d = rz.make_config(w.batch, 1, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, w.n_sink,
                                   max(w.ctx_len), 1)
            all_r = np.ones(w.n_kv_heads, dtype=np.uint8)
            dcache = rz.RazorCache(cfg_d, w.ctx_len, w.window, all_r, device=dev)
            dcache.compress(0, Kd, Vd, w.ctx_len, all_r, w.window)
            for _ in range(3):
                dcache.decode(0, qs[0], out)
            torch.cuda.synchronize()
            reps = 5
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(reps):
                dcache.decode(0, qs[i % n_q], out)
            b.record()
            torch.cuda.synchronize()
            d_us = a.elapsed_time(b) * 1e3 / reps
            line["dense_decode"] = {"us_per_layer": d_us, "gbs": dense_bytes(w) / (d_us * 1e-6) / 1e9,
                                    "us_per_decode_step": d_us * L,
                                    "speedup_compressed_vs_dense": d_us / us_per_launch}
            dcache.close()
            del dcache
        except Exception as ex:   # e.g. not enough memory for a dense layer beside the compressed stack
            line["dense_decode"] = {"unavailable": str(ex)[:200]}

    # ------------------------------------------------------------------ the 128K grouped-query shape, decode only
    if not args.no_dense and rank == 0 and args.workload == "cfg3" and not args.layers:
        try:
            line["decode_128k_gqa"] = decode_only(rz, synth, "cfg4", 32, dev, peak, reps=96, with_append=True)
        except Exception as ex:
            line["decode_128k_gqa"] = {"unavailable": str(ex)[:200]}
        try:   # retrieval-head identification scores (Section 3.3)
            line["head_scores"] = head_scores_leg(rz, synth, dev)
        except Exception as ex:
            line["head_scores"] = {"unavailable": str(ex)[:200]}
        try:   # a cfg3 layer built chunk by chunk from an empty one (chunked prefill)
            line["chunked_prefill"] = chunked_prefill_leg(rz, synth, dev, peak)
        except Exception as ex:
            line["chunked_prefill"] = {"unavailable": str(ex)[:200]}
        try:   # the ALiBi variant on the 32K MHA shape
            line["alibi_32k"] = decode_only(rz, synth, "cfg2", 3, dev, peak, alibi=True)
        except Exception as ex:
            line["alibi_32k"] = {"unavailable": str(ex)[:200]}
        try:   # a 512-token round (follow-up prompt) on the 32K MHA shape: the query-tiled kernel
            line["round_of_512_tokens_32k"] = long_round_leg(rz, synth, dev)
        except Exception as ex:
            line["round_of_512_tokens_32k"] = {"unavailable": str(ex)[:200]}
        try:   # a 32-token round (a short user turn): more rows than one launch of the streaming kernel takes, so the
            # query-tiled kernel as well, most of whose 128 rows are then no query
            line["round_of_32_tokens_32k"] = long_round_leg(rz, synth, dev, n_tok=32)
        except Exception as ex:
            line["round_of_32_tokens_32k"] = {"unavailable": str(ex)[:200]}
        try:   # a 4-token round (verify step) on the 32K MHA shape: same pages streamed, four queries per head
            line["round_of_4_tokens_32k"] = decode_only(rz, synth, "cfg2", 3, dev, peak, n_tok=4)
        except Exception as ex:
            line["round_of_4_tokens_32k"] = {"unavailable": str(ex)[:200]}

    # ------------------------------------------------------------------ end to end with HOST buffers
    if not args.no_e2e:
        e2e_steps = max(1, min(args.steps, 2))
        if per_seq:
            host_dense = None
        else:
            host_dense = (torch.empty(Kd.shape, dtype=tdt, pin_memory=True), torch.empty(Vd.shape, dtype=tdt, pin_memory=True))
            host_dense[0].copy_(Kd); host_dense[1].copy_(Vd)
        h_q = [x.cpu().pin_memory() for x in qs]
        h_kv = [(a.cpu().pin_memory(), b.cpu().pin_memory()) for a, b in kvs]
        h_out = torch.empty(out.shape, dtype=torch.float32, pin_memory=True)
        d_q = torch.empty_like(qs[0]); d_k = torch.empty_like(kvs[0][0]); d_v = torch.empty_like(kvs[0][1])
        h2d = d2h = 0

        def e2e_pass(count=False):
            nonlocal h2d, d2h
            for l in range(L):
                if per_seq:
                    for b in range(w.batch):
                        cache.compress_seq(l, b, dense[b][0], dense[b][1], w.ctx_len[b], retr[l], w.window[b])
                else:
                    Kd.copy_(host_dense[0], non_blocking=True)
                    Vd.copy_(host_dense[1], non_blocking=True)
                    if count:
                        h2d += 2 * Kd.numel() * Kd.element_size()
                    cache.compress(l, Kd, Vd, w.ctx_len, retr[l], w.window)
            for t in range(T):
                for l in range(L):
                    d_q.copy_(h_q[t % n_q], non_blocking=True)
                    d_k.copy_(h_kv[t % n_q][0], non_blocking=True)
                    d_v.copy_(h_kv[t % n_q][1], non_blocking=True)
                    cache.decode_step(l, d_k, d_v, d_q, out)
                    h_out.copy_(out, non_blocking=True)
                    if count:
                        h2d += (d_q.numel() + 2 * d_k.numel()) * d_q.element_size()
                        d2h += out.numel() * 4
            torch.cuda.current_stream().synchronize()

        e2e_pass()
        sync_all()
        t0 = time.perf_counter()
        a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(e2e_steps):
            e2e_pass(count=(i == 0))
        b.record()
        sync_all()
        e_ms = max_over_ranks(a.elapsed_time(b) / e2e_steps, dist, dev)
        line["e2e"] = {"value": replica_throughput(world, attended, e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
                       "d2h_bytes_per_step": d2h, "ms_per_step": e_ms, "steps": e2e_steps,
                       "note": "host-pinned dense K/V, q, k_new, v_new copied in and out[] copied back inside the "
                               "timed region" + ("; cfg5 dense K/V stay on the device (75 GB of host staging "
                                                 "does not fit the time budget)" if per_seq else "")}
        del host_dense

    # ------------------------------------------------------------------ CPU oracle on the host cores
    if not args.no_cpu_baseline and rank == 0:
        v, desc, threads, _ = oracle_sample(synth.workload(args.workload))
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc}

    cache.close()
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
