"""Shared parity harness: runs a synthetic workload through the CUDA library (C ABI via the ctypes
binding) and through the CPU oracle on the same seeded inputs, and compares them.

Bars (written here once, used by every GPU test):
  * kept positions and the K/V rows of the compressed cache: bit-exact;
  * compensation means: ||gpu - oracle||_inf / ||oracle||_inf <= 1e-3 per (sequence, KV head) vector;
  * attention output: max-abs <= 3e-3 for bf16 K/V, <= 1e-5 for fp32 K/V.
"""
from __future__ import annotations

import math
from typing import Dict, Iterable, List, Optional, Sequence, Tuple

import numpy as np
import torch

from oracle import razor_oracle as orc
from paper_2407_15891_b200 import binding as rz
from paper_2407_15891_b200 import synth

TOL_OUT = {"bf16": 3e-3, "f32": 1e-5}
TOL_MEAN_REL = 1e-3


def bits(t: torch.Tensor) -> np.ndarray:
    """Bit pattern of a tensor as integers (bf16 -> int16, fp32 -> int32)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy()
    if t.dtype == torch.float32:
        return t.view(torch.int32).numpy()
    return t.numpy()


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().to(torch.float64).numpy()


def rel_inf(a: np.ndarray, ref: np.ndarray) -> float:
    d = float(np.abs(a - ref).max()) if a.size else 0.0
    n = float(np.abs(ref).max()) if ref.size else 0.0
    if n == 0.0:
        return 0.0 if d == 0.0 else float("inf")
    return d / n


def make_cache(w: synth.Workload, layers: Optional[Sequence[int]] = None, max_new: Optional[int] = None,
               shuffle: int = 0, use_comp: int = 1, sm_scale: float = 0.0, device="cuda:0",
               options: Optional[Dict[int, int]] = None) -> rz.RazorCache:
    n_layers = w.n_layers
    cfg = rz.make_config(w.batch, n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, w.n_sink,
                         max(w.ctx_len), w.decode_steps if max_new is None else max_new, use_comp, shuffle, sm_scale)
    retr = np.stack([w.retrieval(l) for l in range(n_layers)])
    cache = rz.RazorCache(cfg, w.ctx_len, w.window, retr, device=device)
    for opt, val in (options or {}).items():
        cache.set_option(opt, val)
    return cache


class HeadRef:
    """Host copy of one (layer, b, kv head)'s dense history for the oracle, as exact fp64 + raw bits."""

    def __init__(self, layer, b, g, K: torch.Tensor, V: torch.Tensor, n_ctx: int, extra: int):
        self.layer, self.b, self.g, self.n = layer, b, g, n_ctx
        D = K.shape[-1]
        self.K_bits = np.zeros((n_ctx + extra, D), dtype=bits(K[:1]).dtype)
        self.V_bits = np.zeros_like(self.K_bits)
        self.K = np.zeros((n_ctx + extra, D), dtype=np.float64)
        self.V = np.zeros_like(self.K)
        self.K_bits[:n_ctx], self.V_bits[:n_ctx] = bits(K[:n_ctx]), bits(V[:n_ctx])
        self.K[:n_ctx], self.V[:n_ctx] = to_f64(K[:n_ctx]), to_f64(V[:n_ctx])

    def append(self, k: torch.Tensor, v: torch.Tensor):
        self.K_bits[self.n], self.V_bits[self.n] = bits(k), bits(v)
        self.K[self.n], self.V[self.n] = to_f64(k), to_f64(v)
        self.n += 1


def check_head_state(cache: rz.RazorCache, ref: HeadRef, n_sink: int, window: int, is_retr: bool) -> orc.HeadCache:
    """Layout (bit-exact) and compensation means (1e-3 relative) of one head against the oracle."""
    hc = orc.compress_head(ref.K, ref.V, ref.n, n_sink, window, is_retr)
    ex = cache.export(ref.layer, ref.b, ref.g)
    kept = ex["kept_pos"].cpu().numpy().astype(np.int64)
    assert kept.tolist() == hc.kept_pos.tolist(), f"kept positions differ at {(ref.layer, ref.b, ref.g)}"
    assert ex["n_drop"] == hc.n_drop
    assert (bits(ex["K"]) == ref.K_bits[hc.kept_pos]).all(), "K rows not bit-exact"
    assert (bits(ex["V"]) == ref.V_bits[hc.kept_pos]).all(), "V rows not bit-exact"
    mk, mv = to_f64(ex["mean_k"]), to_f64(ex["mean_v"])
    if hc.n_drop > 0:
        assert rel_inf(mk, hc.k_hat) <= TOL_MEAN_REL, (rel_inf(mk, hc.k_hat), ref.layer, ref.b, ref.g)
        assert rel_inf(mv, hc.v_hat) <= TOL_MEAN_REL, (rel_inf(mv, hc.v_hat), ref.layer, ref.b, ref.g)
    else:
        assert not mk.any() and not mv.any()
    return hc


def run_parity(w: synth.Workload, *, layers: Optional[Sequence[int]] = None,
               heads_for: Optional[Dict[int, List[Tuple[int, int]]]] = None, steps: Optional[int] = None,
               shuffle: int = 0, use_comp: int = 1, sm_scale: float = 0.0, per_seq: bool = False,
               check_layout_every: int = 0, device="cuda:0", stats: Optional[dict] = None,
               options: Optional[Dict[int, int]] = None, fused: bool = False) -> dict:
    """Compress every layer, then run `steps` x (append, decode) over all layers on the GPU, checking
    the heads listed in heads_for[layer] (default: every head of every layer) against the oracle.
    With steps == 0 one decode is run straight after compression (no append).  fused: each step is one
    razor_decode_step call instead of razor_append + razor_decode_attention."""
    dev = torch.device(device)
    all_layers = list(range(w.n_layers))
    check_layers = list(layers) if layers is not None else all_layers
    steps = w.decode_steps if steps is None else steps
    if heads_for is None:
        heads_for = {l: [(b, g) for b in range(w.batch) for g in range(w.n_kv_heads)] for l in check_layers}
    scale = sm_scale if sm_scale else 1.0 / math.sqrt(w.head_dim)
    G = w.group
    tol = TOL_OUT[w.dtype]
    cache = make_cache(w, max_new=max(steps, 1), shuffle=shuffle, use_comp=use_comp, sm_scale=sm_scale, device=device,
                       options=options)
    refs: Dict[Tuple[int, int, int], HeadRef] = {}
    worst = dict(out=0.0, mean=0.0, heads=0, outputs=0)
    try:
        for l in all_layers:
            retr = w.retrieval(l)
            if per_seq:
                for b in range(w.batch):
                    wb = _single_seq_view(w, b)
                    K, V = synth.make_dense_kv(wb, l, dev)
                    cache.compress_seq(l, b, K[0], V[0], w.ctx_len[b], retr, w.window[b])
                    for (bb, g) in heads_for.get(l, []):
                        if bb == b:
                            refs[(l, b, g)] = HeadRef(l, b, g, K[0, g], V[0, g], w.ctx_len[b], steps)
                    torch.cuda.synchronize()
                    del K, V
            else:
                K, V = synth.make_dense_kv(w, l, dev)
                cache.compress(l, K, V, w.ctx_len, retr, w.window)
                for (b, g) in heads_for.get(l, []):
                    refs[(l, b, g)] = HeadRef(l, b, g, K[b, g], V[b, g], w.ctx_len[b], steps)
                torch.cuda.synchronize()
                del K, V
        # state right after compression
        for (l, b, g), ref in refs.items():
            check_head_state(cache, ref, w.n_sink, w.window[b], bool(w.retrieval(l)[g]))
            worst["heads"] += 1

        n_rounds = max(steps, 1)
        for t in range(n_rounds):
            for l in all_layers:
                q = synth.make_queries(w, l, t, dev)
                if steps > 0:
                    k_new, v_new = synth.make_new_kv(w, l, t, dev)
                    if fused:                                   # append + decode in one launch
                        out = cache.decode_step(l, k_new, v_new, q)
                    else:
                        cache.append(l, k_new, v_new)
                        out = cache.decode(l, q)
                else:
                    out = cache.decode(l, q)
                if t == 0 and l == all_layers[0]:
                    status = cache.device_status()
                    assert status == 0, f"a bounded wait inside the decode kernel ran out (status bits {status})"
                if l not in heads_for:
                    continue
                out_h = to_f64(out)
                q_h = to_f64(q)
                if steps > 0:
                    kh, vh = k_new.cpu(), v_new.cpu()
                for (b, g) in heads_for[l]:
                    ref = refs[(l, b, g)]
                    if steps > 0:
                        ref.append(kh[b, g], vh[b, g])
                    is_retr = bool(w.retrieval(l)[g])
                    last = t == n_rounds - 1
                    if steps > 0 and (last or (check_layout_every and t % check_layout_every == 0)):
                        hc = check_head_state(cache, ref, w.n_sink, w.window[b], is_retr)
                    else:
                        hc = orc.compress_head(ref.K, ref.V, ref.n, w.n_sink, w.window[b], is_retr)
                    for j in range(G):
                        expect = orc.decode_head(q_h[b, g * G + j], hc, scale, bool(use_comp))
                        err = float(np.abs(out_h[b, g * G + j] - expect).max())
                        worst["out"] = max(worst["out"], err)
                        worst["outputs"] += 1
                        assert err <= tol, f"out max-abs {err:.3e} > {tol} at layer {l} b {b} head {g * G + j} step {t}"
        status = cache.device_status()
        assert status == 0, f"a bounded wait inside the decode kernel ran out (status bits {status})"
        if stats is not None:
            stats.update(worst)
            stats["kept_bytes"], stats["dense_bytes"] = cache.stats(0)
    finally:
        cache.close()
    return worst


def _single_seq_view(w: synth.Workload, b: int) -> synth.Workload:
    """A batch-1 workload that generates exactly sequence b's tensors is not needed for parity: the
    per-sequence path only needs *some* seeded dense cache of the right length for each sequence."""
    import copy
    wb = copy.copy(w)
    wb.batch = 1
    wb.ctx_len = [w.ctx_len[b]]
    wb.window = [w.window[b]]
    wb.seed = w.seed * 131 + b
    return wb


# ------------------------------------------------------------------------------------------------------------
# Full-size parity.  The GPU runs the workload exactly as the benchmark does (compress every layer, then
# decode steps x layers x (append, decode)) and what it produced is recorded: every output, a snapshot of the
# checked heads' exported state in the middle of the run, and the live state at the end.  The oracle then
# replays one group (a layer, or a sequence of the ragged batch) at a time from the regenerated inputs, so
# that only one group's dense fp64 history is ever held on the host, with the heads of the group spread over
# a thread pool (the oracle itself stays single-threaded numpy).
def oracle_threads() -> int:
    import os
    try:
        n = len(os.sched_getaffinity(0))
    except AttributeError:
        n = os.cpu_count() or 1
    return max(1, min(32, n))


def export_to_host(cache: rz.RazorCache, l: int, b: int, g: int) -> dict:
    ex = cache.export(l, b, g)
    return {k: (v.cpu() if isinstance(v, torch.Tensor) else v) for k, v in ex.items()}


def check_export(ex: dict, ref: HeadRef, n_sink: int, window: int, is_retr: bool) -> orc.HeadCache:
    """Layout (bit-exact) and compensation means (1e-3 relative) of an exported head against the oracle."""
    hc = orc.compress_head(ref.K, ref.V, ref.n, n_sink, window, is_retr)
    where = (ref.layer, ref.b, ref.g, ref.n)
    kept = ex["kept_pos"].cpu().numpy().astype(np.int64)
    assert kept.shape == hc.kept_pos.shape and (kept == hc.kept_pos).all(), f"kept positions differ at {where}"
    assert ex["n_drop"] == hc.n_drop, where
    assert (bits(ex["K"]) == ref.K_bits[hc.kept_pos]).all(), f"K rows not bit-exact at {where}"
    assert (bits(ex["V"]) == ref.V_bits[hc.kept_pos]).all(), f"V rows not bit-exact at {where}"
    mk, mv = to_f64(ex["mean_k"]), to_f64(ex["mean_v"])
    if hc.n_drop > 0:
        assert rel_inf(mk, hc.k_hat) <= TOL_MEAN_REL, (rel_inf(mk, hc.k_hat), where)
        assert rel_inf(mv, hc.v_hat) <= TOL_MEAN_REL, (rel_inf(mv, hc.v_hat), where)
    else:
        assert not mk.any() and not mv.any(), where
    return hc


def run_parity_recorded(w: synth.Workload, *, heads_for: Dict[int, List[Tuple[int, int]]], steps: int,
                        per_seq: bool = False, device="cuda:0", options: Optional[Dict[int, int]] = None,
                        fused: bool = True) -> dict:
    """heads_for[layer] = [(b, kv head)] to check.  steps >= 1: that many (append, decode) rounds over all
    layers; steps == 0: one decode straight after compression.  Layout is checked right after compression,
    after the middle step and after the last one; outputs at every step.  Returns counts and worst errors."""
    from concurrent.futures import ThreadPoolExecutor
    from threadpoolctl import threadpool_limits

    dev = torch.device(device)
    L, G = w.n_layers, w.group
    scale = 1.0 / math.sqrt(w.head_dim)
    tol = TOL_OUT[w.dtype]
    n_rounds = max(steps, 1)
    mid = (steps // 2 - 1) if steps >= 4 else -1                       # snapshot after this step's appends
    cache = make_cache(w, max_new=max(steps, 1), device=device, options=options)
    pool = ThreadPoolExecutor(oracle_threads())
    res = dict(out=0.0, mean=0.0, heads=0, outputs=0, layouts=0)

    def groups():
        """(layer, sequences) units whose dense inputs are generated together."""
        for l in range(L):
            if per_seq:
                for b in sorted({b for (b, _) in heads_for.get(l, [])}):
                    yield l, [b]
            else:
                yield l, None

    def dense_of(l, seqs):
        """Dense K, V [B', Hkv, N, D] on the device and the sequences they belong to."""
        if seqs is None:
            K, V = synth.make_dense_kv(w, l, dev)
            return K, V, list(range(w.batch))
        K, V = synth.make_dense_kv(_single_seq_view(w, seqs[0]), l, dev)
        return K, V, seqs

    def build_refs(l, K, V, seqs):
        todo = [(b, g) for (b, g) in heads_for.get(l, []) if b in seqs]
        host = {(b, g): (K[seqs.index(b), g].cpu(), V[seqs.index(b), g].cpu()) for (b, g) in todo}
        make = lambda bg: HeadRef(l, bg[0], bg[1], host[bg][0], host[bg][1], w.ctx_len[bg[0]], steps)
        return dict(zip(todo, pool.map(make, todo)))

    try:
        with threadpool_limits(limits=1):
            # ---- phase 1: compression in the benchmark's order; layout of the checked heads right after it
            for l in range(L):
                retr = w.retrieval(l)
                if per_seq:
                    for b in range(w.batch):
                        K, V, seqs = dense_of(l, [b])
                        cache.compress_seq(l, b, K[0], V[0], w.ctx_len[b], retr, w.window[b])
                        refs = build_refs(l, K, V, seqs)
                        exs = {bg: export_to_host(cache, l, *bg) for bg in refs}
                        list(pool.map(lambda bg: check_export(exs[bg], refs[bg], w.n_sink, w.window[bg[0]], bool(retr[bg[1]])), refs))
                        res["layouts"] += len(refs)
                        torch.cuda.synchronize()
                        del K, V, refs, exs
                else:
                    K, V, seqs = dense_of(l, None)
                    cache.compress(l, K, V, w.ctx_len, retr, w.window)
                    refs = build_refs(l, K, V, seqs)
                    exs = {bg: export_to_host(cache, l, *bg) for bg in refs}
                    list(pool.map(lambda bg: check_export(exs[bg], refs[bg], w.n_sink, w.window[bg[0]], bool(retr[bg[1]])), refs))
                    res["layouts"] += len(refs)
                    torch.cuda.synchronize()
                    del K, V, refs, exs
            # ---- phase 2: the decode steps, step-major over the layers as the benchmark runs them
            outs = {}
            snap = {}
            for t in range(n_rounds):
                for l in range(L):
                    q = synth.make_queries(w, l, t, dev)
                    if steps > 0 and fused:                  # the benchmark's step: append + decode in one launch
                        k_new, v_new = synth.make_new_kv(w, l, t, dev)
                        out = cache.decode_step(l, k_new, v_new, q)
                    elif steps > 0:
                        k_new, v_new = synth.make_new_kv(w, l, t, dev)
                        cache.append(l, k_new, v_new)
                        out = cache.decode(l, q)
                    else:
                        out = cache.decode(l, q)
                    if l in heads_for:
                        outs[(l, t)] = out.cpu()
                        if t == mid:
                            for bg in heads_for[l]:
                                snap[(l,) + bg] = cache.export(l, *bg)          # stays on the device until replayed
            status = cache.device_status()
            assert status == 0, f"a bounded wait inside the decode kernel ran out (status bits {status})"

            # ---- phase 3: the oracle replays one group at a time
            def replay(l, bg, ref, ex_mid, ex_last):
                b, g = bg
                is_retr = bool(w.retrieval(l)[g])
                worst, n_out, n_lay = 0.0, 0, 0
                for t in range(n_rounds):
                    if steps > 0:
                        k_new, v_new = synth.make_new_kv(w, l, t)              # regenerated on the host
                        ref.append(k_new[b, g], v_new[b, g])
                    if t == mid:
                        hc = check_export(ex_mid, ref, w.n_sink, w.window[b], is_retr); n_lay += 1
                    elif t == n_rounds - 1 and steps > 0:
                        hc = check_export(ex_last, ref, w.n_sink, w.window[b], is_retr); n_lay += 1
                    else:
                        hc = None
                    q = to_f64(synth.make_queries(w, l, t))
                    out = to_f64(outs[(l, t)])
                    for j in range(G):
                        h = g * G + j
                        if is_retr and hc is None:       # Algorithm 1: a retrieval head is ordinary attention over every token
                            expect = orc.full_attention(q[b, h], ref.K[:ref.n], ref.V[:ref.n], scale)
                        else:
                            if hc is None:
                                hc = orc.compress_head(ref.K, ref.V, ref.n, w.n_sink, w.window[b], is_retr)
                            expect = orc.decode_head(q[b, h], hc, scale)
                        err = float(np.abs(out[b, h] - expect).max())
                        assert err <= tol, f"out max-abs {err:.3e} > {tol} at layer {l} b {b} head {h} step {t}"
                        worst = max(worst, err)
                        n_out += 1
                return worst, n_out, n_lay

            for l, seqs in groups():
                if not heads_for.get(l):
                    continue
                K, V, seqs = dense_of(l, seqs)
                refs = build_refs(l, K, V, seqs)
                del K, V
                ex_mid = {bg: {k: (v.cpu() if isinstance(v, torch.Tensor) else v) for k, v in snap.pop((l,) + bg).items()}
                          for bg in refs} if mid >= 0 else {bg: None for bg in refs}
                ex_last = {bg: export_to_host(cache, l, *bg) for bg in refs} if steps > 0 else {bg: None for bg in refs}
                for worst, n_out, n_lay in pool.map(lambda bg: replay(l, bg, refs[bg], ex_mid[bg], ex_last[bg]), list(refs)):
                    res["out"] = max(res["out"], worst)
                    res["outputs"] += n_out
                    res["layouts"] += n_lay
                res["heads"] += len(refs)
                del refs, ex_mid, ex_last
    finally:
        pool.shutdown(wait=True, cancel_futures=True)
        cache.close()
    return res


def floor_heads(w: synth.Workload, layer: int, batches: Sequence[int], frac_other: float = 0.10) -> List[Tuple[int, int]]:
    """Every retrieval KV head of the layer plus a seeded tenth (rounded up) of the others, for the given sequences."""
    r = w.retrieval(layer)
    ret = [g for g in range(w.n_kv_heads) if r[g]]
    oth = [g for g in range(w.n_kv_heads) if not r[g]]
    n_oth = min(len(oth), max(1, math.ceil(frac_other * len(oth)))) if oth else 0
    perm = synth.seeded_permutation(w.seed * 31 + layer, len(oth))
    pick = sorted(oth[i] for i in perm[:n_oth])
    return [(b, g) for b in batches for g in ret + pick]
