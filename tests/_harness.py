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


def sample_heads(w: synth.Workload, layer: int, n_retr: int, n_other: int, batches: Sequence[int]) -> List[Tuple[int, int]]:
    r = w.retrieval(layer)
    ret = [g for g in range(w.n_kv_heads) if r[g]][:n_retr]
    oth = [g for g in range(w.n_kv_heads) if not r[g]]
    step = max(1, len(oth) // max(1, n_other))
    oth = oth[::step][:n_other]
    return [(b, g) for b in batches for g in ret + oth]


def run_parity(w: synth.Workload, *, layers: Optional[Sequence[int]] = None,
               heads_for: Optional[Dict[int, List[Tuple[int, int]]]] = None, steps: Optional[int] = None,
               shuffle: int = 0, use_comp: int = 1, sm_scale: float = 0.0, per_seq: bool = False,
               check_layout_every: int = 0, device="cuda:0", stats: Optional[dict] = None,
               options: Optional[Dict[int, int]] = None) -> dict:
    """Compress every layer, then run `steps` x (append, decode) over all layers on the GPU, checking
    the heads listed in heads_for[layer] (default: every head of every layer) against the oracle.
    With steps == 0 one decode is run straight after compression (no append)."""
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
                if steps > 0:
                    k_new, v_new = synth.make_new_kv(w, l, t, dev)
                    cache.append(l, k_new, v_new)
                q = synth.make_queries(w, l, t, dev)
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
