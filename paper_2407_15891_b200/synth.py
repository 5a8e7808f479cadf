"""Seeded synthetic inputs shaped like the paper's long-context workloads.

This module holds NONE of the method's arithmetic: it only produces dense K/V
caches, queries, retrieval-head masks, context lengths and windows.  It serves
both the CUDA path (tests, bench) and the CPU oracle's tests, so that both see
bit-identical inputs.

Generator.  Every tensor element is a function of (seed, tag, flat index) only:
a splitmix64 hash of the 4-element group index is cut into four 16-bit lanes,
and each lane indexes a 65536-entry table holding the standard normal quantiles
Phi^-1((i + 0.5) / 65536) rounded to bf16.  The table is computed once on the
host in fp64; hashing and the table lookup are integer operations, so the result
is bit-identical on CPU and on CUDA tensors.  Values are therefore ~N(0,1),
exactly representable in bf16 (and in fp32 for the fp32 configuration).

Workload structure (Section 3.2-3.3, Table 2 of the paper, and the evaluation
models it names): about 15 % of the heads are retrieval heads, 4 attention-sink
tokens at the start of the context (given 4x key norm here), recent-window
length max(4000, N/5), and "needle" keys aligned with the query so that a head
that still holds them recalls their values.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np
import torch

_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_MIX1 = 0xBF58476D1CE4E5B9
_MIX2 = 0x94D049BB133111EB

# tensor tags (mixed into the hash so that K, V, q, ... are independent streams)
TAG_K, TAG_V, TAG_Q, TAG_KNEW, TAG_VNEW, TAG_MISC = 1, 2, 3, 4, 5, 6


def _s64(x: int) -> int:
    """Python int (mod 2^64) -> the signed value torch.int64 holds for it."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def splitmix64_int(x: int) -> int:
    """splitmix64 finaliser on a Python int (host scalars: seeds, positions)."""
    z = (x + _GOLDEN) & _M64
    z = ((z ^ (z >> 30)) * _MIX1) & _M64
    z = ((z ^ (z >> 27)) * _MIX2) & _M64
    return z ^ (z >> 31)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of int64 (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _splitmix64_t(x: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser on an int64 tensor, wrap-around arithmetic."""
    z = x + _s64(_GOLDEN)
    z = (z ^ _lsr(z, 30)) * _s64(_MIX1)
    z = (z ^ _lsr(z, 27)) * _s64(_MIX2)
    return z ^ _lsr(z, 31)


_TABLE_CACHE: dict = {}


def normal_table(device: torch.device | str = "cpu") -> torch.Tensor:
    """65536 standard-normal quantiles, rounded to bf16 (computed on the host in fp64)."""
    key = str(device)
    if key not in _TABLE_CACHE:
        if "cpu" not in _TABLE_CACHE:
            p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
            _TABLE_CACHE["cpu"] = torch.special.ndtri(p).to(torch.bfloat16)
        if key != "cpu":
            _TABLE_CACHE[key] = _TABLE_CACHE["cpu"].to(device)
    return _TABLE_CACHE[key]


def stream_key(seed: int, tag: int, sub: int = 0) -> int:
    """Per-tensor hash key from (seed, tag, sub-stream id)."""
    return splitmix64_int(splitmix64_int(seed) ^ (tag * _MIX1 & _M64) ^ (sub * _MIX2 & _M64))


def normal_bf16(seed: int, tag: int, shape: Sequence[int], device="cpu", sub: int = 0,
                out: Optional[torch.Tensor] = None, chunk: int = 1 << 26, offset: int = 0) -> torch.Tensor:
    """Tensor of N(0,1) values rounded to bf16; element i depends on (seed, tag, sub, offset + i) only.

    `offset` (a multiple of 4) selects a window of a larger virtual tensor, so that one head of a
    layer can be generated without the rest.
    """
    assert offset % 4 == 0
    n = int(np.prod(shape)) if len(shape) else 1
    dev = torch.device(device)
    if out is None:
        out = torch.empty(n, dtype=torch.bfloat16, device=dev)
    flat = out.view(-1)
    assert flat.numel() == n and flat.dtype == torch.bfloat16
    table = normal_table(dev)
    key = _s64(stream_key(seed, tag, sub))
    shifts = torch.tensor([0, 16, 32, 48], dtype=torch.int64, device=dev)
    for start in range(0, n, chunk):
        stop = min(n, start + chunk)
        g0, g1 = (offset + start) >> 2, (offset + stop + 3) >> 2
        g = torch.arange(g0, g1, dtype=torch.int64, device=dev)
        h = _splitmix64_t(g ^ key)
        lanes = ((h.unsqueeze(1) >> shifts) & 0xFFFF).reshape(-1)
        vals = table[lanes]
        lo = offset + start - (g0 << 2)
        flat[start:stop] = vals[lo:lo + (stop - start)]
    return out.view(*shape)


def seeded_permutation(seed: int, n: int) -> List[int]:
    """Fisher-Yates shuffle of range(n) driven by splitmix64."""
    perm = list(range(n))
    state = splitmix64_int(seed)
    for i in range(n - 1, 0, -1):
        state = splitmix64_int(state)
        j = state % (i + 1)
        perm[i], perm[j] = perm[j], perm[i]
    return perm


def retrieval_mask(seed: int, layer: int, n_heads: int, n_retrieval: int) -> np.ndarray:
    """uint8 [n_heads]: 1 for the seeded retrieval heads of this layer."""
    perm = seeded_permutation(seed * 1000003 + 7919 * layer + 17, n_heads)
    m = np.zeros(n_heads, dtype=np.uint8)
    m[perm[:n_retrieval]] = 1
    return m


@dataclass
class Workload:
    """Shape of one synthetic workload (one of the five configurations)."""
    name: str
    batch: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str                      # "bf16" | "f32"
    ctx_len: List[int]              # per sequence
    window: List[int]               # per sequence
    n_sink: int
    n_retrieval_kv: int             # retrieval KV heads per layer
    decode_steps: int
    seed: int
    n_needles: int = 0
    fixed_retrieval: Optional[List[int]] = None
    needle_pos: Optional[List[int]] = None
    notes: str = ""

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def n_max(self) -> int:
        return max(self.ctx_len)

    def retrieval(self, layer: int) -> np.ndarray:
        if self.fixed_retrieval is not None:
            m = np.zeros(self.n_kv_heads, dtype=np.uint8)
            m[self.fixed_retrieval] = 1
            return m
        return retrieval_mask(self.seed, layer, self.n_kv_heads, self.n_retrieval_kv)

    def esz(self) -> int:
        return 2 if self.dtype == "bf16" else 4


def workload(name: str, scale: float = 1.0) -> Workload:
    """The five configurations.  `scale` < 1 shrinks contexts/windows (for quick tests only)."""
    def sc(x: int) -> int:
        return max(1, int(round(x * scale)))

    if name == "cfg1":      # tiny fp32 reference case
        return Workload("cfg1", 1, 1, 4, 4, 64, "f32", [512], [64], 4, 1, 1, 1001,
                        n_needles=1, fixed_retrieval=[0], needle_pos=[200],
                        notes="tiny fp32: head 0 retrieval, needle at 200")
    if name == "cfg2":      # Llama-2-7B-shaped single layer, 32K
        n = sc(32768)
        return Workload("cfg2", 8, 1, 32, 32, 128, "bf16", [n] * 8,
                        [max(sc(4000), n // 5)] * 8, 4, 5, 1, 1002)
    if name == "cfg3":      # Llama-2-13B-64K-shaped full stack
        n = sc(65536)
        return Workload("cfg3", 4, 40, 40, 40, 128, "bf16", [n] * 4, [sc(8192)] * 4, 4, 6, 16, 1003,
                        n_needles=3)
    if name == "cfg4":      # GQA Llama-3-8B-shaped, 128K
        n = sc(131072)
        return Workload("cfg4", 2, 32, 32, 8, 128, "bf16", [n] * 2, [sc(16384)] * 2, 4, 2, 1, 1004)
    if name == "cfg5":      # ragged serving mix
        seed = 1005
        lens = [sc(4096 + splitmix64_int(seed * 65537 + b) % 126977) for b in range(64)]
        return Workload("cfg5", 64, 1, 32, 32, 128, "bf16", lens,
                        [max(sc(4000), n // 5) for n in lens], 4, 5, 64, seed)
    raise KeyError(name)


def torch_dtype(w: Workload) -> torch.dtype:
    return torch.bfloat16 if w.dtype == "bf16" else torch.float32


def make_queries(w: Workload, layer: int, step: int, device="cpu") -> torch.Tensor:
    """q [B, Hq, D] for one decode step of one layer."""
    q = normal_bf16(w.seed, TAG_Q, (w.batch, w.n_q_heads, w.head_dim), device, sub=layer * 100003 + step)
    return q.to(torch_dtype(w))


def make_new_kv(w: Workload, layer: int, step: int, device="cpu"):
    """(k_new, v_new) [B, Hkv, D] appended at decode step `step`."""
    shp = (w.batch, w.n_kv_heads, w.head_dim)
    k = normal_bf16(w.seed, TAG_KNEW, shp, device, sub=layer * 100003 + step)
    v = normal_bf16(w.seed, TAG_VNEW, shp, device, sub=layer * 100003 + step)
    return k.to(torch_dtype(w)), v.to(torch_dtype(w))


def needle_positions(w: Workload, layer: int, b: int, h: int) -> List[int]:
    if w.n_needles == 0:
        return []
    if w.needle_pos is not None:
        return list(w.needle_pos)
    n = w.ctx_len[b]
    base = splitmix64_int(w.seed * 7 + ((layer * 131 + b) * 131 + h))
    out = []
    for i in range(w.n_needles):
        base = splitmix64_int(base + i)
        out.append(w.n_sink + base % max(1, n - w.n_sink))
    return out


def make_dense_kv(w: Workload, layer: int, device="cpu", needle_beta: float = 20.0,
                  out_k: Optional[torch.Tensor] = None, out_v: Optional[torch.Tensor] = None):
    """Dense post-rotary K, V [B, Hkv, N_max, D] of one layer (rows beyond ctx_len[b] are padding).

    Sinks: key rows at positions < n_sink are scaled by 4 (exact in bf16).
    Needles: key = beta * q0 / (sm_scale * |q0|^2), with q0 the step-0 query of the
    first query head of the group, so that its logit is about beta.
    """
    B, H, N, D = w.batch, w.n_kv_heads, w.n_max, w.head_dim
    k = normal_bf16(w.seed, TAG_K, (B, H, N, D), device, sub=layer, out=out_k)
    v = normal_bf16(w.seed, TAG_V, (B, H, N, D), device, sub=layer, out=out_v)
    k[:, :, : w.n_sink, :] *= 4.0
    if w.n_needles:
        q0 = make_queries(w, layer, 0, device).float()          # [B, Hq, D]
        q0 = q0.view(B, H, w.group, D)[:, :, 0, :]              # first q head of each group
        sm_scale = 1.0 / math.sqrt(D)
        needle = (needle_beta * q0 / (sm_scale * (q0 * q0).sum(-1, keepdim=True))).to(torch.bfloat16)
        for b in range(B):
            for h in range(H):
                for p in needle_positions(w, layer, b, h):
                    if p < w.ctx_len[b]:
                        k[b, h, p, :] = needle[b, h]
    if w.dtype == "f32":
        return k.float(), v.float()
    return k, v


def make_dense_head(w: Workload, layer: int, b: int, g: int, device="cpu"):
    """K, V [N_max, D] of one (sequence, KV head): the same values make_dense_kv gives at [b, g],
    generated alone (needle keys excepted: they depend on the queries and are not planted here)."""
    N, D = w.n_max, w.head_dim
    off = ((b * w.n_kv_heads) + g) * N * D
    k = normal_bf16(w.seed, TAG_K, (N, D), device, sub=layer, offset=off)
    v = normal_bf16(w.seed, TAG_V, (N, D), device, sub=layer, offset=off)
    k[: w.n_sink, :] *= 4.0
    if w.dtype == "f32":
        return k.float(), v.float()
    return k, v
