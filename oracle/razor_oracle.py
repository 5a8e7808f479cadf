"""CPU oracle for RazorAttention's hot path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 numpy implementation of what the paper defines: the kept set
of Algorithm 1, the compensation token of Eq. 4, the compensated attention of
Eq. 5 and ordinary softmax attention for retrieval heads.  It exists to check the
CUDA library and to be timed as a CPU baseline.  Only the tests, the smoke check
and the benchmark's cpu-baseline / reference legs may import it; the product
never does.  It shares no code with the CUDA path and imports nothing from it.

Every function names the passage it follows.  There is no blocking, fusion or
reordering here beyond what the definitions state.  Floating point is fp64 after
widening the inputs exactly (bf16 and fp32 both widen exactly to fp64).

Readings taken where the paper is silent (each is also a pinned test):
  * one softmax scale multiplies every logit, the compensation logit included
    (Eq. 3 / Eq. 5 print no 1/sqrt(d); scale = 1 is the literal form);
  * N/C in Algorithm 1 is floored;
  * sinks are the first N0 positions; when N <= N0 + L nothing is dropped and the
    compensation term vanishes (its weight N_d is 0);
  * during decoding the window length stays what it was at compression time, and a
    token leaving the window joins the dropped set, so the state after t appended
    tokens is, by definition, the compression of the (N + t)-token context;
  * grouped-query attention: a KV head is kept in full when any query head of its
    group is a retrieval head (Section 4.1 on Llama-3-8B);
  * a head that holds no token at all (an empty sequence before its first append) has
    nothing to attend to: both sums of Eq. 5 are empty and the output is defined as zeros.

Parity pins: every function below is pinned by tests/test_oracle_pins.py (brute
force, closed forms, library special cases, the paper's 3.125x figure); none is
"parity unpinned".
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np


# --------------------------------------------------------------------------- Algorithm 1
def buffer_length(n_ctx: int, s0: int, c: int) -> int:
    """Algorithm 1 / Table 2: L_h = max(S0, N / C), N / C floored."""
    return max(int(s0), int(n_ctx) // int(c))


def kept_positions(n_ctx: int, n_sink: int, window: int, is_retrieval: bool) -> np.ndarray:
    """Algorithm 1: positions kept by one head, ascending.

    Retrieval heads keep every token.  Any other head keeps the first `n_sink`
    positions and the most recent `window` positions; everything between is dropped.
    """
    n = int(n_ctx)
    if is_retrieval or n <= n_sink + window:
        return np.arange(n, dtype=np.int64)
    head = np.arange(0, n_sink, dtype=np.int64)
    tail = np.arange(n - window, n, dtype=np.int64)
    return np.concatenate([head, tail])


def dropped_positions(n_ctx: int, n_sink: int, window: int, is_retrieval: bool) -> np.ndarray:
    """Algorithm 1: the set {D} of dropped positions (complement of the kept set)."""
    keep = np.zeros(int(n_ctx), dtype=bool)
    keep[kept_positions(n_ctx, n_sink, window, is_retrieval)] = True
    return np.nonzero(~keep)[0].astype(np.int64)


def kv_head_is_retrieval(q_head_flags: Sequence[int], group: int) -> np.ndarray:
    """Section 4.1 (GQA models): a KV group is protected when at least one of its query heads is."""
    f = np.asarray(q_head_flags).astype(bool).reshape(-1, group)
    return f.any(axis=1).astype(np.uint8)


# --------------------------------------------------------------------------- Eq. 4
def compensation_token(K: np.ndarray, V: np.ndarray, dropped: np.ndarray) -> Tuple[np.ndarray, np.ndarray, int]:
    """Eq. 4: k_hat = (1/N_d) sum_{m in D} k_m, v_hat likewise.  K, V are [N, D] of one head.

    Returns (k_hat, v_hat, N_d); both means are zero vectors when nothing is dropped.
    """
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    n_d = int(len(dropped))
    if n_d == 0:
        return np.zeros(K.shape[1]), np.zeros(V.shape[1]), 0
    k_hat = K[dropped].sum(axis=0) / n_d
    v_hat = V[dropped].sum(axis=0) / n_d
    return k_hat, v_hat, n_d


# --------------------------------------------------------------------------- original attention
def full_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float) -> np.ndarray:
    """Softmax attention of one query over all rows of K, V (retrieval heads, Algorithm 1)."""
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    s = scale * (K @ q)
    w = np.exp(s - s.max())
    return (w @ V) / w.sum()


# --------------------------------------------------------------------------- Eq. 5
def compensated_attention(q: np.ndarray, K_kept: np.ndarray, V_kept: np.ndarray,
                          k_hat: np.ndarray, v_hat: np.ndarray, n_d: int, scale: float) -> np.ndarray:
    """Eq. 5: attention over the kept tokens plus the compensation token.

        out = (N_d e^{q.k_hat} v_hat + sum_kept e^{q.k_n} v_n) / (N_d e^{q.k_hat} + sum_kept e^{q.k_n})

    evaluated in the literal product form (N_d multiplies the exponential), with one
    common maximum subtracted from all logits for range.
    """
    q = np.asarray(q, dtype=np.float64)
    K_kept = np.asarray(K_kept, dtype=np.float64)
    V_kept = np.asarray(V_kept, dtype=np.float64)
    if K_kept.shape[0] == 0 and n_d == 0:
        return np.zeros(V_kept.shape[1])         # nothing to attend to: both sums of Eq. 5 are empty (reading: zeros)
    s = scale * (K_kept @ q)
    if n_d > 0:
        s_c = scale * float(np.dot(q, np.asarray(k_hat, dtype=np.float64)))
        m = max(float(s.max()) if s.size else s_c, s_c)
        w = np.exp(s - m)
        w_c = n_d * np.exp(s_c - m)
        num = w_c * np.asarray(v_hat, dtype=np.float64) + w @ V_kept
        den = w_c + w.sum()
    else:
        m = s.max()
        w = np.exp(s - m)
        num = w @ V_kept
        den = w.sum()
    return num / den


# --------------------------------------------------------------------------- one head, end to end
@dataclass
class HeadCache:
    """Compressed cache of one (sequence, KV head): the paper's {K, k_hat}, {V, v_hat} and N_d."""
    kept_pos: np.ndarray        # int64, ascending original positions
    K: np.ndarray               # [len(kept_pos), D], same dtype/bits as the input rows
    V: np.ndarray
    k_hat: np.ndarray           # fp64 [D]
    v_hat: np.ndarray           # fp64 [D]
    n_drop: int


def compress_head(K: np.ndarray, V: np.ndarray, n_ctx: int, n_sink: int, window: int,
                  is_retrieval: bool) -> HeadCache:
    """Algorithm 1 and Eq. 4 for one head.  K, V: [>= n_ctx, D]; rows >= n_ctx ignored."""
    K = np.asarray(K)[:n_ctx]
    V = np.asarray(V)[:n_ctx]
    kept = kept_positions(n_ctx, n_sink, window, is_retrieval)
    drop = dropped_positions(n_ctx, n_sink, window, is_retrieval)
    k_hat, v_hat, n_d = compensation_token(K, V, drop)
    return HeadCache(kept, K[kept].copy(), V[kept].copy(), k_hat, v_hat, n_d)


def decode_head(q: np.ndarray, hc: HeadCache, scale: float, use_compensation: bool = True) -> np.ndarray:
    """Algorithm 1 for one query head: Eq. 5 (or plain attention when nothing was dropped).

    use_compensation=False gives plain truncation (the scheme of Table 1: recent tokens only).
    """
    n_d = hc.n_drop if use_compensation else 0
    return compensated_attention(q, hc.K, hc.V, hc.k_hat, hc.v_hat, n_d, scale)


# --------------------------------------------------------------------------- a layer (batch of heads)
def compress_layer(K: np.ndarray, V: np.ndarray, ctx_len: Sequence[int], head_is_retrieval: Sequence[int],
                   n_sink: int, window: Sequence[int]) -> List[List[HeadCache]]:
    """Compress dense K, V [B, Hkv, N_max, D]; returns caches[b][g]."""
    B, H = K.shape[0], K.shape[1]
    return [[compress_head(K[b, g], V[b, g], int(ctx_len[b]), n_sink, int(window[b]),
                           bool(head_is_retrieval[g])) for g in range(H)] for b in range(B)]


def decode_layer(q: np.ndarray, caches: List[List[HeadCache]], scale: float,
                 use_compensation: bool = True) -> np.ndarray:
    """q [B, Hq, D] -> out [B, Hq, D] fp64.  Query head j reads KV head j // group."""
    B, Hq, D = q.shape
    Hkv = len(caches[0])
    group = Hq // Hkv
    out = np.zeros((B, Hq, D), dtype=np.float64)
    for b in range(B):
        for j in range(Hq):
            out[b, j] = decode_head(q[b, j], caches[b][j // group], scale, use_compensation)
    return out


# --------------------------------------------------------------------------- decoding with appends
class DenseHistory:
    """Dense history of one (sequence, KV head); appending never updates anything incrementally.

    After every appended token the compressed state is recomputed from the definition
    on the whole (N + t)-token history with the window length fixed at compression time.
    """

    def __init__(self, K: np.ndarray, V: np.ndarray, n_ctx: int, n_sink: int, window: int, is_retrieval: bool):
        self.K = [np.asarray(r) for r in np.asarray(K)[:n_ctx]]
        self.V = [np.asarray(r) for r in np.asarray(V)[:n_ctx]]
        self.n_sink, self.window, self.is_retrieval = int(n_sink), int(window), bool(is_retrieval)

    def append(self, k_new: np.ndarray, v_new: np.ndarray) -> None:
        self.K.append(np.asarray(k_new))
        self.V.append(np.asarray(v_new))

    def cache(self) -> HeadCache:
        return compress_head(np.stack(self.K), np.stack(self.V), len(self.K), self.n_sink, self.window,
                             self.is_retrieval)

    def attend(self, q: np.ndarray, scale: float, use_compensation: bool = True) -> np.ndarray:
        return decode_head(q, self.cache(), scale, use_compensation)


# --------------------------------------------------------------------------- accounting (Table 2)
def kept_token_count(n_ctx: int, n_sink: int, window: int, is_retrieval: bool) -> int:
    """Number of cached tokens of one head, counting the compensation token as one token."""
    kept = len(kept_positions(n_ctx, n_sink, window, is_retrieval))
    n_d = n_ctx - kept
    return kept + (1 if n_d > 0 else 0)


def compression_ratio(n_ctx: int, n_heads: int, n_retrieval: int, n_sink: int, s0: int, c: int) -> float:
    """Dense tokens / cached tokens over the heads of one layer under Table 2's settings."""
    w = buffer_length(n_ctx, s0, c)
    cached = n_retrieval * kept_token_count(n_ctx, n_sink, w, True) \
        + (n_heads - n_retrieval) * kept_token_count(n_ctx, n_sink, w, False)
    return n_heads * n_ctx / cached


# --------------------------------------------------------------------------- several new tokens at once
def multi_query_attention(qs: np.ndarray, K_all: np.ndarray, V_all: np.ndarray, n_sink: int, window: int,
                          is_retrieval: bool, scale: float, use_compensation: bool = True) -> np.ndarray:
    """Attention of the LAST T tokens of a sequence, all against the cache as it stands after the T-th one.

    The paper runs Algorithm 1 once on the prompt and is silent on rounds that add several tokens at
    once (a second prompt, a verify step).  Reading taken: the cache holds the compression of the whole
    (N + T)-token history with the window fixed (as for single appends); query t = 0..T-1 sits at
    position N + t and attends, by causality (Section 3.1: n <= m), to the kept tokens at positions
    <= N + t, plus the compensation token of Eq. 4 over every dropped token with its count N_d (Eq. 5).
    All dropped tokens precede every query as long as window >= T, which callers must ensure.

    qs: [T, D]; K_all, V_all: [N + T, D] dense history of one KV head.  Returns [T, D].
    """
    qs = np.asarray(qs, dtype=np.float64)
    T = qs.shape[0]
    total = int(np.asarray(K_all).shape[0])
    hc = compress_head(K_all, V_all, total, n_sink, window, is_retrieval)
    if hc.n_drop > 0:
        assert window >= T, "a query would see the mean of tokens that come after it"
    out = np.zeros((T, qs.shape[1]), dtype=np.float64)
    for t in range(T):
        q_pos = total - T + t
        vis = hc.kept_pos <= q_pos
        n_d = hc.n_drop if use_compensation else 0
        out[t] = compensated_attention(qs[t], np.asarray(hc.K)[vis], np.asarray(hc.V)[vis], hc.k_hat, hc.v_hat, n_d, scale)
    return out


# --------------------------------------------------------------------------- ALiBi heads (Section 3.1)
def alibi_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, positions: np.ndarray, q_pos: int,
                    slope: float, scale: float) -> np.ndarray:
    """Eq. 1: score of the query at position m = q_pos to the key at position n is q.k - l_h (m - n);
    softmax over the given keys (all at positions <= q_pos).  `scale` multiplies q.k only (Eq. 1 prints
    none); the distance penalty is not scaled."""
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    pos = np.asarray(positions, dtype=np.float64)
    s = scale * (K @ q) - slope * (float(q_pos) - pos)
    w = np.exp(s - s.max())
    return (w @ V) / w.sum()


def alibi_decode_head(qs: np.ndarray, K_all: np.ndarray, V_all: np.ndarray, window: int, slope: float,
                      scale: float, n_sink: int = 0) -> np.ndarray:
    """Section 3.1: an ALiBi head keeps only its most recent L_h = `window` tokens (window < 0: all of
    them); the last T tokens of the history are the queries (T = 1: a decode step), each attending with
    Eq. 1 to the kept tokens at positions <= its own.  qs [T, D]; K_all, V_all [N + T, D]."""
    qs = np.asarray(qs, dtype=np.float64)
    T, total = qs.shape[0], int(np.asarray(K_all).shape[0])
    kept = kept_positions(total, n_sink, window if window >= 0 else total, window < 0)
    out = np.zeros_like(qs)
    for t in range(T):
        q_pos = total - T + t
        vis = kept[kept <= q_pos]
        out[t] = alibi_attention(qs[t], np.asarray(K_all)[vis], np.asarray(V_all)[vis], vis, q_pos, slope, scale)
    return out


# --------------------------------------------------------------------------- retrieval-head identification (Section 3.3)
def echo_induction_scores(Q: np.ndarray, K: np.ndarray, period: int, scale: float) -> Tuple[float, float]:
    """Section 3.3 for one head.  The input is `period` random tokens repeated several times; Q, K [N, D] are
    the head's (post-rotary) queries and keys on it.  For the query at position m >= period, the echo
    tokens are the earlier copies of the current token, at m - j*period, and the induction tokens are the
    ones right after them, at m - j*period + 1 (j = 1, 2, ... while the position is >= 0).  The echo
    (induction) score of the head is the causal-softmax attention weight the query puts on its echo
    (induction) tokens, summed over j and averaged over all m >= period."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    n = Q.shape[0]
    echo = induction = 0.0
    for m in range(period, n):
        s = scale * (K[: m + 1] @ Q[m])
        w = np.exp(s - s.max())
        w /= w.sum()
        j = 1
        while m - j * period >= 0:
            echo += w[m - j * period]
            induction += w[m - j * period + 1]
            j += 1
    cnt = max(1, n - period)
    return echo / cnt, induction / cnt


def select_retrieval_heads(echo: Sequence[float], induction: Sequence[float], frac_induction: float = 0.14,
                           frac_echo: float = 0.01) -> np.ndarray:
    """Section 3.3 / Table 2: the retrieval heads are the top 14 % of all heads by induction score plus the
    top 1 % by echo score (counts rounded to the nearest integer, at least one each; ties broken by the
    lower head index).  Returns a uint8 mask over the heads."""
    echo = np.asarray(echo, dtype=np.float64).reshape(-1)
    induction = np.asarray(induction, dtype=np.float64).reshape(-1)
    n = echo.size
    k_i = max(1, int(round(frac_induction * n)))
    k_e = max(1, int(round(frac_echo * n)))
    mask = np.zeros(n, dtype=np.uint8)
    mask[np.argsort(-induction, kind="stable")[:k_i]] = 1
    mask[np.argsort(-echo, kind="stable")[:k_e]] = 1
    return mask
