"""Thin ctypes binding of librazor.so (include/razor.h).  Argument marshalling only.

Every step of the hot path runs in the library's CUDA kernels; torch is used here for device
memory (`torch.empty`, `data_ptr`) and for the current stream.  There is no CPU or PyTorch
fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librazor.so")

RAZOR_F32, RAZOR_BF16 = 0, 1
STATUS = {
    0: "RAZOR_OK", -1: "RAZOR_E_INVALID_ARG", -2: "RAZOR_E_NULL_PTR", -3: "RAZOR_E_UNSUPPORTED_DIM",
    -4: "RAZOR_E_POOL_TOO_SMALL", -5: "RAZOR_E_CAPACITY", -6: "RAZOR_E_NOT_COMPRESSED", -7: "RAZOR_E_CUDA",
    -8: "RAZOR_E_MISALIGNED",
}

# every symbol include/razor.h declares
SYMBOLS = [
    "razor_query_bytes", "razor_cache_create", "razor_compress", "razor_compress_seq", "razor_append",
    "razor_decode_attention", "razor_decode_step", "razor_append_many", "razor_append_plan", "razor_decode_attention_multi", "razor_cache_export", "razor_cache_stats", "razor_schedule_plan",
    "razor_schedule_query", "razor_schedule_combine_heads", "razor_cache_set_option", "razor_cache_device_status", "razor_cache_wait_selftest", "razor_cache_set_alibi", "razor_cache_set_head_windows",
    "razor_compensation_mean_static", "razor_head_scores_scratch_bytes", "razor_head_scores",
    "razor_select_retrieval_heads", "razor_cache_reset", "razor_cache_destroy", "razor_status_string",
    "razor_last_cuda_error", "razor_version",
]


class RazorError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        lib = _lib
        msg = lib.razor_status_string(status).decode() if lib is not None else "?"
        extra = f" (cudaError {lib.razor_last_cuda_error()})" if status == -7 and lib is not None else ""
        super().__init__(f"{where}: {STATUS.get(status, status)}: {msg}{extra}")


class RazorConfig(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("dtype", C.c_int32), ("page_tokens", C.c_int32), ("n_sink", C.c_int32),
        ("max_ctx_len", C.c_int32), ("max_new_tokens", C.c_int32), ("use_compensation", C.c_int32),
        ("page_shuffle_seed", C.c_int32), ("sm_scale", C.c_float),
    ]


_lib: Optional[C.CDLL] = None


def load() -> C.CDLL:
    """Load librazor.so; raises if it has not been built (python -m paper_2407_15891_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2407_15891_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    cfgp = C.POINTER(RazorConfig)
    lib.razor_query_bytes.argtypes = [cfgp, vp, vp, vp, C.POINTER(sz), C.POINTER(sz)]
    lib.razor_cache_create.argtypes = [C.POINTER(vp), cfgp, vp, sz, vp, sz, vp]
    lib.razor_compress.argtypes = [vp, i32, vp, vp, i64, i64, i64, vp, vp, i32, vp, vp]
    lib.razor_compress_seq.argtypes = [vp, i32, i32, vp, vp, i64, i64, i32, vp, i32, i32, vp]
    lib.razor_append.argtypes = [vp, i32, vp, vp, vp]
    lib.razor_decode_attention.argtypes = [vp, i32, vp, vp, vp]
    lib.razor_decode_step.argtypes = [vp, i32, vp, vp, vp, vp, vp]
    lib.razor_append_many.argtypes = [vp, i32, vp, vp, i32, vp]
    lib.razor_append_plan.argtypes = [i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.razor_decode_attention_multi.argtypes = [vp, i32, vp, vp, i32, vp]
    lib.razor_cache_export.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, C.POINTER(i32),
                                       C.POINTER(i32), vp]
    lib.razor_cache_stats.argtypes = [vp, i32, C.POINTER(sz), C.POINTER(sz)]
    lib.razor_schedule_plan.argtypes = [vp, i32, i32, i32, i32, i32, vp, i32, C.POINTER(i32), C.POINTER(i32)]
    lib.razor_cache_set_option.argtypes = [vp, i32, i32]
    lib.razor_cache_device_status.argtypes = [vp, C.POINTER(i32), vp]
    lib.razor_schedule_query.argtypes = [vp, i32, vp, i32, C.POINTER(i32)]
    lib.razor_schedule_combine_heads.argtypes = [vp, i32, vp, i32, C.POINTER(i32)]
    lib.razor_compensation_mean_static.argtypes = [vp, vp, i64, i64, i32, i32, i32, i32, i32, i32, vp, vp,
                                                   C.POINTER(i32), vp]
    lib.razor_cache_wait_selftest.argtypes = [vp, i64, vp]
    lib.razor_cache_set_alibi.argtypes = [vp, vp, vp]
    lib.razor_cache_set_head_windows.argtypes = [vp, i32, vp]
    lib.razor_head_scores_scratch_bytes.argtypes = [i32, i32, C.POINTER(sz)]
    lib.razor_head_scores.argtypes = [vp, vp, i32, i32, i32, i32, i32, C.c_float, vp, vp, vp, sz, vp]
    lib.razor_select_retrieval_heads.argtypes = [vp, vp, i32, C.c_float, C.c_float, vp]
    lib.razor_cache_reset.argtypes = [vp]
    lib.razor_cache_destroy.argtypes = [vp]
    lib.razor_status_string.argtypes = [C.c_int]
    lib.razor_status_string.restype = C.c_char_p
    lib.razor_last_cuda_error.argtypes = []
    lib.razor_version.argtypes = []
    lib.razor_version.restype = C.c_char_p
    for name in SYMBOLS:
        fn = getattr(lib, name)
        if fn.restype is C.c_int and name not in ("razor_status_string", "razor_version"):
            fn.restype = C.c_int
    _lib = lib
    return lib


def _check(status: int, where: str) -> None:
    if status != 0:
        raise RazorError(status, where)


def _i32(a: Sequence[int]) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _u8(a: Sequence[int]) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.uint8))


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return t.data_ptr()
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return int(t)


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    return int(stream) or None


def make_config(batch, n_layers, n_q_heads, n_kv_heads, head_dim, dtype, n_sink, max_ctx_len, max_new_tokens,
                use_compensation=1, page_shuffle_seed=0, sm_scale=0.0, page_tokens=16) -> RazorConfig:
    dt = {torch.float32: RAZOR_F32, torch.bfloat16: RAZOR_BF16, "f32": RAZOR_F32, "bf16": RAZOR_BF16}.get(dtype, dtype)
    return RazorConfig(batch, n_layers, n_q_heads, n_kv_heads, head_dim, dt, page_tokens, n_sink, max_ctx_len,
                       max_new_tokens, use_compensation, page_shuffle_seed, sm_scale)


# ----------------------------------------------------------------------------- the C-ABI calls, same names
def razor_version() -> str:
    return load().razor_version().decode()


def razor_status_string(status: int) -> str:
    return load().razor_status_string(status).decode()


def razor_query_bytes(cfg: RazorConfig, ctx_len, window, head_is_retrieval) -> Tuple[int, int]:
    """-> (pool_bytes, workspace_bytes).  head_is_retrieval: [L*Hkv] (or [L, Hkv])."""
    a, w, r = _i32(ctx_len), _i32(window), _u8(np.asarray(head_is_retrieval).reshape(-1))
    pool, ws = C.c_size_t(0), C.c_size_t(0)
    _check(load().razor_query_bytes(C.byref(cfg), a.ctypes.data, w.ctypes.data, r.ctypes.data, C.byref(pool),
                                    C.byref(ws)), "razor_query_bytes")
    return pool.value, ws.value


def razor_cache_create(cfg: RazorConfig, pool, pool_bytes: int, workspace, workspace_bytes: int, stream=None) -> int:
    h = C.c_void_p(None)
    _check(load().razor_cache_create(C.byref(h), C.byref(cfg), _ptr(pool), pool_bytes, _ptr(workspace),
                                     workspace_bytes, _stream(stream)), "razor_cache_create")
    return h.value


def razor_compress(cache: int, layer: int, K, V, stride_b: int, stride_h: int, stride_n: int, ctx_len,
                   head_is_retrieval, n_sink: int, window, stream=None) -> None:
    a, w, r = _i32(ctx_len), _i32(window), _u8(head_is_retrieval)
    _check(load().razor_compress(cache, layer, _ptr(K), _ptr(V), stride_b, stride_h, stride_n, a.ctypes.data,
                                 r.ctypes.data, n_sink, w.ctypes.data, _stream(stream)), "razor_compress")


def razor_compress_seq(cache: int, layer: int, b: int, K, V, stride_h: int, stride_n: int, ctx_len: int,
                       head_is_retrieval, n_sink: int, window: int, stream=None) -> None:
    r = _u8(head_is_retrieval)
    _check(load().razor_compress_seq(cache, layer, b, _ptr(K), _ptr(V), stride_h, stride_n, ctx_len, r.ctypes.data,
                                     n_sink, window, _stream(stream)), "razor_compress_seq")


def razor_append(cache: int, layer: int, k_new, v_new, stream=None) -> None:
    _check(load().razor_append(cache, layer, _ptr(k_new), _ptr(v_new), _stream(stream)), "razor_append")


def razor_decode_attention(cache: int, layer: int, q, out, stream=None) -> None:
    _check(load().razor_decode_attention(cache, layer, _ptr(q), _ptr(out), _stream(stream)),
           "razor_decode_attention")


def razor_decode_step(cache: int, layer: int, k_new, v_new, q, out, stream=None) -> None:
    _check(load().razor_decode_step(cache, layer, _ptr(k_new), _ptr(v_new), _ptr(q), _ptr(out), _stream(stream)),
           "razor_decode_step")


def razor_append_many(cache: int, layer: int, k_new, v_new, n_tokens: int, stream=None) -> None:
    _check(load().razor_append_many(cache, layer, _ptr(k_new), _ptr(v_new), n_tokens, _stream(stream)),
           "razor_append_many")


def razor_append_plan(len_: int, n_drop: int, ring_head: int, window: int, n_sink: int, n_tokens: int):
    """Host only.  -> (slot[n_tokens] int32, evicts_old[n_tokens] uint8, (len, n_drop, ring_head) after the run)."""
    slot = np.empty(max(1, n_tokens), dtype=np.int32)
    old = np.empty(max(1, n_tokens), dtype=np.uint8)
    after = np.zeros(3, dtype=np.int32)
    _check(load().razor_append_plan(len_, n_drop, ring_head, window, n_sink, n_tokens, slot.ctypes.data, old.ctypes.data,
                                    after[0:].ctypes.data, after[1:].ctypes.data, after[2:].ctypes.data),
           "razor_append_plan")
    return slot[:n_tokens], old[:n_tokens], tuple(int(x) for x in after)


def razor_decode_attention_multi(cache: int, layer: int, q, out, n_tokens: int, stream=None) -> None:
    _check(load().razor_decode_attention_multi(cache, layer, _ptr(q), _ptr(out), n_tokens, _stream(stream)),
           "razor_decode_attention_multi")


def razor_cache_export(cache: int, layer: int, b: int, kv_head: int, kept_pos=None, K=None, V=None, comp_mean_k=None,
                       comp_mean_v=None, comp_sum_k=None, comp_sum_v=None, stream=None) -> Tuple[int, int]:
    """-> (n_kept, n_drop); fills whichever device buffers are given."""
    nk, nd = C.c_int32(0), C.c_int32(0)
    _check(load().razor_cache_export(cache, layer, b, kv_head, _ptr(kept_pos), _ptr(K), _ptr(V), _ptr(comp_mean_k),
                                     _ptr(comp_mean_v), _ptr(comp_sum_k), _ptr(comp_sum_v), C.byref(nk), C.byref(nd),
                                     _stream(stream)), "razor_cache_export")
    return nk.value, nd.value


def razor_cache_stats(cache: int, layer: int) -> Tuple[int, int]:
    """-> (kept_bytes, dense_bytes) of the layer's K+V rows."""
    k, d = C.c_size_t(0), C.c_size_t(0)
    _check(load().razor_cache_stats(cache, layer, C.byref(k), C.byref(d)), "razor_cache_stats")
    return k.value, d.value


def razor_schedule_plan(tokens, n_ctas: int = 148, static_percent: int = 80, tail_items_per_cta: int = 3,
                        min_chunk_pages: int = 16, with_spans: bool = False):
    """Host-only: -> int32 [n_items, 5] = (head, first_page, end_page (-1: open), parts_of_head, job) in job
    order (and the number of span jobs when with_spans is set)."""
    t = _i32(tokens)
    n, ns = C.c_int32(0), C.c_int32(0)
    lib = load()
    args = (t.ctypes.data, len(t), n_ctas, static_percent, tail_items_per_cta, min_chunk_pages)
    _check(lib.razor_schedule_plan(*args, None, 0, C.byref(n), C.byref(ns)), "razor_schedule_plan")
    items = np.zeros((n.value, 5), dtype=np.int32)
    _check(lib.razor_schedule_plan(*args, items.ctypes.data, n.value, C.byref(n), C.byref(ns)), "razor_schedule_plan")
    return (items, ns.value) if with_spans else items


OPT_DECODE_TAIL_ITEMS_PER_SM, OPT_DECODE_MIN_CHUNK_PAGES, OPT_DECODE_RING_KB, OPT_DECODE_CONSUMER_WARPS = 1, 2, 3, 4
OPT_DECODE_TENSOR_CORES, OPT_DECODE_STATIC_PERCENT, OPT_DECODE_EARLY_PREFETCH, OPT_ROUND_TILED_MIN_ROWS = 5, 6, 7, 8


def razor_cache_set_option(cache: int, option: int, value: int) -> None:
    _check(load().razor_cache_set_option(cache, option, value), "razor_cache_set_option")


def razor_cache_device_status(cache: int, stream=None) -> int:
    """Synchronises the stream; -> the device status word (0 = healthy), cleared when non-zero."""
    st = C.c_int32(0)
    _check(load().razor_cache_device_status(cache, C.byref(st), _stream(stream)), "razor_cache_device_status")
    return st.value


def razor_schedule_query(cache: int, layer: int) -> np.ndarray:
    n = C.c_int32(0)
    lib = load()
    _check(lib.razor_schedule_query(cache, layer, None, 0, C.byref(n)), "razor_schedule_query")
    items = np.zeros((n.value, 5), dtype=np.int32)
    _check(lib.razor_schedule_query(cache, layer, items.ctypes.data, n.value, C.byref(n)), "razor_schedule_query")
    return items


def razor_schedule_combine_heads(cache: int, layer: int) -> np.ndarray:
    """Indices (b * Hkv + kv head) of the heads whose partial records the combine kernel folds."""
    n = C.c_int32(0)
    lib = load()
    _check(lib.razor_schedule_combine_heads(cache, layer, None, 0, C.byref(n)), "razor_schedule_combine_heads")
    heads = np.zeros(n.value, dtype=np.int32)
    _check(lib.razor_schedule_combine_heads(cache, layer, heads.ctypes.data, n.value, C.byref(n)), "razor_schedule_combine_heads")
    return heads


def razor_cache_set_alibi(cache: int, slopes, stream=None) -> None:
    """slopes: [L * Hq] (or [L, Hq]) ALiBi slopes l_h; None switches the distance penalty off."""
    if slopes is None:
        _check(load().razor_cache_set_alibi(cache, None, _stream(stream)), "razor_cache_set_alibi")
        return
    a = np.ascontiguousarray(np.asarray(slopes, dtype=np.float32).reshape(-1))
    _check(load().razor_cache_set_alibi(cache, a.ctypes.data, _stream(stream)), "razor_cache_set_alibi")


def razor_cache_set_head_windows(cache: int, layer: int, window_h) -> None:
    """window_h: [Hkv] per-head caps on the recent window for later compressions of `layer`; None removes them."""
    if window_h is None:
        _check(load().razor_cache_set_head_windows(cache, layer, None), "razor_cache_set_head_windows")
        return
    a = _i32(window_h)
    _check(load().razor_cache_set_head_windows(cache, layer, a.ctypes.data), "razor_cache_set_head_windows")


def razor_cache_wait_selftest(cache: int, limit_ns: int, stream=None) -> None:
    """Enqueue the kernel whose (bounded) wait nothing answers; razor_cache_device_status then shows bit 16."""
    _check(load().razor_cache_wait_selftest(cache, limit_ns, _stream(stream)), "razor_cache_wait_selftest")


def razor_compensation_mean_static(K, V, stride_h: int, stride_n: int, n_kv_heads: int, head_dim: int, dtype: int,
                                   ctx_len: int, n_sink: int, window: int, mean_k, mean_v, stream=None) -> int:
    """Means of the dropped K and V rows of one sequence's heads, using only the library's built-in
    scratch array (no pool, no workspace, no allocation).  -> number of rows averaged."""
    nd = C.c_int32(0)
    _check(load().razor_compensation_mean_static(_ptr(K), _ptr(V), stride_h, stride_n, n_kv_heads, head_dim, dtype,
                                                 ctx_len, n_sink, window, _ptr(mean_k), _ptr(mean_v), C.byref(nd),
                                                 _stream(stream)), "razor_compensation_mean_static")
    return nd.value


def razor_head_scores(Q: torch.Tensor, K: torch.Tensor, period: int, sm_scale: float = 0.0, stream=None):
    """Q, K: bf16 device tensors [H, N, D].  -> (echo, induction) fp32 device tensors [H]."""
    assert Q.is_contiguous() and K.is_contiguous() and Q.shape == K.shape and Q.dtype == torch.bfloat16
    H, N, D = Q.shape
    need = C.c_size_t(0)
    _check(load().razor_head_scores_scratch_bytes(H, N, C.byref(need)), "razor_head_scores_scratch_bytes")
    scratch = torch.empty(need.value, dtype=torch.uint8, device=Q.device)
    echo = torch.empty(H, dtype=torch.float32, device=Q.device)
    induction = torch.empty(H, dtype=torch.float32, device=Q.device)
    _check(load().razor_head_scores(_ptr(Q), _ptr(K), H, N, D, RAZOR_BF16, period, sm_scale, _ptr(echo),
                                    _ptr(induction), _ptr(scratch), need.value, _stream(stream)), "razor_head_scores")
    return echo, induction


def razor_select_retrieval_heads(echo, induction, frac_induction: float = 0.14, frac_echo: float = 0.01) -> np.ndarray:
    """Host-only: uint8 mask over the heads (1 = retrieval head)."""
    e = np.ascontiguousarray(np.asarray(echo, dtype=np.float32).reshape(-1))
    i = np.ascontiguousarray(np.asarray(induction, dtype=np.float32).reshape(-1))
    mask = np.zeros(e.size, dtype=np.uint8)
    _check(load().razor_select_retrieval_heads(e.ctypes.data, i.ctypes.data, e.size, frac_induction, frac_echo,
                                               mask.ctypes.data), "razor_select_retrieval_heads")
    return mask


def razor_cache_reset(cache: int) -> None:
    _check(load().razor_cache_reset(cache), "razor_cache_reset")


def razor_cache_destroy(cache: int) -> None:
    _check(load().razor_cache_destroy(cache), "razor_cache_destroy")


# ----------------------------------------------------------------------------- convenience owner of the buffers
class RazorCache:
    """Owns the pool / workspace tensors and the handle.  Still marshalling only."""

    def __init__(self, cfg: RazorConfig, ctx_len, window, head_is_retrieval, device="cuda:0", extra_pool_bytes=0):
        if not torch.cuda.is_available():
            raise RuntimeError("RazorCache needs a CUDA device (there is no CPU path)")
        self.cfg = cfg
        self.device = torch.device(device)
        self.pool_bytes, self.ws_bytes = razor_query_bytes(cfg, ctx_len, window, head_is_retrieval)
        self.pool_bytes += extra_pool_bytes
        with torch.cuda.device(self.device):
            self.pool = torch.empty(self.pool_bytes, dtype=torch.uint8, device=self.device)
            self.workspace = torch.empty(self.ws_bytes, dtype=torch.uint8, device=self.device)
            self.handle = razor_cache_create(cfg, self.pool, self.pool_bytes, self.workspace, self.ws_bytes)
        self.tdtype = torch.bfloat16 if cfg.dtype == RAZOR_BF16 else torch.float32

    def compress(self, layer: int, K: torch.Tensor, V: torch.Tensor, ctx_len, head_is_retrieval, window) -> None:
        """K, V: [B, Hkv, N, D] device tensors (innermost dim contiguous, same strides)."""
        assert K.stride() == V.stride() and K.stride(3) == 1
        razor_compress(self.handle, layer, K, V, K.stride(0), K.stride(1), K.stride(2), ctx_len, head_is_retrieval,
                       self.cfg.n_sink, window)

    def start_empty(self, layer: int, head_is_retrieval, window) -> None:
        """A layer with no tokens yet, its retrieval set and windows fixed: the start of a chunked prefill, whose
        chunks then arrive through append_many."""
        razor_compress(self.handle, layer, None, None, 0, 0, 0, [0] * self.cfg.batch, head_is_retrieval,
                       self.cfg.n_sink, window)

    def compress_seq(self, layer: int, b: int, K: torch.Tensor, V: torch.Tensor, ctx_len: int, head_is_retrieval,
                     window: int) -> None:
        """K, V: [Hkv, N, D] device tensors of one sequence."""
        assert K.stride() == V.stride() and K.stride(2) == 1
        razor_compress_seq(self.handle, layer, b, K, V, K.stride(0), K.stride(1), ctx_len, head_is_retrieval,
                           self.cfg.n_sink, window)

    def append(self, layer: int, k_new: torch.Tensor, v_new: torch.Tensor) -> None:
        assert k_new.is_contiguous() and v_new.is_contiguous()
        razor_append(self.handle, layer, k_new, v_new)

    def decode(self, layer: int, q: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        assert q.is_contiguous()
        if out is None:
            out = torch.empty(q.shape, dtype=torch.float32, device=q.device)
        razor_decode_attention(self.handle, layer, q, out)
        return out

    def decode_step(self, layer: int, k_new: torch.Tensor, v_new: torch.Tensor, q: torch.Tensor,
                    out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """append(k_new, v_new) + decode(q) in one launch."""
        assert k_new.is_contiguous() and v_new.is_contiguous() and q.is_contiguous()
        if out is None:
            out = torch.empty(q.shape, dtype=torch.float32, device=q.device)
        razor_decode_step(self.handle, layer, k_new, v_new, q, out)
        return out

    def append_many(self, layer: int, k_new: torch.Tensor, v_new: torch.Tensor) -> None:
        """k_new, v_new: [B, T, Hkv, D]."""
        assert k_new.is_contiguous() and v_new.is_contiguous()
        razor_append_many(self.handle, layer, k_new, v_new, k_new.shape[1])

    def decode_multi(self, layer: int, q: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """q: [B, T, Hq, D] -> out fp32 [B, T, Hq, D]."""
        assert q.is_contiguous()
        if out is None:
            out = torch.empty(q.shape, dtype=torch.float32, device=q.device)
        razor_decode_attention_multi(self.handle, layer, q, out, q.shape[1])
        return out

    def export(self, layer: int, b: int, kv_head: int):
        """-> dict(kept_pos, K, V, mean_k, mean_v, sum_k, sum_v, n_drop) in logical order (device tensors)."""
        n_kept, n_drop = razor_cache_export(self.handle, layer, b, kv_head)
        D = self.cfg.head_dim
        dev = self.device
        kp = torch.empty(max(n_kept, 1), dtype=torch.int32, device=dev)
        K = torch.empty((max(n_kept, 1), D), dtype=self.tdtype, device=dev)
        V = torch.empty_like(K)
        f = [torch.empty(D, dtype=torch.float32, device=dev) for _ in range(4)]
        razor_cache_export(self.handle, layer, b, kv_head, kp, K, V, f[0], f[1], f[2], f[3])
        return dict(kept_pos=kp[:n_kept], K=K[:n_kept], V=V[:n_kept], mean_k=f[0], mean_v=f[1], sum_k=f[2],
                    sum_v=f[3], n_drop=n_drop)

    def set_option(self, option: int, value: int) -> None:
        razor_cache_set_option(self.handle, option, value)

    def device_status(self) -> int:
        return razor_cache_device_status(self.handle)

    def stats(self, layer: int):
        return razor_cache_stats(self.handle, layer)

    def close(self) -> None:
        if getattr(self, "handle", None):
            razor_cache_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
