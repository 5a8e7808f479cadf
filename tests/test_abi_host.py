"""CPU-side tests of the C-ABI library: it loads, exports every symbol include/razor.h declares,
validates arguments, sizes its buffers as Algorithm 1 line 2-3 dictates, and plans balanced decode
schedules.  No compute call is made here (there is no GPU on this machine)."""
import ctypes as C
import os
import re

import numpy as np
import pytest
import torch

from paper_2407_15891_b200 import binding as rz
from paper_2407_15891_b200 import build as rz_build
from paper_2407_15891_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    rz_build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "razor.h")).read()
    declared = sorted(set(re.findall(r"RAZOR_API\s+[\w\s\*]+?\b(razor_\w+)\s*\(", header)))
    assert len(declared) >= 13
    assert sorted(rz.SYMBOLS) == declared
    lib = rz.load()
    for name in declared:
        assert hasattr(lib, name), name
    assert rz.razor_version() == "0.1"
    assert rz.razor_status_string(0) == "ok"
    assert "unknown" in rz.razor_status_string(-99)
    for code in range(-8, 0):
        assert "unknown" not in rz.razor_status_string(code)


def test_config_struct_matches_header_field_order():
    header = open(os.path.join(ROOT, "include", "razor.h")).read()
    body = header[header.index("typedef struct {"):header.index("} razor_config_t;")]
    fields = re.findall(r"^\s*(?:int32_t|float)\s+(\w+);", body, flags=re.M)
    assert fields == [f[0] for f in rz.RazorConfig._fields_]
    assert C.sizeof(rz.RazorConfig) == 13 * 4


def _cfg(**kw):
    base = dict(batch=2, n_layers=3, n_q_heads=8, n_kv_heads=8, head_dim=128, dtype="bf16", n_sink=4,
                max_ctx_len=1000, max_new_tokens=8)
    base.update(kw)
    return rz.make_config(**base)


def test_query_bytes_counts_pages_per_head():
    cfg = _cfg()
    retr = np.zeros((3, 8), dtype=np.uint8)
    retr[:, 0] = 1
    pool, ws = rz.razor_query_bytes(cfg, [1000, 100], [200, 200], retr)
    page_bytes = 2 * 16 * 128 * 2
    # sequence 0: retrieval heads hold 1000+8 tokens -> 63 pages; others min(1008, 204) -> 13 pages
    # sequence 1: context 100 <= 4+200: retrieval 108 -> 7 pages; others min(108, 204) = 108 -> 7 pages
    pages = 3 * ((63 + 7 * 13) + (7 + 7 * 7))
    assert pool == pages * page_bytes
    assert ws % 256 == 0 and ws > 0
    # the workspace depends on the config only
    _, ws2 = rz.razor_query_bytes(cfg, [5, 5], [1, 1], retr)
    assert ws2 == ws


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4"])
def test_pool_size_tracks_the_compressed_bytes_of_the_paper_shaped_configs(name):
    w = synth.workload(name)
    cfg = rz.make_config(w.batch, w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, w.n_sink,
                         max(w.ctx_len), 0)
    retr = np.stack([w.retrieval(l) for l in range(w.n_layers)])
    pool, _ = rz.razor_query_bytes(cfg, w.ctx_len, w.window, retr)
    kept = sum(w.compressed_bytes(l) for l in range(w.n_layers))
    assert kept <= pool < kept * 1.002            # only page rounding on top
    dense = w.dense_bytes() * w.n_layers
    ratio = dense / kept
    expect = {"cfg2": 3.08, "cfg3": 3.90, "cfg4": 2.91}[name]
    assert abs(ratio - expect) < 0.01


def test_bad_arguments_are_rejected_with_codes():
    lib = rz.load()
    retr = np.zeros(24, dtype=np.uint8)
    for kw, code in [(dict(head_dim=96), -3), (dict(n_q_heads=12), -1), (dict(n_q_heads=24), -3),
                     (dict(page_tokens=32), -3), (dict(batch=0), -1), (dict(n_sink=-1), -1),
                     (dict(dtype=7), -3), (dict(sm_scale=-1.0), -1)]:
        with pytest.raises(rz.RazorError) as e:
            rz.razor_query_bytes(_cfg(**kw), [10, 10], [5, 5], retr)
        assert e.value.status == code, kw
    with pytest.raises(rz.RazorError) as e:
        rz.razor_query_bytes(_cfg(), [2000, 10], [5, 5], retr)      # beyond max_ctx_len
    assert e.value.status == -5
    with pytest.raises(rz.RazorError) as e:
        rz.razor_query_bytes(_cfg(), [10, 10], [5, -1], retr)
    assert e.value.status == -1
    pool, ws = C.c_size_t(), C.c_size_t()
    assert lib.razor_query_bytes(None, None, None, None, C.byref(pool), C.byref(ws)) == -2
    cfg = _cfg()
    assert lib.razor_query_bytes(C.byref(cfg), None, None, None, C.byref(pool), C.byref(ws)) == -2
    # NULL handles
    assert lib.razor_cache_destroy(None) == -2
    assert lib.razor_cache_reset(None) == -2
    assert lib.razor_append(None, 0, None, None, None) == -2
    assert lib.razor_decode_attention(None, 0, None, None, None) == -2
    h = C.c_void_p()
    assert lib.razor_cache_create(C.byref(h), C.byref(cfg), None, 0, None, 0, None) == -2
    assert lib.razor_cache_create(C.byref(h), C.byref(cfg), 256 + 8, 1 << 20, 512, 1 << 20, None) == -8
    assert lib.razor_cache_create(C.byref(h), C.byref(cfg), 256, 1 << 20, 512, 16, None) == -4


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful without a device")
def test_create_fails_loudly_without_a_gpu():
    cfg = _cfg()
    _, ws = rz.razor_query_bytes(cfg, [10, 10], [5, 5], np.zeros(24, dtype=np.uint8))
    h = C.c_void_p()
    rc = rz.load().razor_cache_create(C.byref(h), C.byref(cfg), 256, 1 << 24, 1 << 20, ws, None)
    assert rc == -7 and rz.load().razor_last_cuda_error() != 0
    with pytest.raises(RuntimeError):
        rz.RazorCache(cfg, [10, 10], [5, 5], np.zeros(24, dtype=np.uint8))


# ------------------------------------------------------------------ decode schedule (host only)
def _coverage(items, tokens):
    pages = [(t + 15) // 16 for t in tokens]
    seen = {h: [] for h in range(len(tokens))}
    for head, p0, p1, parts in items:
        seen[head].append((p0, pages[head] if p1 < 0 else p1, parts))
    return pages, seen


@pytest.mark.parametrize("tokens,target,min_chunk", [
    ([65536] * 6 + [8196] * 34, 148 * 24, 8),                  # one sequence of the 64K-shaped stack
    ([131072, 16388, 16388, 16388, 131072, 16388, 16388, 16388], 148 * 24, 8),
    ([0, 1, 15, 16, 17, 100000, 3], 64, 1),
    ([5000] * 2048, 148 * 24, 8),
    ([7], 1, 1),
    ([1 << 20] * 3, 148 * 200, 1),                             # more parts than the item budget: chunk grows
])
def test_schedule_covers_every_page_once_and_is_balanced(tokens, target, min_chunk):
    items = rz.razor_schedule_plan(tokens, target, min_chunk)
    pages, seen = _coverage(items, tokens)
    sizes = []
    for h, parts in seen.items():
        assert len(parts) >= 1                                 # every head gets at least one item (even empty)
        parts.sort()
        assert parts[0][0] == 0 and parts[-1][1] == pages[h]
        assert all(p[2] == len(parts) for p in parts)
        for a, b in zip(parts, parts[1:]):
            assert a[1] == b[0]                                # contiguous, no overlap
        open_ended = [it for it in items if it[0] == h and it[2] < 0]
        assert len(open_ended) == 1                            # the last part grows with appends
        sizes += [p[1] - p[0] for p in parts]
    total = sum(pages)
    chunk = max(min_chunk, -(-total // target))
    if len(tokens) + total // chunk <= 16384:                  # item budget not hit: parts obey the chunk
        assert max(sizes) <= chunk
        assert len(items) <= len(tokens) + total // chunk + 1
    else:                                                      # the chunk grew until the items fit
        assert len(items) <= len(tokens) + 16384
        assert max(sizes) - min(sizes) <= 1
    # heads cut into the most parts first; within equal part counts, longer ranges first
    keys = [(-parts, -((pages[h] if p1 < 0 else p1) - p0)) for h, p0, p1, parts in items]
    assert keys == sorted(keys)


def test_schedule_splits_only_long_heads():
    tokens = [65536] * 2 + [8196] * 10
    items = rz.razor_schedule_plan(tokens, 64, 4)
    parts = {h: n for h, _, _, n in items}
    assert parts[0] > 8 * parts[5] - 8 and parts[5] >= 1
    with pytest.raises(rz.RazorError):
        rz.razor_schedule_plan([-1], 4)
    with pytest.raises(rz.RazorError):
        rz.razor_schedule_plan([100], 4, 0)
