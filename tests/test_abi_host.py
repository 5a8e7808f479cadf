"""CPU-side tests of the C-ABI library: it loads, exports every symbol include/razor.h declares,
validates arguments, sizes its buffers as Algorithm 1 dictates, and plans balanced decode
schedules.  No compute call is made here (there is no GPU on this machine)."""
import ctypes as C
import os
import re

import numpy as np
import pytest
import torch

from oracle import razor_oracle as orc
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
    row = 2 * w.head_dim * w.esz()                # one K row + one V row
    kept = row * sum(len(orc.kept_positions(n, w.n_sink, win, bool(r)))
                     for l in range(w.n_layers) for r in w.retrieval(l) for n, win in zip(w.ctx_len, w.window))
    assert kept <= pool < kept * 1.002            # only page rounding on top
    dense = row * sum(w.ctx_len) * w.n_kv_heads * w.n_layers
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
    pages = [-(-t // 16) for t in tokens]
    seen = {h: [] for h in range(len(tokens))}
    for head, p0, p1, parts, job in items:
        seen[head].append((p0, pages[head] if p1 < 0 else p1, parts, job))
    return pages, seen


@pytest.mark.parametrize("tokens,n_ctas,pct,tail,min_chunk", [
    ([65536] * 24 + [8196] * 136, 148, 85, 4, 8),              # one layer of the 64K-shaped stack
    ([131072, 16388, 16388, 16388, 131072, 16388, 16388, 16388] * 2, 148, 85, 4, 8),
    ([0, 1, 15, 16, 17, 100000, 3], 148, 85, 4, 1),
    ([5000] * 2048, 148, 85, 4, 8),
    ([7], 148, 85, 4, 8),
    ([1 << 20] * 3, 148, 0, 1000, 1),                          # more tail items than the item budget: chunk grows
    ([9000, 37, 700, 9000, 37, 700], 5, 50, 2, 1),
    ([4000] * 10, 148, 100, 1, 1),
])
def test_schedule_covers_every_page_once_and_is_balanced(tokens, n_ctas, pct, tail, min_chunk):
    items, n_spans = rz.razor_schedule_plan(tokens, n_ctas, pct, tail, min_chunk, with_spans=True)
    pages, seen = _coverage(items, tokens)
    for h, parts in seen.items():
        assert len(parts) >= 1                                 # every head gets at least one item (even empty)
        assert parts == sorted(parts)                          # parts of a head come in page order within the job order
        assert parts[0][0] == 0 and parts[-1][1] == pages[h]
        assert all(p[2] == len(parts) for p in parts)
        for a, b in zip(parts, parts[1:]):
            assert a[1] == b[0]                                # contiguous, no overlap
        open_ended = [it for it in items if it[0] == h and it[2] < 0]
        assert len(open_ended) == 1                            # the last part grows with appends
    total = sum(pages)
    jobs = items[:, 4]
    assert (np.diff(jobs) >= 0).all() and jobs[0] == 0         # job order, jobs numbered from 0
    n_jobs = int(jobs[-1]) + 1
    assert 0 <= n_spans <= min(n_ctas, n_jobs)
    size = np.array([(pages[h] if p1 < 0 else p1) - p0 for h, p0, p1, _, _ in items])
    job_pages = np.bincount(jobs, weights=size, minlength=n_jobs)
    if n_spans:
        span = job_pages[0]
        assert (job_pages[:n_spans] == span).all()             # spans are equal
        assert span >= min_chunk
        assert n_spans * span <= total * pct / 100 + 1e-9
        assert n_spans == n_ctas or (n_spans + 1) * span > total * pct // 100
    tail_sizes = job_pages[n_spans:]
    assert (np.bincount(jobs)[n_spans:] == 1).all()            # a tail job is one item
    if len(tail_sizes):
        tail_total = int(tail_sizes.sum())
        first = max(min_chunk, -(-tail_total // (n_ctas * tail)))
        if len(tokens) + n_spans + 4 * n_ctas * tail + tail_total // max(min_chunk, 1) <= 16384:
            # guided sizes: nothing larger than the first chunk (plus the crumb a head's end may add),
            # and the sizes never grow along the stream except where a head ended early
            assert tail_sizes.max() <= first + min_chunk // 2
            left = tail_total
            for sz in tail_sizes:
                bound = max(min_chunk, -(-left // (n_ctas * tail)))
                assert sz <= bound + min_chunk // 2
                left -= int(sz)
    assert len(items) <= len(tokens) + 16384


def test_schedule_gives_long_heads_few_parts():
    tokens = [65536] * 24 + [8196] * 136                       # 6 retrieval heads x 4 sequences, 40 heads each
    items = rz.razor_schedule_plan(tokens)
    parts = {h: n for h, _, _, n, _ in items}
    assert max(parts[h] for h in range(24)) <= 8               # a full-length head spans about four CTAs' shares
    with pytest.raises(rz.RazorError):
        rz.razor_schedule_plan([-1])
    with pytest.raises(rz.RazorError):
        rz.razor_schedule_plan([100], 148, 85, 4, 0)
    with pytest.raises(rz.RazorError):
        rz.razor_schedule_plan([100], 148, 101, 4, 1)


def test_header_is_plain_c():
    """The public header must compile as C99 on its own: no C++ constructs, no CUDA or torch types."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = '#include "razor.h"\nint main(void) { razor_config_t c; (void)c; return razor_version() == 0; }\n'
    r = subprocess.run([gcc, "-std=c99", "-Wall", "-Werror", "-pedantic", "-fsyntax-only", "-I", os.path.join(root, "include"),
                        "-x", "c", "-"], input=src, text=True, capture_output=True)
    assert r.returncode == 0, r.stderr


def _sequential_appends(len0, n_drop0, ring_head0, window, n_sink, n_tokens):
    """The single-token rule applied n_tokens times on a model cache: slots hold token ids (old tokens are
    negative, new token a is a), `folded` collects what went into the compensation sums."""
    slots = {s: -(s + 1) for s in range(len0)}
    length, n_drop, head, folded = len0, n_drop0, ring_head0, []
    for a in range(n_tokens):
        if window < 0 or length < n_sink + window:
            slots[length] = a
            length += 1
        elif window == 0:
            folded.append(a)
            n_drop += 1
        else:
            s = n_sink + head
            folded.append(slots[s])
            slots[s] = a
            n_drop += 1
            head = (head + 1) % window
    return slots, folded, (length, n_drop, head)


def test_append_run_in_closed_form_equals_single_appends():
    """razor_append_plan (the rule of the parallel append kernel and of the host mirror) against the single-token
    rule applied token by token, for every small state: same final slot contents, same set of folded tokens, same
    state."""
    checked = 0
    for n_sink in (0, 1, 3):
        for window in (-1, 0, 1, 2, 5, 8):
            cap = n_sink + max(window, 0)
            for len0 in range(0, (cap if window >= 0 else 12) + 1):
                full = window > 0 and len0 == cap
                for ring_head0 in (range(window) if full else [0]):
                    for n_tokens in (0, 1, 2, 3, 7, 8, 9, 20):
                        want_slots, want_folded, want_state = _sequential_appends(len0, 4, ring_head0, window, n_sink, n_tokens)
                        slot, old, state = rz.razor_append_plan(len0, 4, ring_head0, window, n_sink, n_tokens)
                        assert state == want_state
                        got_slots = {s: -(s + 1) for s in range(len0)}
                        got_folded = []
                        for a in range(n_tokens):
                            if slot[a] < 0:
                                got_folded.append(a)
                                continue
                            if old[a]:
                                got_folded.append(-(int(slot[a]) + 1))          # the old token of that slot
                            got_slots[int(slot[a])] = a
                        assert got_slots == want_slots
                        assert sorted(got_folded) == sorted(want_folded)
                        assert len(set(int(s) for s in slot if s >= 0)) == int((slot >= 0).sum())   # one writer per slot
                        checked += 1
    assert checked > 1000
    with pytest.raises(rz.RazorError):
        rz.razor_append_plan(3, 0, 1, 8, 2, 3)                  # a ring that is still filling starts at index 0
