"""GPU parity of long appended runs (razor_append_many on prompt chunks): a cache built chunk by chunk from an
empty one must be the cache that one compression of the whole context builds (fold-on-evict keeps Eq. 4 over
every dropped token), layout bit-exact, means and decode outputs within the usual tolerances."""
import math

import numpy as np
import pytest
import torch

from oracle import razor_oracle as orc
from paper_2407_15891_b200 import binding as rz
from paper_2407_15891_b200 import synth

from _harness import TOL_MEAN_REL, TOL_OUT, HeadRef, bits, check_head_state, make_cache, rel_inf, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _gen(w, tag, shape, sub):
    t = synth.normal_bf16(w.seed, tag, shape, DEV, sub=sub)      # fp32 workloads hold bf16-representable values
    return t if w.dtype == "bf16" else t.float()


def _chunk(w, T, sub):
    shp = (w.batch, T, w.n_kv_heads, w.head_dim)
    return _gen(w, synth.TAG_KNEW, shp, sub), _gen(w, synth.TAG_VNEW, shp, sub)


@pytest.mark.parametrize("dtype,D,group", [("bf16", 128, 1), ("bf16", 64, 2), ("f32", 64, 1), ("f32", 128, 4)])
def test_cache_built_chunk_by_chunk_from_empty(dtype, D, group):
    """Chunks shorter and longer than the windows, runs below and above the parallel kernel's threshold, a window
    that fills in the middle of a chunk, a chunk that laps the ring several times."""
    Hkv = 3
    chunks = [700, 1, 5, 8, 7, 64, 1500, 735, 100]
    total = sum(chunks)
    w = synth.Workload("chunked", 2, 1, Hkv * group, Hkv, D, dtype, [0, 0], [600, 100], 4, 1, total, 9100 + D + group)
    cache = make_cache(w, max_new=total)
    retr = w.retrieval(0)
    cache.start_empty(0, retr, w.window)                          # an empty layer with its windows and retrieval set
    dummy = torch.zeros((1, D), dtype=torch.bfloat16 if dtype == "bf16" else torch.float32)
    refs = {(b, g): HeadRef(0, b, g, dummy, dummy, 0, total) for b in range(w.batch) for g in range(Hkv)}
    scale = 1.0 / math.sqrt(D)
    for i, T in enumerate(chunks):
        k, v = _chunk(w, T, i)
        cache.append_many(0, k, v)
        kh, vh = k.cpu(), v.cpu()
        q = _gen(w, synth.TAG_Q, (w.batch, w.n_q_heads, D), i)
        out = to_f64(cache.decode(0, q))
        assert cache.device_status() == 0
        qh = to_f64(q)
        for (b, g), ref in refs.items():
            for t in range(T):
                ref.append(kh[b, t, g], vh[b, t, g])
            hc = check_head_state(cache, ref, w.n_sink, w.window[b], bool(retr[g]))
            for j in range(group):
                expect = orc.decode_head(qh[b, g * group + j], hc, scale)
                err = float(np.abs(out[b, g * group + j] - expect).max())
                assert err <= TOL_OUT[dtype], (err, i, b, g, j)
    cache.close()


def test_chunks_of_at_least_the_window_do_not_read_rows_back_and_stay_exact():
    """Chunk after chunk of the window's length or more: the evicted rows' share of the Eq. 4 sums comes from the
    recorded sum of the window, not from reading the rows again.  A one-launch decode step in between makes that
    record stale (the next chunk must read the rows); the chunks after it use the record again."""
    Hkv, D = 4, 128
    plan = [256, 256, 300, 256, "step", 256, 256, 256]
    total = sum(x for x in plan if x != "step") + 1
    w = synth.Workload("window_chunks", 2, 1, Hkv, Hkv, D, "bf16", [0, 0], [256, 128], 4, 1, total, 7321)
    cache = make_cache(w, max_new=total)
    retr = w.retrieval(0)
    cache.start_empty(0, retr, w.window)
    dummy = torch.zeros((1, D), dtype=torch.bfloat16)
    refs = {(b, g): HeadRef(0, b, g, dummy, dummy, 0, total) for b in range(w.batch) for g in range(Hkv)}
    scale = 1.0 / math.sqrt(D)
    for i, T in enumerate(plan):
        q = _gen(w, synth.TAG_Q, (w.batch, w.n_q_heads, D), i)
        if T == "step":
            k1, v1 = synth.make_new_kv(w, 0, i, DEV)
            out = to_f64(cache.decode_step(0, k1, v1, q))
            kh, vh, n = k1.cpu()[:, None], v1.cpu()[:, None], 1
        else:
            k, v = _chunk(w, T, i)
            cache.append_many(0, k, v)
            out = to_f64(cache.decode(0, q))
            kh, vh, n = k.cpu(), v.cpu(), T
        assert cache.device_status() == 0
        qh = to_f64(q)
        for (b, g), ref in refs.items():
            for t in range(n):
                ref.append(kh[b, t, g], vh[b, t, g])
            hc = check_head_state(cache, ref, w.n_sink, w.window[b], bool(retr[g]))
            err = float(np.abs(out[b, g] - orc.decode_head(qh[b, g], hc, scale)).max())
            assert err <= TOL_OUT["bf16"], (err, i, b, g)
    cache.close()


def test_chunked_prefill_equals_one_compression():
    """Same tokens, same windows: the exported caches agree bit for bit in layout, and in the means to rounding."""
    Hkv, D, N = 4, 128, 3000
    w = synth.Workload("oneshot", 2, 1, Hkv, Hkv, D, "bf16", [N, N], [600, 1000], 4, 1, 8, 4242)
    K, V = synth.make_dense_kv(w, 0, DEV)
    retr = w.retrieval(0)
    whole = make_cache(w, max_new=8)
    whole.compress(0, K, V, w.ctx_len, retr, w.window)
    w0 = synth.Workload("chunks", 2, 1, Hkv, Hkv, D, "bf16", [0, 0], [600, 1000], 4, 1, N + 8, 4242)
    parts = make_cache(w0, max_new=N + 8)
    parts.start_empty(0, retr, w0.window)
    at = 0
    for T in [1024, 1024, 952]:
        k = K[:, :, at:at + T, :].permute(0, 2, 1, 3).contiguous()
        v = V[:, :, at:at + T, :].permute(0, 2, 1, 3).contiguous()
        parts.append_many(0, k, v)
        at += T
    for b in range(2):
        for g in range(Hkv):
            a, c = whole.export(0, b, g), parts.export(0, b, g)
            assert a["kept_pos"].cpu().tolist() == c["kept_pos"].cpu().tolist()
            assert a["n_drop"] == c["n_drop"]
            assert (bits(a["K"]) == bits(c["K"])).all() and (bits(a["V"]) == bits(c["V"])).all()
            if a["n_drop"]:
                assert rel_inf(to_f64(c["mean_k"]), to_f64(a["mean_k"])) <= TOL_MEAN_REL
                assert rel_inf(to_f64(c["mean_v"]), to_f64(a["mean_v"])) <= TOL_MEAN_REL
    q = synth.normal_bf16(7, synth.TAG_Q, (2, Hkv, D), DEV)
    o1, o2 = to_f64(whole.decode(0, q)), to_f64(parts.decode(0, q))
    assert float(np.abs(o1 - o2).max()) <= TOL_OUT["bf16"]
    assert whole.device_status() == 0 and parts.device_status() == 0
    whole.close()
    parts.close()
