"""GPU parity tests: the CUDA library (through its C ABI) against the CPU oracle on the same seeded
inputs.  Layout bit-exact; means within 1e-3 relative; outputs within 3e-3 (bf16) / 1e-5 (fp32)."""
import copy
import math

import numpy as np
import pytest
import torch

from oracle import razor_oracle as orc
from paper_2407_15891_b200 import binding as rz
from paper_2407_15891_b200 import synth

from _harness import HeadRef, TOL_OUT, bits, check_head_state, floor_heads, make_cache, run_parity, run_parity_recorded, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def small(name, **kw):
    w = copy.copy(synth.workload(name))
    for k, v in kw.items():
        setattr(w, k, v)
    return w


# ------------------------------------------------------------------ the five configurations
def test_cfg1_tiny_fp32_every_head():
    w = synth.workload("cfg1")
    st = {}
    r = run_parity(w, steps=0, stats=st)
    assert r["heads"] == 4 and r["outputs"] == 4
    # and with one appended token (the query then attends to itself)
    r = run_parity(w, steps=1)
    assert r["out"] <= 1e-5


def test_cfg1_needle_recalled_only_by_retrieval_head():
    w = synth.workload("cfg1")
    cache = make_cache(w)
    K, V = synth.make_dense_kv(w, 0, DEV)
    cache.compress(0, K, V, w.ctx_len, w.retrieval(0), w.window)
    out = cache.decode(0, synth.make_queries(w, 0, 0, DEV)).cpu()
    v200 = V[0, :, 200, :].cpu()
    assert (out[0, 0] - v200[0]).abs().max() < 0.05
    for h in (1, 2, 3):
        assert (out[0, h] - v200[h]).abs().max() > 0.5
    cache.close()


def test_cfg2_llama2_7b_shaped_32k_every_head():
    w = synth.workload("cfg2")
    st = {}
    r = run_parity(w, steps=0, stats=st)
    assert r["heads"] == 8 * 32
    row = 2 * w.head_dim * w.esz()
    kept = row * sum(len(orc.kept_positions(n, w.n_sink, win, bool(f))) for f in w.retrieval(0)
                     for n, win in zip(w.ctx_len, w.window))
    assert st["kept_bytes"] == kept and st["dense_bytes"] == row * sum(w.ctx_len) * w.n_kv_heads


# The three large configurations run on the GPU exactly as the benchmark runs them (all layers compressed, then
# the decode steps step-major over the layers); checked against the oracle are, in EVERY layer and for every
# sequence listed, every retrieval KV head plus a seeded tenth of the others: layout bit-exact and means right
# after compression, after the middle step and after the last one, outputs at every step.
def test_cfg3_llama2_13b_64k_full_stack_16_steps_every_layer():
    w = synth.workload("cfg3")
    heads = {l: floor_heads(w, l, range(w.batch)) for l in range(w.n_layers)}
    assert all(len(heads[l]) == 4 * (6 + 4) for l in heads)                     # 6 retrieval + 4 of the other 34, x 4 sequences
    r = run_parity_recorded(w, heads_for=heads, steps=16)
    assert r["heads"] == 40 * 40 and r["outputs"] == 40 * 40 * 16 and r["layouts"] == 3 * 40 * 40


def test_cfg4_gqa_llama3_8b_shaped_128k_every_layer():
    w = synth.workload("cfg4")
    heads = {l: floor_heads(w, l, range(w.batch)) for l in range(w.n_layers)}
    assert all(len(heads[l]) == 2 * (2 + 1) for l in heads)                     # 2 retrieval + 1 of the other 6 KV heads, x 2
    r = run_parity_recorded(w, heads_for=heads, steps=0)                        # the configuration: compression + one decode
    assert r["heads"] == 32 * 6 and r["outputs"] == 32 * 6 * 4 and r["layouts"] == 32 * 6
    few = {l: heads[l] for l in (0, 15, 31)}
    r = run_parity_recorded(w, heads_for=few, steps=4)                          # and with appended tokens
    assert r["outputs"] == 3 * 6 * 4 * 4 and r["layouts"] == 3 * 3 * 6


def test_cfg5_ragged_serving_mix_64_steps_shortest_median_longest():
    w = synth.workload("cfg5")
    order = [int(i) for i in np.argsort(w.ctx_len)]
    bs = sorted(set(order[:8] + order[28:36] + order[-8:]))                    # the 8 shortest, 8 around the median, 8 longest
    assert len(bs) == 24
    heads = {0: floor_heads(w, 0, bs)}
    assert len(heads[0]) == 24 * (5 + 3)                                        # 5 retrieval + 3 of the other 27
    r = run_parity_recorded(w, heads_for=heads, steps=64, per_seq=True)
    assert r["heads"] == 24 * 8 and r["outputs"] == 24 * 8 * 64 and r["layouts"] == 3 * 24 * 8


# ------------------------------------------------------------------ scaled copies, every head, paged
@pytest.mark.parametrize("name,scale", [("cfg2", 1 / 16), ("cfg3", 1 / 32), ("cfg4", 1 / 32), ("cfg5", 1 / 32)])
def test_scaled_configs_every_head_with_shuffled_pages(name, scale):
    w = synth.workload(name, scale)
    if name == "cfg3":
        w.n_layers = 3
    if name == "cfg4":
        w.n_layers = 2
    if name == "cfg5":
        w.batch, w.ctx_len, w.window = 8, w.ctx_len[:8], w.window[:8]
    w.decode_steps = min(w.decode_steps, 8)
    run_parity(w, steps=w.decode_steps if w.decode_steps > 1 else 0, shuffle=12345, per_seq=(name == "cfg5"),
               check_layout_every=3)


# ------------------------------------------------------------------ property sweep over small shapes
@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("group", [1, 2, 4, 8])
def test_small_shape_sweep(dtype, D, group, fused):
    rng = np.random.default_rng(D * 100 + group + (7 if dtype == "f32" else 0))
    for trial in range(6):
        B = int(rng.integers(1, 4))
        Hkv = int(rng.integers(1, 4))
        n_sink = int(rng.integers(0, 6))
        ctx = [int(rng.integers(0 if trial == 0 else 1, 301)) for _ in range(B)]
        win = [int(rng.integers(0, 80)) for _ in range(B)]
        if trial == 1:
            win = [max(ctx) + 5] * B                         # window covers everything: nothing dropped
        if trial == 2:
            win = [max(0, c - n_sink - 1) for c in ctx]      # exactly one dropped token where possible
        w = synth.Workload(f"sweep{trial}", B, 2, Hkv * group, Hkv, D, dtype, ctx, win, n_sink,
                           n_retrieval_kv=min(1, Hkv - 1) if trial % 2 else 0, decode_steps=5,
                           seed=9000 + trial + D + group)
        run_parity(w, steps=5 if trial != 3 else 0, shuffle=trial, check_layout_every=1, fused=fused)


@pytest.mark.parametrize("group,options", [
    (2, {rz.OPT_DECODE_TENSOR_CORES: 1}),                                   # matrix instructions from group 2
    (1, {rz.OPT_DECODE_TENSOR_CORES: 1}),                                   # ... and for single heads (one row of the tile)
    (2, {rz.OPT_DECODE_TENSOR_CORES: 1, rz.OPT_DECODE_CONSUMER_WARPS: 4}),
    (4, {rz.OPT_DECODE_TENSOR_CORES: 2}),                                   # grouped heads on the CUDA cores
    (4, {rz.OPT_DECODE_CONSUMER_WARPS: 4, rz.OPT_DECODE_TAIL_ITEMS_PER_SM: 64, rz.OPT_DECODE_MIN_CHUNK_PAGES: 1}),
    (4, {rz.OPT_DECODE_STATIC_PERCENT: 0, rz.OPT_DECODE_TAIL_ITEMS_PER_SM: 2, rz.OPT_DECODE_MIN_CHUNK_PAGES: 1}),
    (1, {rz.OPT_DECODE_STATIC_PERCENT: 100, rz.OPT_DECODE_MIN_CHUNK_PAGES: 1}),
    (8, {rz.OPT_DECODE_RING_KB: 64}),
    (1, {rz.OPT_DECODE_CONSUMER_WARPS: 16, rz.OPT_DECODE_RING_KB: 128}),
    (1, {rz.OPT_DECODE_CONSUMER_WARPS: 8, rz.OPT_DECODE_STATIC_PERCENT: 30, rz.OPT_DECODE_TAIL_ITEMS_PER_SM: 200,
         rz.OPT_DECODE_MIN_CHUNK_PAGES: 1}),
])
@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("D", [64, 128])
def test_decode_kernel_variants(group, options, D, fused):
    """Every decode kernel variant the options can select, on a ragged batch whose long head is cut into
    enough parts for a two-level combine tree."""
    w = synth.Workload("variants", 3, 1, 2 * group, 2, D, "bf16", [9000, 37, 700], [300, 300, 100], 4, 1, 3, 2024 + group)
    run_parity(w, steps=3, shuffle=7, options=options, check_layout_every=2, fused=fused)


def test_schedule_reports_which_heads_are_left_to_the_combine_kernel():
    """razor_schedule_combine_heads lists exactly the heads cut into more parts than the streaming kernel folds
    itself (16 record rows: 16 // group parts), and none when every head is in few parts."""
    for group, ctx in ((4, [9000, 37, 700]), (1, [700, 40, 300])):
        w = synth.Workload("combine_list", 3, 1, 2 * group, 2, 128, "bf16", ctx, [300, 300, 100], 4, 1, 1, 99 + group)
        cache = make_cache(w)
        K, V = synth.make_dense_kv(w, 0, DEV)
        cache.compress(0, K, V, w.ctx_len, w.retrieval(0), w.window)
        items = rz.razor_schedule_query(cache.handle, 0)
        want = sorted({int(h) for h, _, _, parts, _ in items.tolist() if parts > 16 // group})
        got = sorted(rz.razor_schedule_combine_heads(cache.handle, 0).tolist())
        assert got == want
        assert (len(got) > 0) == (group == 4)
        cache.close()


@pytest.mark.parametrize("fused", [False, True])
def test_append_many_tokens_crosses_pages_evicts_and_rebuilds_schedule(fused):
    w = synth.Workload("long_append", 2, 1, 4, 4, 128, "bf16", [700, 90], [64, 200], 4, 1, 300, 4242)
    run_parity(w, steps=300, check_layout_every=37, fused=fused)


def test_one_launch_steps_interleaved_with_separate_appends_and_decodes():
    """razor_decode_step mixed with razor_append / razor_decode_attention on the same layers (one of them a
    single-layer cache, where consecutive launches touch the same pages), layout checked after every step."""
    for n_layers in (1, 3):
        w = synth.Workload("mixed_steps", 3, n_layers, 8, 4, 128, "bf16", [900, 30, 260], [40, 100, 16], 4, 1, 60, 808 + n_layers)
        cache = make_cache(w, max_new=60)
        refs = {}
        for l in range(n_layers):
            K, V = synth.make_dense_kv(w, l, DEV)
            cache.compress(l, K, V, w.ctx_len, w.retrieval(l), w.window)
            for b in range(w.batch):
                for g in range(w.n_kv_heads):
                    refs[(l, b, g)] = HeadRef(l, b, g, K[b, g], V[b, g], w.ctx_len[b], 60)
        rng = np.random.default_rng(5 + n_layers)
        scale = 1 / math.sqrt(w.head_dim)
        for t in range(60):
            for l in range(n_layers):
                k_new, v_new = synth.make_new_kv(w, l, t, DEV)
                q = synth.make_queries(w, l, t, DEV)
                if rng.random() < 0.6:
                    out = cache.decode_step(l, k_new, v_new, q)
                else:
                    cache.append(l, k_new, v_new)
                    out = cache.decode(l, q)
                if rng.random() < 0.3:
                    out = cache.decode(l, q)                      # a second decode of the same layer, no append
                out_h, q_h = to_f64(out), to_f64(q)
                for (ll, b, g), ref in refs.items():
                    if ll != l:
                        continue
                    ref.append(k_new[b, g].cpu(), v_new[b, g].cpu())
                    if t % 7 == 0 or t == 59:
                        hc = check_head_state(cache, ref, w.n_sink, w.window[b], bool(w.retrieval(l)[g]))
                    else:
                        hc = orc.compress_head(ref.K, ref.V, ref.n, w.n_sink, w.window[b], bool(w.retrieval(l)[g]))
                    for j in range(w.group):
                        err = np.abs(out_h[b, g * w.group + j] - orc.decode_head(q_h[b, g * w.group + j], hc, scale)).max()
                        assert err <= 3e-3, (err, l, b, g, j, t)
        assert cache.device_status() == 0
        cache.close()


def test_plain_truncation_mode_and_literal_scale():
    w = synth.workload("cfg2", 1 / 32)
    run_parity(w, steps=3, use_comp=0)                      # sinks + window only (no compensation term)
    w1 = synth.workload("cfg1")
    run_parity(w1, steps=2, sm_scale=1.0)                   # Eq. 5 as printed: no 1/sqrt(d)


def test_invariants_on_gpu_window_covers_context_equals_full_attention():
    """A window >= N reproduces full attention; compared here against the oracle's full attention."""
    w = synth.Workload("fullwin", 1, 1, 2, 2, 128, "bf16", [333], [400], 4, 0, 1, 77)
    cache = make_cache(w)
    K, V = synth.make_dense_kv(w, 0, DEV)
    cache.compress(0, K, V, w.ctx_len, w.retrieval(0), w.window)
    q = synth.make_queries(w, 0, 0, DEV)
    out = to_f64(cache.decode(0, q))
    for h in range(2):
        ref = orc.full_attention(to_f64(q[0, h]), to_f64(K[0, h]), to_f64(V[0, h]), 1 / math.sqrt(128))
        assert np.abs(out[0, h] - ref).max() <= 3e-3
    cache.close()


def test_append_directly_behind_the_kernel_that_produces_its_rows():
    """In a decoder the K/V projection is the kernel right before razor_append and writes k_new / v_new into
    the same buffers every step.  Here a small elementwise kernel refills one pair of buffers immediately
    before each of 200 appends (no synchronisation in between); the cache must hold exactly the rows of each
    step: layout bit-exact against the oracle's recompression of the whole history, means within 1e-3."""
    steps = 200
    w = synth.Workload("producer", 3, 2, 4, 4, 128, "bf16", [300, 40, 77], [48, 90, 20], 4, 1, steps, 555)
    cache = make_cache(w, max_new=steps)
    refs = {}
    for l in range(w.n_layers):
        K, V = synth.make_dense_kv(w, l, DEV)
        cache.compress(l, K, V, w.ctx_len, w.retrieval(l), w.window)
        for b in range(w.batch):
            for g in range(w.n_kv_heads):
                refs[(l, b, g)] = HeadRef(l, b, g, K[b, g], V[b, g], w.ctx_len[b], steps)
    rows = [[synth.make_new_kv(w, l, t, DEV) for t in range(steps)] for l in range(w.n_layers)]
    k_buf = torch.empty_like(rows[0][0][0])
    v_buf = torch.empty_like(k_buf)
    q = synth.make_queries(w, 0, 0, DEV)
    out = torch.empty((w.batch, w.n_q_heads, w.head_dim), dtype=torch.float32, device=DEV)
    one = torch.ones((), dtype=torch.bfloat16, device=DEV)
    torch.cuda.synchronize()
    for t in range(steps):
        for l in range(w.n_layers):
            torch.mul(rows[l][t][0], one, out=k_buf)            # the "projection": an elementwise kernel, not a copy
            torch.mul(rows[l][t][1], one, out=v_buf)
            cache.append(l, k_buf, v_buf)
            cache.decode(l, q, out)                              # keeps the append's programmatic launch chain as in a pass
    torch.cuda.synchronize()
    for (l, b, g), ref in refs.items():
        for t in range(steps):
            ref.append(rows[l][t][0][b, g].cpu(), rows[l][t][1][b, g].cpu())
        check_head_state(cache, ref, w.n_sink, w.window[b], bool(w.retrieval(l)[g]))
    assert cache.device_status() == 0
    cache.close()


def test_a_sequence_without_tokens_attends_to_nothing_and_gives_zeros():
    """A head that holds no token has both sums of Eq. 5 empty; library and oracle define the output as zeros."""
    w = synth.Workload("empty", 2, 1, 4, 2, 64, "bf16", [0, 50], [16, 16], 4, 1, 2, 99)
    cache = make_cache(w, max_new=2)
    K, V = synth.make_dense_kv(w, 0, DEV)
    cache.compress(0, K, V, w.ctx_len, w.retrieval(0), w.window)
    q = synth.make_queries(w, 0, 0, DEV)
    out = to_f64(cache.decode(0, q))
    qh = to_f64(q)
    for b in range(2):
        for g in range(2):
            hc = orc.compress_head(to_f64(K[b, g]), to_f64(V[b, g]), w.ctx_len[b], w.n_sink, w.window[b], bool(w.retrieval(0)[g]))
            for j in range(2):
                expect = orc.decode_head(qh[b, g * 2 + j], hc, 1 / math.sqrt(64))
                assert np.abs(out[b, g * 2 + j] - expect).max() <= 3e-3
    assert not out[0].any()                                       # the empty sequence: exact zeros
    cache.close()


# ------------------------------------------------------------------ error paths on a live cache
def test_error_codes_on_a_live_cache():
    w = synth.Workload("err", 2, 2, 2, 2, 64, "bf16", [100, 50], [20, 20], 4, 1, 2, 5)
    cache = make_cache(w)
    q = synth.make_queries(w, 0, 0, DEV)
    out = torch.empty(q.shape, dtype=torch.float32, device=DEV)
    k_new, v_new = synth.make_new_kv(w, 0, 0, DEV)
    with pytest.raises(rz.RazorError) as e:
        cache.decode(0, q)
    assert e.value.status == -6                                   # not compressed
    with pytest.raises(rz.RazorError) as e:
        cache.append(0, k_new, v_new)
    assert e.value.status == -6
    K, V = synth.make_dense_kv(w, 0, DEV)
    retr = w.retrieval(0)
    cache.compress_seq(0, 0, K[0], V[0], 100, retr, 20)
    with pytest.raises(rz.RazorError) as e:
        cache.decode(0, q)
    assert e.value.status == -6                                   # sequence 1 still missing
    with pytest.raises(rz.RazorError) as e:
        cache.compress_seq(0, 1, K[1], V[1], 50, 1 - retr, 20)    # retrieval set must match the layer's
    assert e.value.status == -1
    cache.compress_seq(0, 1, K[1], V[1], 50, retr, 20)
    cache.decode(0, q, out)
    cache.append(0, k_new, v_new)
    cache.append(0, k_new, v_new)
    with pytest.raises(rz.RazorError) as e:
        cache.append(0, k_new, v_new)                             # max_new_tokens = 2
    assert e.value.status == -5
    with pytest.raises(rz.RazorError) as e:
        rz.razor_compress(cache.handle, 0, K, V, K.stride(0), K.stride(1), K.stride(2), [101, 50], retr, 4, [20, 20])
    assert e.value.status == -5                                   # beyond max_ctx_len
    with pytest.raises(rz.RazorError) as e:
        rz.razor_compress(cache.handle, 0, K, V, K.stride(0), K.stride(1), K.stride(2), w.ctx_len, retr, 3, w.window)
    assert e.value.status == -1                                   # n_sink differs from the config
    with pytest.raises(rz.RazorError) as e:
        rz.razor_compress(cache.handle, 0, K.data_ptr() + 2, V, K.stride(0), K.stride(1), K.stride(2), w.ctx_len,
                          retr, 4, w.window)
    assert e.value.status == -8
    with pytest.raises(rz.RazorError) as e:
        rz.razor_compress(cache.handle, 5, K, V, K.stride(0), K.stride(1), K.stride(2), w.ctx_len, retr, 4, w.window)
    assert e.value.status == -1
    # the pool holds every layer once; asking for a bigger plan than the pool has left fails cleanly
    cache.compress(1, K, V, w.ctx_len, w.retrieval(1), w.window)
    big = synth.Workload("err2", 2, 2, 2, 2, 64, "bf16", [100, 100], [90, 90], 4, 2, 2, 5)
    with pytest.raises(rz.RazorError) as e:
        cache.compress(1, K, V, [100, 100], np.ones(2, dtype=np.uint8), [90, 90])
    assert e.value.status == -4
    # the context is still healthy
    cache.decode(0, q, out)
    torch.cuda.synchronize()
    assert torch.isfinite(out).all()
    cache.close()


def test_a_wait_that_nothing_answers_gives_up_and_reports():
    """Failure detection without a fault: the decode kernel's wait routine, pointed at a barrier nobody
    arrives on, returns after its limit, the status word says so, and the cache goes on working."""
    import time
    w = synth.workload("cfg2", 1 / 32)
    cache = make_cache(w)
    K, V = synth.make_dense_kv(w, 0, DEV)
    q = synth.make_queries(w, 0, 0, DEV)
    cache.compress(0, K, V, w.ctx_len, w.retrieval(0), w.window)
    before = cache.decode(0, q).clone()
    assert cache.device_status() == 0
    t0 = time.perf_counter()
    rz.razor_cache_wait_selftest(cache.handle, 2_000_000)           # 2 ms
    status = cache.device_status()                                  # synchronises
    assert time.perf_counter() - t0 < 1.0
    assert status == 16
    assert cache.device_status() == 0                               # reading it cleared it
    assert (bits(cache.decode(0, q)) == bits(before)).all()         # the context and the cache are healthy
    with pytest.raises(rz.RazorError):
        rz.razor_cache_wait_selftest(cache.handle, 10)              # limit out of range
    cache.close()


def test_recompress_reuses_pages_and_reset_frees_them():
    w = synth.workload("cfg2", 1 / 32)
    w.decode_steps = 2
    cache = make_cache(w)
    K, V = synth.make_dense_kv(w, 0, DEV)
    q = synth.make_queries(w, 0, 0, DEV)
    outs = []
    for _ in range(3):                                            # same plan: fits in the same pages
        cache.compress(0, K, V, w.ctx_len, w.retrieval(0), w.window)
        outs.append(cache.decode(0, q).clone())
    assert (bits(outs[0]) == bits(outs[1])).all() and (bits(outs[1]) == bits(outs[2])).all()
    rz.razor_cache_reset(cache.handle)
    with pytest.raises(rz.RazorError):
        cache.decode(0, q)
    cache.compress(0, K, V, w.ctx_len, w.retrieval(0), w.window)
    assert (bits(cache.decode(0, q)) == bits(outs[0])).all()
    cache.close()


def test_strided_dense_input_and_schedule_query():
    """K/V taken as views of a larger buffer (row stride > D, padded context)."""
    w = synth.Workload("strided", 2, 1, 4, 4, 128, "bf16", [500, 260], [100, 100], 4, 1, 1, 31)
    Kc, Vc = synth.make_dense_kv(w, 0, DEV)
    big_k = torch.zeros((2, 4, 520, 256), dtype=torch.bfloat16, device=DEV)
    big_v = torch.zeros_like(big_k)
    big_k[:, :, :500, 64:192] = Kc
    big_v[:, :, :500, 64:192] = Vc
    Kv, Vv = big_k[:, :, :, 64:192], big_v[:, :, :, 64:192]
    cache = make_cache(w)
    cache.compress(0, Kv, Vv, w.ctx_len, w.retrieval(0), w.window)
    q = synth.make_queries(w, 0, 0, DEV)
    a = cache.decode(0, q).clone()
    items = rz.razor_schedule_query(cache.handle, 0)
    assert set(items[:, 0].tolist()) == set(range(8))
    cache.compress(0, Kc, Vc, w.ctx_len, w.retrieval(0), w.window)
    b = cache.decode(0, q)
    assert (bits(a) == bits(b)).all()
    cache.close()
