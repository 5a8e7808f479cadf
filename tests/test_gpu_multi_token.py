"""GPU parity of a round of several new tokens (razor_append_many + razor_decode_attention_multi) against
the oracle's multi_query_attention: layout bit-exact after the bulk append, outputs within 3e-3."""
import math

import numpy as np
import pytest
import torch

from oracle import razor_oracle as orc
from paper_2407_15891_b200 import binding as rz
from paper_2407_15891_b200 import synth

from _harness import TOL_OUT, HeadRef, check_head_state, make_cache, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _round_inputs(w, T, seed_sub):
    shp_kv, shp_q = (w.batch, T, w.n_kv_heads, w.head_dim), (w.batch, T, w.n_q_heads, w.head_dim)
    k = synth.normal_bf16(w.seed, synth.TAG_KNEW, shp_kv, DEV, sub=seed_sub)
    v = synth.normal_bf16(w.seed, synth.TAG_VNEW, shp_kv, DEV, sub=seed_sub)
    q = synth.normal_bf16(w.seed, synth.TAG_Q, shp_q, DEV, sub=seed_sub)
    return k, v, q


@pytest.mark.parametrize("group,T,D", [(1, 2, 128), (1, 4, 128), (1, 8, 128), (2, 4, 128), (4, 2, 128), (1, 4, 64), (2, 2, 64)])
def test_round_of_new_tokens_matches_the_oracle(group, T, D):
    Hkv = 3
    w = synth.Workload("round", 2, 1, Hkv * group, Hkv, D, "bf16", [1500, 77], [200, 40], 4, 1, 3 * T, 555 + T + group)
    cache = make_cache(w, max_new=3 * T, shuffle=5)
    K, V = synth.make_dense_kv(w, 0, DEV)
    retr = w.retrieval(0)
    cache.compress(0, K, V, w.ctx_len, retr, w.window)
    refs = {(b, g): HeadRef(0, b, g, K[b, g], V[b, g], w.ctx_len[b], 3 * T) for b in range(w.batch) for g in range(Hkv)}
    scale = 1.0 / math.sqrt(D)
    worst = 0.0
    for rnd in range(3):                                       # three rounds: windows fill, evict, wrap
        k, v, q = _round_inputs(w, T, rnd)
        cache.append_many(0, k, v)
        out = to_f64(cache.decode_multi(0, q))
        assert cache.device_status() == 0
        kh, vh, qh = k.cpu(), v.cpu(), to_f64(q)
        for (b, g), ref in refs.items():
            for t in range(T):
                ref.append(kh[b, t, g], vh[b, t, g])
            check_head_state(cache, ref, w.n_sink, w.window[b], bool(retr[g]))   # the bulk append is T appends
            for j in range(group):
                expect = orc.multi_query_attention(qh[b, :, g * group + j], ref.K[:ref.n], ref.V[:ref.n], w.n_sink,
                                                   w.window[b], bool(retr[g]), scale)
                err = float(np.abs(out[b, :, g * group + j] - expect).max())
                worst = max(worst, err)
                assert err <= TOL_OUT["bf16"], (err, rnd, b, g, j)
    cache.close()


def test_round_on_a_long_context_with_split_heads():
    """32K context so that heads are cut into several parts (records + combine kernel) in a 4-token round."""
    w = synth.workload("cfg2", 1 / 4)
    w.batch, w.ctx_len, w.window = 2, w.ctx_len[:2], w.window[:2]
    T = 4
    cache = make_cache(w, max_new=T)
    K, V = synth.make_dense_kv(w, 0, DEV)
    retr = w.retrieval(0)
    cache.compress(0, K, V, w.ctx_len, retr, w.window)
    k, v, q = _round_inputs(w, T, 9)
    cache.append_many(0, k, v)
    out = to_f64(cache.decode_multi(0, q))
    assert cache.device_status() == 0
    scale = 1.0 / math.sqrt(w.head_dim)
    heads = [g for g in range(w.n_kv_heads) if retr[g]][:2] + [g for g in range(w.n_kv_heads) if not retr[g]][:3]
    for b in range(w.batch):
        for g in heads:
            Kh = np.concatenate([to_f64(K[b, g]), to_f64(k[b, :, g])])
            Vh = np.concatenate([to_f64(V[b, g]), to_f64(v[b, :, g])])
            expect = orc.multi_query_attention(to_f64(q[b, :, g]), Kh, Vh, w.n_sink, w.window[b], bool(retr[g]), scale)
            assert np.abs(out[b, :, g] - expect).max() <= TOL_OUT["bf16"]
    cache.close()


@pytest.mark.parametrize("tiled", [False, True])
@pytest.mark.parametrize("group,T,D", [(1, 16, 128), (1, 9, 128), (1, 3, 64), (2, 5, 128), (4, 3, 128), (8, 2, 64), (1, 29, 128)])
def test_round_longer_than_one_launch(group, T, D, tiled):
    """Rounds that do not fit one tile of 2, 4 or 8 rows of the streaming kernel.  Block by block on that kernel
    (forced here by the threshold option; it is what ALiBi caches get): blocks of the largest size that fits, the
    last one moved back to end with the round, every block masking the round's tokens that come after it.  And the
    default: the query-tiled kernel, most of whose 128 rows are no query of such a short round."""
    Hkv = 2
    w = synth.Workload("long_round", 2, 1, Hkv * group, Hkv, D, "bf16", [700, 90], [120, 40], 4, 1, T, 777 + T + group)
    cache = make_cache(w, max_new=T, options={rz.OPT_ROUND_TILED_MIN_ROWS: 9 if tiled else 1 << 30})
    K, V = synth.make_dense_kv(w, 0, DEV)
    retr = w.retrieval(0)
    cache.compress(0, K, V, w.ctx_len, retr, w.window)
    refs = {(b, g): HeadRef(0, b, g, K[b, g], V[b, g], w.ctx_len[b], T) for b in range(w.batch) for g in range(Hkv)}
    k, v, q = _round_inputs(w, T, 3)
    cache.append_many(0, k, v)
    out = to_f64(cache.decode_multi(0, q))
    assert cache.device_status() == 0
    kh, vh, qh = k.cpu(), v.cpu(), to_f64(q)
    scale = 1.0 / math.sqrt(D)
    for (b, g), ref in refs.items():
        for t in range(T):
            ref.append(kh[b, t, g], vh[b, t, g])
        for j in range(group):
            expect = orc.multi_query_attention(qh[b, :, g * group + j], ref.K[:ref.n], ref.V[:ref.n], w.n_sink,
                                               w.window[b], bool(retr[g]), scale)
            err = float(np.abs(out[b, :, g * group + j] - expect).max())
            assert err <= TOL_OUT["bf16"], (err, b, g, j)
    cache.close()


@pytest.mark.parametrize("group,T,D", [(1, 64, 128), (1, 200, 128), (4, 40, 128), (2, 300, 64), (8, 16, 128), (1, 512, 64),
                                        (4, 512, 128), (1, 2048, 128), (4, 2048, 64)])
def test_prompt_sized_round_on_the_query_tiled_kernel(group, T, D):
    """Rounds with at least 64 query rows per KV head run on the query-tiled tensor-core kernel: ragged batch (one
    sequence shorter than a block, one whose window evicts and wraps during the rounds), two rounds in a row,
    every row of every head against the oracle, layout bit-exact after the bulk appends."""
    Hkv = 3
    win = max(T, 150)
    w = synth.Workload("tiled_round", 3, 1, Hkv * group, Hkv, D, "bf16", [1500, 70, 700], [win + 60, win, win], 4, 1,
                       2 * T, 900 + T + group)
    cache = make_cache(w, max_new=2 * T, shuffle=11)
    K, V = synth.make_dense_kv(w, 0, DEV)
    retr = w.retrieval(0)
    cache.compress(0, K, V, w.ctx_len, retr, w.window)
    refs = {(b, g): HeadRef(0, b, g, K[b, g], V[b, g], w.ctx_len[b], 2 * T) for b in range(w.batch) for g in range(Hkv)}
    scale = 1.0 / math.sqrt(D)
    for rnd in range(2):
        k, v, q = _round_inputs(w, T, 40 + rnd)
        cache.append_many(0, k, v)
        out = to_f64(cache.decode_multi(0, q))
        assert cache.device_status() == 0
        kh, vh, qh = k.cpu(), v.cpu(), to_f64(q)
        for (b, g), ref in refs.items():
            for t in range(T):
                ref.append(kh[b, t, g], vh[b, t, g])
            check_head_state(cache, ref, w.n_sink, w.window[b], bool(retr[g]))
            for j in range(group):
                expect = orc.multi_query_attention(qh[b, :, g * group + j], ref.K[:ref.n], ref.V[:ref.n], w.n_sink,
                                                   w.window[b], bool(retr[g]), scale)
                err = float(np.abs(out[b, :, g * group + j] - expect).max())
                assert err <= TOL_OUT["bf16"], (err, rnd, b, g, j)
    cache.close()


def test_prompt_sized_round_on_a_long_context_with_split_units():
    """8K context, 4 sequences x 32 heads, a 256-token round: the long heads are cut into several parts (partial
    records of 128 rows each, merged afterwards)."""
    w = synth.workload("cfg2", 1 / 4)
    w.batch, w.ctx_len, w.window = 4, w.ctx_len[:4], w.window[:4]
    T = 256
    cache = make_cache(w, max_new=T)
    K, V = synth.make_dense_kv(w, 0, DEV)
    retr = w.retrieval(0)
    cache.compress(0, K, V, w.ctx_len, retr, w.window)
    k, v, q = _round_inputs(w, T, 19)
    cache.append_many(0, k, v)
    out = to_f64(cache.decode_multi(0, q))
    assert cache.device_status() == 0
    scale = 1.0 / math.sqrt(w.head_dim)
    heads = [g for g in range(w.n_kv_heads) if retr[g]][:3] + [g for g in range(w.n_kv_heads) if not retr[g]][:4]
    for b in range(w.batch):
        for g in heads:
            Kh = np.concatenate([to_f64(K[b, g]), to_f64(k[b, :, g])])
            Vh = np.concatenate([to_f64(V[b, g]), to_f64(v[b, :, g])])
            expect = orc.multi_query_attention(to_f64(q[b, :, g]), Kh, Vh, w.n_sink, w.window[b], bool(retr[g]), scale)
            assert np.abs(out[b, :, g] - expect).max() <= TOL_OUT["bf16"]
    cache.close()


def test_round_limits_are_reported():
    w = synth.Workload("round_err", 1, 1, 2, 2, 64, "bf16", [100], [3], 4, 0, 8, 1)
    cache = make_cache(w, max_new=8)
    K, V = synth.make_dense_kv(w, 0, DEV)
    cache.compress(0, K, V, w.ctx_len, w.retrieval(0), w.window)
    k, v, q = _round_inputs(w, 4, 0)
    cache.append_many(0, k, v)
    with pytest.raises(rz.RazorError) as e:
        cache.decode_multi(0, q)                               # window 3 < 4 tokens of the round
    assert e.value.status == -1
    with pytest.raises(rz.RazorError) as e:
        rz.razor_append_many(cache.handle, 0, k, v, 5)         # beyond max_new_tokens
    assert e.value.status == -5
    wf = synth.Workload("round_f32", 1, 1, 2, 2, 64, "f32", [100], [30], 4, 0, 4, 1)
    cf = make_cache(wf, max_new=4)
    Kf, Vf = synth.make_dense_kv(wf, 0, DEV)
    cf.compress(0, Kf, Vf, wf.ctx_len, wf.retrieval(0), wf.window)
    with pytest.raises(rz.RazorError) as e:
        cf.decode_multi(0, q.float())                          # fp32 has no tile path
    assert e.value.status == -3
    cf.close()
    cache.close()
