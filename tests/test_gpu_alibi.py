"""GPU parity of the ALiBi variant (Section 3.1): per-head recent windows, no sinks, no compensation token,
logits q.k - l_h (m - n) (Eq. 1), against the oracle's alibi_decode_head."""
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


def _slopes(n_layers, n_q_heads):
    # the geometric family ALiBi uses (2^-8i/H), scaled up a little so that the penalty matters at these lengths
    base = np.array([2.0 ** (-8.0 * (i + 1) / n_q_heads) for i in range(n_q_heads)], dtype=np.float32)
    return np.stack([base * (1.0 + 0.25 * l) for l in range(n_layers)])


@pytest.mark.parametrize("dtype,group,D", [("bf16", 1, 128), ("bf16", 2, 128), ("bf16", 4, 128), ("bf16", 8, 64),
                                           ("f32", 1, 64), ("f32", 2, 128)])
def test_alibi_decode_steps_match_the_oracle(dtype, group, D):
    Hkv, n_layers, steps = 4, 2, 6
    w = synth.Workload("alibi", 2, n_layers, Hkv * group, Hkv, D, dtype, [900, 130], [400, 400], 0, 1, steps, 321 + group)
    head_windows = [[64, 400, 17, 250], [400, 33, 128, 5]]     # per layer, per KV head (the retrieval head ignores its own)
    slopes = _slopes(n_layers, w.n_q_heads)
    cache = make_cache(w, max_new=steps, use_comp=0, shuffle=3)
    rz.razor_cache_set_alibi(cache.handle, slopes)
    scale = 1.0 / math.sqrt(D)
    refs = {}
    for l in range(n_layers):
        rz.razor_cache_set_head_windows(cache.handle, l, head_windows[l])
        K, V = synth.make_dense_kv(w, l, DEV)
        cache.compress(l, K, V, w.ctx_len, w.retrieval(l), w.window)
        for b in range(w.batch):
            for g in range(Hkv):
                refs[(l, b, g)] = HeadRef(l, b, g, K[b, g], V[b, g], w.ctx_len[b], steps)
    tol = TOL_OUT[dtype]
    for t in range(steps):
        for l in range(n_layers):
            retr = w.retrieval(l)
            k_new, v_new = synth.make_new_kv(w, l, t, DEV)
            cache.append(l, k_new, v_new)
            q = synth.make_queries(w, l, t, DEV)
            out, qh = to_f64(cache.decode(l, q)), to_f64(q)
            for b in range(w.batch):
                for g in range(Hkv):
                    ref = refs[(l, b, g)]
                    ref.append(k_new[b, g].cpu(), v_new[b, g].cpu())
                    win = -1 if retr[g] else min(w.window[b], head_windows[l][g])
                    if t in (0, steps - 1):
                        check_head_state(cache, ref, 0, win if win >= 0 else 0, bool(retr[g]))
                    for j in range(group):
                        h = g * group + j
                        expect = orc.alibi_decode_head(qh[b, h][None], ref.K[:ref.n], ref.V[:ref.n], win,
                                                       float(slopes[l, h]), scale)[0]
                        err = float(np.abs(out[b, h] - expect).max())
                        assert err <= tol, (err, t, l, b, h)
    assert cache.device_status() == 0
    # switching the penalty off gives plain truncated attention again
    rz.razor_cache_set_alibi(cache.handle, None)
    q = synth.make_queries(w, 0, 99, DEV)
    out = to_f64(cache.decode(0, q))
    ref = refs[(0, 0, 0)]
    win = -1 if w.retrieval(0)[0] else min(w.window[0], head_windows[0][0])
    expect = orc.alibi_decode_head(to_f64(q)[0, 0][None], ref.K[:ref.n], ref.V[:ref.n], win, 0.0, scale)[0]
    assert np.abs(out[0, 0] - expect).max() <= tol
    cache.close()


@pytest.mark.parametrize("T,tiled,group,D", [(4, True, 2, 128), (20, True, 2, 128), (20, False, 2, 128), (37, True, 2, 128),
                                             (37, False, 2, 128), (150, True, 2, 128), (70, True, 1, 64), (9, True, 4, 128),
                                             (33, True, 8, 64), (5, True, 4, 64)])
def test_alibi_in_a_round_of_several_tokens(T, tiled, group, D):
    """T = 4: one launch of the streaming kernel (a tile of 8 rows).  Longer rounds: the query-tiled kernel, which
    adds Eq. 1's distance penalty to every score (heads in position order and ring heads that have wrapped), or -
    forced here by the threshold option - block by block on the streaming kernel, every block masking the round's
    tokens that come after it."""
    Hkv = 3
    w = synth.Workload("alibi_round", 2, 1, Hkv * group, Hkv, D, "bf16", [700, 60], [300, 300], 0, 1, T, 99 + group)
    hw = [max(40, T), 300, max(9, T)]
    slopes = _slopes(1, w.n_q_heads)
    cache = make_cache(w, max_new=T, use_comp=0, options={rz.OPT_ROUND_TILED_MIN_ROWS: 9 if tiled else 1 << 30})
    rz.razor_cache_set_alibi(cache.handle, slopes)
    rz.razor_cache_set_head_windows(cache.handle, 0, hw)
    K, V = synth.make_dense_kv(w, 0, DEV)
    retr = w.retrieval(0)
    cache.compress(0, K, V, w.ctx_len, retr, w.window)
    k = synth.normal_bf16(w.seed, synth.TAG_KNEW, (w.batch, T, Hkv, D), DEV, sub=1)
    v = synth.normal_bf16(w.seed, synth.TAG_VNEW, (w.batch, T, Hkv, D), DEV, sub=1)
    q = synth.normal_bf16(w.seed, synth.TAG_Q, (w.batch, T, w.n_q_heads, D), DEV, sub=1)
    cache.append_many(0, k, v)
    out = to_f64(cache.decode_multi(0, q))
    assert cache.device_status() == 0
    scale = 1.0 / math.sqrt(D)
    for b in range(w.batch):
        for g in range(Hkv):
            Kh = np.concatenate([to_f64(K[b, g, : w.ctx_len[b]]), to_f64(k[b, :, g])])
            Vh = np.concatenate([to_f64(V[b, g, : w.ctx_len[b]]), to_f64(v[b, :, g])])
            win = -1 if retr[g] else min(w.window[b], hw[g])
            for j in range(group):
                h = g * group + j
                expect = orc.alibi_decode_head(to_f64(q[b, :, h]), Kh, Vh, win, float(slopes[0, h]), scale)
                assert np.abs(out[b, :, h] - expect).max() <= TOL_OUT["bf16"]
    cache.close()


def test_alibi_needs_the_compensation_token_off():
    w = synth.Workload("alibi_err", 1, 1, 2, 2, 64, "bf16", [100], [30], 0, 0, 1, 1)
    cache = make_cache(w, use_comp=1)
    with pytest.raises(rz.RazorError) as e:
        rz.razor_cache_set_alibi(cache.handle, np.ones(2, dtype=np.float32))
    assert e.value.status == -1
    with pytest.raises(rz.RazorError) as e:
        rz.razor_cache_set_head_windows(cache.handle, 0, [5, -2])
    assert e.value.status == -1
    cache.close()
