"""Random sessions on the GPU against the oracle: a compression, then a random mix of single appends, short
rounds, long runs (the parallel append kernel), single-token decodes and multi-token rounds of random length,
with the layout checked bit-exact after every step and every output within tolerance.  Shapes, group sizes,
sink counts and windows are drawn per seed."""
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


@pytest.mark.parametrize("seed", list(range(2000, 2016)))
def test_random_session(seed):
    rng = np.random.default_rng(seed)
    group, Hkv = int(rng.choice([1, 2, 4, 8])), int(rng.integers(1, 4))
    D, B = int(rng.choice([64, 128])), int(rng.integers(1, 3))
    n_sink = int(rng.integers(0, 6))
    ctx = [int(rng.integers(0, 400)) for _ in range(B)]
    win = [int(rng.integers(1, 150)) for _ in range(B)]
    budget = 600
    n_retr = int(rng.integers(0, Hkv + 1)) if Hkv > 1 else 0
    w = synth.Workload(f"session{seed}", B, 1, Hkv * group, Hkv, D, "bf16", ctx, win, n_sink, n_retr, budget, 31337 + seed)
    cache = make_cache(w, max_new=budget, shuffle=int(rng.integers(0, 3)))
    K, V = synth.make_dense_kv(w, 0, DEV)
    retr = w.retrieval(0)
    cache.compress(0, K, V, w.ctx_len, retr, w.window)
    refs = {(b, g): HeadRef(0, b, g, K[b, g], V[b, g], w.ctx_len[b], budget) for b in range(B) for g in range(Hkv)}
    scale = 1.0 / math.sqrt(D)
    used, ops = 0, []
    for step in range(8):
        kind = rng.choice(["one", "few", "many", "none"])
        T = {"one": 1, "few": int(rng.integers(2, 20)), "many": int(rng.integers(64, 200)), "none": 0}[kind]
        if used + T > budget:
            T = 0
        if T:
            shp = (B, T, Hkv, D)
            k = synth.normal_bf16(w.seed, synth.TAG_KNEW, shp, DEV, sub=step)
            v = synth.normal_bf16(w.seed, synth.TAG_VNEW, shp, DEV, sub=step)
            if T == 1 and rng.integers(0, 2):
                cache.append(0, k[:, 0].contiguous(), v[:, 0].contiguous())
            else:
                cache.append_many(0, k, v)
            used += T
            kh, vh = k.cpu(), v.cpu()
            for (b, g), ref in refs.items():
                for t in range(T):
                    ref.append(kh[b, t, g], vh[b, t, g])
        ops.append((kind, T))
        hcs = {key: check_head_state(cache, ref, n_sink, w.window[key[0]], bool(retr[key[1]]))
               for key, ref in refs.items()}
        if min(ref.n for ref in refs.values()) == 0:
            continue
        # multi-token round query over the last Tq tokens, when allowed
        Tq = int(rng.integers(1, 12))
        ok_multi = all(ref.n >= Tq for ref in refs.values()) and \
            all(hc.n_drop == 0 or w.window[key[0]] >= Tq for key, hc in hcs.items())
        if Tq > 1 and ok_multi:
            q = synth.normal_bf16(w.seed, synth.TAG_Q, (B, Tq, Hkv * group, D), DEV, sub=100 + step)
            out, qh = to_f64(cache.decode_multi(0, q)), to_f64(q)
            for (b, g), ref in refs.items():
                for j in range(group):
                    exp = orc.multi_query_attention(qh[b, :, g * group + j], ref.K[:ref.n], ref.V[:ref.n], n_sink,
                                                    w.window[b], bool(retr[g]), scale)
                    err = float(np.abs(out[b, :, g * group + j] - exp).max())
                    assert err <= TOL_OUT["bf16"], ("multi", seed, step, ops, b, g, j, err)
        q = synth.normal_bf16(w.seed, synth.TAG_Q, (B, Hkv * group, D), DEV, sub=200 + step)
        out, qh = to_f64(cache.decode(0, q)), to_f64(q)
        for (b, g), ref in refs.items():
            if ref.n == 0:
                continue
            for j in range(group):
                exp = orc.decode_head(qh[b, g * group + j], hcs[(b, g)], scale)
                err = float(np.abs(out[b, g * group + j] - exp).max())
                assert err <= TOL_OUT["bf16"], ("single", seed, step, ops, b, g, j, err)
        assert cache.device_status() == 0
    cache.close()
