"""The entry point for callers that cannot allocate device memory (an application plugin that is only
handed its input and output tensors, code inside a stream capture, a process with a fixed memory
budget): razor_compensation_mean_static keeps its reduction scratch in a fixed array inside the
library.  Checked here, on two calls in a row that share the array, against the cache-building path
(razor_compress + razor_cache_export), which computes the same means with caller-provided workspace, and
against the CPU oracle's Eq. 4 mean over rows [n_sink, ctx_len - window) of the same inputs."""
import numpy as np
import pytest
import torch

from oracle import razor_oracle as orc
from paper_2407_15891_b200 import binding as rz
from paper_2407_15891_b200 import synth

from _harness import TOL_MEAN_REL, make_cache, rel_inf, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _means_via_cache(w, K, V):
    cache = make_cache(w)
    cache.compress(0, K, V, w.ctx_len, w.retrieval(0), w.window)
    mk = np.stack([to_f64(cache.export(0, 0, g)["mean_k"]) for g in range(w.n_kv_heads)])
    mv = np.stack([to_f64(cache.export(0, 0, g)["mean_v"]) for g in range(w.n_kv_heads)])
    nd = [cache.export(0, 0, g)["n_drop"] for g in range(w.n_kv_heads)]
    cache.close()
    return mk, mv, nd


def _check_static(w, strided=False):
    K, V = synth.make_dense_kv(w, 0, DEV)
    H, D = w.n_kv_heads, w.head_dim
    if strided:                                             # the same rows as views into wider, longer buffers
        big_k = torch.zeros((1, H, w.ctx_len[0] + 9, 2 * D), dtype=K.dtype, device=DEV)
        big_v = torch.zeros_like(big_k)
        big_k[:, :, : w.ctx_len[0], D // 2: D // 2 + D] = K
        big_v[:, :, : w.ctx_len[0], D // 2: D // 2 + D] = V
        K, V = big_k[:, :, :, D // 2: D // 2 + D], big_v[:, :, :, D // 2: D // 2 + D]
        assert K.stride(2) == 2 * D
    mean_k = torch.full((H, D), float("nan"), dtype=torch.float32, device=DEV)
    mean_v = torch.full((H, D), float("nan"), dtype=torch.float32, device=DEV)
    dt = rz.RAZOR_BF16 if w.dtype == "bf16" else rz.RAZOR_F32
    n_drop = rz.razor_compensation_mean_static(K[0], V[0], K.stride(1), K.stride(2), H, D, dt, w.ctx_len[0], w.n_sink,
                                               w.window[0], mean_k, mean_v)
    torch.cuda.synchronize()
    ref_k, ref_v, ref_nd = _means_via_cache(w, K, V)
    assert all(n == n_drop for n in ref_nd)                  # no retrieval heads here: every head drops the same rows
    got_k, got_v = to_f64(mean_k), to_f64(mean_v)
    drop = orc.dropped_positions(w.ctx_len[0], w.n_sink, w.window[0], False)
    assert len(drop) == n_drop
    for g in range(H):
        assert rel_inf(got_k[g], ref_k[g]) <= TOL_MEAN_REL, (g, rel_inf(got_k[g], ref_k[g]))
        assert rel_inf(got_v[g], ref_v[g]) <= TOL_MEAN_REL, (g, rel_inf(got_v[g], ref_v[g]))
        k_hat, v_hat, n_d = orc.compensation_token(to_f64(K[0, g]), to_f64(V[0, g]), drop)      # Eq. 4, fp64
        assert n_d == n_drop
        if n_d:
            assert rel_inf(got_k[g], k_hat) <= TOL_MEAN_REL, (g, rel_inf(got_k[g], k_hat))
            assert rel_inf(got_v[g], v_hat) <= TOL_MEAN_REL, (g, rel_inf(got_v[g], v_hat))
        else:
            assert not got_k[g].any() and not got_v[g].any()
    return n_drop


def test_static_scratch_means_match_the_cache_path_on_two_calls_in_a_row():
    # call 1: bf16, 8 heads, 5000 tokens; call 2 reuses the same built-in array with another shape and dtype
    w1 = synth.Workload("noalloc1", 1, 1, 8, 8, 128, "bf16", [5000], [700], 4, 0, 1, 31337)
    w2 = synth.Workload("noalloc2", 1, 1, 3, 3, 64, "f32", [1234], [100], 2, 0, 1, 31338)
    assert _check_static(w1) == 5000 - 4 - 700
    assert _check_static(w2) == 1234 - 2 - 100
    # nothing dropped: zeros, no read of K or V
    w3 = synth.Workload("noalloc3", 1, 1, 2, 2, 128, "bf16", [50], [100], 4, 0, 1, 31339)
    assert _check_static(w3) == 0


def test_static_scratch_with_strided_rows_and_with_the_most_heads_it_takes():
    w1 = synth.Workload("noalloc4", 1, 1, 5, 5, 64, "bf16", [2100], [300], 3, 0, 1, 31340)
    assert _check_static(w1, strided=True) == 2100 - 3 - 300
    w2 = synth.Workload("noalloc5", 1, 1, 64, 64, 128, "bf16", [900], [120], 4, 0, 1, 31341)    # 64 heads: the limit
    assert _check_static(w2) == 900 - 4 - 120


def test_static_scratch_call_on_a_second_stream_ordered_by_an_event():
    """The built-in array is shared by every call on the device: a call on another stream is fine as long as
    it is ordered behind the call before (here by an event), and gives the oracle's means too."""
    w = synth.Workload("noalloc6", 1, 1, 4, 4, 128, "bf16", [3000], [500], 4, 0, 1, 31342)
    K, V = synth.make_dense_kv(w, 0, DEV)
    H, D = w.n_kv_heads, w.head_dim
    out = [torch.empty((H, D), dtype=torch.float32, device=DEV) for _ in range(4)]
    rz.razor_compensation_mean_static(K[0], V[0], K.stride(1), K.stride(2), H, D, rz.RAZOR_BF16, 3000, 4, 500, out[0], out[1])
    done = torch.cuda.Event()
    done.record()
    side = torch.cuda.Stream()
    side.wait_event(done)
    with torch.cuda.stream(side):
        nd = rz.razor_compensation_mean_static(K[0], V[0], K.stride(1), K.stride(2), H, D, rz.RAZOR_BF16, 2000, 4, 300,
                                               out[2], out[3], stream=side.cuda_stream)
    torch.cuda.synchronize()
    assert nd == 2000 - 4 - 300
    for (n, win, mk, mv) in ((3000, 500, out[0], out[1]), (2000, 300, out[2], out[3])):
        drop = orc.dropped_positions(n, 4, win, False)
        for g in range(H):
            k_hat, v_hat, _ = orc.compensation_token(to_f64(K[0, g]), to_f64(V[0, g]), drop)
            assert rel_inf(to_f64(mk)[g], k_hat) <= TOL_MEAN_REL and rel_inf(to_f64(mv)[g], v_hat) <= TOL_MEAN_REL


def test_static_scratch_rejects_what_does_not_fit():
    z = torch.zeros((65, 64), dtype=torch.float32, device=DEV)
    with pytest.raises(rz.RazorError) as e:
        rz.razor_compensation_mean_static(z, z, 64, 64, 65, 64, rz.RAZOR_F32, 1, 0, 0, z, z)
    assert e.value.status == -5                              # more heads than the built-in scratch holds
    with pytest.raises(rz.RazorError) as e:
        rz.razor_compensation_mean_static(z, z, 64, 64, 2, 96, rz.RAZOR_F32, 1, 0, 0, z, z)
    assert e.value.status == -3
