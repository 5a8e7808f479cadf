"""Pins for the CPU oracle: each check ties an oracle function to something other than itself
(brute force on tiny inputs, closed forms, library routines on special cases, the figure the
paper prints under Table 2), and the mutation tests show that plausible mistakes fail them."""
import math
import os

import numpy as np
import pytest
from scipy.special import softmax as scipy_softmax

from oracle import razor_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table2_hyperparameters.txt")


def _golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                out[k] = float(v)
    return out


def _rng(seed):
    return np.random.default_rng(seed)


def brute_full_attention(q, K, V, scale):
    """Textbook softmax attention written with scalar loops (independent of numpy's matmul path)."""
    n, d = len(K), len(q)
    logits = [scale * sum(float(q[i]) * float(K[t][i]) for i in range(d)) for t in range(n)]
    mx = max(logits)
    w = [math.exp(s - mx) for s in logits]
    z = sum(w)
    return np.array([sum(w[t] * float(V[t][i]) for t in range(n)) / z for i in range(len(V[0]))])


# ------------------------------------------------------------------ kept set (Algorithm 1)
def test_kept_set_matches_per_position_rule_exhaustively():
    for n in range(0, 41):
        for n0 in range(0, 6):
            for w in range(0, 41, 1 if n < 12 else 3):
                kept = orc.kept_positions(n, n0, w, False)
                rule = [p for p in range(n) if p < n0 or p >= n - w]     # first N0 + recent W
                assert kept.tolist() == rule, (n, n0, w)
                drop = orc.dropped_positions(n, n0, w, False)
                assert len(drop) == max(0, n - n0 - w)
                assert sorted(set(kept.tolist()) | set(drop.tolist())) == list(range(n))
                if len(drop):
                    assert drop[0] == n0 and drop[-1] == n - w - 1        # one contiguous middle range
                assert orc.kept_positions(n, n0, w, True).tolist() == list(range(n))
                assert len(orc.dropped_positions(n, n0, w, True)) == 0


def test_buffer_length_table2():
    g = _golden()
    s0, c = int(g["buffer_threshold_S0"]), int(g["compression_ratio_C"])
    assert orc.buffer_length(32768, s0, c) == 6553          # floor(32768 / 5)
    assert orc.buffer_length(8000, s0, c) == 4000           # threshold dominates
    assert orc.buffer_length(20000, s0, c) == 4000
    assert orc.buffer_length(20005, s0, c) == 4001
    assert orc.buffer_length(131072, s0, c) == 26214


def test_long_context_compression_matches_paper_3_125x():
    g = _golden()
    frac = g["induction_head_fraction"] + g["echo_head_fraction"]          # 15 % of heads protected
    n_heads = 100
    ratio = orc.compression_ratio(50_000_000, n_heads, int(round(frac * n_heads)), int(g["sink_token_num"]),
                                  int(g["buffer_threshold_S0"]), int(g["compression_ratio_C"]))
    assert abs(ratio - g["long_context_compression"]) < 1e-4
    # closed form at finite N: heads*N / (r*N + (H-r)*(N0 + W + 1))
    n = 32768
    w = orc.buffer_length(n, 4000, 5)
    expect = 32 * n / (5 * n + 27 * (4 + w + 1))
    assert abs(orc.compression_ratio(n, 32, 5, 4, 4000, 5) - expect) < 1e-12
    assert 3.0 < expect < 3.125


def test_gqa_group_rule():
    flags = [0, 0, 0, 0, 0, 1, 0, 0, 0, 0, 0, 0, 1, 1, 1, 1]
    assert orc.kv_head_is_retrieval(flags, 4).tolist() == [0, 1, 0, 1]
    assert orc.kv_head_is_retrieval(flags, 1).tolist() == flags
    assert orc.kv_head_is_retrieval([0] * 8, 4).tolist() == [0, 0]


# ------------------------------------------------------------------ Eq. 4
def test_compensation_token_is_numpy_mean_of_slice():
    r = _rng(1)
    K, V = r.normal(size=(50, 8)), r.normal(size=(50, 8))
    drop = orc.dropped_positions(50, 4, 10, False)
    k_hat, v_hat, n_d = orc.compensation_token(K, V, drop)
    assert n_d == 36
    np.testing.assert_allclose(k_hat, np.mean(K[4:40], axis=0), rtol=0, atol=1e-14)
    np.testing.assert_allclose(v_hat, np.mean(V[4:40], axis=0), rtol=0, atol=1e-14)


def test_compensation_token_special_cases():
    r = _rng(2)
    K, V = r.normal(size=(20, 4)), r.normal(size=(20, 4))
    # one dropped token: the compensation token IS that token, bit for bit
    k_hat, v_hat, n_d = orc.compensation_token(K, V, np.array([7]))
    assert n_d == 1 and (k_hat == K[7]).all() and (v_hat == V[7]).all()
    # constant dropped rows: mean equals the constant
    K2, V2 = K.copy(), V.copy()
    K2[3:9] = K[3]
    V2[3:9] = V[5]
    k_hat, v_hat, _ = orc.compensation_token(K2, V2, np.arange(3, 9))
    np.testing.assert_allclose(k_hat, K[3], atol=1e-15)
    np.testing.assert_allclose(v_hat, V[5], atol=1e-15)
    # linear in K
    a, _, _ = orc.compensation_token(K, V, np.arange(2, 11))
    b, _, _ = orc.compensation_token(3.0 * K + 1.0, V, np.arange(2, 11))
    np.testing.assert_allclose(b, 3.0 * a + 1.0, atol=1e-13)
    # nothing dropped: zero vectors, count zero, never 0/0
    k_hat, v_hat, n_d = orc.compensation_token(K, V, np.array([], dtype=np.int64))
    assert n_d == 0 and not k_hat.any() and not v_hat.any()


# ------------------------------------------------------------------ original attention
def test_full_attention_matches_scalar_brute_force_and_scipy():
    r = _rng(3)
    for n, d in [(1, 3), (7, 5), (33, 8)]:
        q, K, V = r.normal(size=d), r.normal(size=(n, d)), r.normal(size=(n, d))
        for scale in (1.0, 1 / math.sqrt(d)):
            got = orc.full_attention(q, K, V, scale)
            np.testing.assert_allclose(got, brute_full_attention(q, K, V, scale), rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(got, scipy_softmax(scale * K @ q) @ V, rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------ Eq. 5: checks take the implementation
def _razor_out(impl, q, K, V, n0, w, retr, scale):
    n = len(K)
    kept = orc.kept_positions(n, n0, w, retr)
    drop = orc.dropped_positions(n, n0, w, retr)
    k_hat, v_hat, n_d = orc.compensation_token(K, V, drop)
    return impl(q, K[kept], V[kept], k_hat, v_hat, n_d, scale)


def check_window_covers_context(impl):
    r = _rng(10)
    q, K, V = r.normal(size=6), r.normal(size=(30, 6)), r.normal(size=(30, 6))
    for w in (26, 30, 100):
        np.testing.assert_allclose(_razor_out(impl, q, K, V, 4, w, False, 0.7),
                                   brute_full_attention(q, K, V, 0.7), rtol=1e-12, atol=1e-13)


def check_single_dropped_token(impl):
    r = _rng(11)
    q, K, V = r.normal(size=6), r.normal(size=(30, 6)), r.normal(size=(30, 6))
    np.testing.assert_allclose(_razor_out(impl, q, K, V, 4, 25, False, 0.5),
                               brute_full_attention(q, K, V, 0.5), rtol=1e-12, atol=1e-13)


def check_identical_dropped_tokens(impl):
    r = _rng(12)
    q, K, V = r.normal(size=6), r.normal(size=(40, 6)), r.normal(size=(40, 6))
    K[4:30] = r.normal(size=6)
    V[4:30] = r.normal(size=6)
    np.testing.assert_allclose(_razor_out(impl, q, K, V, 4, 10, False, 1.0),
                               brute_full_attention(q, K, V, 1.0), rtol=1e-12, atol=1e-13)


def check_replicated_compensation_token(impl):
    """Eq. 5 == ordinary softmax attention over the kept rows plus (k_hat, v_hat) repeated N_d times."""
    r = _rng(13)
    q, K, V = r.normal(size=5), r.normal(size=(25, 5)), r.normal(size=(25, 5))
    kept = orc.kept_positions(25, 2, 6, False)
    drop = orc.dropped_positions(25, 2, 6, False)
    k_hat, v_hat, n_d = orc.compensation_token(K, V, drop)
    assert n_d == 17
    K_aug = np.vstack([K[kept]] + [k_hat[None]] * n_d)
    V_aug = np.vstack([V[kept]] + [v_hat[None]] * n_d)
    expect = scipy_softmax(0.9 * (K_aug @ q)) @ V_aug
    np.testing.assert_allclose(impl(q, K[kept], V[kept], k_hat, v_hat, n_d, 0.9), expect, rtol=1e-12, atol=1e-13)


def check_log_count_form(impl):
    """N_d * exp(s) == exp(s + ln N_d): the count may enter as an additive term on the logit."""
    r = _rng(14)
    q, K, V = r.normal(size=5), r.normal(size=(9, 5)), r.normal(size=(9, 5))
    k_hat, v_hat, n_d, scale = r.normal(size=5), r.normal(size=5), 37, 0.8
    s = np.concatenate([scale * (K @ q), [scale * (k_hat @ q) + math.log(n_d)]])
    expect = scipy_softmax(s) @ np.vstack([V, v_hat[None]])
    np.testing.assert_allclose(impl(q, K, V, k_hat, v_hat, n_d, scale), expect, rtol=1e-12, atol=1e-13)


def check_large_logits_are_stable(impl):
    r = _rng(15)
    q, K, V = 40 * r.normal(size=5), 40 * r.normal(size=(9, 5)), r.normal(size=(9, 5))
    out = impl(q, K, V, 40 * r.normal(size=5), r.normal(size=5), 5, 1.0)
    assert np.isfinite(out).all()


EQ5_CHECKS = [check_window_covers_context, check_single_dropped_token, check_identical_dropped_tokens,
              check_replicated_compensation_token, check_log_count_form, check_large_logits_are_stable]


@pytest.mark.parametrize("check", EQ5_CHECKS, ids=lambda f: f.__name__)
def test_eq5_pins(check):
    check(orc.compensated_attention)


def _mutants():
    """Plausible mistakes planted in Eq. 5 (on the CPU, in copies of the oracle's formula)."""
    def base(q, K, V, k_hat, v_hat, n_d, scale, *, cnt_num=True, cnt_den=True, sign=1.0, scale_c=True,
             swap=False, sub_max=True):
        s = scale * (K @ q)
        s_c = (scale if scale_c else 1.0) * sign * float(q @ k_hat)
        m = max(s.max(), s_c) if sub_max else 0.0
        w, e_c = np.exp(s - m), float(np.exp(np.float64(s_c - m)))
        vv = k_hat if swap else v_hat
        num = ((n_d if cnt_num else min(n_d, 1)) * e_c) * vv + w @ V
        den = ((n_d if cnt_den else min(n_d, 1)) * e_c) + w.sum()
        return num / den
    return {
        "count_missing_everywhere": lambda *a: base(*a, cnt_num=False, cnt_den=False),
        "count_missing_in_denominator": lambda *a: base(*a, cnt_den=False),
        "count_missing_in_numerator": lambda *a: base(*a, cnt_num=False),
        "compensation_logit_sign": lambda *a: base(*a, sign=-1.0),
        "compensation_logit_unscaled": lambda *a: base(*a, scale_c=False),
        "k_hat_used_as_value": lambda *a: base(*a, swap=True),
        "no_max_subtraction": lambda *a: base(*a, sub_max=False),
    }


@pytest.mark.parametrize("name", list(_mutants()))
def test_eq5_pins_catch_planted_mistakes(name):
    impl = _mutants()[name]
    failed = 0
    for check in EQ5_CHECKS:
        try:
            with np.errstate(all="ignore"):
                check(impl)
        except (AssertionError, OverflowError):
            failed += 1
    assert failed >= 1, f"mutant {name} passed every pin"


def test_kept_set_pins_catch_planted_mistakes():
    """An off-by-one window or a missing sink range must change the kept set on small cases."""
    def off_by_one(n, n0, w):
        return [p for p in range(n) if p < n0 or p > n - w]
    def no_sinks(n, n0, w):
        return [p for p in range(n) if p >= n - w]
    diff1 = diff2 = 0
    for n in range(1, 30):
        got = orc.kept_positions(n, 2, 5, False).tolist()
        diff1 += got != off_by_one(n, 2, 5)
        diff2 += got != no_sinks(n, 2, 5)
    assert diff1 > 0 and diff2 > 0


# ------------------------------------------------------------------ further invariants
def test_jensen_bound_on_denominator():
    """exp is convex: N_d * exp(q.k_hat) <= sum_{m in D} exp(q.k_m)."""
    r = _rng(20)
    for _ in range(20):
        q, K = r.normal(size=8), r.normal(size=(60, 8))
        drop = orc.dropped_positions(60, 4, 12, False)
        k_hat, _, n_d = orc.compensation_token(K, K, drop)
        assert n_d * math.exp(q @ k_hat) <= np.exp(K[drop] @ q).sum() * (1 + 1e-12)


def test_kept_order_does_not_matter_and_scale_folds_into_query():
    r = _rng(21)
    q, K, V = r.normal(size=6), r.normal(size=(12, 6)), r.normal(size=(12, 6))
    k_hat, v_hat = r.normal(size=6), r.normal(size=6)
    a = orc.compensated_attention(q, K, V, k_hat, v_hat, 9, 0.4)
    p = r.permutation(12)
    np.testing.assert_allclose(orc.compensated_attention(q, K[p], V[p], k_hat, v_hat, 9, 0.4), a, rtol=1e-12)
    np.testing.assert_allclose(orc.compensated_attention(0.4 * q, K, V, k_hat, v_hat, 9, 1.0), a, rtol=1e-12)


def test_retrieval_head_is_original_attention():
    r = _rng(22)
    K, V, q = r.normal(size=(64, 8)), r.normal(size=(64, 8)), r.normal(size=8)
    hc = orc.compress_head(K, V, 64, 4, 8, True)
    assert hc.n_drop == 0 and len(hc.kept_pos) == 64
    np.testing.assert_allclose(orc.decode_head(q, hc, 0.3), brute_full_attention(q, K, V, 0.3), rtol=1e-12)


def test_compress_head_keeps_bits_and_ignores_padding_rows():
    r = _rng(23)
    K = r.normal(size=(70, 8)).astype(np.float32)
    V = r.normal(size=(70, 8)).astype(np.float32)
    hc = orc.compress_head(K, V, 50, 4, 10, False)           # rows 50..69 are padding
    assert hc.kept_pos.tolist() == [0, 1, 2, 3] + list(range(40, 50))
    assert hc.K.dtype == np.float32 and (hc.K == K[hc.kept_pos]).all() and (hc.V == V[hc.kept_pos]).all()
    assert hc.n_drop == 36
    np.testing.assert_allclose(hc.k_hat, K[4:40].astype(np.float64).mean(0), atol=1e-15)


def test_no_compensation_is_plain_truncation():
    r = _rng(24)
    K, V, q = r.normal(size=(40, 4)), r.normal(size=(40, 4)), r.normal(size=4)
    hc = orc.compress_head(K, V, 40, 2, 6, False)
    kept = hc.kept_pos
    np.testing.assert_allclose(orc.decode_head(q, hc, 1.0, use_compensation=False),
                               brute_full_attention(q, K[kept], V[kept], 1.0), rtol=1e-12)


def test_append_is_recompression_of_the_longer_context():
    """FIFO eviction: after t appended tokens the kept set is [0,N0) + the last W of N+t positions."""
    r = _rng(25)
    n, n0, w, d = 20, 2, 6, 4
    K, V = r.normal(size=(n, d)), r.normal(size=(n, d))
    hist = orc.DenseHistory(K, V, n, n0, w, False)
    allK, allV = [K], [V]
    for t in range(1, 12):
        kn, vn = r.normal(size=d), r.normal(size=d)
        hist.append(kn, vn)
        allK.append(kn[None])
        allV.append(vn[None])
        hc = hist.cache()
        assert hc.kept_pos.tolist() == list(range(n0)) + list(range(n + t - w, n + t))
        assert hc.n_drop == n + t - n0 - w
        np.testing.assert_allclose(hc.k_hat, np.vstack(allK)[n0:n + t - w].mean(0), atol=1e-14)
        np.testing.assert_allclose(hc.v_hat, np.vstack(allV)[n0:n + t - w].mean(0), atol=1e-14)
    # a short context fills its window before anything is dropped
    hist = orc.DenseHistory(K[:5], V[:5], 5, n0, w, False)
    for t in range(1, 6):
        hist.append(r.normal(size=d), r.normal(size=d))
        hc = hist.cache()
        assert hc.n_drop == max(0, 5 + t - n0 - w)
        assert len(hc.kept_pos) == min(5 + t, n0 + w)


def test_decode_layer_gqa_equals_mha_with_duplicated_kv_heads():
    r = _rng(26)
    B, Hq, Hkv, N, D = 2, 8, 2, 30, 4
    K, V, q = r.normal(size=(B, Hkv, N, D)), r.normal(size=(B, Hkv, N, D)), r.normal(size=(B, Hq, D))
    flags = [1, 0]
    caches = orc.compress_layer(K, V, [N, N - 7], flags, 2, [5, 5])
    out = orc.decode_layer(q, caches, 0.5)
    Kd, Vd = np.repeat(K, 4, axis=1), np.repeat(V, 4, axis=1)
    caches_d = orc.compress_layer(Kd, Vd, [N, N - 7], np.repeat(flags, 4), 2, [5, 5])
    np.testing.assert_allclose(orc.decode_layer(q, caches_d, 0.5), out, rtol=1e-13)


def test_needle_is_recalled_only_by_the_retrieval_head():
    """Tiny configuration: a key aligned with the query at position 200 sits in the dropped range
    [4, 448) of heads 1-3; only head 0 (retrieval) returns (approximately) that token's value."""
    from paper_2407_15891_b200 import synth
    w = synth.workload("cfg1")
    K, V = synth.make_dense_kv(w, 0)
    q = synth.make_queries(w, 0, 0)
    K, V, q = K.numpy(), V.numpy(), q.numpy()
    caches = orc.compress_layer(K, V, w.ctx_len, w.retrieval(0), w.n_sink, w.window)
    out = orc.decode_layer(q, caches, 1 / math.sqrt(w.head_dim))
    assert caches[0][1].n_drop == 444 and caches[0][0].n_drop == 0
    err0 = np.abs(out[0, 0] - V[0, 0, 200]).max()
    assert err0 < 0.05
    for h in (1, 2, 3):
        assert np.abs(out[0, h] - V[0, h, 200]).max() > 0.5


# ------------------------------------------------------------------ several new tokens at once (verify step)
def test_multi_query_single_token_is_the_decode_step():
    rng = _rng(70)
    K, V, q = rng.standard_normal((90, 16)), rng.standard_normal((90, 16)), rng.standard_normal((1, 16))
    for retr in (False, True):
        a = orc.multi_query_attention(q, K, V, 4, 20, retr, 0.3)[0]
        b = orc.decode_head(q[0], orc.compress_head(K, V, 90, 4, 20, retr), 0.3)
        assert np.allclose(a, b, rtol=0, atol=1e-14)


def test_multi_query_on_a_full_cache_is_causal_full_attention():
    """Retrieval head, or a window covering everything: query t equals brute-force attention over the
    first N + t + 1 tokens, and tokens after a query do not influence it."""
    rng = _rng(71)
    n, T, d = 37, 5, 8
    K, V, qs = rng.standard_normal((n + T, d)), rng.standard_normal((n + T, d)), rng.standard_normal((T, d))
    for retr, win in ((True, 3), (False, 100)):
        out = orc.multi_query_attention(qs, K, V, 2, max(win, T), retr, 0.5)
        for t in range(T):
            ref = brute_full_attention(qs[t], K[: n + t + 1], V[: n + t + 1], 0.5)
            assert np.allclose(out[t], ref, rtol=0, atol=1e-12)
    K2, V2 = K.copy(), V.copy()
    K2[n + 2:], V2[n + 2:] = 7.0, -3.0                        # change what comes after query 1
    a = orc.multi_query_attention(qs, K, V, 2, 10, False, 0.5)
    b = orc.multi_query_attention(qs, K2, V2, 2, 10, False, 0.5)
    assert np.allclose(a[:2], b[:2], rtol=0, atol=1e-14) and not np.allclose(a[2:], b[2:])


def test_multi_query_equals_eq5_with_replicated_compensation_token_and_causal_mask():
    rng = _rng(72)
    n, T, d, n0, w = 60, 4, 8, 3, 9
    K, V, qs = rng.standard_normal((n + T, d)), rng.standard_normal((n + T, d)), rng.standard_normal((T, d))
    out = orc.multi_query_attention(qs, K, V, n0, w, False, 0.4)
    total = n + T
    drop = np.arange(n0, total - w)
    k_hat, v_hat = K[drop].mean(0), V[drop].mean(0)
    for t in range(T):
        kept = [p for p in range(total) if (p < n0 or p >= total - w) and p <= n + t]
        Kx = np.concatenate([K[kept], np.repeat(k_hat[None], len(drop), 0)])
        Vx = np.concatenate([V[kept], np.repeat(v_hat[None], len(drop), 0)])
        ref = scipy_softmax(0.4 * Kx @ qs[t]) @ Vx
        assert np.allclose(out[t], ref, rtol=0, atol=1e-12)
    with pytest.raises(AssertionError):
        orc.multi_query_attention(qs, K, V, n0, T - 1, False, 0.4)   # window shorter than the round


# ------------------------------------------------------------------ ALiBi heads (Section 3.1, Eq. 1, Theorem 1)
def test_alibi_matches_scalar_brute_force_and_reduces_to_plain_attention():
    rng = _rng(80)
    n, d = 23, 6
    K, V, q = rng.standard_normal((n, d)), rng.standard_normal((n, d)), rng.standard_normal(d)
    pos = np.arange(n)
    slope, scale = 0.37, 0.8
    logits = [scale * sum(q[i] * K[t][i] for i in range(d)) - slope * ((n - 1) - t) for t in range(n)]
    w = [math.exp(x - max(logits)) for x in logits]
    ref = np.array([sum(w[t] * V[t][i] for t in range(n)) / sum(w) for i in range(d)])
    assert np.allclose(orc.alibi_attention(q, K, V, pos, n - 1, slope, scale), ref, rtol=0, atol=1e-13)
    # slope 0: ordinary attention; shifting every position by a constant changes nothing
    assert np.allclose(orc.alibi_attention(q, K, V, pos, n - 1, 0.0, scale), orc.full_attention(q, K, V, scale), atol=1e-14)
    assert np.allclose(orc.alibi_attention(q, K, V, pos + 1000, n + 999, slope, scale), ref, rtol=0, atol=1e-12)


def test_alibi_far_tokens_weigh_less_than_epsilon_beyond_the_vision_scope():
    """Theorem 1 with the bound on |q.k| taken from the data: if |scale q.k_n| <= B for every n, the weight
    of a key at distance > (2B - ln eps) / l_h is below eps, so truncating there changes the output by
    at most about eps * (number of far tokens) * max|v|."""
    rng = _rng(81)
    n, d, slope, scale, eps = 400, 8, 0.25, 0.5, 1e-3
    K, V, q = rng.standard_normal((n, d)), rng.standard_normal((n, d)), rng.standard_normal(d)
    B = np.abs(scale * K @ q).max()
    L_h = int(math.ceil((2 * B - math.log(eps)) / slope))
    assert L_h < n
    s = scale * (K @ q) - slope * ((n - 1) - np.arange(n))
    wts = np.exp(s - s.max()); wts /= wts.sum()
    assert wts[: n - 1 - L_h].max() <= eps
    full = orc.alibi_decode_head(q[None], K, V, -1, slope, scale)[0]
    cut = orc.alibi_decode_head(q[None], K, V, L_h + 1, slope, scale)[0]
    assert np.abs(full - cut).max() <= 2 * wts[: n - 1 - L_h].sum() * np.abs(V).max()
    assert np.abs(full - cut).max() < 1e-2


def test_alibi_decode_head_keeps_the_recent_window_and_is_causal():
    rng = _rng(82)
    n, T, d, win = 50, 3, 8, 12
    K, V, qs = rng.standard_normal((n + T, d)), rng.standard_normal((n + T, d)), rng.standard_normal((T, d))
    out = orc.alibi_decode_head(qs, K, V, win, 0.1, 0.6)
    total = n + T
    for t in range(T):
        vis = [p for p in range(total - win, total) if p <= n + t]
        ref = orc.alibi_attention(qs[t], K[vis], V[vis], np.array(vis), n + t, 0.1, 0.6)
        assert np.allclose(out[t], ref, rtol=0, atol=1e-13)
    K2 = K.copy(); K2[: total - win] += 5.0                  # tokens outside the window do not matter
    assert np.allclose(orc.alibi_decode_head(qs, K2, V, win, 0.1, 0.6), out, atol=1e-14)
    # slope 0 and a window: plain truncation (the Table 1 scheme) of the decode oracle
    hc = orc.compress_head(K[: n + 1], V[: n + 1], n + 1, 0, win, False)
    assert np.allclose(orc.alibi_decode_head(qs[:1], K[: n + 1], V[: n + 1], win, 0.0, 0.6)[0],
                       orc.decode_head(qs[0], hc, 0.6, use_compensation=False), atol=1e-13)


# ------------------------------------------------------------------ retrieval-head identification (Section 3.3)
def test_scores_of_a_head_with_uniform_attention_have_a_closed_form():
    """q = 0: every causal weight is 1 / (m + 1), so both scores are mean_m (number of earlier copies) / (m + 1)."""
    n, P, d = 40, 10, 4
    K = _rng(90).standard_normal((n, d))
    e, i = orc.echo_induction_scores(np.zeros((n, d)), K, P, 1.0)
    ref = np.mean([(m // P) / (m + 1) for m in range(P, n)])
    assert abs(e - ref) < 1e-14 and abs(i - ref) < 1e-14


def test_scores_single_out_echo_and_induction_heads():
    """Keys that are one-hot in the token identity: a query that looks for its own token is an echo head, a
    query that looks for the token BEFORE a key's position is an induction head (it lands on the successor)."""
    P, reps, beta = 12, 4, 30.0
    n = P * reps
    ids = np.arange(n) % P
    K = np.eye(P)[ids]                                         # key n encodes token id(n)
    q_echo = beta * np.eye(P)[ids]                             # looks for the same token
    K_prev = np.eye(P)[np.roll(ids, 1)]                        # key n encodes the token before n
    e1, i1 = orc.echo_induction_scores(q_echo, K, P, 1.0)
    e2, i2 = orc.echo_induction_scores(q_echo, K_prev, P, 1.0) # same query against "previous token" keys
    # the echo head also sees itself (position m holds the same token), so its echo mass is below 1 but large
    assert e1 > 0.6 and i1 < 1e-6
    assert i2 > 0.6 and e2 < 1e-6
    # brute force of one query
    m = n - 1
    s = np.array([float(q_echo[m] @ K[t]) for t in range(m + 1)])
    w = np.exp(s - s.max()); w /= w.sum()
    assert abs(sum(w[m - j * P] for j in range(1, reps)) - (reps - 1) / reps) < 1e-9


def test_selection_takes_top_induction_and_top_echo_heads():
    ind = np.linspace(0, 1, 100)                               # head 99 has the largest induction score
    echo = np.zeros(100); echo[7] = 0.9; echo[99] = 0.5
    mask = orc.select_retrieval_heads(echo, ind)               # 14 + 1
    assert mask.sum() == 15 and mask[86:].all() and mask[7] == 1 and mask[85] == 0
    assert orc.select_retrieval_heads(np.zeros(8), np.arange(8.0)).sum() == 2    # round(1.12)=1 by induction, 1 by echo (head 0)
    g = _golden()
    assert g["induction_head_fraction"] == 0.14 and g["echo_head_fraction"] == 0.01


def test_attention_over_no_tokens_is_defined_as_zeros():
    """Eq. 5 with an empty kept set and nothing dropped: numerator and denominator are empty sums.  A scalar-loop
    evaluation gives num = 0 and den = 0; the reading taken is out = num (zeros), never 0/0."""
    D = 8
    q = np.arange(D, dtype=np.float64)
    num, den = np.zeros(D), 0.0
    for _ in range(0):                                   # the sums of Eq. 5 over zero kept tokens
        pass
    assert den == 0.0
    hc = orc.compress_head(np.zeros((0, D)), np.zeros((0, D)), 0, 4, 16, False)
    assert len(hc.kept_pos) == 0 and hc.n_drop == 0
    out = orc.decode_head(q, hc, 0.5)
    assert out.shape == (D,) and (out == num).all()
    # one token: attention returns that token's value, whatever the logit
    K1, V1 = np.ones((1, D)), np.arange(D, dtype=np.float64)[None] * 3.0
    assert np.allclose(orc.decode_head(q, orc.compress_head(K1, V1, 1, 4, 16, False), 0.5), V1[0])
