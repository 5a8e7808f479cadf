"""The seeded input generator: deterministic, windowable, N(0,1)-shaped, structured as the workloads say."""
import numpy as np
import torch

from paper_2407_15891_b200 import synth


def test_generator_is_deterministic_and_windowable():
    a = synth.normal_bf16(5, synth.TAG_K, (3, 7, 8), sub=2)
    b = synth.normal_bf16(5, synth.TAG_K, (3, 7, 8), sub=2, chunk=64)
    assert torch.equal(a, b)
    flat = a.reshape(-1)
    win = synth.normal_bf16(5, synth.TAG_K, (40,), sub=2, offset=56)
    assert torch.equal(win, flat[56:96])
    assert not torch.equal(a, synth.normal_bf16(6, synth.TAG_K, (3, 7, 8), sub=2))
    assert not torch.equal(a, synth.normal_bf16(5, synth.TAG_V, (3, 7, 8), sub=2))


def test_values_look_standard_normal():
    x = synth.normal_bf16(1, synth.TAG_Q, (1 << 18,)).double()
    assert abs(x.mean().item()) < 0.01 and abs(x.std().item() - 1.0) < 0.01
    assert 3.5 < x.abs().max().item() < 6.0
    assert abs((x.abs() < 1.0).double().mean().item() - 0.6827) < 0.01


def test_workload_structure():
    w2 = synth.workload("cfg2")
    assert w2.window[0] == 6553 and int(w2.retrieval(0).sum()) == 5
    w3 = synth.workload("cfg3")
    assert all(int(w3.retrieval(l).sum()) == 6 for l in range(40))
    assert len({tuple(w3.retrieval(l)) for l in range(40)}) > 20          # per-layer sets differ
    w4 = synth.workload("cfg4")
    assert w4.group == 4 and int(w4.retrieval(3).sum()) == 2
    w5 = synth.workload("cfg5")
    assert min(w5.ctx_len) >= 4096 and max(w5.ctx_len) <= 131072 and len(set(w5.ctx_len)) == 64
    assert all(wd == max(4000, n // 5) for wd, n in zip(w5.window, w5.ctx_len))
    w1 = synth.workload("cfg1")
    K, V = synth.make_dense_kv(w1, 0)
    assert K.dtype == torch.float32 and K.shape == (1, 4, 512, 64)
    # sinks carry 4x key norm; the needle's logit is about beta = 20
    assert K[0, 1, :4].norm(dim=-1).mean() > 3 * K[0, 1, 4:].norm(dim=-1).mean()
    q = synth.make_queries(w1, 0, 0)
    assert abs(float(q[0, 0] @ K[0, 0, 200]) / 8.0 - 20.0) < 1.0
    kh, vh = synth.make_dense_head(w1, 0, 0, 2)
    keep = torch.ones(512, dtype=torch.bool)
    keep[200] = False                                                     # the planted needle key
    assert torch.equal(kh[keep], K[0, 2][keep]) and torch.equal(vh, V[0, 2])
