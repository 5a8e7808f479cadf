"""Retrieval-head identification (Section 3.3): the CUDA score reduction against the oracle, and the host-side
top-k selection (runs on CPU)."""
import numpy as np
import pytest
import torch

from oracle import razor_oracle as orc
from paper_2407_15891_b200 import binding as rz
from paper_2407_15891_b200 import build as rz_build
from paper_2407_15891_b200 import synth

DEV = "cuda:0"


def test_selection_matches_the_oracle_rule():
    rz_build.build()
    rng = np.random.default_rng(5)
    for n in (8, 32, 40, 100, 1024):
        echo, ind = rng.random(n).astype(np.float32), rng.random(n).astype(np.float32)
        ind[3] = ind[5]                                        # a tie: the lower index wins
        got = rz.razor_select_retrieval_heads(echo, ind)
        assert (got == orc.select_retrieval_heads(echo, ind)).all()
        assert got.sum() <= max(1, round(0.14 * n)) + max(1, round(0.01 * n))
    with pytest.raises(rz.RazorError):
        rz.razor_select_retrieval_heads([0.1], [0.2], frac_induction=1.5)


def _heads(n_heads, n, period, D, seed, dev):
    """Queries and keys of `n_heads` heads on `period` random tokens repeated: head 0 looks for its own token
    (echo head), head 1 for the token that followed its own token's earlier copies (induction head), the rest
    are unstructured.  bf16, built from the seeded generator."""
    emb = synth.normal_bf16(seed, synth.TAG_MISC, (period, D), dev).float()
    ids = torch.arange(n, device=dev) % period
    tok = emb[ids]                                             # [n, D]
    prev = emb[(ids - 1) % period]
    Q = synth.normal_bf16(seed, synth.TAG_Q, (n_heads, n, D), dev).float()
    K = synth.normal_bf16(seed, synth.TAG_K, (n_heads, n, D), dev).float()
    beta = 3.0
    K[0] = tok + 0.3 * K[0]; Q[0] = beta * tok
    if n_heads > 1:
        K[1] = prev + 0.3 * K[1]; Q[1] = beta * tok
    return Q.to(torch.bfloat16).contiguous(), K.to(torch.bfloat16).contiguous()


@pytest.mark.gpu
@pytest.mark.parametrize("D,n,period,heads", [(128, 384, 96, 5), (64, 300, 70, 4), (128, 1000, 333, 3), (64, 130, 64, 2), (64, 1500, 400, 2), (128, 100, 30, 2), (64, 40, 7, 3)])
def test_scores_match_the_oracle_on_small_inputs(D, n, period, heads):
    Q, K = _heads(heads, n, period, D, 4000 + D + n, DEV)
    echo, ind = rz.razor_head_scores(Q, K, period)
    torch.cuda.synchronize()
    scale = 1.0 / np.sqrt(D)
    Qh, Kh = Q.double().cpu().numpy(), K.double().cpu().numpy()
    for h in range(heads):
        e_ref, i_ref = orc.echo_induction_scores(Qh[h], Kh[h], period, scale)
        assert abs(float(echo[h]) - e_ref) <= 1e-5 + 1e-4 * e_ref, (h, float(echo[h]), e_ref)
        assert abs(float(ind[h]) - i_ref) <= 1e-5 + 1e-4 * i_ref, (h, float(ind[h]), i_ref)
    assert float(echo[0]) > 5 * float(echo[heads - 1]) if heads > 2 else True
    # literal scale (Eq. 3 prints no 1/sqrt(d)) on one head
    e1, i1 = rz.razor_head_scores(Q[:1].contiguous(), K[:1].contiguous(), period, sm_scale=0.05)
    e_ref, i_ref = orc.echo_induction_scores(Qh[0], Kh[0], period, 0.05)
    assert abs(float(e1[0]) - e_ref) <= 1e-5 + 1e-4 * e_ref and abs(float(i1[0]) - i_ref) <= 1e-5 + 1e-4 * i_ref


@pytest.mark.gpu
def test_paper_sized_input_and_selection():
    """2500 random tokens repeated 4 times (Section 3.3), 32 heads; the oracle checks the two structured heads
    and one unstructured head, and the selection must pick the structured ones."""
    n_heads, period, D = 32, 2500, 128
    n = 4 * period
    Q, K = _heads(n_heads, n, period, D, 77, DEV)
    echo, ind = rz.razor_head_scores(Q, K, period)
    torch.cuda.synchronize()
    echo, ind = echo.cpu().numpy(), ind.cpu().numpy()
    scale = 1.0 / np.sqrt(D)
    for h in (0, 1, 17):
        e_ref, i_ref = orc.echo_induction_scores(Q[h].double().cpu().numpy(), K[h].double().cpu().numpy(), period, scale)
        assert abs(echo[h] - e_ref) <= 1e-5 + 1e-4 * e_ref and abs(ind[h] - i_ref) <= 1e-5 + 1e-4 * i_ref
    mask = rz.razor_select_retrieval_heads(echo, ind)
    assert mask[0] == 1 and mask[1] == 1 and mask.sum() <= 5   # round(0.14 * 32) = 4 by induction, 1 by echo
    assert (mask == orc.select_retrieval_heads(echo, ind)).all()


@pytest.mark.gpu
def test_score_call_rejects_bad_arguments():
    Q = torch.zeros((2, 64, 64), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(rz.RazorError) as e:
        rz.razor_head_scores(Q, Q, 64)                         # period must be below n_tokens
    assert e.value.status == -1
    Q96 = torch.zeros((2, 64, 96), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(rz.RazorError) as e:
        rz.razor_head_scores(Q96, Q96, 16)
    assert e.value.status == -3
