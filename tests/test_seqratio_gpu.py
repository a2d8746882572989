"""GPU parity of the response-level importance ratio (MRL_RATIO_SEQUENCE; App. H, data-level coupling) on the
logits-in and the hidden-in entry points, against the oracle."""
import pytest
import torch

from oracle import mrl_oracle as O
from paper_2605_07244_b200 import binding as B
from paper_2605_07244_b200 import build

from helpers import GRAD_REL_L2_BF16, GRAD_REL_L2_F32, LOGP_ATOL, LOSS_RTOL, make_lp, oracle_lp, rel_l2, run_gpu_policy_loss
from test_lmhead_gpu import run_gpu_lmhead, toy as lm_toy

pytestmark = pytest.mark.gpu
SEQ_TIE = 1e-4      # |w - clip bound| below this: float32 log-probs summed over a response may decide either way


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    B.lib()


def toy(N, V, S, dtype, seed, mask_p=None, noise=0.08, pad=0):
    g = torch.Generator().manual_seed(seed)
    z = (torch.randn(N, V + pad, generator=g) * 2.0).to(dtype)
    ids = torch.randint(0, V, (N,), generator=g, dtype=torch.int32)
    cuts = sorted(torch.randperm(N - 1, generator=g)[:S - 1].add(1).tolist()) if S > 1 else []
    cu = torch.tensor([0] + cuts + [N], dtype=torch.int32)
    adv = torch.randn(S, generator=g)
    mask = None if mask_p is None else (torch.rand(N, generator=g) < mask_p).to(torch.uint8)
    logp, _, _ = O.token_logprobs(z[:, :V], ids, mask)
    old = (logp + torch.randn(N, generator=g, dtype=torch.float64) * noise).float()
    nllw = (torch.rand(N, generator=g) < 0.2).float()
    return z, ids, mask, cu, adv, old, nllw


def compare(got, ref, dz_got, dz_ref, tol):
    assert got["status"] == 0
    assert (got["logp"].double() - ref["logp"]).abs().max() <= LOGP_ATOL
    tie = ref["seq_margin"] < SEQ_TIE
    assert not tie.any(), "a response sits on the clip boundary: change the seed"
    for k, name, terms in ((0, "loss_pg", "seq_term"), (1, "loss_nll", "nll_term")):
        L = ref[name]
        # Each float32 log-prob carries ~1e-6 of absolute error (|logp| ~ 10); the response-level ratio exponentiates
        # the sum of a response's T of them, so a term's relative error grows like 1e-6 sqrt(T) .. 1e-6 T.  The
        # stated 1e-5 is therefore taken relative to the total magnitude of the terms, not to their cancelling sum.
        scale = max(abs(L), float(ref[terms].abs().sum()))
        assert abs(float(got["loss"][k]) - L) <= LOSS_RTOL * scale + 1e-12, f"{name}: {float(got['loss'][k])} vs {L}"
    assert int(got["stats"][0]) == ref["stats"][0] and int(got["stats"][1]) == ref["stats"][1]
    if dz_got is not None:
        assert torch.isfinite(dz_got).all()
        assert rel_l2(dz_got, dz_ref) <= tol
        zero = ref["g"] == 0
        if zero.any():
            assert float(dz_got[zero].abs().max()) == 0


@pytest.mark.parametrize("N,V,S,dtype,pad,mask_p", [
    (64, 1000, 6, torch.float32, 0, 0.8),          # general kernel, float32
    (40, 999, 5, torch.bfloat16, 3, None),         # general kernel, bf16, unaligned
    (90, 4096, 7, torch.bfloat16, 0, 0.9),         # streaming kernel, 256-bit
    (50, 40008, 4, torch.bfloat16, 0, None),       # streaming kernel, 128-bit, ragged
    (24, 151936, 3, torch.bfloat16, 0, 0.9),       # full vocabulary
])
def test_sequence_ratio_logits_in(N, V, S, dtype, pad, mask_p):
    z, ids, mask, cu, adv, old, nllw = toy(N, V, S, dtype, seed=N + V, mask_p=mask_p, pad=pad)
    lp = make_lp(nll_coeff=0.05, ratio_level=B.RATIO_SEQUENCE)
    got = run_gpu_policy_loss(z, ids, mask, cu, adv, old, None, nllw, lp, V=V)
    ref = O.policy_loss_sequence_ratio(z[:, :V], ids, mask, cu, adv, old, nllw, oracle_lp(lp))
    assert not ref["seq_clipped"].all()          # the comparison sees clipped and unclipped responses
    compare(got, ref, got["dlogits"][:, :V].double(), ref["dlogits"],
            GRAD_REL_L2_BF16 if dtype == torch.bfloat16 else GRAD_REL_L2_F32)
    # forward only gives the same scalars
    fwd = run_gpu_policy_loss(z, ids, mask, cu, adv, old, None, nllw, lp, V=V, want_dlogits=False)
    assert torch.equal(fwd["loss"], got["loss"]) and torch.equal(fwd["logp"], got["logp"])


def test_sequence_ratio_rejects_token_weights_and_unknown_levels():
    z, ids, mask, cu, adv, old, nllw = toy(16, 64, 2, torch.float32, seed=1)
    with pytest.raises(B.MrlError):
        run_gpu_policy_loss(z, ids, None, cu, adv, old, torch.ones(16), None, make_lp(ratio_level=B.RATIO_SEQUENCE))
    with pytest.raises(B.MrlError):
        run_gpu_policy_loss(z, ids, None, cu, adv, old, None, None, make_lp(ratio_level=7))


@pytest.mark.parametrize("N,H,V,S,mask_p", [(300, 128, 1000, 12, None), (260, 192, 40000, 9, 0.8)])
def test_sequence_ratio_hidden_in(N, H, V, S, mask_p):
    hidden, W, ids, mask, cu, adv, _, g = lm_toy(N, H, V, S, seed=N + V, mask_p=mask_p)
    zz = hidden.double() @ W.double().T
    logp, _, _ = O.token_logprobs(zz, ids, mask)
    old = (logp + torch.randn(N, generator=g, dtype=torch.float64) * 0.03).float()
    nllw = (torch.rand(N, generator=g) < 0.2).float()
    lp = make_lp(nll_coeff=0.05, ratio_level=B.RATIO_SEQUENCE)
    got = run_gpu_lmhead(hidden, W, ids, mask, cu, adv, old, None, nllw, lp)
    ref = O.policy_loss_sequence_ratio(zz, ids, mask, cu, adv, old, nllw, oracle_lp(lp))
    compare(got, ref, None, None, 0)
    dz = ref["dlogits"]
    assert rel_l2(got["dH"].double(), dz @ W.double()) <= GRAD_REL_L2_BF16
    assert rel_l2(got["dW"].double(), dz.T @ hidden.double()) <= GRAD_REL_L2_BF16


@pytest.mark.parametrize("N,V,dtype", [(40, 1000, torch.float32), (36, 8192, torch.bfloat16)])
def test_rows_outside_every_sequence_get_no_gradient(N, V, dtype):
    """cu_seqlens may stop short of N (the contract asks for cu[S] = N, but only the device sees the array): the rows
    no response covers must come out with zero gradient rows and logp = 0, and must not disturb the covered rows."""
    S, Nc = 3, N - 9
    z, ids, _, _, adv, old, nllw = toy(N, V, S, dtype, seed=5 + V)
    cu = torch.tensor([0, 7, 19, Nc], dtype=torch.int32)
    lp = make_lp(nll_coeff=0.05, ratio_level=B.RATIO_SEQUENCE)
    got = run_gpu_policy_loss(z, ids, None, cu, adv, old, None, nllw, lp, V=V)
    ref = O.policy_loss_sequence_ratio(z[:Nc, :V], ids[:Nc], None, cu, adv, old[:Nc], nllw[:Nc], oracle_lp(lp))
    assert got["status"] == 0
    assert float(got["dlogits"][Nc:].abs().max()) == 0 and float(got["logp"][Nc:].abs().max()) == 0
    assert (got["logp"][:Nc].double() - ref["logp"]).abs().max() <= LOGP_ATOL
    scale = max(abs(ref["loss_pg"]), float(ref["seq_term"].abs().sum()))
    assert abs(float(got["loss"][0]) - ref["loss_pg"]) <= LOSS_RTOL * scale
    tol = GRAD_REL_L2_BF16 if dtype == torch.bfloat16 else GRAD_REL_L2_F32
    assert rel_l2(got["dlogits"][:Nc, :V].double(), ref["dlogits"]) <= tol
