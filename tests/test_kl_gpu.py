"""The KL penalty of Eq. (1) (beta R(theta): a per-token KL to a reference trace, its own loss term) on the CUDA
path against the oracle: logits-in through both row kernels, with the response-level ratio, through the fused LM
head, across accumulated calls, and together with the zero-row skip."""
import pytest
import torch

from oracle import mrl_oracle as O
from paper_2605_07244_b200 import binding as B
from paper_2605_07244_b200 import build

from helpers import (GRAD_REL_L2_BF16, GRAD_REL_L2_F32, LOGP_ATOL, LOSS_RTOL, KlTerm, compare_policy_loss, dev, make_lp,
                     oracle_lp, rel_l2, run_gpu_policy_loss)
import test_lmhead_gpu as LM
import test_seqratio_gpu as SR

pytestmark = pytest.mark.gpu
ESTIMATORS = [B.KL_K1, B.KL_K2, B.KL_K3]


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    B.lib()


def reference_trace(logp, g, spread=0.4):
    return (logp + spread * torch.randn(logp.numel(), generator=g, dtype=torch.float64)).float()


def check_kl(kl: KlTerm, ref, floor=0.1):
    # k1 is signed, so the term can be a cancelling sum: relative to max(|L|, floor * sum of |terms|)
    L = ref["loss_kl"]
    scale = max(abs(L), floor * float(ref["kl_term"].abs().sum()))
    assert abs(kl.value() - L) <= LOSS_RTOL * scale + 1e-12, f"loss_kl: {kl.value()} vs {L}"


@pytest.mark.parametrize("estimator", ESTIMATORS)
@pytest.mark.parametrize("agg", [B.AGG_TOKEN_MEAN, B.AGG_SEQ_MEAN_TOKEN_MEAN])
@pytest.mark.parametrize("N,V,S,dtype,pad,mask_p", [
    (64, 1000, 6, torch.float32, 0, 0.8),          # general kernel, float32
    (40, 999, 5, torch.bfloat16, 3, None),         # general kernel, bf16, unaligned
    (90, 4096, 7, torch.bfloat16, 0, 0.9),         # streaming kernel, 256-bit
    (50, 40008, 4, torch.bfloat16, 0, None),       # streaming kernel, 128-bit
    (12, 262144 + 16, 3, torch.bfloat16, 0, None),  # rows split over a pair of CTAs
])
def test_kl_term_logits_in(N, V, S, dtype, pad, mask_p, agg, estimator):
    z, ids, mask, cu, adv, old, nllw = SR.toy(N, V, S, dtype, seed=5 + estimator, mask_p=mask_p, pad=pad)
    g = torch.Generator().manual_seed(77)
    logp, _, _ = O.token_logprobs(z[:, :V], ids, mask)
    ref_trace = reference_trace(logp, g)
    tw = torch.rand(N, generator=g) + 0.5
    lp = make_lp(agg=agg, nll_coeff=0.05)
    kl = KlTerm(lp, ref_trace, 0.05, estimator)            # large beta so that the term matters in g
    got = run_gpu_policy_loss(z, ids, mask, cu, adv, old, tw, nllw, lp, V=V)
    ref = O.policy_loss(z[:, :V], ids, mask, cu, adv, old, tw, nllw, oracle_lp(lp), logp_ref=ref_trace)
    assert got["status"] == 0
    # group-centred advantages make the policy-gradient loss a cancelling sum: relative to a tenth of the sum of |terms|
    compare_policy_loss(got, ref, V, dtype, cancelling=True)
    check_kl(kl, ref)


@pytest.mark.parametrize("estimator", ESTIMATORS)
def test_kl_term_alone_and_app_a_coefficient(estimator):
    # no advantage, no NLL: the gradient is the penalty's alone, at the paper's beta = 1e-3
    z, ids, mask, cu, adv, old, _ = SR.toy(70, 8192, 5, torch.bfloat16, seed=3, mask_p=0.9)
    g = torch.Generator().manual_seed(8)
    logp, _, _ = O.token_logprobs(z, ids, mask)
    ref_trace = reference_trace(logp, g, spread=0.2)
    lp = make_lp()
    kl = KlTerm(lp, ref_trace, 1e-3, estimator)
    got = run_gpu_policy_loss(z, ids, mask, cu, torch.zeros(5), old, None, None, lp)
    ref = O.policy_loss(z, ids, mask, cu, torch.zeros(5), old, None, None, oracle_lp(lp), logp_ref=ref_trace)
    assert float(got["loss"][0]) == 0 and float(got["loss"][1]) == 0
    check_kl(kl, ref)
    assert rel_l2(got["dlogits"], ref["dlogits"]) <= GRAD_REL_L2_BF16
    live = ref["g"] != 0
    assert live.sum() == int(mask.sum())
    rows = (got["dlogits"].double()[live] - ref["dlogits"][live]).norm(dim=1) / ref["dlogits"][live].norm(dim=1)
    assert rows.max() <= 2 * GRAD_REL_L2_BF16


def test_rows_stay_live_under_the_zero_row_skip_while_the_term_is_on():
    z, ids, mask, cu, adv, old, _ = SR.toy(48, 4096, 4, torch.bfloat16, seed=9)
    adv = adv.clone()
    adv[1] = 0.0
    g = torch.Generator().manual_seed(1)
    logp, _, _ = O.token_logprobs(z, ids, mask)
    ref_trace = reference_trace(logp, g)
    lp = make_lp(flags=B.FLAG_SKIP_ZERO_ROWS)
    off = run_gpu_policy_loss(z, ids, mask, cu, adv, old, None, None, lp)
    a, b = int(cu[1]), int(cu[2])
    assert off["logp"][a:b].abs().max() == 0 and off["dlogits"][a:b].abs().max() == 0
    assert int(off["stats"][2]) == 48 - (b - a)
    kl = KlTerm(lp, ref_trace, 0.02, B.KL_K3)
    on = run_gpu_policy_loss(z, ids, mask, cu, adv, old, None, None, lp)
    ref = O.policy_loss(z, ids, mask, cu, adv, old, None, None, oracle_lp(lp), logp_ref=ref_trace)
    compare_policy_loss(on, ref, 4096, torch.bfloat16, cancelling=True)
    check_kl(kl, ref)
    assert int(on["stats"][2]) == 48 and on["dlogits"][a:b].abs().max() > 0


def test_kl_term_accumulates_across_calls_and_empty_call_clears_it():
    z, ids, mask, cu, adv, old, nllw = SR.toy(60, 4096, 6, torch.bfloat16, seed=13)
    g = torch.Generator().manual_seed(2)
    logp, _, _ = O.token_logprobs(z, ids, mask)
    ref_trace = reference_trace(logp, g)
    whole = make_lp(pg_den=60.0)
    ref = O.policy_loss(z, ids, mask, cu, adv, old, None, None,
                        O.LossParams(pg_denominator=60.0, kl_coeff=0.01, kl_estimator=O.KL_K3), logp_ref=ref_trace,
                        want_dlogits=False)
    cut_s = 3
    cut = int(cu[cut_s])
    lp = make_lp(pg_den=60.0, flags=B.FLAG_ACCUMULATE_LOSS)
    kl = KlTerm(lp, ref_trace[:cut], 0.01, B.KL_K3, init=0.0)
    first = run_gpu_policy_loss(z[:cut], ids[:cut], None, cu[:cut_s + 1], adv[:cut_s], old[:cut], None, None, lp,
                                loss_init=torch.zeros(2), stats_init=torch.zeros(4, dtype=torch.int64))
    part = kl.value()
    assert 0 < part < ref["loss_kl"]
    ref2 = dev(ref_trace[cut:], torch.float32)
    lp.logp_ref = ref2.data_ptr()
    run_gpu_policy_loss(z[cut:], ids[cut:], None, cu[cut_s:] - cut, adv[cut_s:], old[cut:], None, None, lp,
                        loss_init=first["loss"], stats_init=first["stats"])
    assert abs(kl.value() - ref["loss_kl"]) <= LOSS_RTOL * ref["loss_kl"]
    # an empty call without the accumulate flag writes zero
    lp0 = make_lp()
    kl0 = KlTerm(lp0, torch.zeros(1), 0.01, B.KL_K3, init=5.0)
    loss = torch.ones(2, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.mrl_policy_loss_fwd_bwd(torch.empty(0, 4096, dtype=torch.bfloat16, device="cuda"), torch.empty(0, dtype=torch.int32, device="cuda"),
                              None, torch.zeros(1, dtype=torch.int32, device="cuda"), torch.empty(0, device="cuda"), None,
                              None, None, lp0, None, None, loss, None, status,
                              torch.empty(256, dtype=torch.uint8, device="cuda"), V=4096)
    torch.cuda.synchronize()
    assert kl0.value() == 0 and float(loss.sum()) == 0
    del whole


@pytest.mark.parametrize("estimator", [B.KL_K1, B.KL_K3])
@pytest.mark.parametrize("N,V,S,dtype,pad,mask_p", [
    (64, 1000, 6, torch.float32, 0, 0.8),
    (90, 4096, 7, torch.bfloat16, 0, 0.9),
])
def test_kl_term_with_the_response_level_ratio(N, V, S, dtype, pad, mask_p, estimator):
    z, ids, mask, cu, adv, old, nllw = SR.toy(N, V, S, dtype, seed=21, mask_p=mask_p, pad=pad, noise=0.02)
    g = torch.Generator().manual_seed(4)
    logp, _, _ = O.token_logprobs(z[:, :V], ids, mask)
    ref_trace = reference_trace(logp, g)
    lp = make_lp(nll_coeff=0.05, ratio_level=B.RATIO_SEQUENCE)
    kl = KlTerm(lp, ref_trace, 0.05, estimator)
    got = run_gpu_policy_loss(z, ids, mask, cu, adv, old, None, nllw, lp, V=V)
    ref = O.policy_loss_sequence_ratio(z[:, :V], ids, mask, cu, adv, old, nllw, oracle_lp(lp), logp_ref=ref_trace)
    tol = GRAD_REL_L2_BF16 if dtype == torch.bfloat16 else GRAD_REL_L2_F32
    SR.compare(got, ref, got["dlogits"][:, :V].double(), ref["dlogits"], tol)
    check_kl(kl, ref)


@pytest.mark.parametrize("estimator", ESTIMATORS)
@pytest.mark.parametrize("seq", [False, True])
def test_kl_term_fused_lm_head(estimator, seq):
    N, H, V, S = 300, 128, 20000, 5
    hidden, W, ids, mask, cu, adv, old, g = LM.toy(N, H, V, S, seed=31, mask_p=0.9, noise=0.02 if seq else 0.1)
    logp, _, _ = O.token_logprobs(hidden.double() @ W.double().T, ids, mask)
    ref_trace = reference_trace(logp, g)
    lp = make_lp(ratio_level=B.RATIO_SEQUENCE if seq else B.RATIO_TOKEN)
    kl = KlTerm(lp, ref_trace, 0.05, estimator)
    got = LM.run_gpu_lmhead(hidden, W, ids, mask, cu, adv, old, None, None, lp)
    if seq:
        z = hidden.double() @ W.double().T
        ref = O.policy_loss_sequence_ratio(z, ids, mask, cu, adv, old, None, oracle_lp(lp), logp_ref=ref_trace)
        assert (got["logp"].double() - ref["logp"]).abs().max() <= LOGP_ATOL
        assert rel_l2(got["dH"], ref["dlogits"] @ W.double()) <= GRAD_REL_L2_BF16
        assert rel_l2(got["dW"], ref["dlogits"].T @ hidden.double()) <= GRAD_REL_L2_BF16
    else:
        ref = O.fused_lmhead_loss(hidden, W, ids, mask, cu, adv, old, None, None, oracle_lp(lp), logp_ref=ref_trace)
        LM.compare(got, ref)
    # here every log-prob carries the ~1e-6 absolute error of a float32-accumulated bf16 dot product and k1 is linear
    # in it, so the error of the sum is beta * 1e-6 whatever the sum cancels to: relative to the sum of |terms|
    check_kl(kl, ref, floor=1.0)


def test_kl_arguments_are_checked():
    z, ids, mask, cu, adv, old, _ = SR.toy(8, 1000, 2, torch.float32, seed=1)
    lp = make_lp()
    lp.logp_ref = dev(old).data_ptr()          # no place for the term
    with pytest.raises(B.MrlError):
        run_gpu_policy_loss(z, ids, mask, cu, adv, old, None, None, lp)
    lp = make_lp()
    kl = KlTerm(lp, old, 0.1, 7)               # unknown estimator
    with pytest.raises(B.MrlError):
        run_gpu_policy_loss(z, ids, mask, cu, adv, old, None, None, lp)
    del kl
