"""Pins of the oracle's KL penalty (Eq. (1)'s beta R(theta); App. A: a per-token KL to a reference as its own loss
term) against facts that hold independently of its code: the exact expectation identities of the sampled-token
estimators against scipy's relative entropy, non-negativity, closed forms for a constant log-ratio, finite
differences of the whole loss, and that the term vanishes without a reference."""
import math

import numpy as np
import pytest
import torch
from scipy.special import rel_entr

from oracle import mrl_oracle as O

F64 = torch.float64


def two_policies(V, seed, spread=1.0):
    g = torch.Generator().manual_seed(seed)
    z = torch.randn(V, generator=g, dtype=F64) * 1.5
    zr = z + spread * torch.randn(V, generator=g, dtype=F64)
    return z, zr, torch.softmax(z, 0), torch.softmax(zr, 0)


def per_token_k(z, zr, estimator):
    """k for every possible sampled token a of one position, through the oracle's own entry point (one row per a)."""
    V = z.numel()
    logits = z.repeat(V, 1)
    ids = torch.arange(V)
    logp_ref = torch.log_softmax(zr, 0)
    lp = O.LossParams(kl_coeff=1.0, kl_estimator=estimator, pg_denominator=1.0)    # c_t = 1: the raw estimate
    out = O.policy_loss(logits, ids, None, torch.tensor([0, V]), torch.zeros(1), None, lp=lp, logp_ref=logp_ref,
                        want_dlogits=False)
    return out["kl_term"]


@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("estimator", [O.KL_K1, O.KL_K3])
def test_expectation_under_the_policy_is_the_exact_kl(seed, estimator):
    z, zr, p, q = two_policies(11, seed)
    k = per_token_k(z, zr, estimator)
    want = float(rel_entr(p.numpy(), q.numpy()).sum())
    assert abs(float((p * k).sum()) - want) <= 1e-12 * max(1.0, want)


def test_k2_agrees_to_second_order_and_k3_from_above():
    z, zr, p, q = two_policies(9, 5, spread=1e-3)
    want = float(rel_entr(p.numpy(), q.numpy()).sum())
    k2 = per_token_k(z, zr, O.KL_K2)
    assert abs(float((p * k2).sum()) - want) <= 5e-3 * want            # third-order difference only
    z, zr, p, q = two_policies(9, 5, spread=1.0)
    k2 = per_token_k(z, zr, O.KL_K2)
    assert abs(float((p * k2).sum()) - float(rel_entr(p.numpy(), q.numpy()).sum())) > 1e-3   # and no more than that


def test_k3_is_nonnegative_and_vanishes_only_on_agreement():
    z, zr, p, q = two_policies(13, 7)
    k3 = per_token_k(z, zr, O.KL_K3)
    assert (k3 > 0).all()
    k_same = per_token_k(z, z + 3.0, O.KL_K3)                              # a shift of the logits is the same policy
    assert k_same.abs().max() <= 1e-15
    k1 = per_token_k(z, zr, O.KL_K1)
    assert (k1 < 0).any() and (k1 > 0).any()                               # k1 is signed; only its mean is a KL


@pytest.mark.parametrize("agg", [O.AGG_TOKEN_MEAN, O.AGG_SEQ_MEAN_TOKEN_MEAN])
def test_constant_log_ratio_gives_the_closed_form_in_both_aggregations(agg):
    g = torch.Generator().manual_seed(3)
    N, V, d0, beta = 23, 17, 0.3, 1e-3
    logits = torch.randn(N, V, generator=g, dtype=F64)
    ids = torch.randint(0, V, (N,), generator=g)
    mask = torch.ones(N, dtype=torch.uint8)
    mask[[2, 9, 22]] = 0
    cu = torch.tensor([0, 5, 5, 14, 23])
    logp, _, _ = O.token_logprobs(logits, ids, mask)
    n_seq = 3 if agg == O.AGG_SEQ_MEAN_TOKEN_MEAN else 4
    for est, k in [(O.KL_K1, d0), (O.KL_K2, d0 * d0 / 2), (O.KL_K3, math.exp(-d0) - 1 + d0)]:
        lp = O.LossParams(agg_mode=agg, kl_coeff=beta, kl_estimator=est, seq_denominator=float(n_seq))
        out = O.policy_loss(logits, ids, mask, cu, torch.zeros(4), None, lp=lp, logp_ref=logp - d0, want_dlogits=False)
        assert abs(out["loss_kl"] - beta * k) <= 1e-15                      # the coefficients sum to one
        assert out["loss_pg"] == 0 and out["loss_nll"] == 0
        assert (out["kl_term"][mask == 0] == 0).all() and (out["g"][mask == 0] == 0).all()


def total_loss(logits, ids, mask, cu, adv, logp_old, tw, nw, lp, logp_ref, seq):
    f = O.policy_loss_sequence_ratio if seq else O.policy_loss
    kw = dict(nll_weight=nw, lp=lp, want_dlogits=False, logp_ref=logp_ref)
    if not seq:
        kw["tok_weight"] = tw
    out = f(logits, ids, mask, cu, adv, logp_old, **kw)
    return out["loss_pg"] + out["loss_nll"] + out["loss_kl"]


@pytest.mark.parametrize("seq", [False, True])
@pytest.mark.parametrize("estimator", [O.KL_K1, O.KL_K2, O.KL_K3])
def test_dlogits_with_the_penalty_match_finite_differences(estimator, seq):
    g = torch.Generator().manual_seed(11 + estimator)
    N, V = 12, 9
    logits = torch.randn(N, V, generator=g, dtype=F64)
    ids = torch.randint(0, V, (N,), generator=g)
    mask = torch.ones(N, dtype=torch.uint8)
    mask[4] = 0
    cu = torch.tensor([0, 4, 9, 12])
    adv = torch.tensor([0.8, -1.1, 0.0], dtype=F64)
    logp, _, _ = O.token_logprobs(logits, ids, mask)
    logp_old = logp + 0.03 * torch.randn(N, generator=g, dtype=F64)        # inside the clip band: smooth loss
    logp_ref = logp + 0.5 * torch.randn(N, generator=g, dtype=F64)
    tw = None if seq else torch.rand(N, generator=g, dtype=F64) + 0.5
    nw = torch.zeros(N, dtype=F64)
    nw[9:] = 1.0
    lp = O.LossParams(kl_coeff=0.7, kl_estimator=estimator, nll_coeff=0.2,
                      ratio_level=O.RATIO_SEQUENCE if seq else O.RATIO_TOKEN)
    f = O.policy_loss_sequence_ratio if seq else O.policy_loss
    kw = dict(nll_weight=nw, lp=lp, logp_ref=logp_ref)
    if not seq:
        kw["tok_weight"] = tw
    dz = f(logits, ids, mask, cu, adv, logp_old, **kw)["dlogits"]
    h = 1e-6
    for (t, v) in [(0, int(ids[0])), (1, 3), (5, int(ids[5])), (6, 0), (10, int(ids[10])), (11, 2), (4, 1)]:
        zp, zm = logits.clone(), logits.clone()
        zp[t, v] += h
        zm[t, v] -= h
        fd = (total_loss(zp, ids, mask, cu, adv, logp_old, tw, nw, lp, logp_ref, seq)
              - total_loss(zm, ids, mask, cu, adv, logp_old, tw, nw, lp, logp_ref, seq)) / (2 * h)
        assert abs(fd - float(dz[t, v])) <= 1e-8, (t, v)


def test_no_reference_or_zero_beta_leaves_the_pass_unchanged():
    g = torch.Generator().manual_seed(2)
    N, V = 10, 8
    logits = torch.randn(N, V, generator=g, dtype=F64)
    ids = torch.randint(0, V, (N,), generator=g)
    cu = torch.tensor([0, 6, 10])
    adv = torch.tensor([1.0, -0.5], dtype=F64)
    logp, _, _ = O.token_logprobs(logits, ids, None)
    old = logp + 0.1 * torch.randn(N, generator=g, dtype=F64)
    base = O.policy_loss(logits, ids, None, cu, adv, old)
    z0 = O.policy_loss(logits, ids, None, cu, adv, old, lp=O.LossParams(kl_coeff=0.0), logp_ref=logp - 1.0)
    assert base["loss_kl"] == 0 and z0["loss_kl"] == 0
    assert torch.equal(base["dlogits"], z0["dlogits"]) and torch.equal(base["g"], z0["g"])
    on = O.policy_loss(logits, ids, None, cu, adv, old, lp=O.LossParams(kl_coeff=1e-3), logp_ref=logp - 1.0)
    assert on["loss_pg"] == base["loss_pg"] and on["loss_kl"] > 0          # the penalty is its own term
    # k3' = 1 - e^{-d} > 0 for d > 0: the penalty pushes the sampled token's log-prob down, i.e. g down
    assert (on["g"] < base["g"]).all()
