"""Pins of the oracle's response-level importance ratio (App. H, data-level coupling): relations to the
token-level pass it must reduce to, closed forms, hand-worked clip cases and finite differences."""
import math

import pytest
import torch

from oracle import mrl_oracle as O

F64 = torch.float64


def _toy(N=30, V=11, S=5, seed=3):
    g = torch.Generator().manual_seed(seed)
    z = torch.randn(N, V, generator=g, dtype=F64) * 2
    ids = torch.randint(0, V, (N,), generator=g)
    cuts = sorted(torch.randperm(N - 1, generator=g)[:S - 1].add(1).tolist())
    cu = torch.tensor([0] + cuts + [N])
    adv = torch.randn(S, generator=g, dtype=F64)
    mask = (torch.rand(N, generator=g) < 0.85).to(torch.uint8)
    logp, _, _ = O.token_logprobs(z, ids, mask)
    old = logp + torch.randn(N, generator=g, dtype=F64) * 0.05
    return z, ids, mask, cu, adv, old, g


def test_sequence_ratio_is_the_product_of_token_ratios():
    z, ids, mask, cu, adv, old, _ = _toy()
    lp = O.LossParams(ratio_level=O.RATIO_SEQUENCE)
    seq = O.policy_loss_sequence_ratio(z, ids, mask, cu, adv, old, None, lp, want_dlogits=False)
    tok = O.policy_loss(z, ids, mask, cu, adv, old, None, None, O.LossParams(), want_dlogits=False)
    for s in range(5):
        a, b = int(cu[s]), int(cu[s + 1])
        v = tok["valid"][a:b]
        assert abs(float(seq["w"][s]) - float(torch.prod(tok["rho"][a:b][v]))) <= 1e-12 * float(seq["w"][s])


def test_single_token_responses_reduce_to_the_token_level_pass():
    # one token per response: response-level and token-level ratios coincide, and so does Eq. (1)'s aggregation
    z, ids, _, _, _, _, g = _toy(N=12, S=12)
    cu = torch.arange(13)
    adv = torch.randn(12, generator=g, dtype=F64)
    logp, _, _ = O.token_logprobs(z, ids)
    old = logp + torch.randn(12, generator=g, dtype=F64) * 0.3         # wide enough to clip some
    seq = O.policy_loss_sequence_ratio(z, ids, None, cu, adv, old, None, O.LossParams(ratio_level=O.RATIO_SEQUENCE))
    tok = O.policy_loss(z, ids, None, cu, adv, old, None, None, O.LossParams(agg_mode=O.AGG_SEQ_MEAN_TOKEN_MEAN))
    assert abs(seq["loss_pg"] - tok["loss_pg"]) <= 1e-14
    assert (seq["dlogits"] - tok["dlogits"]).abs().max() <= 1e-15
    assert seq["seq_clipped"].any() and not seq["seq_clipped"].all()


def test_ratio_one_gives_minus_mean_advantage_over_responses():
    z, ids, mask, cu, adv, _, _ = _toy()
    out = O.policy_loss_sequence_ratio(z, ids, mask, cu, adv, None, None, O.LossParams(ratio_level=O.RATIO_SEQUENCE),
                                       want_dlogits=False)
    assert abs(out["loss_pg"] + float(adv.mean())) <= 1e-14 and (out["w"] == 1).all()


def test_clip_cases_by_hand():
    # two tokens, uniform logits over V = 4: logp = -log 4 each.  L_old chosen so that w = 1.5 resp. 0.5.
    z = torch.zeros(2, 4, dtype=F64)
    ids = torch.tensor([1, 2])
    cu = torch.tensor([0, 2])
    lp = O.LossParams(ratio_level=O.RATIO_SEQUENCE)
    L = -2 * math.log(4.0)
    for w, A, want_s, clipped in ((1.5, 2.0, 1.2 * 2.0, True), (1.5, -2.0, 1.5 * -2.0, False),
                                  (0.5, 2.0, 0.5 * 2.0, False), (0.5, -2.0, 0.8 * -2.0, True)):
        old = torch.full((2,), (L - math.log(w)) / 2, dtype=F64)
        out = O.policy_loss_sequence_ratio(z, ids, None, cu, torch.tensor([A]), old, None, lp)
        assert abs(out["loss_pg"] + want_s) <= 1e-12
        assert bool(out["seq_clipped"][0]) == clipped
        if clipped:
            assert out["dlogits"].abs().max() == 0
        else:   # every token of the response carries the same multiplier A w
            assert abs(float(out["g"][0]) - A * w) <= 1e-12 and abs(float(out["g"][1]) - A * w) <= 1e-12


@pytest.mark.parametrize("V", [3, 64])
def test_finite_differences_agree_with_dlogits(V):
    z, ids, mask, cu, adv, old, g = _toy(N=14, V=V, S=4, seed=5)
    nllw = (torch.rand(14, generator=g) < 0.4).to(F64)
    lp = O.LossParams(ratio_level=O.RATIO_SEQUENCE, nll_coeff=0.3)
    out = O.policy_loss_sequence_ratio(z, ids, mask, cu, adv, old, nllw, lp)
    assert (out["seq_margin"] > 1e-3).all()
    def L(zz):
        o = O.policy_loss_sequence_ratio(zz, ids, mask, cu, adv, old, nllw, lp, want_dlogits=False)
        return o["loss_pg"] + o["loss_nll"]
    h = 1e-6
    gen = torch.Generator().manual_seed(1)
    for _ in range(40):
        t, v = int(torch.randint(0, 14, (1,), generator=gen)), int(torch.randint(0, V, (1,), generator=gen))
        zp, zm = z.clone(), z.clone()
        zp[t, v] += h
        zm[t, v] -= h
        fd = (L(zp) - L(zm)) / (2 * h)
        assert abs(fd - float(out["dlogits"][t, v])) <= 1e-7 * max(1.0, abs(fd))
    assert (out["dlogits"].sum(dim=1).abs() <= 1e-13).all()


def test_responses_without_valid_tokens_and_zero_advantage_contribute_nothing():
    z, ids, mask, cu, adv, old, _ = _toy()
    mask = mask.clone()
    mask[int(cu[1]):int(cu[2])] = 0
    adv = adv.clone()
    adv[3] = 0.0
    out = O.policy_loss_sequence_ratio(z, ids, mask, cu, adv, old, None, O.LossParams(ratio_level=O.RATIO_SEQUENCE))
    assert float(out["seq_term"][1]) == 0 and float(out["seq_term"][3]) == 0
    assert out["dlogits"][int(cu[1]):int(cu[2])].abs().max() == 0 and out["dlogits"][int(cu[3]):int(cu[4])].abs().max() == 0
