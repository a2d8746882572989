"""Pins for the CPU oracle: closed forms, brute force, finite differences, the paper's printed example.

None of these re-types the oracle's own formula with the same routine: each compares it with
something the paper or the mathematics fixes independently.
"""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch
from scipy.special import logsumexp as scipy_lse

from oracle import mrl_oracle as O

F64 = torch.float64
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- log-probs (Sec. 3)

@pytest.mark.parametrize("V", [1, 2, 7, 1024, 151936])
def test_uniform_logits_give_minus_log_V(V):
    z = torch.full((3, V), 0.37, dtype=torch.float32)
    ids = torch.tensor([0, V // 2, V - 1])
    logp, lse, valid = O.token_logprobs(z, ids)
    assert valid.all()
    assert torch.allclose(logp, torch.full((3,), -math.log(V), dtype=F64), atol=1e-12, rtol=0)


def test_logprob_brute_force_python_loops():
    g = torch.Generator().manual_seed(1)
    z = torch.randn(5, 8, generator=g, dtype=F64) * 3
    ids = torch.randint(0, 8, (5,), generator=g)
    logp, lse, _ = O.token_logprobs(z, ids)
    for t in range(5):
        tot = math.fsum(math.exp(float(z[t, v])) for v in range(8))
        assert abs(float(logp[t]) - (float(z[t, ids[t]]) - math.log(tot))) < 1e-12
        assert abs(float(lse[t]) - math.log(tot)) < 1e-12


def test_logprob_matches_scipy_logsumexp_and_shift_invariance():
    g = torch.Generator().manual_seed(2)
    z = (torch.randn(16, 333, generator=g) * 4).bfloat16()
    ids = torch.randint(0, 333, (16,), generator=g)
    logp, lse, _ = O.token_logprobs(z, ids)
    ref = scipy_lse(z.double().numpy(), axis=1)
    assert np.allclose(lse.numpy(), ref, atol=1e-12, rtol=0)
    logp2, _, _ = O.token_logprobs(z.double() + 100.0, ids)
    assert torch.allclose(logp, logp2, atol=1e-10, rtol=0)
    # probabilities over all targets sum to one
    allp = torch.stack([O.token_logprobs(z, torch.full((16,), v))[0] for v in range(333)], 1)
    assert torch.allclose(torch.exp(allp).sum(1), torch.ones(16, dtype=F64), atol=1e-12)


def test_dominant_logit_and_large_magnitudes_are_stable():
    z = torch.zeros(2, 50, dtype=F64)
    z[0, 3] = 800.0      # exp overflows without the max shift
    z[1, 7] = -800.0
    logp, lse, _ = O.token_logprobs(z, torch.tensor([3, 7]))
    assert abs(float(logp[0])) < 1e-12 and abs(float(lse[0]) - 800.0) < 1e-12
    assert abs(float(logp[1]) - (-800.0 - math.log(49.0))) < 1e-9


def test_masked_and_bad_ids_rows_are_zero_and_invalid():
    z = torch.randn(4, 10)
    logp, _, valid = O.token_logprobs(z, torch.tensor([1, -1, 10, 2]), torch.tensor([1, 1, 1, 0]))
    assert valid.tolist() == [True, False, False, False]
    assert logp[1:].abs().max() == 0 and logp[0] < 0


# ---------------------------------------------------------------- advantages (Sec. 3, Sec. 5.1, App. H)

def test_advantages_zero_mean_and_equal_rewards_zero():
    g = torch.Generator().manual_seed(3)
    r = torch.rand(6, 3, 5, generator=g)
    r[2] = 0.25          # a prompt whose rewards are all equal
    r[4, 1] = 1.0        # a group whose rewards are all equal
    for mode in (O.ADV_MEAN_ONLY, O.ADV_GROUP_ZNORM, O.ADV_BATCH_ZNORM):
        own, pool = O.group_advantages(r, mode)
        assert own.sum(dim=2).abs().max() < 1e-9
        assert pool.sum(dim=(1, 2)).abs().max() < 1e-9
        assert own[2].abs().max() == 0 and pool[2].abs().max() == 0
        assert own[4, 1].abs().max() == 0


@pytest.mark.parametrize("K,k", [(5, 1), (8, 3), (16, 15), (4, 2)])
def test_binary_reward_closed_form(K, k):
    # k successes of K with population std sqrt(q(1-q)), q = k/K
    r = torch.zeros(1, 1, K)
    r[0, 0, :k] = 1
    eps = 1e-6
    own, pool = O.group_advantages(r, O.ADV_GROUP_ZNORM, ddof=0, eps=eps)
    q = k / K
    sd = math.sqrt(q * (1 - q))
    assert torch.allclose(own[0, 0, :k], torch.full((k,), (1 - q) / (sd + eps), dtype=F64), atol=1e-12)
    assert torch.allclose(own[0, 0, k:], torch.full((K - k,), -q / (sd + eps), dtype=F64), atol=1e-12)
    assert torch.allclose(own, pool, atol=1e-12)           # M = 1: the pool is the group
    own1, _ = O.group_advantages(r, O.ADV_GROUP_ZNORM, ddof=1, eps=eps)
    assert torch.allclose(own1, own * (sd + eps) / (sd * math.sqrt(K / (K - 1)) + eps), atol=1e-12)


def test_advantages_against_numpy_std_and_pool_permutation_invariance():
    g = torch.Generator().manual_seed(4)
    r = torch.rand(5, 2, 4, generator=g)
    own, pool = O.group_advantages(r, O.ADV_GROUP_ZNORM, ddof=0, eps=1e-6)
    rn = r.double().numpy()
    for p in range(5):
        flat = rn[p].reshape(-1)
        assert np.allclose(pool[p].numpy().reshape(-1), (flat - flat.mean()) / (np.std(flat) + 1e-6))
        for m in range(2):
            assert np.allclose(own[p, m].numpy(), (rn[p, m] - rn[p, m].mean()) / (np.std(rn[p, m]) + 1e-6))
    # the pooled baseline depends only on the multiset of pooled rewards (App. H, XGRPO lemma):
    # permuting the peer's rewards leaves the learner's pooled advantages unchanged
    r2 = r.clone()
    r2[:, 1, :] = r[:, 1, torch.tensor([2, 0, 3, 1])]
    _, pool2 = O.group_advantages(r2, O.ADV_GROUP_ZNORM)
    assert torch.allclose(pool[:, 0], pool2[:, 0], atol=1e-12)


def test_batch_whitening_unit_variance():
    g = torch.Generator().manual_seed(5)
    r = (torch.rand(64, 2, 5, generator=g) < 0.4).float()
    own, pool = O.group_advantages(r, O.ADV_BATCH_ZNORM, ddof=0, eps=0.0)
    for m in range(2):
        assert abs(float((own[:, m] ** 2).mean()) - 1.0) < 1e-9     # zero mean, unit variance over the batch
        assert abs(float(own[:, m].mean())) < 1e-12
    assert abs(float((pool ** 2).mean()) - 1.0) < 1e-9


# ---------------------------------------------------------------- SGT gate (Sec. 5.3, App. B, Def. 7)

def _gate_by_sets(bits, M, G, learner):
    succ = {(m, g) for m in range(M) for g in range(G) if bits[m * G + g]}
    own = {x for x in succ if x[0] == learner}
    peer = succ - own
    return (len(own) == 0) and (len(peer) > 0), sorted(m * G + g for m, g in peer)


@pytest.mark.parametrize("G", [1, 2, 3, 4])
def test_gate_brute_force_all_binary_patterns(G):
    M = 2
    pats = list(itertools.product([0, 1], repeat=M * G))
    r = torch.tensor(pats, dtype=torch.float32).reshape(len(pats), M, G)
    lens = torch.arange(len(pats) * M * G, dtype=torch.int32).reshape(len(pats), M, G) % 5
    for learner in range(M):
        rescue, pick, w, n = O.sgt_gate(r, lens, learner, pick=O.PICK_FIRST)
        for i, bits in enumerate(pats):
            fire, peers = _gate_by_sets(bits, M, G, learner)
            assert bool(rescue[i]) == fire
            assert int(pick[i]) == (peers[0] if fire else -1)
            assert float(w[i].sum()) == (1.0 if fire else 0.0)
        assert n == int(rescue.sum())
        rescue_a, _, w_a, n_a = O.sgt_gate(r, lens, learner, pick=O.PICK_ALL)
        assert torch.equal(rescue_a, rescue)
        for i, bits in enumerate(pats):
            fire, peers = _gate_by_sets(bits, M, G, learner)
            got = sorted(int(x) for x in w_a[i].reshape(-1).nonzero()[:, 0])
            assert got == (peers if fire else [])
        assert n_a == int(w_a.sum())


def test_gate_shortest_pick_and_ties_and_thresholds():
    r = torch.tensor([[[0.0, 0.1], [1.0, 0.9]],      # fires; both peers succeed
                      [[0.0, 0.2], [1.0, 1.0]],      # 0.2 is not < 0.2: no fire
                      [[0.0, 0.0], [0.8, 0.5]],      # 0.8 is not > 0.8: no fire
                      [[0.0, 0.0], [0.0, 0.81]]])    # fires
    lens = torch.tensor([[[5, 5], [9, 4]], [[1, 1], [1, 1]], [[1, 1], [1, 1]], [[3, 3], [7, 7]]],
                        dtype=torch.int32)
    rescue, pick, w, n = O.sgt_gate(r, lens, 0, pick=O.PICK_SHORTEST)
    assert rescue.tolist() == [1, 0, 0, 1] and pick.tolist() == [3, -1, -1, 3] and n == 2
    lens[0, 1, 0] = 4                                   # tie: lowest flat index wins
    _, pick, _, _ = O.sgt_gate(r, lens, 0, pick=O.PICK_SHORTEST)
    assert pick.tolist() == [2, -1, -1, 3]
    _, pick_s, w_s, _ = O.sgt_gate(r, lens, 0, pick=O.PICK_SEEDED, seed=11)
    assert int(pick_s[0]) in (2, 3) and int(pick_s[3]) == 3 and float(w_s.sum()) == 2.0


def test_splitmix64_published_first_outputs():
    # first outputs of the reference SplitMix64 stream started at state 0 (Steele, Lea, Flood 2014;
    # the same vector is used by the xoshiro authors to seed their generators)
    assert O.splitmix64(0) == 0xE220A8397B1DCDAF
    assert O.splitmix64(0x9E3779B97F4A7C15) == 0x6E789E6AA1B965F4


def test_gate_rate_matches_closed_form_and_cost_bound():
    # Def. 7: G_n = (1-p_n)^K [1 - prod_{m != n} (1-p_m)^K], independent Bernoulli rollouts
    g = torch.Generator().manual_seed(6)
    P, M, K = 100000, 3, 4
    p = torch.tensor([0.15, 0.3, 0.1])
    r = (torch.rand(P, M, K, generator=g) < p[None, :, None]).float()
    lens = torch.ones(P, M, K, dtype=torch.int32)
    # vectorised restatement of the gate for speed is NOT used: the oracle's loop runs on a subsample
    sub = 20000
    rescue, pick, w, n = O.sgt_gate(r[:sub], lens[:sub], 0)
    Gn = (1 - 0.15) ** K * (1 - ((1 - 0.3) ** K) * ((1 - 0.1) ** K))
    se = math.sqrt(Gn * (1 - Gn) / sub)
    assert abs(float(rescue.float().mean()) - Gn) < 4 * se
    # App. G: extra sequences <= (M-1)/(M K) of the rollout batch, summed over the learners
    total = 0
    for n_ in range(M):
        total += O.sgt_gate(r[:2000], lens[:2000], n_)[3]
    assert total <= (M - 1) / (M * K) * (2000 * M * K)


# ---------------------------------------------------------------- surrogate and loss (Eq. (1), Eq. (2))

def _toy(N=24, V=13, S=4, seed=7, dtype=F64):
    g = torch.Generator().manual_seed(seed)
    z = (torch.randn(N, V, generator=g) * 2).to(dtype)
    ids = torch.randint(0, V, (N,), generator=g)
    cuts = sorted(torch.randperm(N - 1, generator=g)[:S - 1].add(1).tolist())
    cu = torch.tensor([0] + cuts + [N], dtype=torch.int32)
    adv = torch.randn(S, generator=g, dtype=F64)
    mask = (torch.rand(N, generator=g) < 0.8).to(torch.uint8)
    return z, ids, mask, cu, adv, g


def test_ratio_one_gives_minus_masked_mean_of_A():
    z, ids, mask, cu, adv, g = _toy()
    out = O.policy_loss(z, ids, mask, cu, adv, None)
    A_rows = torch.repeat_interleave(adv, (cu[1:] - cu[:-1]).long())
    m = mask.double()
    assert abs(out["loss_pg"] - float(-(m * A_rows).sum() / m.sum())) < 1e-12
    assert out["loss_nll"] == 0.0
    # Eq. (1) aggregation: mean over sequences of the per-sequence token mean
    out2 = O.policy_loss(z, ids, mask, cu, adv, None, lp=O.LossParams(agg_mode=O.AGG_SEQ_MEAN_TOKEN_MEAN))
    per_seq = [float(adv[s]) if mask[cu[s]:cu[s + 1]].sum() > 0 else 0.0 for s in range(len(adv))]
    assert abs(out2["loss_pg"] - (-sum(per_seq) / len(adv))) < 1e-12


def test_clip_cases_by_hand():
    # one row per case; V = 2 with known probabilities
    z = torch.log(torch.tensor([[0.5, 0.5]] * 6, dtype=F64))
    ids = torch.zeros(6, dtype=torch.long)
    cu = torch.arange(7, dtype=torch.int32)
    adv = torch.tensor([1.0, 1.0, 1.0, -1.0, -1.0, -1.0], dtype=F64)
    rho = torch.tensor([1.5, 0.5, 1.1, 1.5, 0.5, 0.9], dtype=F64)
    logp_old = math.log(0.5) - torch.log(rho)
    out = O.policy_loss(z, ids, None, cu, adv, logp_old, lp=O.LossParams(pg_denominator=1.0))
    s = -out["pg_term"]
    assert torch.allclose(s, torch.tensor([1.2, 0.5, 1.1, -1.5, -0.8, -0.9], dtype=F64), atol=1e-12)
    assert out["clipped"].tolist() == [True, False, False, False, True, False]
    # gradient w.r.t. logp is rho*A where unclipped, else 0
    assert torch.allclose(out["g"], torch.tensor([0, 0.5, 1.1, -1.5, 0, -0.9], dtype=F64), atol=1e-12)
    # |clip(rho)| <= 1 + eps (App. H, PRP bias/variance theorem): clipped surrogate magnitude bound
    assert (s.abs() <= torch.maximum(rho, torch.tensor(1.2, dtype=F64)) + 1e-12).all()
    assert out["stats"] == (6, 2)


def test_clip_boundary_equality_counts_as_unclipped():
    z = torch.zeros(2, 4, dtype=F64)
    ids = torch.zeros(2, dtype=torch.long)
    cu = torch.tensor([0, 1, 2], dtype=torch.int32)
    lp = O.LossParams(eps_lo=0.25, eps_hi=0.25, pg_denominator=1.0)   # 1.25 and 0.75 are exact in binary
    logp = math.log(0.25)
    logp_old = torch.tensor([logp - math.log(1.25), logp - math.log(0.75)], dtype=F64)
    out = O.policy_loss(z, ids, None, cu, torch.tensor([1.0, -1.0], dtype=F64), logp_old, lp=lp)
    # exp(log(1.25)) may round either side of 1.25; the rule under test is the comparison itself
    rho = out["rho"]
    exp_clip = [bool(rho[0] > 1.25), bool(rho[1] < 0.75)]
    assert out["clipped"].tolist() == exp_clip
    sur = O.surrogate(torch.tensor([0.0, 0.0], dtype=F64), torch.tensor([0.0, 0.0], dtype=F64),
                      torch.tensor([1.0, -1.0], dtype=F64), torch.ones(2, dtype=F64),
                      torch.zeros(2, dtype=F64), O.LossParams(eps_lo=0.0, eps_hi=0.0))
    assert sur["clipped"].tolist() == [False, False]          # rho == bound exactly: unclipped


def test_infinite_eps_is_importance_weighted_reinforce():
    z, ids, mask, cu, adv, g = _toy(seed=8)
    logp, _, valid = O.token_logprobs(z, ids, mask)
    logp_old = logp + torch.randn(len(logp), generator=g, dtype=F64) * 0.3
    out = O.policy_loss(z, ids, mask, cu, adv, logp_old, lp=O.LossParams(eps_lo=1.0, eps_hi=1e30))
    A_rows = torch.repeat_interleave(adv, (cu[1:] - cu[:-1]).long())
    m = valid.double()
    ref = -(m * torch.exp(logp - logp_old) * A_rows).sum() / m.sum()
    assert abs(out["loss_pg"] - float(ref)) < 1e-12
    assert not out["clipped"][valid & (A_rows > 0)].any()


def test_nll_only_is_token_mean_cross_entropy():
    z, ids, mask, cu, adv, g = _toy(seed=9)
    nllw = torch.ones(len(ids), dtype=torch.float32)
    lam, n_gated = 0.1, len(adv)
    out = O.policy_loss(z, ids, mask, cu, torch.zeros_like(adv), None, None, nllw,
                        lp=O.LossParams(nll_coeff=lam / n_gated))
    assert out["loss_pg"] == 0.0
    ce = torch.nn.functional.cross_entropy(z, ids, reduction="none")
    tot = 0.0
    for s in range(len(adv)):
        a, b = int(cu[s]), int(cu[s + 1])
        m = mask[a:b].double()
        if m.sum() > 0:
            tot += float((ce[a:b] * m).sum() / m.sum())
    assert abs(out["loss_nll"] - lam * tot / n_gated) < 1e-12


def test_stop_grad_token_weight_scales_terms():
    z, ids, mask, cu, adv, g = _toy(seed=10)
    logp, _, _ = O.token_logprobs(z, ids, mask)
    logp_old = logp + torch.randn(len(logp), generator=g, dtype=F64) * 0.2
    u = torch.rand(len(ids), generator=g, dtype=F64) + 0.5
    a = O.policy_loss(z, ids, mask, cu, adv, logp_old)
    b = O.policy_loss(z, ids, mask, cu, adv, logp_old, tok_weight=u)
    assert torch.allclose(b["pg_term"], a["pg_term"] * u, atol=1e-14)
    assert torch.allclose(b["dlogits"], a["dlogits"] * u[:, None], atol=1e-14)


# ---------------------------------------------------------------- backward

def test_dlogits_rows_sum_to_zero_and_masked_rows_are_zero():
    z, ids, mask, cu, adv, g = _toy(seed=11)
    logp, _, _ = O.token_logprobs(z, ids, mask)
    logp_old = logp + torch.randn(len(logp), generator=g, dtype=F64) * 0.2
    out = O.policy_loss(z, ids, mask, cu, adv, logp_old, nll_weight=torch.ones(len(ids)),
                        lp=O.LossParams(nll_coeff=0.05))
    assert out["dlogits"].sum(dim=1).abs().max() < 1e-14
    assert out["dlogits"][mask == 0].abs().max() == 0


@pytest.mark.parametrize("agg", [O.AGG_TOKEN_MEAN, O.AGG_SEQ_MEAN_TOKEN_MEAN])
@pytest.mark.parametrize("V", [3, 64])
def test_finite_differences_agree_with_dlogits(agg, V):
    z, ids, mask, cu, adv, g = _toy(N=12, V=V, S=3, seed=12 + V)
    logp, _, _ = O.token_logprobs(z, ids, mask)
    logp_old = logp + torch.randn(len(logp), generator=g, dtype=F64) * 0.25
    u = torch.rand(len(ids), generator=g, dtype=F64) + 0.5
    nllw = (torch.rand(len(ids), generator=g) < 0.5).float()
    lp = O.LossParams(agg_mode=agg, nll_coeff=0.07)
    out = O.policy_loss(z, ids, mask, cu, adv, logp_old, u, nllw, lp)
    assert out["margin"][out["valid"]].min() > 1e-4         # no ratio sits on the clip kink
    assert out["clipped"].any() and (~out["clipped"]).any()

    def L(zz):
        o = O.policy_loss(zz, ids, mask, cu, adv, logp_old, u, nllw, lp, want_dlogits=False)
        return o["loss_pg"] + o["loss_nll"]

    h = 1e-6
    fd = torch.zeros_like(z)
    for t in range(z.shape[0]):
        for v in range(V):
            zp, zm = z.clone(), z.clone()
            zp[t, v] += h
            zm[t, v] -= h
            fd[t, v] = (L(zp) - L(zm)) / (2 * h)
    assert (fd - out["dlogits"]).abs().max() < 1e-8


def _read_prop1():
    rows = []
    with open(os.path.join(GOLDEN, "prop1_anti_align.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            parts = [p.strip() for p in line.split("|")]
            fr = lambda s: [Fraction(x) for x in s.split()]
            rows.append((Fraction(parts[0]), fr(parts[1]), fr(parts[2]), Fraction(parts[3]), Fraction(parts[4])))
    return rows


@pytest.mark.parametrize("row", _read_prop1())
def test_prop1_three_action_bandit_printed_gradients(row):
    eta, g_on, g_naive, inner, chi2 = row
    e = float(eta)
    pi = torch.tensor([1 / 3, 2 / 3 - e, e], dtype=F64)
    mu = torch.tensor([e, e, 1 - 2 * e], dtype=F64)
    A = torch.tensor([2 / 3, -1 / 3, -1 / 3], dtype=F64)
    z = torch.log(pi).repeat(3, 1)                # one row per action, logits = log pi
    ids = torch.arange(3)
    cu = torch.arange(4, dtype=torch.int32)
    lp = O.LossParams(pg_denominator=1.0, eps_lo=0.2, eps_hi=0.2)

    def grad(weights):                            # E_{a ~ weights}[A(a) grad log pi(a)] = -dL/dz
        out = O.policy_loss(z, ids, None, cu, A, None, tok_weight=weights, lp=lp)
        return -out["dlogits"].sum(dim=0)

    got_on, got_naive = grad(pi), grad(mu)
    assert torch.allclose(got_on, torch.tensor([float(x) for x in g_on], dtype=F64), atol=1e-14)
    assert torch.allclose(got_naive, torch.tensor([float(x) for x in g_naive], dtype=F64), atol=1e-14)
    ip = float((got_on * got_naive).sum())
    assert abs(ip - float(inner)) < 1e-14 and ip < 0
    assert abs(ip - (2 / 3 * e ** 3 - e ** 2 + 5 / 9 * e - 2 / 81)) < 1e-14
    assert abs(float(((pi ** 2) / mu).sum() - 1) - float(chi2)) < 1e-9


# ---------------------------------------------------------------- hidden-in path

def test_lmhead_gradients_by_finite_differences_and_column_sum():
    g = torch.Generator().manual_seed(21)
    N, H, V, S = 10, 5, 9, 2
    hdn = torch.randn(N, H, generator=g, dtype=F64)
    W = torch.randn(V, H, generator=g, dtype=F64) * 0.5
    ids = torch.randint(0, V, (N,), generator=g)
    cu = torch.tensor([0, 4, 10], dtype=torch.int32)
    adv = torch.tensor([0.7, -1.1], dtype=F64)
    mask = torch.ones(N, dtype=torch.uint8)
    mask[3] = 0
    logp, _, _ = O.token_logprobs(hdn @ W.T, ids, mask)
    logp_old = logp + torch.randn(N, generator=g, dtype=F64) * 0.2
    out = O.fused_lmhead_loss(hdn, W, ids, mask, cu, adv, logp_old)
    assert out["margin"][out["valid"]].min() > 1e-4
    assert out["dW"].sum(dim=0).abs().max() < 1e-13       # rows of dZ sum to zero

    def L(hh, ww):
        o = O.policy_loss(hh @ ww.T, ids, mask, cu, adv, logp_old, want_dlogits=False)
        return o["loss_pg"] + o["loss_nll"]

    h = 1e-6
    for (t, k) in [(0, 0), (3, 2), (9, 4), (5, 1)]:
        hp, hm = hdn.clone(), hdn.clone()
        hp[t, k] += h
        hm[t, k] -= h
        assert abs((L(hp, W) - L(hm, W)) / (2 * h) - float(out["dHidden"][t, k])) < 1e-8
    for (v, k) in [(0, 0), (8, 4), (int(ids[0]), 2), (4, 3)]:
        wp, wm = W.clone(), W.clone()
        wp[v, k] += h
        wm[v, k] -= h
        assert abs((L(hdn, wp) - L(hdn, wm)) / (2 * h) - float(out["dW"][v, k])) < 1e-8


def test_lmhead_degenerate_H1_N1():
    hdn = torch.tensor([[2.0]], dtype=F64)
    W = torch.tensor([[0.5], [-0.5], [0.0]], dtype=F64)
    out = O.fused_lmhead_loss(hdn, W, torch.tensor([1]), None, torch.tensor([0, 1], dtype=torch.int32),
                              torch.tensor([1.0], dtype=F64), None)
    p = torch.softmax(torch.tensor([1.0, -1.0, 0.0], dtype=F64), 0)
    dz = p - torch.tensor([0.0, 1.0, 0.0], dtype=F64)
    assert torch.allclose(out["dW"][:, 0], dz * 2.0, atol=1e-14)
    assert abs(float(out["dHidden"][0, 0]) - float((dz * W[:, 0]).sum())) < 1e-14
