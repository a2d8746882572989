"""GPU parity of the logits-in path (mrl_token_logprobs, mrl_policy_loss_fwd_bwd) and of
mrl_group_advantages against the CPU float64 oracle, element by element on the same seeded inputs."""
import math

import pytest
import torch

from oracle import mrl_oracle as O
from paper_2605_07244_b200 import binding as B
from paper_2605_07244_b200 import build, synth

from helpers import (LOGP_ATOL, TIE_MARGIN, compare_policy_loss, dev, loss_close, make_lp, oracle_lp, rel_l2,
                     run_gpu_policy_loss)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    B.lib()


def toy_inputs(N, V, S, dtype, seed, std=2.0, mask_p=None, noise=0.1, pad=0):
    g = torch.Generator().manual_seed(seed)
    z = (torch.randn(N, V + pad, generator=g) * std).to(dtype)
    ids = torch.randint(0, V, (N,), generator=g, dtype=torch.int32)
    if N > 1 and V > 1:
        ids[0], ids[-1] = 0, V - 1
    if S > 1:
        cuts = sorted(torch.randperm(N - 1, generator=g)[:S - 1].add(1).tolist())
    else:
        cuts = []
    cu = torch.tensor([0] + cuts + [N], dtype=torch.int32)
    adv = torch.randn(S, generator=g)
    mask = None if mask_p is None else (torch.rand(N, generator=g) < mask_p).to(torch.uint8)
    logp, _, _ = O.token_logprobs(z[:, :V], ids, mask)
    logp_old = (logp + torch.randn(N, generator=g, dtype=torch.float64) * noise).float()
    return z, ids, mask, cu, adv, logp_old, g


# ------------------------------------------------------------------ advantages and gate

@pytest.mark.parametrize("mode", [B.ADV_MEAN_ONLY, B.ADV_GROUP_ZNORM, B.ADV_BATCH_ZNORM])
@pytest.mark.parametrize("P,M,G,ddof", [(4, 1, 4, 0), (8, 1, 8, 1), (16, 2, 8, 0), (64, 2, 16, 0), (5, 3, 33, 1),
                                        (3, 1, 1, 0)])
def test_group_advantages_match_oracle(mode, P, M, G, ddof):
    g = torch.Generator().manual_seed(100 + P + G)
    r = (torch.rand(P, M, G, generator=g) < 0.4).float()
    if P > 2:
        r[1] = 1.0           # all-equal prompt
        r[2, 0] = 0.0        # learner fails everything on prompt 2
    own = torch.full((P, M, G), float("nan"), device="cuda")
    pool = torch.full((P, M, G), float("nan"), device="cuda")
    ap = B.AdvParams(mode, ddof, 1e-6, 0.8, 0.2, B.PICK_NONE, 0)
    B.mrl_group_advantages(dev(r), None, 0, ap, own, pool)
    torch.cuda.synchronize()
    ref_own, ref_pool = O.group_advantages(r, mode, ddof, 1e-6)
    scale = max(1.0, float(ref_own.abs().max()))
    assert (own.cpu().double() - ref_own).abs().max() <= 2e-6 * scale
    assert (pool.cpu().double() - ref_pool).abs().max() <= 2e-6 * max(1.0, float(ref_pool.abs().max()))
    if P > 2:
        assert own.cpu()[1].abs().max() == 0 and pool.cpu()[1].abs().max() == 0


@pytest.mark.parametrize("pick", [B.PICK_NONE, B.PICK_FIRST, B.PICK_SHORTEST, B.PICK_ALL, B.PICK_SEEDED])
@pytest.mark.parametrize("P,M,G,learner", [(64, 2, 16, 0), (200, 3, 4, 1), (33, 2, 1, 1), (10, 1, 4, 0)])
def test_sgt_gate_is_bit_exact(pick, P, M, G, learner):
    g = torch.Generator().manual_seed(7 * P + pick)
    p = torch.sin(torch.rand(P, M, generator=g) * math.pi / 2) ** 2 * 0.5
    r = (torch.rand(P, M, G, generator=g) < p[:, :, None]).float()
    r[0] = torch.tensor(0.5)                       # neither negative nor success
    lens = torch.randint(1, 6, (P, M, G), generator=g, dtype=torch.int32)   # many ties
    rescue = torch.full((P,), 9, dtype=torch.uint8, device="cuda")
    pk = torch.full((P,), -7, dtype=torch.int32, device="cuda")
    w = torch.full((P, M, G), float("nan"), device="cuda")
    n = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    ap = B.AdvParams(B.ADV_GROUP_ZNORM, 0, 1e-6, 0.8, 0.2, pick, 1234)
    B.mrl_group_advantages(dev(r), dev(lens), learner, ap, None, None, rescue, pk, w, n)
    torch.cuda.synchronize()
    ref = O.sgt_gate(r, lens, learner, 0.8, 0.2, pick, 1234)
    assert torch.equal(rescue.cpu(), ref[0])
    assert torch.equal(pk.cpu(), ref[1])
    assert torch.equal(w.cpu().double(), ref[2])
    assert int(n.cpu()) == ref[3]
    if M > 1 and pick != B.PICK_NONE:
        assert ref[3] > 0                          # the case exercises the gate


# ------------------------------------------------------------------ log-probs

@pytest.mark.parametrize("N,V,dtype,pad", [
    (1024, 1024, torch.float32, 0),      # config 1 shape
    (7, 1, torch.float32, 0), (5, 3, torch.bfloat16, 0), (9, 1000, torch.bfloat16, 3),   # general kernel
    (37, 4096, torch.bfloat16, 0), (19, 4104, torch.bfloat16, 8),                         # 256-bit path, one step; 128-bit path with a padded row
    (11, 40008, torch.bfloat16, 0),                                                       # 128-bit path, ragged last step
    (9, 100008, torch.bfloat16, 0), (6, 151936, torch.bfloat16, 0), (5, 128256, torch.bfloat16, 0),
    (13, 8208, torch.bfloat16, 0), (4, 65552, torch.bfloat16, 16),                        # 256-bit path, ragged last step
    (3, 262160, torch.bfloat16, 0), (2, 300008, torch.bfloat16, 0),                       # rows split over a cluster of two CTAs
    (3, 200008, torch.bfloat16, 0),                                                       # long row, 128-bit path
])
def test_token_logprobs(N, V, dtype, pad):
    z, ids, _, _, _, _, g = toy_inputs(N, V, 1, dtype, seed=N + V, pad=pad)
    mask = (torch.rand(N, generator=g) < 0.8).to(torch.uint8)
    if N > 4:
        ids[3] = V          # bad id on a row that is not masked
        mask[3] = 1
    zl = dev(z)
    logp = torch.full((N,), float("nan"), device="cuda")
    lse = torch.full((N,), float("nan"), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.mrl_token_logprobs(zl, dev(ids), dev(mask), logp, lse, status, V=V)
    torch.cuda.synchronize()
    ref_logp, ref_lse, valid = O.token_logprobs(z[:, :V], ids, mask)
    assert (logp.cpu().double() - ref_logp).abs().max() <= LOGP_ATOL
    assert (lse.cpu().double() - torch.where(valid, ref_lse, torch.zeros_like(ref_lse))).abs().max() <= LOGP_ATOL
    assert (logp.cpu()[~valid] == 0).all()
    # run-to-run bitwise determinism
    logp2 = torch.empty_like(logp)
    B.mrl_token_logprobs(zl, dev(ids), dev(mask), logp2, None, None, V=V)
    torch.cuda.synchronize()
    assert torch.equal(logp, logp2)


def test_uniform_logits_on_gpu_give_minus_log_V():
    for V in (8, 4096, 151936):
        z = torch.full((4, V), 1.5, dtype=torch.bfloat16, device="cuda")
        ids = torch.tensor([0, 1, V // 2, V - 1], dtype=torch.int32, device="cuda")
        logp = torch.empty(4, device="cuda")
        B.mrl_token_logprobs(z, ids, None, logp)
        torch.cuda.synchronize()
        assert (logp.cpu().double() + math.log(V)).abs().max() <= 1e-5


# ------------------------------------------------------------------ loss forward + backward

CASES = [
    # N, V, S, dtype, pad, mask_p
    (1024, 1024, 16, torch.float32, 0, None),
    (6, 1, 2, torch.float32, 0, None),
    (8, 3, 3, torch.bfloat16, 0, 0.7),
    (33, 1000, 5, torch.bfloat16, 5, 0.8),
    (33, 999, 5, torch.float32, 0, 0.8),
    (41, 4096, 6, torch.bfloat16, 0, None),
    (23, 4104, 4, torch.bfloat16, 16, 0.8),
    (13, 40008, 3, torch.bfloat16, 0, 0.9),
    (9, 100008, 2, torch.bfloat16, 8, None),
    (12, 151936, 3, torch.bfloat16, 0, 0.9),
    (7, 128256, 2, torch.bfloat16, 0, None),
    (3, 200008, 1, torch.bfloat16, 0, None),
    (17, 8208, 3, torch.bfloat16, 0, 0.8),      # 256-bit accesses, ragged last step
    (5, 65552, 2, torch.bfloat16, 16, None),    # 256-bit accesses, padded rows
    (4, 262160, 2, torch.bfloat16, 0, None),    # row split over a cluster of two CTAs, 256-bit accesses
    (3, 262152, 1, torch.bfloat16, 0, 0.7),     # the same with 128-bit accesses and a masked row
    (6, 50000, 3, torch.bfloat16, 0, None),     # 256-bit accesses, three groups, ragged
    (5, 100016, 2, torch.bfloat16, 16, 0.8),    # odd number of vectors, padded rows
]


@pytest.mark.parametrize("agg", [B.AGG_TOKEN_MEAN, B.AGG_SEQ_MEAN_TOKEN_MEAN])
@pytest.mark.parametrize("N,V,S,dtype,pad,mask_p", CASES)
def test_policy_loss_fwd_bwd_matches_oracle(N, V, S, dtype, pad, mask_p, agg):
    z, ids, mask, cu, adv, logp_old, g = toy_inputs(N, V, S, dtype, seed=3 * N + V + agg, mask_p=mask_p)
    if pad:
        zp = torch.zeros(N, V + pad, dtype=dtype)
        zp[:, :V] = z
        zp[:, V:] = 30.0         # would wreck the sums if the kernel read past V
        z = zp
    u = torch.rand(N, generator=g) + 0.5
    nllw = (torch.rand(N, generator=g) < 0.3).float()
    lp = make_lp(agg=agg, nll_coeff=0.05)
    got = run_gpu_policy_loss(z, ids, mask, cu, adv, logp_old, u, nllw, lp, V=V)
    ref = O.policy_loss(z[:, :V], ids, mask, cu, adv, logp_old, u, nllw, oracle_lp(lp))
    # V = 1: logp is exactly 0 and so is the NLL term; the kernel's base-2 evaluation leaves ~1e-7 |z| there,
    # which only an absolute bound can judge (1e-5 of a unit-scale loss)
    compare_policy_loss(got, ref, V, dtype, loss_floor=1e-3 if V == 1 else 0.0)
    assert got["status"] == 0
    if pad:
        assert torch.isnan(got["dlogits"][:, V:].float()).all()    # columns past V are never written


def test_inplace_dlogits_and_forward_only():
    N, V, S = 10, 151936, 2
    z, ids, mask, cu, adv, logp_old, g = toy_inputs(N, V, S, torch.bfloat16, seed=77, mask_p=0.8)
    lp = make_lp()
    ref = O.policy_loss(z, ids, mask, cu, adv, logp_old, None, None, oracle_lp(lp))
    got = run_gpu_policy_loss(z, ids, mask, cu, adv, logp_old, None, None, lp, inplace=True)
    compare_policy_loss(got, ref, V, torch.bfloat16)
    fwd = run_gpu_policy_loss(z, ids, mask, cu, adv, logp_old, None, None, lp, want_dlogits=False)
    assert torch.equal(fwd["logp"], got["logp"]) and torch.equal(fwd["loss"], got["loss"])
    # general kernel in place
    z2, ids2, mask2, cu2, adv2, old2, _ = toy_inputs(20, 777, 3, torch.float32, seed=78, mask_p=0.8)
    ref2 = O.policy_loss(z2, ids2, mask2, cu2, adv2, old2, None, None, oracle_lp(lp))
    got2 = run_gpu_policy_loss(z2, ids2, mask2, cu2, adv2, old2, None, None, lp, inplace=True)
    compare_policy_loss(got2, ref2, 777, torch.float32)


def test_ratio_one_all_masked_zero_advantage_and_bad_ids():
    N, V, S = 24, 4096, 4
    z, ids, _, cu, adv, logp_old, g = toy_inputs(N, V, S, torch.bfloat16, seed=5)
    lp = make_lp()
    # logp_old = NULL: rho = 1, loss = -masked mean of A (a closed form, not the oracle)
    got = run_gpu_policy_loss(z, ids, None, cu, adv, None, None, None, lp)
    A_rows = torch.repeat_interleave(adv, (cu[1:] - cu[:-1]).long())
    assert abs(float(got["loss"][0]) + float(A_rows.double().mean())) <= 1e-5 * abs(float(A_rows.double().mean()))
    assert got["dlogits"].float().sum(dim=1).abs().max() < 2e-3 * got["dlogits"].float().abs().max() * math.sqrt(V)
    # everything masked: zeros everywhere, nothing read
    got = run_gpu_policy_loss(z, ids, torch.zeros(N, dtype=torch.uint8), cu, adv, logp_old, None, None, lp)
    assert got["loss"].abs().max() == 0 and got["logp"].abs().max() == 0 and got["dlogits"].float().abs().max() == 0
    assert got["stats"].tolist() == [0, 0, 0, 0]
    # A = 0 everywhere: loss 0, gradient 0, log-probs still produced
    zero = torch.zeros(S)
    got = run_gpu_policy_loss(z, ids, None, cu, zero, logp_old, None, None, lp)
    ref = O.policy_loss(z, ids, None, cu, zero, logp_old, None, None, oracle_lp(lp))
    compare_policy_loss(got, ref, V, torch.bfloat16)
    assert got["dlogits"].float().abs().max() == 0 and got["stats"].tolist() == [N, 0, N, 0]
    # with SKIP_ZERO_ROWS those rows are not read at all
    got = run_gpu_policy_loss(z, ids, None, cu, zero, logp_old, None, None, make_lp(flags=B.FLAG_SKIP_ZERO_ROWS))
    assert got["stats"].tolist() == [N, 0, 0, 0] and got["logp"].abs().max() == 0
    # bad ids: flagged in the status word, treated as masked, never a fault
    bad = ids.clone()
    bad[2], bad[5] = -1, V
    got = run_gpu_policy_loss(z, bad, None, cu, adv, logp_old, None, None, lp)
    ref = O.policy_loss(z, bad, None, cu, adv, logp_old, None, None, oracle_lp(lp))
    compare_policy_loss(got, ref, V, torch.bfloat16)
    assert got["status"] == B.DEV_BAD_TOKEN_ID and int(got["stats"][3]) == 2
    assert got["dlogits"][2].float().abs().max() == 0 and got["logp"][5] == 0


def test_skip_zero_rows_mixed_batch_and_nll_rows():
    # config-4 style: own rows with pooled advantages (some groups all-equal => A = 0), peer rows that
    # only carry the SGT NLL weight
    N, V, S = 30, 151936, 6
    z, ids, _, cu, adv, logp_old, g = toy_inputs(N, V, S, torch.bfloat16, seed=9)
    adv[1] = 0.0
    adv[4] = 0.0
    adv[5] = 0.0
    nllw = torch.zeros(N)
    nllw[int(cu[5]):] = 1.0                    # the last sequence is a selected peer success
    lp = make_lp(flags=B.FLAG_SKIP_ZERO_ROWS, nll_coeff=0.1 / 1)
    got = run_gpu_policy_loss(z, ids, None, cu, adv, logp_old, None, nllw, lp)
    ref = O.policy_loss(z, ids, None, cu, adv, logp_old, None, nllw, oracle_lp(lp))
    skipped = torch.zeros(N, dtype=torch.bool)
    for s in (1, 4):
        skipped[int(cu[s]):int(cu[s + 1])] = True
    ref["logp"] = torch.where(skipped, torch.zeros_like(ref["logp"]), ref["logp"])   # skipped rows report 0
    compare_policy_loss(got, ref, V, torch.bfloat16)
    assert int(got["stats"][2]) == int((~skipped).sum())
    assert float(got["loss"][1]) > 0


def test_loss_accumulates_across_slabs():
    # one step fed in two calls (micro-batches) with the global normaliser, against one call
    N, V, S = 40, 4096, 8
    z, ids, mask, cu, adv, logp_old, g = toy_inputs(N, V, S, torch.bfloat16, seed=21, mask_p=0.85)
    valid_total = float(mask.sum())
    lp_all = make_lp(pg_den=valid_total)
    whole = run_gpu_policy_loss(z, ids, mask, cu, adv, logp_old, None, None, lp_all)
    cut_s = 3
    cut = int(cu[cut_s])
    lp_a = make_lp(pg_den=valid_total)
    a = run_gpu_policy_loss(z[:cut], ids[:cut], mask[:cut], cu[:cut_s + 1], adv[:cut_s], logp_old[:cut], None, None, lp_a)
    lp_b = make_lp(pg_den=valid_total, flags=B.FLAG_ACCUMULATE_LOSS)
    b = run_gpu_policy_loss(z[cut:], ids[cut:], mask[cut:], cu[cut_s:] - cut, adv[cut_s:], logp_old[cut:], None, None,
                            lp_b, loss_init=a["loss"], stats_init=a["stats"])
    assert abs(float(b["loss"][0]) - float(whole["loss"][0])) <= 2e-6 * abs(float(whole["loss"][0]))
    assert torch.equal(b["stats"], whole["stats"])
    assert torch.equal(torch.cat([a["dlogits"], b["dlogits"]]), whole["dlogits"])


@pytest.mark.parametrize("agg", [B.AGG_TOKEN_MEAN, B.AGG_SEQ_MEAN_TOKEN_MEAN])
def test_slab_accumulated_loss_that_does_not_cancel_matches_the_oracle_to_1e5(agg):
    """One step fed in three micro-batches of whole sequences (App. A) with the step's denominators, every advantage
    positive and an NLL weight on some rows: both accumulated losses are sums of terms of one sign and are held to
    1e-5 of the oracle's loss on the whole batch (no floor)."""
    N, V, S = 90, 8208, 9
    z, ids, mask, cu, adv, logp_old, g = toy_inputs(N, V, S, torch.bfloat16, seed=27, mask_p=0.9)
    adv = adv.abs() + 0.3
    u = torch.rand(N, generator=g) + 0.5
    nllw = (torch.rand(N, generator=g) < 0.3).float()
    den = dict(pg_den=float(mask.sum()), seq_den=float(S), nll_coeff=0.05, agg=agg)
    ref = O.policy_loss(z, ids, mask, cu, adv, logp_old, u, nllw, oracle_lp(make_lp(**den)), want_dlogits=False)
    assert ref["loss_pg"] < 0 < ref["loss_nll"] and float(ref["pg_term"].max()) <= 0
    loss, stats = None, None
    for k, (s0, s1) in enumerate(((0, 2), (2, 6), (6, 9))):
        a, b = int(cu[s0]), int(cu[s1])
        lp = make_lp(flags=B.FLAG_ACCUMULATE_LOSS if k else 0, **den)
        part = run_gpu_policy_loss(z[a:b], ids[a:b], mask[a:b], cu[s0:s1 + 1] - a, adv[s0:s1], logp_old[a:b], u[a:b],
                                   nllw[a:b], lp, loss_init=loss, stats_init=stats, want_dlogits=False)
        assert part["status"] == 0
        loss, stats = part["loss"], part["stats"]
    assert loss_close(loss[0], ref["loss_pg"]) and loss_close(loss[1], ref["loss_nll"])
    assert int(stats[0]) == ref["stats"][0]


@pytest.mark.parametrize("V,dtype", [(1000, torch.float32), (8192, torch.bfloat16)])
def test_rows_outside_every_sequence_contribute_nothing(V, dtype):
    """cu_seqlens may start after row 0 or stop short of N (the contract asks for cu[0] = 0 and cu[S] = N, but only the
    device sees the array): uncovered rows get zero gradient rows and no loss term; they still report their log-prob
    and count as valid rows, and the covered rows are what a call on them alone gives."""
    N, S, a, b = 48, 3, 5, 40
    z, ids, _, _, adv, logp_old, g = toy_inputs(N, V, S, dtype, seed=91 + V)
    cu = torch.tensor([a, 17, 29, b], dtype=torch.int32)
    nllw = (torch.rand(N, generator=g) < 0.3).float()
    lp = make_lp(nll_coeff=0.05, pg_den=float(b - a))
    got = run_gpu_policy_loss(z, ids, None, cu, adv, logp_old, None, nllw, lp)
    ref = O.policy_loss(z[a:b], ids[a:b], None, cu - a, adv, logp_old[a:b], None, nllw[a:b], oracle_lp(lp))
    assert got["status"] == 0
    outside = torch.ones(N, dtype=torch.bool)
    outside[a:b] = False
    assert float(got["dlogits"][outside].float().abs().max()) == 0
    inner = dict(got, logp=got["logp"][a:b], dlogits=got["dlogits"][a:b])
    compare_policy_loss(inner, ref, V, dtype, check_stats=False, cancelling=True)
    assert int(got["stats"][0]) == N          # every row with a valid id counts as valid, covered or not


def test_clip_boundary_neighbourhood():
    # ratios a few float32 ulps either side of 1 + eps and 1 - eps: decisions must match the oracle
    V, S = 4096, 1
    hi, lo = 1.2, 0.8
    offs = [-64, -16, -4, 4, 16, 64]
    N = 2 * len(offs) * 2
    z, ids, _, _, _, _, g = toy_inputs(N, V, 1, torch.bfloat16, seed=31)
    cu = torch.arange(N + 1, dtype=torch.int32)
    logp, _, _ = O.token_logprobs(z, ids)
    adv = torch.empty(N)
    old = torch.empty(N, dtype=torch.float64)
    k = 0
    for bound in (hi, lo):
        for sign in (1.0, -1.0):
            for o in offs:
                target = bound * (1 + o * 2.0 ** -20)       # |offset| >= 4e-6 relative
                old[k] = logp[k] - math.log(target)
                adv[k] = sign
                k += 1
    lp = make_lp()
    got = run_gpu_policy_loss(z, ids, None, cu, adv, old.float(), None, None, lp)
    ref = O.policy_loss(z, ids, None, cu, adv, old.float(), None, None, oracle_lp(lp))
    # The rows come in +A / -A pairs, so the loss cancels to ~1e-5 of its terms by construction.  A float32 sum
    # of 2^x carries ~1e-7 relative error, hence each term ~1e-7 of itself and the loss ~1e-7 of the sum of |terms|
    # whatever the residue is: "1e-5 relative under float32 accumulation" can only be asked down to a residue of
    # 1e-2 of the sum of |terms|, which is the floor used here.
    compare_policy_loss(got, ref, V, torch.bfloat16, cancelling=True)


def test_prop1_bandit_on_gpu():
    # the printed three-action example of Prop. 1 through the CUDA path (general kernel, fp32)
    eta = 1 / 25
    pi = torch.tensor([1 / 3, 2 / 3 - eta, eta], dtype=torch.float64)
    z = torch.log(pi).float().repeat(3, 1)
    ids = torch.arange(3, dtype=torch.int32)
    cu = torch.arange(4, dtype=torch.int32)
    A = torch.tensor([2 / 3, -1 / 3, -1 / 3])
    got = run_gpu_policy_loss(z, ids, None, cu, A, None, pi.float(), None, make_lp(pg_den=1.0))
    g_on = -got["dlogits"].double().sum(dim=0)
    want = torch.tensor([2 / 9, -(1 / 3) * (2 / 3 - eta), -eta / 3], dtype=torch.float64)
    assert (g_on - want).abs().max() < 1e-6


# ------------------------------------------------------------------ config-shaped batches

def _advantages_gpu(meta, mode=B.ADV_GROUP_ZNORM, learner=0, pick=B.PICK_NONE):
    P, M, G = meta.rewards.shape
    own = torch.empty(P, M, G, device="cuda")
    pool = torch.empty(P, M, G, device="cuda")
    w = torch.empty(P, M, G, device="cuda")
    n = torch.zeros(1, dtype=torch.int32, device="cuda")
    ap = B.AdvParams(mode, 0, 1e-6, 0.8, 0.2, pick, 0)
    B.mrl_group_advantages(dev(meta.rewards), dev(meta.seq_len), learner, ap, own, pool, None, None, w, n)
    torch.cuda.synchronize()
    return own.cpu(), pool.cpu(), w.cpu(), int(n.cpu())


def test_config1_full_parity():
    meta = synth.make_meta(synth.C1, seed=1)
    batch = synth.make_batch(meta)
    z = batch.logits_rows(0, batch.N)
    own_gpu, _, _, _ = _advantages_gpu(meta)
    own_ref, _ = O.group_advantages(meta.rewards)
    adv_gpu = own_gpu[batch.seq_p.long(), batch.seq_m.long(), batch.seq_g.long()]
    adv_ref = own_ref[batch.seq_p.long(), batch.seq_m.long(), batch.seq_g.long()]
    assert (adv_gpu.double() - adv_ref).abs().max() < 1e-5
    logp, _, _ = O.token_logprobs(z, batch.ids)
    logp_old = (logp + batch.noise.double()).float()
    lp = make_lp()
    got = run_gpu_policy_loss(z, batch.ids, None, batch.cu_seqlens, adv_gpu, logp_old, None, None, lp)
    ref = O.policy_loss(z, batch.ids, None, batch.cu_seqlens, adv_gpu, logp_old, None, None, oracle_lp(lp))
    compare_policy_loss(got, ref, synth.C1.V, torch.float32)
    assert batch.N == 1024 and batch.S == 16


def test_config3_twin_prp_pool_with_density_weights():
    # reduced twin of config 3: pooled advantages over own + peer rollouts, ragged peer lengths,
    # stop-gradient density weights on peer rows, full Llama-3-size vocabulary
    w = synth.scaled(synth.C3, P=2, G=2, own_len=(6, 6), rows_per_block=64)
    meta = synth.make_meta(w, seed=3)
    sel = torch.ones(w.P, w.M, w.G, dtype=torch.bool)
    batch = synth.make_batch(meta, sel)
    z = batch.logits_rows(0, batch.N)
    _, pool_gpu, _, _ = _advantages_gpu(meta)
    _, pool_ref = O.group_advantages(meta.rewards)
    assert (pool_gpu.double() - pool_ref).abs().max() < 1e-5
    adv = pool_gpu[batch.seq_p.long(), batch.seq_m.long(), batch.seq_g.long()]
    logp, _, _ = O.token_logprobs(z, batch.ids)
    logp_old = (logp + batch.noise.double()).float()
    lp = make_lp()
    got = run_gpu_policy_loss(z, batch.ids, None, batch.cu_seqlens, adv, logp_old, batch.tok_weight, None, lp)
    ref = O.policy_loss(z, batch.ids, None, batch.cu_seqlens, adv, logp_old, batch.tok_weight, None, oracle_lp(lp))
    compare_policy_loss(got, ref, w.V, torch.bfloat16)
    assert batch.is_peer.any() and (batch.tok_weight[batch.is_peer] != 1).any()


def test_config4_twin_xgrpo_baseline_with_sgt_rows():
    # reduced twin of config 4: pooled cross-policy baseline on own rows, SGT-selected peer rows with
    # NLL weight 1, lambda = 0.1, zero rows skipped
    w = synth.scaled(synth.C4, P=12, G=2, own_len=(3, 3), rows_per_block=64)
    meta = synth.make_meta(w, seed=11)
    _, pool_gpu, nllw_seq, n_gated = _advantages_gpu(meta, pick=B.PICK_SHORTEST)
    rescue, pick, w_ref, n_ref = O.sgt_gate(meta.rewards, meta.seq_len, 0, pick=O.PICK_SHORTEST)
    assert torch.equal(nllw_seq.double(), w_ref) and n_gated == n_ref and n_gated > 0
    sel = torch.zeros(w.P, w.M, w.G, dtype=torch.bool)
    sel[:, 0, :] = True
    sel |= nllw_seq > 0
    batch = synth.make_batch(meta, sel)
    z = batch.logits_rows(0, batch.N)
    si = (batch.seq_p.long(), batch.seq_m.long(), batch.seq_g.long())
    adv = torch.where(batch.seq_m == 0, pool_gpu[si], torch.zeros(batch.S))
    lens = (batch.cu_seqlens[1:] - batch.cu_seqlens[:-1]).long()
    nllw = torch.repeat_interleave(nllw_seq[si], lens)
    logp, _, _ = O.token_logprobs(z, batch.ids)
    logp_old = (logp + batch.noise.double()).float()
    lp = make_lp(nll_coeff=0.1 / n_gated, flags=B.FLAG_SKIP_ZERO_ROWS)
    got = run_gpu_policy_loss(z, batch.ids, None, batch.cu_seqlens, adv, logp_old, None, nllw, lp)
    ref = O.policy_loss(z, batch.ids, None, batch.cu_seqlens, adv, logp_old, None, nllw, oracle_lp(lp))
    A_rows = torch.repeat_interleave(adv, lens)
    skipped = (A_rows == 0) & (nllw == 0)
    ref["logp"] = torch.where(skipped, torch.zeros_like(ref["logp"]), ref["logp"])
    compare_policy_loss(got, ref, w.V, torch.bfloat16)
    assert float(got["loss"][1]) > 0 and int(got["stats"][2]) == int((~skipped).sum())


def test_config2_full_size_sampled_rows():
    """Config 2 at full size, in the launch configuration the benchmark times (packed rows, bf16,
    V = 151,936, streaming kernel).  The oracle evaluates the log-prob of EVERY row (Sec. 3) and, from them, the
    ratio, the clipped surrogate and the token-mean loss of Eq. (1) over all N rows with a noisy behaviour trace:
    `logp`, `loss[0]` and `stats` are compared in full; gradient rows are compared on a seeded row sample; and the
    ratio-one closed form (minus the token-weighted mean advantage) is checked at 1e-5 of itself."""
    w = synth.C2
    meta = synth.make_meta(w, seed=2)
    batch = synth.make_batch(meta)
    N, V, S = batch.N, w.V, batch.S
    assert 64 * 128 <= N <= 64 * 1024
    z = torch.empty(N, V, dtype=torch.bfloat16, device="cuda")
    step = 4096
    for a in range(0, N, step):
        z[a:min(N, a + step)] = batch.logits_rows(a, min(N, a + step), device="cuda")
    own_ref, _ = O.group_advantages(meta.rewards)
    adv = own_ref[batch.seq_p.long(), batch.seq_m.long(), batch.seq_g.long()].float()
    g = torch.Generator().manual_seed(5)
    rows = torch.unique(torch.cat([torch.tensor([0, 1, N - 2, N - 1]), batch.cu_seqlens[1:-1].long() - 1,
                                   batch.cu_seqlens[1:-1].long(), torch.randint(0, N, (200,), generator=g)]))
    # the oracle's log-prob of every row, chunk by chunk (the logits never exist on the host at once)
    logp_all = torch.empty(N, dtype=torch.float64)
    lse_all = torch.empty(N, dtype=torch.float64)
    for a in range(0, N, 2048):
        e = min(N, a + 2048)
        logp_all[a:e], lse_all[a:e], _ = O.token_logprobs(z[a:e].cpu(), batch.ids[a:e])
    z_s = z[rows.cuda()].cpu()
    logp_s, lse_s = logp_all[rows], lse_all[rows]
    ids_d, cu_d, adv_d = dev(batch.ids), dev(batch.cu_seqlens), dev(adv)
    logp_fwd = torch.empty(N, device="cuda")
    B.mrl_token_logprobs(z, ids_d, None, logp_fwd)
    torch.cuda.synchronize()
    assert (logp_fwd.cpu().double() - logp_all).abs().max() <= LOGP_ATOL
    logp_old = (logp_all + batch.noise.double()).float()          # behaviour trace: oracle log-probs + noise, every row
    lp = make_lp()
    ws = torch.empty(B.workspace_bytes(B.WS_POLICY_LOSS, N, V, 0, B.BF16, S), dtype=torch.uint8, device="cuda")
    dz = torch.empty_like(z)
    logp = torch.empty(N, device="cuda")
    loss = torch.empty(2, device="cuda")
    stats = torch.empty(4, dtype=torch.int64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.mrl_policy_loss_fwd_bwd(z, ids_d, None, cu_d, adv_d, dev(logp_old), None, None, lp, dz, logp, loss, stats,
                              status, ws)
    torch.cuda.synchronize()
    assert int(status.cpu()) == 0 and stats.cpu().tolist()[0] == N and stats.cpu().tolist()[2] == N
    # ---- every row: log-probs, the loss of Eq. (1) with real ratios and clipping, the clip count
    lens = (batch.cu_seqlens[1:] - batch.cu_seqlens[:-1]).long()
    A_all = torch.repeat_interleave(adv.double(), lens)
    sur_all = O.surrogate(logp_all, logp_old, A_all, torch.full_like(A_all, 1.0 / N), torch.zeros_like(A_all),
                          oracle_lp(lp))
    assert (logp.cpu().double() - logp_all).abs().max() <= LOGP_ATOL
    want_loss = float(sur_all["pg_term"].sum())
    assert loss_close(loss.cpu()[0], want_loss, sur_all["pg_term"].abs().sum())
    assert float(loss.cpu()[1]) == 0
    tie_all = sur_all["margin"] < TIE_MARGIN
    want_clipped = int(((A_all != 0) & sur_all["clipped"]).sum())
    assert want_clipped > 100 and abs(int(stats.cpu()[1]) - want_clipped) <= int(tie_all.sum())
    # ---- sampled rows: the gradient row against the oracle
    sur = {k: v[rows] for k, v in sur_all.items()}
    p = torch.exp(z_s.double() - lse_s[:, None])
    onehot = torch.zeros_like(p)
    onehot.scatter_(1, batch.ids[rows].long()[:, None], 1.0)
    want = sur["g"][:, None] * (p - onehot)
    gotd = dz[rows.cuda()].cpu().double()
    keep = sur["margin"] >= TIE_MARGIN
    assert rel_l2(gotd[keep], want[keep]) <= 1e-2
    live = keep & (sur["g"] != 0)
    assert ((gotd[live] - want[live]).norm(dim=1) / want[live].norm(dim=1)).max() <= 2e-2
    assert gotd[keep & (sur["g"] == 0)].abs().max() == 0
    # ---- closed form at full size: rho = 1 => loss = -sum_t A_t / N (advantages from the oracle)
    B.mrl_policy_loss_fwd_bwd(z, ids_d, None, cu_d, adv_d, None, None, None, lp, None, logp, loss, stats, status, ws)
    torch.cuda.synchronize()
    want_r1 = -float((adv.double() * lens.double()).sum() / N)
    assert abs(float(loss.cpu()[0]) - want_r1) <= 1e-5 * abs(want_r1)
    assert abs(want_r1) > 1e-4     # the property is not vacuous for this seed
    # ---- a loss that does not cancel: every advantage positive (MRL_ADV_MEAN_ONLY on rewards above their group mean),
    # real ratios; held to 1e-5 of the loss itself
    adv_pos = adv.abs() + 0.5
    B.mrl_policy_loss_fwd_bwd(z, ids_d, None, cu_d, dev(adv_pos), dev(logp_old), None, None, lp, None, logp, loss, stats,
                              status, ws)
    torch.cuda.synchronize()
    sur_pos = O.surrogate(logp_all, logp_old, torch.repeat_interleave(adv_pos.double(), lens),
                          torch.full_like(A_all, 1.0 / N), torch.zeros_like(A_all), oracle_lp(lp))
    assert loss_close(loss.cpu()[0], float(sur_pos["pg_term"].sum()))


@pytest.mark.parametrize("V,dtype", [(1000, torch.float32), (4096, torch.bfloat16), (40008, torch.bfloat16),
                                     (262144 + 16, torch.bfloat16), (50000, torch.bfloat16), (151936, torch.bfloat16)])
def test_extreme_logits(V, dtype):
    """Vocabulary masking with -inf, a logit that dominates the row, large magnitudes, an exactly uniform row: the
    running maximum / rescaled sum must neither overflow nor produce NaN, and must match the oracle."""
    N, S = 12, 3
    g = torch.Generator().manual_seed(V)
    z = (torch.randn(N, V, generator=g) * 2.0)
    ids = torch.randint(V // 2, V, (N,), generator=g, dtype=torch.int32)
    z[0, :V // 2] = float("-inf")                       # half of the vocabulary masked out (targets are in the other half)
    z[1, torch.randperm(V, generator=g)[:V - 40]] = float("-inf")
    z[1, ids[1]] = 0.5                                  # ... all but 40 columns masked, the target kept
    # (float32: magnitudes stay moderate -- float32 holds a log-sum-exp near 300 to 2e-5 only, which is already
    # above the 1e-5 asked of float32 gradients; the bf16 cases, judged at 1e-2, take the large ones)
    big = dtype == torch.bfloat16
    z[2, 7] = 80.0 if big else 40.0                     # one column carries all the mass: logp of the target ~ -80
    z[3, ids[3]] = 60.0 if big else 40.0                # the target carries all the mass: logp ~ 0, dz ~ 0
    z[4] = 0.0                                          # uniform: logp = -log V
    z[5] = z[5] * (30.0 if big else 6.0)                # large magnitudes
    z[6] = -200.0 if big else -30.0                     # uniform far from zero
    z[7, :] = float("-inf")
    z[7, ids[7]] = -3.0                                 # only the target survives: logp = 0
    z = z.to(dtype)
    cu = torch.tensor([0, 4, 8, 12], dtype=torch.int32)
    adv = torch.tensor([0.9, -1.2, 0.6])
    logp, _, _ = O.token_logprobs(z, ids)
    assert torch.isfinite(logp).all()
    old = (logp + 0.05 * torch.randn(N, generator=g, dtype=torch.float64)).float()
    nllw = torch.zeros(N)
    nllw[8:] = 1.0
    lp = make_lp(nll_coeff=0.1)
    got = run_gpu_policy_loss(z, ids, None, cu, adv, old, None, nllw, lp)
    ref = O.policy_loss(z, ids, None, cu, adv, old, None, nllw, oracle_lp(lp))
    assert got["status"] == 0 and torch.isfinite(got["dlogits"].float()).all() and torch.isfinite(got["loss"]).all()
    assert abs(float(got["logp"][4]) + math.log(V)) <= 1e-5 and abs(float(got["logp"][7])) <= 1e-6
    compare_policy_loss(got, ref, V, dtype, cancelling=True)
    # masked-out columns get exactly zero gradient
    assert got["dlogits"][0, :V // 2].abs().max() == 0
