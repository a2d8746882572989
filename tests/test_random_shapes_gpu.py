"""Seeded random shapes and option mixes through both loss entry points, against the oracle.

The hand-picked cases elsewhere pin each kernel path; this sweep draws the combinations nobody thought of:
empty sequences between non-empty ones, one-row batches, masks that empty a whole sequence, token weights with
exact zeros, either aggregation, a given or a derived denominator, the KL term on or off, forward only or with
the gradient, padded rows.  Every draw is a pure function of its seed.
"""
import pytest
import torch

from oracle import mrl_oracle as O
from paper_2605_07244_b200 import binding as B
from paper_2605_07244_b200 import build

from helpers import KlTerm, compare_policy_loss, loss_close, make_lp, oracle_lp, run_gpu_policy_loss
from test_lmhead_gpu import compare as compare_lmhead
from test_lmhead_gpu import run_gpu_lmhead

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    B.lib()


def _cuts_with_empty_sequences(N, S, g):
    """cu_seqlens of S sequences over N rows, non-decreasing, some sequences empty."""
    inner = torch.sort(torch.randint(0, N + 1, (S - 1,), generator=g)).values.tolist() if S > 1 else []
    return torch.tensor([0] + inner + [N], dtype=torch.int32)


def _draw_logits_case(seed):
    g = torch.Generator().manual_seed(1000 + seed)
    pick = lambda xs: xs[int(torch.randint(0, len(xs), (1,), generator=g))]
    dtype = pick([torch.bfloat16, torch.bfloat16, torch.float32])
    V = pick([1, 2, 7, 130, 1000, 4096, 4100, 8192 + 16, 12296, 40000 + 8])
    N = pick([1, 2, 3, 17, 64, 150])
    S = pick([1, 2, 5, 9])
    pad = pick([0, 0, 8, 16, 5])
    z = (torch.randn(N, V + pad, generator=g) * 2.0).to(dtype)
    z[:, V:] = 25.0                                    # would wreck the sums if anything read past V
    ids = torch.randint(0, V, (N,), generator=g, dtype=torch.int32)
    cu = _cuts_with_empty_sequences(N, S, g)
    adv = torch.randn(S, generator=g)
    adv[torch.rand(S, generator=g) < 0.25] = 0.0       # zero-advantage sequences
    mask = None
    if pick([True, False]):
        mask = (torch.rand(N, generator=g) < 0.75).to(torch.uint8)
        if S > 1 and int(cu[1]) > 0:
            mask[:int(cu[1])] = 0                       # the first sequence has no valid token at all
    logp, _, _ = O.token_logprobs(z[:, :V], ids, mask)
    logp_old = (logp + 0.15 * torch.randn(N, generator=g, dtype=torch.float64)).float()
    u = None
    if pick([True, False]):
        u = torch.rand(N, generator=g) + 0.25
        u[torch.rand(N, generator=g) < 0.2] = 0.0
    nllw = (torch.rand(N, generator=g) < 0.3).float() if pick([True, False]) else None
    agg = pick([B.AGG_TOKEN_MEAN, B.AGG_SEQ_MEAN_TOKEN_MEAN])
    n_valid = int(N if mask is None else mask.sum())
    given = pick([True, False])
    lp = make_lp(agg=agg, nll_coeff=0.07 if nllw is not None else 0.0, pg_den=float(n_valid + 11) if given else 0.0,
                 seq_den=float(S + 2) if given else 0.0,
                 flags=B.FLAG_SKIP_ZERO_ROWS if pick([True, False, False]) else 0)
    ref_trace = (logp + 0.3 * torch.randn(N, generator=g, dtype=torch.float64)).float() if pick([True, False, False]) else None
    return dict(z=z, V=V, ids=ids, mask=mask, cu=cu, adv=adv, logp_old=logp_old, u=u, nllw=nllw, lp=lp, dtype=dtype,
                ref_trace=ref_trace, want_grad=pick([True, True, False]), estimator=pick([B.KL_K1, B.KL_K2, B.KL_K3]))


@pytest.mark.parametrize("seed", range(24))
def test_logits_in_random_case(seed):
    c = _draw_logits_case(seed)
    lp = c["lp"]
    kl = KlTerm(lp, c["ref_trace"], 0.01, c["estimator"]) if c["ref_trace"] is not None else None
    got = run_gpu_policy_loss(c["z"], c["ids"], c["mask"], c["cu"], c["adv"], c["logp_old"], c["u"], c["nllw"], lp,
                              V=c["V"], want_dlogits=c["want_grad"])
    ref = O.policy_loss(c["z"][:, :c["V"]], c["ids"], c["mask"], c["cu"], c["adv"], c["logp_old"], c["u"], c["nllw"],
                        oracle_lp(lp), logp_ref=c["ref_trace"])
    assert got["status"] == 0
    if lp.flags & B.FLAG_SKIP_ZERO_ROWS:
        # rows whose multiplier is known to be zero beforehand are not read: they report logp = 0 (and still count)
        dead = ref["valid"] & ((ref["cu"] == 0) | (ref["A"] == 0)) & (ref["cn"] == 0)
        if c["ref_trace"] is not None:
            dead = torch.zeros_like(dead)           # the KL term keeps every valid row live
        if dead.any():
            assert float(got["logp"][dead].abs().max()) == 0
        # ... and cannot be classified as clipped or not
        clipped = int((ref["valid"] & ~dead & (ref["A"] != 0) & ref["clipped"]).sum())
        ref = dict(ref, logp=torch.where(dead, torch.zeros_like(ref["logp"]), ref["logp"]), stats=(ref["stats"][0], clipped))
    # A float32 log-prob carries about 1e-7 of absolute error, so an NLL term whose |logp| is tiny (a two-word
    # vocabulary with a dominant logit) cannot be held to 1e-5 of itself: floor at 2e-2 of the sum of its coefficients (2e-7 absolute per log-prob).
    compare_policy_loss(got, ref, c["V"], c["dtype"], cancelling=True, loss_floor=2e-2 * float(ref["cn"].abs().sum()))
    if kl is not None:
        # (every estimator's slope is at most max(1, |d|) and a float32 log-prob is good to about 1e-6: the term is off
        # by up to that times the coefficients, which sum to beta = 0.01, however small its own value is)
        scale = max(abs(ref["loss_kl"]), 0.1 * float(ref["kl_term"].abs().sum()))
        assert abs(kl.value() - ref["loss_kl"]) <= 1e-5 * scale + 1e-6 * 0.01


def _draw_lmhead_case(seed):
    g = torch.Generator().manual_seed(5000 + seed)
    pick = lambda xs: xs[int(torch.randint(0, len(xs), (1,), generator=g))]
    N = pick([1, 31, 128, 129, 300, 513])
    H = pick([64, 128, 192, 320])
    V = pick([37, 256, 1000, 4099, 16384 + 64, 20000])
    S = pick([1, 3, 6])
    hidden = torch.randn(N, H, generator=g).to(torch.bfloat16)
    W = (torch.randn(V, H, generator=g) * (2.0 / H ** 0.5)).to(torch.bfloat16)
    ids = torch.randint(0, V, (N,), generator=g, dtype=torch.int32)
    cu = _cuts_with_empty_sequences(N, S, g)
    adv = torch.randn(S, generator=g)
    adv[torch.rand(S, generator=g) < 0.2] = 0.0
    mask = (torch.rand(N, generator=g) < 0.8).to(torch.uint8) if pick([True, False]) else None
    zz = hidden.double() @ W.double().T
    logp, _, _ = O.token_logprobs(zz, ids, mask)
    logp_old = (logp + 0.1 * torch.randn(N, generator=g, dtype=torch.float64)).float()
    u = (torch.rand(N, generator=g) + 0.5) if pick([True, False]) else None
    nllw = (torch.rand(N, generator=g) < 0.25).float() if pick([True, False]) else None
    lp = make_lp(agg=pick([B.AGG_TOKEN_MEAN, B.AGG_SEQ_MEAN_TOKEN_MEAN]), nll_coeff=0.05 if nllw is not None else 0.0,
                 flags=B.FLAG_PAIR_TILES if pick([True, False, False]) else 0)
    return hidden, W, ids, mask, cu, adv, logp_old, u, nllw, lp


@pytest.mark.parametrize("seed", range(12))
def test_hidden_in_random_case(seed):
    hidden, W, ids, mask, cu, adv, logp_old, u, nllw, lp = _draw_lmhead_case(seed)
    got = run_gpu_lmhead(hidden, W, ids, mask, cu, adv, logp_old, u, nllw, lp)
    ref = O.fused_lmhead_loss(hidden, W, ids, mask, cu, adv, logp_old, u, nllw, oracle_lp(lp))
    tie = bool((ref["valid"] & (ref["margin"] < 2e-5)).any())
    no_gradient = float(ref["g"].abs().max()) == 0
    if no_gradient:
        assert float(got["dH"].float().abs().max()) == 0 and float(got["dW"].float().abs().max()) == 0
    compare_lmhead(got, ref, check_grads=not tie and not no_gradient)


def _draw_sequence_ratio_case(seed):
    g = torch.Generator().manual_seed(9000 + seed)
    pick = lambda xs: xs[int(torch.randint(0, len(xs), (1,), generator=g))]
    dtype = pick([torch.bfloat16, torch.float32])
    V = pick([3, 130, 1000, 4096, 8192 + 16, 40000 + 8])
    N = pick([1, 5, 33, 90])
    S = pick([1, 2, 4, 7])
    z = (torch.randn(N, V, generator=g) * 2.0).to(dtype)
    ids = torch.randint(0, V, (N,), generator=g, dtype=torch.int32)
    cu = _cuts_with_empty_sequences(N, S, g)
    adv = torch.randn(S, generator=g)
    adv[torch.rand(S, generator=g) < 0.25] = 0.0
    mask = None
    if pick([True, False]):
        mask = (torch.rand(N, generator=g) < 0.8).to(torch.uint8)
        if S > 1 and int(cu[1]) > 0:
            mask[:int(cu[1])] = 0                       # a response without a valid token
    logp, _, _ = O.token_logprobs(z, ids, mask)
    old = (logp + 0.06 * torch.randn(N, generator=g, dtype=torch.float64)).float()
    nllw = (torch.rand(N, generator=g) < 0.3).float() if pick([True, False]) else None
    lp = make_lp(nll_coeff=0.05 if nllw is not None else 0.0, ratio_level=B.RATIO_SEQUENCE)
    return dict(z=z, V=V, ids=ids, mask=mask, cu=cu, adv=adv, old=old, nllw=nllw, lp=lp, dtype=dtype,
                want_grad=pick([True, True, False]))


@pytest.mark.parametrize("seed", range(16))
def test_sequence_ratio_random_case(seed):
    """Response-level ratio (App. H) on drawn shapes: empty responses, responses with every token masked, zero
    advantages, with and without the NLL rows, forward only or with the gradient."""
    from helpers import GRAD_REL_L2_BF16, GRAD_REL_L2_F32, LOGP_ATOL, LOSS_RTOL, rel_l2
    c = _draw_sequence_ratio_case(seed)
    got = run_gpu_policy_loss(c["z"], c["ids"], c["mask"], c["cu"], c["adv"], c["old"], None, c["nllw"], c["lp"],
                              V=c["V"], want_dlogits=c["want_grad"])
    ref = O.policy_loss_sequence_ratio(c["z"], c["ids"], c["mask"], c["cu"], c["adv"], c["old"], c["nllw"],
                                       oracle_lp(c["lp"]))
    assert got["status"] == 0
    assert (got["logp"].double() - ref["logp"]).abs().max() <= LOGP_ATOL
    assert not (ref["seq_margin"] < 1e-4).any(), "a response sits on the clip boundary: change the seed"
    for k, name, terms in ((0, "loss_pg", "seq_term"), (1, "loss_nll", "nll_term")):
        # the response-level tolerance: 1e-5 of the total magnitude of the terms (a ratio exponentiates a sum of
        # float32 log-probs), plus 2e-7 absolute per NLL coefficient for log-probs near zero
        scale = max(abs(ref[name]), float(ref[terms].abs().sum()))
        floor = 2e-7 * float(ref["cn"].abs().sum()) if name == "loss_nll" else 0.0
        assert abs(float(got["loss"][k]) - ref[name]) <= LOSS_RTOL * scale + floor + 1e-12, name
    assert int(got["stats"][0]) == ref["stats"][0] and int(got["stats"][1]) == ref["stats"][1]
    if c["want_grad"]:
        dz = got["dlogits"][:, :c["V"]].double()
        assert torch.isfinite(dz).all()
        if float(ref["g"].abs().max()) == 0:
            assert float(dz.abs().max()) == 0
        else:
            assert rel_l2(dz, ref["dlogits"]) <= (GRAD_REL_L2_BF16 if c["dtype"] == torch.bfloat16 else GRAD_REL_L2_F32)
        zero = ref["g"] == 0
        if zero.any():
            assert float(dz[zero].abs().max()) == 0


@pytest.mark.parametrize("seed", range(20))
def test_group_advantages_and_gate_random_case(seed):
    """Sec. 3 advantages (own, pooled, batch-whitened) and the SGT gate of Sec. 5.3 on drawn group shapes and reward
    laws: binary, graded in [0, 1], constant groups, any learner index, every pick rule."""
    g = torch.Generator().manual_seed(13000 + seed)
    pick = lambda xs: xs[int(torch.randint(0, len(xs), (1,), generator=g))]
    P, M, G = pick([1, 2, 7, 64, 300]), pick([1, 2, 3, 4]), pick([1, 2, 4, 8, 16, 33])
    law = pick(["binary", "graded", "sparse"])
    if law == "binary":
        r = (torch.rand(P, M, G, generator=g) < torch.rand(P, M, 1, generator=g)).float()
    elif law == "graded":
        r = (torch.rand(P, M, G, generator=g) * 4).round() / 4          # 0, 1/4, ..., 1: many ties
    else:
        r = (torch.rand(P, M, G, generator=g) < 0.05).float()           # mostly all-zero groups
    if P > 1:
        r[P // 2] = float(pick([0, 1]))                                  # a prompt where every candidate agrees
    lens = torch.randint(1, 9, (P, M, G), generator=g, dtype=torch.int32)
    learner = int(torch.randint(0, M, (1,), generator=g))
    mode = pick([B.ADV_MEAN_ONLY, B.ADV_GROUP_ZNORM, B.ADV_BATCH_ZNORM])
    ddof = pick([0, 1])
    rule = pick([B.PICK_NONE, B.PICK_FIRST, B.PICK_SHORTEST, B.PICK_ALL, B.PICK_SEEDED])
    seed64 = int(torch.randint(0, 2 ** 31 - 1, (1,), generator=g))
    ap = B.AdvParams(mode, ddof, 1e-6, 0.8, 0.2, rule, seed64)
    dev = lambda t: t.cuda()
    own = torch.full((P, M, G), float("nan"), device="cuda")
    pool = torch.full((P, M, G), float("nan"), device="cuda")
    rescue = torch.full((P,), 9, dtype=torch.uint8, device="cuda")
    pk = torch.full((P,), -7, dtype=torch.int32, device="cuda")
    w = torch.full((P, M, G), float("nan"), device="cuda")
    n = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    B.mrl_group_advantages(dev(r), dev(lens), learner, ap, own, pool, rescue, pk, w, n)
    torch.cuda.synchronize()
    ref_own, ref_pool = O.group_advantages(r, mode, ddof, 1e-6)
    for got, ref in ((own, ref_own), (pool, ref_pool)):
        assert torch.isfinite(got).all()
        assert (got.cpu().double() - ref).abs().max() <= 2e-6 * max(1.0, float(ref.abs().max()))
    gate = O.sgt_gate(r, lens, learner, 0.8, 0.2, rule, seed64)
    assert torch.equal(rescue.cpu(), gate[0]) and torch.equal(pk.cpu(), gate[1])
    assert torch.equal(w.cpu().double(), gate[2]) and int(n.cpu()) == gate[3]


@pytest.mark.parametrize("seed", range(12))
def test_hidden_in_random_options(seed):
    """The fused LM head with its options drawn together: KL term (any estimator), entropy output, dW accumulated in
    float32, zero-multiplier rows skipped, pair tiles — logits, gradients and terms against the float64 oracle."""
    hidden, W, ids, mask, cu, adv, logp_old, u, nllw, lp = _draw_lmhead_case(100 + seed)
    g = torch.Generator().manual_seed(17000 + seed)
    pick = lambda xs: xs[int(torch.randint(0, len(xs), (1,), generator=g))]
    N, V = hidden.shape[0], W.shape[0]
    zz = hidden.double() @ W.double().T
    logp64, _, _ = O.token_logprobs(zz, ids, mask)
    with_kl, with_ent, accum = pick([True, False]), pick([True, False]), pick([True, False])
    if pick([True, False, False]):
        lp.flags |= B.FLAG_SKIP_ZERO_ROWS
    if accum:
        lp.flags |= B.FLAG_ACCUMULATE_DW
    ref_trace = (logp64 + 0.3 * torch.randn(N, generator=g, dtype=torch.float64)).float() if with_kl else None
    kl = KlTerm(lp, ref_trace, 0.02, pick([B.KL_K1, B.KL_K2, B.KL_K3])) if with_kl else None
    ent = torch.full((N,), float("nan"), device="cuda") if with_ent else None
    if with_ent:
        lp.entropy = ent.data_ptr()
    dW_init = torch.randn(V, hidden.shape[1], generator=g) * 0.01 if accum else None
    got = run_gpu_lmhead(hidden, W, ids, mask, cu, adv, logp_old, u, nllw, lp, dW_init=dW_init)
    ref = O.fused_lmhead_loss(hidden, W, ids, mask, cu, adv, logp_old, u, nllw, oracle_lp(lp), logp_ref=ref_trace)
    if lp.flags & B.FLAG_SKIP_ZERO_ROWS and not with_kl:
        dead = ref["valid"] & ((ref["cu"] == 0) | (ref["A"] == 0)) & (ref["cn"] == 0)
        # blocks of 256 rows made of dead or masked rows are not produced: such rows report logp = 0; a dead row in a
        # live block may report either
        lg = got["logp"].double()
        both = dead & (lg == 0)
        ref = dict(ref, logp=torch.where(both, torch.zeros_like(ref["logp"]), ref["logp"]))
    tie = bool((ref["valid"] & (ref["margin"] < 2e-5)).any())
    no_gradient = float(ref["g"].abs().max()) == 0
    compare_lmhead(got, ref, check_grads=not tie and not no_gradient, dW_base=dW_init)
    if kl is not None:
        # k1 is linear in a log-prob that carries the error of a float32-accumulated bf16 dot product (a few 1e-7, and
        # not zero-mean: the tensor core does not round its accumulator to nearest), so the term is held relative to
        # the sum of its |terms|, as in tests/test_kl_gpu.py
        # (and every estimator's slope is at most max(1, |d|): a one-token batch whose d is small has a term far below
        # the 4e-6 this path's log-probs are good to at H <= 320, times the coefficients, which sum to beta = 0.02)
        scale = max(abs(ref["loss_kl"]), float(ref["kl_term"].abs().sum()))
        assert abs(kl.value() - ref["loss_kl"]) <= 1e-5 * scale + 4e-6 * 0.02
    if with_ent:
        ref_ent = O.token_entropy(zz, ids, mask)
        e = ent.cpu().double()
        read = e != 0 if lp.flags & B.FLAG_SKIP_ZERO_ROWS else torch.ones(N, dtype=torch.bool)
        assert torch.isfinite(e).all()
        if read.any():
            assert (e - ref_ent)[read].abs().max() <= 1e-4


@pytest.mark.parametrize("seed", range(12))
def test_host_pipeline_random_case(seed):
    """The host-buffer entry point on drawn batches — empty sequences between others, masks, either aggregation, any
    micro-batch size from one sequence to everything, token or response level — against one device call on the whole
    batch: per-row outputs bit for bit, the loss up to the order of its sums."""
    from test_host_pipeline_gpu import run_host
    g = torch.Generator().manual_seed(21000 + seed)
    pick = lambda xs: xs[int(torch.randint(0, len(xs), (1,), generator=g))]
    dtype = pick([torch.bfloat16, torch.bfloat16, torch.float32])
    V = pick([1008, 4096, 8192 + 16, 40000])          # the entry point wants rows of whole 32-byte units
    N = pick([1, 40, 150, 300])
    S = pick([1, 3, 8, 20])
    z = (torch.randn(N, V, generator=g) * 2.0).to(dtype)
    ids = torch.randint(0, V, (N,), generator=g, dtype=torch.int32)
    cu = _cuts_with_empty_sequences(N, S, g)
    adv = torch.randn(S, generator=g)
    adv[torch.rand(S, generator=g) < 0.25] = 0.0
    mask = (torch.rand(N, generator=g) < 0.8).to(torch.uint8) if pick([True, False]) else None
    logp, _, _ = O.token_logprobs(z, ids, mask)
    seq_level = pick([False, False, True])
    old = (logp + (0.03 if seq_level else 0.15) * torch.randn(N, generator=g, dtype=torch.float64)).float()
    tw = (torch.rand(N, generator=g) + 0.5) if (not seq_level and pick([True, False])) else None
    nllw = (torch.rand(N, generator=g) < 0.3).float() if pick([True, False]) else None
    agg = pick([B.AGG_TOKEN_MEAN, B.AGG_SEQ_MEAN_TOKEN_MEAN])
    longest = max(1, int((cu[1:] - cu[:-1]).max()))
    slab_rows = max(longest, pick([1, 7, 64, 100000]))
    mk = lambda: make_lp(agg=agg, nll_coeff=0.05 if nllw is not None else 0.0,
                         ratio_level=B.RATIO_SEQUENCE if seq_level else B.RATIO_TOKEN)
    one = run_gpu_policy_loss(z, ids, mask, cu, adv, old, tw, nllw, mk())
    got = run_host(z, ids, mask, cu, adv, old, tw, nllw, mk(), slab_rows)
    assert got["status"] == 0 and one["status"] == 0
    bits = torch.int16 if dtype == torch.bfloat16 else torch.int32
    assert torch.equal(got["logp"], one["logp"])
    assert torch.equal(got["dlogits"].view(bits), one["dlogits"].view(bits))
    assert torch.equal(got["stats"], one["stats"])
    # the loss: float32 sums in another order (per micro-batch, then accumulated), so the two agree to a few float32
    # roundings of the total magnitude of the terms, which the oracle provides (the loss itself may cancel to far less)
    if seq_level:
        ref = O.policy_loss_sequence_ratio(z, ids, mask, cu, adv, old, nllw, oracle_lp(mk()), want_dlogits=False)
        mags = (float(ref["seq_term"].abs().sum()), float(ref["nll_term"].abs().sum()))
    else:
        ref = O.policy_loss(z, ids, mask, cu, adv, old, tw, nllw, oracle_lp(mk()), want_dlogits=False)
        mags = (float(ref["pg_term"].abs().sum()), float(ref["nll_term"].abs().sum()))
    for k in range(2):
        a, b = float(got["loss"][k]), float(one["loss"][k])
        assert abs(a - b) <= 2e-6 * max(abs(a), abs(b), mags[k]) + 1e-12
