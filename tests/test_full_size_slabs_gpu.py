"""Configs 3 and 4 at full size, streamed through mrl_policy_loss_fwd_bwd in slabs of whole sequences with loss
accumulation (the logits of one step are 136 GB and 159 GB and never exist at once).  Per slab the oracle checks a
seeded sample of rows in full (log-prob, gradient row); the accumulated loss is checked through what is exact at
any size: with ratio one it equals minus the weighted mean advantage of the inputs, and config 4's gated NLL term
is recomputed by the oracle over every selected peer row."""
import pytest
import torch

from oracle import mrl_oracle as O
from paper_2605_07244_b200 import binding as B
from paper_2605_07244_b200 import build, synth

from helpers import LOGP_ATOL, dev, loss_close, make_lp, oracle_lp, rel_l2

pytestmark = pytest.mark.gpu
SLAB_ROWS = 16384


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    B.lib()


def slabs_of_whole_sequences(cu, target_rows):
    """[(first sequence, one past the last)] with about target_rows rows each."""
    out, s0 = [], 0
    S = cu.numel() - 1
    while s0 < S:
        s1 = s0 + 1
        while s1 < S and int(cu[s1 + 1]) - int(cu[s0]) <= target_rows:
            s1 += 1
        out.append((s0, s1))
        s0 = s1
    return out


def stream_and_check(batch, V, adv_seq, tok_weight, nll_weight, nll_coeff, rows_per_slab_checked, seed, flags=0,
                     all_rows_of=None, slab_rows=SLAB_ROWS, kl=None):
    """Runs the whole batch slab by slab twice (behaviour trace = log-prob + noise; then ratio one), checks sampled
    rows against the oracle, returns the accumulated losses / stats and, for `all_rows_of` (bool [N]), the device
    log-probs of those rows next to the oracle's.  `kl` = (beta, estimator, delta f32[N]) switches the KL penalty on
    with the reference trace logp - delta (logp from the oracle on the sampled rows, from the library's forward pass
    elsewhere), so that the accumulated term has the closed form beta / N * sum_t k(delta_t)."""
    N, cu = batch.N, batch.cu_seqlens
    g = torch.Generator().manual_seed(seed)
    lp = make_lp(pg_den=float(N), nll_coeff=nll_coeff, flags=flags | B.FLAG_ACCUMULATE_LOSS)
    loss = torch.zeros(2, device="cuda")
    loss_r1 = torch.zeros(2, device="cuda")
    stats = torch.zeros(4, dtype=torch.int64, device="cuda")
    stats_r1 = torch.zeros(4, dtype=torch.int64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    picked_logp_gpu, picked_logp_ref, picked_idx = [], [], []
    worst_logp, n_checked = 0.0, 0
    kl_loss = torch.zeros(1, device="cuda")
    kl_loss_r1 = torch.zeros(1, device="cuda")
    if kl is not None:
        lp.kl_coeff, lp.kl_estimator = kl[0], kl[1]
    for s0, s1 in slabs_of_whole_sequences(cu, slab_rows):
        a, b = int(cu[s0]), int(cu[s1])
        n = b - a
        z = batch.logits_rows(a, b, device="cuda")
        ids = batch.ids[a:b]
        cu_l = dev(cu[s0:s1 + 1] - a)
        adv_l = dev(adv_seq[s0:s1])
        tw = None if tok_weight is None else tok_weight[a:b]
        nw = None if nll_weight is None else nll_weight[a:b]
        ws = torch.empty(B.workspace_bytes(B.WS_POLICY_LOSS, n, V, 0, B.BF16, s1 - s0), dtype=torch.uint8, device="cuda")
        fwd = torch.empty(n, device="cuda")
        B.mrl_token_logprobs(z, dev(ids), None, fwd)
        rows = torch.unique(torch.cat([torch.tensor([0, n - 1]), torch.randint(0, n, (rows_per_slab_checked,), generator=g)]))
        if all_rows_of is not None:
            rows = torch.unique(torch.cat([rows, all_rows_of[a:b].nonzero()[:, 0]]))
        z_s = z[rows.cuda()].cpu()
        logp_s, lse_s, _ = O.token_logprobs(z_s, ids[rows])
        logp_old = fwd.cpu() + batch.noise[a:b]
        logp_old[rows] = (logp_s + batch.noise[a:b][rows].double()).float()
        logp_ref = ref_d = None
        if kl is not None:
            logp_ref = fwd.cpu() - kl[2][a:b]
            logp_ref[rows] = (logp_s - kl[2][a:b][rows].double()).float()
            ref_d = dev(logp_ref)
            lp.logp_ref = ref_d.data_ptr()
        dz = torch.empty_like(z)
        logp = torch.empty(n, device="cuda")
        lp.kl_loss = kl_loss.data_ptr() if kl is not None else None
        B.mrl_policy_loss_fwd_bwd(z, dev(ids), None, cu_l, adv_l, dev(logp_old), dev(tw), dev(nw), lp, dz, logp, loss,
                                  stats, status, ws)
        lp.kl_loss = kl_loss_r1.data_ptr() if kl is not None else None
        B.mrl_policy_loss_fwd_bwd(z, dev(ids), None, cu_l, adv_l, None, dev(tw), dev(nw), lp, None, logp, loss_r1,
                                  stats_r1, status, ws)
        torch.cuda.synchronize()
        # ---- the sampled rows against the oracle
        lens = (cu[s0 + 1:s1 + 1] - cu[s0:s1]).long()
        A_rows = torch.repeat_interleave(adv_seq[s0:s1].double(), lens)[rows]
        len_rows = torch.repeat_interleave(lens, lens)[rows].double()
        u = torch.ones(rows.numel(), dtype=torch.float64) if tw is None else tw[rows].double()
        cn = torch.zeros(rows.numel(), dtype=torch.float64) if nw is None else nll_coeff * nw[rows].double() / len_rows
        sur = O.surrogate(logp_s, logp_old[rows], A_rows, u / N, cn, oracle_lp(lp))
        if kl is not None:
            pen = O.kl_penalty(logp_s, logp_ref[rows], torch.full_like(u, 1.0 / N), oracle_lp(lp))
            sur["g"] = sur["g"] + pen["g_kl"]
        skipped = (flags & B.FLAG_SKIP_ZERO_ROWS) and True
        got_logp = logp.cpu()[rows].double()
        dead = ((A_rows == 0) | (u == 0)) & (cn == 0) if skipped else torch.zeros_like(A_rows, dtype=torch.bool)
        worst_logp = max(worst_logp, float((got_logp - logp_s)[~dead].abs().max()) if (~dead).any() else 0.0)
        assert float(got_logp[dead].abs().max()) == 0 if dead.any() else True
        p = torch.exp(z_s.double() - lse_s[:, None])
        onehot = torch.zeros_like(p)
        onehot.scatter_(1, ids[rows].long()[:, None], 1.0)
        want = sur["g"][:, None] * (p - onehot)
        gotd = dz[rows.cuda()].cpu().double()
        keep = sur["margin"] >= 2e-5
        live = keep & (sur["g"] != 0)
        if live.any():
            assert rel_l2(gotd[live], want[live]) <= 1e-2
            assert ((gotd[live] - want[live]).norm(dim=1) / want[live].norm(dim=1)).max() <= 2e-2
        zero = keep & (sur["g"] == 0)
        if zero.any():
            assert gotd[zero].abs().max() == 0
        n_checked += int(rows.numel())
        if all_rows_of is not None:
            sel = all_rows_of[a:b][rows]
            picked_logp_gpu.append(got_logp[sel])
            picked_logp_ref.append(logp_s[sel])
            picked_idx.append(rows[sel] + a)
        del z, dz, ws
    assert int(status.cpu()) == 0
    assert worst_logp <= LOGP_ATOL
    out = dict(loss=loss.cpu(), loss_r1=loss_r1.cpu(), stats=stats.cpu(), n_checked=n_checked,
               kl_loss=float(kl_loss.cpu()), kl_loss_r1=float(kl_loss_r1.cpu()))
    if all_rows_of is not None:
        out.update(picked_gpu=torch.cat(picked_logp_gpu), picked_ref=torch.cat(picked_logp_ref), picked_idx=torch.cat(picked_idx))
    return out


def test_config3_full_size_prp_pool_in_slabs():
    w = synth.C3
    meta = synth.make_meta(w, seed=3)
    batch = synth.make_batch(meta, torch.ones(w.P, w.M, w.G, dtype=torch.bool))     # own and peer rollouts: the pool
    assert batch.N > 500_000 and batch.S == 256
    _, pool = O.group_advantages(meta.rewards)                                       # normalised over the 16 candidates
    adv_seq = pool[batch.seq_p.long(), batch.seq_m.long(), batch.seq_g.long()].float()
    res = stream_and_check(batch, w.V, adv_seq, batch.tok_weight, None, 0.0, rows_per_slab_checked=6, seed=1)
    assert int(res["stats"][0]) == batch.N and res["n_checked"] > 150
    lens = (batch.cu_seqlens[1:] - batch.cu_seqlens[:-1]).long()
    A_rows = torch.repeat_interleave(adv_seq.double(), lens)
    want = -float((A_rows * batch.tok_weight.double()).sum() / batch.N)              # ratio one: minus the weighted mean of A
    terms = float((A_rows.abs() * batch.tok_weight.double()).sum() / batch.N)
    assert loss_close(res["loss_r1"][0], want, terms)
    assert torch.isfinite(res["loss"]).all() and float(res["loss"][1]) == 0


def test_config4_full_size_xgrpo_baseline_with_sgt_rows_in_slabs():
    w = synth.C4
    meta = synth.make_meta(w, seed=4)
    rescue, pick, nllw_seq, n_gated = O.sgt_gate(meta.rewards, meta.seq_len, 0, pick=O.PICK_SHORTEST)
    assert n_gated > 0
    sel = torch.zeros(w.P, w.M, w.G, dtype=torch.bool)
    sel[:, 0, :] = True
    sel |= nllw_seq > 0
    batch = synth.make_batch(meta, sel)
    assert batch.N == 64 * 16 * 512 + n_gated * 512
    _, pool = O.group_advantages(meta.rewards)                                       # pooled cross-policy baseline
    si = (batch.seq_p.long(), batch.seq_m.long(), batch.seq_g.long())
    adv_seq = torch.where(batch.seq_m == 0, pool[si].float(), torch.zeros(batch.S))
    lens = (batch.cu_seqlens[1:] - batch.cu_seqlens[:-1]).long()
    nllw = torch.repeat_interleave(nllw_seq[si].float(), lens)
    coeff = 0.1 / n_gated
    res = stream_and_check(batch, w.V, adv_seq, None, nllw, coeff, rows_per_slab_checked=4, seed=2,
                           flags=B.FLAG_SKIP_ZERO_ROWS, all_rows_of=nllw > 0)
    assert int(res["stats"][0]) == batch.N
    # every row of the selected peer successes: log-probs, and the gated NLL term recomputed by the oracle
    assert res["picked_idx"].numel() == n_gated * 512
    assert (res["picked_gpu"] - res["picked_ref"]).abs().max() <= LOGP_ATOL
    want_nll = -float((coeff / 512.0) * res["picked_ref"].sum())
    assert abs(float(res["loss"][1]) - want_nll) <= 1e-5 * abs(want_nll)
    assert abs(float(res["loss_r1"][1]) - want_nll) <= 1e-5 * abs(want_nll)
    A_rows = torch.repeat_interleave(adv_seq.double(), lens)
    want = -float(A_rows.sum() / batch.N)
    terms = float(A_rows.abs().sum() / batch.N)
    assert loss_close(res["loss_r1"][0], want, terms)


def test_app_a_setup_pool_of_two_policies_in_16k_token_micro_batches():
    """The training setup of App. A as one step: groups of 5 rollouts from each of two policies, responses up to 3,072
    tokens, group-centred advantages whitened over the batch, clip 0.2, KL penalty with coefficient 1e-3, log-prob
    micro-batches of at most 16,384 tokens with the loss accumulated across them."""
    w = synth.C6
    meta = synth.make_meta(w, seed=6)
    batch = synth.make_batch(meta, torch.ones(w.P, w.M, w.G, dtype=torch.bool))
    assert batch.S == 40 and 60_000 < batch.N < 110_000
    assert int((batch.cu_seqlens[1:] - batch.cu_seqlens[:-1]).max()) <= 3072
    # advantages from the library (batch whitening), checked against the oracle before they are used
    P, M, G = w.P, w.M, w.G
    ap = B.AdvParams(B.ADV_BATCH_ZNORM, 0, 1e-6, 0.8, 0.2, B.PICK_NONE, 0)
    adv_own = torch.empty(P, M, G, device="cuda")
    adv_pool = torch.empty(P, M, G, device="cuda")
    B.mrl_group_advantages(dev(meta.rewards), dev(meta.seq_len), 0, ap, adv_own, adv_pool, None, None, None, None)
    own_ref, pool_ref = O.group_advantages(meta.rewards, mode=O.ADV_BATCH_ZNORM)
    assert (adv_pool.cpu().double() - pool_ref).abs().max() <= 2e-6 and (adv_own.cpu().double() - own_ref).abs().max() <= 2e-6
    adv_seq = adv_pool.cpu()[batch.seq_p.long(), batch.seq_m.long(), batch.seq_g.long()]
    assert adv_seq.abs().max() > 0
    g = torch.Generator().manual_seed(66)
    delta = 0.2 * torch.randn(batch.N, generator=g)
    beta = 1e-3
    res = stream_and_check(batch, w.V, adv_seq, batch.tok_weight, None, 0.0, rows_per_slab_checked=8, seed=3,
                           slab_rows=16384, kl=(beta, B.KL_K3, delta))
    assert int(res["stats"][0]) == batch.N and res["n_checked"] >= 40
    lens = (batch.cu_seqlens[1:] - batch.cu_seqlens[:-1]).long()
    A_rows = torch.repeat_interleave(adv_seq.double(), lens)
    want = -float((A_rows * batch.tok_weight.double()).sum() / batch.N)
    terms = float((A_rows.abs() * batch.tok_weight.double()).sum() / batch.N)
    assert loss_close(res["loss_r1"][0], want, terms)
    # the accumulated penalty against its closed form (the reference trace is logp - delta by construction; the float32
    # rounding of that difference moves k3 ~ delta^2 / 2 by a relative 2e-6 / |delta| per token, with random sign)
    d = delta.double()
    want_kl = beta * float((torch.expm1(-d) + d).sum()) / batch.N
    assert abs(res["kl_loss"] - want_kl) <= 1e-5 * want_kl and abs(res["kl_loss_r1"] - want_kl) <= 1e-5 * want_kl
