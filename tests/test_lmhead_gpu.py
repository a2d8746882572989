"""GPU parity of the hidden-in path (mrl_fused_lmhead_loss_fwd_bwd) against the CPU float64 oracle:
log-probs, loss terms, statistics, dHidden and dW on the same seeded inputs, through the C ABI."""
import pytest
import torch

from oracle import mrl_oracle as O
from paper_2605_07244_b200 import binding as B
from paper_2605_07244_b200 import build, synth

from helpers import GRAD_REL_L2_BF16, LOGP_ATOL, LOSS_RTOL, TIE_MARGIN, dev, loss_close, make_lp, oracle_lp, rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    B.lib()


def run_gpu_lmhead(hidden, W, ids, mask, cu, adv, logp_old, tok_weight, nll_weight, lp, want_grads=True,
                   dW_init=None):
    """CPU tensors in, CPU results of the CUDA path out."""
    h, w = dev(hidden), dev(W)
    N, H = h.shape
    V = w.shape[0]
    S = cu.numel() - 1
    ws = torch.empty(max(B.workspace_bytes(B.WS_FUSED_LMHEAD, N, V, H, B.BF16, S), 256), dtype=torch.uint8,
                     device="cuda")
    dH = dW = None
    if want_grads:
        dH = torch.full((N, H), float("nan"), dtype=torch.bfloat16, device="cuda")
        if lp.flags & B.FLAG_ACCUMULATE_DW:
            dW = dev(dW_init, torch.float32)
        else:
            dW = torch.full((V, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    logp = torch.full((N,), float("nan"), device="cuda")
    loss = torch.full((2,), float("nan"), device="cuda")
    stats = torch.full((4,), -1, dtype=torch.int64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.mrl_fused_lmhead_loss_fwd_bwd(h, w, dev(ids, torch.int32), dev(mask, torch.uint8), dev(cu, torch.int32),
                                    dev(adv, torch.float32), dev(logp_old, torch.float32),
                                    dev(tok_weight, torch.float32), dev(nll_weight, torch.float32), lp, dH, dW, logp,
                                    loss, stats, status, ws)
    torch.cuda.synchronize()
    return dict(logp=logp.cpu(), loss=loss.cpu(), stats=stats.cpu(), status=int(status.cpu()),
                dH=None if dH is None else dH.cpu(), dW=None if dW is None else dW.cpu())


def toy(N, H, V, S, seed, mask_p=None, h_std=1.0, w_std=None, noise=0.1):
    g = torch.Generator().manual_seed(seed)
    w_std = w_std if w_std is not None else 2.0 / H ** 0.5       # logits of a few units, like an LM head
    hidden = (torch.randn(N, H, generator=g) * h_std).to(torch.bfloat16)
    W = (torch.randn(V, H, generator=g) * w_std).to(torch.bfloat16)
    ids = torch.randint(0, V, (N,), generator=g, dtype=torch.int32)
    if N > 1:
        ids[0], ids[-1] = 0, V - 1
    cuts = sorted(torch.randperm(N - 1, generator=g)[:S - 1].add(1).tolist()) if S > 1 else []
    cu = torch.tensor([0] + cuts + [N], dtype=torch.int32)
    adv = torch.randn(S, generator=g)
    mask = None if mask_p is None else (torch.rand(N, generator=g) < mask_p).to(torch.uint8)
    z = hidden.double() @ W.double().T
    logp, _, _ = O.token_logprobs(z, ids, mask)
    logp_old = (logp + torch.randn(N, generator=g, dtype=torch.float64) * noise).float()
    return hidden, W, ids, mask, cu, adv, logp_old, g


def compare(got, ref, check_grads=True, dW_base=None, strict=False):
    assert got["status"] == 0
    assert torch.isfinite(got["logp"]).all()
    err = (got["logp"].double() - ref["logp"]).abs().max()
    assert err <= LOGP_ATOL, f"logp abs err {err}"
    # Advantages of mixed sign make the policy-gradient term a cancelling sum: the floor of helpers.loss_close
    # applies (strict=True: every term has one sign, the loss is held to 1e-5 of itself).
    for k, name, terms in ((0, "loss_pg", "pg_term"), (1, "loss_nll", "nll_term")):
        L = ref[name]
        assert loss_close(got["loss"][k], L, 0.0 if strict else ref[terms].abs().sum()), f"{name}: {float(got['loss'][k])} vs {L}"
    tie = ref["valid"] & (ref["margin"] < TIE_MARGIN)
    assert int(got["stats"][0]) == ref["stats"][0]
    assert abs(int(got["stats"][1]) - ref["stats"][1]) <= int(tie.sum())
    if not check_grads:
        return
    assert not tie.any(), "a row sits on the clip boundary: pick another seed for a gradient comparison"
    dH, dW = got["dH"].double(), got["dW"].double()
    assert torch.isfinite(dH).all() and torch.isfinite(dW).all()
    want_dW = ref["dW"] if dW_base is None else ref["dW"] + dW_base.double()
    e_h, e_w = rel_l2(dH, ref["dHidden"]), rel_l2(dW, want_dW)
    assert e_h <= GRAD_REL_L2_BF16, f"dHidden rel L2 {e_h}"
    assert e_w <= GRAD_REL_L2_BF16, f"dW rel L2 {e_w}"
    # rows without gradient are exactly zero
    zero_rows = ref["g"] == 0
    if zero_rows.any():
        assert dH[zero_rows].abs().max() == 0
    # no row of dHidden hides behind the global norm
    live = ref["g"] != 0
    if live.any():
        num = (dH[live] - ref["dHidden"][live]).norm(dim=1)
        den = ref["dHidden"][live].norm(dim=1)
        assert (num / den).max() <= 4 * GRAD_REL_L2_BF16


CASES = [
    # N, H, V, S, mask_p                      what it exercises
    (300, 128, 1000, 5, None),      # ragged row tile, ragged column tile, one chunk
    (128, 64, 256, 1, None),        # exactly one tile
    (1, 64, 37, 1, None),           # N = 1, V below one vector
    (260, 192, 40000, 7, 0.8),      # three vocabulary chunks with a ragged last one, masked rows
    (700, 256, 16384 + 8, 3, None),  # second chunk of 8 columns
]


@pytest.mark.parametrize("agg", [B.AGG_TOKEN_MEAN, B.AGG_SEQ_MEAN_TOKEN_MEAN])
@pytest.mark.parametrize("N,H,V,S,mask_p", CASES)
def test_fused_lmhead_matches_oracle(N, H, V, S, mask_p, agg):
    hidden, W, ids, mask, cu, adv, logp_old, g = toy(N, H, V, S, seed=N + V + agg, mask_p=mask_p)
    tokw = torch.exp(torch.randn(N, generator=g) * 0.5)
    nllw = (torch.rand(N, generator=g) < 0.2).float()
    lp = make_lp(agg=agg, nll_coeff=0.05)
    got = run_gpu_lmhead(hidden, W, ids, mask, cu, adv, logp_old, tokw, nllw, lp)
    ref = O.fused_lmhead_loss(hidden, W, ids, mask, cu, adv, logp_old, tokw, nllw, oracle_lp(lp))
    compare(got, ref)


@pytest.mark.parametrize("N,H,V,S,mask_p", [(300, 128, 1000, 5, None), (700, 256, 16384 + 8, 3, 0.8), (1, 64, 37, 1, None)])
def test_pair_tiles_give_the_same_results(N, H, V, S, mask_p):
    """MRL_FLAG_PAIR_TILES: every product on 256-row tiles shared by two CTAs; checked against the oracle."""
    hidden, W, ids, mask, cu, adv, logp_old, g = toy(N, H, V, S, seed=3 * N + V, mask_p=mask_p)
    nllw = (torch.rand(N, generator=g) < 0.2).float()
    lp = make_lp(nll_coeff=0.05, flags=B.FLAG_PAIR_TILES)
    got = run_gpu_lmhead(hidden, W, ids, mask, cu, adv, logp_old, None, nllw, lp)
    ref = O.fused_lmhead_loss(hidden, W, ids, mask, cu, adv, logp_old, None, nllw, oracle_lp(lp))
    compare(got, ref)


def test_forward_only_and_dw_accumulation_in_float32():
    N, H, V, S = 200, 128, 3000, 4
    hidden, W, ids, mask, cu, adv, logp_old, g = toy(N, H, V, S, seed=9)
    lp = make_lp()
    ref = O.fused_lmhead_loss(hidden, W, ids, mask, cu, adv, logp_old, None, None, oracle_lp(lp))
    fwd = run_gpu_lmhead(hidden, W, ids, mask, cu, adv, logp_old, None, None, lp, want_grads=False)
    compare(fwd, ref, check_grads=False)
    base = torch.randn(V, H, generator=g) * float(ref["dW"].abs().mean())
    lp_acc = make_lp(flags=B.FLAG_ACCUMULATE_DW)
    got = run_gpu_lmhead(hidden, W, ids, mask, cu, adv, logp_old, None, None, lp_acc, dW_init=base)
    assert got["dW"].dtype == torch.float32
    compare(got, ref, dW_base=base)


def test_degenerate_batches():
    N, H, V, S = 96, 64, 500, 3
    hidden, W, ids, mask, cu, adv, logp_old, g = toy(N, H, V, S, seed=21)
    lp = make_lp()
    # every row masked: zero loss, zero gradients
    zeros = torch.zeros(N, dtype=torch.uint8)
    got = run_gpu_lmhead(hidden, W, ids, zeros, cu, adv, logp_old, None, None, lp)
    assert got["status"] == 0 and float(got["loss"].abs().max()) == 0
    assert float(got["dH"].float().abs().max()) == 0 and float(got["dW"].float().abs().max()) == 0
    assert got["stats"][0] == 0
    # a bad id is reported, masked, and changes nothing else
    bad = ids.clone()
    bad[5] = V + 3
    got = run_gpu_lmhead(hidden, W, bad, None, cu, adv, logp_old, None, None, lp)
    assert got["status"] & B.DEV_BAD_TOKEN_ID
    ref = O.fused_lmhead_loss(hidden, W, bad, None, cu, adv, logp_old, None, None, oracle_lp(lp))
    got["status"] = 0
    compare(got, ref)
    # ratio one (no behaviour trace): loss = - masked mean of A
    got = run_gpu_lmhead(hidden, W, ids, None, cu, adv, None, None, None, lp)
    lens = (cu[1:] - cu[:-1]).double()
    want = -float((adv.double() * lens).sum() / lens.sum())
    assert abs(float(got["loss"][0]) - want) <= LOSS_RTOL * abs(want)


def test_dW_columns_sum_to_zero_and_matches_logits_in_path():
    """dz rows sum to zero, so sum_v dW[v, :] = 0 up to rounding; and the log-probs agree with the logits-in
    kernel fed the bf16-rounded logits only to that rounding (a cross-check of the two kernel families)."""
    N, H, V, S = 512, 256, 4096, 8
    hidden, W, ids, mask, cu, adv, logp_old, g = toy(N, H, V, S, seed=33)
    lp = make_lp()
    got = run_gpu_lmhead(hidden, W, ids, None, cu, adv, logp_old, None, None, lp)
    col = got["dW"].double().sum(dim=0)
    scale = got["dW"].double().abs().sum(dim=0)
    assert (col.abs() <= 2e-2 * scale + 1e-12).all()


def test_config5_reduced_twin():
    """Config 5's recipe at N = 4,096, H = 1,024, V = 32,768 (two vocabulary chunks), checked in full."""
    w = synth.scaled(synth.C5, P=16, G=16, own_len=(16, 16), V=32768, H=1024)
    meta = synth.make_meta(w, seed=3)
    batch = synth.make_batch(meta)
    N = batch.N
    assert N == 4096
    hidden = batch.hidden_rows(0, N)
    W = batch.lm_head()
    adv, _ = O.group_advantages(meta.rewards)
    adv_seq = adv[batch.seq_p.long(), batch.seq_m.long(), batch.seq_g.long()].float()
    z = hidden.double() @ W.double().T
    logp, _, _ = O.token_logprobs(z, batch.ids)
    logp_old = (logp + batch.noise.double()).float()
    lp = make_lp()
    got = run_gpu_lmhead(hidden, W, batch.ids, None, batch.cu_seqlens, adv_seq, logp_old, None, None, lp)
    ref = O.fused_lmhead_loss(hidden, W, batch.ids, None, batch.cu_seqlens, adv_seq, logp_old, None, None,
                              oracle_lp(lp))
    tie = ref["valid"] & (ref["margin"] < TIE_MARGIN)
    if tie.any():        # rows on the clip boundary may go either way: compare everything but the gradients
        compare(got, ref, check_grads=False)
    else:
        compare(got, ref)


# ------------------------------------------------------------------ config 5 at full size

def _c5_device_inputs(seed):
    """Config 5's hidden states and LM-head weight drawn on the device (the generator is seeded per block, so the
    same bits come out on either device type); returns the packed batch description as well."""
    w = synth.C5
    meta = synth.make_meta(w, seed)
    batch = synth.make_batch(meta)
    hidden = torch.empty(batch.N, w.H, dtype=w.dtype, device="cuda")
    for a in range(0, batch.N, w.rows_per_block):
        e = min(batch.N, a + w.rows_per_block)
        hidden[a:e] = batch.hidden_rows(a, e, device="cuda")
    W = batch.lm_head(device="cuda")
    adv, _ = O.group_advantages(meta.rewards)
    adv_seq = adv[batch.seq_p.long(), batch.seq_m.long(), batch.seq_g.long()].float()
    return w, batch, hidden, W, adv_seq


def _call_lmhead_on_device(hidden, W, ids, mask, cu, adv_seq, logp_old, lp):
    N, H = hidden.shape
    V = W.shape[0]
    S = cu.numel() - 1
    ws = torch.empty(B.workspace_bytes(B.WS_FUSED_LMHEAD, N, V, H, B.BF16, S), dtype=torch.uint8, device="cuda")
    out = dict(dH=torch.full((N, H), float("nan"), dtype=torch.bfloat16, device="cuda"),
               dW=torch.full((V, H), float("nan"), dtype=torch.bfloat16, device="cuda"),
               logp=torch.full((N,), float("nan"), device="cuda"), loss=torch.full((2,), float("nan"), device="cuda"),
               stats=torch.full((4,), -1, dtype=torch.int64, device="cuda"),
               status=torch.zeros(1, dtype=torch.int32, device="cuda"))
    B.mrl_fused_lmhead_loss_fwd_bwd(hidden, W, dev(ids, torch.int32), dev(mask, torch.uint8), dev(cu, torch.int32),
                                    dev(adv_seq, torch.float32), dev(logp_old, torch.float32), None, None, lp,
                                    out["dH"], out["dW"], out["logp"], out["loss"], out["stats"], out["status"], ws)
    torch.cuda.synchronize()
    del ws
    return out


def test_config5_full_size_with_a_sparse_mask_is_checked_in_full():
    """N = 65,536, H = 4,096, V = 151,936 as the benchmark launches it, with all but 192 rows masked: every output
    then depends on those rows only, which the oracle can afford in float64 -- loss, log-probs, the 192 dHidden
    rows and the whole of dW are compared; masked rows must come out exactly zero."""
    w, batch, hidden, W, adv_seq = _c5_device_inputs(seed=11)
    N, V, H = batch.N, w.V, w.H
    g = torch.Generator().manual_seed(5)
    keep = torch.sort(torch.randperm(N, generator=g)[:192]).values
    mask = torch.zeros(N, dtype=torch.uint8)
    mask[keep] = 1
    # the oracle's view: the kept rows as a packed batch of their own (same sequences, same advantages)
    seq_of_row = torch.repeat_interleave(torch.arange(batch.S), (batch.cu_seqlens[1:] - batch.cu_seqlens[:-1]).long())
    counts = torch.bincount(seq_of_row[keep], minlength=batch.S)
    sub_cu = torch.zeros(batch.S + 1, dtype=torch.int32)
    sub_cu[1:] = torch.cumsum(counts, 0)
    h_sub, W_cpu, ids_sub = hidden[keep.cuda()].cpu(), W.cpu(), batch.ids[keep]
    z_sub = h_sub.double() @ W_cpu.double().T
    logp_sub, _, _ = O.token_logprobs(z_sub, ids_sub)
    del z_sub
    old_sub = (logp_sub + batch.noise[keep].double()).float()
    logp_old = torch.zeros(N)
    logp_old[keep] = old_sub
    lp = make_lp()
    got = _call_lmhead_on_device(hidden, W, batch.ids, mask, batch.cu_seqlens, adv_seq, logp_old, lp)
    ref = O.fused_lmhead_loss(h_sub, W_cpu, ids_sub, None, sub_cu, adv_seq, old_sub, None, None, oracle_lp(lp))
    assert int(got["status"].cpu()) == 0
    assert int(got["stats"].cpu()[0]) == 192
    logp = got["logp"].cpu()
    assert (logp[keep].double() - ref["logp"]).abs().max() <= LOGP_ATOL
    assert float(logp[mask == 0].abs().max()) == 0
    assert loss_close(got["loss"].cpu()[0], ref["loss_pg"], ref["pg_term"].abs().sum())
    tie = ref["margin"] < TIE_MARGIN
    assert not tie.any(), "a kept row sits on the clip boundary: change the seed"
    dH = got["dH"].cpu()
    assert float(dH[mask == 0].float().abs().max()) == 0
    assert rel_l2(dH[keep], ref["dHidden"]) <= GRAD_REL_L2_BF16
    assert rel_l2(got["dW"].cpu(), ref["dW"]) <= GRAD_REL_L2_BF16


def test_config5_full_size_unmasked_sampled_rows_and_invariants():
    """The same launch with every row live and ratio one (no behaviour trace): the loss has the closed form
    -mean A; log-probs and dHidden are checked on 48 sampled rows the oracle evaluates one by one (g_t = A_t / N
    needs nothing from other rows); dz rows sum to zero, so the columns of dW must sum to ~0."""
    w, batch, hidden, W, adv_seq = _c5_device_inputs(seed=12)
    N, V, H = batch.N, w.V, w.H
    lp = make_lp()
    got = _call_lmhead_on_device(hidden, W, batch.ids, None, batch.cu_seqlens, adv_seq, None, lp)
    assert int(got["status"].cpu()) == 0 and int(got["stats"].cpu()[0]) == N
    lens = (batch.cu_seqlens[1:] - batch.cu_seqlens[:-1]).double()
    want_loss = -float((adv_seq.double() * lens).sum() / lens.sum())
    terms = float((adv_seq.double().abs() * lens).sum() / lens.sum())
    assert loss_close(got["loss"].cpu()[0], want_loss, terms)
    g = torch.Generator().manual_seed(6)
    rows = torch.sort(torch.randperm(N, generator=g)[:48]).values
    seq_of_row = torch.repeat_interleave(torch.arange(batch.S), lens.long())
    W64 = W.cpu().double()
    z = hidden[rows.cuda()].cpu().double() @ W64.T
    logp, lse, _ = O.token_logprobs(z, batch.ids[rows])
    assert (got["logp"].cpu()[rows].double() - logp).abs().max() <= LOGP_ATOL
    gt = adv_seq.double()[seq_of_row[rows]] / N                       # rho = 1, token mean over all N rows
    dz = torch.exp(z - lse[:, None])
    dz[torch.arange(48), batch.ids[rows].long()] -= 1.0
    dz *= gt[:, None]
    want_dH = dz @ W64
    assert rel_l2(got["dH"].cpu()[rows], want_dH) <= GRAD_REL_L2_BF16
    dW = got["dW"].cpu().double()
    assert torch.isfinite(dW).all()
    col, mag = dW.sum(dim=0), dW.abs().sum(dim=0)
    assert (col.abs() <= 2e-2 * mag + 1e-12).all()


@pytest.mark.parametrize("pair", [False, True])
def test_two_runs_give_the_same_bits(pair):
    # every sum has a fixed order (tile partials merged in tile order, chunks accumulated in sequence, float64 loss sums
    # in one block): the pass is reproducible bit for bit
    N, H, V, S = 700, 256, 40000, 6
    hidden, W, ids, mask, cu, adv, old, g = toy(N, H, V, S, seed=77, mask_p=0.9)
    lp = make_lp(flags=B.FLAG_PAIR_TILES if pair else 0)
    a = run_gpu_lmhead(hidden, W, ids, mask, cu, adv, old, None, None, lp)
    b = run_gpu_lmhead(hidden, W, ids, mask, cu, adv, old, None, None, lp)
    for k in ("logp", "loss", "stats", "dH", "dW"):
        assert torch.equal(a[k].view(torch.int16) if a[k].dtype == torch.bfloat16 else a[k],
                           b[k].view(torch.int16) if b[k].dtype == torch.bfloat16 else b[k]), k


@pytest.mark.parametrize("agg", [B.AGG_TOKEN_MEAN, B.AGG_SEQ_MEAN_TOKEN_MEAN])
@pytest.mark.parametrize("N,H,V,S,mask_p", [(300, 128, 1000, 5, None), (260, 192, 40000, 7, 0.8), (700, 256, 16384 + 8, 3, None)])
def test_losses_that_do_not_cancel_are_held_to_1e5_of_themselves(N, H, V, S, mask_p, agg):
    """Every advantage positive (what MRL_ADV_MEAN_ONLY gives on rewards above their group mean) and an NLL weight on
    a fifth of the rows: all policy-gradient terms share one sign and so do all NLL terms, so nothing cancels and
    both losses of the fused LM head are held to 1e-5 relative of the loss itself (no floor)."""
    hidden, W, ids, mask, cu, adv, logp_old, g = toy(N, H, V, S, seed=11 + N + V + agg, mask_p=mask_p)
    adv = adv.abs() + 0.25
    tokw = torch.exp(torch.randn(N, generator=g) * 0.5)
    nllw = (torch.rand(N, generator=g) < 0.2).float()
    lp = make_lp(agg=agg, nll_coeff=0.05)
    got = run_gpu_lmhead(hidden, W, ids, mask, cu, adv, logp_old, tokw, nllw, lp)
    ref = O.fused_lmhead_loss(hidden, W, ids, mask, cu, adv, logp_old, tokw, nllw, oracle_lp(lp))
    assert float(ref["pg_term"].max()) <= 0 and float(ref["nll_term"].min()) >= 0 and ref["loss_nll"] > 0 > ref["loss_pg"]
    compare(got, ref, check_grads=not bool((ref["valid"] & (ref["margin"] < TIE_MARGIN)).any()), strict=True)


def test_nll_only_batch_is_held_to_1e5_of_the_loss():
    """Eq. (2) alone (every advantage zero, NLL weight on every row): the loss is a plain token-mean cross-entropy
    per sequence, a sum of terms of one sign."""
    N, H, V, S = 300, 128, 5000, 4
    hidden, W, ids, mask, cu, _, logp_old, g = toy(N, H, V, S, seed=3)
    lp = make_lp(nll_coeff=0.25)
    got = run_gpu_lmhead(hidden, W, ids, mask, cu, torch.zeros(S), logp_old, None, torch.ones(N), lp)
    ref = O.fused_lmhead_loss(hidden, W, ids, mask, cu, torch.zeros(S), logp_old, None, torch.ones(N), oracle_lp(lp))
    assert ref["loss_pg"] == 0 and ref["loss_nll"] > 0.5
    compare(got, ref, strict=True)


def test_long_k_twin_every_row_live_dW_and_dHidden_element_by_element():
    """The long-K product at the benchmark's K: N = 65,536 rows (all K-blocks listed, every row with a gradient)
    against H = 256, V = 2,048, small enough for the oracle's float64 GEMMs.  dW = dZ^T hidden sums over all 65,536
    rows; it and dHidden are compared element by element, and the loss (advantages of one sign) to 1e-5 of itself."""
    N, H, V, S = 65536, 256, 2048, 128
    g = torch.Generator().manual_seed(21)
    hidden = torch.randn(N, H, generator=g).to(torch.bfloat16)
    W = (torch.randn(V, H, generator=g) * (2.0 / H ** 0.5)).to(torch.bfloat16)
    ids = torch.randint(0, V, (N,), generator=g, dtype=torch.int32)
    cu = torch.arange(0, N + 1, N // S, dtype=torch.int32)
    adv = torch.rand(S, generator=g) + 0.5
    z = hidden.double() @ W.double().T
    logp, _, _ = O.token_logprobs(z, ids)
    del z
    logp_old = (logp + 0.1 * torch.randn(N, generator=g, dtype=torch.float64)).float()
    lp = make_lp()
    got = run_gpu_lmhead(hidden, W, ids, None, cu, adv, logp_old, None, None, lp)
    ref = O.fused_lmhead_loss(hidden, W, ids, None, cu, adv, logp_old, None, None, oracle_lp(lp))
    assert got["status"] == 0 and int(got["stats"][0]) == N
    assert (got["logp"].double() - ref["logp"]).abs().max() <= LOGP_ATOL
    assert loss_close(got["loss"][0], ref["loss_pg"])                      # strict: all terms negative
    keep = ref["margin"] >= TIE_MARGIN                                     # rows within 2e-5 of the clip bound may go either way
    assert int((~keep).sum()) <= 64
    assert 0 < int(ref["clipped"].sum()) < N                              # clipped and unclipped rows are both present
    assert rel_l2(got["dH"][keep].double(), ref["dHidden"][keep]) <= GRAD_REL_L2_BF16
    # dW sums over the rows: the near-tie rows carry at most 64 / 65,536 of its mass, far inside the tolerance
    err = got["dW"].double() - ref["dW"]
    assert rel_l2(got["dW"].double(), ref["dW"]) <= GRAD_REL_L2_BF16
    # element by element: every entry within bf16 rounding of its value plus the float32 accumulation over 65,536 rows
    tol = 2.0 ** -7 * ref["dW"].abs() + 1e-2 * float(ref["dW"].abs().mean())
    assert bool((err.abs() <= tol).all()), f"worst dW entry off by {float((err.abs() - tol).max())} beyond its bound"
    rows_err = (got["dH"][keep].double() - ref["dHidden"][keep]).norm(dim=1) / ref["dHidden"][keep].norm(dim=1).clamp_min(1e-30)
    live = ref["g"][keep] != 0
    assert float(rows_err[live].max()) <= 4 * GRAD_REL_L2_BF16


def test_tall_tile_dW_matches_oracle_with_dead_row_blocks():
    """A dW product large enough for the 256-row tiles of a single CTA (K = 8,192 rows, 64 x 3 tall tiles): the step's
    last launch must be that kernel, and dW / dHidden must match the oracle with whole 256-row blocks of rows dead
    (zero-advantage sequences), i.e. with the K-block list of the long product in use."""
    N, H, V, S = 8192, 768, 16384, 32
    g = torch.Generator().manual_seed(33)
    hidden = torch.randn(N, H, generator=g).to(torch.bfloat16)
    W = (torch.randn(V, H, generator=g) * (2.0 / H ** 0.5)).to(torch.bfloat16)
    ids = torch.randint(0, V, (N,), generator=g, dtype=torch.int32)
    cu = torch.arange(0, N + 1, N // S, dtype=torch.int32)
    adv = torch.randn(S, generator=g)
    adv[::4] = 0.0                                                  # every fourth sequence (256 rows) has no gradient
    z = hidden.double() @ W.double().T
    logp, _, _ = O.token_logprobs(z, ids)
    del z
    logp_old = (logp + 0.1 * torch.randn(N, generator=g, dtype=torch.float64)).float()
    # A token whose ratio sits on a clip bound may be clipped on one side only, and its gradient row reaches every row
    # of dW: such tokens (one or two in 8,192) are masked out, so that the element-wise comparison below is decided
    rho = torch.exp(logp - logp_old.double())
    mask = (torch.minimum((rho - 0.8).abs(), (rho - 1.2).abs()) >= 1e-4).to(torch.uint8)
    assert int((mask == 0).sum()) <= 16
    lp = make_lp()
    with B.DominantKernelTimer(8) as timer:
        got = run_gpu_lmhead(hidden, W, ids, mask, cu, adv, logp_old, None, None, lp)
    assert "tall" in timer.last_kernel, timer.last_kernel
    ref = O.fused_lmhead_loss(hidden, W, ids, mask, cu, adv, logp_old, None, None, oracle_lp(lp))
    assert got["status"] == 0 and not bool((ref["valid"] & (ref["margin"] < TIE_MARGIN)).any())
    assert (got["logp"].double() - ref["logp"]).abs().max() <= LOGP_ATOL
    assert loss_close(got["loss"][0], ref["loss_pg"], ref["pg_term"].abs().sum())
    assert rel_l2(got["dH"].double(), ref["dHidden"]) <= GRAD_REL_L2_BF16
    assert float(got["dH"][ref["g"] == 0].float().abs().max()) == 0
    assert rel_l2(got["dW"].double(), ref["dW"]) <= GRAD_REL_L2_BF16
    # Element by element.  Every entry of dW is a sum over the tokens of terms of both signs; it is held against the same
    # product taken from the oracle's dZ rounded to bf16 (the tensor-core operand type), where only the float32
    # accumulation order, the bf16 rounding of the output and one-ulp differences between the two roundings of dZ remain
    # (the kernel's dZ is good to 1e-5, so a few per mille of its elements round the other way, each by one bf16 ulp, at most 2^-7
    # of its own term): the bound is 2^-7 of the sum of the magnitudes of an entry's terms, half a typical entry here,
    # where a tile read from the wrong place would be off by whole entries.
    dq = ref["dlogits"].bfloat16().double()
    dW_q = dq.T @ hidden.double()
    tol = 2.0 ** -7 * (dq.abs().T @ hidden.double().abs()) + 2.0 ** -8 * dW_q.abs()
    bad = (got["dW"].double() - dW_q).abs() > tol
    assert not bool(bad.any()), f"{int(bad.sum())} dW entries beyond their bound, rows {bad.any(dim=1).nonzero()[:8, 0].tolist()}"
    assert float(tol.mean()) < float(dW_q.abs().mean())                 # the bound is tighter than the entries
