"""Shared plumbing of the GPU parity tests: run the C ABI on one set of inputs, run the oracle on the
same inputs, compare.  Tolerances: ids / masks / gate outputs bit-exact,
log-probs 1e-4 absolute, loss 1e-5 relative, bf16 gradients 1e-2 relative L2 (fp32 gradients 1e-5).

What "loss 1e-5 relative" is relative to.  A loss whose terms all have one sign (every advantage positive, an
NLL-only batch, the KL penalty) is held to 1e-5 of the loss itself.  With group-centred advantages the policy-gradient
term is a cancelling sum: |L| can be a thousandth of the sum of |terms|, while every term inherits the absolute
error of its float32 log-prob (about 1e-6, through rho = exp(logp - logp_old)), so the error of the sum is about
1e-6 of the sum of |terms| whatever L is.  Such a loss is held to 1e-5 * max(|L|, LOSS_FLOOR_FRACTION * sum |terms|):
with the fraction at 0.1 the floor is exactly that 1e-6 of the sum of |terms|.  One fraction, used everywhere."""
from __future__ import annotations

import torch

from oracle import mrl_oracle as O
from paper_2605_07244_b200 import binding as B

LOGP_ATOL = 1e-4
LOSS_RTOL = 1e-5
LOSS_FLOOR_FRACTION = 0.1   # see the module docstring
GRAD_REL_L2_BF16 = 1e-2
GRAD_REL_L2_F32 = 1e-5
TIE_MARGIN = 2e-5     # |rho - clip bound| below this: fp32 and fp64 may legitimately disagree on "clipped"


def dev(t, dtype=None):
    if t is None:
        return None
    t = torch.as_tensor(t)
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda().contiguous()


def make_lp(eps_lo=0.2, eps_hi=0.2, agg=0, flags=0, pg_den=0.0, seq_den=0.0, nll_coeff=0.0, ratio_level=0):
    return B.LossParams(eps_lo, eps_hi, agg, flags, pg_den, seq_den, nll_coeff, ratio_level)


def oracle_lp(lp: B.LossParams) -> O.LossParams:
    # float32 parameters are upcast exactly, as the kernel sees them
    return O.LossParams(eps_lo=float(lp.eps_lo), eps_hi=float(lp.eps_hi), agg_mode=lp.agg_mode,
                        pg_denominator=lp.pg_denominator, seq_denominator=lp.seq_denominator,
                        nll_coeff=float(lp.nll_coeff), ratio_level=lp.ratio_level,
                        kl_coeff=float(lp.kl_coeff), kl_estimator=lp.kl_estimator)


class KlTerm:
    """Switches the KL penalty on in `lp`: uploads the reference trace, provides the device scalar the term is
    written to, and keeps both alive for as long as `lp` is used."""

    def __init__(self, lp, logp_ref, beta, estimator, init=float("nan")):
        self.ref = dev(logp_ref, torch.float32)
        self.out = torch.full((1,), init, dtype=torch.float32, device="cuda")
        lp.logp_ref, lp.kl_loss = self.ref.data_ptr(), self.out.data_ptr()
        lp.kl_coeff, lp.kl_estimator = beta, estimator

    def value(self):
        return float(self.out.cpu())


def run_gpu_policy_loss(logits, ids, mask, cu, adv, logp_old, tok_weight, nll_weight, lp, V=None,
                        inplace=False, want_dlogits=True, loss_init=None, stats_init=None):
    """All arguments are CPU tensors (or None); returns CPU results of the CUDA path."""
    zl = dev(logits)
    N = zl.shape[0]
    Vv = zl.shape[1] if V is None else V
    S = cu.numel() - 1
    ws = torch.empty(max(B.workspace_bytes(B.WS_POLICY_LOSS, N, Vv, 0, B.BF16, S), 256), dtype=torch.uint8,
                     device="cuda")
    dl = None
    if want_dlogits:
        dl = zl if inplace else torch.full_like(zl, float("nan"))
    logp = torch.full((N,), float("nan"), device="cuda")
    loss = torch.full((2,), float("nan"), device="cuda") if loss_init is None else dev(loss_init)
    stats = torch.full((4,), -1, dtype=torch.int64, device="cuda") if stats_init is None else dev(stats_init)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.mrl_policy_loss_fwd_bwd(zl, dev(ids, torch.int32), dev(mask, torch.uint8), dev(cu, torch.int32),
                              dev(adv, torch.float32), dev(logp_old, torch.float32),
                              dev(tok_weight, torch.float32), dev(nll_weight, torch.float32), lp, dl, logp, loss,
                              stats, status, ws, V=Vv)
    torch.cuda.synchronize()
    return dict(logp=logp.cpu(), loss=loss.cpu(), stats=stats.cpu(), status=int(status.cpu()),
                dlogits=None if dl is None else dl.cpu())


def loss_close(got, want, terms_abs_sum=0.0):
    """|got - want| within 1e-5 of max(|want|, LOSS_FLOOR_FRACTION * sum |terms|); terms_abs_sum = 0 is the strict form."""
    return abs(float(got) - float(want)) <= LOSS_RTOL * max(abs(float(want)), LOSS_FLOOR_FRACTION * float(terms_abs_sum)) + 1e-12


def rel_l2(a, b):
    a, b = a.double(), b.double()
    den = float(b.norm())
    return float((a - b).norm()) / den if den > 0 else float(a.norm())


def compare_policy_loss(got, ref, V, dtype, check_stats=True, loss_floor=0.0, cancelling=False):
    """got: run_gpu_policy_loss output; ref: oracle.policy_loss output (float64, same inputs).
    cancelling: the loss terms have mixed signs; the loss is held relative to max(|L|, the floor of loss_close)."""
    assert torch.isfinite(got["logp"]).all()
    err = (got["logp"].double() - ref["logp"]).abs().max()
    assert err <= LOGP_ATOL, f"logp abs err {err}"
    for k, name, terms in ((0, "loss_pg", "pg_term"), (1, "loss_nll", "nll_term")):
        L = ref[name]
        d = abs(float(got["loss"][k]) - L)
        floor = max(loss_floor, LOSS_FLOOR_FRACTION * float(ref[terms].abs().sum()) if cancelling else 0.0)
        assert d <= LOSS_RTOL * max(abs(L), floor) + 1e-12, f"{name}: got {float(got['loss'][k])} want {L}"
    tie = ref["valid"] & (ref["margin"] < TIE_MARGIN)
    if check_stats:
        assert int(got["stats"][0]) == ref["stats"][0]
        assert abs(int(got["stats"][1]) - ref["stats"][1]) <= int(tie.sum())
    if got["dlogits"] is not None:
        dz = got["dlogits"][:, :V].double()
        want = ref["dlogits"]
        assert torch.isfinite(dz).all()
        keep = ~tie
        tol = GRAD_REL_L2_BF16 if dtype == torch.bfloat16 else GRAD_REL_L2_F32
        # (a row whose softmax is nearly one-hot has dz = g (p - onehot) ~ 0 from 1 - p, which float32 carries to 1e-7
        # absolute, not relative: such a row counts with |g|, the scale of its entries' parts, in the norm below)
        row_scale = torch.maximum(want[keep].norm(dim=1), ref["g"][keep].abs())
        # (and the KL share of g moves one for one with the float32 log-prob: beta c_t 2e-6 per row, see below)
        kl_slack = torch.zeros(())
        if "kl_w" in ref:
            unit = want[keep].norm(dim=1) / ref["g"][keep].abs().clamp_min(1e-300)          # |p - onehot| of the row
            kl_slack = (ref["kl_w"][keep].abs() * 2e-6 * unit).norm()
        err = float((dz[keep] - want[keep]).norm())
        e = max(err - float(kl_slack), 0.0) / max(float(row_scale.norm()), 1e-300)
        assert e <= tol or err == 0, f"dlogits rel L2 {e}"
        # rows that must be exactly zero are exactly zero
        zero_rows = keep & (ref["g"] == 0)
        assert dz[zero_rows].abs().max() == 0 if zero_rows.any() else True
        # per-row check on rows with a gradient: no single row hides behind the global norm
        live = keep & (ref["g"] != 0)
        if live.any():
            # (g = c u A rho + cn - beta c k'(d) may cancel: the error scales with the magnitudes of its parts, not with |g|)
            num = (dz[live] - want[live]).norm(dim=1)
            g_kl = ref["g_kl"] if "g_kl" in ref else torch.zeros_like(ref["g"])
            cancel = ((ref["g"] - ref["cn"] - g_kl).abs() + ref["cn"].abs() + g_kl.abs())[live] / ref["g"][live].abs()
            # and a row whose softmax is (nearly) one-hot has dz ~ 0: measure against |g|, the scale of g (p - onehot)
            den = torch.maximum(want[live].norm(dim=1), ref["g"][live].abs()) * cancel
            # The slopes k2' = d and k3' = 1 - exp(-d) move one for one with the log-prob, which a float32 carries to
            # about 1e-6 at |logp| ~ 10: that share of g is off by up to beta c_t 2e-6 however small d makes it.
            slack = torch.zeros_like(num)
            if "kl_w" in ref:
                slack = (ref["kl_w"].abs() * 2e-6 / ref["g"].abs())[live] * want[live].norm(dim=1)
            assert ((num - slack).clamp_min(0) / den).max() <= 2 * tol, f"worst row rel L2 {(num / den).max()}"
        for r in tie.nonzero()[:, 0].tolist():      # near-tie rows: either side of the clip is valid
            alt = rel_l2(dz[r], want[r])
            assert alt <= tol or dz[r].abs().max() == 0 or want[r].abs().max() == 0
