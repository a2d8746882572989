"""Plain CPU float64 oracle of the token-level policy-loss pass of Mutual RL.

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg; never by the product path.  It shares no code,
table or helper with the CUDA library and does not import the package.

Everything is a direct evaluation of the paper's definitions with plain
PyTorch CPU ops in float64 (inputs in bf16/fp32 are upcast exactly and never
re-rounded).  The only structure beyond the definitions is a split of the rows
into blocks to bound memory; rows are independent, so this changes no value.

Passages followed (by section / equation of the paper):
  * token log-prob trace  l_theta(x, y)_t = log pi_theta(y_t | x, y_<t)   (Sec. 3, Preliminaries)
  * token importance weight  w = exp(l_theta - l_old)                     (Sec. 3)
  * group-relative advantages  r_bar, A~, A~zn                           (Sec. 3)
  * clipped surrogate, Eq. (1)
  * batch whitening of group-centred advantages                          (App. A, hyperparameters)
  * PRP unified candidate pool, pool-normalised advantages                (Sec. 5.1)
  * XGRPO pooled baseline  mu_pool, sigma_pool                            (App. H, value-level coupling)
  * SGT gate / transfer, Eq. (2), L_SGT "averaged per token and aggregated over
    all gated examples"                                                  (Sec. 5.3, App. B)
  * softmax score  grad log pi(a_i) = e_i - pi                            (App. H, proof of Prop. 1)
  * response-level ratio  w = exp(L_theta - L_behavior)                     (App. H, data-level coupling)
  * policy entropy diagnostic  H_t = - sum_v p_v log p_v                   (Sec. 6, App. B: entropy curves)
  * THL word-level trace alignment  Z_w, C_w, Z_w / max(1, C_w)            (Sec. 4.2; Thm. 1; conventions of App. D)
  * THL WordSpans: maximal non-whitespace runs as character intervals      (App. D, Alg. 2)
  * KL-style regulariser  beta R(theta): a per-token KL to a reference, its own loss term,
    coefficient 1e-3                                                      (Eq. (1); App. A, hyperparameters)

Readings taken where the paper is silent are listed in the repository's
design notes; each is a parameter here with the default stated.

Pins (tests, CPU only): closed forms (uniform logits, V = 1, binary-reward
advantages), brute force on tiny inputs, finite differences, the printed
three-action example of Prop. 1, the rescue-gate probability of Def. 7, and
library special cases (scipy logsumexp, torch cross_entropy), and for the word alignment the per-word mass
conservation and the residual identity of Thm. 1 evaluated from its own set definitions (WordSpans: hand-counted
intervals of the paper's example sentence, maximality and coverage); for the KL penalty
the exact expectation identities E_pi[k1] = E_pi[k3] = KL(pi || ref) against scipy's rel_entr, second-order
agreement of k2, non-negativity, closed forms for a constant log-ratio, and finite differences.
Functions without a pin: none.
"""
from __future__ import annotations

import math
import re
from dataclasses import dataclass

import torch

F64 = torch.float64

# advantage modes (Sec. 3 gives A~ and A~zn; App. A gives batch whitening)
ADV_MEAN_ONLY = 0
ADV_GROUP_ZNORM = 1
ADV_BATCH_ZNORM = 2

# SGT pick rules (App. B: "random choice or the configured shorter-response heuristic")
PICK_NONE = 0
PICK_FIRST = 1
PICK_SHORTEST = 2
PICK_ALL = 3
PICK_SEEDED = 4

# importance ratio level: per token (Sec. 3, Eq. (1)) or per response (App. H, data-level coupling)
RATIO_TOKEN = 0
RATIO_SEQUENCE = 1

# token aggregation (Eq. (1) E_tok then 1/K; or one masked mean over all tokens)
AGG_TOKEN_MEAN = 0
AGG_SEQ_MEAN_TOKEN_MEAN = 1

# per-token estimate of KL(pi_theta || pi_ref) from the sampled token's log-ratio d = logp - logp_ref.  The paper
# says only "per-token KL between policy and reference" (App. A); the three usual sampled-token estimators are offered.
KL_K1 = 0   # d
KL_K2 = 1   # d^2 / 2
KL_K3 = 2   # exp(-d) - 1 + d   (>= 0; like k1, its expectation under pi_theta is the KL exactly)

_ROW_BLOCK = 128


def _std(x: torch.Tensor, dim, ddof: int) -> torch.Tensor:
    """Standard deviation about the sample mean with divisor (n - ddof)."""
    n = 1
    dims = dim if isinstance(dim, (tuple, list)) else (dim,)
    for d in dims:
        n *= x.shape[d]
    mean = x.mean(dim=dims, keepdim=True)
    ss = ((x - mean) ** 2).sum(dim=dims, keepdim=True)
    den = max(n - ddof, 1)
    return torch.sqrt(ss / den)


def group_advantages(rewards, mode: int = ADV_GROUP_ZNORM, ddof: int = 0, eps: float = 1e-6):
    """Group-relative advantages (Sec. 3) and their pooled counterpart (Sec. 5.1, App. H).

    rewards: [P, M, G]  (prompt, policy, rollout).
    Returns (adv_own, adv_pool), both [P, M, G] float64.
      adv_own : each policy's rollouts centred / normalised within its own group of G.
      adv_pool: centred / normalised over all M*G rewards of the prompt
                (PRP's unified pool; XGRPO's mu_pool / sigma_pool).
    mode: MEAN_ONLY  A = r - r_bar
          GROUP_ZNORM A = (r - r_bar) / (std_group + eps)
          BATCH_ZNORM A = (r - r_bar) / (std_batch + eps), std_batch over the group-centred
                      values of the policy's whole batch (own) or of all policies (pool).
    """
    r = torch.as_tensor(rewards).to(F64)
    P, M, G = r.shape
    own_c = r - r.mean(dim=2, keepdim=True)
    pool_c = r - r.mean(dim=(1, 2), keepdim=True)
    if mode == ADV_MEAN_ONLY:
        return own_c, pool_c
    if mode == ADV_GROUP_ZNORM:
        own = own_c / (_std(r, 2, ddof) + eps)
        pool = pool_c / (_std(r, (1, 2), ddof) + eps)
        return own, pool
    if mode == ADV_BATCH_ZNORM:
        own = own_c / (_std(own_c, (0, 2), ddof) + eps)        # per policy: over its P*G values
        pool = pool_c / (_std(pool_c, (0, 1, 2), ddof) + eps)  # over all P*M*G values
        return own, pool
    raise ValueError("unknown advantage mode")


def splitmix64(x: int) -> int:
    """The published SplitMix64 output function (Steele, Lea, Flood 2014), on Python ints."""
    mask = (1 << 64) - 1
    x = (x + 0x9E3779B97F4A7C15) & mask
    z = x
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & mask
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & mask
    return z ^ (z >> 31)


def sgt_gate(rewards, seq_len, learner: int, success_thr: float = 0.8, negative_thr: float = 0.2,
             pick: int = PICK_SHORTEST, seed: int = 0):
    """Success-gated transfer: rescue gate and selection of y* (Sec. 5.3; App. A; App. B).

    Gate for learner n on prompt p: every own reward is a negative (r < negative_thr, the
    strict configuration) and at least one peer reward is a success (r > success_thr).
    One peer success is selected per (learner, prompt): FIRST = lowest flat index m*G+g,
    SHORTEST = smallest seq_len (ties: lowest flat index), SEEDED = the
    (splitmix64(seed*2^32 + p) mod n_success)-th success in flat order, ALL = every peer
    success, NONE = no selection.  Thresholds are compared in the rewards' own precision
    (float32 inputs and float32 thresholds, both upcast exactly).
    Returns rescue u8[P], pick i32[P] (-1 if none; lowest selected index for ALL),
    nll_seq_weight f64[P, M, G] (1 on selected rollouts), n_gated int (number selected).
    """
    r = torch.as_tensor(rewards).to(F64)
    P, M, G = r.shape
    succ = float(torch.tensor(success_thr, dtype=torch.float32))
    neg = float(torch.tensor(negative_thr, dtype=torch.float32))
    rescue = torch.zeros(P, dtype=torch.uint8)
    picks = torch.full((P,), -1, dtype=torch.int32)
    w = torch.zeros(P, M, G, dtype=F64)
    n_gated = 0
    for p in range(P):
        own_all_negative = all(float(r[p, learner, g]) < neg for g in range(G))
        peer_succ = [m * G + g for m in range(M) if m != learner for g in range(G)
                     if float(r[p, m, g]) > succ]
        if not (own_all_negative and peer_succ):
            continue
        rescue[p] = 1
        if pick == PICK_NONE:
            continue
        if pick == PICK_FIRST:
            chosen = [peer_succ[0]]
        elif pick == PICK_SHORTEST:
            best = peer_succ[0]
            for f in peer_succ[1:]:
                if int(seq_len[p, f // G, f % G]) < int(seq_len[p, best // G, best % G]):
                    best = f
            chosen = [best]
        elif pick == PICK_ALL:
            chosen = peer_succ
        elif pick == PICK_SEEDED:
            h = splitmix64(((seed & 0xFFFFFFFF) << 32) | (p & 0xFFFFFFFF))
            chosen = [peer_succ[h % len(peer_succ)]]
        else:
            raise ValueError("unknown pick rule")
        picks[p] = chosen[0]
        for f in chosen:
            w[p, f // G, f % G] = 1.0
        n_gated += len(chosen)
    return rescue, picks, w, n_gated


def token_logprobs(logits, ids, mask=None):
    """Token log-prob trace (Sec. 3): logp_t = z[t, ids_t] - log sum_v exp(z[t, v]).

    logits [N, V] any float dtype, ids [N] int, mask [N] (None = all ones).
    Rows that are masked or whose id lies outside [0, V) give logp = 0 (and count as masked).
    Returns (logp f64[N], lse f64[N], valid bool[N]).
    """
    logits = torch.as_tensor(logits)
    N, V = logits.shape
    ids = torch.as_tensor(ids).long()
    valid = (ids >= 0) & (ids < V)
    if mask is not None:
        valid = valid & (torch.as_tensor(mask) != 0)
    lse = torch.empty(N, dtype=F64)
    tgt = torch.empty(N, dtype=F64)
    safe_ids = torch.where((ids >= 0) & (ids < V), ids, torch.zeros_like(ids))
    for a in range(0, N, _ROW_BLOCK):
        z = logits[a:a + _ROW_BLOCK].to(F64)
        m = z.max(dim=1, keepdim=True).values
        lse[a:a + _ROW_BLOCK] = (m + torch.log(torch.exp(z - m).sum(dim=1, keepdim=True)))[:, 0]
        tgt[a:a + _ROW_BLOCK] = z.gather(1, safe_ids[a:a + _ROW_BLOCK, None])[:, 0]
    logp = torch.where(valid, tgt - lse, torch.zeros_like(lse))
    return logp, lse, valid


def token_entropy(logits, ids=None, mask=None):
    """Entropy of the policy's next-token distribution at every row, H_t = - sum_v p_v log p_v with
    p = softmax(z_t) -- the quantity behind the entropy diagnostics of Sec. 6 / App. B (Fig. 5, 6).
    Evaluated as the definition; rows that are masked or have an out-of-range id give 0 (as for log-probs)."""
    logits = torch.as_tensor(logits)
    N, V = logits.shape
    H = torch.empty(N, dtype=F64)
    for a in range(0, N, _ROW_BLOCK):
        z = logits[a:a + _ROW_BLOCK].to(F64)
        logp = z - torch.logsumexp(z, dim=1, keepdim=True)
        p = torch.exp(logp)
        H[a:a + _ROW_BLOCK] = -(torch.where(p > 0, p * logp, torch.zeros_like(p))).sum(dim=1)
    valid = torch.ones(N, dtype=torch.bool)
    if ids is not None:
        ids = torch.as_tensor(ids).long()
        valid &= (ids >= 0) & (ids < V)
    if mask is not None:
        valid &= torch.as_tensor(mask) != 0
    return torch.where(valid, H, torch.zeros_like(H))


@dataclass
class LossParams:
    eps_lo: float = 0.2           # clip band [1 - eps_lo, 1 + eps_hi] (Eq. (1); App. A: width 0.2)
    eps_hi: float = 0.2
    agg_mode: int = AGG_TOKEN_MEAN
    pg_denominator: float = 0.0   # <= 0: number of valid tokens in this call
    seq_denominator: float = 0.0  # <= 0: number of sequences in this call
    nll_coeff: float = 0.0        # lambda_SGT / n_gated (Eq. (2); App. B)
    ratio_level: int = RATIO_TOKEN
    kl_coeff: float = 0.0         # beta of Eq. (1); App. A: 1e-3.  Used only when a reference trace is given
    kl_estimator: int = KL_K3


def row_coefficients(valid, cu_seqlens, adv_seq, tok_weight, nll_weight, lp: LossParams):
    """Per-row multipliers of the aggregate (Eq. (1), Eq. (2)).

    c_t   = m_t / D                     (TOKEN_MEAN; D = all valid tokens)
          = m_t / (S * len_s)           (SEQ_MEAN_TOKEN_MEAN: Eq. (1)'s E_tok, then the mean over sequences)
    cn_t  = nll_coeff * m_t * nll_weight_t / len_s   (per-token average of -log pi(y*|x))
    Returns (A_t, cu_t = c_t * u_t, cn_t), each f64[N].
    """
    valid = torch.as_tensor(valid).bool()
    N = valid.shape[0]
    cu = torch.as_tensor(cu_seqlens).long()
    S = cu.shape[0] - 1
    adv_seq = torch.as_tensor(adv_seq).to(F64)
    A = torch.zeros(N, dtype=F64)
    c = torch.zeros(N, dtype=F64)
    cn = torch.zeros(N, dtype=F64)
    u = torch.ones(N, dtype=F64) if tok_weight is None else torch.as_tensor(tok_weight).to(F64)
    nw = torch.zeros(N, dtype=F64) if nll_weight is None else torch.as_tensor(nll_weight).to(F64)
    total_valid = float(valid.sum())
    D = lp.pg_denominator if lp.pg_denominator > 0 else total_valid
    Sd = lp.seq_denominator if lp.seq_denominator > 0 else float(S)
    for s in range(S):
        a, b = int(cu[s]), int(cu[s + 1])
        if b <= a:
            continue
        v = valid[a:b].to(F64)
        len_s = float(v.sum())
        A[a:b] = adv_seq[s]
        if len_s == 0:
            continue
        if lp.agg_mode == AGG_TOKEN_MEAN:
            if D > 0:
                c[a:b] = v / D
        elif lp.agg_mode == AGG_SEQ_MEAN_TOKEN_MEAN:
            c[a:b] = v / (Sd * len_s)
        else:
            raise ValueError("unknown aggregation mode")
        cn[a:b] = lp.nll_coeff * v * nw[a:b] / len_s
    return A, c * u, cn


def surrogate(logp, logp_old, A, cu, cn, lp: LossParams):
    """Clipped surrogate per token (Eq. (1)) plus the gated NLL (Eq. (2)), from log-probs.

    rho = exp(logp - logp_old); s = min(rho A, clip(rho, 1-eps_lo, 1+eps_hi) A).
    A token is clipped (zero gradient) iff (A > 0 and rho > 1+eps_hi) or (A < 0 and
    rho < 1-eps_lo); equality counts as unclipped; A = 0 gives no gradient.
    Rows whose multiplier cu*A is zero contribute exactly 0 (no inf*0).
    Returns dict with per-row pg_term (= -cu*s), nll_term (= -cn*logp), g (dL/dlogp = -g),
    rho, clipped (bool), margin (distance of rho to the active clip bound).
    """
    logp = torch.as_tensor(logp).to(F64)
    logp_old = torch.as_tensor(logp_old).to(F64)
    rho = torch.exp(logp - logp_old)
    lo, hi = 1.0 - lp.eps_lo, 1.0 + lp.eps_hi
    s = torch.minimum(rho * A, torch.clamp(rho, lo, hi) * A)
    live = (cu != 0) & (A != 0)
    pg_term = torch.where(live, -cu * s, torch.zeros_like(s))
    nll_term = torch.where(cn != 0, -cn * logp, torch.zeros_like(s))
    clipped = ((A > 0) & (rho > hi)) | ((A < 0) & (rho < lo))
    bound = torch.where(A > 0, torch.full_like(rho, hi), torch.full_like(rho, lo))
    margin = torch.where(A != 0, (rho - bound).abs(), torch.full_like(rho, math.inf))
    g = torch.where(live & ~clipped, cu * A * rho, torch.zeros_like(s)) + cn
    return dict(pg_term=pg_term, nll_term=nll_term, g=g, rho=rho, clipped=clipped, margin=margin)


def kl_penalty(logp, logp_ref, c, lp: LossParams):
    """beta R(theta) of Eq. (1) as App. A describes it: a separate loss term, the per-token KL between the policy and
    a reference, scaled by beta.  With only the sampled token's reference log-prob at hand, the per-token KL is one of
    the sampled estimators k(d), d = logp_t - logp_ref_t (KL_K1 / KL_K2 / KL_K3 above), aggregated with the same
    token coefficients c_t as the surrogate (without the stop-gradient weight u_t):

        L_KL = beta * sum_t c_t k(d_t),      dL_KL/dlogp_t = beta c_t k'(d_t),
        k1' = 1,  k2' = d,  k3' = 1 - exp(-d).

    Returns dict: kl_term f64[N] (beta c_t k_t), g_kl f64[N] (the part of g_t: -dL_KL/dlogp_t), d, w (beta c_t).
    """
    logp = torch.as_tensor(logp).to(F64)
    d = logp - torch.as_tensor(logp_ref).to(F64)
    if lp.kl_estimator == KL_K1:
        k, dk = d, torch.ones_like(d)
    elif lp.kl_estimator == KL_K2:
        k, dk = 0.5 * d * d, d
    elif lp.kl_estimator == KL_K3:
        k, dk = torch.expm1(-d) + d, -torch.expm1(-d)
    else:
        raise ValueError("unknown KL estimator")
    w = lp.kl_coeff * c
    on = w != 0
    zero = torch.zeros_like(d)
    return dict(kl_term=torch.where(on, w * k, zero), g_kl=torch.where(on, -w * dk, zero), d=d, w=w)


def policy_loss(logits, ids, mask, cu_seqlens, adv_seq, logp_old, tok_weight=None, nll_weight=None,
                lp: LossParams | None = None, want_dlogits: bool = True, rows=None, logp_ref=None):
    """The whole logits-in pass: log-probs, ratio, clipped surrogate, aggregation, dlogits.

    dlogits[t, v] = g_t * (softmax(z_t)[v] - 1[v == ids_t])  (score e_i - pi, App. H).
    `rows` (optional LongTensor) restricts the dlogits that are materialised to those rows;
    every scalar output still covers all N rows.
    With `logp_ref` (f32/f64 [N]) the KL penalty of kl_penalty() is added: loss_kl, and its part of g.
    Returns dict: loss_pg, loss_nll, loss_kl (python floats), logp, lse, valid, g, rho, clipped, margin,
    A, cu, cn, stats (active, clipped), dlogits f64[len(rows) or N, V] (if requested).
    """
    lp = lp or LossParams()
    logits = torch.as_tensor(logits)
    N, V = logits.shape
    ids_l = torch.as_tensor(ids).long()
    logp, lse, valid = token_logprobs(logits, ids_l, mask)
    A, cu, cn = row_coefficients(valid, cu_seqlens, adv_seq, tok_weight, nll_weight, lp)
    if logp_old is None:
        logp_old = logp
    sur = surrogate(logp, logp_old, A, cu, cn, lp)
    out = dict(sur)
    out.update(logp=logp, lse=lse, valid=valid, A=A, cu=cu, cn=cn)
    out["loss_pg"] = float(sur["pg_term"].sum())
    out["loss_nll"] = float(sur["nll_term"].sum())
    out["loss_kl"] = 0.0
    if logp_ref is not None:
        _, c, _ = row_coefficients(valid, cu_seqlens, adv_seq, None, None, lp)     # c_t alone (u_t = 1)
        kl = kl_penalty(logp, logp_ref, c, lp)
        out["g"] = sur["g"] = sur["g"] + kl["g_kl"]
        out["g_kl"], out["kl_w"] = kl["g_kl"], kl["w"]     # the penalty's share of g and beta c_t, kept for the tests' error scale
        out["kl_term"] = kl["kl_term"]
        out["loss_kl"] = float(kl["kl_term"].sum())
    out["stats"] = (int(valid.sum()), int((valid & (A != 0) & sur["clipped"]).sum()))
    if want_dlogits:
        sel = torch.arange(N) if rows is None else torch.as_tensor(rows).long()
        dz = torch.empty(len(sel), V, dtype=F64)
        g = torch.where(valid, sur["g"], torch.zeros_like(sur["g"]))
        for a in range(0, len(sel), _ROW_BLOCK):
            idx = sel[a:a + _ROW_BLOCK]
            z = logits[idx].to(F64)
            p = torch.exp(z - lse[idx, None])
            onehot = torch.zeros_like(p)
            safe = torch.where(valid[idx], ids_l[idx], torch.zeros_like(ids_l[idx]))
            onehot.scatter_(1, safe[:, None], 1.0)
            dz[a:a + _ROW_BLOCK] = g[idx, None] * (p - onehot)
        out["dlogits"] = dz
    return out


def sequence_ratio_surrogate(logp, logp_old, valid, cu_seqlens, adv_seq, nll_weight, lp: LossParams):
    """Response-level importance ratio of App. H (data-level coupling): with L = sum_t l_t over the valid tokens
    of a response,  w = exp(L_theta - L_behavior),  s = min(w A, clip(w, 1-eps_lo, 1+eps_hi) A), and the loss is
    the mean of -s over the responses (the 1/K sum of Eq. (1) with E_tok replaced by the response-level term).
    A response is clipped iff (A > 0 and w > 1+eps_hi) or (A < 0 and w < 1-eps_lo); responses without a valid
    token contribute nothing.  The gated NLL term of Eq. (2) is unchanged (token level).
    Returns dict: seq_term f64[S] (= -s / S_d), w f64[S], seq_clipped bool[S], seq_margin f64[S], per-row
    g (dL/dlogp = -g), nll_term, cn.
    """
    logp = torch.as_tensor(logp).to(F64)
    logp_old = torch.as_tensor(logp_old).to(F64)
    valid = torch.as_tensor(valid).bool()
    cu = torch.as_tensor(cu_seqlens).long()
    S = cu.shape[0] - 1
    N = logp.shape[0]
    adv_seq = torch.as_tensor(adv_seq).to(F64)
    nw = torch.zeros(N, dtype=F64) if nll_weight is None else torch.as_tensor(nll_weight).to(F64)
    Sd = lp.seq_denominator if lp.seq_denominator > 0 else float(S)
    lo, hi = 1.0 - lp.eps_lo, 1.0 + lp.eps_hi
    seq_term = torch.zeros(S, dtype=F64)
    w = torch.ones(S, dtype=F64)
    seq_clipped = torch.zeros(S, dtype=torch.bool)
    seq_margin = torch.full((S,), math.inf, dtype=F64)
    g = torch.zeros(N, dtype=F64)
    cn = torch.zeros(N, dtype=F64)
    for s_ in range(S):
        a, b = int(cu[s_]), int(cu[s_ + 1])
        v = valid[a:b]
        n_valid = int(v.sum())
        if n_valid == 0:
            continue
        cn[a:b] = lp.nll_coeff * v.to(F64) * nw[a:b] / n_valid
        A = float(adv_seq[s_])
        L_theta = float(logp[a:b][v].sum())
        L_beh = float(logp_old[a:b][v].sum())
        ws = math.exp(L_theta - L_beh)
        w[s_] = ws
        if A == 0:
            continue
        sur = min(ws * A, min(max(ws, lo), hi) * A)
        seq_term[s_] = -sur / Sd
        clipped = (A > 0 and ws > hi) or (A < 0 and ws < lo)
        seq_clipped[s_] = clipped
        seq_margin[s_] = abs(ws - (hi if A > 0 else lo))
        if not clipped:
            g[a:b] = v.to(F64) * (A * ws / Sd)
    nll_term = torch.where(cn != 0, -cn * logp, torch.zeros_like(logp))
    return dict(seq_term=seq_term, w=w, seq_clipped=seq_clipped, seq_margin=seq_margin, g=g + cn, cn=cn,
                nll_term=nll_term)


def policy_loss_sequence_ratio(logits, ids, mask, cu_seqlens, adv_seq, logp_old, nll_weight=None,
                               lp: LossParams | None = None, want_dlogits: bool = True, logp_ref=None):
    """The logits-in pass with the response-level ratio: log-probs, sequence_ratio_surrogate, and
    dlogits[t, v] = g_t (softmax(z_t)[v] - 1[v == ids_t]) with the same g for every token of a response."""
    lp = lp or LossParams(ratio_level=RATIO_SEQUENCE)
    logits = torch.as_tensor(logits)
    N, V = logits.shape
    ids_l = torch.as_tensor(ids).long()
    logp, lse, valid = token_logprobs(logits, ids_l, mask)
    if logp_old is None:
        logp_old = logp
    sur = sequence_ratio_surrogate(logp, logp_old, valid, cu_seqlens, adv_seq, nll_weight, lp)
    out = dict(sur)
    out.update(logp=logp, lse=lse, valid=valid)
    out["loss_pg"] = float(sur["seq_term"].sum())
    out["loss_nll"] = float(sur["nll_term"].sum())
    out["loss_kl"] = 0.0
    if logp_ref is not None:       # the penalty stays per token (App. A) whatever the ratio's level
        _, c, _ = row_coefficients(valid, cu_seqlens, adv_seq, None, None, lp)
        kl = kl_penalty(logp, logp_ref, c, lp)
        out["g"] = sur["g"] = sur["g"] + kl["g_kl"]
        out["g_kl"], out["kl_w"] = kl["g_kl"], kl["w"]     # the penalty's share of g and beta c_t, kept for the tests' error scale
        out["kl_term"] = kl["kl_term"]
        out["loss_kl"] = float(kl["kl_term"].sum())
    cu = torch.as_tensor(cu_seqlens).long()
    lens = cu[1:] - cu[:-1]
    row_clipped = torch.repeat_interleave(sur["seq_clipped"], lens) & valid
    out["stats"] = (int(valid.sum()), int(row_clipped.sum()))
    if want_dlogits:
        dz = torch.empty(N, V, dtype=F64)
        for a in range(0, N, _ROW_BLOCK):
            z = logits[a:a + _ROW_BLOCK].to(F64)
            p = torch.exp(z - lse[a:a + _ROW_BLOCK, None])
            onehot = torch.zeros_like(p)
            safe = torch.where(valid[a:a + _ROW_BLOCK], ids_l[a:a + _ROW_BLOCK], torch.zeros_like(ids_l[a:a + _ROW_BLOCK]))
            onehot.scatter_(1, safe[:, None], 1.0)
            dz[a:a + _ROW_BLOCK] = sur["g"][a:a + _ROW_BLOCK, None] * (p - onehot)
        out["dlogits"] = dz
    return out


def fused_lmhead_loss(hidden, W, ids, mask, cu_seqlens, adv_seq, logp_old, tok_weight=None,
                      nll_weight=None, lp: LossParams | None = None, logp_ref=None):
    """Hidden-in pass: z = hidden W^T (float64), then policy_loss; dHidden = dZ W, dW = dZ^T hidden."""
    h = torch.as_tensor(hidden).to(F64)
    w = torch.as_tensor(W).to(F64)
    z = h @ w.T
    out = policy_loss(z, ids, mask, cu_seqlens, adv_seq, logp_old, tok_weight, nll_weight, lp, logp_ref=logp_ref)
    dz = out["dlogits"]
    out["dHidden"] = dz @ w
    out["dW"] = dz.T @ h
    out["logits"] = z
    return out


# ---------------------------------------------------------------------------------------------------------------
# THL word-level trace alignment (Sec. 4.2; Thm. 1; App. D)
# ---------------------------------------------------------------------------------------------------------------

def thl_word_align_logprobs(src_logp, src_word, src_cu, tgt_word, tgt_cu, ignore_value: float = 0.0):
    """Word-level trace alignment, written out from its definition (Sec. 4.2; Thm. 1 of App. H), on packed response
    tokens.  Within one sequence, with S_w the source tokens and T_w the target tokens attributed to word w:

        Z_w = sum_{s in S_w} l_src[s]          (word-level mass; 0 for a word with no source token)
        C_w = |T_w|                            (target tokens of the word)
        aligned[t] = Z_{w(t)} / max(1, C_{w(t)})   for every target token t that has a word

    Sequence i owns source tokens [src_cu[i], src_cu[i+1]) and target tokens [tgt_cu[i], tgt_cu[i+1]); a word id
    below zero means "no word".  Two conventions come from the routine of App. D rather than from the formula:
    tokens without a word keep `ignore_value`, and so does every target token of a sequence in which no source
    token has a word (such a sequence carries no mass to distribute).  The response masks m_src, m_tgt of the
    formula are already applied: only response tokens are passed.
    Returns f64[N_tgt].
    """
    src_logp = torch.as_tensor(src_logp).to(F64)
    src_word = torch.as_tensor(src_word).long()
    tgt_word = torch.as_tensor(tgt_word).long()
    src_cu = torch.as_tensor(src_cu).long()
    tgt_cu = torch.as_tensor(tgt_cu).long()
    out = torch.full((int(tgt_cu[-1]) if tgt_cu.numel() else 0,), float(ignore_value), dtype=F64)
    for i in range(src_cu.numel() - 1):
        sw = src_word[int(src_cu[i]):int(src_cu[i + 1])]
        tw = tgt_word[int(tgt_cu[i]):int(tgt_cu[i + 1])]
        s_has, t_has = sw >= 0, tw >= 0
        if not bool(s_has.any()):
            continue
        n_words = int(max(sw.max(), tw.max() if tw.numel() else -1)) + 1
        Z = torch.zeros(n_words, dtype=F64).index_add_(0, sw[s_has], src_logp[int(src_cu[i]):int(src_cu[i + 1])][s_has])
        C = torch.bincount(tw[t_has], minlength=n_words)
        w_t = tw[t_has]
        seg = out[int(tgt_cu[i]):int(tgt_cu[i + 1])]
        seg[t_has] = Z[w_t] / torch.clamp(C[w_t], min=1).to(F64)
    return out


def thl_word_spans(text: str):
    """WordSpans (App. D, Alg. 2) as the paper defines it: one (start, end) character interval, end exclusive, per
    match of the regular expression for a maximal run of non-whitespace characters, in order of appearance."""
    return [(m.start(), m.end()) for m in re.finditer(r"\S+", text)]


def thl_sequence_totals(src_logp, src_cu, aligned, tgt_word, tgt_cu, has_source):
    """L_mu (all source response tokens) and L~_mu (aligned values on target tokens with a word) per sequence,
    the two sides of Thm. 1.  `has_source[i]`: sequence i was not skipped by the algorithm."""
    src_logp = torch.as_tensor(src_logp).to(F64)
    aligned = torch.as_tensor(aligned).to(F64)
    tgt_word = torch.as_tensor(tgt_word).long()
    B = len(src_cu) - 1
    L_src, L_tgt = torch.zeros(B, dtype=F64), torch.zeros(B, dtype=F64)
    for i in range(B):
        L_src[i] = src_logp[int(src_cu[i]):int(src_cu[i + 1])].sum()
        if has_source[i]:
            a, b = int(tgt_cu[i]), int(tgt_cu[i + 1])
            L_tgt[i] = aligned[a:b][tgt_word[a:b] >= 0].sum()
    return L_src, L_tgt
