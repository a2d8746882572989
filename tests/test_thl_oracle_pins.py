"""Pins of the oracle's THL word alignment (App. D, Alg. 3) against what the paper and arithmetic fix:
the closed formula of Sec. 4.2, per-word mass conservation and the residual identity of Thm. 1 evaluated from
the theorem's own sets, the zero prefix leak of App. C.2, hand-worked cases, and degenerate maps."""
import torch

from oracle import mrl_oracle as O
from paper_2605_07244_b200 import synth

F64 = torch.float64


def _per_word(values, word, lo, hi, nw):
    tot = torch.zeros(nw, dtype=F64)
    for p in range(lo, hi):
        if int(word[p]) >= 0:
            tot[int(word[p])] += float(values[p])
    return tot


def test_hand_worked_two_word_example():
    # word 0: source tokens (-1.0, -0.5) -> Z = -1.5 over three target tokens; word 1: source (-2.0) over one
    src_logp = torch.tensor([-1.0, -0.5, -2.0])
    out = O.thl_word_align_logprobs(src_logp, [0, 0, 1], [0, 3], [0, 0, 0, 1], [0, 4], ignore_value=-100.0)
    assert torch.allclose(out, torch.tensor([-0.5, -0.5, -0.5, -2.0], dtype=F64), atol=0, rtol=0)


def test_closed_formula_of_section_4_2_on_random_maps():
    # l~_t = Z_{w(t)} / max(1, C_{w(t)}) on target tokens with a word, for sequences that have source mass
    wm = synth.make_word_maps(B=40, words=(1, 30), seed=4)
    out = O.thl_word_align_logprobs(wm.src_logp, wm.src_word, wm.src_cu, wm.tgt_word, wm.tgt_cu, ignore_value=7.0)
    for i in range(40):
        nw = int(wm.word_cu[i + 1] - wm.word_cu[i])
        a, b, c, d = int(wm.src_cu[i]), int(wm.src_cu[i + 1]), int(wm.tgt_cu[i]), int(wm.tgt_cu[i + 1])
        Z = _per_word(wm.src_logp, wm.src_word, a, b, nw)
        C = torch.bincount(wm.tgt_word[c:d][wm.tgt_word[c:d] >= 0].long(), minlength=nw)
        for p in range(c, d):
            w = int(wm.tgt_word[p])
            want = 7.0 if w < 0 else float(Z[w]) / max(1, int(C[w]))
            assert abs(float(out[p]) - want) <= 1e-12


def test_per_word_mass_is_conserved_and_prefix_leak_is_zero():
    # Thm. 1: sum over the target tokens of a word = sum over its source tokens whenever C_w > 0; the running sum
    # of per-word differences (prefix leak, App. C.2) therefore stays at zero over covered words
    wm = synth.make_word_maps(B=60, words=(5, 80), seed=9, p_uncovered=0.0, p_source_gap=0.0)
    out = O.thl_word_align_logprobs(wm.src_logp, wm.src_word, wm.src_cu, wm.tgt_word, wm.tgt_cu)
    worst, leak = 0.0, 0.0
    for i in range(60):
        nw = int(wm.word_cu[i + 1] - wm.word_cu[i])
        Zs = _per_word(wm.src_logp, wm.src_word, int(wm.src_cu[i]), int(wm.src_cu[i + 1]), nw)
        Zt = _per_word(out, wm.tgt_word, int(wm.tgt_cu[i]), int(wm.tgt_cu[i + 1]), nw)
        worst = max(worst, float((Zs - Zt).abs().max()))
        leak = max(leak, float(torch.cumsum(Zs - Zt, 0).abs().max()))
    assert worst <= 1e-12 and leak <= 1e-11


def test_residual_identity_of_theorem_1_from_its_own_sets():
    # L_mu - L~_mu = sum over unassigned source tokens + sum of Z_w over source-covered words without a target slot
    wm = synth.make_word_maps(B=80, words=(3, 40), seed=13, p_uncovered=0.15, p_leading_none=0.6)
    out = O.thl_word_align_logprobs(wm.src_logp, wm.src_word, wm.src_cu, wm.tgt_word, wm.tgt_cu, ignore_value=-5.0)
    has = [bool((wm.src_word[int(wm.src_cu[i]):int(wm.src_cu[i + 1])] >= 0).any()) for i in range(80)]
    L_src, L_tgt = O.thl_sequence_totals(wm.src_logp, wm.src_cu, out, wm.tgt_word, wm.tgt_cu, has)
    saw_w0 = saw_b = False
    for i in range(80):
        if not has[i]:
            continue
        nw = int(wm.word_cu[i + 1] - wm.word_cu[i])
        a, b, c, d = int(wm.src_cu[i]), int(wm.src_cu[i + 1]), int(wm.tgt_cu[i]), int(wm.tgt_cu[i + 1])
        sw, tw = wm.src_word[a:b].long(), wm.tgt_word[c:d].long()
        B_src = wm.src_logp[a:b].double()[sw < 0].sum()
        Z = _per_word(wm.src_logp, wm.src_word, a, b, nw)
        S_nonempty = torch.bincount(sw[sw >= 0], minlength=nw) > 0
        C = torch.bincount(tw[tw >= 0], minlength=nw)
        W0 = S_nonempty & (C == 0)
        R = float(B_src + Z[W0].sum())
        saw_w0 |= bool(W0.any())
        saw_b |= bool((sw < 0).any())
        assert abs(float(L_src[i] - L_tgt[i]) - R) <= 1e-10
        bound = float(wm.src_logp[a:b].double()[sw < 0].abs().sum() + sum(
            wm.src_logp[a:b].double()[sw == w].abs().sum() for w in W0.nonzero()[:, 0].tolist()))
        assert abs(float(L_src[i] - L_tgt[i])) <= bound + 1e-12
    assert saw_w0 and saw_b


def test_self_alignment_reproduces_the_word_totals_and_single_token_words_exactly():
    # same map on both sides: every word keeps its total; words of one token keep their value bit for bit
    wm = synth.make_word_maps(B=20, words=(5, 50), seed=2, p_uncovered=0.0, p_source_gap=0.0)
    out = O.thl_word_align_logprobs(wm.src_logp, wm.src_word, wm.src_cu, wm.src_word, wm.src_cu, ignore_value=0.0)
    w = wm.src_word.long()
    single = torch.ones_like(w, dtype=torch.bool)
    single[1:] &= w[1:] != w[:-1]
    single[:-1] &= w[:-1] != w[1:]
    single &= w >= 0
    assert torch.equal(out[single], wm.src_logp.double()[single])
    for i in range(20):
        nw = int(wm.word_cu[i + 1] - wm.word_cu[i])
        a, b = int(wm.src_cu[i]), int(wm.src_cu[i + 1])
        assert (_per_word(out, wm.src_word, a, b, nw) - _per_word(wm.src_logp, wm.src_word, a, b, nw)).abs().max() <= 1e-12


def test_degenerate_maps():
    ig = -100.0
    # a sequence whose source tokens have no word is skipped: everything stays at ignore_value
    out = O.thl_word_align_logprobs([-1.0, -2.0], [-1, -1], [0, 2], [0, 0, 1], [0, 3], ignore_value=ig)
    assert torch.equal(out, torch.full((3,), ig, dtype=F64))
    # a target word without source tokens gets 0 (the sum defaults to 0), a target token without a word is ignored
    out = O.thl_word_align_logprobs([-1.0], [0], [0, 1], [-1, 0, 1, 1], [0, 4], ignore_value=ig)
    assert torch.equal(out, torch.tensor([ig, -1.0, 0.0, 0.0], dtype=F64))
    # empty sequences and an empty batch
    out = O.thl_word_align_logprobs([-1.0], [0], [0, 0, 1], [0], [0, 0, 1], ignore_value=ig)
    assert torch.equal(out, torch.tensor([-1.0], dtype=F64))
    assert O.thl_word_align_logprobs([], [], [0], [], [0]).numel() == 0
