"""GPU parity of mrl_thl_word_align_logprobs (THL word-level trace alignment, App. D Alg. 3) against the oracle."""
import pytest
import torch

from oracle import mrl_oracle as O
from paper_2605_07244_b200 import binding as B
from paper_2605_07244_b200 import build, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    B.lib()


def run_gpu(wm, ignore_value):
    total_words = int(wm.word_cu[-1])
    Bn = wm.src_cu.numel() - 1
    out = torch.full((int(wm.tgt_cu[-1]),), float("nan"), device="cuda")
    src_total = torch.full((Bn,), float("nan"), device="cuda")
    tgt_total = torch.full((Bn,), float("nan"), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(max(B.workspace_bytes(B.WS_THL_WORD_ALIGN, total_words, 0), 256), dtype=torch.uint8, device="cuda")
    B.mrl_thl_word_align_logprobs(wm.src_logp.cuda(), wm.src_word.cuda(), wm.src_cu.cuda(), wm.tgt_word.cuda(),
                                  wm.tgt_cu.cuda(), wm.word_cu.cuda(), total_words, ignore_value, out, src_total,
                                  tgt_total, status, ws)
    torch.cuda.synchronize()
    return out.cpu(), src_total.cpu(), tgt_total.cpu(), int(status.cpu())


def check(wm, ignore_value):
    out, src_total, tgt_total, status = run_gpu(wm, ignore_value)
    ref = O.thl_word_align_logprobs(wm.src_logp, wm.src_word, wm.src_cu, wm.tgt_word, wm.tgt_cu, ignore_value)
    assert status == 0
    # which positions carry a value is index work: exact
    assigned_ref = torch.zeros(ref.numel(), dtype=torch.bool)
    Bn = wm.src_cu.numel() - 1
    has = []
    for i in range(Bn):
        h = bool((wm.src_word[int(wm.src_cu[i]):int(wm.src_cu[i + 1])] >= 0).any())
        has.append(h)
        a, b = int(wm.tgt_cu[i]), int(wm.tgt_cu[i + 1])
        assigned_ref[a:b] = h & (wm.tgt_word[a:b] >= 0)
    assert torch.equal(out[~assigned_ref], torch.full((int((~assigned_ref).sum()),), float(ignore_value)))
    # float32 sums of a handful of log-probs, then one division: a few ulps of the word's absolute mass
    mass = O.thl_word_align_logprobs(wm.src_logp.abs(), wm.src_word, wm.src_cu, wm.tgt_word, wm.tgt_cu, 0.0)
    err = (out.double() - ref).abs()[assigned_ref]
    assert (err <= 4e-7 * mass[assigned_ref] + 1e-12).all()
    L_src, L_tgt = O.thl_sequence_totals(wm.src_logp, wm.src_cu, ref, wm.tgt_word, wm.tgt_cu, has)
    scale = O.thl_sequence_totals(wm.src_logp.abs(), wm.src_cu, mass, wm.tgt_word, wm.tgt_cu, has)
    assert ((src_total.double() - L_src).abs() <= 2e-6 * scale[0] + 1e-9).all()
    assert ((tgt_total.double() - L_tgt).abs() <= 2e-6 * scale[1] + 1e-9).all()
    return out


@pytest.mark.parametrize("Bn,words,seed", [(1, (1, 1), 1), (7, (1, 12), 2), (64, (5, 80), 3), (300, (50, 400), 4),
                                           (3, (3000, 5000), 5)])
def test_word_align_matches_oracle(Bn, words, seed):
    wm = synth.make_word_maps(Bn, words, seed, p_uncovered=0.1, p_leading_none=0.5, p_source_gap=0.05)
    check(wm, ignore_value=-100.0)
    check(wm, ignore_value=0.0)


def test_reproducible_and_conserves_word_mass():
    wm = synth.make_word_maps(128, (5, 120), seed=8, p_uncovered=0.0, p_source_gap=0.0)
    a = check(wm, -1.0)
    b, _, _, _ = run_gpu(wm, -1.0)
    assert torch.equal(a, b)                        # fixed summation order: bit for bit the same
    for i in range(128):                            # Thm. 1: the word totals of the aligned trace are the source's
        nw = int(wm.word_cu[i + 1] - wm.word_cu[i])
        s = torch.zeros(nw, dtype=torch.float64).index_add_(
            0, wm.src_word[int(wm.src_cu[i]):int(wm.src_cu[i + 1])].clamp_min(0).long(),
            torch.where(wm.src_word[int(wm.src_cu[i]):int(wm.src_cu[i + 1])] >= 0,
                        wm.src_logp[int(wm.src_cu[i]):int(wm.src_cu[i + 1])].double(), torch.zeros(1, dtype=torch.float64)))
        tw = wm.tgt_word[int(wm.tgt_cu[i]):int(wm.tgt_cu[i + 1])]
        t = torch.zeros(nw, dtype=torch.float64).index_add_(
            0, tw.clamp_min(0).long(), torch.where(tw >= 0, a[int(wm.tgt_cu[i]):int(wm.tgt_cu[i + 1])].double(),
                                                   torch.zeros(1, dtype=torch.float64)))
        assert (s - t).abs().max() <= 1e-5


def test_degenerate_and_bad_maps():
    ig = -100.0
    i32 = lambda x: torch.tensor(x, dtype=torch.int32)
    wm = synth.WordMaps(i32([-1, -1, 0]), i32([0, 2, 3]), i32([0, 0, 1, -1, 0, 1]), i32([0, 3, 6]), i32([0, 2, 4]),
                        torch.tensor([-1.0, -2.0, -3.0]))
    out, _, _, status = run_gpu(wm, ig)
    assert status == 0
    assert torch.equal(out, torch.tensor([ig, ig, ig, ig, -3.0, 0.0]))   # first sequence skipped, target word 1 gets 0
    # a word id in two separate runs, and one outside the sequence's range: reported, nothing faults
    bad = synth.WordMaps(i32([0, 1, 0]), i32([0, 3]), i32([0, 1, 7]), i32([0, 3]), i32([0, 2]),
                         torch.tensor([-1.0, -2.0, -3.0]))
    _, _, _, status = run_gpu(bad, ig)
    assert status & B.DEV_BAD_WORD_MAP
    # empty sequences between non-empty ones
    gaps = synth.WordMaps(i32([0]), i32([0, 0, 1, 1]), i32([0, 0]), i32([0, 0, 2, 2]), i32([0, 0, 1, 1]),
                          torch.tensor([-4.0]))
    out, src_total, tgt_total, status = run_gpu(gaps, ig)
    assert status == 0 and torch.equal(out, torch.tensor([-2.0, -2.0]))
    assert torch.equal(src_total, torch.tensor([0.0, -4.0, 0.0])) and torch.equal(tgt_total, torch.tensor([0.0, -4.0, 0.0]))
    # B = 0 is a no-op, null pointers with B > 0 are refused on the host
    f = B.lib().mrl_thl_word_align_logprobs
    assert f(None, None, None, None, None, None, 0, 0, 0, 0, 0.0, None, None, None, None, None, 0, None) == 0
    assert f(None, None, None, None, None, None, 1, 0, 0, 0, 0.0, None, None, None, None, None, 0, None) == 1


def test_offsets_beyond_the_arrays_are_reported_and_stay_inside_the_buffers():
    """Offset arrays live in device memory, so only the kernel can check them.  Offsets that run past the token
    arrays or the word total are cut to the arrays and reported through the status word; the cells beyond the
    arrays' stated lengths (guard cells here) are neither read into the result nor written."""
    ig = -7.0
    i32 = lambda x: torch.tensor(x, dtype=torch.int32)
    n_src, n_tgt, n_words, guard = 3, 4, 2, 64
    src_logp = torch.cat([torch.tensor([-1.0, -0.5, -2.0]), torch.full((guard,), 1e30)]).cuda()
    src_word = torch.cat([i32([0, 0, 1]), torch.zeros(guard, dtype=torch.int32)]).cuda()
    tgt_word = torch.cat([i32([0, 0, 0, 1]), torch.zeros(guard, dtype=torch.int32)]).cuda()
    out = torch.full((n_tgt + guard,), 123.0, device="cuda")
    ws = torch.full((2 * 256 + 4 * guard,), 0x5A, dtype=torch.uint8, device="cuda")
    for src_cu, tgt_cu, word_cu in (([0, 3 + 40], [0, 4], [0, 2]),          # source range past N_src
                                    ([0, 3], [0, 4 + 40], [0, 2]),          # target range past N_tgt
                                    ([0, 3], [0, 4], [0, 2 + 40]),          # word range past total_words
                                    ([0, 3], [2, 1], [0, 2])):              # decreasing offsets
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        out.fill_(123.0)
        d_src_cu, d_tgt_cu, d_word_cu = i32(src_cu).cuda(), i32(tgt_cu).cuda(), i32(word_cu).cuda()
        rc = B.lib().mrl_thl_word_align_logprobs(
            src_logp.data_ptr(), src_word.data_ptr(), d_src_cu.data_ptr(), tgt_word.data_ptr(),
            d_tgt_cu.data_ptr(), d_word_cu.data_ptr(), 1, n_src, n_tgt, n_words, ig,
            out.data_ptr(), None, None, status.data_ptr(), ws.data_ptr(), 2 * 256, None)
        torch.cuda.synchronize()
        assert rc == 0
        assert int(status.cpu()) & B.DEV_BAD_WORD_MAP
        assert bool((out[n_tgt:] == 123.0).all())                  # nothing written past N_tgt
        assert bool((ws[2 * 256:] == 0x5A).all())                   # nothing written past the stated workspace
        assert bool(torch.isfinite(out[:n_tgt]).all()) and float(out[:n_tgt].abs().max()) < 1e3   # guard values unread
