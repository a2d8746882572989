"""WordSpans (App. D, Alg. 2): the oracle's regular-expression definition pinned on hand-worked texts, and the
package's scanning helper compared with it."""
import random

from oracle import mrl_oracle as O
from paper_2605_07244_b200 import thl_words


def test_oracle_on_the_caption_sentence_of_the_word_alignment_figure():
    # the sentence the paper's word-alignment figure uses; intervals counted by hand
    text = "Thinking small is a self-fulfilling prophecy"
    want = [(0, 8), (9, 14), (15, 17), (18, 19), (20, 35), (36, 44)]
    assert O.thl_word_spans(text) == want
    assert [text[s:e] for s, e in want] == text.split()


def test_oracle_hand_cases():
    assert O.thl_word_spans("") == []
    assert O.thl_word_spans(" \t\n ") == []
    assert O.thl_word_spans("a") == [(0, 1)]
    assert O.thl_word_spans("  ab   c ") == [(2, 4), (7, 8)]          # leading / repeated / trailing delimiters
    assert O.thl_word_spans("x\ny\tz") == [(0, 1), (2, 3), (4, 5)]
    # indices count characters, not UTF-8 bytes; a no-break space and an ideographic space delimit too
    assert O.thl_word_spans("é ü ß　道") == [(0, 1), (2, 3), (4, 5), (6, 7)]


def test_spans_are_maximal_disjoint_and_cover_every_non_space_character():
    rng = random.Random(3)
    alphabet = "ab,.é道 \t\n  "
    for _ in range(300):
        text = "".join(rng.choice(alphabet) for _ in range(rng.randrange(0, 40)))
        spans = O.thl_word_spans(text)
        covered = set()
        prev_end = -1
        for s, e in spans:
            assert 0 <= s < e <= len(text) and s > prev_end          # ordered, separated by at least one delimiter
            assert not any(c.isspace() for c in text[s:e])
            assert s == 0 or text[s - 1].isspace()                    # maximal on both sides
            assert e == len(text) or text[e].isspace()
            covered.update(range(s, e))
            prev_end = e
        assert covered == {i for i, c in enumerate(text) if not c.isspace()}


def test_package_helper_matches_the_oracle():
    rng = random.Random(11)
    alphabet = "abcXYZ09-_'é道😀 \t\n\r  　"
    cases = ["", " ", "word", " lead", "trail ", "Thinking small is a self-fulfilling prophecy"]
    cases += ["".join(rng.choice(alphabet) for _ in range(rng.randrange(0, 80))) for _ in range(500)]
    for text in cases:
        assert thl_words.word_spans(text) == O.thl_word_spans(text), repr(text)
        cw = thl_words.char_to_word(text)
        assert len(cw) == len(text)
        for k, (s, e) in enumerate(O.thl_word_spans(text)):
            assert cw[s:e] == [k] * (e - s)
        assert all((w == -1) == c.isspace() for w, c in zip(cw, text))
