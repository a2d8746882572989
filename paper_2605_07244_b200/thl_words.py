"""Host-side text helper of the THL word alignment: WordSpans (App. D, Alg. 2).

The word-alignment kernel (mrl_thl_word_align_logprobs) works on integer token-to-word maps; the words
themselves come from the response text.  WordSpans fixes that coordinate system: the maximal runs of
non-whitespace characters of the text, as (start, end) character intervals with an exclusive end, in text
order.  The intervals depend on the text alone, not on any tokenizer.  This is plain host code (a single
scan over the characters); no device work is involved.
"""
from __future__ import annotations


def word_spans(text: str) -> list[tuple[int, int]]:
    """Character intervals (start, end), end exclusive, of every maximal non-whitespace run of `text`.

    Whitespace is what `str.isspace` says (Unicode whitespace, the class a regular expression's `\\S`
    excludes).  Indices count characters (code points), not bytes.  An empty or all-whitespace text has
    no spans.
    """
    spans = []
    start = -1
    for i, ch in enumerate(text):
        if ch.isspace():
            if start >= 0:
                spans.append((start, i))
                start = -1
        elif start < 0:
            start = i
    if start >= 0:
        spans.append((start, len(text)))
    return spans


def char_to_word(text: str) -> list[int]:
    """Word index of every character of `text` under word_spans (-1 on whitespace): the lookup a tokenizer's
    character offsets are mapped through when token-to-word maps are built from offsets."""
    out = [-1] * len(text)
    for k, (s, e) in enumerate(word_spans(text)):
        for i in range(s, e):
            out[i] = k
    return out
