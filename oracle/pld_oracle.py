"""CPU oracle for prompt-lookup drafting. TEST INFRASTRUCTURE ONLY.

Section 2.3 of the paper (multi-level acceleration) speeds up the drafter with prompt lookup
decoding, which it describes only as a simple n-gram retrieval; the rule below is the cited
method's, stated plainly: the last n tokens of the sequence are the query; among the earlier
positions where the same n tokens occur, the EARLIEST one wins; the tokens that followed it
are proposed, at most K of them and never past the end of the sequence.  n is tried from
max_ngram down to min_ngram and the first n with a match is used.

Pure Python loops over plain lists; shares nothing with the CUDA path.

Pins (tests/test_oracle_pld.py): hand-worked cases in tests/golden/pld_cases.txt, and an
independent search with the standard library's bytes.find on fixed-width encodings.
"""
from typing import List, Sequence, Tuple


def pld_draft(tokens: Sequence[int], K: int, max_ngram: int = 3, min_ngram: int = 1) -> Tuple[List[int], int, int]:
    """Returns (proposed tokens, match position p or -1, n-gram size used or 0)."""
    L = len(tokens)
    for n in range(max_ngram, min_ngram - 1, -1):
        if n >= L:
            continue                                  # no room for an earlier copy plus a continuation
        query = list(tokens[L - n:])
        for p in range(0, L - n):                     # ascending: the first hit is the earliest
            if list(tokens[p:p + n]) == query:
                start = p + n                         # <= L - 1: at least one token follows
                return list(tokens[start:min(start + K, L)]), p, n
    return [], -1, 0
