"""Pins of the prompt-lookup oracle: hand-worked cases, and an independent search that uses the standard
library's bytes.find on fixed-width token encodings."""
import os
import random

from oracle.pld_oracle import pld_draft

HERE = os.path.dirname(os.path.abspath(__file__))


def golden_cases():
    for line in open(os.path.join(HERE, "golden", "pld_cases.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        toks, params, prop, pos, n = [f.strip() for f in line.split("|")]
        K, mx, mn = [int(x) for x in params.split()]
        yield ([int(x) for x in toks.split()], K, mx, mn, [] if prop == "-" else [int(x) for x in prop.split()],
               int(pos), int(n))


def test_hand_worked_cases():
    cases = list(golden_cases())
    assert len(cases) >= 10
    for toks, K, mx, mn, prop, pos, n in cases:
        assert pld_draft(toks, K, mx, mn) == (prop, pos, n), toks


def find_with_bytes(tokens, K, mx, mn):
    """Independent formulation: tokens as 4-byte records, library substring search, aligned hits only."""
    enc = b"".join(int(t).to_bytes(4, "little") for t in tokens)
    L = len(tokens)
    for n in range(mx, mn - 1, -1):
        if n >= L:
            continue
        query = enc[4 * (L - n):]
        at = -1
        while True:
            at = enc.find(query, at + 1, 4 * (L - 1))        # hits must end before the last token
            if at < 0 or at % 4 == 0:
                break
        if at >= 0:
            p = at // 4
            return list(tokens[p + n:min(p + n + K, L)]), p, n
    return [], -1, 0


def test_against_library_substring_search():
    rng = random.Random(0)
    for trial in range(3000):
        L = rng.randint(1, 40)
        alphabet = rng.choice([2, 3, 5, 50, 70000])
        toks = [rng.randrange(alphabet) for _ in range(L)]
        K, mx = rng.randint(1, 12), rng.randint(1, 8)
        mn = rng.randint(1, mx)
        assert pld_draft(toks, K, mx, mn) == find_with_bytes(toks, K, mx, mn), (toks, K, mx, mn)


def test_properties():
    rng = random.Random(1)
    for trial in range(500):
        toks = [rng.randrange(4) for _ in range(rng.randint(2, 30))]
        prop, p, n = pld_draft(toks, 6, 4, 1)
        if p >= 0:
            assert toks[p:p + n] == toks[len(toks) - n:] and 1 <= len(prop) <= 6
            assert prop == toks[p + n:p + n + len(prop)]
            # no larger n-gram (up to 4) has any earlier copy
            for m in range(n + 1, 5):
                assert m >= len(toks) or all(toks[c:c + m] != toks[len(toks) - m:] for c in range(len(toks) - m))
        else:
            assert prop == [] and toks[-1] not in toks[:-1]
