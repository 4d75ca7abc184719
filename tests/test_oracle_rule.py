"""Pins for the oracle's acceptance rule: hand-worked rounds, exhaustive
agreement of the procedural form (Algorithm 1) with the declarative form
(Eq. 6 - Eq. 11) and with a streaming restatement, the limits the paper
states in words, and invariants."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import fly_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
THETA = 1.0
HI, LO = 2.0, 0.25          # entropies on the Defer / Strict side of THETA


def entropies(gates):
    return [HI if g else LO for g in gates]


def streaming_rule(delta, gates, W):
    """Third statement of the rule, as the introduction tells it: walk the
    positions once; a Defer mismatch opens a window of W positions; another
    mismatch inside an open window rejects the token that opened it; a window
    that cannot close inside the round rejects its token too."""
    K = len(delta)
    open_at = None
    for i in range(1, K + 1):
        if open_at is not None and i > open_at + W:
            open_at = None                       # window closed cleanly: kept
        if delta[i - 1] == 0:
            if open_at is not None:
                return open_at
            if not gates[i - 1]:
                return i
            open_at = i
    if open_at is not None and open_at + W > K:
        return open_at
    return K + 1


def read_cases(name):
    for line in open(os.path.join(GOLDEN, name)):
        line = line.split("#")[0].strip()
        if line:
            yield [f.strip() for f in line.split("|")]


def test_hand_worked_rounds():
    n = 0
    for head, dstr, gstr, s in read_cases("rule_cases.txt"):
        K, W = map(int, head.split())
        delta = [int(c) for c in dstr]
        gates = [c == "D" for c in gstr]
        assert len(delta) == K == len(gates)
        H = entropies(gates)
        assert O.s_fly_procedural(delta, H, THETA, W) == int(s), (head, dstr, gstr)
        assert O.s_fly_declarative(delta, H, THETA, W) == int(s), (head, dstr, gstr)
        n += 1
    assert n >= 15


@pytest.mark.parametrize("K", [1, 2, 3, 4, 5, 6])
def test_procedural_equals_declarative_equals_streaming_exhaustively(K):
    for delta in itertools.product((0, 1), repeat=K):
        for gates in itertools.product((False, True), repeat=K):
            H = entropies(gates)
            for W in range(0, K + 2):
                a = O.s_fly_procedural(delta, H, THETA, W)
                b = O.s_fly_declarative(delta, H, THETA, W)
                c = streaming_rule(delta, gates, W)
                assert a == b == c, (delta, gates, W, a, b, c)
                assert 1 <= a <= K + 1


def test_gate_is_strict_below_and_defer_at_or_above_theta():
    # Eq. 6: h < theta Strict, h >= theta Defer (equality defers)
    assert O.gate(0.999, 1.0) == "Strict"
    assert O.gate(1.0, 1.0) == "Defer"
    assert O.gate(1.001, 1.0) == "Defer"
    delta = [1, 0, 1, 1, 1]
    assert O.s_fly_procedural(delta, [9, 1.0, 9, 9, 9], 1.0, 2) == 6
    assert O.s_fly_procedural(delta, [9, 0.9999, 9, 9, 9], 1.0, 2) == 2


@pytest.mark.parametrize("K", [1, 3, 5, 8])
def test_infinite_threshold_is_standard_speculative_decoding(K):
    # the ablation text: at the top of the theta range every mismatch is
    # rejected and the method degenerates to exact-match acceptance (Eq. 3)
    rng = np.random.default_rng(K)
    for delta in itertools.product((0, 1), repeat=K):
        H = list(rng.uniform(0, 12, size=K))
        for W in (0, 1, 3, K):
            assert O.s_fly_procedural(delta, H, math.inf, W) == O.s_standard(delta)
            assert O.s_fly_declarative(delta, H, math.inf, W) == O.s_standard(delta)
    assert O.s_standard([1] * K) == K + 1
    assert O.s_standard([1] * (K - 1) + [0]) == K
    assert O.s_standard([0] + [1] * (K - 1)) == 1


@pytest.mark.parametrize("K", [1, 2, 4, 7])
def test_no_window_and_no_gate_accepts_everything(K):
    # W = 0: every deferred mismatch is accepted; theta = 0: every mismatch defers
    for delta in itertools.product((0, 1), repeat=K):
        H = [0.0] * K
        assert O.s_fly_procedural(delta, H, 0.0, 0) == K + 1
        assert O.s_fly_declarative(delta, H, -1.0, 0) == K + 1


def test_invariants_over_random_rounds():
    rng = np.random.default_rng(0)
    for _ in range(3000):
        K = int(rng.integers(1, 20))
        delta = list((rng.random(K) < 0.75).astype(int))
        H = list(rng.uniform(0, 3, size=K))
        W = int(rng.integers(0, 8))
        th = float(rng.uniform(0, 3))
        s = O.s_fly_procedural(delta, H, th, W)
        assert s >= O.s_standard(delta)                      # never worse than exact match
        assert s <= O.s_fly_procedural(delta, H, th, max(W - 1, 0))   # longer window: no more accepted
        assert s <= O.s_fly_procedural(delta, H, th * 0.5, W)         # lower threshold: no fewer
        if s <= K:
            assert delta[s - 1] == 0                         # a round is only ever cut at a mismatch
        # a mismatch in the last W positions is never kept (boundary sentence)
        for j in range(max(K - W + 1, 1), K + 1):
            if delta[j - 1] == 0:
                assert s <= j


def test_emission():
    draft = [10, 11, 12, 13]
    y = [10, 21, 12, 23, 99]
    assert O.emit_tokens(draft, y, 5) == [10, 11, 12, 13, 99]      # accept all: drafts + bonus
    assert O.emit_tokens(draft, y, 2) == [10, 21, -1, -1, -1]      # cut at 2: draft 1, target 2
    assert O.emit_tokens(draft, y, 1) == [10, -1, -1, -1, -1]
    assert O.emit_tokens(draft, y, 4) == [10, 11, 12, 23, -1]      # accepted mismatch 2 keeps the DRAFT token
    assert O.match_indicator(draft, y[:4]) == [1, 0, 1, 0]


def test_verify_batch_end_to_end_tiny():
    # V = 4.  Row peaked on token t: logit 9 there, 0 elsewhere (H ~ 0.005 nats);
    # flat row with a slight preference: H ~ log 4.
    def peaked(t):
        r = [0.0] * 4; r[t] = 9.0; return r

    def flat(t):
        r = [0.0] * 4; r[t] = 0.1; return r

    K, W = 4, 1
    logits = np.array([
        # seq 0: flat mismatch at 1 then clean -> kept; accept all
        [flat(2), peaked(1), peaked(3), peaked(0), peaked(2)],
        # seq 1: peaked mismatch at 2 -> Strict reject there
        [peaked(0), peaked(1), peaked(3), peaked(0), peaked(2)],
        # seq 2: flat mismatch at 4 -> 4+1 > 4, boundary reject
        [peaked(0), peaked(1), peaked(3), flat(0), peaked(2)],
    ])
    draft = np.array([[1, 1, 3, 0], [0, 2, 3, 0], [0, 1, 3, 3]])
    r = O.verify_batch(logits, draft, theta=1.0, W=W)
    assert list(r.accept_len) == [5, 2, 4]
    assert r.out_tokens.tolist() == [[1, 1, 3, 0, 2], [0, 1, -1, -1, -1], [0, 1, 3, 0, -1]]
    assert r.target_argmax.tolist() == [[2, 1, 3, 0, 2], [0, 1, 3, 0, 2], [0, 1, 3, 0, 2]]
    assert (r.rollback == 0).all() and (r.state_out == [0, 0, -1]).all()
    # same call with the paper's normalised threshold on h = H / log V
    r2 = O.verify_batch(logits, draft, theta=1.0 / math.log(4), W=W, theta_unit="normalized")
    assert list(r2.accept_len) == [5, 2, 4]
    # out-of-vocabulary draft id: a mismatch, flagged
    bad = draft.copy(); bad[1, 0] = 4
    r3 = O.verify_batch(logits, bad, theta=1.0, W=W)
    assert r3.accept_len[1] == 1 and r3.row_flags[1, 0] == O.FLAG_BAD_DRAFT


def test_caller_supplied_target_tokens_replace_the_argmax_in_eq2_and_in_the_output():
    # extension outside the paper's text (which defines y_i as the argmax only)
    import numpy as np
    from oracle import fly_oracle as O
    rng = np.random.default_rng(0)
    B, K, V = 3, 5, 11
    logits = rng.normal(size=(B, K + 1, V)) * 3
    y = logits.argmax(axis=2)
    draft = y[:, :K].copy()
    draft[0, 2] = (draft[0, 2] + 1) % V                    # one mismatch against the argmax
    base = O.verify_batch(logits, draft, theta=1e9, W=2)    # exact-match acceptance
    same = O.verify_batch(logits, draft, theta=1e9, W=2, target_tokens=y)
    assert np.array_equal(base.accept_len, same.accept_len) and np.array_equal(base.out_tokens, same.out_tokens)
    assert base.accept_len[0] == 3
    tt = y.copy()
    tt[0, 2] = draft[0, 2]                                 # the caller's sample agrees with the draft there ...
    tt[1, 0] = (y[1, 0] + 3) % V                           # ... and disagrees with a draft that matched the argmax
    tt[2, K] = V + 4                                       # bonus token out of range
    got = O.verify_batch(logits, draft, theta=1e9, W=2, target_tokens=tt)
    assert got.accept_len.tolist() == [K + 1, 1, K + 1]
    assert got.out_tokens[1, 0] == tt[1, 0] and got.out_tokens[0, K] == y[0, K]
    assert got.row_flags[2, K] == O.FLAG_BAD_TARGET and got.out_tokens[2, K] == 0
    assert np.array_equal(got.target_argmax, y)            # the argmax is still reported as such


# ---------------------------------------------------------------------------
# Invalid input.  The paper does not treat it; the reading (a flagged position is a mismatch that the
# gate never defers, so an invalid or placeholder token id can never be kept or emitted as a draft)
# protects Eq. 2 and Eq. 6.  Every expected value below is written out by hand.  All rows are flat
# unless stated (four equal logits: H = ln 4 = 1.386 nats, Defer at every threshold used; the argmax
# of a flat row is token 0, the lowest index).
# ---------------------------------------------------------------------------

def _flat_rows(B, K1, V=4):
    return np.zeros((B, K1, V))


def test_nonfinite_row_cuts_the_round_even_when_its_placeholder_token_equals_the_draft():
    # K = 3, theta = 0, W = 0: every valid mismatch would be deferred and accepted (no window to check).
    # Position 2 holds a NaN: its row has no defined argmax, the reported token is the placeholder 0.
    # The draft at position 2 is 0 as well - if the placeholder were compared like a real token the
    # position would "match" and all four tokens would be appended.  It must cut at 2 instead.
    x = _flat_rows(1, 4)
    x[0, 1, 2] = np.nan
    draft = np.array([[0, 0, 0]])
    r = O.verify_batch(x, draft, theta=0.0, W=0)
    assert r.row_flags.tolist() == [[0, O.FLAG_NONFINITE, 0, 0]]
    assert r.accept_len.tolist() == [2]
    assert r.out_tokens.tolist() == [[0, 0, -1, -1]]          # draft 1, then the placeholder at the cut
    assert r.target_argmax[0, 1] == 0 and r.entropy[0, 1] == 0.0
    # the same with +inf in the row, and with a row that has no finite entry at all
    for bad_row in ([0.0, np.inf, 0.0, 0.0], [-np.inf] * 4):
        x2 = _flat_rows(1, 4)
        x2[0, 1] = bad_row
        r2 = O.verify_batch(x2, draft, theta=0.0, W=0)
        assert r2.row_flags.tolist() == [[0, O.FLAG_NONFINITE, 0, 0]]
        assert r2.accept_len.tolist() == [2] and r2.out_tokens.tolist() == [[0, 0, -1, -1]]
    # a partly masked row is NOT invalid: two entries left, H = ln 2, argmax = first finite maximum
    x3 = _flat_rows(1, 4)
    x3[0, 1] = [-np.inf, 0.0, -np.inf, 0.0]
    r3 = O.verify_batch(x3, np.array([[0, 1, 0]]), theta=0.0, W=0)
    assert r3.row_flags.tolist() == [[0, 0, 0, 0]] and r3.accept_len.tolist() == [4]
    assert r3.target_argmax[0, 1] == 1 and abs(r3.entropy[0, 1] - math.log(2)) < 1e-12


def test_out_of_range_draft_on_a_defer_row_with_a_clean_window_is_cut_not_kept():
    # K = 4, W = 2, theta = 0.5 nats.  Position 2 proposes token 7 (V = 4): a mismatch on a flat (Defer) row
    # whose window 3..4 is clean and fits (2 + 2 <= 4).  For a valid id Eq. 9 says Accept and the DRAFT token
    # would be appended - here that would put id 7 into the text.  The reading cuts at 2 and emits y_2 = 0.
    x = _flat_rows(2, 5)
    draft = np.array([[0, 7, 0, 0],       # invalid id
                      [0, 3, 0, 0]])      # control: a valid mismatch in the same place IS kept (accept all)
    r = O.verify_batch(x, draft, theta=0.5, W=2)
    assert r.row_flags.tolist() == [[0, O.FLAG_BAD_DRAFT, 0, 0, 0], [0, 0, 0, 0, 0]]
    assert r.accept_len.tolist() == [2, 5]
    assert r.out_tokens.tolist() == [[0, 0, -1, -1, -1], [0, 3, 0, 0, 0]]
    # a negative id is out of range too
    r2 = O.verify_batch(x[:1], np.array([[0, 0, -1, 0]]), theta=0.5, W=0)
    assert r2.row_flags.tolist() == [[0, 0, O.FLAG_BAD_DRAFT, 0, 0]]
    assert r2.accept_len.tolist() == [3] and r2.out_tokens.tolist() == [[0, 0, 0, -1, -1]]


def test_out_of_range_caller_token_is_never_accepted_even_when_the_placeholder_equals_the_draft():
    # Caller-supplied target tokens (extension).  Position 2's token is 9 (V = 4): flagged, replaced by the
    # placeholder 0 - which equals the draft there.  theta = 0, W = 0 would accept any valid mismatch.
    x = _flat_rows(1, 4)
    tt = np.array([[0, 9, 0, 0]])
    r = O.verify_batch(x, np.array([[0, 0, 0]]), theta=0.0, W=0, target_tokens=tt)
    assert r.row_flags.tolist() == [[0, O.FLAG_BAD_TARGET, 0, 0]]
    assert r.accept_len.tolist() == [2] and r.out_tokens.tolist() == [[0, 0, -1, -1]]
    # an invalid BONUS token (position K+1) takes no part in Eq. 2: the round is accepted, the placeholder is emitted
    r2 = O.verify_batch(x, np.array([[0, 0, 0]]), theta=0.0, W=0, target_tokens=np.array([[0, 0, 0, -5]]))
    assert r2.row_flags.tolist() == [[0, 0, 0, O.FLAG_BAD_TARGET]]
    assert r2.accept_len.tolist() == [4] and r2.out_tokens.tolist() == [[0, 0, 0, 0]]
    # a non-finite row ignores what the caller drew for it (flag 1 only)
    x3 = _flat_rows(1, 4)
    x3[0, 0, 0] = np.nan
    r3 = O.verify_batch(x3, np.array([[2, 0, 0]]), theta=0.0, W=0, target_tokens=np.array([[2, 0, 0, 0]]))
    assert r3.row_flags.tolist() == [[O.FLAG_NONFINITE, 0, 0, 0]]
    assert r3.accept_len.tolist() == [1] and r3.out_tokens.tolist() == [[0, -1, -1, -1]]


def test_flagged_position_inside_a_carried_window_revokes_it():
    # Carry extension: one window slot is still open (pending = 1, rollback_len = 3, correction = 2).  Position 1
    # of this round holds a NaN and the draft there equals the placeholder 0: it must count as the mismatch that
    # revokes the carried deferral (s = 1, rollback 3, the correction token), not as a match.
    x = _flat_rows(1, 4)
    x[0, 0, 3] = np.nan
    r = O.verify_batch(x, np.array([[0, 0, 0]]), theta=0.0, W=1, boundary="carry", state_in=np.array([[1, 3, 2]]))
    assert r.accept_len.tolist() == [1] and r.rollback.tolist() == [3]
    assert r.out_tokens.tolist() == [[2, -1, -1, -1]] and r.state_out.tolist() == [[0, 0, -1]]


def test_verify_batch_against_an_independent_composition_on_random_tiny_batches():
    # End to end pin of verify_batch's plumbing (which row meets which draft, the bonus row, the threshold unit, the
    # emitted tokens): the expected values come from a different route - the exactly rounded pure-Python row
    # statistics (row_stats_loops) and the streaming restatement of the rule above, neither of which verify_batch uses.
    rng = np.random.default_rng(2511)
    for case in range(300):
        B, K, V = int(rng.integers(1, 4)), int(rng.integers(1, 7)), int(rng.integers(2, 7))
        W = int(rng.integers(0, K + 2))
        unit = "nats" if case % 2 == 0 else "normalized"
        theta = float(rng.uniform(0.05, 1.2)) if unit == "nats" else float(rng.uniform(0.05, 0.95))
        logits = np.round(rng.normal(size=(B, K + 1, V)) * 2.5, 2)            # distinct enough: no accidental ties
        draft = rng.integers(0, V, size=(B, K))
        th_nats = theta if unit == "nats" else theta * math.log(V)
        want_s, want_toks = [], []
        skip = False
        for b in range(B):
            stats = [O.row_stats_loops(list(logits[b, i])) for i in range(K + 1)]
            H = [h for h, _ in stats]
            y = [t for _, t in stats]
            if any(abs(h - th_nats) < 1e-9 for h in H):
                skip = True
            delta = [1 if int(draft[b, i]) == y[i] else 0 for i in range(K)]
            gates = [H[i] >= th_nats for i in range(K)]
            s = streaming_rule(delta, gates, W)
            want_s.append(s)
            want_toks.append([int(t) for t in draft[b, :s - 1]] + [y[s - 1]] + [-1] * (K + 1 - s))
        if skip:
            continue
        got = O.verify_batch(logits, draft, theta, W, theta_unit=unit)
        assert got.accept_len.tolist() == want_s, (case, B, K, V, W)
        assert got.out_tokens.tolist() == want_toks, (case, B, K, V, W)
        assert (got.row_flags == 0).all() and (got.rollback == 0).all()
