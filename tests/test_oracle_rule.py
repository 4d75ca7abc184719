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
