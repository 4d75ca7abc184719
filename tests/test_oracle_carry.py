"""Pins for the cross-round carry extension: chaining R rounds of K drafts in
carry mode must commit exactly the drafts that the paper's rule commits on
the unsplit pattern of R*K drafts (chunking invariant)."""
import itertools
import os

import numpy as np
import pytest

from oracle import fly_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
THETA, HI, LO = 1.0, 2.0, 0.25


def chain(deltas, gates, K, W):
    """Run the rounds in carry mode; stop at the first round that is not
    accept-all.  Returns committed draft count D and the emitted token log."""
    state = O.ZERO_STATE
    D = 0
    log = []
    R = len(deltas) // K
    for t in range(R):
        d = list(deltas[t * K:(t + 1) * K])
        g = gates[t * K:(t + 1) * K]
        H = [HI if x else LO for x in g]
        draft = [1000 * t + i for i in range(1, K + 1)]
        y = [draft[i] if d[i] else -draft[i] - 7 for i in range(K)] + [1000 * t + 999]
        res = O.verify_round_carry(d, H, THETA, W, draft, y, state)
        if res.rollback > 0:
            assert res.accept_len == 1 and res.state_out == O.ZERO_STATE
            assert res.rollback == state.rollback_len
            assert res.out_tokens == [state.correction] + [-1] * K
            del log[len(log) - res.rollback:]
            log.append(res.out_tokens[0])
            D -= res.rollback - 1
            return D, log, O.ZERO_STATE
        log.extend(res.out_tokens[: res.accept_len])
        D += res.accept_len - 1
        state = res.state_out
        if res.accept_len != K + 1:
            assert state == O.ZERO_STATE
            return D, log, state
    if state.pending > 0:
        D -= state.rollback_len - 1
    return D, log, state


def test_hand_worked_chains():
    n = 0
    for line in open(os.path.join(GOLDEN, "carry_cases.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        head, dstr, want = [f.strip() for f in line.split("|")]
        K, R, W = map(int, head.split())
        deltas = [int(c) for c in dstr.replace("/", "")]
        assert len(deltas) == K * R
        D, _, _ = chain(deltas, [True] * (K * R), K, W)
        assert D == int(want), line
        n += 1
    assert n == 4


@pytest.mark.parametrize("K,R", [(1, 2), (2, 2), (2, 3), (3, 2), (3, 3), (4, 2), (4, 3)])
def test_chunking_invariant_exhaustive(K, R):
    n = K * R
    rng = np.random.default_rng(K * 10 + R)
    for deltas in itertools.product((0, 1), repeat=n):
        # all-Defer plus two random gate patterns per Delta pattern
        gate_sets = [[True] * n] + [list(rng.random(n) < 0.6) for _ in range(2)]
        for gates in gate_sets:
            for W in range(0, K + 1):
                D, log, _ = chain(deltas, gates, K, W)
                H = [HI if g else LO for g in gates]
                s_unsplit = O.s_fly_procedural(list(deltas), H, THETA, W)
                assert D == s_unsplit - 1, (deltas, gates, W, D, s_unsplit)


def test_carry_equals_paper_mode_without_boundary_events():
    rng = np.random.default_rng(0)
    for _ in range(2000):
        K = int(rng.integers(1, 12))
        W = int(rng.integers(0, K + 1))
        d = list((rng.random(K) < 0.8).astype(int))
        H = list(rng.uniform(0, 2, size=K))
        draft = list(range(1, K + 1))
        y = [draft[i] if d[i] else 50 + i for i in range(K)] + [99]
        a = O.verify_round_paper(d, H, THETA, W, draft, y)
        b = O.verify_round_carry(d, H, THETA, W, draft, y, O.ZERO_STATE)
        if b.state_out == O.ZERO_STATE:
            assert a == b
        else:
            # carry differs only by keeping a tail mismatch provisionally
            assert b.accept_len == K + 1 and a.accept_len <= K
            j = a.accept_len
            assert b.state_out == O.State(j + W - K, K - j + 2, y[j - 1])
            assert d[j - 1] == 0 and all(d[j:]) and j + W > K


def test_pending_state_fields_and_revoke():
    K, W = 4, 3
    draft = [1, 2, 3, 4]
    y = [1, 2, 30, 4, 5]
    H = [HI] * K
    r1 = O.verify_round_carry([1, 1, 0, 1], H, THETA, W, draft, y, O.ZERO_STATE)
    # j = 3: 3+3 = 6 > 4, position 4 clean: kept provisionally; r = 2 slots remain,
    # L = drafts 3,4 + bonus = 3 tokens, correction = y_3
    assert r1.accept_len == 5 and r1.out_tokens == [1, 2, 3, 4, 5]
    assert r1.state_out == O.State(2, 3, 30)
    # next round: mismatch at position 2 (inside the r = 2 carried slots): revoke
    r2 = O.verify_round_carry([1, 0, 1, 1], H, THETA, W, draft, y, r1.state_out)
    assert (r2.accept_len, r2.rollback, r2.out_tokens) == (1, 3, [30, -1, -1, -1, -1])
    # mismatch at position 3 (outside): the carried token is confirmed, the new one judged alone
    r3 = O.verify_round_carry([1, 1, 0, 1], H, THETA, W, draft, y, r1.state_out)
    assert r3.rollback == 0 and r3.accept_len == 5 and r3.state_out == O.State(2, 3, 30)
    r4 = O.verify_round_carry([1, 1, 0, 1], [HI, HI, LO, HI], THETA, W, draft, y, r1.state_out)
    assert r4.rollback == 0 and r4.accept_len == 3 and r4.state_out == O.ZERO_STATE
    with pytest.raises(ValueError):
        O.verify_round_carry([1] * 4, H, THETA, 5, draft, y, O.ZERO_STATE)


def test_verify_batch_carry_chain_shapes():
    # two sequences, two rounds, V = 3; every row flat enough to Defer
    def flat(t):
        r = [0.0, 0.0, 0.0]; r[t] = 0.05; return r

    K, W = 2, 1
    lg = np.array([[flat(0), flat(1), flat(2)], [flat(0), flat(1), flat(2)]])
    d1 = np.array([[0, 2], [0, 1]])            # seq 0: mismatch at 2 -> pending
    r = O.verify_batch(lg, d1, 1.0, W, boundary="carry")
    assert r.accept_len.tolist() == [3, 3]
    assert r.state_out.tolist() == [[1, 2, 1], [0, 0, -1]]
    d2 = np.array([[1, 1], [0, 1]])            # seq 0: mismatch at 1 -> revoke
    r2 = O.verify_batch(lg, d2, 1.0, W, boundary="carry", state_in=r.state_out)
    assert r2.accept_len.tolist() == [1, 3] and r2.rollback.tolist() == [2, 0]
    assert r2.out_tokens.tolist() == [[1, -1, -1], [0, 1, 2]]


def test_a_state_the_extension_never_writes_is_flagged_and_ignored():
    # V = 4, K = 3, flat rows (Defer everywhere, argmax 0), drafts all 0: an accept-all round from the zero state.
    # A carried state is only honoured if it is one the extension can have written: 0 <= pending <= K,
    # rollback_len >= 0, and a correction inside the vocabulary while a window is pending.
    x = np.zeros((1, 4, 4))
    d = np.array([[0, 0, 0]])
    for bad in ([4, 2, 1], [-1, 2, 1], [1, -3, 1], [2, 2, 9], [1, 2, -1]):
        r = O.verify_batch(x, d, theta=0.0, W=1, boundary="carry", state_in=np.array([bad]))
        assert r.row_flags.tolist() == [[O.FLAG_BAD_STATE, 0, 0, 0]], bad
        assert r.accept_len.tolist() == [4] and r.rollback.tolist() == [0] and r.out_tokens.tolist() == [[0, 0, 0, 0]]
        assert r.state_out.tolist() == [[0, 0, -1]]
    # a legal pending state is used: position 1 mismatches (draft 2 against argmax 0) and revokes it
    r = O.verify_batch(x, np.array([[2, 0, 0]]), theta=0.0, W=1, boundary="carry", state_in=np.array([[1, 2, 3]]))
    assert r.row_flags.tolist() == [[0, 0, 0, 0]] and r.accept_len.tolist() == [1] and r.rollback.tolist() == [2]
    assert r.out_tokens.tolist() == [[3, -1, -1, -1]]
    # with nothing pending the correction field is not looked at (the zero state carries -1 there)
    r = O.verify_batch(x, d, theta=0.0, W=1, boundary="carry", state_in=np.array([[0, 0, -1]]))
    assert r.row_flags.tolist() == [[0, 0, 0, 0]]
