"""fp64 CPU oracle for the FLy verification step. TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what the CUDA path has to compute,
written from the paper's equations and from Algorithm 1. It shares no code
with the CUDA path and imports nothing from the product package. Only the
tests, the smoke check and the benchmark's CPU-baseline leg may call it.

Notation follows the paper: K drafted tokens per round, logits l_1..l_{K+1}
(row K+1 is the bonus position), draft tokens yhat_1..yhat_K, target tokens
y_i, match indicator Delta_i, mismatch set J, entropy h_j, gate threshold
theta, window length W, accepted-token count s.

Everything is per sequence and per round; a batch is a plain loop.

Parity pins (tests/test_oracle_*.py): closed-form entropies (uniform, one-hot,
single spike), shift invariance, scipy's softmax/entropy, brute-force
enumeration of every (Delta, gate, W) pattern against the declarative form of
the rule, the theta -> +inf and W = 0 limits stated in the paper's ablation
text, the chunking invariant for the cross-round carry extension, and
hand-built rounds for invalid input (non-finite rows, token ids out of range).
"Parity unpinned": nothing here says anything about real-model behaviour
(tau, accuracy recovery); that needs weights and datasets.
"""
from __future__ import annotations

import math
from typing import NamedTuple, Optional, Sequence

import numpy as np

# ---------------------------------------------------------------------------
# Row statistics: softmax, argmax (Eq. 1) and entropy (Eq. 5)
# ---------------------------------------------------------------------------

FLAG_NONFINITE = 1  # a NaN or +inf logit, or a row with no finite logit
FLAG_BAD_DRAFT = 2  # a draft token id outside [0, V)
FLAG_BAD_TARGET = 4  # a caller-supplied target token outside [0, V)
FLAG_BAD_STATE = 8   # (position 1) carried state that the carry extension never writes: ignored


def row_stats(x: np.ndarray):
    """Entropy in nats, greedy token and flags for every row of `x`.

    `x` is [R, V] float64 holding the logit bits widened exactly (bf16 and
    fp32 both embed in fp64).  Returns (H[R] float64, y[R] int64,
    flags[R] uint32).

    Eq. 1: p(v) = softmax(l)_v and y = argmax_v p(v).  softmax is monotone in
    the logit, so the argmax is taken on the logits; among equal maxima the
    smallest index wins (the paper does not say; this is the reading both
    sides use).
    Eq. 5 numerator: H = -sum_v p(v) log p(v), natural log, with the usual
    convention 0 log 0 = 0 (a -inf logit has p = 0).  Division by log|V|
    (the normalised h of Eq. 5) is done by `normalized_entropy`.
    """
    x = np.asarray(x, dtype=np.float64)
    assert x.ndim == 2
    R, V = x.shape
    H = np.zeros(R, dtype=np.float64)
    y = np.zeros(R, dtype=np.int64)
    flags = np.zeros(R, dtype=np.uint32)
    for r in range(R):
        row = x[r]
        bad = np.isnan(row).any() or np.isposinf(row).any() or not np.isfinite(row).any()
        if bad:
            flags[r] |= FLAG_NONFINITE
            H[r] = 0.0
            y[r] = 0
            continue
        m = row.max()
        y[r] = int(np.argmax(row))  # numpy documents: first occurrence of the maximum
        e = np.exp(row - m)         # exp(-inf) = 0
        S = e.sum()
        p = e / S
        pos = p > 0.0
        H[r] = -(p[pos] * np.log(p[pos])).sum()
    return H, y, flags


def row_stats_loops(row: Sequence[float]):
    """Same as `row_stats` for ONE finite row, in pure Python with exactly
    rounded sums (math.fsum): the brute-force statement used on tiny inputs."""
    V = len(row)
    m = -math.inf
    y = 0
    for v in range(V):
        if row[v] > m:          # strict: the first maximum keeps its index
            m = row[v]
            y = v
    S = math.fsum(math.exp(row[v] - m) for v in range(V))
    terms = []
    for v in range(V):
        p = math.exp(row[v] - m) / S
        if p > 0.0:
            terms.append(p * math.log(p))
    return -math.fsum(terms), y


def normalized_entropy(H_nats: np.ndarray, V: int) -> np.ndarray:
    """Eq. 5: h = H / log|V|, in [0, 1]."""
    return np.asarray(H_nats, dtype=np.float64) / math.log(V)


def theta_in_nats(theta: float, unit: str, V: int) -> float:
    """The gate compares entropies in nats.  unit 'nats': theta is used as
    given.  unit 'normalized': theta is the paper's threshold on h of Eq. 5,
    i.e. theta * log|V| nats (h < theta  <=>  H < theta log|V|)."""
    if unit == "nats":
        return float(theta)
    if unit == "normalized":
        return float(theta) * math.log(V)
    raise ValueError(unit)


# ---------------------------------------------------------------------------
# Match indicator (Eq. 2), standard acceptance (Eq. 3)
# ---------------------------------------------------------------------------

def match_indicator(draft: Sequence[int], y: Sequence[int]):
    """Eq. 2: Delta_i = 1[yhat_i = y_i], 1 <= i <= K (0-based lists here)."""
    K = len(draft)
    return [1 if int(draft[i]) == int(y[i]) else 0 for i in range(K)]


def s_standard(delta: Sequence[int]) -> int:
    """Eq. 3: the first mismatch position (1-based), else K+1."""
    K = len(delta)
    for i in range(1, K + 1):
        if delta[i - 1] == 0:
            return i
    return K + 1


# ---------------------------------------------------------------------------
# The FLy rule, procedural form: Algorithm 1, steps 3 and 4
# ---------------------------------------------------------------------------

def s_fly_procedural(delta: Sequence[int], H: Sequence[float], theta: float, W: int) -> int:
    """Accepted-token count s of one round, following Algorithm 1.

    delta[i-1] = Delta_i and H[i-1] = entropy at position i (same unit as
    theta) for i = 1..K.  s = j when the round is cut at mismatch j (j-1
    drafts kept plus the target's own token y_j), s = K+1 when every draft
    is kept (plus the bonus token).
    """
    K = len(delta)
    J = [j for j in range(1, K + 1) if delta[j - 1] == 0]       # mismatch set
    if not J:                                                    # all matched
        return K + 1
    for j in J:                                                  # ascending
        if H[j - 1] < theta:                                     # Strict: reject
            return j
        # Defer: count mismatches over the next W positions.  Positions past K
        # do not exist; the sum stops at K (they cannot turn a reject into an
        # accept because j + W <= K is required as well).
        M_W = sum(1 - delta[i - 1] for i in range(j + 1, min(j + W, K) + 1))
        if M_W == 0 and j + W <= K:
            continue                                             # benign, keep draft
        return j                                                 # harmful: reject
    return K + 1                                                 # accept all


# ---------------------------------------------------------------------------
# The FLy rule, declarative form: Eq. 6 - Eq. 11 (independent restatement)
# ---------------------------------------------------------------------------

def gate(h_j: float, theta: float) -> str:
    """Eq. 6."""
    return "Strict" if h_j < theta else "Defer"


def s_gate(delta, H, theta) -> int:
    """Eq. 7."""
    K = len(delta)
    strict = [j for j in range(1, K + 1) if delta[j - 1] == 0 and gate(H[j - 1], theta) == "Strict"]
    return min(strict) if strict else K + 1


def N_W(delta, j: int, W: int) -> int:
    """Eq. 8, with Delta_i read as a mismatch-free position for i > K (those
    positions only arise when j + W > K, which Eq. 9 rejects anyway)."""
    K = len(delta)
    return sum(1 - delta[i - 1] for i in range(j + 1, j + W + 1) if i <= K)


def defer_decide(delta, H, theta, W, j: int) -> str:
    """Eq. 9."""
    K = len(delta)
    if H[j - 1] >= theta and N_W(delta, j, W) == 0 and j + W <= K:
        return "Accept"
    return "Reject"


def s_defer(delta, H, theta, W) -> int:
    """Eq. 10."""
    K = len(delta)
    rej = [j for j in range(1, K + 1)
           if delta[j - 1] == 0 and defer_decide(delta, H, theta, W, j) == "Reject"]
    return min(rej) if rej else K + 1


def s_fly_declarative(delta, H, theta, W) -> int:
    """Eq. 11: s_FLy = min(s_gate, s_defer)."""
    return min(s_gate(delta, H, theta), s_defer(delta, H, theta, W))


# ---------------------------------------------------------------------------
# Token emission (Algorithm 1: the three concat lines)
# ---------------------------------------------------------------------------

def emit_tokens(draft: Sequence[int], y: Sequence[int], s: int):
    """Tokens appended this round, padded with -1 to length K+1.

    Cut at j = s <= K: yhat_1..yhat_{j-1}, y_j.  Accept all (s = K+1):
    yhat_1..yhat_K, y_{K+1}.  A mismatch that the window accepted keeps the
    DRAFT token.
    """
    K = len(draft)
    out = [int(t) for t in draft[: s - 1]] + [int(y[s - 1])]
    return out + [-1] * (K + 1 - len(out))


# ---------------------------------------------------------------------------
# One round for one sequence
# ---------------------------------------------------------------------------

class State(NamedTuple):
    """Deferred state carried across rounds (the carry extension only).

    pending      r: how many draft positions of the NEXT round still lie in
                    an open window (0 = nothing pending)
    rollback_len L: tokens appended since and including the provisionally
                    kept mismatch (what a revoke removes)
    correction   c: the target's own token at that mismatch
    """
    pending: int = 0
    rollback_len: int = 0
    correction: int = -1


ZERO_STATE = State(0, 0, -1)


class RoundResult(NamedTuple):
    accept_len: int
    rollback: int
    out_tokens: list
    state_out: State


def verify_round_paper(delta, H, theta, W, draft, y) -> RoundResult:
    """The paper's rule (a window that would cross the round end is rejected
    at once).  No cross-round state exists in this mode."""
    s = s_fly_procedural(delta, H, theta, W)
    return RoundResult(s, 0, emit_tokens(draft, y, s), ZERO_STATE)


def verify_round_carry(delta, H, theta, W, draft, y, state_in: State) -> RoundResult:
    """Carry extension: relaxes ONLY the boundary sentence of the paper (a
    Defer mismatch whose window does not fit in the round).  Requires W <= K.

    1. A window is pending (r > 0) and one of this round's first r positions
       mismatches: the carried deferral is revoked, exactly as a mismatch
       inside a window rejects the deferred token within a round.  The caller
       removes the last L tokens and appends the correction c; nothing else
       of this round is used (its logits were conditioned on revoked text).
    2. Otherwise walk J as in Algorithm 1, except: a Defer mismatch j with
       j + W > K and no further mismatch in j+1..K is kept provisionally;
       every draft and the bonus token are emitted and the state records the
       r = j + W - K window slots still to be checked next round.
    3. Every other outcome leaves the zero state.  The bonus token does not
       consume a window slot.
    """
    K = len(delta)
    if W > K:
        raise ValueError("carry mode requires W <= K")
    r, L, c = state_in
    if r > 0 and any(delta[i - 1] == 0 for i in range(1, r + 1)):
        toks = [int(c)] + [-1] * K
        return RoundResult(1, int(L), toks, ZERO_STATE)
    J = [j for j in range(1, K + 1) if delta[j - 1] == 0]
    for j in J:
        if H[j - 1] < theta:
            return RoundResult(j, 0, emit_tokens(draft, y, j), ZERO_STATE)
        later = sum(1 - delta[i - 1] for i in range(j + 1, min(j + W, K) + 1))
        if later == 0 and j + W <= K:
            continue
        if later == 0 and j + W > K:
            st = State(j + W - K, K - j + 2, int(y[j - 1]))
            return RoundResult(K + 1, 0, emit_tokens(draft, y, K + 1), st)
        return RoundResult(j, 0, emit_tokens(draft, y, j), ZERO_STATE)
    return RoundResult(K + 1, 0, emit_tokens(draft, y, K + 1), ZERO_STATE)


# ---------------------------------------------------------------------------
# Whole verification step over a batch
# ---------------------------------------------------------------------------

class BatchResult(NamedTuple):
    accept_len: np.ndarray      # [B] int32
    rollback: np.ndarray        # [B] int32
    out_tokens: np.ndarray      # [B, K+1] int32
    target_argmax: np.ndarray   # [B, K+1] int32
    entropy: np.ndarray         # [B, K+1] float64, nats
    row_flags: np.ndarray       # [B, K+1] uint32
    state_out: np.ndarray       # [B, 3] int32


def verify_batch(logits: np.ndarray, draft: np.ndarray, theta: float, W: int,
                 theta_unit: str = "nats", boundary: str = "reject",
                 state_in: Optional[np.ndarray] = None,
                 target_tokens: Optional[np.ndarray] = None,
                 temperature: float = 1.0) -> BatchResult:
    """One verification step.  logits [B, K+1, V] float64 (exactly widened
    input bits), draft [B, K] integer.  Entropy is computed for every row
    (the paper needs it only at mismatches; the extra rows change nothing).
    A draft id outside [0, V) counts as a mismatch and is flagged.

    target_tokens [B, K+1] (optional, an extension outside the paper's method text, which defines y_i
    only as the argmax of Eq. 1): tokens the caller drew from the target distributions.  They take the
    place of y_i in Eq. 2 and in the emitted tokens; the gate still uses the entropy of the logits and
    target_argmax still reports the argmax.  An id outside [0, V) is flagged and never accepted.

    temperature T > 0 (an extension for the paper's temperature-1 result columns; its method text is
    greedy): the distribution of Eq. 1 / Eq. 5 is softmax(l / T), i.e. the statistics are those of the
    logits divided by T.  Dividing by a positive number keeps the order, so y_i is unchanged."""
    logits = np.asarray(logits, dtype=np.float64)
    if not (temperature > 0.0):
        raise ValueError("temperature must be positive")
    if temperature != 1.0:
        logits = logits / float(temperature)
    B, K1, V = logits.shape
    K = K1 - 1
    draft = np.asarray(draft).reshape(B, K)
    th = theta_in_nats(theta, theta_unit, V)
    H, y, flags = row_stats(logits.reshape(B * K1, V))
    H = H.reshape(B, K1)
    y = y.reshape(B, K1)
    flags = flags.reshape(B, K1).copy()
    acc = np.zeros(B, dtype=np.int32)
    rb = np.zeros(B, dtype=np.int32)
    toks = np.full((B, K1), -1, dtype=np.int32)
    st_out = np.zeros((B, 3), dtype=np.int32)
    y_used = y.copy()
    if target_tokens is not None:
        tt = np.asarray(target_tokens).reshape(B, K1)
        for b in range(B):
            for i in range(K1):
                if flags[b, i] & FLAG_NONFINITE:
                    continue                      # the row is unusable whatever the caller drew
                if 0 <= int(tt[b, i]) < V:
                    y_used[b, i] = int(tt[b, i])
                else:
                    flags[b, i] |= FLAG_BAD_TARGET
                    y_used[b, i] = 0
    for b in range(B):
        for i in range(K):
            if not (0 <= int(draft[b, i]) < V):
                flags[b, i] |= FLAG_BAD_DRAFT
        delta = match_indicator(draft[b], y_used[b, :K])
        # The paper does not treat invalid input.  Reading used by both sides: a
        # flagged position counts as a mismatch that the gate never defers, so
        # an invalid token id can never be emitted.
        Hg = [(-math.inf if flags[b, i] else H[b, i]) for i in range(K)]
        for i in range(K):
            if flags[b, i]:
                delta[i] = 0
        if boundary == "reject":
            res = verify_round_paper(delta, Hg, th, W, draft[b], y_used[b])
        elif boundary == "carry":
            sin = ZERO_STATE if state_in is None else State(*[int(t) for t in state_in[b]])
            # The extension only ever writes 0 <= pending <= W <= K, rollback_len >= 0 and, with a window
            # pending, a correction token inside the vocabulary.  Any other state is not the extension's:
            # it is flagged on position 1 and the round is verified from the zero state.
            if sin.pending < 0 or sin.pending > K or sin.rollback_len < 0 or \
                    (sin.pending > 0 and not (0 <= sin.correction < V)):
                flags[b, 0] |= FLAG_BAD_STATE
                sin = ZERO_STATE
            res = verify_round_carry(delta, Hg, th, W, draft[b], y_used[b], sin)
        else:
            raise ValueError(boundary)
        acc[b] = res.accept_len
        rb[b] = res.rollback
        toks[b] = res.out_tokens
        st_out[b] = list(res.state_out)
    return BatchResult(acc, rb, toks, y.astype(np.int32), H, flags, st_out)


# ---------------------------------------------------------------------------
# Fused LM-head variant: the logits are the last linear layer of the target
# forward pass, hidden @ weight, taken exactly (fp64 product of the inputs).
# ---------------------------------------------------------------------------

def lm_head_logits(hidden: np.ndarray, weight: np.ndarray) -> np.ndarray:
    """hidden [R, D] and weight [D, V], both float64 holding exactly widened
    bf16 values.  Returns the fp64 logits [R, V]."""
    return np.asarray(hidden, dtype=np.float64) @ np.asarray(weight, dtype=np.float64)
