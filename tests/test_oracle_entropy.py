"""Pins for the oracle's row statistics (Eq. 1 argmax, Eq. 5 entropy) against
closed forms, invariants, brute force and library routines - never against
the oracle's own formula."""
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats
import torch

from oracle import fly_oracle as O


def H_of(row):
    H, y, f = O.row_stats(np.asarray(row, dtype=np.float64)[None, :])
    assert f[0] == 0
    return H[0], int(y[0])


@pytest.mark.parametrize("V", [1, 2, 7, 33, 257, 32000, 128256])
def test_uniform_row_has_entropy_log_V(V):
    # every p = 1/V  =>  H = log V, normalised h = 1 (upper end of Eq. 5's range)
    for c in (0.0, -3.5, 88.0):
        H, y = H_of(np.full(V, c))
        assert H == pytest.approx(math.log(V), abs=1e-12)
        assert y == 0                      # all tied: the lowest index wins
    if V > 1:
        assert O.normalized_entropy(np.array([H]), V)[0] == pytest.approx(1.0, abs=1e-13)


@pytest.mark.parametrize("V", [2, 33, 128256])
def test_one_hot_row_has_zero_entropy(V):
    row = np.full(V, -np.inf)
    row[V // 3] = 1.25
    H, y = H_of(row)
    assert H == 0.0 and y == V // 3
    # a spike so tall that every other p underflows behaves the same
    row = np.zeros(V)
    row[V - 1] = 800.0
    H, y = H_of(row)
    assert H == pytest.approx(0.0, abs=1e-300) and y == V - 1


@pytest.mark.parametrize("V,a", [(32000, 12.0), (128256, 8.0), (128256, 16.0), (152064, 11.3), (5, -2.0)])
def test_single_spike_closed_form(V, a):
    # one logit a, V-1 logits 0:  Z = e^a + V - 1,
    # H = log Z - a e^a / Z   (textbook: H = log Z - E[l])
    Z = math.exp(a) + V - 1
    want = math.log(Z) - a * math.exp(a) / Z
    row = np.zeros(V)
    row[17 % V] = a
    H, y = H_of(row)
    assert H == pytest.approx(want, rel=1e-12)
    assert y == (17 % V if a > 0 else 0)


def test_two_outcome_row_is_binary_entropy():
    for a in (-30.0, -1.0, 0.0, 0.3, 5.0, 40.0):
        p = 1.0 / (1.0 + math.exp(-a))
        want = 0.0
        for q in (p, 1 - p):
            if q > 0:
                want -= q * math.log(q)
        H, y = H_of([a, 0.0])
        assert H == pytest.approx(want, abs=1e-14)
        assert y == (0 if a >= 0 else 1)


def test_shift_invariance_and_scale_sensitivity():
    rng = np.random.default_rng(1)
    row = rng.normal(size=4097) * 3
    H0, y0 = H_of(row)
    for c in (-1000.0, 7.25, 1e4):
        H, y = H_of(row + c)
        assert H == pytest.approx(H0, abs=1e-9) and y == y0
    # sharpening the distribution lowers the entropy (catches a sign slip in the exponent)
    assert H_of(2 * row)[0] < H0 < H_of(0.5 * row)[0]


def test_against_scipy_and_torch_fp64():
    rng = np.random.default_rng(2)
    x = rng.normal(size=(6, 5001)) * rng.uniform(0.3, 5, size=(6, 1))
    x[1, 77] += 14
    x[4, 3] = -np.inf
    H, y, f = O.row_stats(x)
    assert (f == 0).all()
    for r in range(6):
        p = scipy.special.softmax(x[r])
        assert H[r] == pytest.approx(scipy.stats.entropy(p), rel=1e-12)
        t = torch.distributions.Categorical(logits=torch.from_numpy(x[r])).entropy().item()
        assert H[r] == pytest.approx(t, rel=1e-10)
        assert y[r] == int(torch.argmax(torch.from_numpy(x[r])))


def test_against_pure_python_brute_force():
    rng = np.random.default_rng(3)
    for V in (1, 2, 3, 11, 200):
        for _ in range(5):
            row = (rng.normal(size=V) * 4).round(1)      # rounding makes ties likely
            Hn, yn = H_of(row)
            Hl, yl = O.row_stats_loops(list(row))
            assert Hn == pytest.approx(Hl, abs=1e-13)
            assert yn == yl


def test_argmax_lowest_index_wins_ties():
    rng = np.random.default_rng(4)
    for _ in range(50):
        V = int(rng.integers(2, 300))
        row = rng.normal(size=V)
        top = row.max() + 1.0
        where = np.sort(rng.choice(V, size=int(rng.integers(1, min(V, 6) + 1)), replace=False))
        row[where] = top
        _, y = H_of(row)
        assert y == where[0]
    # the value decides before the index does
    assert H_of([0.0, 1.0, 3.0, 2.0, 3.0, -1.0])[1] == 2
    assert H_of([5.0, 1.0, 5.0])[1] == 0
    assert H_of([-np.inf, -2.0, -np.inf, -2.0])[1] == 1


def test_entropy_range_and_gaussian_rows():
    # h in [0, 1]; for iid N(0, sigma^2) logits with small sigma, H ~ log V - sigma^2/2
    rng = np.random.default_rng(5)
    V = 128256
    for sigma in (0.5, 1.0, 1.5):
        x = rng.normal(size=(1, V)) * sigma
        H = O.row_stats(x)[0][0]
        assert 0.0 <= H <= math.log(V)
        assert H == pytest.approx(math.log(V) - sigma * sigma / 2, abs=0.03)


def test_bf16_and_fp32_widen_exactly():
    g = torch.Generator().manual_seed(0)
    x = (torch.randn(3, 1000, generator=g) * 3).to(torch.bfloat16)
    wide = x.double().numpy()
    assert (torch.from_numpy(wide).to(torch.bfloat16) == x).all()
    H, y, _ = O.row_stats(wide)
    for r in range(3):
        vals = wide[r]
        assert vals[y[r]] == vals.max() and (vals[: y[r]] < vals.max()).all()


def test_nonfinite_rows_are_flagged_not_computed():
    x = np.zeros((4, 9))
    x[0, 3] = np.nan
    x[1, 8] = np.inf
    x[2, :] = -np.inf
    x[3, 0] = -np.inf          # a masked entry alone is fine
    H, y, f = O.row_stats(x)
    assert list(f) == [O.FLAG_NONFINITE] * 3 + [0]
    assert H[3] == pytest.approx(math.log(8), abs=1e-13) and y[3] == 1


def test_theta_units():
    V = 128256
    assert O.theta_in_nats(1.0, "nats", V) == 1.0
    assert O.theta_in_nats(0.3, "normalized", V) == pytest.approx(0.3 * math.log(V))
    # h < theta  <=>  H < theta log V  (Eq. 5 with Eq. 6)
    H = np.array([3.0, 4.0])
    h = O.normalized_entropy(H, V)
    th = 0.3
    assert list(h < th) == list(H < O.theta_in_nats(th, "normalized", V))
    with pytest.raises(ValueError):
        O.theta_in_nats(1.0, "bits", V)


def test_lm_head_logits_is_the_plain_product():
    rng = np.random.default_rng(6)
    h = torch.from_numpy(rng.normal(size=(5, 64))).to(torch.bfloat16).double().numpy()
    w = torch.from_numpy(rng.normal(size=(64, 37)) * 0.02).to(torch.bfloat16).double().numpy()
    got = O.lm_head_logits(h, w)
    want = np.zeros((5, 37))
    for r in range(5):
        for v in range(37):
            want[r, v] = math.fsum(h[r, d] * w[d, v] for d in range(64))
    assert np.allclose(got, want, rtol=0, atol=1e-13)
    # operands are not transposed: a non-square, asymmetric case
    e = np.zeros((1, 64)); e[0, 5] = 1.0
    assert np.array_equal(O.lm_head_logits(e, w)[0], w[5])
    t = torch.matmul(torch.from_numpy(h), torch.from_numpy(w)).numpy()
    assert np.allclose(got, t, rtol=0, atol=1e-12)


def test_temperature_divides_the_logits():
    # Entropy of softmax(l / T).  Pins: T = 1 changes nothing; single spike of height a over a flat row has the
    # closed form with a / T in place of a; a large T flattens any finite row towards ln V; a small T sharpens a
    # row with a unique maximum towards 0; the greedy token never moves.
    V, a = 1000, 6.0
    row = np.zeros((1, 1, V)); row[0, 0, 123] = a
    draft = np.zeros((1, 0), dtype=np.int64)

    def closed(h):
        return math.log(math.exp(h) + V - 1) - h * math.exp(h) / (math.exp(h) + V - 1)

    for T in (0.5, 0.7, 1.0, 1.5, 3.0):
        r = O.verify_batch(row, draft, theta=1.0, W=0, temperature=T)
        assert abs(r.entropy[0, 0] - closed(a / T)) < 1e-12 and r.target_argmax[0, 0] == 123
    rng = np.random.default_rng(5)
    x = rng.normal(size=(2, 3, 64)) * 4
    d = np.zeros((2, 2), dtype=np.int64)
    base = O.verify_batch(x, d, theta=1.0, W=1)
    same = O.verify_batch(x, d, theta=1.0, W=1, temperature=1.0)
    assert np.array_equal(base.entropy, same.entropy) and np.array_equal(base.out_tokens, same.out_tokens)
    hot = O.verify_batch(x, d, theta=1.0, W=1, temperature=1e4)
    assert np.all(np.abs(hot.entropy - math.log(64)) < 1e-5)
    cold = O.verify_batch(x, d, theta=1.0, W=1, temperature=1e-3)
    assert np.all(cold.entropy < 1e-9)
    for r in (hot, cold):
        assert np.array_equal(r.target_argmax, base.target_argmax)
    # scipy on the divided logits (library restatement of the definition)
    from scipy.special import softmax
    from scipy.stats import entropy
    r = O.verify_batch(x, d, theta=1.0, W=1, temperature=0.7)
    assert np.allclose(r.entropy, entropy(softmax(x / 0.7, axis=-1), axis=-1), atol=1e-12, rtol=0)
    with pytest.raises(ValueError):
        O.verify_batch(x, d, theta=1.0, W=1, temperature=0.0)
