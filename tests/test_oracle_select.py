"""Pins for the oracle's selection (Definition 1 / Eq. 1, Eq. 3, Definition 2 / Eq. 2).

None of the expected values here is produced by the oracle: they come from a
hand-worked example, exact rational arithmetic, a rank-by-counting brute
force, numpy's stable sort, and invariants of the definitions.
"""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle
from conftest import load_hand_example


# ----------------------------------------------------------------- helpers --
def exact_count(frac: Fraction, n: int) -> int:
    """ceil(frac * n) in exact rational arithmetic."""
    v = frac * n
    return min(n, max(0, -((-v.numerator) // v.denominator)))


def is_pos(v: np.float32) -> bool:
    return bool(v > 0) and not math.isnan(float(v))


def brute_select(A, alpha: Fraction, beta: Fraction):
    """Rank every element by counting who beats it (O(N^2)); no sorting."""
    T, N = A.shape
    f = [0] * N
    for t in range(T):
        row = A[t]
        pos = [n for n in range(N) if is_pos(row[n])]
        k = exact_count(alpha, len(pos))
        for n in pos:
            beaten_by = sum(1 for m in pos
                            if row[m] > row[n] or (row[m] == row[n] and m < n))
            if beaten_by < k:
                f[n] += 1
    K = exact_count(beta, N)
    S = [n for n in range(N)
         if sum(1 for m in range(N) if f[m] > f[n] or (f[m] == f[n] and m < n)) < K]
    return np.array(S, dtype=np.int32), np.array(f, dtype=np.int32)


def numpy_select(A, alpha, beta):
    """Library-routine restatement: stable argsort of the negated values."""
    T, N = A.shape
    f = np.zeros(N, dtype=np.int64)
    for t in range(T):
        idx = np.flatnonzero(A[t] > 0)                     # ascending index
        order = idx[np.argsort(-A[t, idx].astype(np.float64), kind="stable")]
        k = exact_count(Fraction(alpha).limit_denominator(10000), len(idx))
        np.add.at(f, order[:k], 1)
    K = exact_count(Fraction(beta).limit_denominator(10000), N)
    S = np.sort(np.argsort(-f, kind="stable")[:K])
    return S.astype(np.int32), f.astype(np.int32)


# ------------------------------------------------------------------- count --
@pytest.mark.parametrize("frac", ["0.1", "0.2", "0.25", "0.4", "0.5", "0.75", "1.0"])
def test_count_matches_exact_rational(frac):
    fr = Fraction(frac)
    fl = float(frac)
    for n in range(0, 40001):
        assert oracle.count(fl, n) == exact_count(fr, n), (frac, n)


def test_count_known_values():
    # products that are integers in decimal but not in binary
    assert oracle.count(0.2, 20480) == 4096
    assert oracle.count(0.25, 11008) == 2752
    assert oracle.count(0.2, 16384) == 3277
    assert oracle.count(0.2, 3072) == 615
    assert oracle.count(0.2, 36864) == 7373
    assert oracle.count(0.4, 5) == 2
    assert oracle.count(0.4, 13) == 6          # an interpolating percentile would give 5
    assert oracle.count(0.4, 0) == 0
    assert oracle.count(1.0, 7) == 7


# ------------------------------------------------------------ hand example --
def test_hand_worked_example():
    A, cases = load_hand_example()
    assert A.shape == (4, 8) and len(cases) >= 3
    for alpha, beta, f_exp, S_exp in cases:
        S, f = oracle.select(A, alpha, beta)
        np.testing.assert_array_equal(f, f_exp)
        np.testing.assert_array_equal(S, S_exp)


def test_hand_example_token_sets():
    A, _ = load_hand_example()
    got = [oracle.token_core(r, 0.5).tolist() for r in A]
    assert got == [[0, 5, 2], [0, 1, 3], [2, 5], []]


# ------------------------------------------------------------- brute force --
ALPHABET = np.array([-1.0, 0.0, 0.5, 1.0], dtype=np.float32)


@pytest.mark.parametrize("alpha,beta", [("0.4", "0.2"), ("0.5", "0.5"), ("1.0", "0.75")])
def test_exhaustive_small_alphabet_two_rows(alpha, beta):
    """All 4^8 matrices with T=2, N=4 over a 4-value alphabet (heavy ties)."""
    fa, fb = Fraction(alpha), Fraction(beta)
    for code in itertools.product(range(4), repeat=8):
        A = ALPHABET[list(code)].reshape(2, 4)
        S, f = oracle.select(A, float(alpha), float(beta))
        S_b, f_b = brute_select(A, fa, fb)
        assert np.array_equal(f, f_b) and np.array_equal(S, S_b), (A, alpha, beta)


def test_exhaustive_small_alphabet_one_row_n6():
    fa, fb = Fraction("0.4"), Fraction("0.5")
    for code in itertools.product(range(4), repeat=6):
        A = ALPHABET[list(code)].reshape(1, 6)
        S, f = oracle.select(A, 0.4, 0.5)
        S_b, f_b = brute_select(A, fa, fb)
        assert np.array_equal(f, f_b) and np.array_equal(S, S_b), A


def test_random_small_vs_brute_force():
    rng = np.random.default_rng(7)
    fracs = ["0.1", "0.2", "0.25", "0.4", "0.5", "0.75", "1.0"]
    for _ in range(1500):
        T, N = int(rng.integers(1, 4)), int(rng.integers(1, 9))
        if rng.random() < 0.5:       # quantised values: many ties
            A = rng.integers(-2, 4, size=(T, N)).astype(np.float32) * 0.25
        else:
            A = rng.standard_normal((T, N)).astype(np.float32)
        a, b = rng.choice(fracs), rng.choice(fracs)
        S, f = oracle.select(A, float(a), float(b))
        S_b, f_b = brute_select(A, Fraction(a), Fraction(b))
        assert np.array_equal(f, f_b) and np.array_equal(S, S_b), (A, a, b)


# --------------------------------------------------------- library routine --
@pytest.mark.parametrize("T,N,alpha,beta,quant", [
    (7, 257, 0.4, 0.2, False), (33, 1000, 0.4, 0.25, True), (64, 3072, 0.4, 0.2, False),
    (5, 4099, 0.1, 0.4, True), (16, 513, 1.0, 1.0, False),
])
def test_matches_numpy_stable_sort(T, N, alpha, beta, quant):
    rng = np.random.default_rng(T * 1000 + N)
    A = rng.standard_normal((T, N)).astype(np.float32)
    if quant:
        A = np.round(A * 4) / 4            # multiples of 0.25: ties inside rows
    S, f = oracle.select(A, alpha, beta)
    S_n, f_n = numpy_select(A, alpha, beta)
    np.testing.assert_array_equal(f, f_n)
    np.testing.assert_array_equal(S, S_n)


# -------------------------------------------------------------- invariants --
def _random_A(rng, T, N):
    A = rng.standard_normal((T, N)).astype(np.float32)
    A[rng.random((T, N)) < 0.3] = 0.0
    return A


def test_invariants():
    rng = np.random.default_rng(11)
    for T, N, alpha, beta in [(1, 64, 0.4, 0.2), (9, 300, 0.4, 0.2), (40, 777, 0.25, 0.5)]:
        A = _random_A(rng, T, N)
        S, f = oracle.select(A, alpha, beta)
        K = exact_count(Fraction(str(beta)), N)
        P = (A > 0).sum(axis=1)
        k = [exact_count(Fraction(str(alpha)), int(p)) for p in P]
        assert f.sum() == sum(k)                                  # Eq. 3 summed over n
        assert f.min() >= 0 and f.max() <= T
        assert len(S) == K and np.all(np.diff(S) > 0)             # |S| = ceil(beta N), ascending
        ever_pos = (A > 0).any(axis=0)
        assert np.all(ever_pos[S[f[S] > 0]])                      # counted members were positive somewhere
        assert np.all(f[~ever_pos] == 0)
        rest = np.setdiff1d(np.arange(N), S)
        if len(rest):
            assert f[S].min() >= f[rest].max()
        if (f > 0).sum() >= K:
            assert np.all(f[S] > 0)                               # zero-count padding only when needed
        # the order of the tokens does not matter
        S_p, f_p = oracle.select(A[rng.permutation(T)], alpha, beta)
        np.testing.assert_array_equal(f_p, f)
        np.testing.assert_array_equal(S_p, S)
        # scaling a row by a positive power of two keeps its order
        A2 = A.copy()
        A2[0] *= 4.0
        A2[-1] *= 0.125
        S_s, f_s = oracle.select(A2, alpha, beta)
        np.testing.assert_array_equal(f_s, f)
        np.testing.assert_array_equal(S_s, S)


def test_special_cases():
    rng = np.random.default_rng(3)
    N = 200
    A = _random_A(rng, 6, N)
    # beta = 1 gives every neuron, whatever alpha
    for alpha in (0.1, 0.4, 1.0):
        S, _ = oracle.select(A, alpha, 1.0)
        np.testing.assert_array_equal(S, np.arange(N))
    # alpha = 1 counts every positive entry
    _, f = oracle.select(A, 1.0, 0.5)
    np.testing.assert_array_equal(f, (A > 0).sum(axis=0))
    # no positive entry anywhere: counts zero, the K lowest indices
    S, f = oracle.select(-np.abs(A), 0.4, 0.2)
    assert f.sum() == 0
    np.testing.assert_array_equal(S, np.arange(40))
    # T identical rows: f in {0, T}; S = lowest members of the token set, then padding
    row = A[:1]
    S, f = oracle.select(np.repeat(row, 5, axis=0), 0.4, 0.2)
    assert set(np.unique(f).tolist()) <= {0, 5}
    members = np.sort(oracle.token_core(row[0], 0.4))
    np.testing.assert_array_equal(S, members[:40] if len(members) >= 40 else
                                  np.sort(np.concatenate([members, np.setdiff1d(np.arange(N), members)[:40 - len(members)]])))


def test_special_floats():
    """Positive is decided on the bit pattern: subnormals and +Inf are positive;
    +-0, negatives and NaN never are."""
    sub = np.float32(1e-45)                       # smallest subnormal
    row = np.array([np.nan, np.inf, -np.inf, 0.0, -0.0, sub, 1.0, -sub], dtype=np.float32)
    assert oracle.token_core(row, 1.0).tolist() == [1, 6, 5]        # +Inf > 1.0 > subnormal
    assert oracle.token_core(row, 0.34).tolist() == [1, 6]          # ceil(0.34 * 3) = 2
    assert oracle.token_core(row, 0.33).tolist() == [1]
    _, f = oracle.select(row[None, :], 1.0, 1.0)
    assert f.tolist() == [0, 1, 0, 0, 0, 1, 1, 0]


def test_planted_subset_is_recovered():
    """Stability picture of Section 3.2: a fixed subset that dominates the
    counts ends up inside the sentence-wise set."""
    rng = np.random.default_rng(5)
    T, N = 128, 2000
    core = rng.permutation(N)[: int(0.15 * N)]
    A = np.where(rng.random((T, N)) < 0.7, 0.0, np.abs(rng.standard_normal((T, N)) * 0.25))
    A[:, core] = rng.exponential(1.0, size=(T, len(core)))
    S, f = oracle.select(A.astype(np.float32), 0.4, 0.2)
    assert np.isin(core, S).all()
    assert f[core].min() > np.delete(f, core).max()
