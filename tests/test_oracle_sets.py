"""Pins of the oracle's set functions (several sentences: prompts in pieces, semantic groups,
set similarity, in-place set updates) against values they did not produce themselves."""
import numpy as np

import oracle


def test_top_by_count_hand_example_and_library_sort():
    # counts of the hand-worked example (alpha = 0.5): f = [2,1,2,1,0,2,0,0]
    f = np.array([2, 1, 2, 1, 0, 2, 0, 0], np.int32)
    np.testing.assert_array_equal(oracle.top_by_count(f, 0.5), [0, 1, 2, 5])
    np.testing.assert_array_equal(oracle.top_by_count(f, 0.75), [0, 1, 2, 3, 4, 5])
    rng = np.random.default_rng(0)
    for N in (1, 7, 64, 1000):
        c = rng.integers(0, 6, size=N).astype(np.int32)
        for frac in (0.1, 0.25, 0.5, 1.0):
            K = oracle.count(frac, N)
            ref = np.sort(np.argsort(-c.astype(np.int64), kind="stable")[:K])
            np.testing.assert_array_equal(oracle.top_by_count(c, frac), ref)


def test_prompt_in_pieces_gives_the_set_of_the_whole_prompt():
    """Eq. 3 is a sum over tokens: the counts of two pieces add up to the counts of the whole."""
    rng = np.random.default_rng(1)
    A = rng.standard_normal((40, 300)).astype(np.float32)
    S, f = oracle.select(A, 0.4, 0.2)
    _, f1 = oracle.select(A[:13], 0.4, 0.2)
    _, f2 = oracle.select(A[13:], 0.4, 0.2)
    np.testing.assert_array_equal(f1 + f2, f)
    np.testing.assert_array_equal(oracle.top_by_count(f1 + f2, 0.2), S)


def test_group_counts_and_group_set():
    sets = [np.array([0, 2, 5], np.int32), np.array([2, 3, 5], np.int32), np.array([1, 2, 7], np.int32)]
    c = oracle.group_counts(sets, 8)
    np.testing.assert_array_equal(c, [1, 1, 3, 1, 0, 2, 0, 1])          # by hand
    np.testing.assert_array_equal(c, np.bincount(np.concatenate(sets), minlength=8))
    np.testing.assert_array_equal(oracle.top_by_count(c, 0.375), [0, 2, 5])   # 3 of 8: counts 3, 2, then the lowest-index 1


def test_core_similarity_against_numpy_set_routines():
    assert oracle.core_similarity([0, 1, 2, 5], [1, 2, 3, 4]) == (2, 6)          # by hand
    assert oracle.core_similarity([3, 4], [3, 4]) == (2, 2)
    assert oracle.core_similarity([0], [9]) == (0, 2)
    rng = np.random.default_rng(2)
    for _ in range(20):
        A = np.sort(rng.choice(500, size=rng.integers(1, 200), replace=False)).astype(np.int32)
        B = np.sort(rng.choice(500, size=rng.integers(1, 200), replace=False)).astype(np.int32)
        assert oracle.core_similarity(A, B) == (len(np.intersect1d(A, B)), len(np.union1d(A, B)))


def test_nearest_centroid():
    C = np.array([[0, 0], [10, 0], [0, 10]], np.float32)
    g, d2 = oracle.nearest_centroid(C, np.array([6, 1], np.float32))
    assert g == 1 and list(d2) == [37.0, 17.0, 117.0]                    # by hand
    assert oracle.nearest_centroid(C, np.array([5, 0], np.float32))[0] == 0   # tie: lower group
    rng = np.random.default_rng(3)
    C = rng.standard_normal((16, 257)).astype(np.float32)
    for g in range(16):
        v = C[g] + 0.01 * rng.standard_normal(257).astype(np.float32)
        got, d2 = oracle.nearest_centroid(C, v)
        ref = ((C.astype(np.float64) - v.astype(np.float64)) ** 2).sum(axis=1)
        assert got == g == int(np.argmin(ref))
        np.testing.assert_allclose(d2, ref, rtol=1e-12)


def test_set_delta():
    slot_neuron = np.array([4, 9, 1, 7], np.int32)                       # rows hold these neurons, any order
    slots, neurons, after = oracle.set_delta(slot_neuron, np.array([1, 2, 7, 8], np.int32))
    np.testing.assert_array_equal(slots, [0, 1])                          # 4 and 9 leave
    np.testing.assert_array_equal(neurons, [2, 8])                        # 2 and 8 enter
    np.testing.assert_array_equal(after, [2, 8, 1, 7])
    rng = np.random.default_rng(4)
    for _ in range(20):
        K = int(rng.integers(1, 60))
        cur = rng.permutation(rng.choice(200, size=K, replace=False)).astype(np.int32)
        new = np.sort(rng.choice(200, size=K, replace=False)).astype(np.int32)
        slots, neurons, after = oracle.set_delta(cur, new)
        np.testing.assert_array_equal(np.sort(after), new)                # the rows now hold exactly the new set
        np.testing.assert_array_equal(neurons, np.setdiff1d(new, cur))
        np.testing.assert_array_equal(np.sort(cur[slots]), np.setdiff1d(cur, new))
        assert (np.diff(slots) > 0).all() if len(slots) > 1 else True
        untouched = np.setdiff1d(np.arange(K), slots)
        np.testing.assert_array_equal(after[untouched], cur[untouched])   # every other row stays where it is
