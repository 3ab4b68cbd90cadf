"""Pins for the repetition-code oracle: what the paper and arithmetic fix."""
import itertools

import numpy as np
import pytest

import draco_inputs as di
from oracle import draco_oracle as orc


def _group_sums(G, n, s):
    """Honest value each group should contribute: fp32(sum of its gradients)."""
    out = []
    for first, size in orc.rep_groups(n, s):
        out.append(G[first:first + size].astype(np.float64).sum(axis=0).astype(np.float32))
    return np.stack(out)


def test_groups_and_allocation():
    assert orc.rep_groups(15, 2) == [(0, 5), (5, 5), (10, 5)]             # r | n: n / r groups of r
    assert [sz for _, sz in orc.rep_groups(45, 3)] == [8, 8, 8, 7, 7, 7]  # r does not divide n
    assert orc.rep_groups(15, 7) == [(0, 15)]
    for n, s in [(15, 2), (9, 1), (45, 3), (45, 5), (105, 7), (15, 5)]:
        groups = orc.rep_groups(n, s)
        assert sum(sz for _, sz in groups) == n
        assert all(sz >= 2 * s + 1 for _, sz in groups)
        A = orc.rep_allocation(n, s)
        ratio = A.sum() / n                                                # redundancy ratio (Definition 1)
        assert ratio >= 2 * s + 1                                          # Theorem 1
        if n % (2 * s + 1) == 0:
            assert ratio == 2 * s + 1                                      # Theorem 2: optimal
            assert np.array_equal(A, np.kron(np.eye(n // (2 * s + 1), dtype=np.int64),
                                             np.ones((2 * s + 1, 2 * s + 1), dtype=np.int64)))
    with pytest.raises(ValueError):
        orc.rep_groups(4, 2)


def test_streaming_majority_against_sort_and_count():
    rng = np.random.default_rng(0)
    for m in (1, 2, 3, 5, 7, 8, 15):
        L = 400
        items = rng.integers(0, 3, size=(m, L)).astype(np.uint32)
        cand = orc.majority_stream(items)
        for c in range(L):
            vals, counts = np.unique(items[:, c], return_counts=True)
            if 2 * counts.max() > m:                       # a strict majority exists: Alg. 2 must find it
                assert cand[c] == vals[counts.argmax()]
            else:                                          # otherwise it still returns one of the items
                assert cand[c] in items[:, c]


def test_streaming_majority_on_every_short_sequence():
    """Every sequence of up to 7 items over a 3-letter alphabet: whenever one letter holds strictly more than
    half of the positions the vote returns it, and otherwise it returns a letter that occurs in the sequence."""
    for m in range(1, 8):
        seqs = np.array(list(itertools.product(range(3), repeat=m)), dtype=np.uint32).T      # [m][3^m]
        cand = orc.majority_stream(seqs)
        counts = np.stack([(seqs == v).sum(axis=0) for v in range(3)])                        # [3][3^m]
        has_majority = 2 * counts.max(axis=0) > m
        assert has_majority.any() and (m < 2 or (~has_majority).any())
        np.testing.assert_array_equal(cand[has_majority], counts.argmax(axis=0)[has_majority])
        assert all(cand[c] in seqs[:, c] for c in np.flatnonzero(~has_majority))


def test_encode_replicas_identical_and_equal_group_sum():
    n, s, d = 15, 2, 257
    G = di.gradient_rows(3, n, d)
    Z = orc.rep_encode(G, n, s)
    sums = _group_sums(G, n, s)
    for ell, (first, size) in enumerate(orc.rep_groups(n, s)):
        for j in range(first, first + size):
            np.testing.assert_array_equal(Z[j].view(np.uint32), sums[ell].view(np.uint32))


def test_no_adversary_is_plain_sum():
    for n, s in [(15, 2), (45, 3), (9, 4)]:
        G = di.gradient_rows(5, n, 300)
        out = orc.rep_decode(orc.rep_encode(G, n, s), n, s)
        exact = G.astype(np.float64).sum(axis=0)
        assert np.abs(out["u"] - exact).max() <= 1e-6 * np.abs(exact).max()
        assert not out["flags"].any() and out["no_majority"] == 0


@pytest.mark.parametrize("n,s", [(3, 1), (5, 2), (6, 1), (9, 1), (10, 2), (15, 2), (7, 1)])
def test_every_placement_of_up_to_s_adversaries_is_corrected(n, s):
    """Definition 2 / Theorem 2 by brute force: D(Z + N) = G 1_P for every N with <= s non-zero columns."""
    d = 12
    G = di.gradient_rows(11, n, d)
    Z = orc.rep_encode(G, n, s)
    honest = _group_sums(G, n, s).astype(np.float64).sum(axis=0)
    exact = G.astype(np.float64).sum(axis=0)
    attacks = [(di.ADV_REVGRAD, 100.0), (di.ADV_CONST, -100.0), (di.ADV_GAUSS, 1e3)]
    for a in range(s + 1):
        for placement in itertools.combinations(range(n), a):
            for model, param in attacks:
                R = Z.copy()
                di.apply_adversaries(R, placement, [model] * a, [param] * a, seed=2)
                out = orc.rep_decode(R, n, s)
                np.testing.assert_array_equal(out["u"], honest)
                assert np.abs(out["u"] - exact).max() <= 1e-6 * max(1.0, np.abs(exact).max())
                assert set(np.flatnonzero(out["flags"])) == set(placement)
                assert out["no_majority"] == 0
    # a single-coordinate corruption is corrected and flagged too
    R = Z.copy()
    R[n - 1, 7] += np.float32(1.0)
    out = orc.rep_decode(R, n, s)
    np.testing.assert_array_equal(out["u"], honest)
    assert list(np.flatnonzero(out["flags"])) == [n - 1]


def test_failure_beyond_s():
    """Theorem 1: redundancy 2 s + 1 cannot survive s + 1 colluders."""
    n, s, d = 15, 2, 40
    G = di.gradient_rows(4, n, d)
    Z = orc.rep_encode(G, n, s)
    R = Z.copy()
    for j in (5, 6, 7):                                   # s + 1 identical colluders inside group 1
        R[j] = np.float32(1e4)
    out = orc.rep_decode(R, n, s)
    np.testing.assert_array_equal(out["maj"][1], np.full(d, 1e4, dtype=np.float32))
    assert np.abs(out["u"] - G.astype(np.float64).sum(axis=0)).max() > 1e3
    assert set(np.flatnonzero(out["flags"])) == {8, 9}     # the honest minority is blamed
    # s + 1 adversaries sending unrelated noise leave no strict majority instead
    R = Z.copy()
    di.apply_adversaries(R, [5, 6, 7], [di.ADV_GAUSS] * 3, [1e3] * 3, seed=8)
    out = orc.rep_decode(R, n, s)
    assert out["no_majority"] == d


def test_equality_is_on_bit_patterns():
    n, s = 3, 1
    R = np.zeros((3, 4), dtype=np.float32)
    R[0] = -0.0                                            # -0.0 == +0.0 as floats, different bits
    out = orc.rep_decode(R, n, s)
    assert list(out["flags"]) == [True, False, False]
    assert not np.signbit(out["maj"][0]).any()
    R = np.full((3, 4), np.nan, dtype=np.float32)          # NaN != NaN as floats, equal bits
    R[2] = 1.0
    out = orc.rep_decode(R, n, s)
    assert list(out["flags"]) == [False, False, True] and np.isnan(out["maj"][0]).all()
