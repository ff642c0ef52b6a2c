"""Pins for the oracle's validation walk (paper Section 3.3, Fig. 5) and the outer loop.

The walk in the oracle is written as the paper describes it (sequence equality
against a growing ground truth).  Here it is pinned against an independent
brute-force statement: the number of accepted drafts is the index of the first
drafted token that differs from the main model's token for the previous row.
"""
import itertools

import numpy as np
import pytest

from oracle import stairs_oracle as so


def brute_force_accept(draft, predicted):
    for i, d in enumerate(draft):
        if d != predicted[i]:
            return i
    return len(draft)


@pytest.mark.parametrize("k", range(0, 9))
def test_walk_equals_first_mismatch_exhaustive_patterns(k):
    ctx = [5, 6, 7]
    # every match/mismatch pattern over the k drafted tokens
    for pattern in itertools.product([True, False], repeat=k):
        predicted = [10 + i for i in range(k + 1)]
        draft = [predicted[i] if pattern[i] else predicted[i] + 100 for i in range(k)]
        rows = so.stairs_rows(ctx, draft)
        assert len(rows) == k + 1 and all(len(rows[r]) == len(ctx) + r for r in range(k + 1))
        ground, a = so.stairs_validate_walk(rows, predicted)
        assert a == brute_force_accept(draft, predicted)
        assert 0 <= a <= k
        # the ground truth is the context, the accepted drafts and the main model's next token
        assert ground == ctx + draft[:a] + [predicted[a]]
        assert len(ground) - len(ctx) == a + 1


def test_walk_exhaustive_small_alphabet():
    # all drafts and all predictions over a 3-symbol alphabet, k <= 3: catches index slips
    ctx = [1]
    for k in range(0, 4):
        for draft in itertools.product(range(3), repeat=k):
            for predicted in itertools.product(range(3), repeat=k + 1):
                rows = so.stairs_rows(ctx, list(draft))
                ground, a = so.stairs_validate_walk(rows, list(predicted))
                assert a == brute_force_accept(draft, predicted)
                assert ground == ctx + list(draft[:a]) + [predicted[a]]


def test_walk_repeated_tokens_do_not_confuse_the_comparison():
    # a draft that repeats the context's last token must still be compared position-wise
    ctx = [4, 4, 4]
    rows = so.stairs_rows(ctx, [4, 4])
    ground, a = so.stairs_validate_walk(rows, [4, 9, 4])
    assert a == 1 and ground == [4, 4, 4, 4, 9]


def test_rows_are_prefixes_of_each_other():
    rows = so.stairs_rows([1, 2], [3, 4, 5])
    assert rows == [[1, 2], [1, 2, 3], [1, 2, 3, 4], [1, 2, 3, 4, 5]]


def test_argmax_lowest_id_wins_ties():
    lg = np.array([0.0, 2.0, 2.0, 1.0], dtype=np.float32)
    assert so.argmax_lowest(lg) == 1
    assert so.top2_margin(lg) == 0.0
    assert so.top2_margin(np.array([3.0, 1.0, 2.5], dtype=np.float32)) == 0.5
    with pytest.raises(FloatingPointError):
        so.argmax_lowest(np.array([0.0, np.nan], dtype=np.float32))
