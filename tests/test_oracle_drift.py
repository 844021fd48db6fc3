"""CPU pins of the oracle's teacher-drift diagnostics (Section 3.1): entropy / branching factor,
rank of the sampled token, top-k survival."""
import math

import numpy as np
import pytest
import scipy.stats

from oracle import adwin_oracle as O


def test_entropy_of_uniform_and_of_a_subset():
    for V in (1, 2, 8, 1000):
        H, r = O.teacher_drift_row(np.full(V, 3.25), 0)
        assert math.isclose(H, math.log(V), rel_tol=1e-13, abs_tol=1e-15) and r == 1
    # m equally likely tokens, the rest impossible: branching factor exactly m
    u = np.full(50, -1.0e4)
    u[[3, 7, 11, 40]] = 2.0
    H, _ = O.teacher_drift_row(u, 3)
    assert math.isclose(math.exp(H), 4.0, rel_tol=1e-12)


def test_entropy_two_point_closed_form_and_shift_invariance():
    a = 1.7
    q = 1.0 / (1.0 + math.exp(-a))
    want = -(q * math.log(q) + (1 - q) * math.log(1 - q))
    H, _ = O.teacher_drift_row(np.array([a, 0.0]), 0)
    assert math.isclose(H, want, rel_tol=1e-13)
    H2, _ = O.teacher_drift_row(np.array([a + 500.0, 500.0]), 0)
    assert math.isclose(H2, want, rel_tol=1e-12)


def test_entropy_against_scipy():
    rng = np.random.default_rng(0)
    for V, s in ((7, 1.0), (513, 3.0), (4096, 6.0)):
        u = rng.normal(0, s, V)
        q = np.exp(u - u.max())
        q /= q.sum()
        H, _ = O.teacher_drift_row(u, 1)
        assert math.isclose(H, float(scipy.stats.entropy(q)), rel_tol=1e-12)


def test_rank_against_sorting_with_ties_and_bad_tokens():
    rng = np.random.default_rng(1)
    u = rng.normal(0, 2, 200)
    order = np.argsort(-u, kind="stable")
    for pos in (0, 1, 17, 199):
        _, r = O.teacher_drift_row(u, int(order[pos]))
        assert r == pos + 1
    u = np.array([1.0, 5.0, 5.0, 3.0, 5.0, 0.0])
    assert [O.teacher_drift_row(u, y)[1] for y in range(6)] == [5, 1, 1, 4, 1, 6]
    assert O.teacher_drift_row(u, -1)[1] == 0 and O.teacher_drift_row(u, 6)[1] == 0


def test_survival_on_a_worked_example():
    # three rollouts of up to 5 positions
    rank = np.array([[1, 2, 1, 9, 1],
                     [3, 1, 1, 1, 1],
                     [1, 1, 7, 7, 7]])           # rollout 2 ends after 2 positions
    R = np.array([5, 5, 2], dtype=np.int32)
    np.testing.assert_array_equal(O.topk_survival(rank, R, 2), [2 / 3, 2 / 3, 2 / 3, 1 / 3, 1 / 3])
    np.testing.assert_array_equal(O.topk_survival(rank, R, 1), [2 / 3, 1 / 3, 1 / 3, 1 / 3, 1 / 3])
    np.testing.assert_array_equal(O.topk_survival(rank, R, 9), [1, 1, 1, 1, 1])
    np.testing.assert_array_equal(O.topk_survival(rank, None, 3), [1, 1, 2 / 3, 1 / 3, 1 / 3])


@pytest.mark.parametrize("k", [1, 3, 10])
def test_survival_is_monotone_and_matches_a_running_maximum(k):
    rng = np.random.default_rng(2)
    B, T = 40, 60
    rank = rng.integers(1, 15, size=(B, T))
    R = rng.integers(0, T + 1, size=B).astype(np.int32)
    S = O.topk_survival(rank, R, k)
    assert (np.diff(S) <= 0).all() and 0 <= S[-1] <= S[0] <= 1
    masked = np.where(np.arange(T)[None, :] < R[:, None], rank, 0)
    want = (np.maximum.accumulate(masked, axis=1) <= k).mean(axis=0)
    np.testing.assert_allclose(S, want, rtol=0, atol=1e-15)
