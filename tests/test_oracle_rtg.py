"""CPU pins of the oracle's discounted return-to-go (Eq. 3) and of the sampled-token gradient with
a given coefficient: special cases the paper states, closed forms, invariants, brute force."""
import math

import numpy as np
import pytest

from oracle import adwin_oracle as O


def _costs(B, T, seed=3):
    rng = np.random.default_rng(seed)
    return rng.normal(0.2, 1.0, size=(B, T))


def test_gamma_zero_returns_the_costs_themselves():
    # Section 3 / appendix: with gamma = 0 the return-to-go collapses to the immediate cost c_t
    c = _costs(3, 17)
    w = np.array([17, 5, 0], dtype=np.int32)
    G = O.return_to_go(c, w, None, 0.0)
    for b in range(3):
        np.testing.assert_array_equal(G[b, :w[b]], c[b, :w[b]])
        assert (G[b, w[b]:] == 0).all()


def test_gamma_one_gives_suffix_sums():
    # undiscounted form of the derivation: sum_{t'=t}^{T} c_t'
    c = _costs(2, 40)
    w = np.array([40, 23], dtype=np.int32)
    G = O.return_to_go(c, w, None, 1.0)
    for b in range(2):
        want = np.cumsum(c[b, :w[b]][::-1])[::-1]
        np.testing.assert_allclose(G[b, :w[b]], want, rtol=1e-13, atol=1e-13)
        assert (G[b, w[b]:] == 0).all()


@pytest.mark.parametrize("gamma", [0.3, 0.9, 0.999])
def test_constant_cost_gives_the_geometric_closed_form(gamma):
    T, E = 64, 50
    c = np.ones((1, T))
    G = O.return_to_go(c, np.array([E], dtype=np.int32), None, gamma)
    n = E - np.arange(E)
    np.testing.assert_allclose(G[0, :E], (1 - gamma ** n) / (1 - gamma), rtol=1e-12)


@pytest.mark.parametrize("gamma", [0.0, 0.5, 0.97, 1.0])
def test_recurrence_and_last_position(gamma):
    c = _costs(2, 33, seed=9)
    w = np.array([33, 12], dtype=np.int32)
    r = np.array([30, 33], dtype=np.int32)          # sequence 0 ends before its window
    G = O.return_to_go(c, w, r, gamma)
    for b, E in enumerate([30, 12]):
        assert G[b, E - 1] == c[b, E - 1]
        np.testing.assert_allclose(G[b, :E - 1] - gamma * G[b, 1:E], c[b, :E - 1],
                                   rtol=1e-12, atol=1e-12)
        assert (G[b, E:] == 0).all()


def test_brute_force_on_a_tiny_case_and_the_full_range_flag():
    gamma = 0.8
    c = _costs(2, 6, seed=1)
    w = np.array([2, 6], dtype=np.int32)
    r = np.array([5, 4], dtype=np.int32)
    for flags, ends in [(0, [2, 4]), (O.FLAG_RANGE_FULL, [5, 4])]:
        G = O.return_to_go(c, w, r, gamma, flags)
        for b in range(2):
            for t in range(6):
                want = 0.0
                if t < ends[b]:
                    weight = 1.0
                    for tp in range(t, ends[b]):
                        want += weight * c[b, tp]
                        weight *= gamma
                assert math.isclose(G[b, t], want, rel_tol=1e-13, abs_tol=1e-15)


def test_weighted_row_reduces_to_the_sampled_mode_and_is_linear():
    rng = np.random.default_rng(5)
    z, u = rng.normal(0, 2, 50), rng.normal(0, 2, 50)
    y, alpha = 7, -0.75
    ref = O.row(z, u, y, alpha, O.MODE_SAMPLED)
    g, gsq = O.row_weighted(z, y, alpha, ref["c"])          # w = c_t: Eq. 4
    np.testing.assert_allclose(g, ref["g"], rtol=1e-14, atol=1e-300)
    assert math.isclose(gsq, ref["gsq"], rel_tol=1e-13)
    g2, gsq2 = O.row_weighted(z, y, alpha, 3.0 * ref["c"])
    np.testing.assert_allclose(g2, 3.0 * g, rtol=1e-14)
    assert math.isclose(gsq2, 9.0 * gsq, rel_tol=1e-13)


def test_weighted_row_is_w_times_the_gradient_of_log_p_y():
    rng = np.random.default_rng(6)
    z = rng.normal(0, 1.5, 12)
    y, alpha, w = 4, 1.0, 2.5
    g, gsq = O.row_weighted(z, y, alpha, w)
    assert abs(g.sum()) < 1e-14                              # sum_k (1[k=y] - p_k) = 0
    h = 1e-6
    for k in range(12):
        zp, zm = z.copy(), z.copy()
        zp[k] += h
        zm[k] -= h
        fd = w * ((zp[y] - O.logsumexp(zp)) - (zm[y] - O.logsumexp(zm))) / (2 * h)
        assert math.isclose(g[k], fd, rel_tol=1e-6, abs_tol=1e-8)
    assert math.isclose(gsq, float((g * g).sum()), rel_tol=1e-13)
    g_bad, _ = O.row_weighted(z, 99, alpha, w)
    assert np.isnan(g_bad).all()
