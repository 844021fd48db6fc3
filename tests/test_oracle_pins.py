"""Pins of the float64 oracle against facts that do not come from the oracle itself.

Each test targets a plausible mistake: a swapped KL direction, a sign error in c, a dropped
"- KL" term in the gradient, a transposed operand, an off-by-one window, a wrong normaliser.
"""
import math
from fractions import Fraction

import numpy as np
import pytest
import scipy.special
import torch

from oracle import adwin_oracle as O

RNG = np.random.default_rng(1234)


def rand_rows(V, s=2.0, t=1.0):
    z = RNG.normal(0, s, V)
    u = z + RNG.normal(0, t, V)
    return z, u


# ----------------------------------------------------------------------------- log-sum-exp
@pytest.mark.parametrize("V", [1, 2, 7, 1000, 4096])
def test_logsumexp_matches_scipy_and_torch(V):
    v = RNG.normal(0, 5, V)
    assert O.logsumexp(v) == pytest.approx(scipy.special.logsumexp(v), rel=1e-14, abs=1e-14)
    lt = torch.logsumexp(torch.tensor(v, dtype=torch.float64), 0).item()
    assert O.logsumexp(v) == pytest.approx(lt, rel=1e-14, abs=1e-14)


def test_logsumexp_large_offsets_and_shift():
    v = RNG.normal(0, 3, 257)
    for a in (-1e4, 700.0, 1e5):
        assert O.logsumexp(v + a) == pytest.approx(O.logsumexp(v) + a, rel=1e-13)


def test_row_lse_is_log_softmax_normaliser():
    z, u = rand_rows(513)
    r = O.row(z, u, 5)
    lp = torch.log_softmax(torch.tensor(z, dtype=torch.float64), 0).numpy()
    lq = torch.log_softmax(torch.tensor(u, dtype=torch.float64), 0).numpy()
    np.testing.assert_allclose(z - r["lse_s"], lp, rtol=0, atol=1e-13)
    np.testing.assert_allclose(u - r["lse_t"], lq, rtol=0, atol=1e-13)


# ----------------------------------------------------------------------------- KL
def test_kl_of_identical_rows_is_zero_and_shift_invariant():
    z, _ = rand_rows(777)
    assert abs(O.row(z, z.copy(), 0)["kl"]) < 1e-15
    assert abs(O.row(z, z + 3.25, 0)["kl"]) < 1e-13            # u = z + const is the same q
    z, u = rand_rows(777)
    k0 = O.row(z, u, 0)["kl"]
    assert O.row(z + 11.0, u, 0)["kl"] == pytest.approx(k0, rel=1e-12)
    assert O.row(z, u - 7.5, 0)["kl"] == pytest.approx(k0, rel=1e-12)


def test_kl_nonnegative():
    for _ in range(50):
        V = int(RNG.integers(2, 400))
        z, u = rand_rows(V, s=RNG.uniform(0.1, 6), t=RNG.uniform(0.0, 4))
        assert O.row(z, u, 0)["kl"] >= -1e-14


def test_kl_direction_two_point_example():
    # p = (0.9, 0.1), q = (0.5, 0.5):  KL(p||q) = 0.9 ln 1.8 + 0.1 ln 0.2 = 0.368064...
    # the other direction would be      KL(q||p) = 0.5 ln(5/9) + 0.5 ln 5   = 0.510826...
    z = np.log([0.9, 0.1])
    u = np.log([0.5, 0.5])
    kl = O.row(z, u, 0)["kl"]
    assert kl == pytest.approx(0.9 * math.log(1.8) + 0.1 * math.log(0.2), rel=1e-13)
    assert kl == pytest.approx(0.3680642071684971, rel=1e-12)
    assert abs(kl - 0.5108256237659907) > 0.1                   # student first (Eq. 2), not teacher


def test_kl_v2_closed_form():
    for _ in range(20):
        a, b = RNG.normal(0, 3, 2)
        p = 1 / (1 + math.exp(-a))
        q = 1 / (1 + math.exp(-b))
        want = p * math.log(p / q) + (1 - p) * math.log((1 - p) / (1 - q))
        got = O.row(np.array([a, 0.0]), np.array([b, 0.0]), 0)["kl"]
        assert got == pytest.approx(want, rel=1e-11, abs=1e-15)


def test_kl_uniform_student_closed_form():
    # p uniform:  KL = -log V - mean_k log q_k
    V = 300
    _, u = rand_rows(V)
    lq = u - scipy.special.logsumexp(u)
    want = -math.log(V) - lq.mean()
    assert O.row(np.full(V, 2.5), u, 0)["kl"] == pytest.approx(want, rel=1e-12)
    assert abs(O.row(np.zeros(V), np.full(V, -4.0), 0)["kl"]) < 1e-15     # uniform vs uniform


def test_kl_one_hot_student_limit():
    # z_j = +60, rest 0  =>  p ~ e_j  and  KL -> -log q_j
    V, j = 50, 17
    _, u = rand_rows(V)
    z = np.zeros(V)
    z[j] = 60.0
    lq = u - scipy.special.logsumexp(u)
    assert O.row(z, u, 0)["kl"] == pytest.approx(-lq[j], rel=1e-9)


def test_kl_exact_rational_enumeration_tiny_v():
    # logits = log of integers, so p and q are exact rationals; sum the definition term by term.
    for V in (2, 3, 5, 8):
        a = [int(x) for x in RNG.integers(1, 20, V)]
        b = [int(x) for x in RNG.integers(1, 20, V)]
        A, Bt = sum(a), sum(b)
        want = 0.0
        for ak, bk in zip(a, b):
            ratio = Fraction(ak, A) / Fraction(bk, Bt)
            want += float(Fraction(ak, A)) * (math.log(ratio.numerator) - math.log(ratio.denominator))
        got = O.row(np.log(np.array(a, dtype=np.float64)), np.log(np.array(b, dtype=np.float64)), 0)
        assert got["kl"] == pytest.approx(want, rel=1e-12, abs=1e-14)


def test_zero_probability_terms_contribute_zero():
    z = np.array([0.0, -np.inf, 1.0])
    u = np.array([0.3, 0.2, -0.4])
    kl = O.row(z, u, 0)["kl"]
    kl2 = O.row(z[[0, 2]], u[[0, 2]], 0)
    # dropping the impossible token changes q's normaliser only
    lq3 = u - scipy.special.logsumexp(u)
    p = np.exp(z[[0, 2]] - scipy.special.logsumexp(z[[0, 2]]))
    want = float(np.sum(p * (np.log(p) - lq3[[0, 2]])))
    assert kl == pytest.approx(want, rel=1e-13)
    assert np.isfinite(kl2["kl"])


# ----------------------------------------------------------------------------- step-wise cost c
def test_logratio_sign_and_value():
    z = np.log([0.9, 0.1])
    u = np.log([0.5, 0.5])
    assert O.row(z, u, 0)["c"] == pytest.approx(math.log(0.9) - math.log(0.5), rel=1e-13)   # > 0
    assert O.row(z, u, 1)["c"] == pytest.approx(math.log(0.1) - math.log(0.5), rel=1e-13)   # < 0


def test_expected_logratio_under_student_is_kl():
    V = 9
    z, u = rand_rows(V)
    p = np.exp(z - scipy.special.logsumexp(z))
    e = sum(p[y] * O.row(z, u, y)["c"] for y in range(V))
    assert e == pytest.approx(O.row(z, u, 0)["kl"], rel=1e-12)


def test_token_out_of_range_gives_nan_logratio():
    z, u = rand_rows(6)
    assert math.isnan(O.row(z, u, 6)["c"]) and math.isnan(O.row(z, u, -1)["c"])


# ----------------------------------------------------------------------------- gradients
def _kl_numpy(z, u):
    lp = z - scipy.special.logsumexp(z)
    lq = u - scipy.special.logsumexp(u)
    return float(np.sum(np.exp(lp) * (lp - lq)))


def test_full_kl_gradient_matches_finite_differences():
    V = 24
    z, u = rand_rows(V)
    g = O.row(z, u, 3, alpha=1.0, mode=O.MODE_FULL_KL)["g"]
    h = 1e-6
    for k in range(V):
        zp, zm = z.copy(), z.copy()
        zp[k] += h
        zm[k] -= h
        fd = (_kl_numpy(zp, u) - _kl_numpy(zm, u)) / (2 * h)
        assert g[k] == pytest.approx(fd, rel=2e-6, abs=2e-9)


def test_gradient_rows_sum_to_zero_and_vanish_at_equality():
    z, u = rand_rows(333)
    for mode in (O.MODE_FULL_KL, O.MODE_SAMPLED):
        r = O.row(z, u, 10, alpha=0.7, mode=mode)
        assert abs(r["g"].sum()) < 1e-13
    r = O.row(z, z - 2.0, 10, mode=O.MODE_FULL_KL)
    assert np.abs(r["g"]).max() < 1e-14 and r["gsq"] < 1e-27


def test_grad_scale_is_linear_and_gsq_is_the_squared_norm():
    z, u = rand_rows(100)
    for mode in (O.MODE_FULL_KL, O.MODE_SAMPLED):
        r1 = O.row(z, u, 4, alpha=1.0, mode=mode)
        r3 = O.row(z, u, 4, alpha=-3.0, mode=mode)
        np.testing.assert_allclose(r3["g"], -3.0 * r1["g"], rtol=1e-14)
        assert r3["gsq"] == pytest.approx(float(np.sum(r3["g"] ** 2)), rel=1e-13)
        assert r3["gsq"] == pytest.approx(9.0 * r1["gsq"], rel=1e-13)


def test_sampled_gradient_form_and_sign():
    # g = c (e_y - p): at the sampled token the entry is c (1 - p_y), elsewhere -c p_k  (Eq. 4)
    z, u = rand_rows(40)
    y = 7
    r = O.row(z, u, y, mode=O.MODE_SAMPLED)
    p = np.exp(z - scipy.special.logsumexp(z))
    want = -r["c"] * p
    want[y] += r["c"]
    np.testing.assert_allclose(r["g"], want, rtol=1e-12, atol=1e-16)


def test_expected_sampled_gradient_is_the_full_kl_gradient():
    # Appendix A.1: E_{y~p}[c(y) grad log p(y)] = grad KL(p||q) because E[grad log p] = 0.
    V = 11
    z, u = rand_rows(V)
    p = np.exp(z - scipy.special.logsumexp(z))
    acc = np.zeros(V)
    for y in range(V):
        acc += p[y] * O.row(z, u, y, mode=O.MODE_SAMPLED)["g"]
    full = O.row(z, u, 0, mode=O.MODE_FULL_KL)["g"]
    np.testing.assert_allclose(acc, full, rtol=1e-11, atol=1e-15)


def test_gsq_matches_expanded_single_sweep_form():
    # sum_k g_k^2 = [sum p^2 d^2 - 2 KL sum p^2 d + KL^2 sum p^2] with d = log p - log q
    z, u = rand_rows(500)
    r = O.row(z, u, 9, alpha=1.0, mode=O.MODE_FULL_KL)
    lp = z - r["lse_s"]
    d = lp - (u - r["lse_t"])
    p2 = np.exp(2 * lp)
    want = np.sum(p2 * d * d) - 2 * r["kl"] * np.sum(p2 * d) + r["kl"] ** 2 * np.sum(p2)
    assert r["gsq"] == pytest.approx(float(want), rel=1e-11)
    rs = O.row(z, u, 9, alpha=1.0, mode=O.MODE_SAMPLED)
    py = math.exp(lp[9])
    assert rs["gsq"] == pytest.approx(rs["c"] ** 2 * (1 - 2 * py + float(np.sum(p2))), rel=1e-11)


# ----------------------------------------------------------------------------- batch + window
def _small_batch(B=3, T=10, V=16, dtype=np.float32):
    z = RNG.normal(0, 2, (B, T, V)).astype(dtype)
    u = (z + RNG.normal(0, 1, (B, T, V))).astype(dtype)
    y = RNG.integers(0, V, (B, T)).astype(np.int32)
    return z, u, y


def test_batch_equals_row_by_row_inside_window_and_zero_outside():
    z, u, y = _small_batch()
    W = np.array([4, 10, 0], dtype=np.int32)
    R = np.array([10, 7, 10], dtype=np.int32)
    sentinel = np.full(z.shape, 123.0)
    out = O.opd_kl_fwd_bwd(z, u, y, W, R, grad_scale=0.5, grad_init=sentinel)
    for b in range(3):
        E = min(W[b], R[b], 10)
        for t in range(10):
            if t < E:
                r = O.row(z[b, t].astype(np.float64), u[b, t].astype(np.float64), y[b, t], 0.5)
                assert out["kl"][b, t] == r["kl"] and out["logratio"][b, t] == r["c"]
                assert out["gsq"][b, t] == r["gsq"]
                np.testing.assert_array_equal(out["grad"][b, t], r["g"])
            else:
                assert out["kl"][b, t] == 0 and out["logratio"][b, t] == 0 and out["gsq"][b, t] == 0
                assert (out["grad"][b, t] == 123.0).all()          # untouched
    out0 = O.opd_kl_fwd_bwd(z, u, y, W, R, flags=O.FLAG_ZERO_TAIL, grad_init=sentinel)
    assert (out0["grad"][2] == 0).all() and (out0["grad"][0, 4:] == 0).all()
    assert (out0["grad"][1, 7:] == 0).all() and (out0["grad"][1, :7] != 0).any()


def test_range_full_processes_rollout_but_writes_gradient_only_in_window():
    z, u, y = _small_batch()
    W = np.array([4, 10, 0], dtype=np.int32)
    R = np.array([10, 7, 6], dtype=np.int32)
    sentinel = np.full(z.shape, -5.0)
    out = O.opd_kl_fwd_bwd(z, u, y, W, R, flags=O.FLAG_RANGE_FULL, grad_init=sentinel)
    for b in range(3):
        for t in range(10):
            assert (out["kl"][b, t] != 0) == (t < R[b])
            wrote = not (out["grad"][b, t] == -5.0).all()
            assert wrote == (t < min(W[b], R[b]))


def test_bf16_bits_are_widened_exactly():
    zf = torch.randn(2, 3, 8) * 3
    uf = torch.randn(2, 3, 8) * 3
    zb, ub = zf.to(torch.bfloat16), uf.to(torch.bfloat16)
    y = np.zeros((2, 3), dtype=np.int32)
    W = np.array([3, 3], dtype=np.int32)
    a = O.opd_kl_fwd_bwd(zb.view(torch.int16).numpy().view(np.uint16),
                         ub.view(torch.int16).numpy().view(np.uint16), y, W)
    b = O.opd_kl_fwd_bwd(zb.float().numpy(), ub.float().numpy(), y, W)
    np.testing.assert_array_equal(a["kl"], b["kl"])
    np.testing.assert_array_equal(a["grad"], b["grad"])


def test_row_stride_is_respected():
    z, u, y = _small_batch(B=2, T=3, V=8)
    pad = np.full((2, 3, 12), 99.0, dtype=np.float32)
    zp, up = pad.copy(), pad.copy()
    zp[..., :8], up[..., :8] = z, u
    W = np.array([3, 2], dtype=np.int32)
    a = O.opd_kl_fwd_bwd(z, u, y, W)
    bq = O.lib()  # call through the raw entry with ld=12 and V=8
    import ctypes
    kl = np.empty((2, 3)); c = np.empty((2, 3)); gs = np.empty((2, 3))
    rc = bq.adwin_oracle_opd_kl_fwd_bwd(
        zp.ctypes.data_as(ctypes.c_void_p), up.ctypes.data_as(ctypes.c_void_p), 0,
        ctypes.c_int64(2), ctypes.c_int64(3), ctypes.c_int64(8), ctypes.c_int64(12),
        y.ctypes.data_as(ctypes.c_void_p), W.ctypes.data_as(ctypes.c_void_p), None,
        ctypes.c_double(1.0), 0, 0, None, ctypes.c_int64(8),
        kl.ctypes.data_as(ctypes.c_void_p), c.ctypes.data_as(ctypes.c_void_p),
        gs.ctypes.data_as(ctypes.c_void_p), None, None)
    assert rc == 0
    np.testing.assert_array_equal(kl, a["kl"])


def test_invalid_windows_are_rejected():
    z, u, y = _small_batch(B=2, T=3, V=4)
    with pytest.raises(ValueError):
        O.opd_kl_fwd_bwd(z, u, y, np.array([-1, 2], dtype=np.int32))
    with pytest.raises(ValueError):
        O.opd_kl_fwd_bwd(z, u, y, np.array([1, 2], dtype=np.int32), np.array([4, 2], dtype=np.int32))


def test_window_reduce_is_the_brute_force_prefix_sum():
    B, T = 4, 12
    kl = RNG.uniform(0, 2, (B, T))
    c = RNG.normal(0, 1, (B, T))
    gs = RNG.uniform(0, 1, (B, T))
    W = np.array([0, 5, 12, 20], dtype=np.int32)
    R = np.array([12, 3, 12, 9], dtype=np.int32)
    seq, batch = O.window_reduce(kl, c, gs, W, R)
    for b in range(B):
        E = min(W[b], R[b], T)
        assert seq[b, 0] == pytest.approx(kl[b, :E].sum(), rel=1e-14, abs=1e-300)
        assert seq[b, 1] == pytest.approx(c[b, :E].sum(), rel=1e-13, abs=1e-14)
        assert seq[b, 2] == pytest.approx(gs[b, :E].sum(), rel=1e-14, abs=1e-300)
        assert seq[b, 3] == E
    np.testing.assert_allclose(batch, seq.sum(0), rtol=1e-14)
    assert (seq[0] == 0).all()


def test_gsq_term_scale_bounds_the_terms_of_the_one_sweep_form():
    # the scale must dominate each of the three sums the expanded form combines, and the expanded
    # form must equal gsq; with the peak as the sample the scale stays near gsq, off the peak it
    # grows like 1/(1-p_max)^2
    V = 300
    z = RNG.normal(0, 1, V)
    z[7] += 12.0                                   # a peaked row: p_7 ~ 0.99
    u = z + RNG.normal(0, 2, V)
    for y, lo, hi in ((7, 1.0, 20.0), (11, 50.0, 1e9)):
        r = O.row(z, u, y)
        p = np.exp(z - r["lse_s"])
        d = (z - u) - (z[y] - u[y])
        c0 = float(np.sum(p * (z - u))) - (z[y] - u[y])
        B2, B1, B0 = np.sum(p * p * d * d), np.sum(p * p * d), np.sum(p * p)
        assert B2 - 2 * c0 * B1 + c0 * c0 * B0 == pytest.approx(r["gsq"], rel=1e-9)
        sc = O.row_gsq_term_scale(z, u, y)
        assert sc >= max(B2, abs(2 * c0 * B1), c0 * c0 * B0) * (1 - 1e-12)
        assert sc == pytest.approx(2 * (B2 + c0 * c0 * B0), rel=1e-12)
        assert lo <= sc / r["gsq"] <= hi
    s = O.row(z, u, 11, alpha=0.5, mode=O.MODE_SAMPLED)
    p11 = np.exp(z[11] - s["lse_s"])
    want = (0.5 * s["c"]) ** 2 * (np.sum(p * p) + p11 ** 2 + (1 - p11) ** 2)
    assert O.row_gsq_term_scale(z, u, 11, 0.5, O.MODE_SAMPLED) == pytest.approx(want, rel=1e-12)
