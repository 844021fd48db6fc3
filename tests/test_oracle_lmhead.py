"""Pins of the oracle's fused LM-head form (policies given as hidden states times an LM head).

Targets: a transposed operand in either matrix product, a swapped student/teacher head, a dropped
window mask in dH or dW, a wrong chain rule, and a weight-space cosine that silently reduces to the
logit-space one.
"""
import numpy as np
import pytest

from oracle import adwin_oracle as O

RNG = np.random.default_rng(20260528)


def make(B=2, T=6, V=11, ds=4, dt=5, scale=0.7):
    Hs = RNG.normal(0, 1, (B, T, ds))
    Ht = RNG.normal(0, 1, (B, T, dt))
    Ws = RNG.normal(0, scale, (V, ds))
    Wt = RNG.normal(0, scale, (V, dt))
    tok = RNG.integers(0, V, (B, T)).astype(np.int32)
    return Hs, Ws, Ht, Wt, tok


def windowed_loss(Hs, Ws, Ht, Wt, window, rollout):
    """sum over in-window positions of KL(softmax(h_s W_s^T) || softmax(h_t W_t^T)), from scipy."""
    import scipy.special as sp
    tot = 0.0
    for b in range(Hs.shape[0]):
        for t in range(Hs.shape[1]):
            if t < window[b] and t < rollout[b]:
                z = np.array([sum(Hs[b, t, j] * Ws[k, j] for j in range(Hs.shape[2]))
                              for k in range(Ws.shape[0])])
                u = np.array([sum(Ht[b, t, j] * Wt[k, j] for j in range(Ht.shape[2]))
                              for k in range(Wt.shape[0])])
                lp, lq = sp.log_softmax(z), sp.log_softmax(u)
                tot += float(np.sum(np.exp(lp) * (lp - lq)))
    return tot


def test_logits_are_hidden_times_head_transposed():
    Hs, Ws, _, _, _ = make(B=1, T=3, V=5, ds=4)
    z = O.lmhead_logits(Hs, Ws)
    assert z.shape == (1, 3, 5)
    for t in range(3):
        for k in range(5):
            assert z[0, t, k] == pytest.approx(sum(Hs[0, t, j] * Ws[k, j] for j in range(4)),
                                               rel=1e-14, abs=1e-15)


def test_bf16_bits_are_widened_exactly():
    bits = np.array([0x3F80, 0xBF00, 0x4049, 0x0000, 0x7F7F], dtype=np.uint16)
    np.testing.assert_array_equal(
        O.widen(bits), [1.0, -0.5, 3.140625, 0.0, 3.3895313892515355e38])


def test_equals_logit_entry_point_on_materialised_logits():
    # integer hidden states and weights: the logits are small integers, exact in float32
    B, T, V, ds, dt = 2, 7, 9, 3, 4
    Hs = RNG.integers(-2, 3, (B, T, ds)).astype(np.float32)
    Ht = RNG.integers(-2, 3, (B, T, dt)).astype(np.float32)
    Ws = RNG.integers(-1, 2, (V, ds)).astype(np.float32)
    Wt = RNG.integers(-1, 2, (V, dt)).astype(np.float32)
    tok = RNG.integers(0, V, (B, T)).astype(np.int32)
    window, rollout = np.array([4, 7], np.int32), np.array([6, 5], np.int32)
    z = np.einsum("btj,kj->btk", Hs, Ws).astype(np.float32)
    u = np.einsum("btj,kj->btk", Ht, Wt).astype(np.float32)
    for mode in (O.MODE_FULL_KL, O.MODE_SAMPLED):
        for flags in (0, O.FLAG_RANGE_FULL):
            ref = O.opd_kl_fwd_bwd(z, u, tok, window, rollout, grad_scale=0.5, grad_mode=mode,
                                   flags=flags | O.FLAG_ZERO_TAIL)
            got = O.lmhead_fwd_bwd(Hs, Ws, Ht, Wt, tok, window, rollout, grad_scale=0.5,
                                   grad_mode=mode, flags=flags)
            for name in ("kl", "logratio", "gsq", "lse_s", "lse_t"):
                np.testing.assert_allclose(got[name], ref[name], rtol=1e-13, atol=1e-14)
            G = ref["grad"]
            np.testing.assert_allclose(got["dH"], np.einsum("btk,kj->btj", G, Ws.astype(float)),
                                       rtol=1e-12, atol=1e-14)
            np.testing.assert_allclose(got["dW"], np.einsum("btk,btj->kj", G, Hs.astype(float)),
                                       rtol=1e-12, atol=1e-14)


def test_full_kl_gradients_against_central_differences():
    Hs, Ws, Ht, Wt, tok = make()
    window, rollout = np.array([3, 6], np.int32), np.array([6, 4], np.int32)
    out = O.lmhead_fwd_bwd(Hs, Ws, Ht, Wt, tok, window, rollout)
    assert out["kl"][np.arange(6)[None, :] < np.minimum(window, rollout)[:, None]].sum() == \
        pytest.approx(windowed_loss(Hs, Ws, Ht, Wt, window, rollout), rel=1e-12)
    h = 1e-6
    for (b, t, j) in [(0, 0, 0), (0, 2, 3), (1, 3, 1), (0, 4, 2), (1, 5, 0)]:
        Hp, Hm = Hs.copy(), Hs.copy()
        Hp[b, t, j] += h
        Hm[b, t, j] -= h
        fd = (windowed_loss(Hp, Ws, Ht, Wt, window, rollout) -
              windowed_loss(Hm, Ws, Ht, Wt, window, rollout)) / (2 * h)
        assert out["dH"][b, t, j] == pytest.approx(fd, rel=1e-6, abs=1e-8)
    for (k, j) in [(0, 0), (3, 2), (10, 3), (5, 1)]:
        Wp, Wm = Ws.copy(), Ws.copy()
        Wp[k, j] += h
        Wm[k, j] -= h
        fd = (windowed_loss(Hs, Wp, Ht, Wt, window, rollout) -
              windowed_loss(Hs, Wm, Ht, Wt, window, rollout)) / (2 * h)
        assert out["dW"][k, j] == pytest.approx(fd, rel=1e-6, abs=1e-8)


def test_sampled_mode_is_cost_times_score_of_the_sampled_token():
    # Eq. 4 in parameter space: sum over in-window positions of c_t * d log p(y_t) / d(H_s, W_s)
    import scipy.special as sp
    Hs, Ws, Ht, Wt, tok = make(B=1, T=4, V=6, ds=3, dt=3)
    window, rollout = np.array([3], np.int32), np.array([4], np.int32)
    out = O.lmhead_fwd_bwd(Hs, Ws, Ht, Wt, tok, window, rollout, grad_mode=O.MODE_SAMPLED)
    c = out["logratio"][0]

    def surrogate(H, W):
        return sum(c[t] * sp.log_softmax(H[0, t] @ W.T)[tok[0, t]] for t in range(3))

    h = 1e-6
    for (t, j) in [(0, 0), (1, 2), (2, 1), (3, 0)]:
        Hp, Hm = Hs.copy(), Hs.copy()
        Hp[0, t, j] += h
        Hm[0, t, j] -= h
        fd = (surrogate(Hp, Ws) - surrogate(Hm, Ws)) / (2 * h)
        assert out["dH"][0, t, j] == pytest.approx(fd, rel=1e-6, abs=1e-9)
    for (k, j) in [(0, 0), (5, 2), (int(tok[0, 1]), 1)]:
        Wp, Wm = Ws.copy(), Ws.copy()
        Wp[k, j] += h
        Wm[k, j] -= h
        fd = (surrogate(Hs, Wp) - surrogate(Hs, Wm)) / (2 * h)
        assert out["dW"][k, j] == pytest.approx(fd, rel=1e-6, abs=1e-9)


def test_positions_outside_the_window_contribute_nothing():
    Hs, Ws, Ht, Wt, tok = make(B=2, T=8)
    window, rollout = np.array([3, 8], np.int32), np.array([8, 5], np.int32)
    base = O.lmhead_fwd_bwd(Hs, Ws, Ht, Wt, tok, window, rollout, flags=O.FLAG_RANGE_FULL)
    assert (base["dH"][0, 3:] == 0).all() and (base["dH"][1, 5:] == 0).all()
    assert (base["dH"][0, :3] != 0).any()
    assert (base["kl"][0, 3:8] > 0).all()              # scalars over the whole rollout ...
    assert (base["kl"][1, 5:] == 0).all()              # ... and nothing past it
    H2, T2 = Hs.copy(), Ht.copy()
    H2[0, 3:] = RNG.normal(0, 5, H2[0, 3:].shape)      # disturb rows outside every window
    T2[1, 5:] = RNG.normal(0, 5, T2[1, 5:].shape)
    H2[1, 5:] = 1e3
    pert = O.lmhead_fwd_bwd(H2, Ws, T2, Wt, tok, window, rollout, flags=O.FLAG_RANGE_FULL)
    np.testing.assert_array_equal(pert["dW"], base["dW"])
    np.testing.assert_array_equal(pert["dH"], base["dH"])
    # all windows empty: no gradient at all
    none = O.lmhead_fwd_bwd(Hs, Ws, Ht, Wt, tok, np.zeros(2, np.int32), rollout)
    assert (none["dW"] == 0).all() and (none["dH"] == 0).all() and (none["kl"] == 0).all()


def test_gradients_scale_linearly_and_vanish_for_equal_policies():
    Hs, Ws, Ht, Wt, tok = make()
    window = np.array([6, 6], np.int32)
    a = O.lmhead_fwd_bwd(Hs, Ws, Ht, Wt, tok, window)
    b = O.lmhead_fwd_bwd(Hs, Ws, Ht, Wt, tok, window, grad_scale=-2.5)
    np.testing.assert_allclose(b["dW"], -2.5 * a["dW"], rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(b["dH"], -2.5 * a["dH"], rtol=1e-12, atol=1e-15)
    same = O.lmhead_fwd_bwd(Hs, Ws, Hs, Ws, tok, window)       # teacher == student
    assert np.abs(same["kl"]).max() < 1e-14
    assert np.abs(same["dW"]).max() < 1e-13 and np.abs(same["dH"]).max() < 1e-13


# ------------------------------------------------------------------ weight-space cosine
def logit_space_rho(Hs, Ws, Ht, Wt, tok, rollout, cands):
    B, T, _ = Hs.shape
    full = O.lmhead_fwd_bwd(Hs, Ws, Ht, Wt, tok, rollout, rollout)
    al = O.probe_align(full["kl"], full["logratio"], full["gsq"], rollout, rollout,
                       np.array(cands, np.int32), 0.5)
    return al["batch_stats"][:len(cands), 0], al["seq_stats"][:, :len(cands), 3]


def test_weight_cosine_equals_gram_form():
    # <dW^(L), dW^full> = sum_{r in prefix} sum_{r'} (g_r . g_r') (h_r . h_r')
    Hs, Ws, Ht, Wt, tok = make(B=2, T=5, V=7, ds=3, dt=3)
    rollout = np.array([5, 3], np.int32)
    cands = [1, 2, 4]
    got = O.lmhead_weight_cosine(Hs, Ws, Ht, Wt, tok, rollout, cands)
    z, u = O.lmhead_logits(Hs, Ws), O.lmhead_logits(Ht, Wt)
    rows = [(b, t) for b in range(2) for t in range(5) if t < rollout[b]]
    g = {r: O.row(z[r], u[r], int(tok[r]))["g"] for r in rows}
    for j, L in enumerate(cands):
        pre = [r for r in rows if r[1] < L]
        dot = sum(g[a] @ g[b] * (Hs[a] @ Hs[b]) for a in pre for b in rows)
        npre = sum(g[a] @ g[b] * (Hs[a] @ Hs[b]) for a in pre for b in pre)
        nfull = sum(g[a] @ g[b] * (Hs[a] @ Hs[b]) for a in rows for b in rows)
        assert got["micro"][j] == pytest.approx(dot / np.sqrt(npre * nfull), rel=1e-10)


def test_weight_cosine_with_orthonormal_hidden_states_is_the_logit_space_rho():
    # distinct orthonormal h_r make the outer products g_r h_r^T mutually orthogonal: no
    # cross-position term survives and the cosine is sqrt(Q(L)/Q_full), as in logit space
    B, T, V, dt = 2, 4, 6, 3
    ds = B * T
    Q, _ = np.linalg.qr(RNG.normal(size=(ds, ds)))
    Hs = Q.reshape(B, T, ds)
    _, Ws, Ht, Wt, tok = make(B=B, T=T, V=V, ds=ds, dt=dt)
    rollout = np.array([4, 3], np.int32)
    cands = [1, 2, 3, 4]
    got = O.lmhead_weight_cosine(Hs, Ws, Ht, Wt, tok, rollout, cands)
    micro, per_seq = logit_space_rho(Hs, Ws, Ht, Wt, tok, rollout, cands)
    np.testing.assert_allclose(got["micro"], micro, rtol=1e-10)
    np.testing.assert_allclose(got["per_seq"], per_seq, rtol=1e-10)
    np.testing.assert_allclose(got["macro"], per_seq.mean(axis=0), rtol=1e-10)


def test_weight_cosine_with_shared_hidden_state_shows_cross_sample_cancellation():
    # every position has the same hidden state h: dW = (sum_r g_r) h^T, so the cosine is the one
    # between summed logit gradients, where contributions of different positions and sequences can
    # cancel (Figure 5) -- it must differ from the logit-space rho, which has no cross terms
    B, T, V, ds, dt = 2, 4, 6, 3, 3
    _, Ws, Ht, Wt, tok = make(B=B, T=T, V=V, ds=ds, dt=dt)
    h = RNG.normal(size=ds)
    Hs = np.broadcast_to(h, (B, T, ds)).copy()
    rollout = np.array([4, 4], np.int32)
    cands = [1, 2, 4]
    got = O.lmhead_weight_cosine(Hs, Ws, Ht, Wt, tok, rollout, cands)
    z, u = O.lmhead_logits(Hs, Ws), O.lmhead_logits(Ht, Wt)
    g = np.array([[O.row(z[b, t], u[b, t], int(tok[b, t]))["g"] for t in range(T)]
                  for b in range(B)])
    for j, L in enumerate(cands):
        a, f = g[:, :L].sum(axis=(0, 1)), g.sum(axis=(0, 1))
        assert got["micro"][j] == pytest.approx(a @ f / np.sqrt((a @ a) * (f @ f)), rel=1e-10)
    micro, _ = logit_space_rho(Hs, Ws, Ht, Wt, tok, rollout, cands)
    assert np.abs(got["micro"][:2] - micro[:2]).min() > 1e-3
    assert got["micro"][2] == pytest.approx(1.0, rel=1e-12)     # L covers every rollout
    assert np.abs(got["macro"][:2] - got["micro"][:2]).min() > 1e-6   # macro != micro
